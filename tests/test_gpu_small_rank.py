"""The small-rank path (an option; r' <= 8, the fine-tuning ranks 4 and 8 of Sec. 4.2 and 4.3): the step as two
kernels without tensor cores that touch every element of G and W once.  Checked against the fp64 oracle on ragged shapes, against the
tensor-core path on the same inputs, and for the failure semantics it shares with that path."""
import numpy as np
import pytest
import torch

from paper_2410_16029_b200 import workload as wl
from tests.parity_util import TOL_UPDATE, run_side_by_side, to_device_bf16

pytestmark = pytest.mark.gpu

SHAPES = [(72, 40), (40, 72), (200, 104), (24, 64), (136, 1000), (1000, 136), (8, 8), (2100, 200), (520, 328)]


def _make(w, T=None, **kw):
    from paper_2410_16029_b200.ngalore import NGaLore

    return NGaLore([(M, N) for _, M, N in w.shapes], w.r, w.s, w.T if T is None else T, lam=w.lam, lr=w.lr,
                   beta1=w.beta1, beta2=w.beta2, eps=w.eps, wd=w.wd, **kw)


@pytest.mark.parametrize("r,s,T", [(8, 3, 4), (4, 8, 3), (8, 16, 30), (8, 0, 5), (3, 5, 4), (8, 1, 2)])
def test_small_rank_path_against_the_oracle(r, s, T):
    """Strips with ragged tails (columns no multiple of 64), matrices taller than one staged chunk of P, ranks below
    8 (padded rows of P), histories that fill and wrap, s = 0 (plain GaLore)."""
    w = wl.tiny_workload(SHAPES, r=r, s=s, T=T, inner_rank=2, index=76, wd=0.05)
    W0 = [wl.initial_weight(w, i) for i in range(w.n_matrices)]
    for mode in ("A", "B"):
        opt = _make(w, T=0 if mode == "A" else None, small_rank_path=True)
        assert opt.uses_small_rank_path
        errs, _, _ = run_side_by_side(opt, w, max(9, s + 4), mode, W0=W0)
        worst = max(max(row.values()) for row in errs)
        assert worst <= TOL_UPDATE, (mode, worst)
        assert opt.poll_status()[0] == 0


def test_small_rank_path_agrees_with_the_tensor_core_path():
    w = wl.tiny_workload(SHAPES, r=8, s=4, T=0, inner_rank=2, index=77, wd=0.1)
    dev = torch.device("cuda")
    a, b = _make(w, small_rank_path=True), _make(w)
    assert a.uses_small_rank_path and not b.uses_small_rank_path
    grads = [[to_device_bf16(wl.gradient_bits(w, i, k), dev) for i in range(w.n_matrices)] for k in range(7)]
    a.refresh_subspace(grads[0])
    for i in range(w.n_matrices):
        b.set_subspace(i, a.get_subspace(i))
    Wa = [wl.initial_weight_device(w, i, dev) for i in range(w.n_matrices)]
    Wb = [t.clone() for t in Wa]
    for k in range(7):
        before = [t.clone() for t in Wa]
        a.step(Wa, grads[k])
        b.step(Wb, grads[k])
        torch.cuda.synchronize()
        for x, y, z in zip(Wa, Wb, before):
            da, db = (x - z).double(), (y - z).double()
            # the tensor-core path rounds u to fp16 and sums in another order
            assert (torch.linalg.norm(da - db) <= 5e-4 * torch.linalg.norm(db) + 1e-12).item(), k
        for x, y in zip(Wa, Wb):
            y.copy_(x)          # keep both trajectories on the same weights
    assert a.poll_status()[0] == 0 and b.poll_status()[0] == 0


def test_small_rank_path_nonfinite_gradient_checkpoint_and_graph():
    """A NaN gradient is reported, leaves that matrix's W, m and v alone and enters the history as zero; a checkpoint
    round trip is bitwise; a captured step replays."""
    shapes = [(200, 264), (264, 200), (72, 136)]
    w = wl.tiny_workload(shapes, r=8, s=3, T=0, inner_rank=2, index=78)
    dev = torch.device("cuda")
    grads = [[to_device_bf16(wl.gradient_bits(w, i, k), dev) for i in range(3)] for k in range(8)]

    def run(split=-1, poison=-1):
        opt = _make(w, small_rank_path=True)
        assert opt.uses_small_rank_path
        opt.refresh_subspace(grads[0])
        W = [wl.initial_weight_device(w, i, dev) for i in range(3)]
        for k in range(8):
            if k == split:
                blob = opt.export_state()
                opt.close()
                opt = _make(w, small_rank_path=True)
                opt.import_state(blob)
            G = grads[k]
            if k == poison:
                G = [g.clone() for g in G]
                G[1][3, 5] = float("nan")
                before = W[1].clone()
            opt.step(W, G)
            if k == poison:
                torch.cuda.synchronize()
                code, per = opt.poll_status()
                assert code == 7 and per == [0, 7, 0]
                assert torch.equal(W[1], before)
        torch.cuda.synchronize()
        assert opt.poll_status()[0] == 0
        return W

    x, y = run(), run(split=5)
    assert all(torch.equal(p, q) for p, q in zip(x, y))
    z = run(poison=4)
    assert all(bool(torch.isfinite(t).all()) for t in z)
    assert torch.equal(z[0], x[0]) and torch.equal(z[2], x[2]) and not torch.equal(z[1], x[1])
    # graph replay: two replays of a captured step equal two plain steps
    a, b = _make(w, small_rank_path=True), _make(w, small_rank_path=True)
    a.refresh_subspace(grads[0])
    for i in range(3):
        b.set_subspace(i, a.get_subspace(i))
    Wa = [wl.initial_weight_device(w, i, dev) for i in range(3)]
    Wb = [t.clone() for t in Wa]
    a.step(Wa, grads[1])
    b.step(Wb, grads[1])
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        b.step(Wb, grads[1], check=False)
    for _ in range(2):
        a.step(Wa, grads[1])
        g.replay()
    torch.cuda.synchronize()
    assert all(torch.equal(p, q) for p, q in zip(Wa, Wb))
