"""The projection that forms the new Gram row in its epilogue (option gram_fusion, rank-512 class shapes) against
the fp64 oracle and against the same library with the Gram tiles left in the stream kernel.

The option applies where nearly all of the work sits in matrices with at least 512 low-rank rows and a long K,
so these cases use small sets of such shapes: column counts that are not a multiple of the
256-column tile (a 32-column last tile), a 128-row matrix beside the 512-row ones, a one-slot history, a history
that wraps around its ring, and a step whose gradient carries a NaN.
"""
import numpy as np
import pytest
import torch

from paper_2410_16029_b200 import workload as wl
from tests.parity_util import TOL_UPDATE, run_side_by_side, to_device_bf16

pytestmark = pytest.mark.gpu

SHAPES = [(1536, 544), (2048, 512), (1600, 800), (1536, 128)]


def _make(w, **kw):
    from paper_2410_16029_b200.ngalore import NGaLore

    return NGaLore([(M, N) for _, M, N in w.shapes], w.r, w.s, w.T, lam=w.lam, lr=w.lr, beta1=w.beta1, beta2=w.beta2,
                   eps=w.eps, wd=w.wd, **dict(dict(gram_fusion=True), **kw))


@pytest.mark.parametrize("s,steps", [(1, 3), (5, 12), (16, 18)])
def test_against_the_oracle(s, steps):
    w = wl.tiny_workload(SHAPES, r=512, s=s, T=7, inner_rank=8, index=120 + s)
    opt = _make(w)
    errs, _, _ = run_side_by_side(opt, w, steps, "B")
    worst = max(max(row.values()) for row in errs)
    assert worst <= TOL_UPDATE, errs
    assert opt.poll_status()[0] == 0


def test_same_weights_as_with_the_gram_tiles_in_the_stream_kernel():
    """Both arrangements add fp32 products in a different order, so the updates agree to rounding, not bitwise:
    the bound is a tenth of the parity tolerance."""
    w = wl.tiny_workload(SHAPES, r=512, s=6, T=0, inner_rank=8, index=131)
    dev = torch.device("cuda")
    a, b = _make(w), _make(w, gram_fusion=False)
    G0 = [to_device_bf16(wl.gradient_bits(w, i, 0), dev) for i in range(w.n_matrices)]
    a.refresh_subspace(G0)
    torch.cuda.synchronize()
    for i in range(w.n_matrices):
        b.set_subspace(i, a.get_subspace(i))
    for k in range(9):
        G = [to_device_bf16(wl.gradient_bits(w, i, k), dev) for i in range(w.n_matrices)]
        Wa = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
        Wb = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
        a.step(Wa, G)
        b.step(Wb, G)
        torch.cuda.synchronize()
        for x, y in zip(Wa, Wb):
            err = (torch.linalg.norm(x.double() - y.double()) / torch.linalg.norm(y.double())).item()
            assert err <= 0.1 * TOL_UPDATE, (k, err)
    assert a.poll_status()[0] == 0 and b.poll_status()[0] == 0
    assert a.launch_count != b.launch_count       # the two states really took different paths


def test_nonfinite_gradient_is_reported_and_skipped():
    w = wl.tiny_workload(SHAPES[:2], r=512, s=4, T=0, inner_rank=8, index=133)
    opt = _make(w)
    dev = torch.device("cuda")
    G0 = [to_device_bf16(wl.gradient_bits(w, i, 0), dev) for i in range(2)]
    opt.refresh_subspace(G0)
    W = [torch.ones((M, N), device=dev) for _, M, N in w.shapes]
    opt.step(W, G0)
    Wgood = [t.clone() for t in W]
    bad = [G0[0].clone(), G0[1]]
    bad[0][3, 5] = float("nan")
    opt.step(W, bad)
    code, per = opt.poll_status()
    assert code == 7 and per[0] == 7 and per[1] == 0
    assert torch.equal(W[0], Wgood[0])           # matrix 0 untouched
    assert not torch.equal(W[1], Wgood[1])       # matrix 1 stepped
    opt.step(W, G0)                               # recovers: the poisoned slot was cleared
    code, per = opt.poll_status()
    assert code == 0 and all(torch.isfinite(t).all() for t in W)
    assert not torch.equal(W[0], Wgood[0])


def test_two_runs_are_identical():
    w = wl.tiny_workload(SHAPES, r=512, s=4, T=0, inner_rank=8, index=134)
    dev = torch.device("cuda")
    G = [[to_device_bf16(wl.gradient_bits(w, i, k), dev) for i in range(w.n_matrices)] for k in range(6)]
    outs = []
    for _ in range(2):
        opt = _make(w)
        opt.refresh_subspace(G[0])
        W = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
        for k in range(6):
            opt.step(W, G[k])
        torch.cuda.synchronize()
        outs.append([t.clone() for t in W])
        opt.close()
    for x, y in zip(*outs):
        assert torch.equal(x, y)
