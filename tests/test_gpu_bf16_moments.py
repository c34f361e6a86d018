"""Reduced-precision moments (the paper's conclusion names lower-memory optimizer state as future work; Sec. 2.2
defines the moments): m stored as bf16 rounded to nearest, v as bf16 with stochastic rounding driven by a
counter-based generator that both sides implement from its published definition.  The CUDA path is compared
with the oracle running the same option, step by step, and with the fp32-moments oracle for the size of the
deviation the option costs."""
import numpy as np
import pytest
import torch

from oracle import natural_galore as orc
from paper_2410_16029_b200 import workload as wl
from tests.parity_util import TOL_UPDATE, oracle_hyper, rel_err, to_device_bf16

pytestmark = pytest.mark.gpu

SEED = 0x1234ABCD5678EF01


def _make(w, **kw):
    from paper_2410_16029_b200.ngalore import NGaLore

    return NGaLore([(M, N) for _, M, N in w.shapes], w.r, w.s, w.T, lam=w.lam, lr=w.lr, beta1=w.beta1, beta2=w.beta2,
                   eps=w.eps, wd=w.wd, **kw)


@pytest.mark.parametrize("s,history_bf16", [(3, False), (8, False), (16, False), (20, False), (3, True), (16, True)])
def test_bf16_moments_follow_the_oracle_with_the_same_option(s, history_bf16):
    """Ragged shapes, every instantiation of the stream kernel (8, 16 and 32 slots, fp32 and bf16 history), more
    steps than slots.  The oracle rounds with the same generator, key and counters (element group, matrix, step)."""
    shapes = [(136, 264), (264, 136), (72, 1000), (200, 104), (512, 2048)]
    w = wl.tiny_workload(shapes, r=32, s=s, T=0, inner_rank=4, index=74)
    dev = torch.device("cuda")
    opt = _make(w, moments_bf16=True, history_bf16=history_bf16, seed=SEED)
    hp = oracle_hyper(w, moments_bf16=True, history_bf16=history_bf16, rounding_seed=SEED)
    hp32 = oracle_hyper(w, history_bf16=history_bf16)
    states = [orc.MatrixState(M, N, hp, matrix_index=i) for i, (M, N) in enumerate(shapes)]
    full = [orc.MatrixState(M, N, hp32) for M, N in shapes]
    W = [torch.zeros(sh, dtype=torch.float32, device=dev) for sh in shapes]
    worst, worst_cost = 0.0, 0.0
    steps = s + 6
    for k in range(steps):
        bits = [wl.gradient_bits(w, i, k) for i in range(len(shapes))]
        G = [to_device_bf16(b, dev) for b in bits]
        if k == 0:
            opt.refresh_subspace(G)
            torch.cuda.synchronize()
            for i in range(len(shapes)):
                P = opt.get_subspace(i, working=True).cpu().numpy().astype(np.float64)
                states[i].set_subspace(P)
                full[i].set_subspace(P)
        for t in W:
            t.zero_()
        opt.step(W, G)
        torch.cuda.synchronize()
        for i in range(len(shapes)):
            g64 = wl.bf16_bits_to_f64(bits[i])
            dW = states[i].step(np.zeros(shapes[i]), g64, auto_refresh=False)
            dW32 = full[i].step(np.zeros(shapes[i]), g64, auto_refresh=False)
            err = rel_err(W[i].cpu().numpy().astype(np.float64), dW)
            worst = max(worst, err)
            worst_cost = max(worst_cost, rel_err(dW, dW32))
            assert err <= TOL_UPDATE, (k, shapes[i], err)
    print(f"bf16 moments, s = {s}, bf16 history {history_bf16}: worst error against the oracle with the option {worst:.2e}; "
          f"the option itself moves the update by {worst_cost:.2e}")
    assert opt.poll_status()[0] == 0


def test_bf16_moments_halve_the_moment_memory_and_survive_a_checkpoint():
    shapes = [(136, 264), (264, 136)]
    w = wl.tiny_workload(shapes, r=16, s=3, T=0, inner_rank=4, index=75)
    dev = torch.device("cuda")
    grads = [[to_device_bf16(wl.gradient_bits(w, i, k), dev) for i in range(2)] for k in range(8)]
    a, b = _make(w), _make(w, moments_bf16=True)
    rn = sum(16 * N for _, N in shapes)
    assert a.device_bytes - b.device_bytes >= 4 * rn - 2048     # two moments, 2 bytes less each (up to alignment)

    def run(split):
        opt = _make(w, moments_bf16=True, seed=SEED)
        W = [torch.zeros(sh, device=dev) for sh in shapes]
        opt.refresh_subspace(grads[0])
        for k in range(8):
            if k == split:
                blob = opt.export_state()
                opt.close()
                opt = _make(w, moments_bf16=True, seed=SEED)
                opt.import_state(blob)
            opt.step(W, grads[k])
        torch.cuda.synchronize()
        return W

    x, y = run(-1), run(5)
    assert all(torch.equal(p, q) for p, q in zip(x, y))
    from paper_2410_16029_b200.ngalore import NGaLoreError

    with pytest.raises(NGaLoreError):
        _make(w, moments_bf16=True, projection="short_side")
    with pytest.raises(NGaLoreError):
        _make(w).import_state(_make(w, moments_bf16=True).export_state())
