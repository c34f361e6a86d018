"""Reduced-precision history (ngalore_options.history_bf16 = 1): every stored low-rank gradient but the
current one is bf16.  The CUDA path is compared with the oracle that rounds its history the same way, and
with the plain fp32-history oracle, whose update it must still match within the stated tolerance."""
import numpy as np
import pytest
import torch

from paper_2410_16029_b200 import workload as wl
from tests.parity_util import TOL_UPDATE, run_side_by_side, to_device_bf16

pytestmark = pytest.mark.gpu

SHAPES = [(72, 40), (40, 72), (200, 104), (136, 1000), (1000, 136), (8, 8)]


def _make(w, T=None, **kw):
    from paper_2410_16029_b200.ngalore import NGaLore

    return NGaLore([(M, N) for _, M, N in w.shapes], w.r, w.s, w.T if T is None else T, lam=w.lam, lr=w.lr,
                   beta1=w.beta1, beta2=w.beta2, eps=w.eps, wd=w.wd, history_bf16=True, **kw)


def _worst(errs):
    return max(max(row.values()) for row in errs)


@pytest.mark.parametrize("gemm_impl", [0, 1])
@pytest.mark.parametrize("r,s,T,steps", [(16, 3, 4, 10), (32, 5, 3, 13), (8, 1, 2, 5), (24, 20, 12, 24)])
def test_against_the_oracle_with_the_same_rounding(gemm_impl, r, s, T, steps):
    w = wl.tiny_workload(SHAPES, r=r, s=s, T=T, inner_rank=4, index=86)
    opt = _make(w, gemm_impl=gemm_impl)
    errs, _, _ = run_side_by_side(opt, w, steps, "B", oracle_over=dict(history_bf16=True))
    assert _worst(errs) <= TOL_UPDATE, errs
    assert opt.poll_status()[0] == 0


def test_config0_stays_within_tolerance_of_the_fp32_history_oracle():
    """Config 0 (20 steps, T = 10), and its transpose under the short-side rule: against the oracle as the
    paper states it, no rounding of the history."""
    w = wl.WORKLOADS[0]
    opt = _make(w)
    errs, _, _ = run_side_by_side(opt, w, w.steps, "B")
    assert _worst(errs) <= TOL_UPDATE, errs
    w2 = wl.tiny_workload([(1376, 512)], r=128, s=8, T=10, inner_rank=32, index=87)
    errs_short = run_side_by_side(_make(w2, projection="short_side"), w2, 12, "B", projection="short_side")[0]
    assert _worst(errs_short) <= TOL_UPDATE, errs_short


def test_nonfinite_gradient_and_checkpoint():
    """A NaN gradient is reported and skipped, the ring recovers; a checkpoint taken mid-run continues bitwise."""
    w = wl.tiny_workload([(120, 88), (88, 120)], r=16, s=3, T=4, inner_rank=4, index=88)
    dev = torch.device("cuda")
    grads = [[to_device_bf16(wl.gradient_bits(w, i, k), dev) for i in range(2)] for k in range(10)]
    bad = grads[3][1].clone()
    bad[5, 7] = float("nan")

    def run(split, poison):
        opt = _make(w)
        W = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
        codes = []
        for k in range(10):
            if k == split:
                blob = opt.export_state()
                opt.close()
                opt = _make(w)
                opt.import_state(blob)
            G = [grads[k][0], bad] if (poison and k == 3) else grads[k]
            before = W[1].clone()
            opt.step(W, G)
            torch.cuda.synchronize()
            if poison and k == 3:
                assert torch.equal(W[1], before)          # the poisoned matrix is left alone
                codes = opt.poll_status()[1]
        assert all(bool(torch.isfinite(t).all()) for t in W)
        return W, codes

    a, _ = run(-1, False)
    b, _ = run(6, False)
    assert all(torch.equal(x, y) for x, y in zip(a, b))
    _, codes = run(-1, True)
    assert codes[0] == 0 and codes[1] == 7


def test_llama_block_shapes_bf16_history():
    """One Llama-1.1B block (r 512, s 16) in the tensor-core configuration, ring filled and wrapped."""
    shapes = [(2048, 2048), (2048, 256), (2048, 5632)]
    w = wl.tiny_workload(shapes, r=512, s=4, T=200, generator="powerlaw_noise", inner_rank=64, index=89)
    opt = _make(w)
    errs, _, _ = run_side_by_side(opt, w, 6, "B", oracle_over=dict(history_bf16=True))
    assert _worst(errs) <= TOL_UPDATE, errs
    assert opt.poll_status()[0] == 0


def test_option_is_rejected_where_it_cannot_work():
    from paper_2410_16029_b200.ngalore import NGaLore, NGaLoreError

    with pytest.raises(NGaLoreError):
        NGaLore([(64, 64)], 8, 0, 0, history_bf16=True)                  # no history to narrow
    with pytest.raises(NGaLoreError):
        NGaLore([(64, 64)], 8, 4, 0, history_bf16=True, stream_impl=1)   # plain kernels read the fp32 ring
