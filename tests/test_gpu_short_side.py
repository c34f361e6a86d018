"""Short-side projection rule (ngalore_options.projection_rule = 1): matrices with rows >= cols are
projected on the right, R = G Q, and updated with u Q^T; the CUDA path against the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2410_16029_b200 import workload as wl
from tests.parity_util import TOL_PROJECTOR, TOL_UPDATE, projector_distance, run_side_by_side

pytestmark = pytest.mark.gpu

IMPLS = [pytest.param(dict(gemm_impl=0, stream_impl=0), id="tcgen05+fused"),
         pytest.param(dict(gemm_impl=1, stream_impl=1), id="simt+plain")]

# tall, wide and square; rows that are no multiple of 8 (the transposed copy the refresh reads is padded);
# several 128-row tiles with a ragged tail; r' = cols < r; a rank that is no multiple of 8
MIXED = [(200, 104), (104, 200), (136, 136), (1000, 136), (136, 1000), (300, 8), (77, 40)]


def _make(w, T=None, **kw):
    from paper_2410_16029_b200.ngalore import NGaLore

    return NGaLore([(M, N) for _, M, N in w.shapes], w.r, w.s, w.T if T is None else T, lam=w.lam, lr=w.lr,
                   beta1=w.beta1, beta2=w.beta2, eps=w.eps, wd=w.wd, projection="short_side", **kw)


def _worst(errs):
    return max(max(row.values()) for row in errs)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("r,s,T", [(16, 3, 4), (12, 5, 3)])
def test_mixed_orientations_against_oracle(impl, r, s, T):
    w = wl.tiny_workload(MIXED, r=r, s=s, T=T, inner_rank=4, index=95)
    optA = _make(w, T=0, **impl)
    sides = [optA.projects_right(i) for i in range(w.n_matrices)]
    assert sides == [M >= N for _, M, N in w.shapes]
    assert [optA.subspace_rows(i) for i in range(w.n_matrices)] == [N if M >= N else M for _, M, N in w.shapes]
    errs, _, _ = run_side_by_side(optA, w, 9, "A", projection="short_side")
    assert _worst(errs) <= TOL_UPDATE, errs
    assert optA.poll_status()[0] == 0
    optB = _make(w, **impl)
    errs, _, _ = run_side_by_side(optB, w, 9, "B", projection="short_side")
    assert _worst(errs) <= TOL_UPDATE, errs
    assert optB.poll_status()[0] == 0


def test_refreshed_right_subspace_matches_the_right_singular_vectors():
    """A tall matrix with a planted rank-32 signal: the refreshed Q spans the leading right singular subspace."""
    M, N, q = 1376, 512, 32
    w = wl.tiny_workload([(M, N)], r=128, s=4, T=10, inner_rank=q, index=96)
    opt = _make(w)
    assert opt.projects_right(0) and opt.subspace_rows(0) == N
    dev = torch.device("cuda")
    bits = wl.gradient_bits(w, 0, 0)
    G = torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)
    opt.refresh_subspace([G])
    torch.cuda.synchronize()
    Q = opt.get_subspace(0).cpu().numpy().astype(np.float64)
    assert Q.shape == (N, 128)
    assert np.max(np.abs(Q.T @ Q - np.eye(128))) <= 1e-5
    kk, dist = projector_distance(Q, wl.bf16_bits_to_f64(bits).T, opt.rank(0))
    assert kk == q
    assert dist <= TOL_PROJECTOR, dist


def test_llama_block_shapes_short_side():
    """One Llama-1.1B block (r 512, s 16) under the short-side rule in the tensor-core configuration:
    q/o (square) and down (tall) go right, k/v and gate/up stay left."""
    shapes = [(2048, 2048), (2048, 256), (2048, 5632), (5632, 2048)]
    w = wl.tiny_workload(shapes, r=512, s=16, T=200, generator="powerlaw_noise", inner_rank=64, index=97)
    opt = _make(w)
    assert [opt.projects_right(i) for i in range(4)] == [True, True, False, True]
    errs, _, _ = run_side_by_side(opt, w, 3, "B", projection="short_side")
    assert _worst(errs) <= TOL_UPDATE, errs
    assert opt.poll_status()[0] == 0
