"""The refresh returns singular VECTORS, not just a basis of their span (Sec. 1 "GaLore" paragraph: P comes from
the compact SVD of the gradient; Sec. 2.2 runs the Adam moments element by element in the coordinates P defines).

A singular vector is determined (up to its sign) only where its singular value is separated from both neighbours,
so the per-column checks take the columns i whose gaps sigma_{i-1} - sigma_i and sigma_i - sigma_{i+1} are both at
least 1e-2 sigma_1, the separation the projector criterion uses."""
import numpy as np
import pytest
import torch

from oracle import natural_galore as orc
from paper_2410_16029_b200 import workload as wl
from tests.parity_util import TOL_UPDATE, oracle_hyper, rel_err, to_device_bf16

pytestmark = pytest.mark.gpu

TOL_COLUMN = 1e-3   # 1 - |<p_i, u_i>| for a determined column


def _make(w, T=None, **kw):
    from paper_2410_16029_b200.ngalore import NGaLore

    return NGaLore([(M, N) for _, M, N in w.shapes], w.r, w.s, w.T if T is None else T, lam=w.lam, lr=w.lr,
                   beta1=w.beta1, beta2=w.beta2, eps=w.eps, wd=w.wd, **kw)


def determined_columns(sv, rp):
    """Indices i < r' whose singular value is at least 1e-2 sigma_1 away from both neighbours."""
    out = []
    for i in range(min(rp, len(sv))):
        up = sv[i - 1] - sv[i] if i > 0 else np.inf
        down = sv[i] - sv[i + 1] if i + 1 < len(sv) else sv[i]
        if up >= 1e-2 * sv[0] and down >= 1e-2 * sv[0]:
            out.append(i)
    return out


def check_columns(P, G64, rp, label, rotated=256):
    """`rotated`: how many leading columns the refresh turns into Ritz vectors (256 unless the state asks for all);
    the per-column and ordering checks cover those."""
    U, sv, _ = np.linalg.svd(G64, full_matrices=False)
    cols = [i for i in determined_columns(sv, rp) if i < rotated]
    worst = 0.0
    for i in cols:
        worst = max(worst, 1.0 - abs(float(P[:, i] @ U[:, i])))
    assert worst <= TOL_COLUMN, (label, worst, cols[:8])
    # the columns come in falling order of their singular value, the weak ones too: ||G^T p_i|| must not rise by
    # more than rounding (this fails when the strongest directions leak into the weak columns at the 1e-4 level)
    ritz = np.linalg.norm(G64.T @ P, axis=0)[:rotated]
    assert np.all(ritz[1:] <= ritz[:-1] * (1 + 1e-3) + 1e-6 * ritz[0]), (label, ritz[-8:])
    return len(cols), worst


@pytest.mark.parametrize("impl", [pytest.param(dict(gemm_impl=0), id="tcgen05"), pytest.param(dict(gemm_impl=1), id="simt"),
                                  # fewer than four sweeps: every product takes both bf16 parts of the basis;
                                  # eight: the first four take the high part only
                                  pytest.param(dict(gemm_impl=0, power_iterations=3), id="tcgen05-3-sweeps"),
                                  pytest.param(dict(gemm_impl=0, power_iterations=8), id="tcgen05-8-sweeps")])
def test_config0_columns_are_singular_vectors(impl):
    w = wl.WORKLOADS[0]
    dev = torch.device("cuda")
    opt = _make(w, **impl)
    bits = wl.gradient_bits(w, 0, 0)
    opt.refresh_subspace([to_device_bf16(bits, dev)])
    torch.cuda.synchronize()
    P = opt.get_subspace(0).cpu().numpy().astype(np.float64)
    assert np.max(np.abs(P.T @ P - np.eye(P.shape[1]))) <= 1e-5
    n, worst = check_columns(P, wl.bf16_bits_to_f64(bits), opt.rank(0), "config 0")
    assert n >= 4
    print(f"config 0: {n} determined columns, worst 1 - |<p, u>| = {worst:.2e}")
    assert opt.poll_status()[0] == 0


def test_ragged_set_columns_and_right_projection():
    """Ranks that are no multiple of 4 (plain path), a one-block rank, a several-block rank, a right projection."""
    shapes = [(200, 264), (264, 200), (72, 1000), (520, 136), (136, 96)]
    dev = torch.device("cuda")
    # (rank, projection rule, planted signal rank): the rank exceeds the signal rank, so that the subspace iteration
    # itself (which draws exactly r' columns) converges on every planted direction
    for r, proj, q in ((24, "left", 12), (18, "left", 12), (6, "left", 4), (40, "short_side", 12)):
        w = wl.tiny_workload(shapes, r=r, s=2, T=0, generator="powerlaw_noise", inner_rank=q, index=71)
        opt = _make(w, projection=proj)
        bits = [wl.gradient_bits(w, i, 0) for i in range(w.n_matrices)]
        opt.refresh_subspace([to_device_bf16(b, dev) for b in bits])
        torch.cuda.synchronize()
        for i in range(w.n_matrices):
            P = opt.get_subspace(i).cpu().numpy().astype(np.float64)
            G64 = wl.bf16_bits_to_f64(bits[i])
            if opt.projects_right(i):
                G64 = G64.T
            assert np.max(np.abs(P.T @ P - np.eye(P.shape[1]))) <= 1e-5, (r, proj, i)
            n, worst = check_columns(P, G64, opt.rank(i), (r, proj, shapes[i]))
            assert n >= 2, (r, proj, shapes[i], n)
        assert opt.poll_status()[0] == 0


@pytest.mark.parametrize("index,shapes_checked", [(1, 4), (2, 4), (3, 4), (4, 5)])
def test_one_matrix_per_shape_of_the_full_workloads(index, shapes_checked):
    """The whole matrix set refreshes on the GPU (the grouped tensor-core path); one matrix per distinct shape is
    compared column by column with the fp64 SVD."""
    w = wl.WORKLOADS[index]
    dev = torch.device("cuda")
    opt = _make(w, T=0)
    G = [wl.gradient_device(w, i, 0, dev) for i in range(w.n_matrices)]
    opt.refresh_subspace(G)
    torch.cuda.synchronize()
    sample = w.distinct_shapes()
    assert len(sample) == shapes_checked
    for i, M, N in sample:
        if M >= 32000:
            continue                      # the fp64 SVD of the embedding alone takes most of a minute
        P = opt.get_subspace(i).cpu().numpy().astype(np.float64)
        G64 = wl.bf16_bits_to_f64(wl.torch_bf16_to_bits(G[i]))
        n, worst = check_columns(P, G64, opt.rank(i), (index, M, N))
        print(f"workload {index} {M}x{N}: {n} determined columns, worst 1 - |<p, u>| = {worst:.2e}")
    assert opt.poll_status()[0] == 0


@pytest.mark.parametrize("impl", [pytest.param(dict(gemm_impl=0, stream_impl=0), id="tcgen05+fused"),
                                  pytest.param(dict(gemm_impl=1, stream_impl=1), id="simt+plain")])
def test_update_parity_with_the_oracles_own_svd(impl):
    """No projector is handed over: the GPU refreshes by itself, the oracle takes its own exact SVD.  The planted
    spectrum (1, 0.35, 0.19, 0.125 over a noise edge of 0.036) separates all r = 4 leading values, so P is unique
    up to the signs of its columns, and a sign flip of a column leaves P u unchanged: the updates must agree."""
    shapes = [(256, 384), (384, 256)]
    w = wl.tiny_workload(shapes, r=4, s=3, T=0, generator="powerlaw_noise", inner_rank=4, index=72)
    dev = torch.device("cuda")
    opt = _make(w, **impl)
    hp = oracle_hyper(w)
    states = [orc.MatrixState(M, N, hp) for M, N in shapes]
    W = [torch.zeros(s, dtype=torch.float32, device=dev) for s in shapes]
    worst = 0.0
    for k in range(6):
        bits = [wl.gradient_bits(w, i, k) for i in range(2)]
        G = [to_device_bf16(b, dev) for b in bits]
        if k == 0:
            opt.refresh_subspace(G)
            for i, st in enumerate(states):
                st.refresh(wl.bf16_bits_to_f64(bits[i]))
        for t in W:
            t.zero_()
        opt.step(W, G)
        torch.cuda.synchronize()
        for i, st in enumerate(states):
            dW = st.step(np.zeros(shapes[i]), wl.bf16_bits_to_f64(bits[i]), auto_refresh=False)
            err = rel_err(W[i].cpu().numpy().astype(np.float64), dW)
            worst = max(worst, err)
            assert err <= TOL_UPDATE, (k, shapes[i], err)
    print(f"own-SVD parity: worst relative update error {worst:.2e}")
    assert opt.poll_status()[0] == 0


@pytest.mark.parametrize("r", [256, 328])
def test_all_columns_rotated_on_request(r):
    """ritz_columns = -1: every column of the basis is a Ritz vector, in falling order.  r = 328 has 21 blocks of
    16 columns (rounded up to 22): more block pairs per round than one pass of the eigensolver's CTAs takes, and a
    last block that is half padding."""
    shapes = [(768, 1024), (1024, 768)]
    w = wl.tiny_workload(shapes, r=r, s=2, T=0, inner_rank=16, index=73)
    dev = torch.device("cuda")
    opt = _make(w, ritz_columns=-1)
    bits = [wl.gradient_bits(w, i, 0) for i in range(2)]
    opt.refresh_subspace([to_device_bf16(b, dev) for b in bits])
    torch.cuda.synchronize()
    for i in range(2):
        P = opt.get_subspace(i).cpu().numpy().astype(np.float64)
        assert np.max(np.abs(P.T @ P - np.eye(r))) <= 1e-5
        n, worst = check_columns(P, wl.bf16_bits_to_f64(bits[i]), r, shapes[i], rotated=r)
        assert n >= 2
    assert opt.poll_status()[0] == 0
