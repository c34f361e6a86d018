"""Pins for the fp64 oracle: what the paper's equations and plain mathematics fix.

Each test compares the oracle with something that is not the oracle: a dense
solve of the explicit Fisher system, a closed form, an invariant, an
independently written special case, or a library routine.
"""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import natural_galore as orc


def _rand_history(rng, c, rp, N, scale=1.0):
    return [scale * rng.standard_normal((rp, N)) for _ in range(c)]


# ----------------------------------------------------------------------------- P1: Woodbury vs dense

@pytest.mark.parametrize("c,rp,N,lam", [(1, 3, 5, 1e-3), (4, 4, 8, 1e-3), (8, 8, 16, 1e-3), (8, 16, 16, 0.5)])
def test_woodbury_matches_dense_fisher_solve(c, rp, N, lam):
    """Sec. 2.4: F = lambda I + U U^T with U = [vec H_i]/sqrt(c); N~ must equal F^-1 vec(R)."""
    rng = np.random.default_rng(100 + c)
    hist = _rand_history(rng, c, rp, N, scale=1.0 / math.sqrt(rp * N))
    R = hist[-1]  # the current gradient is one of the columns
    F = lam * np.eye(rp * N)
    for H in hist:
        F += np.outer(H.ravel(), H.ravel()) / c
    x = np.linalg.solve(F, R.ravel())
    Nt = orc.natural_gradient(R, hist, lam)
    assert np.linalg.norm(Nt.ravel() - x) / np.linalg.norm(x) <= 1e-9


def test_woodbury_with_gradient_not_in_history():
    """The Woodbury route does not depend on R being a column of U."""
    rng = np.random.default_rng(7)
    hist = _rand_history(rng, 5, 3, 6, scale=0.3)
    R = rng.standard_normal((3, 6))
    lam = 1e-2
    F = lam * np.eye(18) + sum(np.outer(H.ravel(), H.ravel()) for H in hist) / 5
    x = np.linalg.solve(F, R.ravel())
    Nt = orc.natural_gradient(R, hist, lam)
    assert np.linalg.norm(Nt.ravel() - x) / np.linalg.norm(x) <= 1e-9


# ----------------------------------------------------------------------------- P2: push-through closed form

@pytest.mark.parametrize("cur", [0, 3, 7])
def test_push_through_closed_form(cur):
    """vec(R) = sqrt(c) U e_cur  =>  N~ = sum_i w_i H_i with (lambda I + K) w = e_cur."""
    rng = np.random.default_rng(11 + cur)
    c, rp, N, lam = 8, 6, 10, 1e-3
    hist = _rand_history(rng, c, rp, N)
    R = hist[cur]
    K = orc.gram_matrix(hist)
    e = np.zeros(c)
    e[cur] = 1.0
    w = np.linalg.solve(lam * np.eye(c) + K, e)
    closed = sum(w[i] * hist[i] for i in range(c))
    Nt = orc.natural_gradient(R, hist, lam)
    assert np.linalg.norm(Nt - closed) / np.linalg.norm(closed) <= 1e-7


# ----------------------------------------------------------------------------- P3: rank-one cases

def test_single_slot_is_sherman_morrison():
    rng = np.random.default_rng(3)
    R = rng.standard_normal((4, 7))
    lam = 1e-3
    Nt = orc.natural_gradient(R, [R], lam)
    np.testing.assert_allclose(Nt, R / (lam + np.sum(R * R)), rtol=1e-9)


def test_identical_slots_equal_single_slot():
    rng = np.random.default_rng(4)
    R = rng.standard_normal((3, 5))
    lam = 0.05
    Nt = orc.natural_gradient(R, [R.copy() for _ in range(6)], lam)
    np.testing.assert_allclose(Nt, R / (lam + np.sum(R * R)), rtol=1e-9)


def test_orthogonal_slots_closed_form():
    """Mutually orthogonal history: N~ = R / (lambda + |R|^2 / c)."""
    c, lam = 4, 1e-2
    hist = []
    for i in range(c):
        H = np.zeros((2, 4))
        H[i // 4 if c > 4 else 0, i] = 2.0 + i
        hist.append(H)
    R = hist[2]
    Nt = orc.natural_gradient(R, hist, lam)
    np.testing.assert_allclose(Nt, R / (lam + np.sum(R * R) / c), rtol=1e-10)


def test_hand_worked_step():
    """One full step on a 2x2 matrix, worked by hand.

    P = I (r = M = 2), s = 1, lambda = 1, G = [[3, 4], [0, 0]]  =>  R = G, |R|^2 = 25,
    N~ = R / (1 + 25)                                   (Sherman-Morrison case of Sec. 2.4)
    m = (1 - b1) N~ = N~ / 2,  v = (1 - b2) N~^2 = N~^2 / 4     (b1 = 1/2, b2 = 3/4, zero start)
    u = m / sqrt(v + eps) with eps = 7/2704:
        u00 = (3/52) / sqrt(9/2704 + 7/2704) = (3/52) / (4/52) = 3/4
        u01 = (4/52) / sqrt(16/2704 + 7/2704) = 4 / sqrt(23)
        u1j = 0 / sqrt(7/2704) = 0
    W <- W - lr u - lr wd W with lr = 1/2, wd = 1/4, W = [[1, 2], [3, 4]]:
        dW00 = -3/8 - 1/8 = -1/2,  dW01 = -2/sqrt(23) - 1/4,  dW10 = -3/8,  dW11 = -1/2
    """
    hp = orc.Hyper(r=2, s=1, T=0, lam=1.0, lr=0.5, beta1=0.5, beta2=0.75, eps=float(Fraction(7, 2704)), wd=0.25)
    st = orc.MatrixState(2, 2, hp)
    st.set_subspace(np.eye(2))
    W = np.array([[1.0, 2.0], [3.0, 4.0]])
    dW = st.step(W, np.array([[3.0, 4.0], [0.0, 0.0]]))
    expect = np.array([[-0.5, -2.0 / math.sqrt(23.0) - 0.25], [-0.375, -0.5]])
    np.testing.assert_allclose(dW, expect, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(W, np.array([[1.0, 2.0], [3.0, 4.0]]) + expect, rtol=1e-12)
    np.testing.assert_allclose(st.m, np.array([[3 / 52, 4 / 52], [0, 0]]), rtol=1e-12)
    np.testing.assert_allclose(st.v, np.array([[9 / 2704, 16 / 2704], [0, 0]]), rtol=1e-12)


def test_history_fill_divides_by_count_and_ring_wraps():
    """While the history fills the mean is over the c gradients held; after s steps the oldest is dropped."""
    rng = np.random.default_rng(21)
    M, N, s, lam = 4, 6, 3, 1e-2
    hp = orc.Hyper(r=4, s=s, T=0, lam=lam)
    st = orc.MatrixState(M, N, hp)
    st.set_subspace(np.eye(M))
    grads = [rng.standard_normal((M, N)) for _ in range(5)]
    W = np.zeros((M, N))
    for k, G in enumerate(grads):
        st.step(W, G)
        held = grads[max(0, k - s + 1): k + 1]
        c = len(held)
        F = lam * np.eye(M * N) + sum(np.outer(h.ravel(), h.ravel()) for h in held) / c
        x = np.linalg.solve(F, G.ravel()).reshape(M, N)
        assert st.count == c
        np.testing.assert_allclose(st.last_natural_gradient, x, rtol=1e-8, atol=1e-12)


# ----------------------------------------------------------------------------- P4: projection identities

@pytest.mark.parametrize("M,N,r", [(24, 40, 6), (40, 24, 8), (16, 8, 32)])
def test_subspace_is_orthonormal_and_optimal(M, N, r):
    rng = np.random.default_rng(M * N)
    G = rng.standard_normal((M, 5)) @ rng.standard_normal((5, N)) + 0.05 * rng.standard_normal((M, N))
    P = orc.left_singular_basis(G, r)
    rp = min(r, M, N)
    assert P.shape == (M, rp)
    assert np.max(np.abs(P.T @ P - np.eye(rp))) <= 1e-12
    np.testing.assert_allclose(P @ (P.T @ P), P, atol=1e-12)
    # Eckart-Young: residual energy equals the tail of the spectrum, taken from an independent route.
    small = G @ G.T if M <= N else G.T @ G
    ev = np.sort(np.linalg.eigvalsh(small))[::-1]
    tail = float(np.sum(ev[rp:]))
    resid = float(np.sum((G - P @ (P.T @ G)) ** 2))
    assert abs(resid - tail) <= 1e-9 * float(np.sum(ev))
    # no other rank-r' orthonormal basis captures more energy
    Qr, _ = np.linalg.qr(rng.standard_normal((M, rp)))
    assert np.sum((Qr.T @ G) ** 2) <= np.sum((P.T @ G) ** 2) + 1e-9


def test_projection_is_transpose_product():
    """R = P^T G: a transposed operand or a swapped product would change the shape or the values."""
    P = np.array([[1.0, 0.0], [0.0, 1.0], [0.0, 0.0]])
    G = np.arange(12.0).reshape(3, 4)
    np.testing.assert_array_equal(orc.project(P, G), G[:2])


# ----------------------------------------------------------------------------- P5: reductions

def _galore_adam_reference(P, grads, lr, b1, b2, eps):
    """GaLore with the printed Adam equations, written independently of the oracle (Sec. 2.2)."""
    rp, N = P.shape[1], grads[0].shape[1]
    m = np.zeros((rp, N))
    v = np.zeros((rp, N))
    out = []
    for G in grads:
        g = np.einsum("mr,mn->rn", P, G)
        m = b1 * m + (1 - b1) * g
        v = b2 * v + (1 - b2) * g ** 2
        out.append(-lr * np.einsum("mr,rn->mn", P, m / np.sqrt(v + eps)))
    return out


def test_fisher_disabled_reduces_to_galore():
    rng = np.random.default_rng(5)
    M, N, r = 12, 9, 4
    P, _ = np.linalg.qr(rng.standard_normal((M, r)))
    hp = orc.Hyper(r=r, s=0, T=0, lr=3e-3, store_P_as_bf16=False)
    st = orc.MatrixState(M, N, hp)
    st.set_subspace(P)
    grads = [rng.standard_normal((M, N)) * 1e-3 for _ in range(4)]
    ref = _galore_adam_reference(P, grads, hp.lr, hp.beta1, hp.beta2, hp.eps)
    W = rng.standard_normal((M, N))
    for G, d in zip(grads, ref):
        np.testing.assert_allclose(st.step(W, G), d, rtol=1e-11, atol=1e-18)


def test_full_rank_identity_reduces_to_elementwise_adam():
    """r = M with P = I and no Fisher term is textbook Adam when its two switches are on."""
    rng = np.random.default_rng(6)
    M, N = 5, 7
    hp = orc.Hyper(r=M, s=0, T=0, lr=1e-2, eps=1e-8, bias_correction=True, eps_outside=True)
    st = orc.MatrixState(M, N, hp)
    st.set_subspace(np.eye(M))
    W = rng.standard_normal((M, N))
    Wref = W.copy()
    m = np.zeros((M, N))
    v = np.zeros((M, N))
    for t in range(1, 6):
        G = rng.standard_normal((M, N))
        st.step(W, G)
        for i in range(M):
            for j in range(N):
                m[i, j] = 0.9 * m[i, j] + 0.1 * G[i, j]
                v[i, j] = 0.999 * v[i, j] + 0.001 * G[i, j] ** 2
                Wref[i, j] -= 1e-2 * (m[i, j] / (1 - 0.9 ** t)) / (math.sqrt(v[i, j] / (1 - 0.999 ** t)) + 1e-8)
        np.testing.assert_allclose(W, Wref, rtol=1e-12)


@pytest.mark.parametrize("projection,s", [("left", 0), ("left", 3), ("short_side", 0), ("short_side", 3)])
def test_cyclic_shift_projector_gives_the_update_of_the_identity_projector(projection, s):
    """A square projector that is a cyclic shift (a permutation, so not symmetric) only relabels the rows of
    the low-rank gradient (the columns, on the right); Adam is elementwise and the Fisher solve sees the same
    inner products, so projecting and projecting back must give exactly the update of P = I.  A transposed
    P in either product shifts twice instead of shifting there and back."""
    rng = np.random.default_rng(61)
    n = 6
    shift = np.roll(np.eye(n), 1, axis=0)          # row i of shift^T G is row i + 1 of G
    assert not np.array_equal(shift, shift.T)
    hp = orc.Hyper(r=n, s=s, T=0, lr=1e-2, projection=projection)
    a, b = orc.MatrixState(n, n, hp), orc.MatrixState(n, n, hp)
    a.set_subspace(shift)
    b.set_subspace(np.eye(n))
    for _ in range(5):
        G = rng.standard_normal((n, n))
        da = a.step(np.zeros((n, n)), G)
        db = b.step(np.zeros((n, n)), G)
        np.testing.assert_allclose(da, db, rtol=1e-9, atol=1e-15)
    R = orc.project(shift, G)
    for i in range(n):
        np.testing.assert_array_equal(R[i], G[(i + 1) % n])


def test_stored_projector_holds_bf16_values():
    """The projector is kept in the storage format of the step's GEMM operand (bf16): every stored value has
    an 8-bit significand and lies within half a bf16 spacing of what was set."""
    rng = np.random.default_rng(62)
    P, _ = np.linalg.qr(rng.standard_normal((12, 5)))
    st = orc.MatrixState(12, 9, orc.Hyper(r=5, s=0, T=0))
    st.set_subspace(P)
    mant, _ = np.frexp(st.P)
    assert np.array_equal(mant * 256.0, np.round(mant * 256.0))      # 8 significant bits
    assert np.all(np.abs(st.P - P) <= np.abs(P) * 2.0 ** -8)      # half of the spacing 2^(e-7)
    assert np.any(st.P != P)


def test_large_lambda_limit_returns_scaled_gradient():
    rng = np.random.default_rng(8)
    hist = _rand_history(rng, 6, 4, 9)
    lam = 1e12
    Nt = orc.natural_gradient(hist[-1], hist, lam)
    np.testing.assert_allclose(lam * Nt, hist[-1], rtol=1e-6)


# ----------------------------------------------------------------------------- P6: invariants of a whole step

def _run(M, N, r, s, steps, seed, W0=None, perm=None, wd=0.0, T=3):
    rng = np.random.default_rng(seed)
    hp = orc.Hyper(r=r, s=s, T=T, wd=wd)
    st = orc.MatrixState(M, N, hp)
    W = np.zeros((M, N)) if W0 is None else W0.copy()
    out = []
    for _ in range(steps):
        G = rng.standard_normal((M, 3)) @ rng.standard_normal((3, N)) + 1e-2 * rng.standard_normal((M, N))
        if perm is not None:
            G = G[:, perm]
        out.append((st.step(W, G), st.P.copy()))
    return out, W


def test_update_lies_in_range_of_P_and_ignores_W_without_decay():
    M, N, r, s = 16, 12, 5, 4
    a, _ = _run(M, N, r, s, 7, seed=33)
    W0 = np.random.default_rng(1).standard_normal((M, N))
    b, _ = _run(M, N, r, s, 7, seed=33, W0=W0)
    for (dWa, P), (dWb, _) in zip(a, b):
        np.testing.assert_allclose(dWa, dWb, rtol=0, atol=0)
        PtP = P.T @ P
        resid = dWa - P @ np.linalg.solve(PtP, P.T @ dWa)
        assert np.linalg.norm(resid) <= 1e-12 * np.linalg.norm(dWa)


def test_column_permutation_equivariance():
    M, N, r, s = 10, 8, 4, 3
    perm = np.random.default_rng(2).permutation(N)
    a, _ = _run(M, N, r, s, 6, seed=44)
    b, _ = _run(M, N, r, s, 6, seed=44, perm=perm)
    for (dWa, Pa), (dWb, Pb) in zip(a, b):
        # the left singular subspace does not depend on the column order (signs may flip)
        np.testing.assert_allclose(np.abs(Pa.T @ Pb), np.eye(Pa.shape[1]), atol=2e-2)
    # with an injected common P the update permutes exactly
    rng = np.random.default_rng(9)
    P, _ = np.linalg.qr(rng.standard_normal((M, r)))
    res = []
    for pm in (None, perm):
        st = orc.MatrixState(M, N, orc.Hyper(r=r, s=s, T=0, store_P_as_bf16=False))
        st.set_subspace(P)
        g = np.random.default_rng(10)
        W = np.zeros((M, N))
        ds = []
        for _ in range(5):
            G = g.standard_normal((M, N))
            ds.append(st.step(W, G if pm is None else G[:, pm]))
        res.append(ds)
    for da, db in zip(*res):
        np.testing.assert_allclose(da[:, perm], db, rtol=1e-9, atol=1e-15)


def test_weight_decay_is_decoupled_and_uses_pre_update_W():
    M, N, r, s = 9, 7, 3, 2
    W0 = np.random.default_rng(12).standard_normal((M, N))
    a, _ = _run(M, N, r, s, 1, seed=55, W0=W0, wd=0.0)
    b, _ = _run(M, N, r, s, 1, seed=55, W0=W0, wd=0.1)
    np.testing.assert_allclose(b[0][0] - a[0][0], -1e-3 * 0.1 * W0, rtol=1e-12)


def test_gram_is_symmetric_psd_and_S_is_well_conditioned_from_below():
    rng = np.random.default_rng(13)
    hist = _rand_history(rng, 8, 5, 11)
    K = orc.gram_matrix(hist)
    np.testing.assert_allclose(K, K.T, rtol=1e-14)
    assert np.min(np.linalg.eigvalsh(K)) >= -1e-12
    S = np.eye(8) + K / 1e-3
    assert np.min(np.linalg.eigvalsh(S)) >= 1.0 - 1e-9
    # K_ij is the mean-normalised inner product
    assert K[2, 5] == pytest.approx(float(np.vdot(hist[2], hist[5])) / 8, rel=1e-14)


def test_refresh_schedule_and_state_kept_across_refresh():
    """Refresh at k mod T == 0 from the current gradient; m, v and the history survive it."""
    rng = np.random.default_rng(14)
    M, N, r, s, T = 8, 10, 3, 4, 3
    st = orc.MatrixState(M, N, orc.Hyper(r=r, s=s, T=T, store_P_as_bf16=False))
    W = np.zeros((M, N))
    Ps = []
    for k in range(7):
        G = rng.standard_normal((M, N))
        m_before, cnt_before = st.m.copy(), st.count
        st.step(W, G)
        Ps.append(st.P.copy())
        if k % T == 0:
            U = np.linalg.svd(G)[0][:, :r]
            np.testing.assert_allclose(np.abs(U.T @ st.P), np.eye(r), atol=1e-9)
            assert st.count == min(cnt_before + 1, s)
            assert np.linalg.norm(st.m - 0.9 * m_before) > 0  # moments continued, not reset
    assert np.array_equal(Ps[0], Ps[1]) and np.array_equal(Ps[1], Ps[2])
    assert not np.array_equal(Ps[2], Ps[3])
    assert np.array_equal(Ps[3], Ps[5]) and not np.array_equal(Ps[5], Ps[6])


# ----------------------------------------------------------------------------- P7: library cross-checks

@pytest.mark.parametrize("n", [1, 2, 8, 16])
def test_cholesky_solve_matches_library(n):
    rng = np.random.default_rng(n)
    A = rng.standard_normal((n, n + 3))
    S = A @ A.T + 0.1 * np.eye(n)
    y = rng.standard_normal(n)
    np.testing.assert_allclose(orc.cholesky_lower(S), np.linalg.cholesky(S), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(orc.cholesky_solve(S, y), np.linalg.solve(S, y), rtol=1e-9)


def test_cholesky_rejects_indefinite():
    with pytest.raises(np.linalg.LinAlgError):
        orc.cholesky_lower(np.array([[1.0, 2.0], [2.0, 1.0]]))


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -0.3, 1e-30, 65504.0])
    got = orc.round_to_bf16(x)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: even mantissa wins (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == 1.0 + 2 ** -7 and got[3] == 1.0 + 2 ** -6
    assert np.all(np.abs(got - x) <= np.abs(x) * 2 ** -8)


def test_adam_moments_as_printed():
    """eps sits inside the root and there is no bias correction (Sec. 2.2)."""
    m, v, u = orc.adam_moments(np.array([0.0]), np.array([0.0]), np.array([2.0]), 0.9, 0.999, 1e-8)
    assert m[0] == pytest.approx(0.2) and v[0] == pytest.approx(0.004)
    assert u[0] == pytest.approx(0.2 / math.sqrt(0.004 + 1e-8), rel=1e-14)


# ----------------------------------------------------------------------------- short-side projection rule

def test_right_singular_basis_recovers_planted_right_factor():
    """Eckart-Young on the right: G = A diag(sigma) B^T with orthonormal A, B has B[:, :r] as its
    leading right singular subspace."""
    rng = np.random.default_rng(41)
    M, N, r = 40, 24, 5
    A, _ = np.linalg.qr(rng.standard_normal((M, N)))
    B, _ = np.linalg.qr(rng.standard_normal((N, N)))
    sigma = np.array([10.0, 7.0, 5.0, 3.0, 2.0] + [0.1] * (N - 5))
    G = (A * sigma) @ B.T
    Q = orc.right_singular_basis(G, r)
    assert Q.shape == (N, r)
    assert np.max(np.abs(Q.T @ Q - np.eye(r))) <= 1e-12
    assert np.linalg.norm(Q @ Q.T - B[:, :r] @ B[:, :r].T, 2) <= 1e-10


@pytest.mark.parametrize("M,N", [(24, 16), (16, 16)])
def test_right_projection_is_the_left_projection_of_the_transposed_problem(M, N):
    """Projecting G on the right with Q is projecting G^T on the left with the same Q; every later
    step acts on vec() of the low-rank gradient, whose element order the mathematics ignores.  So
    the updates of a tall matrix under the short-side rule are the transposed updates of its
    transpose under the left rule."""
    rng = np.random.default_rng(43)
    hp_short = orc.Hyper(r=4, s=3, T=4, lr=1e-2, wd=0.1, projection="short_side", store_P_as_bf16=False)
    hp_left = orc.Hyper(r=4, s=3, T=4, lr=1e-2, wd=0.1, projection="left", store_P_as_bf16=False)
    a = orc.MatrixState(M, N, hp_short)
    b = orc.MatrixState(N, M, hp_left)
    assert a.right and not b.right
    Wa = rng.standard_normal((M, N))
    Wb = Wa.T.copy()
    for k in range(9):
        G = sum((0.5 ** i) * np.outer(rng.standard_normal(M), rng.standard_normal(N)) for i in range(6))
        if k % 4 == 0:
            # one basis for both: signs of singular vectors are not unique, and the moments kept across
            # a refresh make the update depend on them
            Q = orc.right_singular_basis(G, 4)
            a.set_subspace(Q)
            b.set_subspace(Q)
        da = a.step(Wa, G, auto_refresh=False)
        db = b.step(Wb, G.T.copy(), auto_refresh=False)
        assert np.linalg.norm(da - db.T) <= 1e-9 * np.linalg.norm(db), k
    assert np.linalg.norm(Wa - Wb.T) <= 1e-9 * np.linalg.norm(Wb)
    assert a.m.shape == (M, 4) and b.m.shape == (4, M)


def test_short_side_rule_picks_the_side_and_leaves_wide_matrices_alone():
    """M < N keeps the left projection (identical numbers to the default rule); M >= N projects on the right."""
    rng = np.random.default_rng(47)
    hp_short = orc.Hyper(r=3, s=2, T=3, projection="short_side")
    hp_left = orc.Hyper(r=3, s=2, T=3)
    wide_s, wide_l = orc.MatrixState(8, 16, hp_short), orc.MatrixState(8, 16, hp_left)
    assert not wide_s.right
    assert orc.MatrixState(16, 8, hp_short).right and orc.MatrixState(8, 8, hp_short).right
    Ws, Wl = np.zeros((8, 16)), np.zeros((8, 16))
    for k in range(5):
        G = rng.standard_normal((8, 16))
        assert np.array_equal(wide_s.step(Ws, G), wide_l.step(Wl, G))


def test_right_projected_update_lies_in_the_row_space_of_Q():
    """Delta W = -lr u Q^T (Sec. 2.2 update with the projector on the right): its rows are combinations of Q's columns."""
    rng = np.random.default_rng(53)
    st = orc.MatrixState(20, 12, orc.Hyper(r=3, s=2, T=100, projection="short_side", store_P_as_bf16=False))
    W = np.zeros((20, 12))
    dW = st.step(W, rng.standard_normal((20, 12)))
    Q = st.P
    assert Q.shape == (12, 3)
    assert np.linalg.norm(dW - dW @ Q @ Q.T) <= 1e-12 * np.linalg.norm(dW)
    assert np.linalg.matrix_rank(dW, tol=1e-10) <= 3


# ----------------------------------------------------------------------------- reduced-precision history

def test_bf16_history_keeps_the_current_gradient_exact_and_rounds_the_rest():
    """With history_bf16 the natural gradient of a step is F~^-1 R for F~ = lambda I + (1/c) sum of outer
    products of the stored gradients, where the current R enters exactly and the older ones as their bf16
    roundings: checked by a dense solve, step by step."""
    rng = np.random.default_rng(61)
    M, N, r, s, lam = 6, 8, 3, 3, 1e-2
    st = orc.MatrixState(M, N, orc.Hyper(r=r, s=s, T=0, lam=lam, history_bf16=True, store_P_as_bf16=False))
    P, _ = np.linalg.qr(rng.standard_normal((M, r)))
    st.set_subspace(P)
    stored = []   # what the ring must hold before each step
    for k in range(6):
        G = rng.standard_normal((M, N))
        R = P.T @ G
        held = stored[-(s - 1):] + [R]
        F = lam * np.eye(r * N)
        for H in held:
            F += np.outer(H.ravel(), H.ravel()) / len(held)
        want = np.linalg.solve(F, R.ravel()).reshape(r, N)
        st.step(np.zeros((M, N)), G, auto_refresh=False)
        assert np.linalg.norm(st.last_natural_gradient - want) <= 1e-9 * np.linalg.norm(want), k
        stored.append(orc.round_to_bf16(R))
        ring = [h for h in st.history()]
        assert all(np.array_equal(h, orc.round_to_bf16(h)) for h in ring)


# ----------------------------------------------------------------------------- reduced-precision moments

def test_philox_reproduces_the_published_known_answers():
    """The generator behind the stochastic rounding against the known-answer vectors published with it."""
    import os

    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "philox4x32_10_kat.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for row in rows:
        words = [int(x, 16) for x in row]
        got = orc.philox4x32_10(np.array([words[:4]], dtype=np.uint64), words[4], words[5])[0]
        assert [int(x) for x in got] == words[6:], row


def test_stochastic_rounding_picks_a_neighbour_with_the_right_odds():
    """A value goes to one of its two bf16 neighbours, up with probability (x - down) / (up - down); a bf16 value
    stays; the mean over many draws is the value itself."""
    x = np.float32(1.0) + np.float32(2.0 ** -7) * np.float32(0.3)           # 30 % of the way from 1 to 1 + 2^-7
    n = 200000
    bits = orc.rounding_bits(n, matrix_index=3, step_index=11, seed=12345)
    assert bits.dtype == np.uint32 and bits.max() < 65536 and bits.min() >= 0
    out = orc.stochastic_round_to_bf16(np.full(n, x, dtype=np.float64), bits)
    down, up = 1.0, 1.0 + 2.0 ** -7
    assert set(np.unique(out)) == {down, up}
    frac_up = float(np.mean(out == up))
    assert abs(frac_up - 0.3) <= 4 * np.sqrt(0.3 * 0.7 / n) + 2.0 ** -15
    assert abs(float(np.mean(out)) - float(x)) <= 5e-6
    exact = np.array([0.5, 1.0, 1.0 + 2.0 ** -7, 3.0e-5], dtype=np.float64)
    exact = orc.round_to_bf16(exact)
    assert np.array_equal(orc.stochastic_round_to_bf16(exact, np.full(4, 65535, dtype=np.uint32)), exact)
    # the bits of different steps, matrices and seeds are different streams; the same arguments give the same bits
    a = orc.rounding_bits(64, 0, 0, 1)
    assert np.array_equal(a, orc.rounding_bits(64, 0, 0, 1))
    assert not np.array_equal(a, orc.rounding_bits(64, 0, 1, 1))
    assert not np.array_equal(a, orc.rounding_bits(64, 1, 0, 1))
    assert not np.array_equal(a, orc.rounding_bits(64, 0, 0, 2))
    assert np.array_equal(orc.rounding_bits(61, 0, 0, 1), a[:61])


def test_bf16_moments_store_rounded_values_and_the_second_moment_does_not_freeze():
    """moments_bf16: the direction of a step comes from the unrounded moments, the state holds bf16 values
    (m rounded to nearest), and v keeps following (1 - beta2) g^2 although one step changes it by less than half
    a bf16 unit: its mean over many elements tracks the full-precision recursion, where rounding to nearest would
    leave it at its starting value."""
    M, N, r = 8, 4096, 8
    hp16 = orc.Hyper(r=r, s=0, T=0, lr=1.0, beta1=0.9, beta2=0.999, eps=1e-8, moments_bf16=True, store_P_as_bf16=False)
    hp32 = orc.Hyper(r=r, s=0, T=0, lr=1.0, beta1=0.9, beta2=0.999, eps=1e-8, store_P_as_bf16=False)
    a, b = orc.MatrixState(M, N, hp16, matrix_index=2), orc.MatrixState(M, N, hp32)
    for st in (a, b):
        st.set_subspace(np.eye(M))
    rng = np.random.default_rng(7)
    G0 = rng.standard_normal((M, N))
    # first step from zero moments: both see the same unrounded m, v, hence the same direction
    dWa = a.step(np.zeros((M, N)), G0, auto_refresh=False)
    dWb = b.step(np.zeros((M, N)), G0, auto_refresh=False)
    assert np.array_equal(dWa, dWb)
    assert np.array_equal(a.m, orc.round_to_bf16(b.m))
    assert np.array_equal(a.v, orc.round_to_bf16(a.v)) and not np.array_equal(a.v, orc.round_to_bf16(b.v))
    lo = np.floor(b.v / 2.0 ** np.floor(np.log2(b.v)) * 128) / 128 * 2.0 ** np.floor(np.log2(b.v))   # bf16 below
    assert np.all((a.v == lo) | (a.v == lo + 2.0 ** (np.floor(np.log2(b.v)) - 7)))
    # a long run with a gradient four times larger: v must climb towards 16 g0^2
    for k in range(300):
        a.step(np.zeros((M, N)), 4.0 * G0, auto_refresh=False)
        b.step(np.zeros((M, N)), 4.0 * G0, auto_refresh=False)
    ratio = float(np.sum(a.v) / np.sum(b.v))
    assert abs(ratio - 1.0) <= 2e-3, ratio                      # unbiased: the totals agree
    frozen = orc.round_to_bf16(1e-3 * G0 * G0)                  # what round-to-nearest would still hold
    assert float(np.sum(b.v) / np.sum(frozen)) > 3.0            # the full-precision v has moved far from it
    assert np.array_equal(a.m, orc.round_to_bf16(a.m))
