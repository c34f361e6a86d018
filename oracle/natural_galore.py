"""fp64 CPU oracle of the Natural GaLore per-matrix optimizer update.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
optimizer computes, written from the paper's equations; the tests, the smoke
check and the benchmark's CPU-baseline leg are its only callers.  It shares no
code with the CUDA path and must never be imported by the product package.

Every quantity is float64.  One ``MatrixState`` holds the state of one weight
matrix W (M x N); ``step`` advances it by one optimizer step in the order the
paper gives:

  O0  every T steps: P <- first r' left singular vectors of G        (Sec. 1 "GaLore" paragraph; Sec. 2.2)
  O1  R = P^T G                                                        (Sec. 1, low-rank projection equation)
  O2  push R into the history of the last s low-rank gradients         (Sec. 2.4, stacked matrix G)
  O3  K_ij = <H_i, H_j> / c                                            (Sec. 2.2 empirical FIM, mean of outer products)
  O4  S = I + K / lambda,  y = U^T vec(R),  solve S z = y (Cholesky)   (Sec. 2.4)
  O5  N~ = R / lambda - (1 / lambda^2) U z                             (Sec. 2.4, last equation)
  O6  m, v, u = m / sqrt(v + eps)                                      (Sec. 2.2, Adam equations as printed)
  O7  W <- W - eta P u - eta wd W                                      (Sec. 2.2 update equation; decoupled decay as in AdamW)

with U = [vec(H_1) ... vec(H_c)] / sqrt(c) and c the number of gradients held.

Readings taken where the paper is silent or inconsistent: left projection only (the default; ``Hyper.projection =
"short_side"`` selects the GaLore convention the paper inherits when it says, at
the start of Sec. 2.4, that most steps are those of GaLore: project on the
right, R = G Q with Q the first r' right singular vectors, when M >= N);
r' = min(r, M, N); ``Hyper.history_bf16`` is the reduced-precision state the paper's
conclusion names as future work: every stored gradient but the current one is
rounded to bf16; ``Hyper.moments_bf16`` is the same idea for the Adam moments: m is stored
rounded to nearest, v with stochastic rounding from a counter-based generator (round to nearest
would freeze v, whose relative change per step, 1 - beta2, is below half a bf16 unit); the empirical Fisher is
the *mean* of outer products plus lambda I (the 1/h of the Sec. 2.2 definition
carried into Sec. 2.4); exactly s columns, the current gradient among them;
divide by the number of gradients actually held while the history fills; eps
inside the square root and no bias correction, as printed; scale factor alpha = 1;
decoupled weight decay on the pre-update W; refresh when k mod T == 0 from the
current gradient; moments and history are kept across a refresh.

Parity pins: every function below is pinned by tests/test_oracle_pins.py
(Woodbury against a dense solve, Sherman-Morrison closed forms, Eckart-Young,
the GaLore/Adam reductions, a hand-worked step).  The absolute values of the
update on the benchmark workloads are "parity unpinned" by the paper itself: it
prints no worked example of the optimizer step.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import numpy as np


# ----------------------------------------------------------------------------- small pieces

def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Values of x rounded to the nearest bf16 (ties to even), returned as float64.

    Used to hold the projection matrix in the storage format the update is defined
    on: the optimizer keeps the working copy of P in bf16, so the step (both here
    and in the CUDA path) is the paper's update with P replaced by its bf16 rounding,
    and the rounding of P is then not an error term of the comparison.  Also used by
    the bf16-history option."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


def left_singular_basis(G: np.ndarray, r: int) -> np.ndarray:
    """First r' = min(r, M, N) left singular vectors of G (compact SVD G = P Sigma Q^T, Sec. 1)."""
    G = np.asarray(G, dtype=np.float64)
    rp = min(r, G.shape[0], G.shape[1])
    U, _, _ = np.linalg.svd(G, full_matrices=False)
    return np.ascontiguousarray(U[:, :rp])


def right_singular_basis(G: np.ndarray, r: int) -> np.ndarray:
    """First r' = min(r, M, N) right singular vectors of G, as the columns of an N x r' matrix
    (compact SVD G = P Sigma Q^T, Sec. 1; used by the short-side projection rule)."""
    G = np.asarray(G, dtype=np.float64)
    rp = min(r, G.shape[0], G.shape[1])
    _, _, Vt = np.linalg.svd(G, full_matrices=False)
    return np.ascontiguousarray(Vt[:rp, :].T)


def project(P: np.ndarray, G: np.ndarray) -> np.ndarray:
    """Low-rank gradient R = P^T G (Sec. 1)."""
    return P.T @ G


def gram_matrix(history: List[np.ndarray]) -> np.ndarray:
    """K = U^T U with U = [vec(H_1) ... vec(H_c)] / sqrt(c): K_ij = <H_i, H_j>_F / c."""
    c = len(history)
    K = np.empty((c, c), dtype=np.float64)
    for i in range(c):
        for j in range(c):
            K[i, j] = float(np.sum(history[i] * history[j])) / c
    return K


def cholesky_lower(S: np.ndarray) -> np.ndarray:
    """Lower Cholesky factor L of a symmetric positive definite S (S = L L^T), written out."""
    n = S.shape[0]
    L = np.zeros((n, n), dtype=np.float64)
    for j in range(n):
        d = S[j, j] - float(np.dot(L[j, :j], L[j, :j]))
        if not (d > 0.0) or not math.isfinite(d):
            raise np.linalg.LinAlgError("matrix is not positive definite")
        L[j, j] = math.sqrt(d)
        for i in range(j + 1, n):
            L[i, j] = (S[i, j] - float(np.dot(L[i, :j], L[j, :j]))) / L[j, j]
    return L


def cholesky_solve(S: np.ndarray, y: np.ndarray) -> np.ndarray:
    """Solve S z = y through S = L L^T: forward then backward substitution (Sec. 2.4)."""
    L = cholesky_lower(S)
    n = S.shape[0]
    t = np.zeros(n, dtype=np.float64)
    for i in range(n):
        t[i] = (y[i] - float(np.dot(L[i, :i], t[:i]))) / L[i, i]
    z = np.zeros(n, dtype=np.float64)
    for i in range(n - 1, -1, -1):
        z[i] = (t[i] - float(np.dot(L[i + 1:, i], z[i + 1:]))) / L[i, i]
    return z


def natural_gradient(R: np.ndarray, history: List[np.ndarray], lam: float) -> np.ndarray:
    """N~ = F^-1 vec(R) with F = lambda I + U U^T, by the Woodbury route of Sec. 2.4.

    S = I + (1/lambda) U^T U,  y = U^T vec(R),  S z = y,
    N~ = (1/lambda) R - (1/lambda^2) U z.
    """
    c = len(history)
    rc = math.sqrt(c)
    K = gram_matrix(history)
    S = np.eye(c) + K / lam
    y = np.array([float(np.sum(H * R)) / rc for H in history], dtype=np.float64)
    z = cholesky_solve(S, y)
    Uz = np.zeros_like(R)
    for i in range(c):
        Uz += (z[i] / rc) * history[i]
    return R / lam - Uz / (lam * lam)


def adam_moments(m, v, g, beta1, beta2, eps, *, step_index=0, bias_correction=False, eps_outside=False):
    """m, v and the direction u of the Adam equations in Sec. 2.2.

    As printed: u = m / sqrt(v + eps), no bias correction.  The two switches give
    the textbook form and exist for the reduction pin only."""
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    mh, vh = m, v
    if bias_correction:
        mh = m / (1.0 - beta1 ** (step_index + 1))
        vh = v / (1.0 - beta2 ** (step_index + 1))
    u = mh / (np.sqrt(vh) + eps) if eps_outside else mh / np.sqrt(vh + eps)
    return m, v, u


# ----------------------------------------------------------------------------- reduced-precision moments

PHILOX_M0, PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
PHILOX_W0, PHILOX_W1 = 0x9E3779B9, 0xBB67AE85


def philox4x32_10(counter: np.ndarray, key0: int, key1: int) -> np.ndarray:
    """Philox-4x32 with ten rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
    2011): counter (n, 4) uint32 -> (n, 4) uint32.  One round maps (c0, c1, c2, c3) to
    (hi(M1 c2) ^ c1 ^ k0, lo(M1 c2), hi(M0 c0) ^ c3 ^ k1, lo(M0 c0)); the key is bumped by the Weyl constants
    between rounds."""
    c = np.asarray(counter, dtype=np.uint64).reshape(-1, 4).copy()
    k0, k1 = np.uint64(key0 & 0xFFFFFFFF), np.uint64(key1 & 0xFFFFFFFF)
    mask = np.uint64(0xFFFFFFFF)
    for _ in range(10):
        p0 = np.uint64(PHILOX_M0) * c[:, 0]
        p1 = np.uint64(PHILOX_M1) * c[:, 2]
        n0 = ((p1 >> np.uint64(32)) ^ c[:, 1] ^ k0) & mask
        n1 = p1 & mask
        n2 = ((p0 >> np.uint64(32)) ^ c[:, 3] ^ k1) & mask
        n3 = p0 & mask
        c = np.stack([n0, n1, n2, n3], axis=1)
        k0 = (k0 + np.uint64(PHILOX_W0)) & mask
        k1 = (k1 + np.uint64(PHILOX_W1)) & mask
    return c.astype(np.uint32)


def rounding_bits(n_elements: int, matrix_index: int, step_index: int, seed: int) -> np.ndarray:
    """Sixteen random bits per element of a flattened array for the stochastic rounding of the second moment:
    elements 4 g .. 4 g + 3 take the upper halves of the four words of Philox(counter = (g mod 2^32, g div 2^32,
    matrix index, step index), key = (seed mod 2^32, seed div 2^32))."""
    groups = (n_elements + 3) // 4
    g = np.arange(groups, dtype=np.uint64)
    ctr = np.stack([g & np.uint64(0xFFFFFFFF), g >> np.uint64(32),
                    np.full(groups, matrix_index & 0xFFFFFFFF, dtype=np.uint64),
                    np.full(groups, step_index & 0xFFFFFFFF, dtype=np.uint64)], axis=1)
    words = philox4x32_10(ctr, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    return (words >> np.uint32(16)).reshape(-1)[:n_elements].astype(np.uint32)


def stochastic_round_to_bf16(x: np.ndarray, bits16: np.ndarray) -> np.ndarray:
    """Non-negative values rounded to bf16 up or down with probabilities in proportion to the distances: the
    sixteen random bits are added below the sixteen bits that bf16 keeps of the float32 pattern, and the sum is
    truncated.  Returned as float64."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64).reshape(-1)
    u = (u + bits16.astype(np.uint64).reshape(-1)) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


# ----------------------------------------------------------------------------- the optimizer state

@dataclasses.dataclass
class Hyper:
    r: int
    s: int
    T: int
    lam: float = 1e-3
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    wd: float = 0.0
    bias_correction: bool = False
    eps_outside: bool = False
    reset_history_on_refresh: bool = False
    store_P_as_bf16: bool = True
    projection: str = "left"        # "left": always R = P^T G; "short_side": R = G Q when M >= N
    history_bf16: bool = False      # keep every low-rank gradient but the current one rounded to bf16
    moments_bf16: bool = False      # store m (round to nearest) and v (stochastic rounding) as bf16
    rounding_seed: int = 0x9E3779B97F4A7C15   # key of the generator behind the stochastic rounding


class MatrixState:
    """Optimizer state of one M x N weight matrix."""

    def __init__(self, M: int, N: int, hp: Hyper, matrix_index: int = 0):
        self.M, self.N, self.hp = M, N, hp
        self.matrix_index = matrix_index      # position in the optimizer's matrix list (keys the rounding stream)
        self.rp = min(hp.r, M, N)
        if hp.projection not in ("left", "short_side"):
            raise ValueError(hp.projection)
        # Short-side rule: the projector lives on the shorter side of the matrix; a square matrix
        # takes the right projection, as in GaLore.
        self.right = hp.projection == "short_side" and M >= N
        self.P: Optional[np.ndarray] = None      # M x r' (left) or the N x r' matrix Q (right)
        low_rank_shape = (M, self.rp) if self.right else (self.rp, N)
        self.m = np.zeros(low_rank_shape, dtype=np.float64)
        self.v = np.zeros(low_rank_shape, dtype=np.float64)
        self.slots: List[Optional[np.ndarray]] = [None] * max(hp.s, 0)
        self.head = 0
        self.count = 0
        self.k = 0
        self.last_natural_gradient: Optional[np.ndarray] = None
        self.last_direction: Optional[np.ndarray] = None

    # -- subspace -------------------------------------------------------------
    def set_subspace(self, P: np.ndarray) -> None:
        P = np.asarray(P, dtype=np.float64)
        want = (self.N if self.right else self.M, self.rp)
        assert P.shape == want, (P.shape, want)
        self.P = round_to_bf16(P) if self.hp.store_P_as_bf16 else P.copy()

    def refresh(self, G: np.ndarray) -> None:
        basis = right_singular_basis if self.right else left_singular_basis
        self.set_subspace(basis(G, self.hp.r))
        if self.hp.reset_history_on_refresh:
            self.slots = [None] * max(self.hp.s, 0)
            self.head = 0
            self.count = 0

    def history(self) -> List[np.ndarray]:
        return [self.slots[i] for i in range(self.count)]

    # -- one step ---------------------------------------------------------------
    def step(self, W: np.ndarray, G: np.ndarray, *, auto_refresh: bool = True) -> np.ndarray:
        """Advance by one step; W (float64, M x N) is updated in place; returns Delta W."""
        hp = self.hp
        G = np.asarray(G, dtype=np.float64)
        if auto_refresh and hp.T > 0 and self.k % hp.T == 0:           # O0
            self.refresh(G)
        if self.P is None:
            raise RuntimeError("no subspace: refresh first")
        R = G @ self.P if self.right else project(self.P, G)            # O1
        if hp.s > 0:
            self.slots[self.head] = R                                   # O2
            self.head = (self.head + 1) % hp.s
            self.count = min(self.count + 1, hp.s)
            Nt = natural_gradient(R, self.history(), hp.lam)            # O3-O5
        else:
            Nt = R
        if hp.s > 0 and hp.history_bf16:
            # Reduced-precision history: the gradient of this step took part exactly (the Woodbury form
            # needs it to lie in the span of the stacked matrix); from now on it is held as bf16.
            slot = (self.head - 1) % hp.s
            self.slots[slot] = round_to_bf16(self.slots[slot])
        self.m, self.v, u = adam_moments(self.m, self.v, Nt, hp.beta1, hp.beta2, hp.eps,
                                         step_index=self.k, bias_correction=hp.bias_correction,
                                         eps_outside=hp.eps_outside)    # O6
        if hp.moments_bf16:
            # Reduced-precision moments: the direction u above came from the unrounded moments of this step;
            # what the next step starts from is their bf16 storage.
            self.m = round_to_bf16(self.m)
            bits = rounding_bits(self.v.size, self.matrix_index, self.k, hp.rounding_seed)
            self.v = stochastic_round_to_bf16(self.v, bits.reshape(self.v.shape))
        back = u @ self.P.T if self.right else self.P @ u
        dW = -hp.lr * back - hp.lr * hp.wd * W                          # O7
        W += dW
        self.k += 1
        self.last_natural_gradient = Nt
        self.last_direction = u
        return dW
