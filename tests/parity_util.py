"""Side-by-side driver for the parity tests: the CUDA path (through the C ABI) and the fp64 oracle
run on the same seeded bf16 gradients, sharing the projection matrix P as the protocol requires
(a truncated SVD basis is unique only up to sign and rotation, and r exceeds the signal rank of the
synthetic gradients, so the update is comparable only with a common P)."""
from __future__ import annotations

import numpy as np
import torch

from oracle import natural_galore as orc
from paper_2410_16029_b200 import workload as wl

TOL_UPDATE = 1e-3      # relative Frobenius error of the per-step update (stated target)
TOL_PROJECTOR = 1e-3   # subspace distance ||P_k P_k^T - Q_k Q_k^T||_F / sqrt(k) where the gap criterion holds


def to_device_bf16(bits: np.ndarray, dev) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)


def oracle_hyper(w: wl.Workload, **over) -> orc.Hyper:
    kw = dict(r=w.r, s=w.s, T=w.T, lam=w.lam, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, wd=w.wd)
    kw.update(over)
    return orc.Hyper(**kw)


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    d = float(np.linalg.norm(ref))
    return float(np.linalg.norm(got - ref)) / d if d > 0 else float(np.linalg.norm(got))


def run_side_by_side(opt, w: wl.Workload, steps: int, mode: str, matrices=None, dev=None, wd=None,
                     grads=None, W0=None, projection="left", oracle_over=None):
    """Run `steps` optimizer steps on both sides; returns the per-step, per-matrix relative errors.

    mode "A": the oracle computes each refresh (exact SVD), its bf16-rounded P is injected into the CUDA
              state (created with T = 0).
    mode "B": the CUDA path refreshes by itself (created with T = w.T); the oracle adopts its working P.
    """
    dev = dev or torch.device("cuda", torch.cuda.current_device())
    idx = list(range(w.n_matrices)) if matrices is None else list(matrices)
    over = dict(oracle_over or {}, projection=projection)
    if wd is not None:
        over["wd"] = wd
    hp = oracle_hyper(w, **over)
    states = {i: orc.MatrixState(w.shapes[i][1], w.shapes[i][2], hp) for i in idx}
    errs = []
    Wdev = [torch.zeros((M, N), dtype=torch.float32, device=dev) for _, M, N in w.shapes]
    Wor = {i: np.zeros((states[i].M, states[i].N)) for i in idx}
    if W0 is not None:
        for i in range(w.n_matrices):
            Wdev[i].copy_(torch.from_numpy(W0[i]))
        Wor = {i: W0[i].astype(np.float64) for i in idx}
    for k in range(steps):
        bits = [grads(i, k) if grads else wl.gradient_bits(w, i, k) for i in range(w.n_matrices)]
        G = [to_device_bf16(b, dev) for b in bits]
        refresh_now = w.T > 0 and k % w.T == 0
        if mode == "A" and refresh_now:
            for i in range(w.n_matrices):
                if i in states:
                    states[i].refresh(wl.bf16_bits_to_f64(bits[i]))
                    P = states[i].P
                else:  # matrices outside the compared subset still need some subspace
                    basis = orc.right_singular_basis if opt.projects_right(i) else orc.left_singular_basis
                    P = basis(wl.bf16_bits_to_f64(bits[i]), w.r)
                opt.set_subspace(i, torch.from_numpy(P.astype(np.float32)))
        if W0 is None:
            for t in Wdev:
                t.zero_()
        before = {i: Wdev[i].cpu().numpy().astype(np.float64) for i in idx} if W0 is not None else None
        opt.step(Wdev, G)
        torch.cuda.synchronize()
        row = {}
        for i in idx:
            st = states[i]
            if mode == "B" and refresh_now:
                st.set_subspace(opt.get_subspace(i, working=True).cpu().numpy().astype(np.float64))
            if W0 is None:
                Wor[i][:] = 0.0
            dW = st.step(Wor[i], wl.bf16_bits_to_f64(bits[i]), auto_refresh=False)
            got = Wdev[i].cpu().numpy().astype(np.float64)
            if W0 is not None:
                got = got - before[i]
            row[i] = rel_err(got, dW)
        errs.append(row)
    return errs, states, Wdev


def leading_gap_rank(sv: np.ndarray, rp: int) -> int:
    """Largest k <= r' with sigma_k - sigma_{k+1} >= 1e-2 sigma_1."""
    k = 0
    for j in range(min(rp, len(sv) - 1)):
        if sv[j] - sv[j + 1] >= 1e-2 * sv[0]:
            k = j + 1
    return k


def projector_distance(P_gpu: np.ndarray, G: np.ndarray, rp: int):
    """Distance between the leading-k Ritz subspace of range(P_gpu) w.r.t. G and the true leading-k left
    singular subspace, k from the gap criterion; evaluated without forming M x M projectors."""
    U, sv, _ = np.linalg.svd(G, full_matrices=False)
    k = leading_gap_rank(sv, rp)
    if k == 0:
        return 0, 0.0
    Q, _ = np.linalg.qr(P_gpu)
    B = Q.T @ G
    Ub, _, _ = np.linalg.svd(B, full_matrices=False)
    Pk = Q @ Ub[:, :k]
    overlap = float(np.sum((Pk.T @ U[:, :k]) ** 2))
    return k, float(np.sqrt(max(2.0 * k - 2.0 * overlap, 0.0)) / np.sqrt(k))
