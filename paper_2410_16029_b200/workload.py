"""Seeded synthetic workloads: matrix shapes, hyper-parameters and gradient generators.

This module holds no optimizer arithmetic.  It only describes the matrix sets
(five Llama-shaped pre-training sets and three small-rank fine-tuning sets:
shapes, rank r, history length s, refresh period T)
and draws the synthetic gradients and initial weights that stand in for the
paper's C4 pre-training gradients (Sec. 4.1, Table 1 gives the model sizes and
ranks).  Both the CUDA path and the CPU oracle consume its outputs; neither
shares anything else.

Two gradient recipes:

* ``lowrank_noise``  G = A B^T / sqrt(q) + 1e-3 Z, with A (M x q), B (N x q) and
  Z (M x N) i.i.d. standard normal, redrawn every step.
* ``powerlaw_noise`` G = sum_{i=1..64} i^-1.5 a_i b_i^T + 1e-3 Z with a_i, b_i
  unit-normalised Gaussian columns, redrawn every step.

Gradients are rounded to bf16 (round-to-nearest-even) and handed out as raw
uint16 bit patterns so that every consumer sees identical values.
"""
from __future__ import annotations

import dataclasses
from typing import List, Tuple

import numpy as np

BASE_SEED = 20241016
NOISE_STD = 1e-3
POWERLAW_TERMS = 64
POWERLAW_EXPONENT = 1.5
W_INIT_STD = 0.02


@dataclasses.dataclass(frozen=True)
class Workload:
    index: int
    name: str
    r: int
    s: int
    T: int
    steps: int
    inner_rank: int
    generator: str
    shapes: Tuple[Tuple[str, int, int], ...]  # (label, rows M, cols N)
    lam: float = 1e-3
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    wd: float = 0.0

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def n_matrices(self) -> int:
        return len(self.shapes)

    def rank_of(self, i: int) -> int:
        _, M, N = self.shapes[i]
        return min(self.r, M, N)

    def distinct_shapes(self) -> List[Tuple[int, int, int]]:
        """(first matrix index, M, N) for every distinct shape, in first-seen order."""
        seen, out = set(), []
        for i, (_, M, N) in enumerate(self.shapes):
            if (M, N) not in seen:
                seen.add((M, N))
                out.append((i, M, N))
        return out


def _llama_shapes(layers: int, hidden: int, mlp: int, vocab: int, kv_dim: int | None = None):
    kv = hidden if kv_dim is None else kv_dim
    shapes = [("embed", vocab, hidden)]
    for l in range(layers):
        shapes += [
            (f"l{l}.q", hidden, hidden),
            (f"l{l}.k", hidden, kv),
            (f"l{l}.v", hidden, kv),
            (f"l{l}.o", hidden, hidden),
            (f"l{l}.gate", hidden, mlp),
            (f"l{l}.up", hidden, mlp),
            (f"l{l}.down", mlp, hidden),
        ]
    shapes.append(("lm_head", vocab, hidden))
    return tuple(shapes)


def _encoder_shapes(layers: int, hidden: int, ffn: int):
    shapes = []
    for l in range(layers):
        shapes += [
            (f"l{l}.q", hidden, hidden),
            (f"l{l}.k", hidden, hidden),
            (f"l{l}.v", hidden, hidden),
            (f"l{l}.o", hidden, hidden),
            (f"l{l}.ffn_in", hidden, ffn),
            (f"l{l}.ffn_out", ffn, hidden),
        ]
    return tuple(shapes)


WORKLOADS = {
    0: Workload(0, "single-512x1376", r=128, s=8, T=10, steps=20, inner_rank=32,
                generator="lowrank_noise", shapes=(("w", 512, 1376),)),
    1: Workload(1, "llama-60m", r=128, s=8, T=200, steps=100, inner_rank=32,
                generator="lowrank_noise", shapes=_llama_shapes(8, 512, 1376, 32000)),
    2: Workload(2, "llama-130m", r=256, s=8, T=200, steps=100, inner_rank=64,
                generator="lowrank_noise", shapes=_llama_shapes(12, 768, 2048, 32000)),
    3: Workload(3, "llama-350m", r=256, s=16, T=200, steps=100, inner_rank=64,
                generator="lowrank_noise", shapes=_llama_shapes(24, 1024, 2736, 32000)),
    4: Workload(4, "llama-1.1b", r=512, s=16, T=200, steps=100, inner_rank=POWERLAW_TERMS,
                generator="powerlaw_noise",
                shapes=_llama_shapes(22, 2048, 5632, 32000, kv_dim=256)),
    # Small-rank fine-tuning regime (Sec. 4.2: ranks 4 and 8 on RoBERTa-Base; Sec. 4.3: TinyLlama 1.1B): the
    # attention and feed-forward matrices of the encoder blocks, and the 1.1B shapes again at rank 8.  The
    # planted signal has rank 4, so that the rank-4 and rank-8 subspaces both hold all of it.
    5: Workload(5, "roberta-base-r8", r=8, s=8, T=200, steps=100, inner_rank=4,
                generator="lowrank_noise", shapes=_encoder_shapes(12, 768, 3072), lr=2e-5),
    6: Workload(6, "roberta-base-r4", r=4, s=8, T=200, steps=100, inner_rank=4,
                generator="lowrank_noise", shapes=_encoder_shapes(12, 768, 3072), lr=2e-5),
    7: Workload(7, "tinyllama-1.1b-r8", r=8, s=8, T=200, steps=100, inner_rank=4,
                generator="lowrank_noise", shapes=_llama_shapes(22, 2048, 5632, 32000, kv_dim=256), lr=7e-5),
}


def truncated(wl: "Workload", layers: int) -> "Workload":
    """The same workload with only its first `layers` transformer layers (embedding and lm_head kept):
    a small case with the full-size shapes, for profiler captures."""
    keep = tuple(sh for sh in wl.shapes if not sh[0].startswith("l") or sh[0] == "lm_head"
                 or int(sh[0][1:].split(".")[0]) < layers)
    return dataclasses.replace(wl, name=f"{wl.name}[{layers} layers]", shapes=keep)


def tiny_workload(shapes, r, s, T, generator="lowrank_noise", inner_rank=4, index=90, **kw) -> Workload:
    """A small ad-hoc workload for tests; same recipes, caller-chosen shapes."""
    shp = tuple((f"t{i}", int(M), int(N)) for i, (M, N) in enumerate(shapes))
    return Workload(index, "tiny", r=r, s=s, T=T, steps=0, inner_rank=inner_rank,
                    generator=generator, shapes=shp, **kw)


# --------------------------------------------------------------------------- bf16 bits

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bf16 (nearest-even) and return the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    out = ((u + rounding) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(bits).astype(np.float64)


# --------------------------------------------------------------------------- numpy generators

def _rng(seed: int, step: int, matrix: int) -> np.random.Generator:
    # Counter-based stream keyed by (seed, step, matrix); step -1 is the weight draw.
    key = [np.uint64(seed), np.uint64(((step + 1) << 32) | matrix)]
    return np.random.Generator(np.random.Philox(key=key))


def gradient_f32(wl: Workload, matrix: int, step: int) -> np.ndarray:
    """The un-rounded synthetic gradient (float32) of one matrix at one step."""
    _, M, N = wl.shapes[matrix]
    g = _rng(wl.seed, step, matrix)
    q = wl.inner_rank
    A = g.standard_normal((M, q), dtype=np.float32)
    B = g.standard_normal((N, q), dtype=np.float32)
    Z = g.standard_normal((M, N), dtype=np.float32)
    if wl.generator == "lowrank_noise":
        G = (A @ B.T) / np.float32(np.sqrt(q))
    elif wl.generator == "powerlaw_noise":
        A /= np.linalg.norm(A, axis=0, keepdims=True)
        B /= np.linalg.norm(B, axis=0, keepdims=True)
        sigma = (np.arange(1, q + 1, dtype=np.float32) ** np.float32(-POWERLAW_EXPONENT))
        G = (A * sigma) @ B.T
    else:
        raise ValueError(wl.generator)
    G += np.float32(NOISE_STD) * Z
    return G


def gradient_bits(wl: Workload, matrix: int, step: int) -> np.ndarray:
    """bf16 bit patterns (uint16, M x N, row-major) of one synthetic gradient."""
    return f32_to_bf16_bits(gradient_f32(wl, matrix, step))


def initial_weight(wl: Workload, matrix: int) -> np.ndarray:
    """W0 ~ N(0, 0.02^2) in float32."""
    _, M, N = wl.shapes[matrix]
    g = _rng(wl.seed, -1, matrix)
    return (np.float32(W_INIT_STD) * g.standard_normal((M, N), dtype=np.float32))


# --------------------------------------------------------------------------- torch (device) generators

def _torch_seed(seed: int, step: int, matrix: int) -> int:
    return (seed * 1000003 + (step + 1) * 10007 + matrix) % (2 ** 63 - 1)


def gradient_device(wl: Workload, matrix: int, step: int, device):
    """Same recipes drawn with torch's seeded generator on ``device``; returns a bf16 tensor.

    The values differ from the numpy stream (different generator) but follow the
    same distribution; consumers that need both sides to agree download the tensor.
    """
    import torch

    _, M, N = wl.shapes[matrix]
    gen = torch.Generator(device=device)
    gen.manual_seed(_torch_seed(wl.seed, step, matrix))
    q = wl.inner_rank
    A = torch.randn((M, q), generator=gen, device=device, dtype=torch.float32)
    B = torch.randn((N, q), generator=gen, device=device, dtype=torch.float32)
    if wl.generator == "lowrank_noise":
        G = (A @ B.T) / (q ** 0.5)
    else:
        A = A / A.norm(dim=0, keepdim=True)
        B = B / B.norm(dim=0, keepdim=True)
        sigma = torch.arange(1, q + 1, device=device, dtype=torch.float32) ** (-POWERLAW_EXPONENT)
        G = (A * sigma) @ B.T
    G.add_(torch.randn((M, N), generator=gen, device=device, dtype=torch.float32), alpha=NOISE_STD)
    return G.to(torch.bfloat16)


def initial_weight_device(wl: Workload, matrix: int, device):
    import torch

    _, M, N = wl.shapes[matrix]
    gen = torch.Generator(device=device)
    gen.manual_seed(_torch_seed(wl.seed, -1, matrix))
    return W_INIT_STD * torch.randn((M, N), generator=gen, device=device, dtype=torch.float32)


def torch_bf16_to_bits(t) -> np.ndarray:
    """Download a bf16 tensor as uint16 bit patterns."""
    import torch

    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
