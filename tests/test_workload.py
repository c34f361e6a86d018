"""Host-side checks of the synthetic workload descriptions and generators."""
import numpy as np
import pytest

from paper_2410_16029_b200 import workload as wl


@pytest.mark.parametrize("idx,n_mat,sum_mn", [(0, 1, 704512), (1, 58, 58.1e6), (2, 86, 134.1e6),
                                                (3, 170, 367.9e6), (4, 156, 1100.0e6), (5, 72, 84.9e6),
                                                (6, 72, 84.9e6), (7, 156, 1100.0e6)])
def test_matrix_sets(idx, n_mat, sum_mn):
    w = wl.WORKLOADS[idx]
    assert w.n_matrices == n_mat
    total = sum(M * N for _, M, N in w.shapes)
    assert total == pytest.approx(sum_mn, rel=2e-3)
    assert all(N % 8 == 0 for _, _, N in w.shapes)


def test_rank_is_clamped_to_the_short_side():
    w = wl.WORKLOADS[4]
    ranks = {(M, N): w.rank_of(i) for i, (_, M, N) in enumerate(w.shapes)}
    assert ranks[(2048, 256)] == 256 and ranks[(2048, 5632)] == 512 and ranks[(32000, 2048)] == 512


def test_bf16_bits_roundtrip_and_rounding():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -2.5, 3.0e38, 0.0], dtype=np.float32)
    bits = wl.f32_to_bf16_bits(x)
    back = wl.bf16_bits_to_f32(bits)
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == np.float32(1.0 + 2 ** -6) and back[3] == -2.5
    assert np.array_equal(wl.f32_to_bf16_bits(back), bits)


def test_gradients_are_seeded_and_redrawn_per_step():
    w = wl.WORKLOADS[0]
    a = wl.gradient_bits(w, 0, 3)
    assert a.shape == (512, 1376) and a.dtype == np.uint16
    assert np.array_equal(a, wl.gradient_bits(w, 0, 3))
    assert not np.array_equal(a, wl.gradient_bits(w, 0, 4))
    g = wl.bf16_bits_to_f64(a)
    assert abs(g.std() - 1.0) < 0.1          # unit-variance entries
    sv = np.linalg.svd(g, compute_uv=False)
    assert sv[31] / sv[32] > 100              # rank-32 signal over a 1e-3 noise floor


def test_powerlaw_recipe_spectrum():
    w = wl.tiny_workload([(256, 384)], r=32, s=4, T=10, generator="powerlaw_noise", inner_rank=64)
    g = wl.bf16_bits_to_f64(wl.gradient_bits(w, 0, 0))
    sv = np.linalg.svd(g, compute_uv=False)
    assert sv[0] == pytest.approx(1.0, rel=0.15) and sv[1] == pytest.approx(2 ** -1.5, rel=0.2)
