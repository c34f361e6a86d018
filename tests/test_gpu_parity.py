"""GPU parity tests: the CUDA path, called through the C ABI, against the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2410_16029_b200 import workload as wl
from tests.parity_util import (TOL_PROJECTOR, TOL_UPDATE, projector_distance, rel_err, run_side_by_side,
                               to_device_bf16)

pytestmark = pytest.mark.gpu

IMPLS = [pytest.param(dict(gemm_impl=0, stream_impl=0), id="tcgen05+fused"),
         pytest.param(dict(gemm_impl=1, stream_impl=1), id="simt+plain"),
         pytest.param(dict(gemm_impl=1, stream_impl=0), id="simt+fused"),
         pytest.param(dict(gemm_impl=0, stream_impl=1), id="tcgen05+plain")]


def _make(w, T=None, **kw):
    from paper_2410_16029_b200.ngalore import NGaLore

    return NGaLore([(M, N) for _, M, N in w.shapes], w.r, w.s, w.T if T is None else T, lam=w.lam, lr=w.lr,
                   beta1=w.beta1, beta2=w.beta2, eps=w.eps, wd=w.wd, **kw)


def _assert_errs(errs, tol=TOL_UPDATE):
    worst = max(max(row.values()) for row in errs)
    assert worst <= tol, f"worst relative update error {worst:.3e} > {tol:.1e}: {errs}"


@pytest.mark.parametrize("impl", IMPLS)
def test_config0_shared_P_from_oracle(impl):
    """Config 0 (512x1376, r 128, s 8, T 10, 20 steps): oracle SVD injected at each refresh."""
    w = wl.WORKLOADS[0]
    opt = _make(w, T=0, **impl)
    errs, _, _ = run_side_by_side(opt, w, w.steps, "A")
    _assert_errs(errs)
    assert opt.poll_status()[0] == 0


@pytest.mark.parametrize("impl", IMPLS[:2])
def test_config0_gpu_refresh_end_to_end(impl):
    """Config 0 with the CUDA path refreshing its own subspace; the oracle adopts that P."""
    w = wl.WORKLOADS[0]
    opt = _make(w, **impl)
    errs, states, _ = run_side_by_side(opt, w, w.steps, "B")
    _assert_errs(errs)
    P32 = opt.get_subspace(0).cpu().numpy().astype(np.float64)
    P16 = opt.get_subspace(0, working=True).cpu().numpy().astype(np.float64)
    assert np.max(np.abs(P32.T @ P32 - np.eye(P32.shape[1]))) <= 1e-5
    assert np.max(np.abs(P16.T @ P16 - np.eye(P16.shape[1]))) <= 5e-3
    assert opt.poll_status()[0] == 0


def test_config0_refreshed_subspace_matches_svd():
    """Projector distance on the gap-separated leading directions (k = 32 here)."""
    w = wl.WORKLOADS[0]
    opt = _make(w)
    for k in (0, 10):
        bits = wl.gradient_bits(w, 0, k)
        opt.refresh_subspace([to_device_bf16(bits, torch.device("cuda"))])
        torch.cuda.synchronize()
        P = opt.get_subspace(0).cpu().numpy().astype(np.float64)
        kk, dist = projector_distance(P, wl.bf16_bits_to_f64(bits), opt.rank(0))
        assert kk == 32
        assert dist <= TOL_PROJECTOR, dist


RAGGED = [(72, 40), (40, 72), (200, 104), (24, 64), (136, 1000), (1000, 136), (8, 8)]


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("r,s,T", [(16, 3, 4), (32, 5, 3), (8, 1, 2)])
def test_ragged_shapes(impl, r, s, T):
    """Shapes that are not multiples of any tile, r' < r cases, short histories; several tiles and tails."""
    w = wl.tiny_workload(RAGGED, r=r, s=s, T=T, inner_rank=4, index=92)
    optA = _make(w, T=0, **impl)
    errs, _, _ = run_side_by_side(optA, w, 9, "A")
    _assert_errs(errs)
    optB = _make(w, **impl)
    errs, _, _ = run_side_by_side(optB, w, 9, "B")
    _assert_errs(errs)


@pytest.mark.parametrize("impl", IMPLS[:2])
def test_fisher_disabled_and_weight_decay(impl):
    w = wl.tiny_workload([(96, 160), (160, 96)], r=24, s=0, T=5, inner_rank=6, index=93, wd=0.1)
    opt = _make(w, T=0, **impl)
    W0 = [wl.initial_weight(w, i) for i in range(w.n_matrices)]
    errs, _, _ = run_side_by_side(opt, w, 7, "A", W0=W0)
    _assert_errs(errs, 2e-3)  # the update is differenced from fp32 W here, which costs a little accuracy
    w2 = wl.tiny_workload([(96, 160), (160, 96)], r=24, s=4, T=5, inner_rank=6, index=94, wd=0.1)
    opt2 = _make(w2, T=0, **impl)
    W0 = [wl.initial_weight(w2, i) for i in range(w2.n_matrices)]
    errs, _, _ = run_side_by_side(opt2, w2, 7, "A", W0=W0)
    _assert_errs(errs, 2e-3)


@pytest.mark.parametrize("impl", IMPLS[:2])
def test_nonfinite_gradient_is_reported_and_skipped(impl):
    w = wl.tiny_workload([(64, 96), (96, 64)], r=16, s=4, T=0, inner_rank=4, index=95)
    opt = _make(w, **impl)
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
    opt.step(W, G0)                                # recovers: the poisoned slot was cleared
    code, per = opt.poll_status()
    assert code == 0 and all(torch.isfinite(t).all() for t in W)
    assert not torch.equal(W[0], Wgood[0])


def test_checkpoint_roundtrip_is_bitwise():
    from paper_2410_16029_b200.ngalore import NGaLore

    w = wl.tiny_workload([(120, 88), (88, 120)], r=16, s=3, T=4, inner_rank=4, index=96)
    dev = torch.device("cuda")
    grads = [[to_device_bf16(wl.gradient_bits(w, i, k), dev) for i in range(2)] for k in range(10)]

    def run(split):
        opt = _make(w)
        W = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
        for k in range(10):
            if k == split:
                blob = opt.export_state()
                opt.close()
                opt = _make(w)
                opt.import_state(blob)
            opt.step(W, grads[k])
        torch.cuda.synchronize()
        return W

    a, b = run(-1), run(5)
    assert all(torch.equal(x, y) for x, y in zip(a, b))


def test_two_runs_are_identical():
    w = wl.tiny_workload([(256, 520), (520, 256)], r=32, s=4, T=3, inner_rank=4, index=97)
    dev = torch.device("cuda")
    outs = []
    for _ in range(2):
        opt = _make(w)
        W = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
        for k in range(6):
            opt.step(W, [to_device_bf16(wl.gradient_bits(w, i, k), dev) for i in range(2)])
        torch.cuda.synchronize()
        outs.append([t.clone() for t in W])
    for x, y in zip(*outs):
        assert rel_err(x.cpu().numpy(), y.cpu().numpy()) <= 1e-6


def test_invalid_arguments_are_rejected():
    from paper_2410_16029_b200.ngalore import NGaLore, NGaLoreError

    with pytest.raises(NGaLoreError):
        NGaLore([(64, 36)], 8, 4, 10)            # cols not a multiple of 8
    with pytest.raises(NGaLoreError):
        NGaLore([(64, 64)], 8, 33, 10)           # history too long
    with pytest.raises(NGaLoreError):
        NGaLore([(64, 64)], 8, 4, 10, lam=0.0)   # lambda must be positive with a Fisher term
    with pytest.raises(NGaLoreError):
        NGaLore([(8, 8)] * 65536, 8, 1, 0)       # more matrices than one state takes
    opt = NGaLore([(64, 64)], 8, 4, 0)
    W = [torch.zeros((64, 64), device="cuda")]
    G = [torch.zeros((64, 64), device="cuda", dtype=torch.bfloat16)]
    with pytest.raises(NGaLoreError) as e:
        opt.step(W, G)                            # T == 0 and no subspace yet
    assert e.value.code == 5
    # pointers that are not 16-byte aligned are turned away on the host, before any kernel sees them
    opt.set_subspace(0, torch.eye(64)[:, :8].contiguous())
    flat = torch.zeros(64 * 64 + 4, device="cuda")
    W_off = [flat[1:1 + 64 * 64].view(64, 64)]
    assert W_off[0].data_ptr() % 16 == 4 and W_off[0].is_contiguous()
    with pytest.raises(NGaLoreError) as e:
        opt.step(W_off, G, check=False)
    assert e.value.code == 1
    assert opt.step_count == 0                    # a rejected call leaves the state where it was
    opt.step(W, G)
    assert opt.step_count == 1 and opt.poll_status()[0] == 0


def test_many_small_matrices():
    """400 matrices in one state (more matrices than SMs, more than two per CTA of every grouped launch)."""
    shapes = [(24, 16), (16, 40), (40, 40), (8, 24)] * 100
    w = wl.tiny_workload(shapes, r=8, s=3, T=4, inner_rank=2, index=73)
    opt = _make(w)
    errs, _, _ = run_side_by_side(opt, w, 6, "B", matrices=[0, 1, 2, 3, 199, 398, 399])
    _assert_errs(errs)
    assert opt.poll_status()[0] == 0


@pytest.mark.parametrize("impl", IMPLS[:2])
def test_long_history_uses_the_32_slot_kernels(impl):
    """s = 20 exercises the 32-slot instantiation of the stream kernels; 24 steps fill and wrap the ring."""
    w = wl.tiny_workload([(200, 264), (136, 96), (64, 1032)], r=24, s=20, T=12, inner_rank=4, index=89)
    opt = _make(w, **impl)
    errs, _, _ = run_side_by_side(opt, w, 24, "B")
    _assert_errs(errs)
    assert opt.poll_status()[0] == 0


EDGE = [(1, 8), (3, 16), (16, 8), (5, 40), (129, 24), (24, 136), (1025, 8), (8, 2056), (257, 264)]


@pytest.mark.parametrize("projection", ["left", "short_side"])
@pytest.mark.parametrize("r,s", [(4, 2), (1, 1), (7, 3), (64, 4)])
def test_tiny_dimensions_and_odd_ranks(projection, r, s):
    """One-row and three-row matrices, 8-column matrices, ranks 1 and 7: r' = min(r, M, N) is then no multiple
    of 4 for some matrices, which the tensor-core refresh cannot take (it stores rows of r' floats with 16-byte
    accesses); those matrices are refreshed by the plain path inside the same call."""
    w = wl.tiny_workload(EDGE, r=r, s=s, T=3, inner_rank=2, index=70)
    opt = _make(w, projection=projection)
    errs, _, _ = run_side_by_side(opt, w, 7, "B", projection=projection)
    _assert_errs(errs)
    assert opt.poll_status()[0] == 0


@pytest.mark.parametrize("projection,history_bf16", [("left", False), ("short_side", True)])
def test_large_rank_and_longest_history(projection, history_bf16):
    """r = 768 (not a power of two, near the largest rank the library takes) with s = 32 slots."""
    w = wl.tiny_workload([(1536, 1024), (1024, 1536)], r=768, s=32, T=40, inner_rank=6, index=71)
    opt = _make(w, projection=projection, history_bf16=history_bf16)
    errs, _, _ = run_side_by_side(opt, w, 4, "B", projection=projection,
                                  oracle_over=dict(history_bf16=history_bf16))
    _assert_errs(errs)
    assert opt.poll_status()[0] == 0


def test_rank_beyond_the_limit_is_rejected():
    from paper_2410_16029_b200.ngalore import NGaLore, NGaLoreError

    with pytest.raises(NGaLoreError):
        NGaLore([(2048, 2048)], 1024, 4, 0)


@pytest.mark.parametrize("mix", [0.5, 0.1, 0.01])
def test_correlated_gradient_sequences(mix):
    """Consecutive gradients that share 50 %, 90 % and 99 % of their content, as in training: the Gram matrix
    is then far from diagonal and the s x s system ill conditioned; the update still matches the oracle and no
    solve fails."""
    w = wl.tiny_workload([(512, 1376), (1376, 512)], r=128, s=8, T=10, inner_rank=32, index=72)

    def grads(i, k):
        base = wl.gradient_f32(w, i, 0)
        fresh = wl.gradient_f32(w, i, k + 1)
        return wl.f32_to_bf16_bits(((1 - mix) * base + mix * fresh).astype(np.float32))

    opt = _make(w)
    errs, _, _ = run_side_by_side(opt, w, 14, "B", grads=grads)
    _assert_errs(errs)
    assert opt.poll_status()[0] == 0


def test_step_replays_from_a_cuda_graph():
    """A step enqueues only kernels once its pointer tables are warm (same W and G buffers, T = 0), so it can
    be captured in a CUDA graph; replays must match eager steps (ring position and counters live on the device)."""
    w = wl.tiny_workload([(256, 520), (520, 256)], r=32, s=4, T=0, inner_rank=4, index=99)
    dev = torch.device("cuda")
    shapes = [(M, N) for _, M, N in w.shapes]
    G0 = [to_device_bf16(wl.gradient_bits(w, i, 0), dev) for i in range(2)]
    eager, graphed = _make(w), _make(w)
    for opt in (eager, graphed):
        opt.refresh_subspace(G0)
    Wa = [torch.zeros(s, device=dev) for s in shapes]
    Wb = [torch.zeros(s, device=dev) for s in shapes]
    Gs = [g.clone() for g in G0]                     # static gradient buffers, refilled in place
    for k in range(2):
        for i in range(2):
            Gs[i].copy_(to_device_bf16(wl.gradient_bits(w, i, k), dev))
        eager.step(Wa, Gs)
        graphed.step(Wb, Gs)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        graphed.step(Wb, Gs)
    for k in range(2, 7):
        for i in range(2):
            Gs[i].copy_(to_device_bf16(wl.gradient_bits(w, i, k), dev))
        eager.step(Wa, Gs)
        graph.replay()
        torch.cuda.synchronize()
        for a, b in zip(Wa, Wb):
            assert rel_err(b.cpu().numpy(), a.cpu().numpy()) <= 1e-6
    assert eager.poll_status()[0] == 0 and graphed.poll_status()[0] == 0


def test_full_wrapping_ring_of_sixteen_on_the_default_path():
    """s = 16 with more steps than slots on the default path (tensor-core GEMMs, fused stream kernel, default
    options): the Gram tiles of the 16-slot instantiation of the stream kernel run with every slot held and the
    ring position wrapping, on shapes with several stream tiles and ragged tails, r = 128.  T = 30 puts the only
    refresh at step 0."""
    shapes = [(512, 768), (640, 1000), (1376, 512), (200, 264), (512, 4096)]
    w = wl.tiny_workload(shapes, r=128, s=16, T=30, inner_rank=8, index=95)
    for mode in ("B", "A"):
        opt = _make(w, T=w.T if mode == "B" else 0)
        errs, _, _ = run_side_by_side(opt, w, 22, mode)
        _assert_errs(errs)
        worst_full = max(max(row.values()) for row in errs[16:])
        print(f"16-slot ring, mode {mode}, steps 16..21 (full, wrapping): worst relative update error {worst_full:.2e}")
        assert opt.poll_status()[0] == 0
