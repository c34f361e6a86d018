"""The entry points around the step: host-buffer stepping, learning-rate changes, single-matrix refresh,
history reset on refresh, and checkpoints under the short-side rule."""
import numpy as np
import pytest
import torch

from oracle import natural_galore as orc
from paper_2410_16029_b200 import workload as wl
from tests.parity_util import (TOL_PROJECTOR, TOL_UPDATE, oracle_hyper, projector_distance, rel_err,
                               to_device_bf16)

pytestmark = pytest.mark.gpu


def _make(w, T=None, **kw):
    from paper_2410_16029_b200.ngalore import NGaLore

    return NGaLore([(M, N) for _, M, N in w.shapes], w.r, w.s, w.T if T is None else T, lam=w.lam, lr=w.lr,
                   beta1=w.beta1, beta2=w.beta2, eps=w.eps, wd=w.wd, **kw)


def _grads(w, steps, dev):
    return [[to_device_bf16(wl.gradient_bits(w, i, k), dev) for i in range(w.n_matrices)] for k in range(steps)]


def test_step_host_equals_device_step():
    """ngalore_step_host moves W and G through its own staging and must give the bits ngalore_step gives."""
    w = wl.tiny_workload([(136, 264), (264, 136), (72, 40)], r=16, s=3, T=3, inner_rank=4, index=81, wd=0.05)
    dev = torch.device("cuda")
    grads = _grads(w, 7, dev)
    a, b = _make(w), _make(w)
    Wd = [wl.initial_weight_device(w, i, dev) for i in range(w.n_matrices)]
    Wh = [t.cpu().pin_memory() for t in Wd]
    for k in range(7):
        a.step(Wd, grads[k])
        Gh = [g.cpu().pin_memory() for g in grads[k]]
        b.step_host(Wh, Gh)
    torch.cuda.synchronize()
    for x, y in zip(Wd, Wh):
        assert torch.equal(x.cpu(), y)
    assert a.poll_status()[0] == 0 and b.poll_status()[0] == 0


def test_set_lr_scales_the_next_update_exactly():
    """W <- W - lr P u with W = 0 and wd = 0: doubling lr doubles every element (a power of two is exact in fp32),
    and the oracle with the new rate agrees."""
    w = wl.tiny_workload([(96, 160)], r=16, s=2, T=100, inner_rank=4, index=82)
    dev = torch.device("cuda")
    grads = _grads(w, 3, dev)
    a, b = _make(w), _make(w)
    Wa = [torch.zeros((96, 160), device=dev)]
    Wb = [torch.zeros((96, 160), device=dev)]
    for k in range(2):
        a.step(Wa, grads[k])
        b.step(Wb, grads[k])
    b.set_lr(2.0 * w.lr)
    Wa[0].zero_()
    Wb[0].zero_()
    a.step(Wa, grads[2])
    b.step(Wb, grads[2])
    torch.cuda.synchronize()
    assert torch.equal(Wb[0], 2.0 * Wa[0])
    st = orc.MatrixState(96, 160, oracle_hyper(w))
    st.set_subspace(a.get_subspace(0, working=True).cpu().numpy().astype(np.float64))
    Wo = np.zeros((96, 160))
    for k in range(2):
        st.step(Wo, wl.bf16_bits_to_f64(wl.gradient_bits(w, 0, k)), auto_refresh=False)
    st.hp.lr = 2.0 * w.lr
    dW = st.step(np.zeros((96, 160)), wl.bf16_bits_to_f64(wl.gradient_bits(w, 0, 2)), auto_refresh=False)
    assert rel_err(Wb[0].cpu().numpy().astype(np.float64), dW) <= TOL_UPDATE


@pytest.mark.parametrize("impl", [dict(gemm_impl=0), dict(gemm_impl=1)])
def test_single_matrix_refresh_touches_only_that_matrix(impl):
    w = wl.tiny_workload([(512, 264), (264, 512)], r=32, s=2, T=0, inner_rank=8, index=83)
    dev = torch.device("cuda")
    opt = _make(w, **impl)
    G0 = _grads(w, 1, dev)[0]
    opt.refresh_subspace(G0)
    torch.cuda.synchronize()
    P0 = opt.get_subspace(0).clone()
    P1 = opt.get_subspace(1).clone()
    bits = wl.gradient_bits(w, 1, 5)
    G1 = [G0[0], to_device_bf16(bits, dev)]
    opt.refresh_subspace(G1, matrix_index=1)
    torch.cuda.synchronize()
    assert torch.equal(opt.get_subspace(0), P0)
    Q = opt.get_subspace(1)
    assert not torch.equal(Q, P1)
    Qn = Q.cpu().numpy().astype(np.float64)
    assert np.max(np.abs(Qn.T @ Qn - np.eye(32))) <= 1e-5
    kk, dist = projector_distance(Qn, wl.bf16_bits_to_f64(bits), opt.rank(1))
    assert kk == 8 and dist <= TOL_PROJECTOR, (kk, dist)


def test_reset_history_on_refresh_matches_the_oracle_option():
    w = wl.tiny_workload([(136, 200), (200, 136)], r=16, s=4, T=3, inner_rank=4, index=84)
    dev = torch.device("cuda")
    opt = _make(w, reset_history_on_refresh=True)
    hp = oracle_hyper(w, reset_history_on_refresh=True)
    states = [orc.MatrixState(M, N, hp) for _, M, N in w.shapes]
    W = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
    for k in range(8):
        bits = [wl.gradient_bits(w, i, k) for i in range(2)]
        for t in W:
            t.zero_()
        opt.step(W, [to_device_bf16(b, dev) for b in bits])
        torch.cuda.synchronize()
        for i, st in enumerate(states):
            if k % w.T == 0:
                st.set_subspace(opt.get_subspace(i, working=True).cpu().numpy().astype(np.float64))
                st.slots, st.head, st.count = [None] * w.s, 0, 0
            dW = st.step(np.zeros(W[i].shape), wl.bf16_bits_to_f64(bits[i]), auto_refresh=False)
            assert rel_err(W[i].cpu().numpy().astype(np.float64), dW) <= TOL_UPDATE, (k, i)
    assert opt.poll_status()[0] == 0


def test_checkpoint_roundtrip_under_the_short_side_rule():
    w = wl.tiny_workload([(200, 104), (104, 200)], r=16, s=3, T=4, inner_rank=4, index=85)
    dev = torch.device("cuda")
    grads = _grads(w, 9, dev)

    def run(split):
        opt = _make(w, projection="short_side")
        W = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
        for k in range(9):
            if k == split:
                blob = opt.export_state()
                opt.close()
                opt = _make(w, projection="short_side")
                opt.import_state(blob)
            opt.step(W, grads[k])
        torch.cuda.synchronize()
        return W

    a, b = run(-1), run(5)
    assert all(torch.equal(x, y) for x, y in zip(a, b))
    left = _make(w)
    with pytest.raises(Exception):
        left.import_state(_make(w, projection="short_side").export_state())


def test_steps_on_a_side_stream_match_the_default_stream():
    """The stream argument: the same run enqueued on a non-default stream gives the same bits."""
    w = wl.tiny_workload([(264, 136), (136, 264)], r=16, s=3, T=3, inner_rank=4, index=80)
    dev = torch.device("cuda")
    grads = _grads(w, 7, dev)
    a, b = _make(w), _make(w)
    Wa = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
    Wb = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    for k in range(7):
        a.step(Wa, grads[k])
        b.step(Wb, grads[k], stream=side)
    side.synchronize()
    torch.cuda.synchronize()
    assert all(torch.equal(x, y) for x, y in zip(Wa, Wb))
    assert a.poll_status()[0] == 0 and b.poll_status()[0] == 0


def test_sharded_wrapper_with_one_rank_equals_the_plain_optimizer():
    """One rank owns every matrix: the sharded wrapper (partition, subset stepping, weight exchange over the
    process group) must then give the bits of the plain optimizer.  The refresh draws its random test matrix from
    the seed and the matrix's position, so both sides get the subspaces injected."""
    import os

    import torch.distributed as dist

    from paper_2410_16029_b200.sharding import ShardedNGaLore

    w = wl.tiny_workload([(136, 264), (264, 136), (72, 40), (200, 96)], r=16, s=3, T=0, inner_rank=4, index=83)
    dev = torch.device("cuda")
    shapes = [(M, N) for _, M, N in w.shapes]
    grads = _grads(w, 5, dev)
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29761")
    dist.init_process_group("gloo", rank=0, world_size=1)
    try:
        kw = dict(lam=w.lam, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, wd=w.wd)
        sharded = ShardedNGaLore(shapes, w.r, w.s, 0, **kw)
        assert sharded.mine == [0, 1, 2, 3] and sharded.parts == [[0, 1, 2, 3]]
        plain = _make(w, T=0)
        plain.refresh_subspace(grads[0])
        for i in range(len(shapes)):
            sharded.opt.set_subspace(i, plain.get_subspace(i))
        Wa = [wl.initial_weight_device(w, i, dev) for i in range(w.n_matrices)]
        Wb = [t.clone() for t in Wa]
        for k in range(5):
            plain.step(Wa, grads[k])
            sharded.step(Wb, grads[k])
        torch.cuda.synchronize()
        for x, y in zip(Wa, Wb):
            assert torch.equal(x, y)
    finally:
        dist.destroy_process_group()


def test_import_into_a_state_that_has_stepped_since_the_export():
    """Export, step once more, import the blob back into the SAME state, step again: the bits of a straight run.
    The import brings back the exporting step's epoch; whatever the step in between left in the stream kernel's
    readiness flags must not be taken for the next step's."""
    w = wl.tiny_workload([(136, 264)], r=16, s=3, T=0, inner_rank=4, index=86)
    dev = torch.device("cuda")
    grads = _grads(w, 8, dev)
    P = None

    def run(detour):
        nonlocal P
        opt = _make(w)
        if P is None:
            opt.refresh_subspace(grads[0])
            P = opt.get_subspace(0).clone()
        else:
            opt.set_subspace(0, P)
        W = [torch.zeros((136, 264), device=dev)]
        for k in range(8):
            if detour and k == 5:
                blob = opt.export_state()
                scratch = [W[0].clone()]
                opt.step(scratch, grads[7])      # a step the straight run never makes
                torch.cuda.synchronize()
                opt.import_state(blob)
            opt.step(W, grads[k])
        torch.cuda.synchronize()
        assert opt.poll_status()[0] == 0
        return W[0].clone()

    a, b = run(False), run(True)
    assert torch.equal(a, b)


def test_a_wait_that_runs_out_is_reported_and_skips_only_that_matrix():
    """The bounded wait of the stream kernel's combination tiles: with the testing aid the weights of matrix 1 are
    computed but never announced, its tiles give up after a bounded number of polls, and the step ends by itself: status
    TIMEOUT for matrix 1, its W bitwise untouched, the other matrices updated as usual, and the next step clean."""
    from paper_2410_16029_b200.ngalore import NGaLoreError

    w = wl.tiny_workload([(136, 264), (264, 136), (72, 200)], r=16, s=3, T=0, inner_rank=4, index=87, wd=0.1)
    dev = torch.device("cuda")
    grads = _grads(w, 4, dev)
    a, b = _make(w), _make(w)
    a.refresh_subspace(grads[0])
    for i in range(3):
        b.set_subspace(i, a.get_subspace(i))
    Wa = [wl.initial_weight_device(w, i, dev) for i in range(3)]
    Wb = [t.clone() for t in Wa]
    for k in range(2):
        a.step(Wa, grads[k])
        b.step(Wb, grads[k])
    torch.cuda.synchronize()
    before = Wb[1].clone()
    b.debug_withhold_solution(1, 20000)
    a.step(Wa, grads[2])
    b.step(Wb, grads[2])
    torch.cuda.synchronize()
    code, per = b.poll_status()
    assert code == 8 and per == [0, 8, 0], (code, per)
    assert torch.equal(Wb[1], before)                       # neither decay nor update reached it
    assert torch.equal(Wb[0], Wa[0]) and torch.equal(Wb[2], Wa[2])
    # the aid lasts one step: the next one is regular again for every matrix
    before = [t.clone() for t in Wb]
    b.step(Wb, grads[3])
    torch.cuda.synchronize()
    assert b.poll_status() == (0, [0, 0, 0])
    assert all(not torch.equal(x, y) for x, y in zip(before, Wb))
    with pytest.raises(NGaLoreError):
        b.debug_withhold_solution(7, 20000)


def test_stepping_needs_a_projector_for_every_matrix():
    from paper_2410_16029_b200.ngalore import NGaLoreError

    w = wl.tiny_workload([(72, 40), (40, 72)], r=8, s=2, T=0, inner_rank=4, index=88)
    dev = torch.device("cuda")
    grads = _grads(w, 1, dev)
    opt = _make(w)
    W = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
    ref = _make(w)
    ref.refresh_subspace(grads[0])
    opt.set_subspace(0, ref.get_subspace(0))
    with pytest.raises(NGaLoreError) as e:
        opt.step(W, grads[0])
    assert e.value.code == 5                                 # NO_SUBSPACE: matrix 1 has none yet
    opt.refresh_subspace(grads[0], matrix_index=1)
    opt.step(W, grads[0])
    torch.cuda.synchronize()
    assert opt.poll_status()[0] == 0


def test_more_buffer_sets_than_cached_descriptor_sets():
    """The TMA descriptors of (W, G) pointer arrays are cached; a run that shows more distinct gradient buffers
    than the cache holds (sets get overwritten and come back) gives the bits of a run that always passes the same
    buffer."""
    w = wl.tiny_workload([(136, 264), (264, 136)], r=16, s=3, T=0, inner_rank=4, index=89)
    dev = torch.device("cuda")
    steps = 80
    grads = _grads(w, 40, dev)                               # 40 distinct buffer sets, cycled twice
    a, b = _make(w), _make(w)
    a.refresh_subspace(grads[0])
    for i in range(2):
        b.set_subspace(i, a.get_subspace(i))
    Wa = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
    Wb = [torch.zeros((M, N), device=dev) for _, M, N in w.shapes]
    fixed = [torch.empty_like(g) for g in grads[0]]
    for k in range(steps):
        a.step(Wa, grads[k % 40])
        for f, g in zip(fixed, grads[k % 40]):
            f.copy_(g)
        b.step(Wb, fixed)
    torch.cuda.synchronize()
    assert all(torch.equal(x, y) for x, y in zip(Wa, Wb))
    assert a.poll_status()[0] == 0 and b.poll_status()[0] == 0


def test_update_groups_and_overlapped_exchange_with_one_rank():
    """The weight update in groups with an event after each: same bits as the single launch; a side stream that waits
    for group g sees that group's weights updated; the sharded wrapper with the overlapped exchange (one rank: it
    owns everything) gives the bits of the plain optimizer."""
    import os

    import torch.distributed as dist

    from paper_2410_16029_b200.sharding import ShardedNGaLore

    w = wl.tiny_workload([(136, 264), (264, 136), (72, 40), (200, 96), (128, 512)], r=16, s=3, T=0, inner_rank=4, index=79)
    dev = torch.device("cuda")
    shapes = [(M, N) for _, M, N in w.shapes]
    grads = _grads(w, 4, dev)
    plain, grouped = _make(w), _make(w)
    plain.refresh_subspace(grads[0])
    for i in range(len(shapes)):
        grouped.set_subspace(i, plain.get_subspace(i))
    grouped.set_update_groups(3)
    ranges = grouped.update_groups()
    assert ranges[0][0] == 0 and ranges[-1][1] == len(shapes) and 2 <= len(ranges) <= 3   # about equal sizes, at most 3
    assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
    Wa = [wl.initial_weight_device(w, i, dev) for i in range(len(shapes))]
    Wb = [t.clone() for t in Wa]
    side = torch.cuda.Stream()
    copies = []
    for k in range(4):
        plain.step(Wa, grads[k])
        grouped.step(Wb, grads[k])
        for g, (a, b) in enumerate(ranges):
            grouped.stream_wait_update(g, side)
            with torch.cuda.stream(side):
                copies = [Wb[i].clone() for i in range(a, b)]
            torch.cuda.synchronize()
            assert all(torch.equal(c, Wa[i]) for c, i in zip(copies, range(a, b))), (k, g)
    assert all(torch.equal(x, y) for x, y in zip(Wa, Wb))
    grouped.set_update_groups(0)
    assert grouped.update_groups() == [(0, len(shapes))]
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29763")
    dist.init_process_group("gloo", rank=0, world_size=1)
    try:
        kw = dict(lam=w.lam, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, wd=w.wd)
        sharded = ShardedNGaLore(shapes, w.r, w.s, 0, update_groups=2, **kw)
        ref = _make(w)
        for i in range(len(shapes)):
            ref.set_subspace(i, plain.get_subspace(i))
            sharded.opt.set_subspace(i, plain.get_subspace(i))
        Wc = [wl.initial_weight_device(w, i, dev) for i in range(len(shapes))]
        Wd = [t.clone() for t in Wc]
        for k in range(3):
            ref.step(Wc, grads[k])
            sharded.step(Wd, grads[k])
        torch.cuda.synchronize()
        assert all(torch.equal(x, y) for x, y in zip(Wc, Wd))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("impl", [pytest.param(dict(gemm_impl=0), id="tcgen05"), pytest.param(dict(gemm_impl=1), id="simt")])
def test_refresh_and_step_on_a_zero_gradient(impl):
    """A frozen layer: its gradient is all zeros, at the refresh and in the steps.  There is no subspace to find; what
    is asked of the library is that the projector stays finite, no status is raised for it or for its neighbours, its
    weights only see the decay, and the other matrix is updated as if it were alone."""
    from paper_2410_16029_b200.ngalore import NGaLore

    shapes = [(264, 520), (136, 264)]
    w = wl.tiny_workload(shapes, r=16, s=3, T=0, inner_rank=4, index=91, wd=0.1)
    dev = torch.device("cuda")
    both = _make(w, **impl)
    alone = NGaLore([shapes[1]], w.r, w.s, 0, lam=w.lam, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, wd=w.wd, **impl)
    zero = torch.zeros(shapes[0], dtype=torch.bfloat16, device=dev)
    g1 = [wl.gradient_device(w, 1, k, dev) for k in range(4)]
    both.refresh_subspace([zero, g1[0]])
    alone.refresh_subspace([g1[0]])
    torch.cuda.synchronize()
    P0 = both.get_subspace(0)
    assert torch.isfinite(P0).all()
    alone.set_subspace(0, both.get_subspace(1))          # same projector for the live matrix on both sides
    W = [wl.initial_weight_device(w, i, dev) for i in range(2)]
    Wl = [W[1].clone()]
    W0 = W[0].clone()
    for k in range(4):
        both.step(W, [zero, g1[k]])
        alone.step(Wl, [g1[k]])
    torch.cuda.synchronize()
    assert both.poll_status() == (0, [0, 0])
    assert torch.isfinite(W[0]).all()
    expect = W0 * (1.0 - w.lr * w.wd) ** 4
    assert torch.allclose(W[0], expect, rtol=1e-5, atol=1e-7)     # u = 0 / sqrt(0 + eps) = 0: decay only
    assert torch.equal(W[1], Wl[0])


def test_refresh_on_a_gradient_that_is_not_finite():
    """A NaN in the gradient a refresh is given: that matrix's status says so, its projector becomes the first r' unit
    vectors (finite, orthonormal), the other matrix is refreshed as usual, and a later refresh on a clean gradient is
    regular again."""
    shapes = [(264, 520), (136, 264)]
    w = wl.tiny_workload(shapes, r=16, s=3, T=0, inner_rank=4, index=92)
    dev = torch.device("cuda")
    opt = _make(w)
    good = [wl.gradient_device(w, i, 0, dev) for i in range(2)]
    bad = good[0].clone()
    bad[7, 11] = float("nan")
    opt.refresh_subspace([bad, good[1]])
    torch.cuda.synchronize()
    code, per = opt.poll_status()
    assert code == 7 and per == [7, 0], (code, per)
    P0 = opt.get_subspace(0)
    expect = torch.zeros_like(P0)
    expect[:16, :16] = torch.eye(16, device=dev)
    assert torch.equal(P0, expect)
    P1 = opt.get_subspace(1).double()
    assert torch.allclose(P1.T @ P1, torch.eye(16, device=dev, dtype=torch.float64), atol=1e-5)
    opt.refresh_subspace(good)
    torch.cuda.synchronize()
    assert opt.poll_status() == (0, [0, 0])
    P0 = opt.get_subspace(0).double()
    assert torch.allclose(P0.T @ P0, torch.eye(16, device=dev, dtype=torch.float64), atol=1e-5)
