"""The allocation-free entry point against the regular optimizer step.

Some users of this library run where device allocation is not available to them (a fixed memory
budget carved up at start-up, or a host framework that forbids cudaMalloc once it is running), so they
cannot create an optimizer state.  ngalore_natural_gradient_static serves them with scratch that is
part of the library image.  This test drives it next to ngalore_step on the same gradients and checks
that both produce the same natural gradient, on several calls in a row (the calls share the scratch).

How the comparison works: with M = r (so P can be the identity), beta1 = beta2 = 0 and lr = 1 the step
writes W = -N~ / sqrt(N~^2 + eps) into a zeroed W, where N~ is the natural gradient of the current
low-rank gradient R = G; the static entry point returns N~ itself from a caller-kept history ring.
The same N~ is also computed by the fp64 oracle from a host copy of that ring and compared directly.
"""
import numpy as np
import pytest
import torch

from oracle import natural_galore as orc
from paper_2410_16029_b200 import workload as wl
from tests.parity_util import TOL_UPDATE, rel_err, to_device_bf16

pytestmark = pytest.mark.gpu


def test_static_natural_gradient_matches_step_on_consecutive_calls():
    from paper_2410_16029_b200.ngalore import NGaLore, natural_gradient_static

    dev = torch.device("cuda")
    M, N, s, lam, eps = 64, 320, 4, 1e-3, 1e-6
    n = M * N                                     # 20480 elements: three scratch tiles, the last one ragged
    w = wl.tiny_workload([(M, N)], r=M, s=s, T=0, inner_rank=4, index=98)
    opt = NGaLore([(M, N)], M, s, 0, lam=lam, lr=1.0, beta1=0.0, beta2=0.0, eps=eps)
    opt.set_subspace(0, torch.eye(M))
    H = torch.zeros((s, n), dtype=torch.float32, device=dev)
    K = torch.zeros((s, s), dtype=torch.float64, device=dev)
    out = torch.empty(n, dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    for k in range(6):                            # fills the ring and wraps around it
        G = to_device_bf16(wl.gradient_bits(w, 0, k), dev)
        W = torch.zeros((M, N), dtype=torch.float32, device=dev)
        opt.step([W], [G])
        cur, count = k % s, min(k + 1, s)
        H[cur].copy_(G.float().reshape(-1))
        natural_gradient_static(H, count, cur, lam, K, out, status)
        torch.cuda.synchronize()
        nat = out.double().reshape(M, N)
        expect = -(nat / torch.sqrt(nat * nat + eps))
        err = (torch.linalg.norm(W.double() - expect) / torch.linalg.norm(expect)).item()
        assert err <= TOL_UPDATE, (k, err)
        assert status.item() == 0
        # directly against the oracle: F^-1 applied to the newest gradient over the gradients the ring holds
        ring = H.double().cpu().numpy()
        want = orc.natural_gradient(ring[cur], [ring[j] for j in range(count)], lam)
        assert rel_err(out.double().cpu().numpy(), want) <= TOL_UPDATE, (k, rel_err(out.double().cpu().numpy(), want))
    assert opt.poll_status()[0] == 0


def test_static_entry_rejects_sizes_beyond_its_scratch():
    from paper_2410_16029_b200.ngalore import NGaLoreError, natural_gradient_static

    dev = torch.device("cuda")
    n = 8388608 + 8192
    H = torch.zeros((1, n), dtype=torch.float32, device=dev)
    K = torch.zeros((1, 1), dtype=torch.float64, device=dev)
    out = torch.empty(n, dtype=torch.float32, device=dev)
    with pytest.raises(NGaLoreError) as e:
        natural_gradient_static(H, 1, 0, 1e-3, K, out)
    assert e.value.code == 1
