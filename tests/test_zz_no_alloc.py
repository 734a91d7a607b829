"""The workspace-free forward (hass_topk_distill_fwd_static) against the ordinary forward.

Some users of the library cannot allocate device memory when they call it (the GPU was reserved
up front by their framework, or their plug-in interface passes inputs and outputs only), so one
entry point keeps its scratch in an array compiled into the library. This file checks, through
the C ABI, that it returns what hass_topk_distill_fwd returns, on two consecutive calls with
different inputs (the second call finds the first call's leftovers in the shared array), and that
an oversized problem is refused instead of overrunning the array. The file name makes pytest
collect it after every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import hass_inputs as hi
from parity import compare

pytestmark = pytest.mark.gpu

LOSS_RTOL = 2e-3      # the tolerances of tests/parity.py
LSE_ATOL = 1e-4
Q_RTOL = 1e-3


def _compare(static, ref):
    assert int(static["device_status"].item()) == 0
    assert torch.equal(static["topk_idx"], ref["topk_idx"])
    np.testing.assert_allclose(static["topk_q"].cpu().numpy(), ref["topk_q"].cpu().numpy(), rtol=Q_RTOL)
    np.testing.assert_allclose(static["lse_t"].cpu().numpy(), ref["lse_t"].cpu().numpy(), atol=LSE_ATOL)
    np.testing.assert_allclose(static["lse_d"].cpu().numpy(), ref["lse_d"].cpu().numpy(), atol=LSE_ATOL)
    a, b = static["loss"].cpu().numpy(), ref["loss"].cpu().numpy()
    assert np.all(np.abs(a - b) <= LOSS_RTOL * np.maximum(np.abs(b), 1e-6))


def test_static_scratch_forward_matches_workspace_forward_twice_in_a_row():
    import paper_2408_15766_b200 as hass
    dev = torch.device("cuda:0")
    # two different problems back to back: a ragged one, then a larger one with more slots and K
    for (N, d, V, K, seed) in [(300, 256, 5000, 10, 1), (1000, 512, 33000, 24, 2)]:
        inp = hi.make_custom(N, d, V, K, seed=seed, sigma_w=2.0 / np.sqrt(d))
        H_t, H_d, W = inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev)
        ref = hass.topk_distill_fwd(H_t, H_d, W, K)
        hass.check(ref["workspace"])
        static = hass.topk_distill_fwd_static(H_t, H_d, W, K)
        torch.cuda.synchronize()
        _compare(static, ref)
        # and against the fp64 oracle itself (the forward has no dH_d)
        print(compare(inp.H_t, inp.H_d[0], inp.W, K, {k: v.cpu() for k, v in static.items()}, check_dH=False))
        # and once more on the same inputs, reusing the output tensors (no allocation at all)
        again = hass.topk_distill_fwd_static(H_t, H_d, W, K, out=static)
        torch.cuda.synchronize()
        _compare(again, ref)


@pytest.mark.parametrize("N,K_ok", [(8192, 16), (128, 53)])
def test_static_scratch_limit_is_the_declared_one(N, K_ok):
    """The largest K whose forward scratch fits the array (it depends on the number of row tiles) runs and agrees
    with the ordinary forward; the next K is refused on the host, before anything is launched."""
    import paper_2408_15766_b200 as hass
    dev = torch.device("cuda:0")
    d, V = 64, 128256
    limit = hass.STATIC_SCRATCH_MAX_BYTES
    fits = [K for K in range(1, 129) if hass.topk_distill_fwd_static_scratch_bytes(N, d, V, K) <= limit]
    assert fits == list(range(1, K_ok + 1))
    inp = hi.make_custom(N, d, V, K_ok, seed=7, sigma_w=0.25)
    H_t, H_d, W = inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev)
    ref = hass.topk_distill_fwd(H_t, H_d, W, K_ok)
    hass.check(ref["workspace"])
    static = hass.topk_distill_fwd_static(H_t, H_d, W, K_ok)
    torch.cuda.synchronize()
    _compare(static, ref)
    with pytest.raises(hass.HassError) as e:
        hass.topk_distill_fwd_static(H_t, H_d, W, K_ok + 1)
    assert e.value.status == -2
    torch.cuda.synchronize()


def test_static_scratch_refuses_a_problem_that_does_not_fit():
    import paper_2408_15766_b200 as hass
    dev = torch.device("cuda:0")
    N, d, V, K = 8192, 64, 128256, 128          # forward scratch far above 32 MiB
    assert hass.topk_distill_workspace_bytes(N, d, V, K) > (32 << 20)
    buf = torch.zeros(4096, dtype=torch.uint8, device=dev)
    p = ctypes.c_void_p(buf.data_ptr())
    rc = hass.lib.hass_topk_distill_fwd_static(p, p, p, N, d, V, K, p, p, p, p, p, None, None)
    assert rc == -2 and hass.status_string(rc) == "HASS_ERR_UNSUPPORTED"
    torch.cuda.synchronize()
