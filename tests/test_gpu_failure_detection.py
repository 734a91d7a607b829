"""Failure detection on the device: a bounded wait that runs out must end its kernel, leave a code in the
status word, be reported once by hass_check as HASS_ERR_TIMEOUT, and leave the context usable.

The wait is made to run out in the library's own self-test kernel (a barrier that nothing completes, a limit
of two milliseconds); no real kernel is disturbed, nothing faults, traps or spins beyond its limit."""
import pytest
import torch

import hass_inputs as hi
from parity import compare

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_once_and_the_next_call_is_clean():
    import paper_2408_15766_b200 as hass
    dev = torch.device("cuda:0")
    wl = hi.WORKLOADS["tiny"]
    inp = hi.make_inputs(wl)
    H_t, H_d, W = inp.H_t.to(dev), inp.H_d[0].to(dev), inp.W.to(dev)
    ws = torch.zeros(hass.topk_distill_workspace_bytes(wl.N, wl.d, wl.V, wl.K), dtype=torch.uint8, device=dev)

    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    hass.selftest_wait_expiry(ws, limit_ns=2_000_000)
    t1.record()
    with pytest.raises(hass.HassError) as e:
        hass.check(ws)
    assert e.value.status == -5 and hass.status_string(-5) == "HASS_ERR_TIMEOUT"
    words = ws[:128].view(torch.int32).cpu()
    assert int(words[16]) == 128                      # every thread's wait ended: one by its limit, the rest by the flag
    waited_ms = int(words[17]) / 1e6
    assert 2.0 <= waited_ms < 50.0 and t0.elapsed_time(t1) < 100.0      # gave up at the limit, not at the 2 s default
    hass.check(ws)                                    # the report was cleared: clean from here on

    # the context is intact: an ordinary call on the same workspace gives oracle-exact results
    out = hass.topk_distill_fwd_bwd(H_t, H_d, W, wl.K, dH_dtype=hass.HASS_FP32, workspace=ws)
    hass.check(ws)
    print(compare(inp.H_t, inp.H_d[0], inp.W, wl.K, {k: v.cpu() for k, v in out.items() if k != "workspace"}))

    # limits outside 1 us .. 100 ms are refused on the host
    for bad in (0, 10**9):
        with pytest.raises(hass.HassError) as e:
            hass.selftest_wait_expiry(ws, limit_ns=bad)
        assert e.value.status == -1
