"""A device-side wait that runs out ends the kernel with an error code, not a hang: the bounded wait of the
tensor-core kernels, exercised by the library's diagnostic kernel on a barrier that nothing ever signals.  Nothing
here faults or hangs a GPU; the wait gives up by itself after the stated number of clocks."""
import time

import pytest
import torch

import oracle
import parity
from paper_2508_20407_b200 import binding as tl
from paper_2508_20407_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_expired_wait_is_reported_once_and_the_library_stays_usable():
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0
    waited = torch.zeros(1, dtype=torch.int64, device=DEV)
    limit = 200_000                                  # clocks: about 0.1 ms
    t0 = time.perf_counter()
    tl.tlin_debug_wait_expires(limit, waited)
    assert tl.tlin_last_launch_count() == 1
    status = tl.tlin_get_status()                    # synchronises the stream
    dt = time.perf_counter() - t0
    assert status == tl.ERR_TIMEOUT
    assert "timed out" in tl.status_string(status)
    assert tl.tlin_get_status() == 0                 # reading cleared it
    # the wait served its limit (it polls the clock every 256 tries, so a little more), and only once: the other
    # threads found the abort flag raised instead of waiting again
    assert limit <= int(waited.item()) <= 20 * limit
    assert dt < 5.0
    # the context is intact: an ordinary forward right afterwards is still correct
    wl = synth.Workload("after_timeout", 1, 2, 128, 1500, 200, seed=5)
    q, k, v = synth.forward_inputs(wl, device=DEV)
    out, lse = tl.tlin_attn_forward(q, k, v, causal_window=1)
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0
    ref, ref_lse = oracle.attn_forward(q.cpu(), k.cpu(), v.cpu(), 1)
    parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref, ref_lse, "bf16", "forward after an expired wait")


def test_wait_limit_is_validated_on_the_host():
    for bad in (0, -5, 3_000_000_000):
        with pytest.raises(tl.TlinError) as e:
            tl.tlin_debug_wait_expires(bad)
        assert e.value.status == tl.ERR_INVALID_ARG
