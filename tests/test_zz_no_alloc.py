"""The decode entry point for callers that cannot allocate (scratch built into the library) must give
what tlin_decode_step gives.  Collected last on purpose: a run that stops at the first failure has
then already been through every other test."""
import ctypes

import pytest
import torch

import oracle
import parity
from paper_2508_20407_b200 import binding as tl
from paper_2508_20407_b200 import synth

DEV = "cuda"


# the last two cases fill the built-in array to its last partial slot (256 (b,h) pairs at d = 128, 508 at d = 64)
@pytest.mark.gpu
@pytest.mark.parametrize("B,H,d,N0", [(2, 4, 128, 3000), (1, 3, 64, 700), (8, 32, 128, 40), (4, 127, 64, 9)])
def test_static_scratch_decode_matches_workspace_decode_and_the_oracle_twice_in_a_row(B, H, d, N0):
    wl = synth.Workload("static_dec", B, H, d, N0, 2, seed=77 + N0, decode=True)
    (kc, vc), (qn, kn, vn) = synth.decode_inputs(wl, device=DEV)
    kc2, vc2 = kc.clone(), vc.clone()
    kc_h, vc_h = kc.cpu(), vc.cpu()
    out = torch.empty((wl.B, wl.H, 1, wl.d), dtype=torch.bfloat16, device=DEV)
    lse = torch.empty((wl.B, wl.H), dtype=torch.float32, device=DEV)
    for t in range(wl.W):                      # two calls in a row share the built-in array
        ref_out, ref_lse = tl.tlin_decode_step(qn[t], kn[t], vn[t], kc, vc, wl.N + t)
        tl.tlin_decode_step_static(qn[t], kn[t], vn[t], kc2, vc2, wl.N + t, out, lse)
        assert tl.tlin_last_launch_count() == 2          # counted from zero by every call: split kernel + merge
        torch.cuda.synchronize()
        assert tl.tlin_get_status() == 0
        parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref_out.float().cpu().numpy(),
                     ref_lse.cpu().numpy(), "bf16", f"static scratch against the workspace entry point, step {t}")
        assert torch.equal(kc, kc2) and torch.equal(vc, vc2)
        o_ref, l_ref = oracle.decode_step(qn[t].cpu(), kn[t].cpu(), vn[t].cpu(), kc_h, vc_h, wl.N + t)
        parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), o_ref, l_ref, "bf16", f"static scratch against the oracle, step {t}")
        assert torch.equal(kc2.cpu(), kc_h) and torch.equal(vc2.cpu(), vc_h)


@pytest.mark.gpu
def test_static_scratch_decode_rejects_shapes_beyond_its_array():
    # B*H = 257 pairs at d = 128 is one pair too many; validation happens before any launch
    p = ctypes.c_void_p(torch.zeros(64, dtype=torch.uint8, device=DEV).data_ptr())
    rc = tl.lib().tlin_decode_step_static(p, p, p, p, p, p, None, 257, 1, 16, 3, 128, None)
    assert rc == tl.ERR_WORKSPACE
    assert tl.lib().tlin_decode_step_static(p, p, p, p, p, p, None, 509, 1, 16, 3, 64, None) == tl.ERR_WORKSPACE


def test_static_scratch_decode_validates_arguments_on_the_host():
    one = ctypes.c_void_p(16)
    L = tl.lib()
    assert L.tlin_decode_step_static(None, one, one, one, one, one, None, 1, 1, 8, 3, 128, None) == tl.ERR_INVALID_ARG
    assert L.tlin_decode_step_static(one, one, one, one, one, one, None, 1, 1, 8, 8, 128, None) == tl.ERR_INVALID_ARG
    assert L.tlin_decode_step_static(one, one, one, one, one, one, None, 1, 1, 8, 3, 48, None) == tl.ERR_UNSUPPORTED
    assert L.tlin_decode_step_static(one, one, one, one, one, one, None, 600, 1, 8, 3, 128, None) == tl.ERR_WORKSPACE
