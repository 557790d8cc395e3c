"""GPU parity of the cached decode step against the CPU oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2508_20407_b200 import binding as tl
from paper_2508_20407_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("B,H,d,N0,T", [(2, 3, 128, 1000, 6), (1, 2, 64, 5, 9), (1, 1, 128, 0, 4), (2, 2, 64, 4100, 3),
                                        (1, 4, 128, 20000, 2)])
def test_decode_steps_elementwise_and_cache_bookkeeping(B, H, d, N0, T):
    wl = synth.Workload("dec", B, H, d, N0, T, seed=21 + N0, decode=True)
    (kc, vc), (qn, kn, vn) = synth.decode_inputs(wl, device=DEV)
    # canary rows above the live range: must stay untouched
    pad = 2
    kc = torch.cat([kc, torch.full((B, H, pad, d), -7.0, dtype=kc.dtype, device=DEV)], dim=2).contiguous()
    vc = torch.cat([vc, torch.full((B, H, pad, d), -7.0, dtype=vc.dtype, device=DEV)], dim=2).contiguous()
    kc[:, :, N0:N0 + T] = -7.0
    vc[:, :, N0:N0 + T] = -7.0
    kc_h, vc_h = kc.cpu(), vc.cpu()
    for t in range(T):
        out, lse = tl.tlin_decode_step(qn[t], kn[t], vn[t], kc, vc, N0 + t)
        torch.cuda.synchronize()
        assert tl.tlin_get_status() == 0 and tl.tlin_last_launch_count() >= 1
        ref, ref_lse = oracle.decode_step(qn[t].cpu(), kn[t].cpu(), vn[t].cpu(), kc_h, vc_h, N0 + t)
        parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref, ref_lse, "bf16", f"decode step {t}")
        # bit-exact bookkeeping: appended rows equal the new tokens, everything above is untouched
        assert torch.equal(kc.cpu(), kc_h) and torch.equal(vc.cpu(), vc_h)
        assert (kc[:, :, N0 + t + 1:] == -7.0).all() and (vc[:, :, N0 + t + 1:] == -7.0).all()


def test_decode_equals_rows_of_the_forward_oracle():
    wl = synth.Workload("dec_rows", 1, 2, 128, 700, 5, seed=31, decode=True)
    (kc, vc), (qn, kn, vn) = synth.decode_inputs(wl, device=DEV)
    outs, lses = [], []
    for t in range(wl.W):
        o, l = tl.tlin_decode_step(qn[t], kn[t], vn[t], kc, vc, wl.N + t)
        outs.append(o.clone())
        lses.append(l.clone())
    torch.cuda.synchronize()
    q_all = torch.cat([qn[t] for t in range(wl.W)], dim=2).cpu()
    ref, ref_lse = oracle.attn_forward(q_all, kc.cpu(), vc.cpu(), 1)   # the caches now hold the whole sequence
    got = torch.cat(outs, dim=2).float().cpu().numpy()
    got_lse = torch.stack(lses, dim=2).cpu().numpy()
    parity.check(got, got_lse, ref, ref_lse, "bf16", "decode rows vs forward oracle")


def test_decode_rejects_missing_workspace_and_bad_pos():
    wl = synth.Workload("dec_err", 1, 1, 64, 10, 1, seed=1, decode=True)
    (kc, vc), (qn, kn, vn) = synth.decode_inputs(wl, device=DEV)
    with pytest.raises(tl.TlinError) as e:
        tl.tlin_decode_step(qn[0], kn[0], vn[0], kc, vc, kc.shape[2])
    assert e.value.status == tl.ERR_INVALID_ARG
    saved = tl._workspace_tensor
    tl.set_workspace(None)
    try:
        rc = tl.lib().tlin_decode_step(qn[0].data_ptr(), kn[0].data_ptr(), vn[0].data_ptr(), kc.data_ptr(), vc.data_ptr(),
                                       qn[0].data_ptr(), None, 1, 1, kc.shape[2], 10, 64, None)
        assert rc == tl.ERR_WORKSPACE
    finally:
        tl.set_workspace(saved)


def test_cfg5_full_size_sampled_heads_and_steps():
    wl = synth.WORKLOADS["cfg5_decode"]
    (kc, vc), (qn, kn, vn) = synth.decode_inputs(wl, device=DEV)
    heads = [(0, 0), (3, 17), (7, 31)]
    check_steps = {0, 1, 2, 127, 254, 255}
    host = {bh: (kc[bh[0], bh[1]].cpu().view(1, 1, -1, wl.d).contiguous(), vc[bh[0], bh[1]].cpu().view(1, 1, -1, wl.d).contiguous())
            for bh in heads}
    out = torch.empty((wl.B, wl.H, 1, wl.d), dtype=torch.bfloat16, device=DEV)
    lse = torch.empty((wl.B, wl.H), dtype=torch.float32, device=DEV)
    for t in range(wl.W):
        tl.tlin_decode_step(qn[t], kn[t], vn[t], kc, vc, wl.N + t, out, lse)
        for (b, h) in heads:
            sl = lambda x: x[b:b + 1, h:h + 1].cpu().contiguous()
            kh, vh = host[(b, h)]
            if t in check_steps:
                torch.cuda.synchronize()
                ref, ref_lse = oracle.decode_step(sl(qn[t]), sl(kn[t]), sl(vn[t]), kh, vh, wl.N + t)
                parity.check(sl(out).float().numpy(), sl(lse).numpy(), ref, ref_lse, "bf16", f"cfg5 step {t} head {(b, h)}")
            else:  # keep the host copy of the cache in step without the attention
                kh[0, 0, wl.N + t] = kn[t, b, h, 0].cpu()
                vh[0, 0, wl.N + t] = vn[t, b, h, 0].cpu()
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0
    for (b, h) in heads:
        assert torch.equal(kc[b, h].cpu(), host[(b, h)][0][0, 0]) and torch.equal(vc[b, h].cpu(), host[(b, h)][1][0, 0])
