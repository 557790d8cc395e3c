"""GPU parity of the cached decode step against the CPU oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
import parity
from guards import Guarded
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
    # out, lse and the split workspace sit between filled guard regions, in buffers of exactly the documented sizes
    out_g, lse_g = Guarded((B, H, 1, d), torch.bfloat16, DEV), Guarded((B, H), torch.float32, DEV)
    ws_g = Guarded((tl.workspace_bytes_decode(B, H, kc.shape[2], d),), torch.uint8, DEV)
    saved = tl._workspace_tensor
    tl.set_workspace(ws_g.t)
    for t in range(T):
        out, lse = tl.tlin_decode_step(qn[t], kn[t], vn[t], kc, vc, N0 + t, out_g.t, lse_g.t)
        torch.cuda.synchronize()
        assert tl.tlin_get_status() == 0 and tl.tlin_last_launch_count() >= 1
        assert tl._workspace_tensor is ws_g.t
        for g, name in ((out_g, "out"), (lse_g, "lse"), (ws_g, "workspace")):
            g.check(f"decode step {t} {name}")
        ref, ref_lse = oracle.decode_step(qn[t].cpu(), kn[t].cpu(), vn[t].cpu(), kc_h, vc_h, N0 + t)
        parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref, ref_lse, "bf16", f"decode step {t}")
        # bit-exact bookkeeping: appended rows equal the new tokens, everything above is untouched
        assert torch.equal(kc.cpu(), kc_h) and torch.equal(vc.cpu(), vc_h)
        assert (kc[:, :, N0 + t + 1:] == -7.0).all() and (vc[:, :, N0 + t + 1:] == -7.0).all()
    tl.set_workspace(saved)


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


def _every_head_agrees(out, lse, ref_out, ref_lse, what, lse_gate=1e-3):
    """Two kernel families on the same inputs, both storing bf16: per (b,h) relative L2 <= 1e-2 (rounding of 128 bf16
    values gives about 2e-3) and |lse difference| <= lse_gate."""
    a, b = out.float().flatten(2), ref_out.float().flatten(2)                 # [B,H,d]
    assert torch.isfinite(a).all() and torch.isfinite(lse).all(), what
    rel = ((a - b).pow(2).sum(-1) / b.pow(2).sum(-1).clamp_min(1e-30)).sqrt()
    assert float(rel.max()) <= 1e-2, f"{what}: worst (b,h) rel L2 {float(rel.max()):.3e} at {int(rel.argmax())}"
    dl = (lse.flatten() - ref_lse.flatten()).abs()
    assert float(dl.max()) <= lse_gate, f"{what}: lse differs by {float(dl.max()):.3e} at {int(dl.argmax())}"


def test_cfg5_every_head_against_the_forward_kernels_on_the_cache():
    """The oracle recomputes three heads of cfg5; here every (b,h) of a step is compared with the forward entry point run
    on the same cache (one query row, all cached rows, no mask): a different kernel family, different split of the keys."""
    wl = synth.WORKLOADS["cfg5_decode"]
    (kc, vc), (qn, kn, vn) = synth.decode_inputs(wl, device=DEV, steps=3)
    for t in range(3):
        out, lse = tl.tlin_decode_step(qn[t], kn[t], vn[t], kc, vc, wl.N + t)
        ref_out, ref_lse = tl.tlin_attn_forward_cache(qn[t], kc, vc, wl.N + t + 1, causal_window=0)
        torch.cuda.synchronize()
        assert tl.tlin_get_status() == 0
        _every_head_agrees(out, lse, ref_out, ref_lse, f"cfg5 step {t}")


def test_ragged_decode_one_length_per_sequence():
    """Sequences of one batch at different cache lengths (positions read from device memory): every sequence
    equals the oracle's step at its own length; appended rows are bit-exact; nothing else in the caches moves."""
    B, H, d, T = 4, 3, 128, 3
    lengths = [0, 37, 1500, 4099]
    ncap = max(lengths) + T + 2
    rng = torch.Generator(device="cpu").manual_seed(77)
    kc = (torch.randn((B, H, ncap, d), generator=rng) * 1.0).to(torch.bfloat16)
    vc = (torch.randn((B, H, ncap, d), generator=rng) * 1.0).to(torch.bfloat16)
    for b, n0 in enumerate(lengths):
        kc[b, :, n0:] = -7.0
        vc[b, :, n0:] = -7.0
    kc_h, vc_h = kc.clone(), vc.clone()
    kc, vc = kc.to(DEV), vc.to(DEV)
    pos = torch.tensor(lengths, dtype=torch.int32, device=DEV)
    for t in range(T):
        qn = (torch.randn((B, H, 1, d), generator=rng)).to(torch.bfloat16)
        kn = (torch.randn((B, H, 1, d), generator=rng)).to(torch.bfloat16)
        vn = (torch.randn((B, H, 1, d), generator=rng)).to(torch.bfloat16)
        out, lse = tl.tlin_decode_step_ragged(qn.to(DEV), kn.to(DEV), vn.to(DEV), kc, vc, pos, max(lengths) + t)
        torch.cuda.synchronize()
        assert tl.tlin_get_status() == 0
        for b, n0 in enumerate(lengths):
            sl = slice(b, b + 1)
            ref, ref_lse = oracle.decode_step(qn[sl], kn[sl], vn[sl], kc_h[sl], vc_h[sl], n0 + t)   # updates the host caches in place
            parity.check(out[sl].float().cpu().numpy(), lse[sl].cpu().numpy(), ref, ref_lse, "bf16", f"ragged step {t} seq {b}")
        assert torch.equal(kc.cpu(), kc_h) and torch.equal(vc.cpu(), vc_h)
        pos += 1                                   # advanced on the device


def test_ragged_decode_reports_a_position_beyond_the_bound():
    B, H, d = 2, 2, 64
    kc = torch.zeros((B, H, 64, d), dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    kc_before = kc.clone()
    x = torch.ones((B, H, 1, d), dtype=torch.bfloat16, device=DEV)
    pos = torch.tensor([5, 40], dtype=torch.int32, device=DEV)      # 40 exceeds the bound given below
    kc_h, vc_h = kc.cpu(), vc.cpu()
    out, lse = tl.tlin_decode_step_ragged(x, x, x, kc, vc, pos, 10)
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == tl.ERR_INVALID_ARG
    assert tl.tlin_get_status() == 0                                  # reading clears it
    assert torch.equal(kc[1], kc_before[1])                           # the offending sequence's cache is untouched
    assert (kc[0, :, 5] == 1).all()                                   # the valid one was appended
    # the rejected sequence gets zeros and an empty log-sum-exp, not NaN; the valid one its ordinary result
    assert float(out[1].float().abs().max()) == 0.0 and bool((lse[1] == float("-inf")).all())
    ref, ref_lse = oracle.decode_step(x[:1].cpu(), x[:1].cpu(), x[:1].cpu(), kc_h[:1], vc_h[:1], 5)
    parity.check(out[:1].float().cpu().numpy(), lse[:1].cpu().numpy(), ref, ref_lse, "bf16", "valid sequence beside a rejected one")
    with pytest.raises(tl.TlinError):
        tl.tlin_decode_step_ragged(x, x, x, kc, vc, pos, 64)          # bound outside the cache: rejected on the host


def test_ragged_decode_loop_replays_from_a_cuda_graph():
    """With the positions in device memory a whole decode loop can be recorded once and replayed: the captured
    sequence is [step; pos += 1] and a replay continues where the previous one stopped."""
    B, H, d, n0 = 2, 4, 64, 300
    steps_per_graph, replays = 4, 3
    total = steps_per_graph * replays
    ncap = n0 + total + 8
    wl = synth.Workload("graph", B, H, d, n0, total, seed=91, decode=True)
    (kc0, vc0), (qn, kn, vn) = synth.decode_inputs(wl, device=DEV)
    kc = torch.zeros((B, H, ncap, d), dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    kc[:, :, :n0], vc[:, :, :n0] = kc0[:, :, :n0], vc0[:, :, :n0]
    kc_ref, vc_ref = kc.clone(), vc.clone()
    # eager reference run: the same entry point with the same bound (hence the same split of the key range), call by call
    ref_out = []
    pos_ref = torch.full((B,), n0, dtype=torch.int32, device=DEV)
    for t in range(total):
        o, _ = tl.tlin_decode_step_ragged(qn[t], kn[t], vn[t], kc_ref, vc_ref, pos_ref, ncap - 1)
        pos_ref += 1
        ref_out.append(o.clone())
    torch.cuda.synchronize()
    # captured run: the graph reads its tokens from staging tensors that are refilled before every replay
    tl.ensure_workspace(tl.workspace_bytes_decode(B, H, ncap, d), torch.device(DEV))
    pos = torch.full((B,), n0, dtype=torch.int32, device=DEV)
    q_st, k_st, v_st = (torch.empty((steps_per_graph, B, H, 1, d), dtype=torch.bfloat16, device=DEV) for _ in range(3))
    outs = torch.empty((steps_per_graph, B, H, 1, d), dtype=torch.bfloat16, device=DEV)
    lses = torch.empty((steps_per_graph, B, H), dtype=torch.float32, device=DEV)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        # one eager warm-up step on scratch copies so that nothing is initialised for the first time under capture
        tl.tlin_decode_step_ragged(qn[0], kn[0], vn[0], kc.clone(), vc.clone(), pos.clone(), ncap - 1, stream=stream)
        stream.synchronize()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(steps_per_graph):
                tl.tlin_decode_step_ragged(q_st[i], k_st[i], v_st[i], kc, vc, pos, ncap - 1, outs[i], lses[i], stream=stream)
                pos.add_(1)
    got = []
    for r in range(replays):
        sl = slice(r * steps_per_graph, (r + 1) * steps_per_graph)
        q_st.copy_(qn[sl]); k_st.copy_(kn[sl]); v_st.copy_(vn[sl])
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        got.extend(outs[i].clone() for i in range(steps_per_graph))
    assert tl.tlin_get_status() == 0
    assert int(pos[0]) == n0 + total
    for t in range(total):
        assert torch.equal(got[t], ref_out[t]), f"step {t}"
    assert torch.equal(kc[:, :, :n0 + total], kc_ref[:, :, :n0 + total])


def _fp8_cache(wl, pad):
    """Quantises the seeded bf16 cache of `wl` to E4M3 codes on the host (library conversion, pinned against the oracle's
    codec on the CPU side), one scale per (b,h) such that the largest magnitude maps to 224."""
    (kc, vc), (qn, kn, vn) = synth.decode_inputs(wl, device="cpu")
    B, H, d = wl.B, wl.H, wl.d
    def scales(x):
        amax = x.float().abs().amax(dim=(2, 3)) if x.shape[2] > 0 else torch.ones(B, H)
        return (torch.clamp(amax, min=1e-3) / 224.0).float().contiguous()
    ks, vs = scales(torch.cat([kc, kn.transpose(0, 2).reshape(B, H, -1, d)], 2)), scales(torch.cat([vc, vn.transpose(0, 2).reshape(B, H, -1, d)], 2))
    def codes(x, s):
        c = (x.float() / s[:, :, None, None]).to(torch.float8_e4m3fn).view(torch.uint8)
        c = torch.cat([c, torch.zeros((B, H, pad, d), dtype=torch.uint8)], 2).contiguous()
        c[:, :, wl.N:] = 0x55                # canary in every row that is not live yet
        return c
    return codes(kc, ks), codes(vc, vs), ks, vs, qn, kn, vn


@pytest.mark.parametrize("B,H,d,N0,T", [(2, 3, 128, 1000, 5), (1, 2, 64, 5, 9), (1, 1, 128, 0, 4), (2, 2, 64, 4100, 3)])
def test_fp8_decode_steps_elementwise_and_exact_codes(B, H, d, N0, T):
    wl = synth.Workload("dec8", B, H, d, N0, T, seed=61 + N0, decode=True)
    kc_h, vc_h, ks, vs, qn, kn, vn = _fp8_cache(wl, pad=2)
    kc, vc = kc_h.to(DEV), vc_h.to(DEV)
    ks_d, vs_d = ks.to(DEV), vs.to(DEV)
    for t in range(T):
        out, lse = tl.tlin_decode_step_fp8(qn[t].to(DEV), kn[t].to(DEV), vn[t].to(DEV), kc, vc, ks_d, vs_d, N0 + t)
        torch.cuda.synchronize()
        assert tl.tlin_get_status() == 0 and tl.tlin_last_launch_count() == 2
        ref, ref_lse = oracle.decode_step_fp8(qn[t], kn[t], vn[t], kc_h, vc_h, ks, vs, N0 + t)
        parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref, ref_lse, "bf16", f"fp8 decode step {t}")
        # byte-exact bookkeeping: the appended codes equal the oracle's (same fp32 division, same rounding), the canary
        # rows above are untouched
        assert torch.equal(kc.cpu(), kc_h) and torch.equal(vc.cpu(), vc_h)
        assert (kc[:, :, N0 + t + 1:] == 0x55).all() and (vc[:, :, N0 + t + 1:] == 0x55).all()


def test_fp8_decode_saturates_and_keeps_signed_zero_like_the_oracle():
    B, H, d, Ncap = 1, 2, 64, 8
    kc = torch.zeros(B, H, Ncap, d, dtype=torch.uint8, device=DEV)
    vc = torch.zeros_like(kc)
    ks = torch.full((B, H), 0.01, device=DEV)
    vs = torch.full((B, H), 0.5, device=DEV)
    kn = torch.linspace(-8.0, 8.0, d).repeat(B, H, 1, 1).to(torch.bfloat16)       # |x| / 0.01 goes far beyond 448
    vn = torch.cat([torch.tensor([0.0, -0.0, 1e-4, -1e-4]), torch.linspace(-300, 300, d - 4)]).repeat(B, H, 1, 1).to(torch.bfloat16)
    q = torch.ones(B, H, 1, d).to(torch.bfloat16)
    kc_h, vc_h = kc.cpu(), vc.cpu()
    out, lse = tl.tlin_decode_step_fp8(q.to(DEV), kn.to(DEV), vn.to(DEV), kc, vc, ks, vs, 0)
    torch.cuda.synchronize()
    ref, ref_lse = oracle.decode_step_fp8(q, kn, vn, kc_h, vc_h, ks.cpu(), vs.cpu(), 0)
    assert torch.equal(kc.cpu(), kc_h) and torch.equal(vc.cpu(), vc_h)
    assert int(kc_h[0, 0, 0].max()) <= 0xFE and 0x7E in kc_h[0, 0, 0].tolist() and 0xFE in kc_h[0, 0, 0].tolist()
    got = out.float().cpu().numpy()
    assert np.abs(got - ref).max() <= 2e-2 * max(1.0, float(np.abs(ref).max()))


def test_fp8_decode_at_the_cfg5_size_on_sampled_heads():
    # the benchmarked 8-bit configuration (B8 H32 d128, 65536 cached rows): three heads of three steps against the oracle,
    # the appended codes of those heads byte for byte
    wl = synth.WORKLOADS["cfg5_decode"]
    B, H, d, N = wl.B, wl.H, wl.d, wl.N
    g = torch.Generator(device=DEV).manual_seed(77)
    def codes():
        c = torch.randint(0, 254, (B, H, N + 8, d), generator=g, device=DEV, dtype=torch.int16)
        return (c + (c >= 127).to(torch.int16)).to(torch.uint8).contiguous()       # every finite code, no NaN code
    kc, vc = codes(), codes()
    ks = (torch.rand(B, H, generator=g, device=DEV) * 0.01 + 0.002).float()
    vs = (torch.rand(B, H, generator=g, device=DEV) * 0.01 + 0.002).float()
    q, kn, vn = (torch.randn(3, B, H, 1, d, generator=g, device=DEV).to(torch.bfloat16) for _ in range(3))
    heads = [(0, 0), (3, 17), (7, 31)]
    host = {bh: (kc[bh[0], bh[1]].cpu().view(1, 1, -1, d).contiguous(), vc[bh[0], bh[1]].cpu().view(1, 1, -1, d).contiguous()) for bh in heads}
    for t in range(3):
        out, lse = tl.tlin_decode_step_fp8(q[t], kn[t], vn[t], kc, vc, ks, vs, N + t)
        torch.cuda.synchronize()
        assert tl.tlin_get_status() == 0
        for (b, h) in heads:
            sl = lambda x: x[b:b + 1, h:h + 1].cpu().contiguous()
            kh, vh = host[(b, h)]
            ref, ref_lse = oracle.decode_step_fp8(sl(q[t]), sl(kn[t]), sl(vn[t]), kh, vh, sl(ks), sl(vs), N + t)
            parity.check(sl(out).float().numpy(), sl(lse).numpy(), ref, ref_lse, "bf16", f"8-bit cfg5 step {t} head {(b, h)}")
    for (b, h) in heads:
        assert torch.equal(kc[b, h].cpu(), host[(b, h)][0][0, 0]) and torch.equal(vc[b, h].cpu(), host[(b, h)][1][0, 0])


def test_fp8_decode_at_the_cfg5_size_every_head_against_the_bf16_kernels():
    """Every (b,h) of an 8-bit step against the forward entry point on the same cache after torch has turned the codes into
    bf16 values (code * scale, rounded to bf16).  That rounding moves every key by up to 2^-9 of itself, and with keys
    as large as these (codes up to 448, scales up to 0.012) the scores of the few keys that carry a row move by a few 1e-3:
    the lse gate of this comparison is 1e-2, the output gate the usual one."""
    wl = synth.WORKLOADS["cfg5_decode"]
    B, H, d, N = wl.B, wl.H, wl.d, wl.N
    g = torch.Generator(device=DEV).manual_seed(78)
    def codes():
        c = torch.randint(0, 254, (B, H, N + 8, d), generator=g, device=DEV, dtype=torch.int16)
        return (c + (c >= 127).to(torch.int16)).to(torch.uint8).contiguous()       # every finite code, no NaN code
    kc, vc = codes(), codes()
    ks = (torch.rand(B, H, generator=g, device=DEV) * 0.01 + 0.002).float()
    vs = (torch.rand(B, H, generator=g, device=DEV) * 0.01 + 0.002).float()
    q, kn, vn = (torch.randn(B, H, 1, d, generator=g, device=DEV).to(torch.bfloat16) for _ in range(3))
    out, lse = tl.tlin_decode_step_fp8(q, kn, vn, kc, vc, ks, vs, N)
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0
    def values(c, scale):       # [B,H,N+1,d] bf16, a (b,h) at a time to bound the fp32 temporaries
        v = torch.empty((B, H, N + 1, d), dtype=torch.bfloat16, device=DEV)
        for b in range(B):
            v[b] = (c[b, :, :N + 1].view(torch.float8_e4m3fn).float() * scale[b].view(H, 1, 1)).to(torch.bfloat16)
        return v
    kb, vb = values(kc, ks), values(vc, vs)
    ref_out, ref_lse = tl.tlin_attn_forward_cache(q, kb, vb, N + 1, causal_window=0)
    torch.cuda.synchronize()
    _every_head_agrees(out, lse, ref_out, ref_lse, "8-bit cfg5 step", lse_gate=1e-2)


@pytest.mark.parametrize("B,H,d,hist,W_og,W_oh,extra", [(2, 3, 128, 300, 64, 48, 5), (1, 2, 64, 1000, 130, 40, 3), (1, 2, 72, 90, 20, 8, 2)])
def test_window_slide_cycle_on_the_cache_in_place(B, H, d, hist, W_og, W_oh, extra):
    """Section 4.1 / 5.2: decode W_og cached steps, then the window slides and the layers that look at the history run
    again from scratch -- here directly on the cache buffer (first n rows of a larger allocation, nothing copied) --
    and decoding continues on the same buffers.  Every output against the oracle; the caches bit-equal throughout."""
    if d not in (64, 128):
        steps_ok = False        # the decode kernel serves d in {64,128}; other head sizes exercise the forward over the cache only
    else:
        steps_ok = True
    total = W_og + extra
    wl = synth.Workload("slide", B, H, d, hist, total, seed=500 + hist, decode=True)
    (kc, vc), (qn, kn, vn) = synth.decode_inputs(wl, device=DEV)
    pad = 3                                                    # canary rows above everything that is ever written
    kc = torch.cat([kc, torch.full((B, H, pad, d), -7.0, dtype=kc.dtype, device=DEV)], dim=2).contiguous()
    vc = torch.cat([vc, torch.full((B, H, pad, d), -7.0, dtype=vc.dtype, device=DEV)], dim=2).contiguous()
    kc[:, :, hist:] = -7.0
    vc[:, :, hist:] = -7.0
    kc_h, vc_h = kc.cpu(), vc.cpu()
    dec_out, dec_lse = [], []

    def decode(t):
        if steps_ok:
            o, l = tl.tlin_decode_step(qn[t], kn[t], vn[t], kc, vc, hist + t)
            torch.cuda.synchronize()
            assert tl.tlin_get_status() == 0
        ref, ref_lse = oracle.decode_step(qn[t].cpu(), kn[t].cpu(), vn[t].cpu(), kc_h, vc_h, hist + t)
        if steps_ok:
            parity.check(o.float().cpu().numpy(), l.cpu().numpy(), ref, ref_lse, "bf16", f"decode step {t}")
            assert torch.equal(kc.cpu(), kc_h) and torch.equal(vc.cpu(), vc_h)
            dec_out.append(o.clone())
            dec_lse.append(l.clone())
        else:                                                   # no decode kernel for this head size: place the rows by copy
            kc[:, :, hist + t] = kn[t][:, :, 0]
            vc[:, :, hist + t] = vn[t][:, :, 0]

    for t in range(W_og):                                       # the window fills up
        decode(t)
    pos = hist + W_og                                           # the window slides: all `pos` cached rows are history now
    # (a) summary queries over the new history (focused attention), on the cache in place
    g = torch.Generator(device="cpu").manual_seed(hist)
    q_sum = torch.randn((B, H, W_oh, d), generator=g).to(torch.bfloat16).to(DEV)
    out, lse = tl.tlin_attn_forward_cache(q_sum, kc, vc, pos, causal_window=0)
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0
    ref, ref_lse = oracle.attn_forward(q_sum.cpu(), kc_h[:, :, :pos].contiguous(), vc_h[:, :, :pos].contiguous(), 0)
    parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref, ref_lse, "bf16", "summary queries over the slid history")
    # (b) the window just completed, recomputed as a cache-miss forward: its rows are what the decode steps returned
    q_win = torch.cat([qn[t] for t in range(W_og)], dim=2).contiguous()
    out, lse = tl.tlin_attn_forward_cache(q_win, kc, vc, pos, causal_window=1)
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0
    ref, ref_lse = oracle.attn_forward(q_win.cpu(), kc_h[:, :, :pos].contiguous(), vc_h[:, :, :pos].contiguous(), 1)
    parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref, ref_lse, "bf16", "window recomputed over the cache")
    if steps_ok:
        steps = torch.cat(dec_out, dim=2).float()
        assert float((steps - out.float()).abs().max()) <= 2e-2
        assert float((torch.stack(dec_lse, dim=2) - lse).abs().max()) <= 1e-3
    # the forward calls wrote nothing into the caches, and the rows above `pos` still hold the canary
    assert torch.equal(kc.cpu(), kc_h) and torch.equal(vc.cpu(), vc_h)
    assert (kc[:, :, pos:] == -7.0).all() and (vc[:, :, pos:] == -7.0).all()
    for t in range(W_og, total):                                # decoding continues in the next window
        decode(t)
    assert (kc[:, :, hist + total:] == -7.0).all() and (vc[:, :, hist + total:] == -7.0).all()
    with pytest.raises(tl.TlinError):
        tl.tlin_attn_forward_cache(q_sum, kc, vc, kc.shape[2] + 1, causal_window=0)      # more rows than the cache has


@pytest.mark.parametrize("d,n_problems", [(128, 5), (64, 3), (128, 50)])
def test_batched_decode_table_every_problem_against_the_oracle(d, n_problems):
    """A table of short cached steps in one launch (per-layer rows of a cache-hit step, Appendix A): problems of different
    cache lengths and head counts, some appending the new token, some attending to a finished cache only."""
    rng = torch.Generator(device="cpu").manual_seed(1000 + d + n_problems)
    problems, host = [], []
    for i in range(n_problems):
        bh = int(torch.randint(1, 7, (1,), generator=rng))
        pos = int(torch.randint(1, 1400 if i % 3 else 40, (1,), generator=rng))
        append = i % 2 == 0
        ncap = pos + 3
        kc = torch.randn((1, bh, ncap, d), generator=rng).to(torch.bfloat16)
        vc = torch.randn((1, bh, ncap, d), generator=rng).to(torch.bfloat16)
        kc[:, :, pos:] = -7.0
        vc[:, :, pos:] = -7.0
        qn, kn, vn = (torch.randn((1, bh, 1, d), generator=rng).to(torch.bfloat16) for _ in range(3))
        out = torch.empty((1, bh, 1, d), dtype=torch.bfloat16, device=DEV)
        lse = torch.empty((1, bh), dtype=torch.float32, device=DEV)
        host.append((qn, kn, vn, kc, vc, pos, append))
        problems.append((qn.to(DEV), kn.to(DEV) if append else None, vn.to(DEV) if append else None, kc.to(DEV), vc.to(DEV), pos, out, lse))
    tl.tlin_decode_step_batched(problems)
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0 and tl.tlin_last_launch_count() == -(-n_problems // 48)
    for i, ((qn, kn, vn, kc, vc, pos, append), pr) in enumerate(zip(host, problems)):
        out, lse, kc_d, vc_d = pr[6], pr[7], pr[3], pr[4]
        if append:
            ref, ref_lse = oracle.decode_step(qn, kn, vn, kc, vc, pos)                     # updates kc, vc in place
        else:
            ref, ref_lse = oracle.attn_forward(qn, kc[:, :, :pos].contiguous(), vc[:, :, :pos].contiguous(), 0)
        parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref.reshape(out.shape), ref_lse.reshape(lse.shape), "bf16", f"table problem {i}")
        assert torch.equal(kc_d.cpu(), kc) and torch.equal(vc_d.cpu(), vc)               # appended row bit-exact, the rest untouched
    with pytest.raises(tl.TlinError):
        bad = list(problems[0]); bad[5] = problems[0][3].shape[2]                          # pos beyond the cache
        tl.tlin_decode_step_batched([tuple(bad)])
