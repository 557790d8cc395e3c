"""GPU parity of the forward entry points against the CPU oracle (element by element on the same
seeded inputs; sampled rows at the full benchmark sizes).  Everything goes through the C-ABI."""
from concurrent.futures import ThreadPoolExecutor

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


def run_impl(impl, fn, *a, **kw):
    prev = tl.tlin_set_forward_impl(impl)
    try:
        out = fn(*a, **kw)
        torch.cuda.synchronize()
        assert tl.tlin_get_status() == 0
        assert tl.tlin_last_launch_count() >= 1
        return out
    finally:
        tl.tlin_set_forward_impl(prev)


def impls_for(d):
    return [1, 2] if d in (64, 128) and TC_AVAILABLE else [1]


def _tc_available():
    try:
        prev = tl.tlin_set_forward_impl(2)
        try:
            p = tl.tlin_plan_forward(1, 1, 128, 128, 64, 0)
            if not torch.cuda.is_available():
                return False
            q = torch.zeros(1, 1, 128, 64, dtype=torch.bfloat16, device=DEV)
            tl.tlin_attn_forward(q, q, q, causal_window=0)
            torch.cuda.synchronize()
            return bool(p.tensor_path)
        finally:
            tl.tlin_set_forward_impl(prev)
    except tl.TlinError:
        return False


TC_AVAILABLE = _tc_available() if torch.cuda.is_available() else False


def full_compare(wl, impl, kind="bf16", causal=None):
    causal = wl.causal_window if causal is None else causal
    dtype = torch.bfloat16 if kind == "bf16" else torch.float32
    q, k, v = synth.forward_inputs(wl, device=DEV, dtype=dtype)
    fn = tl.tlin_attn_forward if kind == "bf16" else tl.tlin_attn_forward_f32
    out, lse = run_impl(impl, fn, q, k, v, causal_window=causal)
    ref, ref_lse = oracle.attn_forward(q.cpu(), k.cpu(), v.cpu(), causal)
    return parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref, ref_lse, kind, f"{wl.name} impl={impl}")


@pytest.mark.parametrize("impl", [0, 1, 2])
def test_cfg1_tiny_elementwise(impl):
    if impl == 2 and not TC_AVAILABLE:
        pytest.skip("tensor path not built")
    full_compare(synth.WORKLOADS["cfg1_tiny"], impl)


SHAPES = [  # B, H, N, W, d, causal
    (1, 1, 1, 1, 64, 1), (1, 2, 129, 1, 64, 1), (2, 1, 128, 128, 64, 1), (1, 2, 300, 300, 128, 1),
    (1, 3, 1000, 77, 128, 1), (2, 2, 515, 130, 64, 0), (1, 2, 257, 255, 128, 0), (1, 1, 4096, 384, 128, 1),
    (1, 2, 2049, 129, 64, 1), (1, 1, 100, 300, 128, 0), (1, 1, 640, 512, 128, 1), (3, 2, 1111, 200, 64, 1),
]


def guarded_compare(wl, impl):
    """full_compare with out, lse and the split workspace inside guarded buffers of exactly the documented sizes."""
    causal = wl.causal_window
    q, k, v = synth.forward_inputs(wl, device=DEV)
    out_g = Guarded(q.shape, torch.bfloat16, DEV)
    lse_g = Guarded((wl.B, wl.H, wl.W), torch.float32, DEV)
    saved = tl._workspace_tensor
    prev = tl.tlin_set_forward_impl(impl)
    try:
        need = tl.workspace_bytes_forward(wl.B, wl.H, wl.N, wl.W, wl.d, causal)
        ws_g = Guarded((max(need, 16),), torch.uint8, DEV)
        tl.set_workspace(ws_g.t)
        out, lse = tl.tlin_attn_forward(q, k, v, out_g.t, lse_g.t, causal_window=causal)
        torch.cuda.synchronize()
        assert tl.tlin_get_status() == 0 and tl.tlin_last_launch_count() >= 1
        assert tl._workspace_tensor is ws_g.t          # the call used the guarded workspace, nothing larger
    finally:
        tl.tlin_set_forward_impl(prev)
        tl.set_workspace(saved)
    for g, name in ((out_g, "out"), (lse_g, "lse"), (ws_g, "workspace")):
        g.check(f"{wl.name} impl={impl} {name}")
    ref, ref_lse = oracle.attn_forward(q.cpu(), k.cpu(), v.cpu(), causal)
    return parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref, ref_lse, "bf16", f"{wl.name} impl={impl}")


@pytest.mark.parametrize("B,H,N,W,d,causal", SHAPES)
def test_awkward_shapes_bf16(B, H, N, W, d, causal):
    wl = synth.Workload("shape", B, H, d, N, W, seed=100 + N + W, causal_window=causal)
    for impl in impls_for(d):
        guarded_compare(wl, impl)


def partials_per_head(plan):
    """For a schedule-0 plan: how many groups (= partial results per query row) each (b,h) is spread over."""
    starts = [tl.tlin_plan_group_start(plan, g) for g in range(plan.n_groups + 1)]
    T = plan.key_tiles
    counts = []
    for bh in range(plan.total_units // T):
        lo, hi = bh * T, (bh + 1) * T
        counts.append(sum(1 for g in range(plan.n_groups) if starts[g] < hi and starts[g + 1] > lo))
    return counts


def random_shapes(seed, count, budget=4e9):
    """Seeded shapes that no one picked by hand: tile edges +-1, window rule on and off, few and many (b,h), key ranges that
    are split between CTAs and ones that are not; B*H*W*N*d bounded so that the oracle stays within a second per shape."""
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        d = int(rng.choice([64, 128]))
        causal = int(rng.integers(0, 2))
        kind = int(rng.integers(0, 4))
        if kind == 0:       # long keys, few queries
            W, N, BH = int(rng.integers(1, 700)), int(rng.integers(700, 9000)), int(rng.integers(1, 5))
        elif kind == 1:     # square-ish
            W = int(rng.integers(1, 1400)); N, BH = W + int(rng.integers(0, 400)), int(rng.integers(1, 7))
        elif kind == 2:     # tile edges
            W = max(1, 128 * int(rng.integers(1, 9)) + int(rng.integers(-1, 2)))
            N, BH = max(1, 128 * int(rng.integers(1, 30)) + int(rng.integers(-1, 2))), int(rng.integers(1, 9))
        else:               # many queries, few keys
            W, N, BH = int(rng.integers(300, 3000)), int(rng.integers(1, 700)), int(rng.integers(1, 6))
        if causal and N < W:
            N = W
        while BH > 1 and BH * W * N * d > budget:
            BH -= 1
        if BH * W * N * d > budget:
            continue
        B = 2 if BH % 2 == 0 and rng.integers(0, 2) else 1
        out.append((B, BH // B, N, W, d, causal))
    return out


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_forward_random_shapes_against_the_oracle(seed):
    if not TC_AVAILABLE:
        pytest.skip("tensor path not built")
    for (B, H, N, W, d, causal) in random_shapes(seed, 10):
        wl = synth.Workload(f"random B{B} H{H} N{N} W{W} d{d} causal{causal}", B, H, d, N, W, seed=seed * 1000 + N + W,
                            causal_window=causal)
        guarded_compare(wl, 2)


@pytest.mark.parametrize("seed", [15, 16])
def test_forward_random_shapes_cuda_core_kernels_and_fp32(seed):
    # the same generator through the kernels that serve every other head size, in bf16 and in fp32 (the paper's d = 36 included)
    rng = np.random.default_rng(seed)
    for (B, H, N, W, d, causal) in random_shapes(seed, 8, budget=1e9):
        d16 = int(rng.choice([8, 40, 64, 96, 128, 200, 256]))
        d32 = int(rng.choice([4, 36, 64, 100, 128, 256]))
        N, W = min(N, 3000), min(W, 1000)
        if causal and N < W:
            N = W
        guarded_compare(synth.Workload(f"random B{B} H{H} N{N} W{W} d{d16} causal{causal}", B, H, d16, N, W, seed=seed * 1000 + N,
                                       causal_window=causal), 1)
        full_compare(synth.Workload(f"random f32 B{B} H{H} N{N} W{W} d{d32} causal{causal}", B, H, d32, N, W, seed=seed * 1000 + W,
                                    causal_window=causal), 0, kind="f32")


def test_awkward_shapes_reach_both_branches_of_the_split_merge():
    # the merge kernel combines up to 8 partial results per row from registers and more than 8 in a loop: the shapes
    # above must keep exercising both, whatever the planner turns into
    if not TC_AVAILABLE:
        pytest.skip("tensor path not built")
    few = many = False
    prev = tl.tlin_set_forward_impl(2)
    try:
        for (B, H, N, W, d, causal) in SHAPES:
            plan = tl.tlin_plan_forward(B, H, N, W, d, causal)
            if not (plan.tensor_path and plan.schedule == 0 and plan.uses_workspace):
                continue
            c = partials_per_head(plan)
            few = few or any(2 <= x <= 8 for x in c)
            many = many or any(x > 8 for x in c)
    finally:
        tl.tlin_set_forward_impl(prev)
    assert few, "no awkward shape is split into 2..8 partial results per row"
    assert many, "no awkward shape is split into more than 8 partial results per row"


@pytest.mark.parametrize("B,H,N,W,d,causal", [(1, 2, 333, 40, 36, 1), (1, 1, 1024, 128, 64, 1), (2, 2, 200, 200, 128, 1),
                                              (1, 2, 77, 5, 256, 0), (1, 1, 1, 1, 4, 1), (1, 1, 2000, 9, 100, 1)])
def test_fp32_path(B, H, N, W, d, causal):
    wl = synth.Workload("f32", B, H, d, N, W, seed=7 + d, causal_window=causal)
    full_compare(wl, 0, kind="f32")


@pytest.mark.parametrize("B,H,N,W,d,causal", [(1, 2, 256, 40000, 128, 0), (2, 1, 300, 38000, 64, 0), (6, 16, 1024, 1000, 64, 1),
                                              (1, 160, 384, 512, 64, 0),
                                              # window rule with several query tiles and at least three problems per CTA:
                                              # the CTAs share the problems by cost, runs cross (b,h) borders, ragged tails
                                              (2, 40, 1600, 1500, 128, 1), (3, 50, 900, 900, 64, 1)])
def test_many_queries_few_keys_schedule(B, H, N, W, d, causal):
    """Restoring cross-attention shape (Section 3): every history token queries a few summary tokens.
    The planner hands whole (b,h,query tile) problems to the CTAs; parity on sampled heads and rows."""
    wl = synth.Workload("wide", B, H, d, N, W, seed=300 + N, causal_window=causal)
    assert tl.tlin_plan_forward(B, H, N, W, d, causal).schedule == 1
    q, k, v = synth.forward_inputs(wl, device=DEV)
    out, lse = run_impl(2 if TC_AVAILABLE else 1, tl.tlin_attn_forward, q, k, v, causal_window=causal)
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
    rng = np.random.default_rng(N)
    for (b, h) in {(0, 0), (B - 1, H - 1)}:
        rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, W - 1], rng.integers(0, W, 250)]))
        qs = q[b:b + 1, h:h + 1, rows].contiguous().cpu()
        if causal:      # row i sees keys j <= N - W + i: compare row by row through the unmasked oracle call
            for idx in np.unique(np.linspace(0, len(rows) - 1, 40).astype(int)):      # 40 rows spread over all query tiles
                i = rows[idx]
                lim = N - W + int(i) + 1
                if lim < 1:
                    continue
                ref, ref_lse = oracle.attn_forward(qs[:, :, idx:idx + 1], k[b:b + 1, h:h + 1, :lim].cpu(), v[b:b + 1, h:h + 1, :lim].cpu(), 0)
                parity.check(out[b, h, int(i)].float().cpu().numpy()[None], lse[b, h, int(i)].cpu().numpy()[None], ref.reshape(1, -1), ref_lse.reshape(1), "bf16", f"wide causal row {i}")
        else:
            ref, ref_lse = oracle.attn_forward(qs, k[b:b + 1, h:h + 1].cpu(), v[b:b + 1, h:h + 1].cpu(), 0)
            parity.check(out[b, h, rows].float().cpu().numpy(), lse[b, h, rows].cpu().numpy(), ref[0, 0], ref_lse[0, 0], "bf16", f"wide head {(b, h)}")


def test_bf16_fallback_head_dims():
    for d in (8, 72, 256):
        full_compare(synth.Workload("odd_d", 1, 2, d, 300, 33, seed=d), 0)


def test_peaky_keys_stress_rescaling():
    wl = synth.Workload("peaky", 1, 2, 128, 3000, 256, seed=2, peaky=(100, 8.0))
    for impl in impls_for(128):
        full_compare(wl, impl)


def test_future_tokens_do_not_change_earlier_rows():
    wl = synth.Workload("causal_inv", 1, 2, 64, 700, 200, seed=11)
    q, k, v = synth.forward_inputs(wl, device=DEV)
    for impl in impls_for(64):
        out0, lse0 = run_impl(impl, tl.tlin_attn_forward, q, k, v, causal_window=1)
        i = 57
        k2, v2 = k.clone(), v.clone()
        k2[:, :, wl.N - wl.W + i + 1:] += 3.0
        v2[:, :, wl.N - wl.W + i + 1:] -= 2.0
        out1, lse1 = run_impl(impl, tl.tlin_attn_forward, q, k2, v2, causal_window=1)
        assert torch.equal(out0[:, :, :i + 1], out1[:, :, :i + 1]) and torch.equal(lse0[:, :, :i + 1], lse1[:, :, :i + 1])
        assert not torch.equal(out0[:, :, i + 1:], out1[:, :, i + 1:])


def test_run_to_run_bitwise_determinism():
    wl = synth.Workload("det", 2, 4, 128, 5000, 300, seed=12)
    q, k, v = synth.forward_inputs(wl, device=DEV)
    for impl in impls_for(128):
        a, la = run_impl(impl, tl.tlin_attn_forward, q, k, v, causal_window=1)
        b, lb = run_impl(impl, tl.tlin_attn_forward, q, k, v, causal_window=1)
        assert torch.equal(a, b) and torch.equal(la, lb)


def test_merge_joins_history_and_window_calls():
    wl = synth.Workload("merge", 1, 2, 64, 900, 128, seed=13)
    q, k, v = synth.forward_inputs(wl, device=DEV)
    joint, joint_lse = tl.tlin_attn_forward(q, k, v, causal_window=1)
    hist = wl.N - wl.W
    oh, lh = tl.tlin_attn_forward(q, k[:, :, :hist].contiguous(), v[:, :, :hist].contiguous(), causal_window=0)
    ow, lw = tl.tlin_attn_forward(q, k[:, :, hist:].contiguous(), v[:, :, hist:].contiguous(), causal_window=1)
    out, lse = tl.tlin_merge_lse(oh, lh, ow, lw)
    torch.cuda.synchronize()
    ref, ref_lse = oracle.attn_forward(q.cpu(), k.cpu(), v.cpu(), 1)
    parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref, ref_lse, "bf16", "merge of two calls")
    parity.check(joint.float().cpu().numpy(), joint_lse.cpu().numpy(), ref, ref_lse, "bf16", "joint call")
    # fp32 merge against the oracle's merge on the same partials, empty side included
    oa = torch.randn(50, 64, device=DEV)
    ob = torch.randn(50, 64, device=DEV)
    la = torch.randn(50, device=DEV) * 3
    lb = torch.randn(50, device=DEV) * 3
    lb[3] = float("-inf")
    la[7] = float("-inf")
    la[9] = lb[9] = float("-inf")
    o, l = tl.tlin_merge_lse(oa, la, ob, lb)
    torch.cuda.synchronize()
    r, rl = oracle.merge_lse(oa.cpu().double().numpy(), la.cpu().double().numpy(), ob.cpu().double().numpy(), lb.cpu().double().numpy())
    assert np.abs(o.cpu().numpy() - r).max() < 1e-5
    fin = np.isfinite(rl)
    assert np.abs(l.cpu().numpy()[fin] - rl[fin]).max() < 1e-5 and (l.cpu().numpy()[~fin] == -np.inf).all()


def sampled_rows_compare(wl, impl, rows_per_head, heads, causal):
    """Full-size run; the oracle recomputes sampled query rows one by one (row i alone over keys [0, limit))."""
    q, k, v = synth.forward_inputs(wl, device=DEV)
    out, lse = run_impl(impl, tl.tlin_attn_forward, q, k, v, causal_window=causal)
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
    rng = np.random.default_rng(wl.seed)
    jobs = []
    for (b, h) in heads:
        kh, vh = k[b, h].cpu(), v[b, h].cpu()
        rows = sorted(set([0, wl.W - 1] + [int(x) for x in rng.integers(0, wl.W, rows_per_head)]))
        for i in rows:
            limit = wl.N - wl.W + i + 1 if causal else wl.N
            jobs.append((b, h, i, q[b, h, i].cpu().view(1, 1, 1, wl.d), kh[:limit].view(1, 1, limit, wl.d), vh[:limit].view(1, 1, limit, wl.d)))
    with ThreadPoolExecutor(max_workers=8) as ex:
        refs = list(ex.map(lambda j: oracle.attn_forward(j[3], j[4], j[5], 0), jobs))
    got = np.stack([out[b, h, i].float().cpu().numpy() for (b, h, i, *_rest) in jobs])
    got_lse = np.array([lse[b, h, i].item() for (b, h, i, *_rest) in jobs])
    ref = np.stack([r[0].reshape(-1) for r in refs])
    ref_lse = np.array([r[1].item() for r in refs])
    return parity.check(got, got_lse, ref, ref_lse, "bf16", f"{wl.name} impl={impl} sampled rows")


def test_cfg2_mid_sampled_heads_full_rows():
    wl = synth.WORKLOADS["cfg2_mid"]
    q, k, v = synth.forward_inputs(wl, device=DEV)
    for impl in impls_for(wl.d):
        out, lse = run_impl(impl, tl.tlin_attn_forward, q, k, v, causal_window=1)
        for (b, h) in [(0, 0), (3, 15), (1, 7)]:
            sl = lambda t: t[b:b + 1, h:h + 1].contiguous().cpu()
            ref, ref_lse = oracle.attn_forward(sl(q), sl(k), sl(v), 1)
            parity.check(sl(out).float().numpy(), sl(lse).numpy(), ref, ref_lse, "bf16", f"cfg2 head {(b, h)} impl={impl}")


def stratified_rows(wl, b, h, per_tile):
    """`per_tile` hashed rows in every 128-row query tile of head (b,h): each CTA of any plan (256 query rows of one or
    several heads) then has sampled rows in both of its query tiles, in its first and in its last head."""
    rng = np.random.default_rng(wl.seed * 1000003 + b * 131 + h)
    rows = []
    for r0 in range(0, wl.W, 128):
        r1 = min(r0 + 128, wl.W)
        rows.extend(int(x) for x in rng.choice(np.arange(r0, r1), size=min(per_tile, r1 - r0), replace=False))
    return sorted(rows)


@pytest.mark.parametrize("name,causal", [("cfg3_long", 1), ("cfg3_long", 0), ("cfg4_vlong", 1), ("cfg4_vlong", 0)])
def test_full_size_sampled_rows(name, causal):
    """The benchmarked launch at full size: every row of heads {0, H/2, H-1} and 16 hashed rows of every other head
    against the oracle.  The rows are spread over all 128-row query tiles, so every CTA of the plan, whose key range
    may start or end inside a head (partial results, merged by the second kernel), has checked rows in the first and
    in the last head it works on."""
    wl = synth.WORKLOADS[name]
    impl = 2 if TC_AVAILABLE else 1
    q, k, v = synth.forward_inputs(wl, device=DEV)
    out, lse = run_impl(impl, tl.tlin_attn_forward, q, k, v, causal_window=causal)
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
    full_heads = [(0, 0), (0, wl.H // 2), (0, wl.H - 1)]
    per_tile = max(1, 16 // ((wl.W + 127) // 128))
    sampled = {(b, h): stratified_rows(wl, b, h, per_tile) for b in range(wl.B) for h in range(wl.H) if (b, h) not in full_heads}
    # every CTA = (group, 256-row query tile pair) has checked rows in the first and the last head of its unit range
    plan = tl.tlin_plan_forward(wl.B, wl.H, wl.N, wl.W, wl.d, causal)
    if plan.tensor_path and plan.schedule == 0:
        starts = [tl.tlin_plan_group_start(plan, g) for g in range(plan.n_groups + 1)]
        for g in range(plan.n_groups):
            for bh in {starts[g] // plan.key_tiles, (starts[g + 1] - 1) // plan.key_tiles}:
                head = (bh // wl.H, bh % wl.H)
                rows = range(wl.W) if head in full_heads else sampled[head]
                for qt in range(plan.q_tiles):
                    for half in range(2):
                        lo = qt * 256 + half * 128
                        if lo < wl.W:
                            assert any(lo <= r < lo + 128 for r in rows), (g, head, qt, half)
    for (b, h) in full_heads:
        sl = lambda t: t[b:b + 1, h:h + 1].contiguous().cpu()
        ref, ref_lse = oracle.attn_forward(sl(q), sl(k), sl(v), causal)
        parity.check(sl(out).float().numpy(), sl(lse).numpy(), ref, ref_lse, "bf16", f"{name} causal={causal} head {(b, h)}, all rows")
    got, got_lse, ref, ref_lse = [], [], [], []
    for (b, h), rows in sampled.items():
        kh, vh = k[b, h].cpu(), v[b, h].cpu()
        qh = q[b, h].cpu()
        if causal:      # row i alone over the keys it may use, through the unmasked oracle call
            jobs = []
            for i in rows:
                limit = wl.N - wl.W + i + 1
                jobs.append((qh[i].view(1, 1, 1, wl.d), kh[:limit].view(1, 1, limit, wl.d), vh[:limit].view(1, 1, limit, wl.d)))
            with ThreadPoolExecutor(max_workers=8) as ex:
                res = list(ex.map(lambda j: oracle.attn_forward(j[0], j[1], j[2], 0), jobs))
            ref.extend(r[0].reshape(-1) for r in res)
            ref_lse.extend(float(r[1].reshape(-1)[0]) for r in res)
        else:
            r, rl = oracle.attn_forward(qh[rows].view(1, 1, len(rows), wl.d), kh.view(1, 1, wl.N, wl.d), vh.view(1, 1, wl.N, wl.d), 0)
            ref.extend(r[0, 0])
            ref_lse.extend(rl[0, 0])
        got.extend(out[b, h, rows].float().cpu().numpy())
        got_lse.extend(lse[b, h, rows].cpu().numpy())
    parity.check(np.stack(got), np.array(got_lse), np.stack(ref), np.array(ref_lse), "bf16", f"{name} causal={causal}, hashed rows of the other heads")


@pytest.mark.parametrize("name", ["cfg3_long", "cfg4_vlong"])
def test_full_size_tensor_core_path_agrees_with_the_cuda_core_path_everywhere(name):
    # CUDA against CUDA, a supplement to the oracle checks above (it proves nothing by itself): the two kernels share no
    # tiling, schedule or split, and the CUDA-core one is the path verified element by element on the small shapes
    if not TC_AVAILABLE:
        pytest.skip("tensor path not built")
    wl = synth.WORKLOADS[name]
    q, k, v = synth.forward_inputs(wl, device=DEV)
    a, la = run_impl(2, tl.tlin_attn_forward, q, k, v, causal_window=1)
    b, lb = run_impl(1, tl.tlin_attn_forward, q, k, v, causal_window=1)
    # both sides are rounded to bf16, so besides the absolute gate of the oracle comparison two values may sit one last
    # place (2^-7 relative) apart; the peaked rows of the long configuration reach magnitudes of several units
    af, bf = a.float(), b.float()
    excess = (af - bf).abs() - (2.0 ** -7) * torch.maximum(af.abs(), bf.abs())
    assert float(excess.max()) <= 2e-2
    assert float((af - bf).abs().mean()) <= 2e-3
    assert float((af - bf).norm() / bf.norm()) <= 2e-2
    assert float((la - lb).abs().max()) <= 1e-3


def test_whole_sequence_causal_attention_sampled_rows():
    # N = W = 4096 over B4 H32: whole (b,h,query tile) problems per CTA, shared between the CTAs by cost, so a CTA's
    # run of problems crosses (b,h) borders; rows sampled in the first, a middle and the last (b,h)
    wl = synth.WORKLOADS["train_seq"]
    impl = 2 if TC_AVAILABLE else 1
    plan = tl.tlin_plan_forward(wl.B, wl.H, wl.N, wl.W, wl.d, 1)
    if impl == 2:
        assert plan.schedule == 1 and plan.uses_workspace == 0
    sampled_rows_compare(wl, impl, 14, [(0, 0), (1, 17), (wl.B - 1, wl.H - 1)], 1)


def test_chunk_scheduled_forward_equals_per_chunk_calls_and_full_causal_attention():
    # Sliding-window training (Section 5.1): C windows of W tokens, window c attends to everything up to its own end.
    # One call over shared k, v; each chunk must equal the oracle on the key prefix, and the chunks laid end to end are
    # the rows of plain causal attention over the whole sequence.
    if not TC_AVAILABLE:
        pytest.skip("tensor path not built")
    C, B, H, W, d = 5, 2, 2, 96, 128
    L = C * W
    wl = synth.Workload("chunks", B, H, d, L, L, seed=41, causal_window=1)
    q_all, k, v = synth.forward_inputs(wl, device=DEV, dtype=torch.bfloat16)          # q_all [B,H,L,d]
    q = q_all.view(B, H, C, W, d).permute(2, 0, 1, 3, 4).contiguous()                 # [C,B,H,W,d]
    n_keys = [(c + 1) * W for c in range(C)]
    out, lse = tl.tlin_attn_forward_prefixes(q, k, v, n_keys, causal_window=1)
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0 and tl.tlin_last_launch_count() >= C
    for c in range(C):
        ref, ref_lse = oracle.attn_forward(q[c].cpu(), k[:, :, :n_keys[c]].contiguous().cpu(), v[:, :, :n_keys[c]].contiguous().cpu(), 1)
        parity.check(out[c].float().cpu().numpy(), lse[c].cpu().numpy(), ref, ref_lse, "bf16", f"chunk {c}")
    full, full_lse = tl.tlin_attn_forward(q_all, k, v, causal_window=1)
    stitched = out.permute(1, 2, 0, 3, 4).reshape(B, H, L, d)
    assert float((stitched.float() - full.float()).abs().max()) <= 2e-2
    assert float((lse.permute(1, 2, 0, 3).reshape(B, H, L) - full_lse).abs().max()) <= 1e-3


def test_chunk_scheduled_forward_ragged_prefixes_without_mask():
    # focused attention of every chunk over its own history: W summary queries, unmasked, arbitrary prefix lengths
    if not TC_AVAILABLE:
        pytest.skip("tensor path not built")
    C, B, H, W, d, L = 3, 1, 3, 40, 64, 1000
    wl = synth.Workload("prefixes", B, H, d, L, C * W, seed=43, causal_window=0)
    q_all, k, v = synth.forward_inputs(wl, device=DEV, dtype=torch.bfloat16)
    q = q_all.view(B, H, C, W, d).permute(2, 0, 1, 3, 4).contiguous()
    n_keys = [100, 333, 1000]
    out, lse = tl.tlin_attn_forward_prefixes(q, k, v, n_keys, causal_window=0)
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0
    for c in range(C):
        ref, ref_lse = oracle.attn_forward(q[c].cpu(), k[:, :, :n_keys[c]].contiguous().cpu(), v[:, :, :n_keys[c]].contiguous().cpu(), 0)
        parity.check(out[c].float().cpu().numpy(), lse[c].cpu().numpy(), ref, ref_lse, "bf16", f"prefix {n_keys[c]}")
    with pytest.raises(tl.TlinError):
        tl.tlin_attn_forward_prefixes(q, k, v, [100, 333, 1001], causal_window=0)      # beyond the key tensor


def _batched_case(d, specs, seed):
    """specs: (B, H, rows, n_keys, W, causal); k, v hold `rows` rows per head of which the first n_keys are used."""
    problems, refs = [], []
    for i, (B, H, rows, n_keys, W, causal) in enumerate(specs):
        wl = synth.Workload(f"tab{i}", B, H, d, rows, W, seed=seed + i, causal_window=causal)
        q, k, v = synth.forward_inputs(wl, device=DEV)
        out_g = Guarded(q.shape, torch.bfloat16, DEV)
        lse_g = Guarded((B, H, W), torch.float32, DEV)
        problems.append((q, k, v, out_g.t, lse_g.t, n_keys, causal))
        refs.append((out_g, lse_g))
    return problems, refs


@pytest.mark.parametrize("d,specs", [
    (128, [(1, 6, 300, 300, 300, 0), (1, 6, 700, 700, 300, 1), (2, 2, 1000, 100, 40, 0), (2, 2, 1000, 333, 40, 0),
           (2, 2, 1000, 1000, 40, 0), (1, 3, 520, 520, 520, 1), (1, 1, 77, 77, 1, 1)]),
    (64, [(2, 5, 1111, 1111, 200, 1), (1, 2, 129, 100, 600, 0), (3, 1, 2049, 2049, 129, 1)]),
    (128, [(1, 1, 64 + 8 * i, 64 + 8 * i, 30 + i, i % 2) for i in range(27)]),      # more than one launch's table
])
def test_batched_forward_every_problem_against_the_oracle(d, specs):
    """A table of independent problems of different shapes and masks as one launch (inner layers of a block, key
    prefixes of one sequence read in place): each problem equals the oracle, guard regions around every output stay
    untouched, and a problem that a call of its own would also run unsplit comes out bit-identical."""
    if not TC_AVAILABLE:
        pytest.skip("tensor path not built")
    problems, guards = _batched_case(d, specs, seed=900 + d)
    tl.tlin_attn_forward_batched(problems)
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0
    assert tl.tlin_last_launch_count() == -(-len(specs) // 24)
    for i, ((q, k, v, out, lse, n_keys, causal), (og, lg)) in enumerate(zip(problems, guards)):
        og.check(f"problem {i} out")
        lg.check(f"problem {i} lse")
        ks, vs = k[:, :, :n_keys].contiguous(), v[:, :, :n_keys].contiguous()
        ref, ref_lse = oracle.attn_forward(q.cpu(), ks.cpu(), vs.cpu(), causal)
        parity.check(out.float().cpu().numpy(), lse.cpu().numpy(), ref, ref_lse, "bf16", f"batched problem {i} {specs[i]}")
        B, H, W = q.shape[0], q.shape[1], q.shape[2]
        if tl.tlin_plan_forward(B, H, n_keys, W, d, causal).schedule == 1:
            single, single_lse = run_impl(2, tl.tlin_attn_forward, q, ks, vs, causal_window=causal)
            assert torch.equal(single, out) and torch.equal(single_lse, lse), f"problem {i}: differs from its own call"


def test_batched_forward_runs_a_sliding_window_pass_with_arbitrary_prefixes_in_one_launch():
    # Section 5.1: every chunk of W_og tokens attends to everything up to its own end; here as one table over one k, v
    if not TC_AVAILABLE:
        pytest.skip("tensor path not built")
    C, B, H, W, d = 6, 2, 3, 160, 128
    L = C * W
    wl = synth.Workload("chunks1", B, H, d, L, L, seed=47, causal_window=1)
    q_all, k, v = synth.forward_inputs(wl, device=DEV)
    q = q_all.view(B, H, C, W, d).permute(2, 0, 1, 3, 4).contiguous()
    out = torch.empty_like(q)
    lse = torch.empty((C, B, H, W), dtype=torch.float32, device=DEV)
    tl.tlin_attn_forward_batched([(q[c], k, v, out[c], lse[c], (c + 1) * W, 1) for c in range(C)])
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0 and tl.tlin_last_launch_count() == 1
    ref, ref_lse = oracle.attn_forward(q_all.cpu(), k.cpu(), v.cpu(), 1)         # plain causal attention over the whole sequence
    got = out.permute(1, 2, 0, 3, 4).reshape(B, H, L, d)
    parity.check(got.float().cpu().numpy(), lse.permute(1, 2, 0, 3).reshape(B, H, L).cpu().numpy(), ref, ref_lse, "bf16", "chunks in one launch")


def test_chunk_scheduled_forward_with_many_units_is_one_launch():
    # enough (chunk, b*h, query tile) problems to fill the SMs: the prefixes entry point issues all chunks as one table launch
    if not TC_AVAILABLE:
        pytest.skip("tensor path not built")
    C, B, H, W, d = 4, 2, 40, 200, 64
    L = C * W + 37                                   # the last chunk does not reach the end of k, v
    wl = synth.Workload("chunks_table", B, H, d, L, C * W, seed=49, causal_window=1)
    q_all, k, v = synth.forward_inputs(wl, device=DEV)
    q = q_all.view(B, H, C, W, d).permute(2, 0, 1, 3, 4).contiguous()
    n_keys = [(c + 1) * W for c in range(C)]
    out, lse = tl.tlin_attn_forward_prefixes(q, k, v, n_keys, causal_window=1)
    torch.cuda.synchronize()
    assert tl.tlin_get_status() == 0 and tl.tlin_last_launch_count() == 1
    for c in (0, C - 1):
        for (b, h) in ((0, 0), (B - 1, H - 1)):
            sl = lambda t: t[b:b + 1, h:h + 1].contiguous().cpu()
            ref, ref_lse = oracle.attn_forward(sl(q[c]), sl(k[:, :, :n_keys[c]]), sl(v[:, :, :n_keys[c]]), 1)
            parity.check(sl(out[c]).float().numpy(), sl(lse[c]).numpy(), ref, ref_lse, "bf16", f"chunk {c} head {(b, h)}")
    # every chunk equals its own call bit for bit when that call does not split the keys either
    for c in range(C):
        if tl.tlin_plan_forward(B, H, n_keys[c], W, d, 1).schedule == 1:
            o1, l1 = run_impl(2, tl.tlin_attn_forward, q[c], k[:, :, :n_keys[c]].contiguous(), v[:, :, :n_keys[c]].contiguous(), causal_window=1)
            assert torch.equal(o1, out[c]) and torch.equal(l1, lse[c])
