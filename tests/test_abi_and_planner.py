"""CPU-side tests of the C-ABI library: it loads without a GPU, exports every symbol the header
declares, rejects bad arguments before touching a device, and its integer planning is exact."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import cost_model
from paper_2508_20407_b200 import binding as tl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "tlin.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(tlin_[a-z0-9_]+)\s*\(", header))
    assert len(declared) >= 18
    raw = ctypes.CDLL(tl.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), f"{name} is declared in tlin.h but not exported"
    assert declared == set(tl.SIGNATURES), declared ^ set(tl.SIGNATURES)


def test_version_and_status_strings():
    assert "sm_100a" in tl.version()
    assert tl.status_string(0) == "ok"
    for s in range(-6, 0):
        assert tl.status_string(s) not in ("ok", "unknown status")


def test_argument_errors_are_found_on_the_host():
    L = tl.lib()
    one = ctypes.c_void_p(16)  # aligned, never dereferenced: every call below fails validation first
    odd = ctypes.c_void_p(24 + 2)
    fwd = lambda *a: L.tlin_attn_forward(*a, None)
    assert fwd(None, one, one, one, one, 1, 1, 8, 4, 64, 1) == tl.ERR_INVALID_ARG
    assert fwd(one, one, one, one, one, 0, 1, 8, 4, 64, 1) == tl.ERR_INVALID_ARG
    assert fwd(one, one, one, one, one, 1, 1, 4, 8, 64, 1) == tl.ERR_INVALID_ARG      # N < W with a window
    assert fwd(odd, one, one, one, one, 1, 1, 8, 4, 64, 1) == tl.ERR_INVALID_ARG      # misaligned
    assert fwd(one, one, one, one, one, 1, 1, 8, 4, 64, 2) == tl.ERR_INVALID_ARG      # causal flag
    assert fwd(one, one, one, one, one, 1, 1, 8, 4, 36, 1) == tl.ERR_UNSUPPORTED      # bf16 path needs d % 8 == 0
    assert L.tlin_attn_forward_f32(one, one, one, one, one, 1, 1, 8, 4, 258, 1, None) == tl.ERR_UNSUPPORTED
    dec = lambda *a: L.tlin_decode_step(*a, None)
    assert dec(one, one, one, one, one, one, one, 1, 1, 8, -1, 64) == tl.ERR_INVALID_ARG
    assert dec(one, one, one, one, one, one, one, 1, 1, 8, 8, 64) == tl.ERR_INVALID_ARG
    assert dec(one, one, one, one, one, one, one, 1, 1, 8, 3, 48) == tl.ERR_UNSUPPORTED
    assert L.tlin_set_workspace(None, 16) == tl.ERR_INVALID_ARG
    assert L.tlin_set_forward_impl(7) == tl.ERR_INVALID_ARG


def test_mask_predicate_matches_the_causal_rule_bit_for_bit():
    for N in range(1, 10):
        for W in range(1, N + 1):
            for i in range(W):
                for j in range(-1, N + 1):
                    assert tl.tlin_allowed(i, j, N, W, 1) == int(0 <= j < N and j <= N - W + i)
                    assert tl.tlin_allowed(i, j, N, W, 0) == int(0 <= j < N)


@pytest.mark.parametrize("N,W,causal,tm,tn", [(1000, 300, 1, 128, 128), (512, 512, 1, 128, 128), (777, 130, 0, 128, 128),
                                              (1024, 128, 1, 128, 128), (300, 7, 1, 8, 32), (4096, 256, 1, 256, 128)])
def test_tile_classes_against_brute_force_and_pair_count(N, W, causal, tm, tn):
    i = np.arange(W)[:, None]
    j = np.arange(((N + tn - 1) // tn) * tn)[None, :]
    allowed = (j < N) & ((j <= N - W + i) if causal else (i >= 0))
    total = 0
    for qt in range((W + tm - 1) // tm):
        for kt in range((N + tn - 1) // tn):
            blk = allowed[qt * tm:(qt + 1) * tm, kt * tn:(kt + 1) * tn]
            cls = tl.tlin_tile_class(N, W, causal, tm, tn, qt, kt)
            if cls == 0:
                assert not blk.any()
            elif cls == 1:
                assert blk.all() and blk.shape[1] == tn
            else:
                assert cls == 2 and blk.any() and not (blk.all() and blk.shape[1] == tn)
            if cls:
                total += int(blk.sum())
    # the pairs the planned tiles cover are exactly the pairs the method evaluates
    assert total == cost_model.allowed_pairs(N, W, causal)


CONFIGS = [(1, 4, 1024, 128, 64, 1), (4, 16, 8192, 256, 64, 1), (1, 32, 32768, 512, 128, 1),
           (1, 32, 131072, 1024, 128, 1), (3, 5, 1000, 77, 128, 0), (1, 1, 100, 100, 64, 1), (2, 2, 129, 1, 64, 1)]


def _plan_tc(B, H, N, W, d, causal):
    prev = tl.tlin_set_forward_impl(2)
    try:
        return tl.tlin_plan_forward(B, H, N, W, d, causal, num_sms=148)
    finally:
        tl.tlin_set_forward_impl(prev)


def _check_plan(p, B, H, N, W, d, causal):
    """Whatever the schedule, the groups partition the units and so cover every (query tile, key tile) once."""
    assert p.tensor_path == 1 and p.tile_n == 128 and p.schedule in (0, 1)
    assert p.q_tiles == -(-W // p.tile_m) and p.key_tiles == -(-N // p.tile_n)
    starts = [tl.tlin_plan_group_start(p, g) for g in range(p.n_groups + 1)]
    assert starts[0] == 0 and starts[-1] == p.total_units
    sizes = np.diff(starts)
    by_cost = p.schedule == 1 and causal and p.q_tiles > 1 and p.total_units >= 3 * p.n_groups
    if by_cost:
        # window rule, whole problems per CTA: problem qt may use ceil((N-W+min(W,256(qt+1)))/128) key tiles; the groups take
        # contiguous runs of problems, and the costliest run (cost = tiles + 3 per problem) must be the optimum over all ways
        # of cutting the list into n_groups runs, found here by bisection over a plain greedy pass
        cost = [min(p.key_tiles, -(-(N - W + min(W, 256 * (qt + 1))) // 128)) + 3 for qt in range(p.q_tiles)]
        all_costs = cost * (p.total_units // p.q_tiles)
        loads = [sum(all_costs[a:b]) for a, b in zip(starts, starts[1:])]

        def runs_needed(cap):
            n, cur = 1, 0
            for c in all_costs:
                if cur + c > cap:
                    n, cur = n + 1, c
                else:
                    cur += c
            return n

        lo, hi = max(cost), sum(all_costs)
        while lo < hi:
            mid = (lo + hi) // 2
            lo, hi = (lo, mid) if runs_needed(mid) <= p.n_groups else (mid + 1, hi)
        mean = sum(all_costs) / p.n_groups
        assert (sizes >= 0).all() and lo <= mean + max(cost)
        if sum(cost) >= 10 * p.q_tiles:
            assert max(loads) == lo and min(loads) > 0
        else:       # short problems: every group starts where the cost before it reaches its share of the total
            assert max(loads) <= mean + max(cost) and min(loads) >= mean - max(cost)
    else:
        assert (sizes >= 1).all() and sizes.max() - sizes.min() <= 1
    if p.schedule == 0:
        # unit = (b,h,key tile); a group is q_tiles CTAs (one per pair of query tiles) walking the same units
        assert p.total_units == B * H * p.key_tiles
        assert 1 <= p.n_groups <= p.total_units and p.n_ctas == p.n_groups * p.q_tiles
        assert p.n_ctas <= 148 or p.n_groups == 1
        split = any(s % p.key_tiles for s in starts[1:-1])
        assert bool(p.uses_workspace) == split
        assert p.workspace_bytes == (p.n_ctas * 2 * p.tile_m * (d + 1) * 4 if split else 0)
        covered = int(sizes.sum()) * p.q_tiles
    else:
        # unit = whole (b,h,query tile pair) problem: all its key tiles, never split, nothing to merge
        assert p.total_units == B * H * p.q_tiles
        assert p.n_ctas == p.n_groups == min(148, p.total_units)
        assert p.uses_workspace == 0 and p.workspace_bytes == 0
        covered = int(sizes.sum()) * p.key_tiles
    assert covered == B * H * p.q_tiles * p.key_tiles


@pytest.mark.parametrize("B,H,N,W,d,causal", CONFIGS)
def test_forward_plan_partitions_the_units(B, H, N, W, d, causal):
    p = _plan_tc(B, H, N, W, d, causal)
    _check_plan(p, B, H, N, W, d, causal)
    if N >= 8192:
        # few query rows over a long context (focused attention, generation window): key ranges are split
        assert p.schedule == 0 and p.n_ctas == 148
    assert tl.workspace_bytes_forward(B, H, N, W, d, causal) in (0, p.workspace_bytes) or tl.tlin_set_forward_impl(0) == 0


WIDE = [(1, 32, 1024, 130048, 128, 0), (1, 32, 512, 32256, 128, 0), (2, 3, 300, 40000, 64, 0), (8, 16, 1024, 1024, 64, 1),
        (1, 32, 1024, 1024, 128, 0), (1, 32, 2048, 1024, 128, 1),
        # plain causal attention over whole sequences: problems of very different cost, shared between the CTAs by cost
        (4, 32, 4096, 4096, 128, 1), (1, 32, 8192, 8192, 128, 1), (1, 8, 16384, 16384, 128, 1), (2, 40, 1600, 1500, 128, 1),
        (3, 50, 900, 900, 64, 1), (4, 32, 4096, 2048, 128, 1)]


@pytest.mark.parametrize("B,H,N,W,d,causal", WIDE)
def test_forward_plan_many_queries_few_keys(B, H, N, W, d, causal):
    """Restoring cross-attention and the inner layers (Section 3): many (b,h,query tile) problems over a short
    key range go to the CTAs whole; the evaluated pairs are unchanged (Appendix A: D*(N-W_og)*W_oh)."""
    p = _plan_tc(B, H, N, W, d, causal)
    _check_plan(p, B, H, N, W, d, causal)
    assert p.schedule == 1


def test_forward_plan_keeps_key_splitting_when_kv_exceed_l2():
    """Whole problems per CTA would read every K/V tile q_tiles times from HBM once K and V no longer fit in L2."""
    p = _plan_tc(1, 64, 16384, 1024, 128, 1)        # 512 MB of K and V
    assert p.schedule == 0


def test_forward_plan_fallback_path_never_splits():
    p = tl.tlin_plan_forward(2, 3, 500, 50, 36, 1, is_f32=True)
    assert p.tensor_path == 0 and p.uses_workspace == 0 and p.workspace_bytes == 0
    assert p.tile_m == 8 and p.n_ctas == 6 * 7


@pytest.mark.parametrize("B,H,L,d", [(8, 32, 65537, 128), (8, 32, 65792, 128), (1, 1, 1, 64), (1, 4, 300, 64),
                                     (2, 2, 100000, 128), (64, 32, 4096, 128)])
def test_decode_plan_covers_every_key_once(B, H, L, d):
    p = tl.tlin_plan_decode(B, H, L, d, 148)
    assert 1 <= p.splits <= 64 and p.keys_per_split % 8 == 0
    assert p.n_ctas == B * H * p.splits
    covered = 0
    for s in range(p.splits):
        lo, hi = s * p.keys_per_split, min(L, (s + 1) * p.keys_per_split)
        assert hi > lo
        covered += hi - lo
    assert covered == L
    assert p.workspace_bytes == B * H * 64 * (d + 1) * 4 == tl.workspace_bytes_decode(B, H, max(L, 1), d)
    if L >= 2 * 256:
        assert p.keys_per_split >= 256


def test_decode_plan_balances_the_benchmark_shape():
    p = tl.tlin_plan_decode(8, 32, 65537, 128, 148)
    waves = -(-p.n_ctas // 296)
    ideal = 65537 * 256 / 296
    assert waves * p.keys_per_split <= 1.05 * ideal


def test_backward_workspace_covers_row_statistics_and_partial_sums():
    # host arithmetic only: 2 floats per padded query row (lse*log2e, delta) plus, when the key range of a (b,h) is split
    # between groups, two 256 x d fp32 slots per CTA of the dQ kernel; never less than the CUDA-core path's needs
    # (one float per row + an fp32 dQ accumulator)
    for B, H, N, W, d in [(1, 32, 131072, 1024, 128), (4, 32, 8192, 1024, 128), (4, 16, 8192, 256, 64), (1, 1, 1, 1, 64), (2, 3, 1000, 300, 128)]:
        got = tl.workspace_bytes_backward(B, H, N, W, d)
        rows = B * H * W
        simt = 4 * ((rows + 3) // 4 * 4 + rows * d)
        wpad = (W + 127) // 128 * 128
        need = simt
        for causal in (0, 1):
            if causal and N < W:
                continue
            plan = tl.tlin_plan_forward(B, H, N, W, d, causal)
            tc = 4 * (2 * B * H * wpad + (plan.n_ctas * 2 * 256 * d if plan.uses_workspace else 0))
            need = max(need, tc)
        if d == 128:        # the one-kernel arrangement: row statistics plus an fp32 dQ buffer on padded rows
            need = max(need, 4 * B * H * wpad * (d + 2))
        assert got == need, (B, H, N, W, d, got, need)
    assert tl.workspace_bytes_backward(0, 1, 1, 1, 64) == 0


def test_prefix_workspace_is_the_largest_of_the_chunks():
    import ctypes
    B, H, W, d = 1, 8, 512, 128
    n_keys = [512, 4096, 32768, 65536]
    arr = (ctypes.c_int32 * len(n_keys))(*n_keys)
    for causal in (0, 1):
        got = int(tl.lib().tlin_workspace_bytes_forward_prefixes(B, H, W, d, len(n_keys), arr, causal))
        assert got == max(tl.workspace_bytes_forward(B, H, n, W, d, causal) for n in n_keys)
    assert int(tl.lib().tlin_workspace_bytes_forward_prefixes(B, H, W, d, 0, arr, 1)) == 0


def test_backward_key_tile_shares_cover_everything_and_balance_the_steps():
    import random
    L = tl.lib()
    rnd = random.Random(3)
    cases = [(1, 32, 32768, 512, 1), (4, 32, 8192, 1024, 1), (2, 3, 1024, 1024, 1), (1, 1, 1, 1, 1), (2, 5, 4000, 700, 0)]
    cases += [(rnd.randint(1, 3), rnd.randint(1, 9), 0, rnd.randint(1, 1500), 1) for _ in range(40)]
    for B, H, N, W, causal in cases:
        if N == 0:
            N = W + rnd.choice([0, 1, 127, 128, 129, rnd.randint(0, 5000)])
        T, Qt = (N + 127) // 128, (W + 127) // 128
        total = B * H * T
        G = min(total, 148)
        starts = [L.tlin_plan_backward_share_start(B, H, N, W, causal, c, G) for c in range(G + 1)]
        assert starts[0] == 0 and starts[-1] == total
        assert all(a <= b for a, b in zip(starts, starts[1:]))                 # contiguous, disjoint, complete

        def steps(u):                                                          # query tiles key tile u % T has to visit
            f = (u % T) * 128 - (N - W)
            return Qt - (0 if (not causal or f <= 0) else f // 128)
        loads = [sum(steps(u) for u in range(a, b)) for a, b in zip(starts, starts[1:])]
        assert all(steps(u) >= 1 for u in range(min(total, 2 * T)))
        mean = sum(loads) / G
        assert max(loads) <= mean + Qt and min(loads) >= mean - Qt             # within one key tile's full cost of the mean
    assert L.tlin_plan_backward_share_start(1, 1, 10, 20, 1, 0, 4) == -1       # N < W with the window rule


def _problem_array(specs):
    """ctypes Problem array from (BH, n_keys, n_queries, causal) with dummy aligned pointers (never dereferenced)."""
    arr = (tl.Problem * len(specs))()
    for i, (bh, n, w, causal) in enumerate(specs):
        arr[i] = tl.Problem(16, 32, 48, 64, None, bh, n, 0, w, causal, 0)
    return arr


def _unit_costs(specs):
    costs = []
    for (bh, n, w, causal) in specs:
        key_tiles, q_tiles = -(-n // 128), -(-w // 256)
        per_qt = []
        for qt in range(q_tiles):
            if causal:
                rows_end = min(w, (qt + 1) * 256)
                per_qt.append(min(key_tiles, -(-(n - w + rows_end) // 128)) + 3)
            else:
                per_qt.append(key_tiles + 2)
        costs.extend(per_qt * bh)
    return costs


@pytest.mark.parametrize("specs", [
    [(32, 1024, 1024, 0), (32, 2048, 1024, 1)],                     # an inner context layer and an inner generation layer
    [(3, 100, 40, 0), (3, 333, 40, 0), (3, 1000, 40, 0)],            # three key prefixes of one sequence
    [(1, 128, 128, 1)],                                               # a single unit
    [(8, 4096, 4096, 1), (2, 300, 5000, 0), (40, 64, 64, 1)],         # very uneven units
    [(1, 256, 256, 1)] * 24,
])
def test_batched_plan_gives_every_cta_a_contiguous_non_empty_run_with_the_cheapest_possible_maximum(specs):
    costs = _unit_costs(specs)
    U = len(costs)
    starts = tl.tlin_plan_batched(_problem_array(specs))
    G = len(starts) - 1
    assert G == min(148, U) and starts[0] == 0 and starts[-1] == U
    assert all(b > a for a, b in zip(starts, starts[1:]))
    runs = [sum(costs[a:b]) for a, b in zip(starts, starts[1:])]
    # the cheapest possible maximum over all splits into G contiguous non-empty runs, by bisection with a greedy check
    def fits(cap):
        g, acc = 1, 0
        for c in costs:
            if c > cap:
                return False
            if acc + c > cap:
                g, acc = g + 1, 0
            acc += c
        return g <= G
    lo, hi = max(costs), sum(costs)
    while lo < hi:
        mid = (lo + hi) // 2
        lo, hi = (lo, mid) if fits(mid) else (mid + 1, hi)
    assert max(runs) == lo


def test_batched_plan_rejects_bad_problems_on_the_host():
    L = tl.lib()
    out = (ctypes.c_int64 * 200)()
    n = ctypes.c_int32()
    call = lambda arr, count: L.tlin_plan_batched(ctypes.cast(arr, ctypes.c_void_p), count, 0, ctypes.cast(out, ctypes.c_void_p),
                                                  ctypes.cast(ctypes.pointer(n), ctypes.c_void_p))
    ok = _problem_array([(2, 300, 100, 1)])
    assert call(ok, 1) == 0
    assert call(ok, 0) == tl.ERR_INVALID_ARG
    assert call(_problem_array([(2, 50, 100, 1)]), 1) == tl.ERR_INVALID_ARG          # window rule with N < W
    assert call(_problem_array([(0, 300, 100, 0)]), 1) == tl.ERR_INVALID_ARG
    bad = _problem_array([(2, 300, 100, 0)])
    bad[0].kv_rows = 200                                                             # allocation smaller than the keys used
    assert call(bad, 1) == tl.ERR_INVALID_ARG
    bad = _problem_array([(2, 300, 100, 0)])
    bad[0].q = 24                                                                    # misaligned
    assert call(bad, 1) == tl.ERR_INVALID_ARG
    assert call(_problem_array([(1, 128, 128, 0)] * 25), 25) == tl.ERR_INVALID_ARG    # more than one launch's table
    assert L.tlin_attn_forward_batched(ctypes.cast(ok, ctypes.c_void_p), 1, 36, None) == tl.ERR_UNSUPPORTED
    assert L.tlin_attn_forward_batched(None, 1, 64, None) == tl.ERR_INVALID_ARG
    assert L.tlin_attn_forward_cache(ctypes.c_void_p(16), ctypes.c_void_p(16), ctypes.c_void_p(16), ctypes.c_void_p(16), None,
                                     1, 1, 100, 101, 8, 64, 0, None) == tl.ERR_INVALID_ARG
