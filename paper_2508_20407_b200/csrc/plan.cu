// Host-side planning: pure integer arithmetic, no CUDA calls.  The paper does not schedule
// anything; what it fixes is the set of (query,key) pairs a call evaluates (Section 3, causal
// rule; Appendix A, cost terms), and every function here is tested against that count.
#include "tlin_internal.h"
#include <algorithm>
#include <vector>

using namespace tlin;

extern "C" int tlin_allowed(int64_t i, int64_t j, int64_t N, int64_t W, int causal_window) {
    if (i < 0 || i >= W || j < 0 || j >= N) return 0;
    if (causal_window) return j <= (N - W) + i ? 1 : 0;
    return 1;
}

extern "C" int tlin_tile_class(int64_t N, int64_t W, int causal_window, int tile_m, int tile_n, int qt, int kt) {
    if (tile_m <= 0 || tile_n <= 0 || qt < 0 || kt < 0) return 0;
    const int64_t i0 = (int64_t)qt * tile_m, j0 = (int64_t)kt * tile_n;
    if (i0 >= W || j0 >= N) return 0;
    const int64_t i1 = (i0 + tile_m < W ? i0 + tile_m : W) - 1;   // last query row of the tile
    const int64_t j1 = j0 + tile_n - 1;                           // last key column, may lie beyond N
    if (causal_window) {
        if (j0 > (N - W) + i1) return 0;                          // even the last row sees nothing
        if (j1 < N && j1 <= (N - W) + i0) return 1;               // even the first row sees everything
        return 2;
    }
    return j1 < N ? 1 : 2;
}

void tlin::fwd_group_starts(const tlin_fwd_plan& plan, GroupStarts* starts) {
    const int G = plan.n_groups;
    const long long U = plan.total_units;
    const bool by_cost = plan.schedule != 0 && plan.causal_window && plan.q_tiles > 1 && U >= 3LL * G;
    if (!by_cost) {
        for (int g = 0; g <= G; ++g) starts->u[g] = (long long)(((unsigned long long)g * (unsigned long long)U) / (unsigned)G);
        return;
    }
    // prefix[n] = cost of the first n problems of a (b,h)
    thread_local std::vector<long long> prefix;
    prefix.assign((size_t)plan.q_tiles + 1, 0);
    for (int qt = 0; qt < plan.q_tiles; ++qt)
        prefix[qt + 1] = prefix[qt] + fwd_problem_cost(plan.n_keys, plan.n_queries, plan.key_tiles, qt);
    const long long q = plan.q_tiles, n_bh = U / q, per_bh = prefix[q], total = per_bh * n_bh;
    long long biggest = 0;
    for (int qt = 0; qt < q; ++qt) biggest = std::max(biggest, prefix[qt + 1] - prefix[qt]);
    // The costs repeat with every (b,h): P(x) = cost of the first x problems, and its two inverses
    auto P = [&](long long x) { return (x / q) * per_bh + prefix[x % q]; };
    auto last_le = [&](long long v) {        // largest x <= U with P(x) <= v   (v >= 0)
        const long long bh = v / per_bh;
        if (bh >= n_bh) return U;
        return bh * q + ((std::upper_bound(prefix.begin(), prefix.end(), v - bh * per_bh) - prefix.begin()) - 1);
    };
    auto first_ge = [&](long long v) {       // smallest x >= 0 with P(x) >= v   (v <= total)
        if (v <= 0) return 0LL;
        const long long bh = v / per_bh;
        return bh * q + (long long)(std::lower_bound(prefix.begin(), prefix.end(), v - bh * per_bh) - prefix.begin());
    };
    auto proportional = [&](int g) {         // group g starts where the cost before it reaches g/G of the total
        return first_ge((long long)(((unsigned long long)g * (unsigned long long)total) / (unsigned)G));
    };
    starts->u[G] = U;
    if (per_bh < 10 * q) {
        // short problems (10 key-tile times on average, overheads included): the cost model is too coarse for more than
        // the proportional split (measured: the exact optimum below is 5-10 % slower at N = W = 1024, 3-8 % faster from 2048 on)
        for (int g = 0; g < G; ++g) starts->u[g] = proportional(g);
        return;
    }
    // G contiguous runs, none costlier than cap: possible iff filling every run to the brim reaches the end
    auto feasible = [&](long long cap) {
        long long pos = 0;
        for (int g = 0; g < G && pos < U; ++g) pos = last_le(P(pos) + cap);
        return pos >= U;
    };
    // the slowest CTA decides the kernel's time: smallest cap that works (between the mean and one problem above it)
    long long cap = std::max(biggest, (total + G - 1) / G), hi = (total + G - 1) / G + biggest;
    while (cap < hi) {
        const long long mid = (cap + hi) / 2;
        if (feasible(mid)) hi = mid; else cap = mid + 1;
    }
    // Among the splits that respect cap, stay as close as possible to the proportional one (group g starting where the cost
    // before it reaches g/G of the total), so that no CTA is left without work when it can be helped.  earliest[g]: first
    // problem group g may start at such that the groups from g on can still take the rest.
    long long earliest[kMaxGroups + 1];
    earliest[G] = U;
    for (int g = G - 1; g >= 0; --g) earliest[g] = first_ge(P(earliest[g + 1]) - cap);
    starts->u[0] = 0;
    for (int g = 0; g + 1 < G; ++g) {
        const long long from = starts->u[g];
        const long long lo = std::max(earliest[g + 1], from), up = last_le(P(from) + cap);
        starts->u[g + 1] = std::min(std::max(proportional(g + 1), lo), up);
    }
    starts->u[G] = U;
}

// Contiguous runs of units, one per CTA, every run non-empty: the costliest run as cheap as contiguous runs allow, and
// within that as close as possible to equal shares of the total (run c starting where the cost before it reaches
// c/n of the total).
void tlin::balanced_run_starts(const long long* prefix, long long U, int G, long long* starts) {
    const long long total = prefix[U];
    long long biggest = 0;
    for (long long x = 0; x < U; ++x) biggest = std::max(biggest, prefix[x + 1] - prefix[x]);
    auto last_le = [&](long long v) { return (long long)(std::upper_bound(prefix, prefix + U + 1, v) - prefix) - 1; };   // largest x with prefix[x] <= v
    auto first_ge = [&](long long v) { return (long long)(std::lower_bound(prefix, prefix + U + 1, v) - prefix); };       // smallest x with prefix[x] >= v
    auto feasible = [&](long long cap) {
        long long pos = 0;
        for (int g = 0; g < G && pos < U; ++g) pos = last_le(prefix[pos] + cap);
        return pos >= U;
    };
    long long cap = std::max(biggest, (total + G - 1) / G), hi = (total + G - 1) / G + biggest;
    while (cap < hi) {
        const long long mid = (cap + hi) / 2;
        if (feasible(mid)) hi = mid; else cap = mid + 1;
    }
    std::vector<long long> earliest((size_t)G + 1);
    earliest[G] = U;
    for (int g = G - 1; g >= 0; --g) earliest[g] = first_ge(prefix[earliest[g + 1]] - cap);
    starts[0] = 0;
    for (int g = 0; g + 1 < G; ++g) {
        const long long from = starts[g];
        const long long lo = std::max(earliest[g + 1], from), up = last_le(prefix[from] + cap);
        const long long want = first_ge((long long)(((unsigned long long)(g + 1) * (unsigned long long)total) / (unsigned)G));
        long long x = std::min(std::max(want, lo), up);
        // no run is empty (G <= U): at least one unit for this CTA, and one left for each of the CTAs after it
        x = std::max(x, from + 1);
        x = std::min(x, U - (G - 1 - g));
        starts[g + 1] = x;
    }
    starts[G] = U;
}

static int check_problem(const tlin_problem& pb) {
    if (!pb.q || !pb.k || !pb.v || !pb.out) return TLIN_ERR_INVALID_ARG;
    if (pb.BH <= 0 || pb.n_keys <= 0 || pb.n_queries <= 0) return TLIN_ERR_INVALID_ARG;
    if (pb.causal_window != 0 && pb.causal_window != 1) return TLIN_ERR_INVALID_ARG;
    if (pb.causal_window && pb.n_keys < pb.n_queries) return TLIN_ERR_INVALID_ARG;
    if (pb.kv_rows != 0 && pb.kv_rows < pb.n_keys) return TLIN_ERR_INVALID_ARG;
    const uintptr_t all = (uintptr_t)pb.q | (uintptr_t)pb.k | (uintptr_t)pb.v | (uintptr_t)pb.out;
    if (all & 15u) return TLIN_ERR_INVALID_ARG;
    if (pb.lse && ((uintptr_t)pb.lse & 3u)) return TLIN_ERR_INVALID_ARG;
    return TLIN_OK;
}

extern "C" int tlin_plan_batched(const tlin_problem* problems, int n_problems, int num_sms, int64_t* starts, int32_t* n_ctas) {
    if (!problems || !starts || !n_ctas || n_problems <= 0 || n_problems > kMaxBatch) return TLIN_ERR_INVALID_ARG;
    if (num_sms <= 0) num_sms = kDefaultSMs;
    if (num_sms > kMaxGroups) num_sms = kMaxGroups;
    std::vector<long long> prefix(1, 0);
    for (int i = 0; i < n_problems; ++i) {
        const tlin_problem& pb = problems[i];
        const int rc = check_problem(pb);
        if (rc != TLIN_OK) return rc;
        const int key_tiles = (pb.n_keys + kTileN - 1) / kTileN, q_tiles = (pb.n_queries + 255) / 256;
        if ((long long)pb.BH * pb.n_queries > 0x7fffffffLL) return TLIN_ERR_UNSUPPORTED;
        for (int bh = 0; bh < pb.BH; ++bh)
            for (int qt = 0; qt < q_tiles; ++qt)
                prefix.push_back(prefix.back() + (pb.causal_window ? fwd_problem_cost(pb.n_keys, pb.n_queries, key_tiles, qt) : key_tiles + 2));
    }
    const long long U = (long long)prefix.size() - 1;
    const int G = (int)std::min<long long>(num_sms, U);
    std::vector<long long> st((size_t)G + 1);
    balanced_run_starts(prefix.data(), U, G, st.data());
    for (int g = 0; g <= G; ++g) starts[g] = st[g];
    *n_ctas = G;
    return TLIN_OK;
}

extern "C" int64_t tlin_plan_group_start(const tlin_fwd_plan* plan, int g) {
    if (!plan || plan->n_groups <= 0) return 0;
    if (g <= 0) return 0;
    if (g >= plan->n_groups) return plan->total_units;
    if (!plan->tensor_path || plan->n_groups > kMaxGroups)      // CUDA-core path: one group per (b,h), equal counts
        return (int64_t)(((unsigned long long)g * (unsigned long long)plan->total_units) / (unsigned)plan->n_groups);
    GroupStarts starts;
    fwd_group_starts(*plan, &starts);
    return starts.u[g];
}

extern "C" int tlin_plan_forward(int B, int H, int N, int W, int d, int causal_window, int is_f32,
                                 int num_sms, tlin_fwd_plan* plan) {
    if (!plan) return TLIN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || N <= 0 || W <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    if (causal_window && N < W) return TLIN_ERR_INVALID_ARG;
    if (num_sms <= 0) num_sms = kDefaultSMs;
    const int impl = forward_impl();
    const bool tc_shape = !is_f32 && (d == 64 || d == 128);
    if (impl == 2 && !tc_shape) return TLIN_ERR_UNSUPPORTED;
    if (is_f32 ? (d % 4 != 0 || d > 256) : (d % 8 != 0 || d > 256)) return TLIN_ERR_UNSUPPORTED;
    const bool tc = tc_shape && impl != 1;
    tlin_fwd_plan p = {};
    const int64_t bh = (int64_t)B * H;
    p.tensor_path = tc ? 1 : 0;
    p.causal_window = causal_window;
    p.n_keys = N;
    p.n_queries = W;
    if (!tc) {
        p.tile_m = kSimtRows;
        p.tile_n = kSimtKeys;
        p.q_tiles = (W + p.tile_m - 1) / p.tile_m;
        p.key_tiles = (N + p.tile_n - 1) / p.tile_n;
        p.total_units = bh * p.key_tiles;
        p.n_groups = (int32_t)(bh < INT32_MAX ? bh : INT32_MAX);   // one group per (b,h): never split
        if ((int64_t)p.n_groups * p.q_tiles > INT32_MAX) return TLIN_ERR_UNSUPPORTED;
        p.n_ctas = p.n_groups * p.q_tiles;
        p.uses_workspace = 0;
        p.workspace_bytes = 0;
        *plan = p;
        return TLIN_OK;
    }
    if (num_sms > kMaxGroups) num_sms = kMaxGroups;   // size of the table of group starts handed to the kernels
    p.tile_m = 256;            // two 128-row Q tiles per CTA
    p.tile_n = kTileN;
    p.q_tiles = (W + p.tile_m - 1) / p.tile_m;
    p.key_tiles = (N + p.tile_n - 1) / p.tile_n;
    // Two ways to share the work out (both evaluate exactly the same (query,key) pairs):
    //   schedule 0: groups of q_tiles CTAs stream ranges of (b,h,key tile) units; a (b,h) may be split between
    //               groups, whose partial results a second kernel merges.  Fills the SMs however few (b,h) there are,
    //               and the CTAs of a group read each K/V tile at the same time (once from HBM).
    //   schedule 1: every CTA works through whole (b,h,query tile) problems; no split, no merge, but a K/V tile
    //               is read by the q_tiles problems of its (b,h) at unrelated times, so K and V have to stay in L2.
    // Costs in key-tile times per CTA; the constants (merge pass ~ 6 tiles, start/finish of a problem ~ 2 tiles)
    // are measured on B200.
    bool wide = false;
    {
        int64_t groups0 = num_sms / p.q_tiles;
        if (groups0 < 1) groups0 = 1;
        if (groups0 > bh * p.key_tiles) groups0 = bh * p.key_tiles;
        const int64_t waves0 = (p.q_tiles + num_sms - 1) / num_sms;              // > 1 only if q_tiles exceeds the SMs
        const int64_t per_group = (bh * p.key_tiles + groups0 - 1) / groups0;
        const bool splits0 = (bh * p.key_tiles) % groups0 != 0 || (bh * p.key_tiles / groups0) % p.key_tiles != 0;
        const int64_t segments0 = per_group / p.key_tiles + 1;                   // (b,h) pieces a group walks through
        const int64_t cost0 = waves0 * (per_group + 2 * segments0) + (splits0 ? 6 : 0);
        const int64_t problems = bh * p.q_tiles;
        const int64_t ctas1 = num_sms < problems ? num_sms : problems;
        const int64_t kv_bytes = 2 * bh * (int64_t)N * d * 2;
        const bool kv_in_l2 = p.q_tiles == 1 || kv_bytes <= (int64_t)64 << 20;
        int64_t cost1 = ((problems + ctas1 - 1) / ctas1) * ((int64_t)p.key_tiles + 2);
        bool allow1 = kv_in_l2;
        if (causal_window && p.q_tiles > 1) {
            // With the window rule a problem only needs the key tiles its rows may use, and under schedule 0 the CTAs of
            // the early query tiles would idle while the last one finishes.  Problems are shared by cost (the same
            // arithmetic as the kernel's); an indivisible problem can leave a CTA half its cost above the mean.  When K and
            // V exceed L2 the tiles come from HBM at unrelated times: measured about 15 % slower per tile.
            int64_t per_bh = 0, biggest = 0;
            for (int qt = 0; qt < p.q_tiles; ++qt) {
                const int64_t c = fwd_problem_cost(N, W, p.key_tiles, qt);
                per_bh += c;
                if (c > biggest) biggest = c;
            }
            cost1 = (per_bh * bh + ctas1 - 1) / ctas1 + (problems > ctas1 ? biggest / 2 : 0);
            if (cost1 < biggest) cost1 = biggest;
            if (!kv_in_l2) cost1 += cost1 * 15 / 100;
            allow1 = true;
        }
        wide = allow1 && cost1 < cost0;
    }
    if (wide) {
        p.schedule = 1;
        p.total_units = bh * p.q_tiles;
        if (p.total_units > INT32_MAX) return TLIN_ERR_UNSUPPORTED;
        int64_t ctas = num_sms < p.total_units ? num_sms : p.total_units;
        p.n_groups = (int32_t)ctas;
        p.n_ctas = (int32_t)ctas;
        p.uses_workspace = 0;
        p.workspace_bytes = 0;
        *plan = p;
        return TLIN_OK;
    }
    p.total_units = bh * p.key_tiles;
    int64_t groups = num_sms / p.q_tiles;
    if (groups < 1) groups = 1;
    if (groups > p.total_units) groups = p.total_units;
    p.n_groups = (int32_t)groups;
    p.n_ctas = p.n_groups * p.q_tiles;
    p.uses_workspace = 0;
    GroupStarts starts;
    fwd_group_starts(p, &starts);
    for (int g = 1; g < p.n_groups; ++g)
        if (starts.u[g] % p.key_tiles != 0) { p.uses_workspace = 1; break; }
    // two partial slots per CTA (first and last segment of its unit range), each tile_m x (d + 1) floats
    p.workspace_bytes = p.uses_workspace ? (int64_t)p.n_ctas * 2 * p.tile_m * (d + 1) * (int64_t)sizeof(float) : 0;
    *plan = p;
    return TLIN_OK;
}

extern "C" int tlin_plan_decode(int B, int H, int L, int d, int num_sms, tlin_decode_plan* plan) {
    if (!plan) return TLIN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || L <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    if (num_sms <= 0) num_sms = kDefaultSMs;
    const int64_t bh = (int64_t)B * H;
    const int64_t slots = (int64_t)num_sms * kDecodeCtasPerSM;
    int max_s = (L + kDecodeMinKeys - 1) / kDecodeMinKeys;
    if (max_s > kDecodeMaxSplits) max_s = kDecodeMaxSplits;
    if (max_s < 1) max_s = 1;
    int best_s = 1;
    int64_t best_cost = -1;
    for (int s = 1; s <= max_s; ++s) {
        int64_t kps = (L + s - 1) / s;
        kps = (kps + 7) / 8 * 8;
        const int64_t waves = (bh * s + slots - 1) / slots;
        const int64_t cost = waves * (kps + 64);   // + a fixed per-CTA overhead, in keys
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_s = s; }
    }
    tlin_decode_plan p = {};
    int64_t kps = (L + best_s - 1) / best_s;
    kps = (kps + 7) / 8 * 8;
    p.keys_per_split = (int32_t)kps;
    p.splits = (int32_t)((L + kps - 1) / kps);     // drop splits that rounding left empty
    if (bh * p.splits > INT32_MAX) return TLIN_ERR_UNSUPPORTED;
    p.n_ctas = (int32_t)(bh * p.splits);
    p.workspace_bytes = bh * kDecodeMaxSplits * (int64_t)(d + 1) * (int64_t)sizeof(float);
    *plan = p;
    return TLIN_OK;
}

extern "C" size_t tlin_workspace_bytes_forward(int B, int H, int N, int W, int d, int causal_window) {
    tlin_fwd_plan p;
    if (tlin_plan_forward(B, H, N, W, d, causal_window, 0, 0, &p) != TLIN_OK) return 0;
    // sized for a 148-SM part; a device with another SM count is re-planned and re-checked at call time
    return (size_t)p.workspace_bytes;
}

extern "C" size_t tlin_workspace_bytes_decode(int B, int H, int Ncap, int d) {
    tlin_decode_plan p;
    if (tlin_plan_decode(B, H, Ncap > 0 ? Ncap : 1, d, 0, &p) != TLIN_OK) return 0;
    return (size_t)p.workspace_bytes;
}

extern "C" int64_t tlin_plan_backward_share_start(int B, int H, int N, int W, int causal_window, int share, int n_shares) {
    if (B <= 0 || H <= 0 || N <= 0 || W <= 0 || n_shares <= 0 || share < 0) return -1;
    if (causal_window && N < W) return -1;
    const int key_tiles = (N + kTileN - 1) / kTileN;
    return tlin::bwd_first_unit_of_share(N, W, causal_window, (long long)B * H * key_tiles, key_tiles, (unsigned)share, (unsigned)n_shares);
}
