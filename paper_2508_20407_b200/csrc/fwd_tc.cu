// Tensor-core forward kernel for sm_100a: exact softmax attention of W queries over N keys
// (Section 3 attention formula; causal rule j <= N-W+i inside the window), bf16 in, fp32 accumulate.
//
// One CTA owns 256 query rows of one (b,h) (two 128-row Q tiles) and streams a contiguous range of
// 128-key tiles.  K and V tiles arrive by TMA (128-byte swizzle) into a shared-memory ring; one thread
// issues tcgen05.mma: S_i = Q_i K_j^T into TMEM, then O_i += P_i V_j with P_i read from TMEM and V_j
// as an MN-major shared-memory operand.  Two softmax warpgroups (one per Q tile, one thread per row)
// read a whole row of S_i from TMEM into registers once, keep a running max / sum in base-2 units, write
// P_i (bf16) over S_i, and rescale O_i only when the running max has grown by more than 2^32 (the final
// O/l is exact either way).  A fixed share of the exponentials is evaluated by a cubic on the FMA pipe,
// the rest by the special-function unit, so that neither pipe alone bounds the softmax.
// While one warpgroup does its exponentials the tensor pipe works on the other Q tile.
//
// CTAs are numbered group*q_tiles + q_tile: the q_tiles CTAs of a group walk the same (b,h,key-tile)
// units at the same time, so K/V tiles are fetched from HBM once and re-read from L2.  A group's unit
// range may start or end in the middle of a (b,h); such partial results (normalised o, lse) go to the
// workspace and fwd_merge_kernel combines them with log-sum-exp weights.
//
// Every wait is bounded: on expiry the CTA sets the library's error word, drains and exits.
#include "tlin_internal.h"
#include "sm100_ptx.cuh"
#include "tc_common.cuh"
#include <math_constants.h>
#include <mutex>
#include <string.h>

namespace tlin {
namespace {

using namespace ptx;
using namespace tc;

constexpr int kProducerWarp = 8;
constexpr int kMmaWarp = 9;
constexpr int kThreads = 32 * 12;          // warps 10 and 11 only lend their registers
constexpr int kSoftmaxRegs = 216, kOtherRegs = 72;   // 256*224 + 128*56 = 384*168 registers
// an increase beyond what the other warpgroup released would wait for ever
static_assert(256 * kSoftmaxRegs + 128 * kOtherRegs <= kThreads * 168, "register budget of the CTA exceeded");
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kPolyPairs = 5;                // of every 16 column pairs, this many get 2^x from the polynomial
constexpr float kRescaleThreshold = 32.0f;  // base-2 units: P stays below 2^32, far inside bf16/fp32 range

// 2^x for a packed pair without the special-function unit: x = n + f with n = floor(x) (taken by adding
// 1.5*2^23 rounding down, which leaves n in the low mantissa bits), 2^f on [0,1) by a cubic fitted for
// minimum relative error (7.9e-5, well below the 2^-9 rounding of P to bf16), n added into the exponent field.
// x is clamped to [-126, inf) first; values the caller produces stay far below the upper exponent limit.
__device__ __forceinline__ void exp2_poly2(uint64_t x2, float& p0, float& p1) {
    float x0, x1;
    f2_unpack(x2, x0, x1);
    x0 = fmaxf(x0, -126.f);
    x1 = fmaxf(x1, -126.f);
    const uint64_t xc = f2_pack(x0, x1);
    const uint64_t magic = f2_pack(12582912.f, 12582912.f);
    const uint64_t xf = f2_add_rm(xc, magic);
    const uint64_t fr = f2_sub(xc, f2_sub(xf, magic));
    uint64_t y = f2_fma(f2_pack(0.07806939631700516f, 0.07806939631700516f), fr, f2_pack(0.22593535482883453f, 0.22593535482883453f));
    y = f2_fma(y, fr, f2_pack(0.6959162950515747f, 0.6959162950515747f));
    y = f2_fma(y, fr, f2_pack(0.9999210238456726f, 0.9999210238456726f));
    uint32_t n0, n1, y0, y1;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(n0), "=r"(n1) : "l"(xf));
    asm("mov.b64 {%0, %1}, %2;" : "=r"(y0), "=r"(y1) : "l"(y));
    p0 = __uint_as_float(y0 + (n0 << 23));
    p1 = __uint_as_float(y1 + (n1 << 23));
}

template <int D>
struct Cfg {
    static constexpr int kTileBytes = kQTile * D * 2;          // one 128-row tile of Q, K or V
    static constexpr int kBoxes = D / 64;                      // 64-element (128-byte) column blocks per tile
    static constexpr int kSlots = D == 128 ? 4 : 8;            // K/V ring slots
    static constexpr int kSmemTiles = (2 + kSlots) * kTileBytes;
    static constexpr int kStageBytes = 8 * 32 * 128;           // per softmax warp 32 rows x 128 bytes: result rows on their way out
    static constexpr int kNumBars = 10 + 2 * kSlots;
    static constexpr int kSmemBytes = kSmemTiles + kStageBytes + kNumBars * 8 + 16 + 1024;   // + alignment slack
    // TMEM columns: S0, S1 (128 each), O0, O1 (D each)
    static constexpr uint32_t kColS = 0, kColO = 256;
};

// One problem of a batched launch as the kernel sees it (the field names N, W, causal, key_tiles are the ones the
// helpers shared with the single-problem kernel read).
struct ProblemDev {
    void* out;            // [BH, W, D] bf16
    float* lse;           // [BH, W] or null
    long long unit0;      // first unit of this problem in the launch's list: unit = unit0 + bh * q_tiles + q tile pair
    int N, W, causal, key_tiles, q_tiles;
};
// What a launch reads its tensors through: three tensor maps, or a table of them with the problems' shapes.
template <bool kBatched> struct KernelMaps;
template <> struct KernelMaps<false> { CUtensorMap q, k, v; };
template <> struct KernelMaps<true> {
    CUtensorMap q[kMaxBatch], k[kMaxBatch], v[kMaxBatch];
    ProblemDev prob[kMaxBatch];
    int n;
};

struct Params {
    void* out;            // [B*H, W, D] bf16
    float* lse;           // [B*H, W] or null
    float* ws;            // partial slots
    int* status;
    long long total_units;
    int n_groups, q_tiles, key_tiles;
    int N, W, causal;
    int schedule;         // 0: groups of q_tiles CTAs stream key ranges; 1: every CTA walks whole (b,h,q-tile) problems
    float scale_log2e;
};

// Walks the units of a batched launch: whole problems, in table order.
struct BatchWalker {
    long long u, u1;
    const ProblemDev* prob;
    int n, pi;
    __device__ BatchWalker(const KernelMaps<true>& m, const GroupStarts& starts)
        : u(starts.u[blockIdx.x]), u1(starts.u[blockIdx.x + 1]), prob(m.prob), n(m.n), pi(0) {}
    __device__ bool next(Segment& s) {
        if (u >= u1) return false;
        while (pi + 1 < n && u >= prob[pi + 1].unit0) ++pi;
        const long long r = u - prob[pi].unit0;
        s.bh = (int)(r / prob[pi].q_tiles);
        s.qt = (int)(r - (long long)s.bh * prob[pi].q_tiles);
        s.t_begin = 0;
        s.t_end = prob[pi].key_tiles;
        s.prob = pi;
        ++u;
        return true;
    }
};
template <bool kBatched>
__device__ __forceinline__ auto make_walker(const KernelMaps<kBatched>& m, const Params& p, const GroupStarts& starts) {
    if constexpr (kBatched) return BatchWalker(m, starts);
    else return SegmentWalker(p, starts);
}
// shape (N, W, causal, key_tiles) and result pointers of the problem a segment belongs to
template <bool kBatched>
__device__ __forceinline__ decltype(auto) problem_of(const KernelMaps<kBatched>& m, const Params& p, const Segment& s) {
    if constexpr (kBatched) return (m.prob[s.prob]);
    else return (p);
}

template <int D, bool kBatched>
__global__ void __launch_bounds__(kThreads, 1)
fwd_tc_kernel(const __grid_constant__ KernelMaps<kBatched> maps, const __grid_constant__ Params p,
              const __grid_constant__ GroupStarts starts) {
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem;                               // 2 tiles
    uint8_t* sRing = smem + 2 * C::kTileBytes;        // kSlots tiles
    uint8_t* sStage = smem + C::kSmemTiles;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kSmemTiles + C::kStageBytes);
    uint64_t* q_full = bars + 0;
    uint64_t* q_empty = bars + 1;
    uint64_t* s_full = bars + 2;      // [2]
    uint64_t* p_full = bars + 4;      // [2]
    uint64_t* pv_done = bars + 6;     // [2]
    uint64_t* p_half = bars + 8;      // [2]  first 64 keys of P written (PV may start on them)
    uint64_t* kv_full = bars + 10;    // [kSlots]
    uint64_t* kv_empty = bars + 10 + C::kSlots;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::kNumBars);
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(q_full, 1);
        mbar_init(q_empty, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s_full[i], 1);
            mbar_init(&p_full[i], kQTile);
            mbar_init(&p_half[i], kQTile);
            mbar_init(&pv_done[i], 1);
        }
        for (int s = 0; s < C::kSlots; ++s) {
            mbar_init(&kv_full[s], 1);
            mbar_init(&kv_empty[s], 1);
        }
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if constexpr (!kBatched) {
        if (warp == kProducerWarp && lane == 0) {
            prefetch_tensormap(&maps.q);
            prefetch_tensormap(&maps.k);
            prefetch_tensormap(&maps.v);
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    volatile int* abort_p = &abort_flag;
    // the softmax warpgroups hold a whole row of S in registers; the third warpgroup gives them its share

    if (warp >= 8) {
    setmaxnreg_dec<kOtherRegs>();
    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;           // ring counter
            uint32_t seg_idx = 0;
            bool ok = true;
            auto walk = make_walker<kBatched>(maps, p, starts);
            Segment s;
            while (ok && walk.next(s)) {
                const auto& pr = problem_of<kBatched>(maps, p, s);
                const CUtensorMap* map_q_p;
                const CUtensorMap* map_k_p;
                const CUtensorMap* map_v_p;
                if constexpr (kBatched) { map_q_p = &maps.q[s.prob]; map_k_p = &maps.k[s.prob]; map_v_p = &maps.v[s.prob]; }
                else { map_q_p = &maps.q; map_k_p = &maps.k; map_v_p = &maps.v; }
                const int row0 = s.qt * kTileM;
                const int c0 = seg_count(s, tiles_allowed(pr, row0, 0)), c1 = seg_count(s, tiles_allowed(pr, row0, 1));
                const int cnt = c0 > c1 ? c0 : c1;
                if (cnt == 0) continue;
                if (seg_idx > 0) ok = mbar_wait(q_empty, (seg_idx - 1) & 1, abort_p);
                if (!ok) break;
                mbar_arrive_expect_tx(q_full, 2 * C::kTileBytes);
                for (int i = 0; i < 2; ++i)
                    for (int b = 0; b < C::kBoxes; ++b)
                        tma_load_3d(sQ + i * C::kTileBytes + b * (kQTile * 128), map_q_p, q_full, b * 64, row0 + i * kQTile, s.bh);
                for (int j = 0; j < cnt && ok; ++j) {
                    const int t = s.t_begin + j;
                    for (int kv = 0; kv < 2 && ok; ++kv) {
                        const uint32_t slot = it % C::kSlots, round = it / C::kSlots;
                        ok = mbar_wait(&kv_empty[slot], (round & 1) ^ 1, abort_p);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&kv_full[slot], C::kTileBytes);
                        uint8_t* dst = sRing + slot * C::kTileBytes;
                        for (int b = 0; b < C::kBoxes; ++b)
                            tma_load_3d(dst + b * (kQTile * 128), kv == 0 ? map_k_p : map_v_p, &kv_full[slot], b * 64, t * kTileN, s.bh);
                        ++it;
                    }
                }
                ++seg_idx;
            }
            if (!ok) {
                // leave no copy in flight: every slot armed in its latest round must have landed
                for (uint32_t back = 0; back < (uint32_t)C::kSlots && back < it; ++back) {
                    const uint32_t id = it - 1 - back, slot = id % C::kSlots, round = id / C::kSlots;
                    int dummy = 0;
                    mbar_wait(&kv_full[slot], round & 1, &dummy, 200000000LL);
                }
                // seg_idx counts the Q loads armed so far; the last one may still be on its way
                if (seg_idx > 0) {
                    int dummy = 0;
                    mbar_wait(q_full, (seg_idx - 1) & 1, &dummy, 200000000LL);
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer
        // The whole warp walks the schedule (every value below is the same in all lanes) and one elected
        // lane issues: descriptors and addresses then live in uniform registers and an MMA costs a few
        // instructions, which matters because the tensor pipe takes the next MMA only when it has room.
        {
            const uint32_t idesc_qk = make_idesc_bf16(kQTile, kTileN, 0, 0);
            const uint32_t idesc_pv = make_idesc_bf16(kQTile, D, 0, 1);
            // Descriptors are built once; per MMA only the 14-bit address field of the low word moves
            // (one 32-bit add of a compile-time constant).
            const uint64_t q_desc = make_smem_desc_sw128(smem_u32(sQ), 16, 1024);
            const uint64_t k_desc = make_smem_desc_sw128(smem_u32(sRing), 16, 1024);            // K-major tile (K)
            const uint64_t v_desc = make_smem_desc_sw128(smem_u32(sRing), kQTile * 128, 1024);  // MN-major tile (V)
            const uint32_t desc_hi = (uint32_t)(q_desc >> 32);        // identical for all three
            const uint32_t q_lo[2] = {(uint32_t)q_desc, (uint32_t)q_desc + (C::kTileBytes >> 4)};
            const uint32_t k_lo0 = (uint32_t)k_desc, v_lo0 = (uint32_t)v_desc;
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
            const uint32_t tS0 = tmem_u + C::kColS, tO0 = tmem_u + C::kColO;
            uint32_t it = 0, seg_idx = 0;
            uint32_t n_pv[2] = {0, 0};
            bool ok = true;
            auto issue_qk = [&](int i, uint32_t k_slot) {
                const uint32_t a_lo = q_lo[i], b_lo = k_lo0 + k_slot * (C::kTileBytes >> 4), d = tS0 + i * kTileN;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off16 = ((kk >> 2) * (kQTile * 128) + (kk & 3) * 32) >> 4;
                    if (elect_one()) mma_ss_parts(d, a_lo + off16, b_lo + off16, desc_hi, idesc_qk, kk > 0);
                }
                commit_elected(&s_full[i]);
            };
            auto issue_pv_half = [&](int i, uint32_t v_slot, bool accumulate, int half) {
                const uint32_t b_lo = v_lo0 + v_slot * (C::kTileBytes >> 4), d = tO0 + i * D, a = tS0 + i * kTileN;
#pragma unroll
                for (int k4 = 0; k4 < kTileN / 32; ++k4) {
                    const int kk = half * (kTileN / 32) + k4;
                    if (elect_one()) mma_ts_parts(d, a + kk * 8, b_lo + kk * (2048 >> 4), desc_hi, idesc_pv, (accumulate || kk > 0) ? 1u : 0u);
                }
                if (half == 1) commit_elected(&pv_done[i]);
            };
            auto walk = make_walker<kBatched>(maps, p, starts);
            Segment s;
            while (ok && walk.next(s)) {
                const auto& pr = problem_of<kBatched>(maps, p, s);
                const int row0 = s.qt * kTileM;
                const int c0 = seg_count(s, tiles_allowed(pr, row0, 0)), c1 = seg_count(s, tiles_allowed(pr, row0, 1));
                const int cnt = c0 > c1 ? c0 : c1;
                if (cnt == 0) continue;
                const int cq[2] = {c0, c1};
                ok = __all_sync(0xffffffffu, mbar_wait(q_full, seg_idx & 1, abort_p));
                if (!ok) break;
                // first K tile
                uint32_t k_slot = it % C::kSlots;
                ok = __all_sync(0xffffffffu, mbar_wait(&kv_full[k_slot], (it / C::kSlots) & 1, abort_p));
                if (!ok) break;
                tc_fence_after();
                for (int i = 0; i < 2; ++i)
                    if (cq[i] > 0) issue_qk(i, k_slot);
                commit_elected(&kv_empty[k_slot]);
                if (cnt == 1) commit_elected(q_empty);      // the segment's last use of Q is issued: its successor may load
                ++it;
                for (int j = 0; j < cnt && ok; ++j) {
                    const uint32_t v_slot = it % C::kSlots, v_par = (it / C::kSlots) & 1;
                    ++it;
                    const bool have_next = j + 1 < cnt;
                    uint32_t nk_slot = 0, nk_par = 0;
                    if (have_next) {
                        nk_slot = it % C::kSlots;
                        nk_par = (it / C::kSlots) & 1;
                        ++it;
                    }
                    // both tiles are usually there already: ask both barriers at once (the two answers travel together), and
                    // wait one after the other only if one is missing
                    {
                        const bool v_there = mbar_try_wait(&kv_full[v_slot], v_par);
                        const bool k_there = have_next ? mbar_try_wait(&kv_full[nk_slot], nk_par) : true;
                        if (!__all_sync(0xffffffffu, v_there && k_there)) {
                            ok = __all_sync(0xffffffffu, mbar_wait(&kv_full[v_slot], v_par, abort_p));
                            if (!ok) break;
                            if (have_next) {
                                ok = __all_sync(0xffffffffu, mbar_wait(&kv_full[nk_slot], nk_par, abort_p));
                                if (!ok) break;
                            }
                        }
                    }
                    tc_fence_after();
                    for (int i = 0; i < 2 && ok; ++i) {
                        if (j < cq[i]) {
                            ok = __all_sync(0xffffffffu, mbar_wait(&p_half[i], n_pv[i] & 1, abort_p));
                            if (!ok) break;
                            tc_fence_after();
                            issue_pv_half(i, v_slot, j > 0, 0);
                            ok = __all_sync(0xffffffffu, mbar_wait(&p_full[i], n_pv[i] & 1, abort_p));
                            if (!ok) break;
                            tc_fence_after();
                            issue_pv_half(i, v_slot, j > 0, 1);
                            ++n_pv[i];
                        }
                        if (i == 1) commit_elected(&kv_empty[v_slot]);
                        if (have_next && j + 1 < cq[i]) issue_qk(i, nk_slot);
                        if (have_next && i == 1) {
                            commit_elected(&kv_empty[nk_slot]);
                            // Q is last read by the S of the segment's last key tile: releasing it here lets the
                            // producer fetch the next segment's Q while this one finishes
                            if (j + 2 == cnt) commit_elected(q_empty);
                        }
                    }
                }
                if (!ok) break;
                ++seg_idx;
            }
        }
    }
    } else {
        // ------------------------------------------------------------------ softmax warpgroups (one per Q tile)
        setmaxnreg_inc<kSoftmaxRegs>();
        const int i = warp >> 2;                           // Q tile
        const int r = (warp & 3) * 32 + lane;              // row inside the Q tile == TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + lane_addr + C::kColS + i * kTileN;
        const uint32_t tO = tmem_base + lane_addr + C::kColO + i * D;
        uint32_t n = 0;     // tiles processed by this warpgroup (phase counter of s_full/p_full/pv_done)
        bool ok = true;
        auto walk = make_walker<kBatched>(maps, p, starts);
        int bh_first = 0;                                  // (b,h) of this CTA's first unit (used under schedule 0 only)
        if constexpr (!kBatched) bh_first = (int)(walk.u / p.key_tiles);
        Segment s;
        while (ok && walk.next(s)) {
            const auto& pr = problem_of<kBatched>(maps, p, s);
            const int row0 = s.qt * kTileM;
            const int row = row0 + i * kQTile + r;         // row inside W (may lie beyond W: computed, never stored)
            const int allowed_i = tiles_allowed(pr, row0, i);
            // keys visible to this row, and to the first row of this warp (the smallest in the warp)
            const long long lim_row_ll = pr.causal ? (long long)pr.N - pr.W + row + 1 : (long long)pr.N;
            const int lim_row = (int)(lim_row_ll < pr.N ? lim_row_ll : pr.N);
            const long long lim_warp_ll = pr.causal ? (long long)pr.N - pr.W + (row - lane) + 1 : (long long)pr.N;
            const int lim_warp = (int)(lim_warp_ll < pr.N ? lim_warp_ll : pr.N);
            const int cnt_i = seg_count(s, allowed_i);
            float m_ref = -CUDART_INF_F;
            uint64_t l2[2] = {0ull, 0ull};          // four partial row sums as two packed fp32 pairs
            for (int j = 0; j < cnt_i; ++j) {
                ok = mbar_wait(&s_full[i], n & 1, abort_p);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const int k0 = (s.t_begin + j) * kTileN;
                const bool masked = k0 + kTileN > lim_warp;   // warp-uniform: some column of some lane is masked
                const int nvalid = lim_row - k0;              // columns [0, nvalid) of this tile are allowed for this row
                // the whole row of S (128 fp32) comes into registers once
                uint32_t sv[kTileN / 32][32];
#pragma unroll
                for (int c = 0; c < kTileN / 32; ++c) tmem_ld32_async(tS + c * 32, sv[c]);
#pragma unroll
                for (int c = 0; c < kTileN / 32; ++c) tmem_wait_ld(sv[c]);
                if (masked) {
#pragma unroll
                    for (int e = 0; e < kTileN; ++e)
                        if (e >= nvalid) sv[e >> 5][e & 31] = 0xff800000u;   // -inf
                }
                float mx[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};   // independent chains
#pragma unroll
                for (int e = 0; e < kTileN / 2; ++e)
                    mx[e & 3] = max3(mx[e & 3], __uint_as_float(sv[e >> 4][(2 * e) & 31]), __uint_as_float(sv[e >> 4][(2 * e + 1) & 31]));
                const float tmax = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                const float m_new = fmaxf(m_ref, tmax * p.scale_log2e);
                const bool need = m_new > m_ref + kRescaleThreshold;
                if (__any_sync(0xffffffffu, need)) {
                    const float alpha = need ? ex2(m_ref - m_new) : 1.f;     // m_ref = -inf -> 0
                    if (j > 0) {
                        ok = mbar_wait(&pv_done[i], (n - 1) & 1, abort_p);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < D / 8; ++c) {      // narrow pieces: the row of S stays in registers meanwhile
                            uint32_t o[8];
                            tmem_ld8(tO + c * 8, o);
#pragma unroll
                            for (int e = 0; e < 8; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                            tmem_st8(tO + c * 8, o);
                        }
                    }
                    const uint64_t alpha2 = f2_pack(alpha, alpha);
                    l2[0] = f2_mul(l2[0], alpha2);
                    l2[1] = f2_mul(l2[1], alpha2);
                    if (need) m_ref = m_new;
                }
                const float m_use = m_ref == -CUDART_INF_F ? 0.f : m_ref;
                // P = 2^(s*scale - m) as bf16 over the columns of S; kPolyPairs of every 16 pairs take the
                // polynomial route (FMA pipe), the rest the special-function unit
                {
                    const uint64_t scale2 = f2_pack(p.scale_log2e, p.scale_log2e), negm2 = f2_pack(-m_use, -m_use);
#pragma unroll
                    for (int c = 0; c < kTileN / 32; ++c) {
                        float pe[32];
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const uint64_t x2 = f2_fma(f2_pack_bits(sv[c][2 * e], sv[c][2 * e + 1]), scale2, negm2);
                            if ((e % 16) * kPolyPairs / 16 != ((e % 16) + 1) * kPolyPairs / 16) {
                                exp2_poly2(x2, pe[2 * e], pe[2 * e + 1]);
                            } else {
                                float x0, x1;
                                f2_unpack(x2, x0, x1);
                                pe[2 * e] = ex2(x0);
                                pe[2 * e + 1] = ex2(x1);
                            }
                        }
                        if (masked) {          // the polynomial gives 2^-126, not 0, for a masked column
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (c * 32 + e >= nvalid) pe[e] = 0.f;
                        }
                        uint32_t pk[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            l2[e & 1] = f2_add(l2[e & 1], f2_pack(pe[2 * e], pe[2 * e + 1]));
                            pk[e] = pack_bf16x2(pe[2 * e], pe[2 * e + 1]);
                        }
                        tmem_st16(tS + c * 16, pk);
                        if (c == kTileN / 64 - 1) {        // first 64 keys are in place: let the PV MMAs start on them
                            tc_wait_st();
                            tc_fence_before();
                            mbar_arrive(&p_half[i]);
                        }
                    }
                }
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(&p_full[i]);
                ++n;
            }
            if (!ok) break;
            if (allowed_i == 0) continue;                  // this Q tile does not exist: nothing to write
            // ---------------------------------------------------------------- epilogue of the segment
            const bool whole = kBatched || (s.t_begin == 0 && s.t_end == p.key_tiles);
            if (cnt_i > 0) {
                ok = mbar_wait(&pv_done[i], (n - 1) & 1, abort_p);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
            }
            float l;
            {
                float a, b, c, d2;
                f2_unpack(l2[0], a, b);
                f2_unpack(l2[1], c, d2);
                l = (a + b) + (c + d2);
            }
            const float inv_l = l > 0.f ? 1.f / l : 0.f;
            const float lse_val = l > 0.f ? (m_ref + log2f(l)) * kLn2 : -CUDART_INF_F;
            const bool store = row < pr.W;
            // partial result -> workspace slot (0: first segment of this CTA's range, 1: a later one)
            float* pbase = p.ws + ((long long)blockIdx.x * 2 + (s.bh == bh_first ? 0 : 1)) * (long long)kTileM * (D + 1);
            // A thread holds one row.  Stored straight from the registers a warp's store would touch 32 different lines, so
            // the warp passes its rows through shared memory 128 bytes at a time (16-byte pieces, piece index xor row: no
            // bank conflicts beyond the minimum on either side) and every store instruction writes four whole lines.
            uint8_t* stage = sStage + warp * (32 * 128);
            const int row_warp = row - lane;                   // row of lane 0
            if (whole) {
                __nv_bfloat16* owarp = reinterpret_cast<__nv_bfloat16*>(pr.out) + ((long long)s.bh * pr.W + row_warp) * D;
#pragma unroll
                for (int h = 0; h < D / 64; ++h) {             // 64 bf16 columns per pass
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t o[16];
                        if (cnt_i > 0) {
                            tmem_ld16_async(tO + h * 64 + c * 16, o);
                            tmem_wait_ld16(o);
                        } else {
#pragma unroll
                            for (int e = 0; e < 16; ++e) o[e] = 0u;
                        }
#pragma unroll
                        for (int v4 = 0; v4 < 2; ++v4) {
                            uint4 w;
                            w.x = pack_bf16x2(__uint_as_float(o[v4 * 8 + 0]) * inv_l, __uint_as_float(o[v4 * 8 + 1]) * inv_l);
                            w.y = pack_bf16x2(__uint_as_float(o[v4 * 8 + 2]) * inv_l, __uint_as_float(o[v4 * 8 + 3]) * inv_l);
                            w.z = pack_bf16x2(__uint_as_float(o[v4 * 8 + 4]) * inv_l, __uint_as_float(o[v4 * 8 + 5]) * inv_l);
                            w.w = pack_bf16x2(__uint_as_float(o[v4 * 8 + 6]) * inv_l, __uint_as_float(o[v4 * 8 + 7]) * inv_l);
                            *reinterpret_cast<uint4*>(stage + lane * 128 + (((c * 2 + v4) ^ (lane & 7)) << 4)) = w;
                        }
                    }
                    __syncwarp();
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int rrow = it * 4 + (lane >> 3), piece = lane & 7;
                        const uint4 w = *reinterpret_cast<const uint4*>(stage + rrow * 128 + ((piece ^ (rrow & 7)) << 4));
                        if (row_warp + rrow < pr.W) *reinterpret_cast<uint4*>(owarp + (long long)rrow * D + h * 64 + piece * 8) = w;
                    }
                    __syncwarp();
                }
            } else {
                float* pwarp = pbase + (long long)(i * kQTile + (warp & 3) * 32) * D;
#pragma unroll
                for (int h = 0; h < D / 32; ++h) {             // 32 fp32 columns per pass
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t o[16];
                        if (cnt_i > 0) {
                            tmem_ld16_async(tO + h * 32 + c * 16, o);
                            tmem_wait_ld16(o);
                        } else {
#pragma unroll
                            for (int e = 0; e < 16; ++e) o[e] = 0u;
                        }
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) {
                            float4 w;
                            w.x = __uint_as_float(o[v4 * 4 + 0]) * inv_l;
                            w.y = __uint_as_float(o[v4 * 4 + 1]) * inv_l;
                            w.z = __uint_as_float(o[v4 * 4 + 2]) * inv_l;
                            w.w = __uint_as_float(o[v4 * 4 + 3]) * inv_l;
                            *reinterpret_cast<float4*>(stage + lane * 128 + (((c * 4 + v4) ^ (lane & 7)) << 4)) = w;
                        }
                    }
                    __syncwarp();
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int rrow = it * 4 + (lane >> 3), piece = lane & 7;
                        const float4 w = *reinterpret_cast<const float4*>(stage + rrow * 128 + ((piece ^ (rrow & 7)) << 4));
                        *reinterpret_cast<float4*>(pwarp + (long long)rrow * D + h * 32 + piece * 4) = w;
                    }
                    __syncwarp();
                }
            }
            if (whole) {
                if (store && pr.lse != nullptr) pr.lse[(long long)s.bh * pr.W + row] = lse_val;
            } else {
                pbase[(long long)kTileM * D + i * kQTile + r] = lse_val;
            }
            tc_fence_before();      // TMEM reads of O are complete before the next segment's arrive lets PV overwrite it
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(p.status, (int)TLIN_ERR_TIMEOUT);
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// Combines the partial results of every (b,h) whose key tiles were split between groups.
// One CTA per 8 query rows of a (b,h, q-tile pair): 8 warps, one row each, 4 (or 2) columns per lane.
constexpr int kMergeRows = 8;            // one row per warp: many small CTAs hide the latency of the scattered partial reads
constexpr int kMaxParts = 8;          // more partials than this per row are merged in a slower loop

template <int D>
__global__ void __launch_bounds__(256)
fwd_merge_kernel(const Params p) {
    constexpr int CPL = D / 32;                           // columns per lane
    const int blocks_per_tile = kTileM / kMergeRows;
    const int quarter = blockIdx.x % blocks_per_tile;
    const int tile_id = blockIdx.x / blocks_per_tile;     // bh * q_tiles + qt
    const int bh = tile_id / p.q_tiles, qt = tile_id - bh * p.q_tiles;
    __shared__ const float* part_base[kMaxParts];
    __shared__ int n_parts_s, g_lo_s;
    if (threadIdx.x == 0) {
        const unsigned long long T = (unsigned long long)p.key_tiles, U = (unsigned long long)p.total_units, G = (unsigned)p.n_groups;
        // groups holding the first and the last unit of this (b,h): largest g with floor(g*U/G) <= x
        const unsigned long long x0 = (unsigned long long)bh * T, x1 = x0 + T - 1;
        const int g_lo = (int)(((x0 + 1) * G - 1) / U), g_hi = (int)(((x1 + 1) * G - 1) / U);
        g_lo_s = g_lo;
        n_parts_s = g_hi - g_lo + 1;
        for (int g = g_lo; g <= g_hi && g - g_lo < kMaxParts; ++g) {
            const int cta = g * p.q_tiles + qt;
            const int slot = bh == (int)((((unsigned long long)g * U) / G) / T) ? 0 : 1;
            part_base[g - g_lo] = p.ws + ((long long)cta * 2 + slot) * (long long)kTileM * (D + 1);
        }
    }
    __syncthreads();
    const int n_parts = n_parts_s;
    if (n_parts <= 1) return;                             // written directly by the attention kernel
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int rq = warp; rq < kMergeRows; rq += 8) {
        const int rr = quarter * kMergeRows + rq;         // row inside the 256-row tile
        const int row = qt * kTileM + rr;
        if (row >= p.W) break;
        float m = -CUDART_INF_F;
        if (n_parts <= kMaxParts) {
            float ls[kMaxParts];
#pragma unroll
            for (int i = 0; i < kMaxParts; ++i) {
                ls[i] = i < n_parts ? part_base[i][(long long)kTileM * D + rr] : -CUDART_INF_F;
                m = fmaxf(m, ls[i]);
            }
            float z = 0.f, acc[CPL];
#pragma unroll
            for (int e = 0; e < CPL; ++e) acc[e] = 0.f;
#pragma unroll
            for (int i = 0; i < kMaxParts; ++i) {
                if (i < n_parts) {
                    const float w = expf(ls[i] - m);      // -inf (empty part) -> 0
                    z += w;
                    const float* src = part_base[i] + (long long)rr * D + lane * CPL;
#pragma unroll
                    for (int e = 0; e < CPL; ++e) acc[e] = fmaf(w, src[e], acc[e]);
                }
            }
            const float inv = 1.f / z;
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + ((long long)bh * p.W + row) * D + lane * CPL;
#pragma unroll
            for (int e = 0; e < CPL; e += 2)
                *reinterpret_cast<uint32_t*>(dst + e) = pack_bf16x2(acc[e] * inv, acc[e + 1] * inv);
            if (p.lse != nullptr && lane == 0) p.lse[(long long)bh * p.W + row] = m + logf(z);
        } else {
            // many small groups per (b,h): recompute the slot addresses on the fly
            const unsigned long long T = (unsigned long long)p.key_tiles, U = (unsigned long long)p.total_units, G = (unsigned)p.n_groups;
            auto base_of = [&](int g) {
                const int cta = g * p.q_tiles + qt;
                const int slot = bh == (int)((((unsigned long long)g * U) / G) / T) ? 0 : 1;
                return p.ws + ((long long)cta * 2 + slot) * (long long)kTileM * (D + 1);
            };
            for (int i = 0; i < n_parts; ++i) m = fmaxf(m, base_of(g_lo_s + i)[(long long)kTileM * D + rr]);
            float z = 0.f, acc[CPL];
#pragma unroll
            for (int e = 0; e < CPL; ++e) acc[e] = 0.f;
            for (int i = 0; i < n_parts; ++i) {
                const float* base = base_of(g_lo_s + i);
                const float w = expf(base[(long long)kTileM * D + rr] - m);
                z += w;
#pragma unroll
                for (int e = 0; e < CPL; ++e) acc[e] = fmaf(w, base[(long long)rr * D + lane * CPL + e], acc[e]);
            }
            const float inv = 1.f / z;
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + ((long long)bh * p.W + row) * D + lane * CPL;
#pragma unroll
            for (int e = 0; e < CPL; e += 2)
                *reinterpret_cast<uint32_t*>(dst + e) = pack_bf16x2(acc[e] * inv, acc[e + 1] * inv);
            if (p.lse != nullptr && lane == 0) p.lse[(long long)bh * p.W + row] = m + logf(z);
        }
    }
}

template <int D>
int launch_d(const void* q, const void* k, const void* v, void* out, float* lse, int B, int H, int N, int W,
             int causal, const tlin_fwd_plan& plan, float* ws, long long kv_rows_alloc, cudaStream_t st) {
    using C = Cfg<D>;
    const long long bh = (long long)B * H;
    KernelMaps<false> maps;
    int rc = make_map(&maps.q, q, D, W, bh);
    if (rc == TLIN_OK) rc = make_map(&maps.k, k, D, N, bh, kQTile, kv_rows_alloc);
    if (rc == TLIN_OK) rc = make_map(&maps.v, v, D, N, bh, kQTile, kv_rows_alloc);
    if (rc != TLIN_OK) return rc;
    Params p;
    p.out = out; p.lse = lse; p.ws = ws; p.status = status_word();
    if (!p.status) return TLIN_ERR_CUDA;
    p.total_units = plan.total_units; p.n_groups = plan.n_groups; p.q_tiles = plan.q_tiles; p.key_tiles = plan.key_tiles;
    p.N = N; p.W = W; p.causal = causal; p.schedule = plan.schedule;
    p.scale_log2e = kLog2e / sqrtf((float)D);
    static bool smem_allowed[64] = {};
    TLIN_CUDA_CHECK(allow_dynamic_smem(fwd_tc_kernel<D, false>, C::kSmemBytes, smem_allowed));
    if (plan.n_groups > kMaxGroups) return TLIN_ERR_UNSUPPORTED;
    GroupStarts starts;
    fwd_group_starts(plan, &starts);
    fwd_tc_kernel<D, false><<<plan.n_ctas, kThreads, C::kSmemBytes, st>>>(maps, p, starts);
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch();
    if (plan.uses_workspace) {
        fwd_merge_kernel<D><<<(unsigned)(bh * plan.q_tiles * (kTileM / kMergeRows)), 256, 0, st>>>(p);
        TLIN_CUDA_CHECK(cudaGetLastError());
        count_launch();
    }
    return TLIN_OK;
}

// A table of problems as one launch: every CTA walks a contiguous run of whole (problem, b*h, query tile pair) units.
template <int D>
int launch_batched_d(const tlin_problem* problems, int n, const long long* starts_in, int n_ctas, cudaStream_t st) {
    using C = Cfg<D>;
    static_assert(sizeof(KernelMaps<true>) + sizeof(Params) + sizeof(GroupStarts) < 32000, "launch parameters exceed the limit");
    KernelMaps<true> maps;
    memset(&maps, 0, sizeof(maps));
    maps.n = n;
    long long unit = 0;
    for (int i = 0; i < n; ++i) {
        const tlin_problem& pb = problems[i];
        const long long kv_rows = pb.kv_rows > 0 ? pb.kv_rows : pb.n_keys;
        int rc = make_map(&maps.q[i], pb.q, D, pb.n_queries, pb.BH);
        if (rc == TLIN_OK) rc = make_map(&maps.k[i], pb.k, D, pb.n_keys, pb.BH, kQTile, kv_rows);
        if (rc == TLIN_OK) rc = make_map(&maps.v[i], pb.v, D, pb.n_keys, pb.BH, kQTile, kv_rows);
        if (rc != TLIN_OK) return rc;
        ProblemDev& pd = maps.prob[i];
        pd.out = pb.out; pd.lse = pb.lse; pd.unit0 = unit;
        pd.N = pb.n_keys; pd.W = pb.n_queries; pd.causal = pb.causal_window;
        pd.key_tiles = (pb.n_keys + kTileN - 1) / kTileN;
        pd.q_tiles = (pb.n_queries + kTileM - 1) / kTileM;
        unit += (long long)pb.BH * pd.q_tiles;
    }
    Params p;
    memset(&p, 0, sizeof(p));
    p.status = status_word();
    if (!p.status) return TLIN_ERR_CUDA;
    p.total_units = unit; p.n_groups = n_ctas; p.q_tiles = 1; p.key_tiles = 1; p.schedule = 1;
    p.scale_log2e = kLog2e / sqrtf((float)D);
    if (n_ctas > kMaxGroups) return TLIN_ERR_UNSUPPORTED;
    GroupStarts starts;
    for (int g = 0; g <= n_ctas; ++g) starts.u[g] = starts_in[g];
    static bool smem_allowed[64] = {};
    TLIN_CUDA_CHECK(allow_dynamic_smem(fwd_tc_kernel<D, true>, C::kSmemBytes, smem_allowed));
    fwd_tc_kernel<D, true><<<n_ctas, kThreads, C::kSmemBytes, st>>>(maps, p, starts);
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch();
    return TLIN_OK;
}

}  // namespace

int launch_fwd_tc_batched(const tlin_problem* problems, int n, int d, const long long* starts, int n_ctas, cudaStream_t st) {
    if (n <= 0 || n > kMaxBatch) return TLIN_ERR_INVALID_ARG;
    if (d == 128) return launch_batched_d<128>(problems, n, starts, n_ctas, st);
    if (d == 64) return launch_batched_d<64>(problems, n, starts, n_ctas, st);
    return TLIN_ERR_UNSUPPORTED;
}

int launch_fwd_tc(const void* q, const void* k, const void* v, void* out, float* lse,
                  int B, int H, int N, int W, int d, int causal, const tlin_fwd_plan& plan,
                  float* ws, long long kv_rows_alloc, cudaStream_t st) {
    if (plan.tile_m != kTileM || plan.tile_n != kTileN) return TLIN_ERR_UNSUPPORTED;
    if ((long long)B * H * W > 0x7fffffffLL) return TLIN_ERR_UNSUPPORTED;
    if (d == 128) return launch_d<128>(q, k, v, out, lse, B, H, N, W, causal, plan, ws, kv_rows_alloc, st);
    if (d == 64) return launch_d<64>(q, k, v, out, lse, B, H, N, W, causal, plan, ws, kv_rows_alloc, st);
    return TLIN_ERR_UNSUPPORTED;
}

}  // namespace tlin
