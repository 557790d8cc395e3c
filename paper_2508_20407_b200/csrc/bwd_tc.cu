// Tensor-core backward pass for sm_100a (bf16 in and out, fp32 accumulate): the chain rule of the Section 3
// attention formula with the window rule j <= N-W+i.  Training runs every layer as forward + backward ("cache miss"
// throughout, Section 4.1); the paper gives no gradient algorithm of its own.
//
//   p = exp(q k^T / sqrt(d) - lse)    dp = dout v^T    ds = p * (dp - delta) / sqrt(d),  delta_i = dout_i . out_i
//   dv = p^T dout      dk = ds^T q      dq = ds k
//
// Two kernels, neither with atomics, both recomputing p from the saved lse (the default):
//
// bwd_dkdv_tc_kernel   A CTA owns one 128-key tile of a (b,h) at a time and walks the 128-row query tiles that may
//   see it.  Scores are computed TRANSPOSED (S^T = K Q^T, dP^T = V dout^T: TMEM lane = key, column = query) so that
//   P^T and dS^T, written back to TMEM as bf16, are directly the A operands of dV += P^T dout and dK += dS^T Q, whose
//   B operands are the dout / Q tiles already in shared memory (read MN-major).  dK and dV stay in TMEM for the whole
//   key tile and are written once.  Each 128-query tile is worked on as two independent chains of 64 queries, one per
//   warpgroup (thread = key row): [S^T_x | dP^T_x] by the tensor pipe, then P^T_x and dS^T_x written over them in
//   place, then the two accumulating MMAs; while one chain does its elementwise work the tensor pipe serves the other.
//
// bwd_dq_tc_kernel     The forward's structure: a CTA owns 256 query rows (two Q tiles, one warpgroup each, one
//   thread per row) and streams 128-key tiles; per tile S = Q K^T -> p (kept in registers), then dP = dout V^T into
//   the same TMEM columns -> dS (bf16, in place) -> dQ += dS K with K read MN-major.  The work is scheduled like the
//   forward (groups that split the key range write fp32 partial dQ to the workspace; a small kernel adds them).
//
// bwd_fused_tc_kernel  (d = 128, on request)  The dK/dV kernel with a third accumulating product per chain step,
//   dQ^T_x = K^T dS^T_x (K read MN-major, dS^T_x also written to shared memory as the B operand) into the chain's dead
//   dP^T_x columns, which the chain's threads read back and add to an fp32 dQ buffer with reductions in L2; a small kernel
//   scales and rounds it.  Five matrix products instead of seven, but 32 KB of reductions per chain step, and an SM gets
//   about 25 bytes per clock of those: measured within +-10 % of the two kernels.
//
// A preparation kernel writes lse*log2(e) and delta per query row, padded to a multiple of 128 rows per (b,h) with
// +inf / 0: a padded row then gives p = 0 without any test.
//
// Every wait is bounded: on expiry the CTA sets the library's error word, drains and exits.
#include "tlin_internal.h"
#include "sm100_ptx.cuh"
#include "tc_common.cuh"
#include <math_constants.h>

namespace tlin {
namespace {

using namespace ptx;
using namespace tc;

constexpr int kProducerWarp = 8;
constexpr int kMmaWarp = 9;
constexpr int kKvWarp = 10;                 // dK/dV kernel only
constexpr float kLog2e = 1.4426950408889634f;

struct BwdParams {
    const float* lse2;        // [B*H, Wpad]  lse * log2(e), +inf beyond W
    const float* delta;       // [B*H, Wpad]  dout . out,   0 beyond W
    void* dq;                 // [B*H, W, D] bf16
    void* dk;                 // [B*H, N, D] bf16
    void* dv;
    float* ws;                // partial dQ slots of the dq kernel
    int* status;
    long long total_units;    // dk/dv kernel: B*H*key_tiles; dq kernel: the plan's units
    int n_groups, q_tiles, key_tiles, schedule;   // dq kernel: the forward's plan fields
    int q_tiles128;           // ceil(W / 128)
    int N, W, Wpad, causal;
    int wide_stores;          // dq and the workspace are 32-byte aligned: the dQ kernel may use 32-byte stores
    float scale_log2e, scale;
};

// ------------------------------------------------------------------------------------------ preparation
// Row statistics of the backward pass: lse2 = lse * log2(e) and delta = sum_c out*dout, on rows padded to 128 per (b,h)
// (padding rows: +inf and 0).  D/8 lanes share a row with one 16-byte load per tensor each; a warp keeps kPrepPasses
// groups of rows in flight, so that enough bytes are outstanding to stream at HBM speed.
constexpr int kPrepPasses = 4;
template <int D>
__host__ __device__ constexpr int prep_rows_per_block() { return 8 * (32 / (D / 8)) * kPrepPasses; }

template <int D>
__global__ void __launch_bounds__(256)
bwd_prep_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout, const float* __restrict__ lse,
                float* __restrict__ lse2, float* __restrict__ delta, int W, int Wpad, long long rows_padded) {
    constexpr int LPR = D / 8;              // lanes per row
    constexpr int RPP = 32 / LPR;           // rows per pass of a warp
    const int lane = threadIdx.x & 31, sub = lane / LPR, l = lane % LPR;
    const long long first = ((long long)blockIdx.x * 8 + (threadIdx.x >> 5)) * (RPP * kPrepPasses) + sub;
    uint4 a[kPrepPasses], b[kPrepPasses];
    long long row[kPrepPasses];
#pragma unroll
    for (int ps = 0; ps < kPrepPasses; ++ps) {
        const long long prow = first + ps * RPP;
        const long long bh = prow / Wpad;
        const int i = (int)(prow - bh * Wpad);
        row[ps] = (prow < rows_padded && i < W) ? bh * W + i : -1;
        a[ps] = b[ps] = make_uint4(0u, 0u, 0u, 0u);
        if (row[ps] >= 0) {
            a[ps] = *reinterpret_cast<const uint4*>(out + row[ps] * D + l * 8);
            b[ps] = *reinterpret_cast<const uint4*>(dout + row[ps] * D + l * 8);
        }
    }
#pragma unroll
    for (int ps = 0; ps < kPrepPasses; ++ps) {
        const uint32_t* aw = reinterpret_cast<const uint32_t*>(&a[ps]);
        const uint32_t* bw = reinterpret_cast<const uint32_t*>(&b[ps]);
        float acc = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&aw[e]));
            const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bw[e]));
            acc = fmaf(x.x, y.x, fmaf(x.y, y.y, acc));
        }
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        const long long prow = first + ps * RPP;
        if (l == 0 && prow < rows_padded) {
            lse2[prow] = row[ps] >= 0 ? lse[row[ps]] * kLog2e : CUDART_INF_F;
            delta[prow] = row[ps] >= 0 ? acc : 0.f;
        }
    }
}

// ------------------------------------------------------------------------------------------ dK / dV
template <int D>
struct ACfg {
    static constexpr int kTileBytes = kQTile * D * 2;          // one 128-row tile (K or V)
    static constexpr int kHalfBytes = 64 * D * 2;              // one 64-row tile (Q or dout of a chain step)
    static constexpr int kBoxes = D / 64;
    static constexpr int kSlots = D == 128 ? 4 : 8;            // ring of chain steps: Q (64 rows), dout (64 rows), 64 lse2 + 64 delta
    static constexpr int kSlotBytes = 2 * kHalfBytes;
    static constexpr int kOffKV = 0;
    static constexpr int kOffRing = 2 * kTileBytes;
    static constexpr int kOffStats = kOffRing + kSlots * kSlotBytes;
    static constexpr int kOffStage = kOffStats + kSlots * 512;  // per compute warp 32 rows x D bytes: dK / dV rows on their way out
    static constexpr int kOffBars = kOffStage + 8 * 32 * D;
    static constexpr int kNumBars = 8 + 2 * kSlots;
    static constexpr int kSmemBytes = kOffBars + kNumBars * 8 + 16;
    // TMEM columns: dK, dV (D each); per chain x (64 queries of the tile) 128 columns: S^T_x (64 fp32) and dP^T_x
    // (64 fp32); P^T_x and dS^T_x (bf16, 32 columns each) are written over the first half of S^T_x and dP^T_x
    static constexpr uint32_t kColDK = 0, kColDV = D, kColR = 2 * D;
    static constexpr int kThreads = 32 * 11;
};

// first 128-row query tile that may use a key of key tile t
__device__ __forceinline__ int first_q_tile(const BwdParams& p, int t) {
    if (!p.causal) return 0;
    const long long f = (long long)t * kTileN - ((long long)p.N - p.W);
    return f <= 0 ? 0 : (int)(f / kQTile);
}

template <int D>
__global__ void __launch_bounds__(ACfg<D>::kThreads, 1)
bwd_dkdv_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do, const BwdParams p) {
    using C = ACfg<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* sKV = smem + C::kOffKV;          // K, V
    uint8_t* sRing = smem + C::kOffRing;      // [kSlots][Q 64 rows | dout 64 rows]
    float* sStats = reinterpret_cast<float*>(smem + C::kOffStats);   // [kSlots][lse2 64 | delta 64]
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kOffBars);
    uint64_t* kv_full = bars + 0;
    uint64_t* kv_empty = bars + 1;
    uint64_t* sdp_full = bars + 2;    // [2] S^T_x and dP^T_x of a step are in TMEM
    uint64_t* pds_full = bars + 4;    // [2] the chain's threads have stored P^T_x and dS^T_x
    uint64_t* acc_full = bars + 6;    // dK, dV of the key tile are complete
    uint64_t* acc_empty = bars + 7;   // all threads have read them
    uint64_t* slot_full = bars + 8;   // [kSlots]
    uint64_t* slot_empty = slot_full + C::kSlots;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::kNumBars);
    int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool base_ok = (smem_u32(smem) & 1023u) == 0;   // the swizzled tiles need 1024-byte alignment

    if (threadIdx.x == 0) {
        *abort_flag = base_ok ? 0 : 1;
        mbar_init(kv_full, 1);
        mbar_init(kv_empty, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sdp_full[i], 1);
            mbar_init(&pds_full[i], 128);
        }
        for (int i = 0; i < C::kSlots; ++i) {
            mbar_init(&slot_full[i], 1);
            mbar_init(&slot_empty[i], 1);
        }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, 256);
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == kProducerWarp && lane == 0) {
        prefetch_tensormap(&map_q);
        prefetch_tensormap(&map_k);
        prefetch_tensormap(&map_v);
        prefetch_tensormap(&map_do);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    volatile int* abort_p = abort_flag;

    // The CTAs share the (b,h,key tile) units by cost (query tiles a key tile has to visit), not by count: with the
    // window rule the last key tiles of a (b,h) are cheaper, down to one step.
    const long long u_begin = bwd_first_unit_of_share(p.N, p.W, p.causal, p.total_units, p.key_tiles, blockIdx.x, gridDim.x);
    const long long u_end = bwd_first_unit_of_share(p.N, p.W, p.causal, p.total_units, p.key_tiles, blockIdx.x + 1, gridDim.x);

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ TMA producer: Q / dout / row statistics ring
        // The ring runs ahead of the key tiles: the first chain steps of the next key tile are loaded while the
        // current one is still being worked on.
        if (lane == 0) {
            bool ok = base_ok;
            uint32_t hh = 0;                // chain steps (64 queries each) issued
            for (long long u = u_begin; u < u_end && ok; ++u) {
                const int bh = (int)(u / p.key_tiles), t = (int)(u - (long long)bh * p.key_tiles);
                const int row_first = first_q_tile(p, t) * kQTile, row_end = p.q_tiles128 * kQTile;
                for (int row = row_first; row < row_end && ok; row += 64, ++hh) {
                    const uint32_t slot = hh % C::kSlots, round = hh / C::kSlots;
                    ok = mbar_wait(&slot_empty[slot], (round & 1) ^ 1, abort_p);
                    if (!ok) break;
                    uint8_t* dst = sRing + slot * C::kSlotBytes;
                    mbar_arrive_expect_tx(&slot_full[slot], C::kSlotBytes + 512);
                    for (int x = 0; x < C::kBoxes; ++x) {
                        tma_load_3d(dst + x * (64 * 128), &map_q, &slot_full[slot], x * 64, row, bh);
                        tma_load_3d(dst + C::kHalfBytes + x * (64 * 128), &map_do, &slot_full[slot], x * 64, row, bh);
                    }
                    bulk_load_1d(sStats + slot * 128, p.lse2 + (long long)bh * p.Wpad + row, 256, &slot_full[slot]);
                    bulk_load_1d(sStats + slot * 128 + 64, p.delta + (long long)bh * p.Wpad + row, 256, &slot_full[slot]);
                }
            }
            if (!ok && base_ok) {
                int dummy = 0;              // leave no copy in flight: the barriers armed last must complete (bounded)
                for (uint32_t back = 1; back <= (uint32_t)C::kSlots && back <= hh; ++back) {
                    const uint32_t id = hh - back;
                    mbar_wait(&slot_full[id % C::kSlots], (id / C::kSlots) & 1, &dummy, 200000000LL);
                }
            }
        }
    } else if (warp == kKvWarp) {
        // ------------------------------------------------------------------ TMA producer: K, V of the key tiles
        if (lane == 0) {
            bool ok = base_ok;
            uint32_t n = 0;
            for (long long u = u_begin; u < u_end && ok; ++u, ++n) {
                const int bh = (int)(u / p.key_tiles), t = (int)(u - (long long)bh * p.key_tiles);
                if (u + 1 < u_end) {        // K, V have one buffer: the next tile's rows come as far as L2 meanwhile
                    const int bh_n = (int)((u + 1) / p.key_tiles), t_n = (int)(u + 1 - (long long)bh_n * p.key_tiles);
                    for (int x = 0; x < C::kBoxes; ++x) {
                        tma_prefetch_l2_3d(&map_k, x * 64, t_n * kTileN, bh_n);
                        tma_prefetch_l2_3d(&map_v, x * 64, t_n * kTileN, bh_n);
                    }
                }
                ok = mbar_wait(kv_empty, (n & 1) ^ 1, abort_p);
                if (!ok) break;
                mbar_arrive_expect_tx(kv_full, 2 * C::kTileBytes);
                for (int x = 0; x < C::kBoxes; ++x) {
                    tma_load_3d(sKV + x * (kQTile * 128), &map_k, kv_full, x * 64, t * kTileN, bh);
                    tma_load_3d(sKV + C::kTileBytes + x * (kQTile * 128), &map_v, kv_full, x * 64, t * kTileN, bh);
                }
            }
            if (!ok && base_ok && n > 0) {
                int dummy = 0;
                mbar_wait(kv_full, (n - 1) & 1, &dummy, 200000000LL);
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer (all lanes walk, one issues)
        const uint32_t idesc_st = make_idesc_bf16(kQTile, 64, 0, 0);         // S^T, dP^T of a chain: M = keys, N = 64 queries
        const uint32_t idesc_acc = make_idesc_bf16(kQTile, D, 0, 1);         // dV, dK: A in TMEM, B MN-major
        const uint64_t kmaj = make_smem_desc_sw128(smem_u32(smem), 16, 1024);
        const uint64_t mnmaj = make_smem_desc_sw128(smem_u32(smem), 64 * 128, 1024);   // 64-row tiles: 8 KB between column blocks
        const uint32_t desc_hi = (uint32_t)(kmaj >> 32);
        const uint32_t kmaj_lo = (uint32_t)kmaj, mnmaj_lo = (uint32_t)mnmaj;
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t tDK = tmem_u + C::kColDK, tDV = tmem_u + C::kColDV;
        const uint32_t k_off = (uint32_t)(C::kOffKV >> 4), v_off = (uint32_t)((C::kOffKV + C::kTileBytes) >> 4);
        // [S^T_x | dP^T_x] = [K Q_x^T | V dout_x^T]: A a 128-row K-major tile, B the 64-row K-major tile of the slot
        auto issue_sdp = [&](int x, uint32_t slot) {
            const uint32_t q_off = (uint32_t)((C::kOffRing + slot * C::kSlotBytes) >> 4), do_off = q_off + (uint32_t)(C::kHalfBytes >> 4);
            const uint32_t d = tmem_u + C::kColR + x * 128;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t a16 = ((kk >> 2) * (kQTile * 128) + (kk & 3) * 32) >> 4, b16 = ((kk >> 2) * (64 * 128) + (kk & 3) * 32) >> 4;
                if (elect_one()) mma_ss_parts(d, kmaj_lo + k_off + a16, kmaj_lo + q_off + b16, desc_hi, idesc_st, kk > 0);
            }
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t a16 = ((kk >> 2) * (kQTile * 128) + (kk & 3) * 32) >> 4, b16 = ((kk >> 2) * (64 * 128) + (kk & 3) * 32) >> 4;
                if (elect_one()) mma_ss_parts(d + 64, kmaj_lo + v_off + a16, kmaj_lo + do_off + b16, desc_hi, idesc_st, kk > 0);
            }
            commit_elected(&sdp_full[x]);
        };
        // dV += P^T_x dout_x, dK += dS^T_x Q_x: A in TMEM (64 queries = 32 columns), B the slot's 64-row tile read MN-major
        auto issue_acc = [&](int x, uint32_t slot, bool accumulate) {
            const uint32_t q_off = (uint32_t)((C::kOffRing + slot * C::kSlotBytes) >> 4), do_off = q_off + (uint32_t)(C::kHalfBytes >> 4);
            const uint32_t a = tmem_u + C::kColR + x * 128;
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                if (elect_one()) mma_ts_parts(tDV, a + kk * 8, mnmaj_lo + do_off + kk * (2048 >> 4), desc_hi, idesc_acc, (accumulate || kk > 0) ? 1u : 0u);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                if (elect_one()) mma_ts_parts(tDK, a + 64 + kk * 8, mnmaj_lo + q_off + kk * (2048 >> 4), desc_hi, idesc_acc, (accumulate || kk > 0) ? 1u : 0u);
            commit_elected(&slot_empty[slot]);
        };
        bool ok = base_ok;
        uint32_t g = 0, n = 0;              // 128-query steps done, key tiles done; chain x of step g uses ring entry 2g + x
        int t = (int)(u_begin % p.key_tiles);
        for (long long u = u_begin; u < u_end && ok; ++u, ++n, t = t + 1 == p.key_tiles ? 0 : t + 1) {
            const int steps = p.q_tiles128 - first_q_tile(p, t);
            ok = __all_sync(0xffffffffu, mbar_wait(kv_full, n & 1, abort_p));
            if (!ok) break;
            for (int x = 0; x < 2 && ok; ++x) {
                const uint32_t hh = 2 * g + x;
                ok = __all_sync(0xffffffffu, mbar_wait(&slot_full[hh % C::kSlots], (hh / C::kSlots) & 1, abort_p));
                if (!ok) break;
                issue_sdp(x, hh % C::kSlots);
            }
            if (!ok) break;
            if (steps == 1) commit_elected(kv_empty);       // K, V have been read for the last time: the next tile's may load
            for (int s = 0; s < steps && ok; ++s, ++g) {
                const bool have_next = s + 1 < steps;
                for (int x = 0; x < 2 && ok; ++x) {
                    const uint32_t hh = 2 * g + x;
                    ok = __all_sync(0xffffffffu, mbar_wait(&pds_full[x], g & 1, abort_p));
                    if (!ok) break;
                    if (s == 0 && x == 0 && n > 0) {        // the previous key tile's dK, dV must have been read out
                        ok = __all_sync(0xffffffffu, mbar_wait(acc_empty, (n - 1) & 1, abort_p));
                        if (!ok) break;
                    }
                    tc_fence_after();
                    issue_acc(x, hh % C::kSlots, s > 0 || x > 0);
                    if (have_next) {
                        const uint32_t hn = hh + 2;
                        ok = __all_sync(0xffffffffu, mbar_wait(&slot_full[hn % C::kSlots], (hn / C::kSlots) & 1, abort_p));
                        if (!ok) break;
                        issue_sdp(x, hn % C::kSlots);
                    }
                }
                if (!ok) break;
                if (have_next && s + 2 == steps) commit_elected(kv_empty);
            }
            if (!ok) break;
            commit_elected(acc_full);
        }
    } else if (warp < 8) {
        // ------------------------------------------------------------------ elementwise threads
        const int wg = warp >> 2;                              // chain: which 64 queries of every tile
        const int r = (warp & 3) * 32 + lane;                  // key row inside the tile == TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + lane_addr + C::kColR + wg * 128;
        const uint32_t tDP = tS + 64;
        bool ok = base_ok;
        uint32_t g = 0, n = 0;
        int bh = (int)(u_begin / p.key_tiles), t = (int)(u_begin - (long long)bh * p.key_tiles);
        for (long long u = u_begin; u < u_end && ok; ++u, ++n, ++t) {
            if (t == p.key_tiles) {
                t = 0;
                ++bh;
            }
            const int key = t * kTileN + r;
            const int i_first = first_q_tile(p, t);
            const long long shift = (long long)p.N - p.W;       // query q may use key k iff q >= k - shift
            const int q_min = p.causal ? (int)((long long)key - shift) : -0x7fffffff;
            const int q_min_warp = p.causal ? (int)((long long)key - lane + 31 - shift) : -0x7fffffff;   // largest in the warp
            for (int i = i_first; i < p.q_tiles128; ++i, ++g) {
                const uint32_t hh = 2 * g + wg, slot = hh % C::kSlots;
                const float* st = sStats + slot * 128;
                const int q0 = i * kQTile + wg * 64;              // first query of this thread's columns
                ok = __all_sync(0xffffffffu, mbar_wait(&sdp_full[wg], g & 1, abort_p));
                if (!ok) break;
                // already complete (the MMAs waited for it); observing it here orders the bulk-copied lse2 / delta
                // before this thread's reads
                ok = __all_sync(0xffffffffu, mbar_wait(&slot_full[slot], (hh / C::kSlots) & 1, abort_p));
                if (!ok) break;
                tc_fence_after();
                const bool masked = q0 < q_min_warp;              // warp-uniform: some element of some lane is masked
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t sv[32], dv_[32];
                    tmem_ld32_async(tS + h * 32, sv);
                    tmem_ld32_async(tDP + h * 32, dv_);
                    tmem_wait_ld(sv);
                    tmem_wait_ld(dv_);
                    uint32_t pk[16], dk_[16];
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        const float4 l4 = *reinterpret_cast<const float4*>(st + h * 32 + c);
                        const float4 d4 = *reinterpret_cast<const float4*>(st + 64 + h * 32 + c);
                        const float lv[4] = {l4.x, l4.y, l4.z, l4.w}, dlv[4] = {d4.x, d4.y, d4.z, d4.w};
                        float pe[4], de[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            pe[e] = ex2(fmaf(__uint_as_float(sv[c + e]), p.scale_log2e, -lv[e]));
                            if (masked && q0 + h * 32 + c + e < q_min) pe[e] = 0.f;
                            de[e] = pe[e] * (__uint_as_float(dv_[c + e]) - dlv[e]);
                        }
                        pk[c / 2] = pack_bf16x2(pe[0], pe[1]);
                        pk[c / 2 + 1] = pack_bf16x2(pe[2], pe[3]);
                        dk_[c / 2] = pack_bf16x2(de[0], de[1]);
                        dk_[c / 2 + 1] = pack_bf16x2(de[2], de[3]);
                    }
                    // bf16 P^T over columns of S^T, dS^T over columns of dP^T, that are already in registers
                    tmem_st16(tS + h * 16, pk);
                    tmem_st16(tDP + h * 16, dk_);
                }
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(&pds_full[wg]);
            }
            if (!ok) break;
            // ---------------------------------------------------------------- dK, dV of this key tile
            ok = __all_sync(0xffffffffu, mbar_wait(acc_full, n & 1, abort_p));
            if (!ok) break;
            tc_fence_after();
            // Each thread holds half a row (D/2 columns) of dK and of dV.  Written straight from the registers a warp's store
            // would touch 32 different lines; the warp passes its 32 x D bytes through shared memory (16-byte pieces, piece
            // index xor row so that neither side has bank conflicts beyond the minimum) and stores whole lines instead.
            constexpr int kPieces = D / 16;                    // 16-byte pieces per half row
            constexpr int kRowsPerStore = 32 / kPieces;
            uint8_t* stage = smem + C::kOffStage + warp * (32 * D);
            const int key_warp = t * kTileN + (warp & 3) * 32;     // key of lane 0
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const uint32_t tA = tmem_base + lane_addr + (which == 0 ? C::kColDK : C::kColDV) + wg * (D / 2);
                const float f = which == 0 ? p.scale : 1.f;
#pragma unroll
                for (int c = 0; c < D / 64; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tA + c * 32, o);
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(o[v4 * 8 + 0]) * f, __uint_as_float(o[v4 * 8 + 1]) * f);
                        w.y = pack_bf16x2(__uint_as_float(o[v4 * 8 + 2]) * f, __uint_as_float(o[v4 * 8 + 3]) * f);
                        w.z = pack_bf16x2(__uint_as_float(o[v4 * 8 + 4]) * f, __uint_as_float(o[v4 * 8 + 5]) * f);
                        w.w = pack_bf16x2(__uint_as_float(o[v4 * 8 + 6]) * f, __uint_as_float(o[v4 * 8 + 7]) * f);
                        const int piece = c * 4 + v4;
                        *reinterpret_cast<uint4*>(stage + lane * D + ((piece ^ (lane & (kPieces - 1))) << 4)) = w;
                    }
                }
                __syncwarp();
                __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(which == 0 ? p.dk : p.dv) +
                                     ((long long)bh * p.N + key_warp) * D + wg * (D / 2);
#pragma unroll
                for (int it = 0; it < 32 / kRowsPerStore; ++it) {
                    const int rrow = it * kRowsPerStore + lane / kPieces, piece = lane % kPieces;
                    const uint4 w = *reinterpret_cast<const uint4*>(stage + rrow * D + ((piece ^ (rrow & (kPieces - 1))) << 4));
                    if (key_warp + rrow < p.N) *reinterpret_cast<uint4*>(dst + (long long)rrow * D + piece * 8) = w;
                }
                __syncwarp();
            }
            tc_fence_before();
            mbar_arrive(acc_empty);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, base_ok ? (int)TLIN_ERR_TIMEOUT : (int)TLIN_ERR_CUDA);
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------ dK / dV / dQ in one kernel
// The dK/dV kernel with a third accumulating product per chain step: dQ^T_x = K^T dS^T_x goes into the chain's dead dP^T_x
// columns (dS^T_x now sits beside P^T_x over S^T_x), is read back by the chain's threads and added to an fp32 dQ buffer in the
// workspace with reductions in L2.  Scores are computed once: five matrix products per (query, key) pair instead of seven.
// Columns of a chain: [P^T q0-31 | dS^T q0-31 | P^T q32-63 | dS^T q32-63] (16 each, written over S^T_x half by half) and dQ^T_x (64).
template <int D>
__global__ void __launch_bounds__(ACfg<D>::kThreads, 1)
bwd_fused_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do, const BwdParams p) {
    using C = ACfg<D>;
    static_assert(D == 128, "the transposed dQ accumulator needs M = d = 128");
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* sKV = smem + C::kOffKV;          // K, V
    uint8_t* sRing = smem + C::kOffRing;      // [kSlots][Q 64 rows | dout 64 rows]
    float* sStats = reinterpret_cast<float*>(smem + C::kOffStats);   // [kSlots][lse2 64 | delta 64]
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kOffBars);
    uint64_t* kv_full = bars + 0;
    uint64_t* kv_empty = bars + 1;
    uint64_t* sdp_full = bars + 2;    // [2] S^T_x and dP^T_x of a step are in TMEM
    uint64_t* pds_full = bars + 4;    // [2] the chain's threads have stored P^T_x and dS^T_x
    uint64_t* acc_full = bars + 6;    // dK, dV of the key tile are complete
    uint64_t* acc_empty = bars + 7;   // all threads have read them
    uint64_t* slot_full = bars + 8;   // [kSlots]
    uint64_t* slot_empty = slot_full + C::kSlots;
    uint64_t* dqt_full = bars + C::kNumBars;        // [2] dQ^T_x of a chain step is in TMEM
    uint64_t* dq_drained = dqt_full + 2;            // [2] the chain's threads hold it in registers: its columns are free
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::kNumBars + 4);
    int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool base_ok = (smem_u32(smem) & 1023u) == 0;   // the swizzled tiles need 1024-byte alignment

    if (threadIdx.x == 0) {
        *abort_flag = base_ok ? 0 : 1;
        mbar_init(kv_full, 1);
        mbar_init(kv_empty, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sdp_full[i], 1);
            mbar_init(&pds_full[i], 128);
            mbar_init(&dqt_full[i], 1);
            mbar_init(&dq_drained[i], 128);
        }
        for (int i = 0; i < C::kSlots; ++i) {
            mbar_init(&slot_full[i], 1);
            mbar_init(&slot_empty[i], 1);
        }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, 256);
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == kProducerWarp && lane == 0) {
        prefetch_tensormap(&map_q);
        prefetch_tensormap(&map_k);
        prefetch_tensormap(&map_v);
        prefetch_tensormap(&map_do);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    volatile int* abort_p = abort_flag;

    // The CTAs take the (b,h,key tile) units in turn (CTA c: units c, c + CTAs, ...), so that at any time all of them work on
    // the key tiles of two or three (b,h): the rows of the fp32 dQ buffer they add to, and the Q / dout tiles they read, then
    // stay in L2 whatever the size of the call.  With the window rule the last key tiles of a (b,h) are cheaper; taking units in
    // turn spreads those evenly.
    const long long u_begin = blockIdx.x, u_end = p.total_units, u_step = gridDim.x;

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ TMA producer: Q / dout / row statistics ring
        // The ring runs ahead of the key tiles: the first chain steps of the next key tile are loaded while the
        // current one is still being worked on.
        if (lane == 0) {
            bool ok = base_ok;
            uint32_t hh = 0;                // chain steps (64 queries each) issued
            for (long long u = u_begin; u < u_end && ok; u += u_step) {
                const int bh = (int)(u / p.key_tiles), t = (int)(u - (long long)bh * p.key_tiles);
                const int row_first = first_q_tile(p, t) * kQTile, row_end = p.q_tiles128 * kQTile;
                for (int row = row_first; row < row_end && ok; row += 64, ++hh) {
                    const uint32_t slot = hh % C::kSlots, round = hh / C::kSlots;
                    ok = mbar_wait(&slot_empty[slot], (round & 1) ^ 1, abort_p);
                    if (!ok) break;
                    uint8_t* dst = sRing + slot * C::kSlotBytes;
                    mbar_arrive_expect_tx(&slot_full[slot], C::kSlotBytes + 512);
                    for (int x = 0; x < C::kBoxes; ++x) {
                        tma_load_3d(dst + x * (64 * 128), &map_q, &slot_full[slot], x * 64, row, bh);
                        tma_load_3d(dst + C::kHalfBytes + x * (64 * 128), &map_do, &slot_full[slot], x * 64, row, bh);
                    }
                    bulk_load_1d(sStats + slot * 128, p.lse2 + (long long)bh * p.Wpad + row, 256, &slot_full[slot]);
                    bulk_load_1d(sStats + slot * 128 + 64, p.delta + (long long)bh * p.Wpad + row, 256, &slot_full[slot]);
                }
            }
            if (!ok && base_ok) {
                int dummy = 0;              // leave no copy in flight: the barriers armed last must complete (bounded)
                for (uint32_t back = 1; back <= (uint32_t)C::kSlots && back <= hh; ++back) {
                    const uint32_t id = hh - back;
                    mbar_wait(&slot_full[id % C::kSlots], (id / C::kSlots) & 1, &dummy, 200000000LL);
                }
            }
        }
    } else if (warp == kKvWarp) {
        // ------------------------------------------------------------------ TMA producer: K, V of the key tiles
        if (lane == 0) {
            bool ok = base_ok;
            uint32_t n = 0;
            for (long long u = u_begin; u < u_end && ok; u += u_step, ++n) {
                const int bh = (int)(u / p.key_tiles), t = (int)(u - (long long)bh * p.key_tiles);
                if (u + u_step < u_end) {   // K, V have one buffer: the next tile's rows come as far as L2 meanwhile
                    const int bh_n = (int)((u + u_step) / p.key_tiles), t_n = (int)(u + u_step - (long long)bh_n * p.key_tiles);
                    for (int x = 0; x < C::kBoxes; ++x) {
                        tma_prefetch_l2_3d(&map_k, x * 64, t_n * kTileN, bh_n);
                        tma_prefetch_l2_3d(&map_v, x * 64, t_n * kTileN, bh_n);
                    }
                }
                ok = mbar_wait(kv_empty, (n & 1) ^ 1, abort_p);
                if (!ok) break;
                mbar_arrive_expect_tx(kv_full, 2 * C::kTileBytes);
                for (int x = 0; x < C::kBoxes; ++x) {
                    tma_load_3d(sKV + x * (kQTile * 128), &map_k, kv_full, x * 64, t * kTileN, bh);
                    tma_load_3d(sKV + C::kTileBytes + x * (kQTile * 128), &map_v, kv_full, x * 64, t * kTileN, bh);
                }
            }
            if (!ok && base_ok && n > 0) {
                int dummy = 0;
                mbar_wait(kv_full, (n - 1) & 1, &dummy, 200000000LL);
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer (all lanes walk, one issues)
        const uint32_t idesc_st = make_idesc_bf16(kQTile, 64, 0, 0);         // S^T, dP^T of a chain: M = keys, N = 64 queries
        const uint32_t idesc_acc = make_idesc_bf16(kQTile, D, 0, 1);         // dV, dK: A in TMEM, B MN-major
        const uint32_t idesc_dqt = make_idesc_bf16(D, 64, 1, 1);             // dQ^T_x = K^T dS^T_x: M = d, N = 64 queries, K = keys; both MN-major
        const uint64_t kmaj = make_smem_desc_sw128(smem_u32(smem), 16, 1024);
        const uint64_t mnmaj = make_smem_desc_sw128(smem_u32(smem), 64 * 128, 1024);   // 64-row tiles: 8 KB between column blocks
        const uint32_t desc_hi = (uint32_t)(kmaj >> 32);
        const uint32_t kmaj_lo = (uint32_t)kmaj, mnmaj_lo = (uint32_t)mnmaj;
        const uint32_t mnmaj128_lo = (uint32_t)make_smem_desc_sw128(smem_u32(smem), kQTile * 128, 1024);   // 128-row tile: 16 KB between column blocks
        const uint32_t ds_off = (uint32_t)(C::kOffStage >> 4);              // dS^T_x tiles: chain x at + x * 16 KB
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t tDK = tmem_u + C::kColDK, tDV = tmem_u + C::kColDV;
        const uint32_t k_off = (uint32_t)(C::kOffKV >> 4), v_off = (uint32_t)((C::kOffKV + C::kTileBytes) >> 4);
        // [S^T_x | dP^T_x] = [K Q_x^T | V dout_x^T]: A a 128-row K-major tile, B the 64-row K-major tile of the slot
        auto issue_sdp = [&](int x, uint32_t slot) {
            const uint32_t q_off = (uint32_t)((C::kOffRing + slot * C::kSlotBytes) >> 4), do_off = q_off + (uint32_t)(C::kHalfBytes >> 4);
            const uint32_t d = tmem_u + C::kColR + x * 128;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t a16 = ((kk >> 2) * (kQTile * 128) + (kk & 3) * 32) >> 4, b16 = ((kk >> 2) * (64 * 128) + (kk & 3) * 32) >> 4;
                if (elect_one()) mma_ss_parts(d, kmaj_lo + k_off + a16, kmaj_lo + q_off + b16, desc_hi, idesc_st, kk > 0);
            }
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t a16 = ((kk >> 2) * (kQTile * 128) + (kk & 3) * 32) >> 4, b16 = ((kk >> 2) * (64 * 128) + (kk & 3) * 32) >> 4;
                if (elect_one()) mma_ss_parts(d + 64, kmaj_lo + v_off + a16, kmaj_lo + do_off + b16, desc_hi, idesc_st, kk > 0);
            }
            commit_elected(&sdp_full[x]);
        };
        // dV += P^T_x dout_x, dK += dS^T_x Q_x: A in TMEM (64 queries = 32 columns), B the slot's 64-row tile read MN-major
        auto issue_acc = [&](int x, uint32_t slot, bool accumulate) {
            const uint32_t q_off = (uint32_t)((C::kOffRing + slot * C::kSlotBytes) >> 4), do_off = q_off + (uint32_t)(C::kHalfBytes >> 4);
            const uint32_t a = tmem_u + C::kColR + x * 128;
            // dQ^T_x (d x 64 queries, over the dead dP^T_x columns) = K^T (the K tile read MN-major) dS^T_x (shared memory,
            // MN-major); first, so that the chain's threads can take it away while dV and dK are in the pipe
#pragma unroll
            for (int kk = 0; kk < kTileN / 16; ++kk)
                if (elect_one()) mma_ss_parts(a + 64, mnmaj128_lo + k_off + kk * (2048 >> 4), mnmaj_lo + ds_off + x * (16384 >> 4) + kk * (2048 >> 4),
                                              desc_hi, idesc_dqt, kk > 0 ? 1u : 0u);
            commit_elected(&dqt_full[x]);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                if (elect_one()) mma_ts_parts(tDV, a + (kk >> 1) * 32 + (kk & 1) * 8, mnmaj_lo + do_off + kk * (2048 >> 4), desc_hi, idesc_acc, (accumulate || kk > 0) ? 1u : 0u);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                if (elect_one()) mma_ts_parts(tDK, a + (kk >> 1) * 32 + 16 + (kk & 1) * 8, mnmaj_lo + q_off + kk * (2048 >> 4), desc_hi, idesc_acc, (accumulate || kk > 0) ? 1u : 0u);
            commit_elected(&slot_empty[slot]);
        };
        bool ok = base_ok;
        uint32_t g = 0, n = 0;              // 128-query steps done, key tiles done; chain x of step g uses ring entry 2g + x
        for (long long u = u_begin; u < u_end && ok; u += u_step, ++n) {
            const int t = (int)(u % p.key_tiles);
            const int steps = p.q_tiles128 - first_q_tile(p, t);
            ok = __all_sync(0xffffffffu, mbar_wait(kv_full, n & 1, abort_p));
            if (!ok) break;
            for (int x = 0; x < 2 && ok; ++x) {
                const uint32_t hh = 2 * g + x;
                ok = __all_sync(0xffffffffu, mbar_wait(&slot_full[hh % C::kSlots], (hh / C::kSlots) & 1, abort_p));
                if (!ok) break;
                if (g > 0) {                                // dP^T_x is written over the chain's previous dQ^T_x
                    ok = __all_sync(0xffffffffu, mbar_wait(&dq_drained[x], (g - 1) & 1, abort_p));
                    if (!ok) break;
                }
                issue_sdp(x, hh % C::kSlots);
            }
            if (!ok) break;
            for (int s = 0; s < steps && ok; ++s, ++g) {
                const bool have_next = s + 1 < steps;
                for (int x = 0; x < 2 && ok; ++x) {
                    const uint32_t hh = 2 * g + x;
                    ok = __all_sync(0xffffffffu, mbar_wait(&pds_full[x], g & 1, abort_p));
                    if (!ok) break;
                    if (s == 0 && x == 0 && n > 0) {        // the previous key tile's dK, dV must have been read out
                        ok = __all_sync(0xffffffffu, mbar_wait(acc_empty, (n - 1) & 1, abort_p));
                        if (!ok) break;
                    }
                    tc_fence_after();
                    issue_acc(x, hh % C::kSlots, s > 0 || x > 0);
                }
                if (!ok) break;
                if (!have_next) commit_elected(kv_empty);   // K (read by the dQ^T products) and V are free for the next key tile
                // the next score products of a chain overwrite its dQ^T_x: they follow its drain, which runs while the
                // other chain's products are in the pipe
                for (int x = 0; x < 2 && ok && have_next; ++x) {
                    const uint32_t hn = 2 * g + x + 2;
                    ok = __all_sync(0xffffffffu, mbar_wait(&slot_full[hn % C::kSlots], (hn / C::kSlots) & 1, abort_p));
                    if (!ok) break;
                    ok = __all_sync(0xffffffffu, mbar_wait(&dq_drained[x], g & 1, abort_p));
                    if (!ok) break;
                    tc_fence_after();
                    issue_sdp(x, hn % C::kSlots);
                }
                if (!ok) break;
            }
            if (!ok) break;
            commit_elected(acc_full);
        }
    } else if (warp < 8) {
        // ------------------------------------------------------------------ elementwise threads
        const int wg = warp >> 2;                              // chain: which 64 queries of every tile
        const int r = (warp & 3) * 32 + lane;                  // key row inside the tile == TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + lane_addr + C::kColR + wg * 128;
        const uint32_t tDP = tS + 64;
        bool ok = base_ok;
        // the second half of a step's dQ^T_x values waits in registers and is handed to L2 while the next step's products run
        uint32_t held[32];
        float* held_row = nullptr;
        uint32_t g = 0, n = 0;
        for (long long u = u_begin; u < u_end && ok; u += u_step, ++n) {
            const int bh = (int)(u / p.key_tiles), t = (int)(u - (long long)bh * p.key_tiles);
            const int key = t * kTileN + r;
            const int i_first = first_q_tile(p, t);
            const long long shift = (long long)p.N - p.W;       // query q may use key k iff q >= k - shift
            const int q_min = p.causal ? (int)((long long)key - shift) : -0x7fffffff;
            const int q_min_warp = p.causal ? (int)((long long)key - lane + 31 - shift) : -0x7fffffff;   // largest in the warp
            for (int i = i_first; i < p.q_tiles128; ++i, ++g) {
                const uint32_t hh = 2 * g + wg, slot = hh % C::kSlots;
                const float* st = sStats + slot * 128;
                const int q0 = i * kQTile + wg * 64;              // first query of this thread's columns
                ok = __all_sync(0xffffffffu, mbar_wait(&sdp_full[wg], g & 1, abort_p));
                if (!ok) break;
                // already complete (the MMAs waited for it); observing it here orders the bulk-copied lse2 / delta
                // before this thread's reads
                ok = __all_sync(0xffffffffu, mbar_wait(&slot_full[slot], (hh / C::kSlots) & 1, abort_p));
                if (!ok) break;
                tc_fence_after();
                const bool masked = q0 < q_min_warp;              // warp-uniform: some element of some lane is masked
                // 32 queries at a time: P^T and dS^T of a half go over the 32 columns of S^T_x that have just been read
                uint8_t* ds_row = smem + C::kOffStage + wg * 16384 + r * 128;       // this key's row of the dS^T_x tile
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t sv[32], dv_[32];
                    tmem_ld32_async(tS + h * 32, sv);
                    tmem_ld32_async(tDP + h * 32, dv_);
                    tmem_wait_ld(sv);
                    tmem_wait_ld(dv_);
                    uint32_t pk[16], dk_[16];
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        const float4 l4 = *reinterpret_cast<const float4*>(st + h * 32 + c);
                        const float4 d4 = *reinterpret_cast<const float4*>(st + 64 + h * 32 + c);
                        const float lv[4] = {l4.x, l4.y, l4.z, l4.w}, dlv[4] = {d4.x, d4.y, d4.z, d4.w};
                        float pe[4], de[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            pe[e] = ex2(fmaf(__uint_as_float(sv[c + e]), p.scale_log2e, -lv[e]));
                            if (masked && q0 + h * 32 + c + e < q_min) pe[e] = 0.f;
                            de[e] = pe[e] * (__uint_as_float(dv_[c + e]) - dlv[e]);
                        }
                        pk[c / 2] = pack_bf16x2(pe[0], pe[1]);
                        pk[c / 2 + 1] = pack_bf16x2(pe[2], pe[3]);
                        dk_[c / 2] = pack_bf16x2(de[0], de[1]);
                        dk_[c / 2 + 1] = pack_bf16x2(de[2], de[3]);
                    }
                    tmem_st16(tS + h * 32, pk);
                    tmem_st16(tS + h * 32 + 16, dk_);
                    // and dS^T_x once more as the B operand of the dQ^T product: row = key, 64 queries = 128 bytes, 16-byte
                    // pieces at (piece xor row mod 8), the layout the 128-byte swizzle of the descriptors expects
#pragma unroll
                    for (int c4 = 0; c4 < 4; ++c4)
                        *reinterpret_cast<uint4*>(ds_row + (((h * 4 + c4) ^ (r & 7)) << 4)) =
                            make_uint4(dk_[c4 * 4], dk_[c4 * 4 + 1], dk_[c4 * 4 + 2], dk_[c4 * 4 + 3]);
                }
                tc_wait_st();
                fence_proxy_async_smem();             // the tile was written with ordinary stores and is read by the MMA
                tc_fence_before();
                mbar_arrive(&pds_full[wg]);
                // ------------------------------------------------------------ dQ^T_x -> fp32 dQ (reductions in L2)
                // For one query the 32 lanes of a warp hold 32 consecutive floats of its row of the fp32 dQ buffer: one
                // reduction instruction adds 128 consecutive bytes.  The half kept from the previous step goes first, while
                // this step's products are in the pipe.
                if (held_row != nullptr) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) atomicAdd(held_row + (long long)e * D, __uint_as_float(held[e]));
                }
                ok = __all_sync(0xffffffffu, mbar_wait(&dqt_full[wg], g & 1, abort_p));
                if (!ok) break;
                tc_fence_after();
                // TMEM lane = column of dQ (this thread: r), TMEM column = query.  Once the values are in registers the columns
                // are free for the chain's next score products.
                uint32_t o[32];
                tmem_ld32_async(tDP, o);
                tmem_ld32_async(tDP + 32, held);
                tmem_wait_ld(o);
                tmem_wait_ld(held);
                tc_fence_before();
                mbar_arrive(&dq_drained[wg]);
                float* drow = p.ws + ((long long)bh * p.Wpad + q0) * D + r;
#pragma unroll
                for (int e = 0; e < 32; ++e) atomicAdd(drow + (long long)e * D, __uint_as_float(o[e]));
                held_row = drow + 32LL * D;
            }
            if (!ok) break;
            // ---------------------------------------------------------------- dK, dV of this key tile
            ok = __all_sync(0xffffffffu, mbar_wait(acc_full, n & 1, abort_p));
            if (!ok) break;
            tc_fence_after();
            // Each thread holds half a row (D/2 columns) of dK and of dV.  Written straight from the registers a warp's store
            // would touch 32 different lines; the warp passes its 32 x D bytes through shared memory (16-byte pieces, piece
            // index xor row so that neither side has bank conflicts beyond the minimum) and stores whole lines instead.
            constexpr int kPieces = D / 16;                    // 16-byte pieces per half row
            constexpr int kRowsPerStore = 32 / kPieces;
            uint8_t* stage = smem + C::kOffStage + warp * (32 * D);
            const int key_warp = t * kTileN + (warp & 3) * 32;     // key of lane 0
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const uint32_t tA = tmem_base + lane_addr + (which == 0 ? C::kColDK : C::kColDV) + wg * (D / 2);
                const float f = which == 0 ? p.scale : 1.f;
#pragma unroll
                for (int c = 0; c < D / 64; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tA + c * 32, o);
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(o[v4 * 8 + 0]) * f, __uint_as_float(o[v4 * 8 + 1]) * f);
                        w.y = pack_bf16x2(__uint_as_float(o[v4 * 8 + 2]) * f, __uint_as_float(o[v4 * 8 + 3]) * f);
                        w.z = pack_bf16x2(__uint_as_float(o[v4 * 8 + 4]) * f, __uint_as_float(o[v4 * 8 + 5]) * f);
                        w.w = pack_bf16x2(__uint_as_float(o[v4 * 8 + 6]) * f, __uint_as_float(o[v4 * 8 + 7]) * f);
                        const int piece = c * 4 + v4;
                        *reinterpret_cast<uint4*>(stage + lane * D + ((piece ^ (lane & (kPieces - 1))) << 4)) = w;
                    }
                }
                __syncwarp();
                __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(which == 0 ? p.dk : p.dv) +
                                     ((long long)bh * p.N + key_warp) * D + wg * (D / 2);
#pragma unroll
                for (int it = 0; it < 32 / kRowsPerStore; ++it) {
                    const int rrow = it * kRowsPerStore + lane / kPieces, piece = lane % kPieces;
                    const uint4 w = *reinterpret_cast<const uint4*>(stage + rrow * D + ((piece ^ (rrow & (kPieces - 1))) << 4));
                    if (key_warp + rrow < p.N) *reinterpret_cast<uint4*>(dst + (long long)rrow * D + piece * 8) = w;
                }
                __syncwarp();
            }
            tc_fence_before();
            mbar_arrive(acc_empty);
        }
        if (held_row != nullptr) {
#pragma unroll
            for (int e = 0; e < 32; ++e) atomicAdd(held_row + (long long)e * D, __uint_as_float(held[e]));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, base_ok ? (int)TLIN_ERR_TIMEOUT : (int)TLIN_ERR_CUDA);
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------ dQ
template <int D>
struct BCfg {
    static constexpr int kTileBytes = kQTile * D * 2;
    static constexpr int kBoxes = D / 64;
    static constexpr int kKSlots = D == 128 ? 2 : 4;           // K tiles live for a whole step (S, then dQ)
    static constexpr int kVSlots = D == 128 ? 1 : 2;           // V tiles only for the dP MMAs
    static constexpr int kOffQ = 0;                            // 2 tiles
    static constexpr int kOffDO = 2 * kTileBytes;              // 2 tiles
    static constexpr int kOffK = 4 * kTileBytes;
    static constexpr int kOffV = (4 + kKSlots) * kTileBytes;
    static constexpr int kOffBars = (4 + kKSlots + kVSlots) * kTileBytes;
    static constexpr int kNumBars = 11 + 2 * kKSlots + 2 * kVSlots;
    static constexpr int kSmemBytes = kOffBars + kNumBars * 8 + 32;   // + TMEM slot, abort flag, unit range
    // TMEM columns: R0, R1 (S, then dP, then dS as bf16; 128 each), dQ0, dQ1 (D each)
    static constexpr uint32_t kColR = 0, kColDQ = 256;
    static constexpr int kThreads = 32 * 12;                   // warps 10 and 11 only lend their registers
    // setmaxnreg moves registers between warpgroups; the CTA starts with 168 per thread (65536 / 384, rounded down to a
    // multiple of 8), and an increase beyond what the other warpgroup released would wait for ever
    static constexpr int kComputeRegs = 200, kOtherRegs = 104;
    static_assert(256 * kComputeRegs + 128 * kOtherRegs <= kThreads * 168, "register budget of the CTA exceeded");
};

template <int D>
__global__ void __launch_bounds__(BCfg<D>::kThreads, 1)
bwd_dq_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do, const BwdParams p,
                 const __grid_constant__ GroupStarts starts) {
    using C = BCfg<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* sQ = smem + C::kOffQ;
    uint8_t* sDO = smem + C::kOffDO;
    uint8_t* sK = smem + C::kOffK;
    uint8_t* sV = smem + C::kOffV;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kOffBars);
    uint64_t* qdo_full = bars + 0;
    uint64_t* qdo_empty = bars + 1;
    uint64_t* dq_done = bars + 2;
    uint64_t* s_full = bars + 3;      // [2]
    uint64_t* p_ready = bars + 5;     // [2]  every thread of the tile has read S
    uint64_t* dp_full = bars + 7;     // [2]
    uint64_t* ds_full = bars + 9;     // [2]
    uint64_t* k_full = bars + 11;
    uint64_t* k_empty = k_full + C::kKSlots;
    uint64_t* v_full = k_empty + C::kKSlots;
    uint64_t* v_empty = v_full + C::kVSlots;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::kNumBars);
    int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool base_ok = (smem_u32(smem) & 1023u) == 0;

    if (threadIdx.x == 0) {
        *abort_flag = base_ok ? 0 : 1;
        mbar_init(qdo_full, 1);
        mbar_init(qdo_empty, 1);
        mbar_init(dq_done, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s_full[i], 1);
            mbar_init(&p_ready[i], kQTile);
            mbar_init(&dp_full[i], 1);
            mbar_init(&ds_full[i], kQTile);
        }
        for (int s = 0; s < C::kKSlots; ++s) {
            mbar_init(&k_full[s], 1);
            mbar_init(&k_empty[s], 1);
        }
        for (int s = 0; s < C::kVSlots; ++s) {
            mbar_init(&v_full[s], 1);
            mbar_init(&v_empty[s], 1);
        }
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == kProducerWarp && lane == 0) {
        prefetch_tensormap(&map_q);
        prefetch_tensormap(&map_k);
        prefetch_tensormap(&map_v);
        prefetch_tensormap(&map_do);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    volatile int* abort_p = abort_flag;

    if (warp >= 8) {
    setmaxnreg_dec<C::kOtherRegs>();
    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t kit = 0, vit = 0, seg_idx = 0;
            bool ok = base_ok;
            SegmentWalker walk(p, starts);
            Segment s;
            while (ok && walk.next(s)) {
                const int row0 = s.qt * kTileM;
                const int c0 = seg_count(s, tiles_allowed(p, row0, 0)), c1 = seg_count(s, tiles_allowed(p, row0, 1));
                const int cnt = c0 > c1 ? c0 : c1;
                if (cnt == 0) continue;
                if (seg_idx > 0) ok = mbar_wait(qdo_empty, (seg_idx - 1) & 1, abort_p);
                if (!ok) break;
                mbar_arrive_expect_tx(qdo_full, 4 * C::kTileBytes);
                for (int i = 0; i < 2; ++i)
                    for (int x = 0; x < C::kBoxes; ++x) {
                        tma_load_3d(sQ + i * C::kTileBytes + x * (kQTile * 128), &map_q, qdo_full, x * 64, row0 + i * kQTile, s.bh);
                        tma_load_3d(sDO + i * C::kTileBytes + x * (kQTile * 128), &map_do, qdo_full, x * 64, row0 + i * kQTile, s.bh);
                    }
                for (int j = 0; j < cnt && ok; ++j) {
                    const int t = s.t_begin + j;
                    {
                        const uint32_t slot = kit % C::kKSlots, round = kit / C::kKSlots;
                        ok = mbar_wait(&k_empty[slot], (round & 1) ^ 1, abort_p);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&k_full[slot], C::kTileBytes);
                        for (int x = 0; x < C::kBoxes; ++x)
                            tma_load_3d(sK + slot * C::kTileBytes + x * (kQTile * 128), &map_k, &k_full[slot], x * 64, t * kTileN, s.bh);
                        ++kit;
                    }
                    {
                        const uint32_t slot = vit % C::kVSlots, round = vit / C::kVSlots;
                        ok = mbar_wait(&v_empty[slot], (round & 1) ^ 1, abort_p);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&v_full[slot], C::kTileBytes);
                        for (int x = 0; x < C::kBoxes; ++x)
                            tma_load_3d(sV + slot * C::kTileBytes + x * (kQTile * 128), &map_v, &v_full[slot], x * 64, t * kTileN, s.bh);
                        ++vit;
                    }
                }
                ++seg_idx;
            }
            if (!ok && base_ok) {
                int dummy = 0;          // leave no copy in flight: what was armed last must land (bounded)
                for (uint32_t back = 0; back < (uint32_t)C::kKSlots && back < kit; ++back) {
                    const uint32_t id = kit - 1 - back;
                    mbar_wait(&k_full[id % C::kKSlots], (id / C::kKSlots) & 1, &dummy, 200000000LL);
                }
                for (uint32_t back = 0; back < (uint32_t)C::kVSlots && back < vit; ++back) {
                    const uint32_t id = vit - 1 - back;
                    mbar_wait(&v_full[id % C::kVSlots], (id / C::kVSlots) & 1, &dummy, 200000000LL);
                }
                if (seg_idx > 0) mbar_wait(qdo_full, (seg_idx - 1) & 1, &dummy, 200000000LL);
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer (all lanes walk, one issues)
        const uint32_t idesc_s = make_idesc_bf16(kQTile, kTileN, 0, 0);      // S, dP: M = queries, N = keys
        const uint32_t idesc_dq = make_idesc_bf16(kQTile, D, 0, 1);          // dQ: A = dS in TMEM, B = K MN-major
        const uint64_t kmaj = make_smem_desc_sw128(smem_u32(smem), 16, 1024);
        const uint64_t mnmaj = make_smem_desc_sw128(smem_u32(smem), kQTile * 128, 1024);
        const uint32_t desc_hi = (uint32_t)(kmaj >> 32);
        const uint32_t kmaj_lo = (uint32_t)kmaj, mnmaj_lo = (uint32_t)mnmaj;
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
        auto issue_r = [&](int i, int a_byte_off, int b_byte_off) {        // R_i = A B^T (contraction over d)
            const uint32_t a_lo = kmaj_lo + (uint32_t)(a_byte_off >> 4), b_lo = kmaj_lo + (uint32_t)(b_byte_off >> 4);
            const uint32_t d = tmem_u + C::kColR + i * kTileN;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off16 = ((kk >> 2) * (kQTile * 128) + (kk & 3) * 32) >> 4;
                if (elect_one()) mma_ss_parts(d, a_lo + off16, b_lo + off16, desc_hi, idesc_s, kk > 0);
            }
        };
        auto issue_dq = [&](int i, int k_byte_off, bool accumulate) {       // dQ_i += dS_i K (contraction over keys)
            const uint32_t b_lo = mnmaj_lo + (uint32_t)(k_byte_off >> 4);
            const uint32_t d = tmem_u + C::kColDQ + i * D, a = tmem_u + C::kColR + i * kTileN;
#pragma unroll
            for (int kk = 0; kk < kTileN / 16; ++kk)
                if (elect_one()) mma_ts_parts(d, a + kk * 8, b_lo + kk * (2048 >> 4), desc_hi, idesc_dq, (accumulate || kk > 0) ? 1u : 0u);
        };
        uint32_t kit = 0, vit = 0, seg_idx = 0;
        uint32_t n_step[2] = {0, 0};
        bool ok = base_ok;
        SegmentWalker walk(p, starts);
        Segment s;
        while (ok && walk.next(s)) {
            const int row0 = s.qt * kTileM;
            const int c0 = seg_count(s, tiles_allowed(p, row0, 0)), c1 = seg_count(s, tiles_allowed(p, row0, 1));
            const int cnt = c0 > c1 ? c0 : c1;
            if (cnt == 0) continue;
            const int cq[2] = {c0, c1};
            ok = __all_sync(0xffffffffu, mbar_wait(qdo_full, seg_idx & 1, abort_p));
            if (!ok) break;
            uint32_t ks = kit % C::kKSlots;
            ok = __all_sync(0xffffffffu, mbar_wait(&k_full[ks], (kit / C::kKSlots) & 1, abort_p));
            if (!ok) break;
            tc_fence_after();
            for (int i = 0; i < 2; ++i)
                if (cq[i] > 0) {
                    issue_r(i, C::kOffQ + i * C::kTileBytes, C::kOffK + ks * C::kTileBytes);
                    commit_elected(&s_full[i]);
                }
            for (int j = 0; j < cnt && ok; ++j) {
                const uint32_t vs = vit % C::kVSlots;
                ok = __all_sync(0xffffffffu, mbar_wait(&v_full[vs], (vit / C::kVSlots) & 1, abort_p));
                if (!ok) break;
                ++vit;
                for (int i = 0; i < 2 && ok; ++i) {
                    if (j < cq[i]) {
                        ok = __all_sync(0xffffffffu, mbar_wait(&p_ready[i], n_step[i] & 1, abort_p));
                        if (!ok) break;
                        tc_fence_after();
                        issue_r(i, C::kOffDO + i * C::kTileBytes, C::kOffV + vs * C::kTileBytes);   // dP over S
                        commit_elected(&dp_full[i]);
                    }
                }
                if (!ok) break;
                commit_elected(&v_empty[vs]);
                const bool have_next = j + 1 < cnt;
                if (!have_next) commit_elected(qdo_empty);       // Q and dout of this segment have been read for the last time
                uint32_t nks = 0;
                if (have_next) {
                    nks = (kit + 1) % C::kKSlots;
                    ok = __all_sync(0xffffffffu, mbar_wait(&k_full[nks], ((kit + 1) / C::kKSlots) & 1, abort_p));
                    if (!ok) break;
                }
                for (int i = 0; i < 2 && ok; ++i) {
                    if (j < cq[i]) {
                        ok = __all_sync(0xffffffffu, mbar_wait(&ds_full[i], n_step[i] & 1, abort_p));
                        if (!ok) break;
                        tc_fence_after();
                        issue_dq(i, C::kOffK + ks * C::kTileBytes, j > 0);
                        ++n_step[i];
                    }
                    if (have_next && j + 1 < cq[i]) {
                        tc_fence_after();
                        issue_r(i, C::kOffQ + i * C::kTileBytes, C::kOffK + nks * C::kTileBytes);
                        commit_elected(&s_full[i]);
                    }
                }
                if (!ok) break;
                commit_elected(&k_empty[ks]);
                ++kit;
                ks = nks;
            }
            if (!ok) break;
            commit_elected(dq_done);
            ++seg_idx;
        }
    }
    } else {
        // ------------------------------------------------------------------ elementwise warpgroups (one per Q tile)
        setmaxnreg_inc<C::kComputeRegs>();
        const int i = warp >> 2;
        const int r = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tR = tmem_base + lane_addr + C::kColR + i * kTileN;
        const uint32_t tDQ = tmem_base + lane_addr + C::kColDQ + i * D;
        uint32_t n = 0, seg_idx = 0;
        bool ok = base_ok;
        SegmentWalker walk(p, starts);
        const int bh_first = (int)(walk.u / p.key_tiles);     // (b,h) of this CTA's first unit (used under schedule 0 only)
        Segment s;
        while (ok && walk.next(s)) {
            const int row0 = s.qt * kTileM;
            const int row = row0 + i * kQTile + r;
            const int a0 = tiles_allowed(p, row0, 0), a1 = tiles_allowed(p, row0, 1);
            const int c0 = seg_count(s, a0), c1 = seg_count(s, a1);
            // No tile of the segment is visible to either Q tile: the MMA warp and the producer skip it and it takes no
            // barrier phase, but its partial slot is still read by the reduce kernel and has to hold zeros.
            const bool skipped = (c0 > c1 ? c0 : c1) == 0;
            const int allowed_i = i == 0 ? a0 : a1, cnt_i = i == 0 ? c0 : c1;
            const long long lim_row_ll = p.causal ? (long long)p.N - p.W + row + 1 : (long long)p.N;
            const int lim_row = (int)(lim_row_ll < p.N ? lim_row_ll : p.N);
            const long long lim_warp_ll = p.causal ? (long long)p.N - p.W + (row - lane) + 1 : (long long)p.N;
            const int lim_warp = (int)(lim_warp_ll < p.N ? lim_warp_ll : p.N);
            const bool row_ok = row < p.W;
            const float l2 = row_ok ? p.lse2[(long long)s.bh * p.Wpad + row] : CUDART_INF_F;
            const float dl = row_ok ? p.delta[(long long)s.bh * p.Wpad + row] : 0.f;
            for (int j = 0; j < cnt_i; ++j) {
                ok = __all_sync(0xffffffffu, mbar_wait(&s_full[i], n & 1, abort_p));
                if (!ok) break;
                tc_fence_after();
                const int k0 = (s.t_begin + j) * kTileN;
                const bool masked = k0 + kTileN > lim_warp;
                const int nvalid = lim_row - k0;
                uint32_t sv[kTileN / 32][32];
#pragma unroll
                for (int c = 0; c < kTileN / 32; ++c) tmem_ld32_async(tR + c * 32, sv[c]);
#pragma unroll
                for (int c = 0; c < kTileN / 32; ++c) tmem_wait_ld(sv[c]);
                tc_fence_before();
                mbar_arrive(&p_ready[i]);                      // S is in registers: dP may overwrite it
                // p = 2^(s*scale*log2e - lse*log2e), kept as fp32 in the registers that held s
#pragma unroll
                for (int e = 0; e < kTileN; ++e) {
                    float pe = ex2(fmaf(__uint_as_float(sv[e >> 5][e & 31]), p.scale_log2e, -l2));
                    if (masked && e >= nvalid) pe = 0.f;
                    sv[e >> 5][e & 31] = __float_as_uint(pe);
                }
                ok = __all_sync(0xffffffffu, mbar_wait(&dp_full[i], n & 1, abort_p));
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < kTileN / 16; ++c) {
                    uint32_t dp[16];
                    tmem_ld16_async(tR + c * 16, dp);
                    tmem_wait_ld16(dp);
                    uint32_t pk[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const float d0 = __uint_as_float(sv[c >> 1][(c & 1) * 16 + 2 * e]) * (__uint_as_float(dp[2 * e]) - dl);
                        const float d1 = __uint_as_float(sv[c >> 1][(c & 1) * 16 + 2 * e + 1]) * (__uint_as_float(dp[2 * e + 1]) - dl);
                        pk[e] = pack_bf16x2(d0, d1);
                    }
                    tmem_st8(tR + c * 8, pk);                 // bf16 dS over columns of dP that are already in registers
                }
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(&ds_full[i]);
                ++n;
            }
            if (!ok) break;
            const uint32_t my_seg = seg_idx;
            if (!skipped) ++seg_idx;
            if (allowed_i == 0) continue;                      // this Q tile does not exist
            // ---------------------------------------------------------------- dQ of the segment
            if (cnt_i > 0) {
                ok = __all_sync(0xffffffffu, mbar_wait(dq_done, my_seg & 1, abort_p));
                if (!ok) break;
                tc_fence_after();
            }
            const bool whole = s.t_begin == 0 && s.t_end == p.key_tiles;
            __nv_bfloat16* drow = reinterpret_cast<__nv_bfloat16*>(p.dq) + ((long long)s.bh * p.W + row) * D;
            // partial sum -> workspace slot (0: first segment of this CTA's range, 1: a later one); unscaled fp32
            float* prow = p.ws + ((long long)blockIdx.x * 2 + (s.bh == bh_first ? 0 : 1)) * (long long)kTileM * D + (long long)(i * kQTile + r) * D;
            const float f = whole ? p.scale : 1.f;
#pragma unroll 1
            for (int c = 0; c < D / 16; ++c) {
                uint32_t o[16];
                if (cnt_i > 0) {
                    tmem_ld16_async(tDQ + c * 16, o);
                    tmem_wait_ld16(o);
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) o[e] = 0u;
                }
                // a thread holds one row: 32-byte stores halve the number of (scattered) store instructions
                // (taken when dq and the workspace are 32-byte aligned; the interface only promises 16)
                if (whole) {
                    if (row_ok) {
                        uint32_t w[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) w[e] = pack_bf16x2(__uint_as_float(o[2 * e]) * f, __uint_as_float(o[2 * e + 1]) * f);
                        if (p.wide_stores) {
                            st_global_v8(drow + c * 16, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
                        } else {
                            *reinterpret_cast<uint4*>(drow + c * 16) = make_uint4(w[0], w[1], w[2], w[3]);
                            *reinterpret_cast<uint4*>(drow + c * 16 + 8) = make_uint4(w[4], w[5], w[6], w[7]);
                        }
                    }
                } else if (p.wide_stores) {
                    st_global_v8(prow + c * 16, o[0], o[1], o[2], o[3], o[4], o[5], o[6], o[7]);
                    st_global_v8(prow + c * 16 + 8, o[8], o[9], o[10], o[11], o[12], o[13], o[14], o[15]);
                } else {
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4)
                        *reinterpret_cast<uint4*>(prow + c * 16 + v4 * 4) = make_uint4(o[v4 * 4], o[v4 * 4 + 1], o[v4 * 4 + 2], o[v4 * 4 + 3]);
                }
            }
            tc_fence_before();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, base_ok ? (int)TLIN_ERR_TIMEOUT : (int)TLIN_ERR_CUDA);
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// Adds the partial dQ of every (b,h) whose key tiles were split between groups, scales and rounds to bf16.
// One CTA per 8 query rows of a (b,h, 256-row tile): one warp per row.
template <int D>
__global__ void __launch_bounds__(256)
bwd_dq_reduce_kernel(const BwdParams p) {
    constexpr int CPL = D / 32;
    const int blocks_per_tile = kTileM / 8;
    const int part = blockIdx.x % blocks_per_tile;
    const int tile_id = blockIdx.x / blocks_per_tile;       // bh * q_tiles + qt
    const int bh = tile_id / p.q_tiles, qt = tile_id - bh * p.q_tiles;
    const unsigned long long T = (unsigned long long)p.key_tiles, U = (unsigned long long)p.total_units, G = (unsigned)p.n_groups;
    // groups holding the first and the last unit of this (b,h): largest g with floor(g*U/G) <= x
    const unsigned long long x0 = (unsigned long long)bh * T, x1 = x0 + T - 1;
    const int g_lo = (int)(((x0 + 1) * G - 1) / U), g_hi = (int)(((x1 + 1) * G - 1) / U);
    if (g_hi == g_lo) return;                               // written directly by the dQ kernel
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rr = part * 8 + warp;
    const int row = qt * kTileM + rr;
    if (row >= p.W) return;
    float acc[CPL];
#pragma unroll
    for (int e = 0; e < CPL; ++e) acc[e] = 0.f;
    for (int g = g_lo; g <= g_hi; ++g) {
        const int cta = g * p.q_tiles + qt;
        const int slot = bh == (int)((((unsigned long long)g * U) / G) / T) ? 0 : 1;
        const float* src = p.ws + ((long long)cta * 2 + slot) * (long long)kTileM * D + (long long)rr * D + lane * CPL;
#pragma unroll
        for (int e = 0; e < CPL; ++e) acc[e] += src[e];
    }
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.dq) + ((long long)bh * p.W + row) * D + lane * CPL;
#pragma unroll
    for (int e = 0; e < CPL; e += 2)
        *reinterpret_cast<uint32_t*>(dst + e) = pack_bf16x2(acc[e] * p.scale, acc[e + 1] * p.scale);
}

// ------------------------------------------------------------------------------------------ host side
template <int D>
int launch_d(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
             void* dq, void* dk, void* dv, int B, int H, int N, int W, int causal, const tlin_fwd_plan& plan,
             float* ws, int num_sms, cudaStream_t st) {
    const long long bh = (long long)B * H;
    const int Wpad = (W + kQTile - 1) / kQTile * kQTile;
    CUtensorMap mq, mk, mv, mdo, mq64, mdo64;
    int rc = make_map(&mq, q, D, W, bh);
    if (rc == TLIN_OK) rc = make_map(&mk, k, D, N, bh);
    if (rc == TLIN_OK) rc = make_map(&mv, v, D, N, bh);
    if (rc == TLIN_OK) rc = make_map(&mdo, dout, D, W, bh);
    if (rc == TLIN_OK) rc = make_map(&mq64, q, D, W, bh, 64);
    if (rc == TLIN_OK) rc = make_map(&mdo64, dout, D, W, bh, 64);
    if (rc != TLIN_OK) return rc;
    BwdParams p;
    float* lse2 = ws;
    float* delta = ws + bh * Wpad;
    p.lse2 = lse2; p.delta = delta; p.dq = dq; p.dk = dk; p.dv = dv;
    p.ws = ws + 2 * bh * Wpad;
    p.status = status_word();
    if (!p.status) return TLIN_ERR_CUDA;
    p.key_tiles = (N + kTileN - 1) / kTileN;
    p.q_tiles128 = Wpad / kQTile;
    p.N = N; p.W = W; p.Wpad = Wpad; p.causal = causal;
    p.scale = 1.f / sqrtf((float)D);
    p.scale_log2e = kLog2e * p.scale;
    p.wide_stores = ((reinterpret_cast<uintptr_t>(dq) | reinterpret_cast<uintptr_t>(ws)) & 31u) == 0;
    static bool smem_allowed_a[64] = {}, smem_allowed_b[64] = {};
    TLIN_CUDA_CHECK(allow_dynamic_smem(bwd_dkdv_tc_kernel<D>, ACfg<D>::kSmemBytes, smem_allowed_a));
    TLIN_CUDA_CHECK(allow_dynamic_smem(bwd_dq_tc_kernel<D>, BCfg<D>::kSmemBytes, smem_allowed_b));
    const long long rows_padded = bh * Wpad;
    bwd_prep_kernel<D><<<(unsigned)((rows_padded + prep_rows_per_block<D>() - 1) / prep_rows_per_block<D>()), 256, 0, st>>>(
        (const __nv_bfloat16*)out, (const __nv_bfloat16*)dout, lse, lse2, delta, W, Wpad, rows_padded);
    TLIN_CUDA_CHECK(cudaGetLastError());
    // dK, dV: the units are (b,h,key tile); a CTA takes a contiguous run of them
    BwdParams pa = p;
    pa.total_units = bh * p.key_tiles;
    pa.n_groups = 0; pa.q_tiles = 0; pa.schedule = 0;
    const long long ctas_a = pa.total_units < num_sms ? pa.total_units : num_sms;
    bwd_dkdv_tc_kernel<D><<<(unsigned)ctas_a, ACfg<D>::kThreads, ACfg<D>::kSmemBytes, st>>>(mq64, mk, mv, mdo64, pa);
    TLIN_CUDA_CHECK(cudaGetLastError());
    // dQ: the forward's plan
    BwdParams pb = p;
    pb.total_units = plan.total_units; pb.n_groups = plan.n_groups; pb.q_tiles = plan.q_tiles; pb.schedule = plan.schedule;
    if (plan.n_groups > kMaxGroups) return TLIN_ERR_UNSUPPORTED;
    GroupStarts starts;
    fwd_group_starts(plan, &starts);
    bwd_dq_tc_kernel<D><<<plan.n_ctas, BCfg<D>::kThreads, BCfg<D>::kSmemBytes, st>>>(mq, mk, mv, mdo, pb, starts);
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch(3);
    if (plan.uses_workspace) {
        bwd_dq_reduce_kernel<D><<<(unsigned)(bh * plan.q_tiles * (kTileM / 8)), 256, 0, st>>>(pb);
        TLIN_CUDA_CHECK(cudaGetLastError());
        count_launch();
    }
    return TLIN_OK;
}

// fp32 dQ sums (rows padded to 128 per (b,h)) -> scaled bf16 dQ; 8 elements per thread
template <int D>
__global__ void __launch_bounds__(256)
bwd_dq_convert_kernel(const float* __restrict__ dq32, __nv_bfloat16* __restrict__ dq, int W, int Wpad, long long rows, float scale) {
    constexpr int TPR = D / 8;              // threads per row
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    const long long row = idx / TPR;
    const int piece = (int)(idx - row * TPR);
    if (row >= rows) return;
    const long long bh = row / W;
    const int i = (int)(row - bh * W);
    const float4* src = reinterpret_cast<const float4*>(dq32 + (bh * Wpad + i) * D + piece * 8);
    const float4 a = src[0], b = src[1];
    uint4 w;
    w.x = pack_bf16x2(a.x * scale, a.y * scale);
    w.y = pack_bf16x2(a.z * scale, a.w * scale);
    w.z = pack_bf16x2(b.x * scale, b.y * scale);
    w.w = pack_bf16x2(b.z * scale, b.w * scale);
    *reinterpret_cast<uint4*>(dq + row * D + piece * 8) = w;
}

// One kernel for dK, dV and dQ (five matrix products per pair; dQ summed in fp32 by reductions in L2, then rounded).
int launch_fused_128(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
                     void* dq, void* dk, void* dv, int B, int H, int N, int W, int causal, float* ws, int num_sms, cudaStream_t st) {
    constexpr int D = 128;
    const long long bh = (long long)B * H;
    const int Wpad = (W + kQTile - 1) / kQTile * kQTile;
    CUtensorMap mk, mv, mq64, mdo64;
    int rc = make_map(&mk, k, D, N, bh);
    if (rc == TLIN_OK) rc = make_map(&mv, v, D, N, bh);
    if (rc == TLIN_OK) rc = make_map(&mq64, q, D, W, bh, 64);
    if (rc == TLIN_OK) rc = make_map(&mdo64, dout, D, W, bh, 64);
    if (rc != TLIN_OK) return rc;
    BwdParams p;
    float* lse2 = ws;
    float* delta = ws + bh * Wpad;
    float* dq32 = ws + 2 * bh * Wpad;
    p.lse2 = lse2; p.delta = delta; p.dq = dq; p.dk = dk; p.dv = dv;
    p.ws = dq32;
    p.status = status_word();
    if (!p.status) return TLIN_ERR_CUDA;
    p.key_tiles = (N + kTileN - 1) / kTileN;
    p.q_tiles128 = Wpad / kQTile;
    p.N = N; p.W = W; p.Wpad = Wpad; p.causal = causal;
    p.scale = 1.f / sqrtf((float)D);
    p.scale_log2e = kLog2e * p.scale;
    p.wide_stores = 0;
    p.total_units = bh * p.key_tiles;
    p.n_groups = 0; p.q_tiles = 0; p.schedule = 0;
    static bool smem_allowed[64] = {};
    constexpr int kSmem = ACfg<D>::kSmemBytes + 32;             // four more barriers than the dK/dV kernel
    TLIN_CUDA_CHECK(allow_dynamic_smem(bwd_fused_tc_kernel<D>, kSmem, smem_allowed));
    const long long rows_padded = bh * Wpad;
    bwd_prep_kernel<D><<<(unsigned)((rows_padded + prep_rows_per_block<D>() - 1) / prep_rows_per_block<D>()), 256, 0, st>>>(
        (const __nv_bfloat16*)out, (const __nv_bfloat16*)dout, lse, lse2, delta, W, Wpad, rows_padded);
    TLIN_CUDA_CHECK(cudaGetLastError());
    TLIN_CUDA_CHECK(cudaMemsetAsync(dq32, 0, (size_t)rows_padded * D * sizeof(float), st));
    const long long ctas = p.total_units < num_sms ? p.total_units : num_sms;
    bwd_fused_tc_kernel<D><<<(unsigned)ctas, ACfg<D>::kThreads, kSmem, st>>>(mq64, mk, mv, mdo64, p);
    TLIN_CUDA_CHECK(cudaGetLastError());
    const long long rows = bh * W, threads = rows * (D / 8);
    bwd_dq_convert_kernel<D><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(dq32, (__nv_bfloat16*)dq, W, Wpad, rows, p.scale);
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch(3);
    return TLIN_OK;
}

}  // namespace

// row statistics (lse2, delta, padded) + the fp32 dQ sums, rows padded to 128 per (b,h)
size_t bwd_fused_workspace_bytes(long long B, long long H, long long W, int d) {
    const long long bh = B * H, Wpad = (W + tc::kQTile - 1) / tc::kQTile * tc::kQTile;
    return (size_t)(2 * bh * Wpad + bh * Wpad * d) * sizeof(float);
}

int launch_bwd_fused(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
                     void* dq, void* dk, void* dv, int B, int H, int N, int W, int d, int causal, float* ws, int num_sms, cudaStream_t st) {
    if (d != 128) return TLIN_ERR_UNSUPPORTED;
    if ((long long)B * H * W > 0x7fffffffLL || (long long)B * H > 0x7fffffffLL) return TLIN_ERR_UNSUPPORTED;
    return launch_fused_128(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, causal, ws, num_sms, st);
}

// row statistics (lse2, delta, padded) + the dQ kernel's partial slots
size_t bwd_tc_workspace_bytes(long long B, long long H, long long W, int d, const tlin_fwd_plan& plan) {
    const long long bh = B * H, Wpad = (W + tc::kQTile - 1) / tc::kQTile * tc::kQTile;
    long long floats = 2 * bh * Wpad;
    if (plan.uses_workspace) floats += (long long)plan.n_ctas * 2 * tc::kTileM * d;
    return (size_t)floats * sizeof(float);
}

int launch_bwd_tc(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
                  void* dq, void* dk, void* dv, int B, int H, int N, int W, int d, int causal, const tlin_fwd_plan& plan,
                  float* ws, int num_sms, cudaStream_t st) {
    if (plan.tile_m != tc::kTileM || plan.tile_n != kTileN || !plan.tensor_path) return TLIN_ERR_UNSUPPORTED;
    if ((long long)B * H * W > 0x7fffffffLL || (long long)B * H > 0x7fffffffLL) return TLIN_ERR_UNSUPPORTED;
    if (d == 128) return launch_d<128>(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, causal, plan, ws, num_sms, st);
    if (d == 64) return launch_d<64>(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, causal, plan, ws, num_sms, st);
    return TLIN_ERR_UNSUPPORTED;
}

}  // namespace tlin
