// Cached decode step: append the new key/value row, then one query row per (b,h) over the whole
// cache.  Appendix A ("Cache Hit": only the newest token takes part) and Section 5.2 (the history
// cache is static; nothing is re-concatenated).  Pure HBM streaming: every cached K/V byte is read
// exactly once with 16-byte loads, CUDA cores do the arithmetic in fp32.
//
// Grid: (b,h) x splits.  Split s owns keys [s*kps, min(L,(s+1)*kps)), L = pos+1.  Inside a CTA
// each warp-load covers 512 contiguous bytes (32/LPR rows); the LPR lanes that share a row reduce
// their partial dot products with xor-shuffles.  Every row-group keeps its own running max/sum and
// they are combined at the end; the CTA writes one normalised partial (o, lse) to the workspace and
// a second kernel merges the splits (log-sum-exp weights).
#include "tlin_internal.h"
#include <cuda_fp16.h>
#include <math_constants.h>
#include <mutex>
#include <string.h>

namespace tlin {
namespace {

constexpr int kWarps = 8;
constexpr int kUnroll = 4;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ float dot8(const uint4& kv, const float (&qf)[8]) {
    float s = bf_lo(kv.x) * qf[0];
    s = fmaf(bf_hi(kv.x), qf[1], s);
    s = fmaf(bf_lo(kv.y), qf[2], s);
    s = fmaf(bf_hi(kv.y), qf[3], s);
    s = fmaf(bf_lo(kv.z), qf[4], s);
    s = fmaf(bf_hi(kv.z), qf[5], s);
    s = fmaf(bf_lo(kv.w), qf[6], s);
    s = fmaf(bf_hi(kv.w), qf[7], s);
    return s;
}
__device__ __forceinline__ void axpy8(float p, const uint4& vv, float (&acc)[8]) {
    acc[0] = fmaf(p, bf_lo(vv.x), acc[0]);
    acc[1] = fmaf(p, bf_hi(vv.x), acc[1]);
    acc[2] = fmaf(p, bf_lo(vv.y), acc[2]);
    acc[3] = fmaf(p, bf_hi(vv.y), acc[3]);
    acc[4] = fmaf(p, bf_lo(vv.z), acc[4]);
    acc[5] = fmaf(p, bf_hi(vv.z), acc[5]);
    acc[6] = fmaf(p, bf_lo(vv.w), acc[6]);
    acc[7] = fmaf(p, bf_hi(vv.w), acc[7]);
}

// merge (m2,l2,a2) into (m,l,a); both in log2 units
__device__ __forceinline__ void combine(float& m, float& l, float (&a)[8], float m2, float l2, const float (&a2)[8]) {
    const float mn = fmaxf(m, m2);
    const float ms = mn == -CUDART_INF_F ? 0.f : mn;
    const float c1 = exp2f(m - ms), c2 = exp2f(m2 - ms);
    l = l * c1 + l2 * c2;
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] = a[e] * c1 + a2[e] * c2;
    m = mn;
}

// One query row of one (b,h) over keys [j0, j1) of its cache, by all threads of the CTA: the row `pos` (the token being
// appended in this launch, or -1) is taken from k_new / v_new instead of the cache.  Returns, in threads 0..D-1, column
// c = threadIdx.x of the un-normalised result `a`, the row sum `ll` and the running maximum `mm` (log2 units).
template <int D>
__device__ __forceinline__ void attend_key_range(const uint4* __restrict__ q_row, const uint4* __restrict__ kn, const uint4* __restrict__ vn,
                                                 const uint4* __restrict__ kc, const uint4* __restrict__ vc, int j0, int j1, int pos,
                                                 float scale_log2e, float& a, float& ll, float& mm) {
    constexpr int LPR = D / 8;           // lanes (16-byte chunks) per row
    constexpr int RPW = 32 / LPR;        // rows per warp-load
    constexpr int ROWS_PER_IT = kWarps * RPW * kUnroll;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane % LPR, rsel = lane / LPR;
    float qf[8];
    {
        const uint4 qv = q_row[sub];
        qf[0] = bf_lo(qv.x) * scale_log2e; qf[1] = bf_hi(qv.x) * scale_log2e;
        qf[2] = bf_lo(qv.y) * scale_log2e; qf[3] = bf_hi(qv.y) * scale_log2e;
        qf[4] = bf_lo(qv.z) * scale_log2e; qf[5] = bf_hi(qv.z) * scale_log2e;
        qf[6] = bf_lo(qv.w) * scale_log2e; qf[7] = bf_hi(qv.w) * scale_log2e;
    }

    float m = -CUDART_INF_F, l = 0.f;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;

    for (int base = j0; base < j1; base += ROWS_PER_IT) {
        uint4 kv[kUnroll], vv[kUnroll];
        bool ok[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int j = base + (u * kWarps + warp) * RPW + rsel;
            ok[u] = j < j1;
            kv[u] = make_uint4(0, 0, 0, 0);
            vv[u] = make_uint4(0, 0, 0, 0);
            if (ok[u]) {
                const bool fresh = j == pos;
                const uint4* kp = fresh ? kn + sub : kc + (int64_t)j * LPR + sub;
                const uint4* vp = fresh ? vn + sub : vc + (int64_t)j * LPR + sub;
                kv[u] = ld_stream(kp);
                vv[u] = ld_stream(vp);
            }
        }
        float s[kUnroll];
        float mb = m;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            float x = dot8(kv[u], qf);
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            s[u] = ok[u] ? x : -CUDART_INF_F;
            mb = fmaxf(mb, s[u]);
        }
        const float ms = mb == -CUDART_INF_F ? 0.f : mb;
        const float corr = exp2f(m - ms);
        l *= corr;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] *= corr;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const float p = exp2f(s[u] - ms);
            l += p;
            axpy8(p, vv[u], acc);
        }
        m = mb;
    }

    // combine the row-groups of the warp
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
        const float l2 = __shfl_xor_sync(0xffffffffu, l, o);
        float a2[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) a2[e] = __shfl_xor_sync(0xffffffffu, acc[e], o);
        combine(m, l, acc, m2, l2, a2);
    }
    __shared__ float sm_m[kWarps], sm_l[kWarps];
    __shared__ float sm_a[kWarps][D];
    if (rsel == 0) {
#pragma unroll
        for (int e = 0; e < 8; ++e) sm_a[warp][sub * 8 + e] = acc[e];
        if (sub == 0) { sm_m[warp] = m; sm_l[warp] = l; }
    }
    __syncthreads();
    a = 0.f; ll = 0.f; mm = -CUDART_INF_F;
    if (threadIdx.x < D) {
        const int c = threadIdx.x;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) mm = fmaxf(mm, sm_m[w]);
        const float ms = mm == -CUDART_INF_F ? 0.f : mm;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float c1 = exp2f(sm_m[w] - ms);
            ll += sm_l[w] * c1;
            a += sm_a[w][c] * c1;
        }
    }
}

template <int D>
__global__ void __launch_bounds__(kWarps * 32, kDecodeCtasPerSM)
decode_splitk_kernel(const uint4* __restrict__ q_new, const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                     uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                     float* __restrict__ part_o, float* __restrict__ part_lse,
                     int Ncap, int pos_all, const int* __restrict__ pos_per_seq, int H, int* __restrict__ status,
                     int splits, int kps, float scale_log2e) {
    constexpr int LPR = D / 8;           // lanes (16-byte chunks) per row
    const int bh = blockIdx.x / splits, sp = blockIdx.x - bh * splits;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // one position for the whole batch, or one per sequence read from device memory (ragged batch)
    int pos = pos_all;
    if (pos_per_seq != nullptr) {
        pos = pos_per_seq[bh / H];
        if (pos < 0 || pos >= Ncap || pos > pos_all) {   // pos_all is the caller's bound, which sized the splits; the host
                                                          // cannot see the entries: report, and leave this (b,h) alone
            if (threadIdx.x == 0) {
                atomicExch(status, (int)TLIN_ERR_INVALID_ARG);
                part_lse[(int64_t)bh * splits + sp] = -CUDART_INF_F;
            }
            if (threadIdx.x < D) part_o[((int64_t)bh * splits + sp) * D + threadIdx.x] = 0.f;
            return;
        }
    }
    const int L = pos + 1;
    const int j0 = sp * kps, j1 = min(L, j0 + kps);

    const uint4* kc = k_cache + (int64_t)bh * Ncap * LPR;
    const uint4* vc = v_cache + (int64_t)bh * Ncap * LPR;
    const uint4* kn = k_new + (int64_t)bh * LPR;
    const uint4* vn = v_new + (int64_t)bh * LPR;

    // append (bit-exact copy) by the CTA whose range holds row `pos`; nobody reads that row from the
    // cache in this launch -- the lanes below take it from k_new / v_new.
    if (pos >= j0 && pos < j1 && warp == 0 && lane < LPR) {
        k_cache[((int64_t)bh * Ncap + pos) * LPR + lane] = kn[lane];
        v_cache[((int64_t)bh * Ncap + pos) * LPR + lane] = vn[lane];
    }

    float a, ll, mm;
    attend_key_range<D>(q_new + (int64_t)bh * LPR, kn, vn, kc, vc, j0, j1, pos, scale_log2e, a, ll, mm);
    if (threadIdx.x < D) {
        const int c = threadIdx.x;
        const int64_t slot = (int64_t)bh * splits + sp;
        part_o[slot * D + c] = ll > 0.f ? a / ll : 0.f;
        if (c == 0) part_lse[slot] = ll > 0.f ? (mm + log2f(ll)) * kLn2 : -CUDART_INF_F;
    }
}

// A table of decode problems as one launch: one CTA per (problem, b*h), whole key range, result written directly (no
// split, no second kernel).  Meant for the per-layer caches of a block, which are short (Appendix A, cache hit: the
// (H+1) D W_oh term -- one row against the W_oh summary tokens of a layer -- and the row inside the window).
struct DecodeProblemDev {
    const uint4* q_new; const uint4* k_new; const uint4* v_new;   // k_new == null: attend only, nothing is appended
    uint4* k_cache; uint4* v_cache;
    __nv_bfloat16* out; float* lse;
    int cta0, Ncap, pos;
};
constexpr int kMaxDecodeBatch = 48;
struct DecodeTable { DecodeProblemDev prob[kMaxDecodeBatch]; int n; };

template <int D>
__global__ void __launch_bounds__(kWarps * 32, kDecodeCtasPerSM)
decode_table_kernel(const __grid_constant__ DecodeTable tbl, float scale_log2e) {
    constexpr int LPR = D / 8;
    int pi = 0;
    while (pi + 1 < tbl.n && (int)blockIdx.x >= tbl.prob[pi + 1].cta0) ++pi;
    const DecodeProblemDev& pr = tbl.prob[pi];
    const int bh = blockIdx.x - pr.cta0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool append = pr.k_new != nullptr;
    const int pos = append ? pr.pos : -1;              // row taken from k_new / v_new instead of the cache
    const int L = append ? pr.pos + 1 : pr.pos;
    const uint4* kc = pr.k_cache + (int64_t)bh * pr.Ncap * LPR;
    const uint4* vc = pr.v_cache + (int64_t)bh * pr.Ncap * LPR;
    const uint4* kn = append ? pr.k_new + (int64_t)bh * LPR : kc;
    const uint4* vn = append ? pr.v_new + (int64_t)bh * LPR : vc;
    if (append && warp == 0 && lane < LPR) {
        pr.k_cache[((int64_t)bh * pr.Ncap + pos) * LPR + lane] = kn[lane];
        pr.v_cache[((int64_t)bh * pr.Ncap + pos) * LPR + lane] = vn[lane];
    }
    float a, ll, mm;
    attend_key_range<D>(pr.q_new + (int64_t)bh * LPR, kn, vn, kc, vc, 0, L, pos, scale_log2e, a, ll, mm);
    if (threadIdx.x < D) {
        const int c = threadIdx.x;
        pr.out[(int64_t)bh * D + c] = __float2bfloat16_rn(ll > 0.f ? a / ll : 0.f);
        if (pr.lse != nullptr && c == 0) pr.lse[bh] = ll > 0.f ? (mm + log2f(ll)) * kLn2 : -CUDART_INF_F;
    }
}

// One CTA per (b,h): out = sum_s w_s o_s / sum_s w_s with w_s = exp(lse_s - max lse).
template <int D>
__global__ void __launch_bounds__(D)
decode_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse,
                    __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int splits) {
    const int bh = blockIdx.x, c = threadIdx.x;
    const float* pl = part_lse + (int64_t)bh * splits;
    float mm = -CUDART_INF_F;
    for (int s = 0; s < splits; ++s) mm = fmaxf(mm, pl[s]);
    if (mm == -CUDART_INF_F) {          // every split empty (a ragged sequence whose position was rejected): zeros, not NaN
        out[(int64_t)bh * D + c] = __float2bfloat16_rn(0.f);
        if (lse != nullptr && c == 0) lse[bh] = -CUDART_INF_F;
        return;
    }
    float z = 0.f, a = 0.f;
    for (int s = 0; s < splits; ++s) {
        const float w = expf(pl[s] - mm);
        z += w;
        a = fmaf(w, part_o[((int64_t)bh * splits + s) * D + c], a);
    }
    out[(int64_t)bh * D + c] = __float2bfloat16_rn(a / z);
    if (lse != nullptr && c == 0) lse[bh] = mm + logf(z);
}

// ---------------------------------------------------------------------------------------------------------------
// The same step over an 8-bit cache (E4M3 codes, value = decode(code) * scale[b,h]; not in the paper: it halves the
// bytes the step streams and the memory Section 5.2 accounts for).  A lane owns 16 columns of a row: one 16-byte load
// each for K and V, codes widened in pairs by cvt.rn.f16x2.e4m3x2 (exact).  The key scale is folded into q, the value
// scale into the final normalisation.  The new row is stored as encode(x / scale) (fp32 division, round to nearest
// even, saturating) and every lane that meets it takes the same codes from k_new / v_new instead of the cache.
__device__ __forceinline__ float2 e4m3x2_to_f32x2(uint32_t two_codes) {      // low byte -> x, next byte -> y
    uint32_t h2;
    asm("{\n\t.reg .b16 c;\n\tcvt.u16.u32 c, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, c;\n\t}" : "=r"(h2) : "r"(two_codes));
    return __half22float2(*reinterpret_cast<const __half2*>(&h2));
}
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float lo, float hi) {     // lo -> low byte, hi -> next byte
    uint32_t r;
    asm("{\n\t.reg .b16 c;\n\tcvt.rn.satfinite.e4m3x2.f32 c, %1, %2;\n\tcvt.u32.u16 %0, c;\n\t}" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// sum += k . q for the 16 codes of `c` against 16 f16 values of q (8 packed words): codes widened to f16 pairs (exact),
// products and sum in fp32 by the mixed-precision fma
__device__ __forceinline__ float dot16_codes(const uint4& c, const uint32_t (&qh)[8]) {
    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        asm("{\n\t.reg .b16 c0, c1, k0, k1, k2, k3, q0, q1, q2, q3;\n\t.reg .b32 h0, h1;\n\t"
            "mov.b32 {c0, c1}, %1;\n\t"
            "cvt.rn.f16x2.e4m3x2 h0, c0;\n\tcvt.rn.f16x2.e4m3x2 h1, c1;\n\t"
            "mov.b32 {k0, k1}, h0;\n\tmov.b32 {k2, k3}, h1;\n\t"
            "mov.b32 {q0, q1}, %2;\n\tmov.b32 {q2, q3}, %3;\n\t"
            "fma.rn.f32.f16 %0, k0, q0, %0;\n\tfma.rn.f32.f16 %0, k1, q1, %0;\n\t"
            "fma.rn.f32.f16 %0, k2, q2, %0;\n\tfma.rn.f32.f16 %0, k3, q3, %0;\n\t}"
            : "+f"(s) : "r"(w[i]), "r"(qh[2 * i]), "r"(qh[2 * i + 1]));
    }
    return s;
}
// acc[e] += p * v_e for the 16 codes of `c`; p given twice in one word as f16 (weights lie in (0,1]: rounding them to
// 11 mantissa bits is far below the bf16 rounding of the output), codes widened to f16 (exact), products and sums in fp32
__device__ __forceinline__ void axpy16_codes(uint32_t p2, const uint4& c, float (&acc)[16]) {
    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        asm("{\n\t.reg .b16 c0, c1, v0, v1, v2, v3, p0, p1;\n\t.reg .b32 h0, h1;\n\t"
            "mov.b32 {c0, c1}, %4;\n\t"
            "cvt.rn.f16x2.e4m3x2 h0, c0;\n\tcvt.rn.f16x2.e4m3x2 h1, c1;\n\t"
            "mov.b32 {v0, v1}, h0;\n\tmov.b32 {v2, v3}, h1;\n\t"
            "mov.b32 {p0, p1}, %5;\n\t"
            "fma.rn.f32.f16 %0, v0, p0, %0;\n\tfma.rn.f32.f16 %1, v1, p0, %1;\n\t"
            "fma.rn.f32.f16 %2, v2, p0, %2;\n\tfma.rn.f32.f16 %3, v3, p0, %3;\n\t}"
            : "+f"(acc[4 * i]), "+f"(acc[4 * i + 1]), "+f"(acc[4 * i + 2]), "+f"(acc[4 * i + 3]) : "r"(w[i]), "r"(p2));
    }
}
__device__ __forceinline__ void widen16(const uint4& c, float (&x)[16]) {
    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 a = e4m3x2_to_f32x2(w[i] & 0xffffu), b = e4m3x2_to_f32x2(w[i] >> 16);
        x[4 * i + 0] = a.x; x[4 * i + 1] = a.y; x[4 * i + 2] = b.x; x[4 * i + 3] = b.y;
    }
}
// 16 bf16 values (two 16-byte words) divided by `scale` and encoded
__device__ __forceinline__ uint4 quantise16(const uint4& lo8, const uint4& hi8, float scale) {
    const uint32_t w[8] = {lo8.x, lo8.y, lo8.z, lo8.w, hi8.x, hi8.y, hi8.z, hi8.w};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t a = f32x2_to_e4m3x2(__fdiv_rn(bf_lo(w[2 * i]), scale), __fdiv_rn(bf_hi(w[2 * i]), scale));
        const uint32_t b = f32x2_to_e4m3x2(__fdiv_rn(bf_lo(w[2 * i + 1]), scale), __fdiv_rn(bf_hi(w[2 * i + 1]), scale));
        o[i] = a | (b << 16);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

template <int D>
__global__ void __launch_bounds__(kWarps * 32, kDecodeCtasPerSM)
decode_fp8_splitk_kernel(const uint4* __restrict__ q_new, const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                         uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                         const float* __restrict__ k_scale, const float* __restrict__ v_scale,
                         float* __restrict__ part_o, float* __restrict__ part_lse,
                         int Ncap, int pos, int splits, int kps, float scale_log2e) {
    constexpr int LPR = D / 16;          // lanes (16-byte chunks of codes) per row
    constexpr int RPW = 32 / LPR;        // rows per warp-load
    constexpr int ROWS_PER_IT = kWarps * RPW * kUnroll;
    const int bh = blockIdx.x / splits, sp = blockIdx.x - bh * splits;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane % LPR, rsel = lane / LPR;
    const int L = pos + 1;
    const int j0 = sp * kps, j1 = min(L, j0 + kps);
    const float ks = k_scale[bh], vs = v_scale[bh];

    const uint4* kc = k_cache + (int64_t)bh * Ncap * LPR;
    const uint4* vc = v_cache + (int64_t)bh * Ncap * LPR;
    // the new row's codes for this lane's 16 columns (bf16: two 16-byte words per lane)
    const uint4 kn_codes = quantise16(k_new[(int64_t)bh * (D / 8) + 2 * sub], k_new[(int64_t)bh * (D / 8) + 2 * sub + 1], ks);
    const uint4 vn_codes = quantise16(v_new[(int64_t)bh * (D / 8) + 2 * sub], v_new[(int64_t)bh * (D / 8) + 2 * sub + 1], vs);
    // append by the CTA whose range holds row `pos`; nobody reads that row from the cache in this launch
    if (pos >= j0 && pos < j1 && warp == 0 && lane < LPR) {
        k_cache[((int64_t)bh * Ncap + pos) * LPR + lane] = kn_codes;
        v_cache[((int64_t)bh * Ncap + pos) * LPR + lane] = vn_codes;
    }

    // q * log2(e)/sqrt(d) as f16 pairs (|q| of a few units: no range issue; 11 mantissa bits against the 8 of the bf16
    // input); the key scale multiplies the finished dot product
    uint32_t qh[8];
    {
        const uint4 q0 = q_new[(int64_t)bh * (D / 8) + 2 * sub], q1 = q_new[(int64_t)bh * (D / 8) + 2 * sub + 1];
        const uint32_t w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const __half2 h = __floats2half2_rn(bf_lo(w[i]) * scale_log2e, bf_hi(w[i]) * scale_log2e);
            qh[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
    }

    float m = -CUDART_INF_F, l = 0.f;
    float acc[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) acc[e] = 0.f;

    for (int base = j0; base < j1; base += ROWS_PER_IT) {
        uint4 kv[kUnroll], vv[kUnroll];
        bool ok[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int j = base + (u * kWarps + warp) * RPW + rsel;
            ok[u] = j < j1;
            kv[u] = make_uint4(0, 0, 0, 0);
            vv[u] = make_uint4(0, 0, 0, 0);
            if (ok[u]) {
                if (j == pos) {
                    kv[u] = kn_codes;
                    vv[u] = vn_codes;
                } else {
                    kv[u] = ld_stream(kc + (int64_t)j * LPR + sub);
                    vv[u] = ld_stream(vc + (int64_t)j * LPR + sub);
                }
            }
        }
        float s[kUnroll];
        float mb = m;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            float x = dot16_codes(kv[u], qh);
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            s[u] = ok[u] ? x * ks : -CUDART_INF_F;
            mb = fmaxf(mb, s[u]);
        }
        const float ms = mb == -CUDART_INF_F ? 0.f : mb;
        const float corr = exp2f(m - ms);
        l *= corr;
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[e] *= corr;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const float pr = exp2f(s[u] - ms);
            const __half2 ph = __float2half2_rn(pr);
            l += __low2float(ph);                 // the same rounded weight in the numerator and the denominator
            axpy16_codes(*reinterpret_cast<const uint32_t*>(&ph), vv[u], acc);
        }
        m = mb;
    }

    // combine the row-groups of the warp
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
        const float l2 = __shfl_xor_sync(0xffffffffu, l, o);
        const float mn = fmaxf(m, m2);
        const float mz = mn == -CUDART_INF_F ? 0.f : mn;
        const float c1 = exp2f(m - mz), c2 = exp2f(m2 - mz);
        l = l * c1 + l2 * c2;
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[e] = acc[e] * c1 + __shfl_xor_sync(0xffffffffu, acc[e], o) * c2;
        m = mn;
    }
    __shared__ float sm_m[kWarps], sm_l[kWarps];
    __shared__ float sm_a[kWarps][D];
    if (rsel == 0) {
#pragma unroll
        for (int e = 0; e < 16; ++e) sm_a[warp][sub * 16 + e] = acc[e];
        if (sub == 0) { sm_m[warp] = m; sm_l[warp] = l; }
    }
    __syncthreads();
    if (threadIdx.x < D) {
        const int c = threadIdx.x;
        float mm = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) mm = fmaxf(mm, sm_m[w]);
        const float ms = mm == -CUDART_INF_F ? 0.f : mm;
        float ll = 0.f, a = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float c1 = exp2f(sm_m[w] - ms);
            ll += sm_l[w] * c1;
            a += sm_a[w][c] * c1;
        }
        const int64_t slot = (int64_t)bh * splits + sp;
        part_o[slot * D + c] = ll > 0.f ? a * vs / ll : 0.f;          // the value scale applied once per output element
        if (c == 0) part_lse[slot] = ll > 0.f ? (mm + log2f(ll)) * kLn2 : -CUDART_INF_F;
    }
}

template <int D>
int launch_d(const void* q_new, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
             void* out, float* lse, int B, int H, int Ncap, int pos, const int* pos_per_seq, const tlin_decode_plan& plan,
             float* ws, cudaStream_t st) {
    const int64_t bh = (int64_t)B * H;
    float* part_o = ws;
    float* part_lse = ws + bh * kDecodeMaxSplits * D;
    const float scale_log2e = kLog2e / sqrtf((float)D);
    decode_splitk_kernel<D><<<plan.n_ctas, kWarps * 32, 0, st>>>(
        (const uint4*)q_new, (const uint4*)k_new, (const uint4*)v_new, (uint4*)k_cache, (uint4*)v_cache,
        part_o, part_lse, Ncap, pos, pos_per_seq, H, status_word(), plan.splits, plan.keys_per_split, scale_log2e);
    TLIN_CUDA_CHECK(cudaGetLastError());
    decode_merge_kernel<D><<<(unsigned)bh, D, 0, st>>>(part_o, part_lse, (__nv_bfloat16*)out, lse, plan.splits);
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch(2);
    return TLIN_OK;
}

template <int D>
int launch_fp8_d(const void* q_new, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                 const float* k_scale, const float* v_scale, void* out, float* lse, int B, int H, int Ncap, int pos,
                 const tlin_decode_plan& plan, float* ws, cudaStream_t st) {
    const int64_t bh = (int64_t)B * H;
    float* part_o = ws;
    float* part_lse = ws + bh * kDecodeMaxSplits * D;
    const float scale_log2e = kLog2e / sqrtf((float)D);
    decode_fp8_splitk_kernel<D><<<plan.n_ctas, kWarps * 32, 0, st>>>(
        (const uint4*)q_new, (const uint4*)k_new, (const uint4*)v_new, (uint4*)k_cache, (uint4*)v_cache, k_scale, v_scale,
        part_o, part_lse, Ncap, pos, plan.splits, plan.keys_per_split, scale_log2e);
    TLIN_CUDA_CHECK(cudaGetLastError());
    decode_merge_kernel<D><<<(unsigned)bh, D, 0, st>>>(part_o, part_lse, (__nv_bfloat16*)out, lse, plan.splits);
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch(2);
    return TLIN_OK;
}

template <int D>
int launch_table_d(const tlin_decode_problem* problems, int n, cudaStream_t st) {
    DecodeTable tbl;
    memset(&tbl, 0, sizeof(tbl));
    tbl.n = n;
    long long ctas = 0;
    for (int i = 0; i < n; ++i) {
        const tlin_decode_problem& pb = problems[i];
        DecodeProblemDev& pd = tbl.prob[i];
        pd.q_new = (const uint4*)pb.q_new; pd.k_new = (const uint4*)pb.k_new; pd.v_new = (const uint4*)pb.v_new;
        pd.k_cache = (uint4*)pb.k_cache; pd.v_cache = (uint4*)pb.v_cache;
        pd.out = (__nv_bfloat16*)pb.out; pd.lse = pb.lse;
        pd.cta0 = (int)ctas; pd.Ncap = pb.Ncap; pd.pos = pb.pos;
        ctas += pb.BH;
    }
    if (ctas > 0x7fffffffLL) return TLIN_ERR_UNSUPPORTED;
    decode_table_kernel<D><<<(unsigned)ctas, kWarps * 32, 0, st>>>(tbl, kLog2e / sqrtf((float)D));
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch();
    return TLIN_OK;
}

}  // namespace

int decode_table_max_problems() { return kMaxDecodeBatch; }
int launch_decode_table(const tlin_decode_problem* problems, int n, int d, cudaStream_t st) {
    if (n <= 0 || n > kMaxDecodeBatch) return TLIN_ERR_INVALID_ARG;
    if (d == 128) return launch_table_d<128>(problems, n, st);
    if (d == 64) return launch_table_d<64>(problems, n, st);
    return TLIN_ERR_UNSUPPORTED;
}

int launch_decode_fp8(const void* q_new, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                      const float* k_scale, const float* v_scale, void* out, float* lse, int B, int H, int Ncap, int pos,
                      int d, const tlin_decode_plan& plan, float* ws, cudaStream_t st) {
    if (d == 128) return launch_fp8_d<128>(q_new, k_new, v_new, k_cache, v_cache, k_scale, v_scale, out, lse, B, H, Ncap, pos, plan, ws, st);
    if (d == 64) return launch_fp8_d<64>(q_new, k_new, v_new, k_cache, v_cache, k_scale, v_scale, out, lse, B, H, Ncap, pos, plan, ws, st);
    return TLIN_ERR_UNSUPPORTED;
}

int launch_decode(const void* q_new, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                  void* out, float* lse, int B, int H, int Ncap, int pos, const int* pos_per_seq, int d,
                  const tlin_decode_plan& plan, float* ws, cudaStream_t st) {
    if (d == 128) return launch_d<128>(q_new, k_new, v_new, k_cache, v_cache, out, lse, B, H, Ncap, pos, pos_per_seq, plan, ws, st);
    if (d == 64) return launch_d<64>(q_new, k_new, v_new, k_cache, v_cache, out, lse, B, H, Ncap, pos, pos_per_seq, plan, ws, st);
    return TLIN_ERR_UNSUPPORTED;
}

}  // namespace tlin

// ------------------------------------------------------------------------------------------------
// Decode step for callers that cannot allocate device memory.
//
// Some hosts of this library never get to call cudaMalloc: a plugin running inside another
// framework's memory pool, a worker that may only touch buffers handed to it, a process whose device
// memory budget is fixed up front.  For them the split-K partials live in the array below, which is part of
// the library image: every GPU that loads libtlin holds these 8.1 MiB until the process exits.
// Everything else is as in tlin_decode_step; the caller still owns inputs, caches and outputs.
namespace tlin {
namespace {

constexpr size_t kStaticScratchFloats = (size_t)256 * kDecodeMaxSplits * 129;   // 8 454 144 bytes
static __device__ __align__(256) float g_decode_static_scratch[kStaticScratchFloats];

std::mutex g_static_mu;
float* g_static_ptr[64] = {};      // device address of the array, per device, filled on first use
int g_static_major[64] = {};
int g_static_sms[64] = {};

// In host code the array's name is only a handle: the address a kernel can use has to be asked for,
// with the device current.  Done once per device.
int static_scratch_setup(int dev, float** ptr, int* sms) {
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (g_static_ptr[dev] == nullptr) {
        float* p = nullptr;
        TLIN_CUDA_CHECK(cudaGetSymbolAddress((void**)&p, g_decode_static_scratch));
        TLIN_CUDA_CHECK(cudaDeviceGetAttribute(&g_static_major[dev], cudaDevAttrComputeCapabilityMajor, dev));
        TLIN_CUDA_CHECK(cudaDeviceGetAttribute(&g_static_sms[dev], cudaDevAttrMultiProcessorCount, dev));
        g_static_ptr[dev] = p;
    }
    if (g_static_major[dev] != 10) return TLIN_ERR_ARCH;
    *ptr = g_static_ptr[dev];
    *sms = g_static_sms[dev];
    return TLIN_OK;
}

}  // namespace
}  // namespace tlin

extern "C" int tlin_decode_step_static(const void* q_new, const void* k_new, const void* v_new,
                                       void* k_cache, void* v_cache, void* out, float* lse,
                                       int B, int H, int Ncap, int pos, int d, tlin_stream_t stream) {
    using namespace tlin;
    reset_launches();
    if (!q_new || !k_new || !v_new || !k_cache || !v_cache || !out) return TLIN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || Ncap <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    if (pos < 0 || pos >= Ncap) return TLIN_ERR_INVALID_ARG;
    const uintptr_t all = (uintptr_t)q_new | (uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache |
                          (uintptr_t)v_cache | (uintptr_t)out;
    if (all & 15u) return TLIN_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return TLIN_ERR_UNSUPPORTED;
    const size_t need = (size_t)B * H * kDecodeMaxSplits * (size_t)(d + 1);
    if (need > kStaticScratchFloats) {
        fprintf(stderr, "libtlin: tlin_decode_step_static needs %zu bytes of scratch for B*H=%lld, d=%d but the "
                        "built-in array holds %zu bytes; use tlin_decode_step with a workspace instead\n",
                need * sizeof(float), (long long)B * H, d, kStaticScratchFloats * sizeof(float));
        return TLIN_ERR_WORKSPACE;
    }
    int dev = 0;
    TLIN_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return TLIN_ERR_CUDA;
    float* scratch = nullptr;
    int sms = 0;
    int rc = static_scratch_setup(dev, &scratch, &sms);
    if (rc != TLIN_OK) return rc;
    tlin_decode_plan plan;
    rc = tlin_plan_decode(B, H, pos + 1, d, sms, &plan);
    if (rc != TLIN_OK) return rc;
    return launch_decode(q_new, k_new, v_new, k_cache, v_cache, out, lse, B, H, Ncap, pos, nullptr, d, plan, scratch,
                         (cudaStream_t)stream);
}
