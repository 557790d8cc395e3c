// CUDA-core forward kernel: exact softmax attention, fp32 arithmetic, any head dimension up to 256.
// Serves the fp32 entry point (error bar 1e-4) and bf16 shapes the tensor path does not take.
// Section 3 attention formula; causal rule j <= N-W+i; online (running max / running sum) softmax.
//
// One CTA = 8 warps = 8 consecutive query rows of one (b,h).  Keys/values are staged 32 rows at a
// time in shared memory (converted to fp32); lane l scores key l of the tile, the warp reduces max
// and sum with shuffles, and lane c accumulates output columns c, c+32, ...
#include "tlin_internal.h"
#include <math_constants.h>

namespace tlin {
namespace {

constexpr int ROWS = kSimtRows;
constexpr int KT = kSimtKeys;
constexpr int MAXR = 8;  // d <= 256 -> at most 8 output columns per lane

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_out(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

template <typename T>
__global__ void __launch_bounds__(ROWS * 32)
fwd_simt_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                T* __restrict__ out, float* __restrict__ lse,
                int N, int W, int d, int causal, int q_tiles, float scale, int64_t kv_rows) {
    extern __shared__ float smem[];
    const int kstride = d + 4;                 // padded: lanes reading different rows hit different banks
    float* Qs = smem;                          // [ROWS][d]
    float* Ks = Qs + ROWS * d;                 // [KT][d+4]
    float* Vs = Ks + KT * kstride;             // [KT][d]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t bh = blockIdx.x / q_tiles;
    const int row0 = (blockIdx.x % q_tiles) * ROWS;
    const int i = row0 + warp;
    const bool row_ok = i < W;
    const T* qb = q + (bh * W + row0) * (int64_t)d;
    const T* kb = k + bh * kv_rows * d;        // kv_rows >= N: rows per (b,h) of the key/value allocation
    const T* vb = v + bh * kv_rows * d;

    const int rows_here = min(ROWS, W - row0);
    for (int idx = threadIdx.x; idx < rows_here * d; idx += blockDim.x) Qs[idx] = to_f32(qb[idx]);

    // keys this CTA needs: up to the limit of its last row
    const int64_t last_i = row0 + rows_here - 1;
    const int64_t klimit_blk = causal ? min((int64_t)N, (int64_t)(N - W) + last_i + 1) : (int64_t)N;
    const int64_t klimit_row = causal ? (int64_t)(N - W) + i + 1 : (int64_t)N;  // keys j < klimit_row allowed

    float m = -CUDART_INF_F, l = 0.f;
    float acc[MAXR];
#pragma unroll
    for (int r = 0; r < MAXR; ++r) acc[r] = 0.f;

    for (int64_t t0 = 0; t0 < klimit_blk; t0 += KT) {
        __syncthreads();
        const int nk = (int)min((int64_t)KT, (int64_t)N - t0);
        for (int idx = threadIdx.x; idx < KT * d; idx += blockDim.x) {
            const int r = idx / d, c = idx - r * d;
            float kv = 0.f, vv = 0.f;
            if (r < nk) {
                kv = to_f32(kb[(t0 + r) * d + c]);
                vv = to_f32(vb[(t0 + r) * d + c]);
            }
            Ks[r * kstride + c] = kv;
            Vs[r * d + c] = vv;
        }
        __syncthreads();
        if (!row_ok) continue;
        const int64_t j = t0 + lane;
        const bool ok = j < N && j < klimit_row;
        float s = 0.f;
        const float4* q4 = reinterpret_cast<const float4*>(Qs + warp * d);
        const float4* k4 = reinterpret_cast<const float4*>(Ks + lane * kstride);
        for (int c = 0; c < d / 4; ++c) {
            const float4 a = q4[c], b = k4[c];
            s = fmaf(a.x, b.x, s); s = fmaf(a.y, b.y, s); s = fmaf(a.z, b.z, s); s = fmaf(a.w, b.w, s);
        }
        s = ok ? s * scale : -CUDART_INF_F;
        const float m_new = fmaxf(m, warp_max(s));
        if (m_new == -CUDART_INF_F) continue;          // nothing allowed for this row so far
        const float corr = expf(m - m_new);            // m = -inf -> 0
        const float p = ok ? expf(s - m_new) : 0.f;
        l = l * corr + warp_sum(p);
        m = m_new;
#pragma unroll
        for (int r = 0; r < MAXR; ++r) acc[r] *= corr;
        for (int jj = 0; jj < KT; ++jj) {
            const float pj = __shfl_sync(0xffffffffu, p, jj);
#pragma unroll
            for (int r = 0; r < MAXR; ++r) {
                const int c = lane + 32 * r;
                if (c < d) acc[r] = fmaf(pj, Vs[jj * d + c], acc[r]);
            }
        }
    }
    if (!row_ok) return;
    const float inv_l = 1.f / l;
    T* ob = out + (bh * W + i) * (int64_t)d;
#pragma unroll
    for (int r = 0; r < MAXR; ++r) {
        const int c = lane + 32 * r;
        if (c < d) store_out(ob + c, acc[r] * inv_l);
    }
    if (lse != nullptr && lane == 0) lse[bh * W + i] = m + logf(l);
}

template <typename T>
int launch(const T* q, const T* k, const T* v, T* out, float* lse, int B, int H, int N, int W, int d,
           int causal, long long kv_rows_alloc, cudaStream_t st) {
    const int q_tiles = (W + ROWS - 1) / ROWS;
    const int64_t blocks = (int64_t)B * H * q_tiles;
    const size_t smem = sizeof(float) * ((size_t)ROWS * d + (size_t)KT * (d + 4) + (size_t)KT * d);
    TLIN_CUDA_CHECK(cudaFuncSetAttribute(fwd_simt_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    fwd_simt_kernel<T><<<(unsigned)blocks, ROWS * 32, smem, st>>>(q, k, v, out, lse, N, W, d, causal, q_tiles,
                                                                   1.0f / sqrtf((float)d),
                                                                   kv_rows_alloc > 0 ? (int64_t)kv_rows_alloc : (int64_t)N);
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch();
    return TLIN_OK;
}

}  // namespace

int launch_fwd_simt_bf16(const void* q, const void* k, const void* v, void* out, float* lse,
                         int B, int H, int N, int W, int d, int causal, long long kv_rows_alloc, cudaStream_t st) {
    return launch<__nv_bfloat16>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v,
                                 (__nv_bfloat16*)out, lse, B, H, N, W, d, causal, kv_rows_alloc, st);
}
int launch_fwd_simt_f32(const float* q, const float* k, const float* v, float* out, float* lse,
                        int B, int H, int N, int W, int d, int causal, long long kv_rows_alloc, cudaStream_t st) {
    return launch<float>(q, k, v, out, lse, B, H, N, W, d, causal, kv_rows_alloc, st);
}

}  // namespace tlin
