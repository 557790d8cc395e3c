// Backward pass of the attention layer on the CUDA cores (fp32 arithmetic, bf16 in and out): the chain rule
// applied to the Section 3 attention formula with the window mask.  Training runs every layer as a forward and
// a backward pass ("cache miss" throughout, Section 4.1); the paper gives no separate algorithm for the gradient.
//
//   p_ij  = exp(s_ij - lse_i),  s_ij = q_i.k_j / sqrt(d)      (lse saved by the forward, so no second softmax pass)
//   delta_i = dout_i . out_i   ( = sum_j p_ij dp_ij )
//   dv_j  = sum_i p_ij dout_i          dp_ij = dout_i . v_j          ds_ij = p_ij (dp_ij - delta_i) / sqrt(d)
//   dq_i  = sum_j ds_ij k_j            dk_j  = sum_i ds_ij q_i
//
// Three kernels.  delta: one warp per query row.  dk/dv: one CTA per block of 32 keys of a (b,h), looping over the
// query tiles that can see it; every dk/dv element has one owner, so nothing is atomic.  dq: one CTA per tile of 32
// query rows and per slice of the key range; the slices add their partial dq into an fp32 buffer in the workspace
// (cleared first), which a last kernel rounds to bf16.
//
// This is the first correct path for the gradient (the counterpart of fwd_simt.cu); it is not a roofline target.
#include "tlin_internal.h"
#include <math_constants.h>

namespace tlin {
namespace {

constexpr int kTB = 32;                 // query rows per tile and keys per block
constexpr int kBwdThreads = 256;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float bf2f(__nv_bfloat16 x) { return __bfloat162float(x); }

// rows [r0, r0+32) of a [rows_total, D] bf16 matrix into padded fp32 shared memory; rows beyond rows_total become 0
template <int D>
__device__ __forceinline__ void load_tile(float (*dst)[D + 1], const __nv_bfloat16* src, long long r0, long long rows_total) {
    for (int x = threadIdx.x; x < kTB * (D / 8); x += kBwdThreads) {
        const int r = x / (D / 8), c8 = x % (D / 8);
        uint4 w = make_uint4(0, 0, 0, 0);
        if (r0 + r < rows_total) w = *reinterpret_cast<const uint4*>(src + (r0 + r) * D + c8 * 8);
        const __nv_bfloat16* h = reinterpret_cast<const __nv_bfloat16*>(&w);
#pragma unroll
        for (int e = 0; e < 8; ++e) dst[r][c8 * 8 + e] = bf2f(h[e]);
    }
}

// delta_i = dout_i . out_i, one warp per row
template <int D>
__global__ void __launch_bounds__(256)
bwd_delta_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout, float* __restrict__ delta, long long rows) {
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int lane = threadIdx.x & 31;
    float acc = 0.f;
    for (int c = lane; c < D; c += 32) acc = fmaf(bf2f(out[row * D + c]), bf2f(dout[row * D + c]), acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) delta[row] = acc;
}

// Scores, probabilities and ds of one 32 x 32 (query, key) tile, written to Ps / dSs (both [row][key]).
// Thread t handles key j = t % 32 and rows i = t / 32 + 8 m: the row operands are warp-uniform (broadcast), the key
// operands hit 32 different banks thanks to the padding.
template <int D>
__device__ __forceinline__ void tile_p_ds(const float (*Qs)[D + 1], const float (*dOs)[D + 1], const float (*Ks)[D + 1],
                                          const float (*Vs)[D + 1], const float* lse_s, const float* delta_s,
                                          float (*Ps)[kTB + 1], float (*dSs)[kTB + 1],
                                          long long i0, long long j0, long long N, long long W, int causal, float scale) {
    const int j = threadIdx.x & 31, ib = threadIdx.x >> 5;
    float s[4] = {0.f, 0.f, 0.f, 0.f}, dp[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
    for (int c = 0; c < D; ++c) {
        const float kc = Ks[j][c], vc = Vs[j][c];
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            s[m] = fmaf(Qs[ib + 8 * m][c], kc, s[m]);
            dp[m] = fmaf(dOs[ib + 8 * m][c], vc, dp[m]);
        }
    }
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        const int il = ib + 8 * m;
        const long long i = i0 + il, jj = j0 + j;
        const bool ok = i < W && jj < N && (!causal || jj <= (N - W) + i);
        const float p = ok ? exp2f((s[m] * scale - lse_s[il]) * kLog2e) : 0.f;
        Ps[il][j] = p;
        dSs[il][j] = p * (dp[m] - delta_s[il]) * scale;
    }
}

template <int D>
struct BwdSmem {
    float Qs[kTB][D + 1], dOs[kTB][D + 1], Ks[kTB][D + 1], Vs[kTB][D + 1];
    float Ps[kTB][kTB + 1], dSs[kTB][kTB + 1];
    float lse_s[kTB], delta_s[kTB];
};

template <int D>
__global__ void __launch_bounds__(kBwdThreads)
bwd_dkdv_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                const __nv_bfloat16* __restrict__ dout, const float* __restrict__ lse, const float* __restrict__ delta,
                __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv, long long N, long long W, int causal, float scale) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    BwdSmem<D>& sm = *reinterpret_cast<BwdSmem<D>*>(smem_raw);
    const long long bh = blockIdx.y, j0 = (long long)blockIdx.x * kTB;
    const __nv_bfloat16* qb = q + bh * W * D;
    const __nv_bfloat16* dob = dout + bh * W * D;
    load_tile<D>(sm.Ks, k + bh * N * D, j0, N);
    load_tile<D>(sm.Vs, v + bh * N * D, j0, N);
    // thread t owns key jo = t / 8 and columns co + 8 m
    const int jo = threadIdx.x >> 3, co = threadIdx.x & 7;
    float acc_dk[D / 8], acc_dv[D / 8];
#pragma unroll
    for (int m = 0; m < D / 8; ++m) acc_dk[m] = acc_dv[m] = 0.f;
    // the first query row that may use a key of this block (window rule j <= N-W+i)
    long long i_first = 0;
    if (causal) {
        i_first = j0 - (N - W);
        if (i_first < 0) i_first = 0;
    }
    for (long long i0 = (i_first / kTB) * kTB; i0 < W; i0 += kTB) {
        __syncthreads();
        load_tile<D>(sm.Qs, qb, i0, W);
        load_tile<D>(sm.dOs, dob, i0, W);
        if (threadIdx.x < kTB) {
            const long long i = i0 + threadIdx.x;
            sm.lse_s[threadIdx.x] = i < W ? lse[bh * W + i] : 0.f;
            sm.delta_s[threadIdx.x] = i < W ? delta[bh * W + i] : 0.f;
        }
        __syncthreads();
        tile_p_ds<D>(sm.Qs, sm.dOs, sm.Ks, sm.Vs, sm.lse_s, sm.delta_s, sm.Ps, sm.dSs, i0, j0, N, W, causal, scale);
        __syncthreads();
#pragma unroll 4
        for (int i = 0; i < kTB; ++i) {
            const float p = sm.Ps[i][jo], ds = sm.dSs[i][jo];
#pragma unroll
            for (int m = 0; m < D / 8; ++m) {
                acc_dv[m] = fmaf(p, sm.dOs[i][co + 8 * m], acc_dv[m]);
                acc_dk[m] = fmaf(ds, sm.Qs[i][co + 8 * m], acc_dk[m]);
            }
        }
    }
    if (j0 + jo < N) {
#pragma unroll
        for (int m = 0; m < D / 8; ++m) {
            dk[(bh * N + j0 + jo) * D + co + 8 * m] = __float2bfloat16_rn(acc_dk[m]);
            dv[(bh * N + j0 + jo) * D + co + 8 * m] = __float2bfloat16_rn(acc_dv[m]);
        }
    }
}

template <int D>
__global__ void __launch_bounds__(kBwdThreads)
bwd_dq_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
              const __nv_bfloat16* __restrict__ dout, const float* __restrict__ lse, const float* __restrict__ delta,
              float* __restrict__ dq_acc, long long N, long long W, int causal, float scale, int blocks_per_split) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    BwdSmem<D>& sm = *reinterpret_cast<BwdSmem<D>*>(smem_raw);
    const long long bh = blockIdx.y, i0 = (long long)blockIdx.x * kTB;
    load_tile<D>(sm.Qs, q + bh * W * D, i0, W);
    load_tile<D>(sm.dOs, dout + bh * W * D, i0, W);
    if (threadIdx.x < kTB) {
        const long long i = i0 + threadIdx.x;
        sm.lse_s[threadIdx.x] = i < W ? lse[bh * W + i] : 0.f;
        sm.delta_s[threadIdx.x] = i < W ? delta[bh * W + i] : 0.f;
    }
    // thread t owns row io = t / 8 and columns co + 8 m
    const int io = threadIdx.x >> 3, co = threadIdx.x & 7;
    float acc[D / 8];
#pragma unroll
    for (int m = 0; m < D / 8; ++m) acc[m] = 0.f;
    const long long key_blocks = (N + kTB - 1) / kTB;
    long long b0 = (long long)blockIdx.z * blocks_per_split, b1 = b0 + blocks_per_split;
    if (b1 > key_blocks) b1 = key_blocks;
    if (causal) {                                  // keys beyond the last row's limit are never used by this tile
        const long long i_last = (i0 + kTB < W ? i0 + kTB : W) - 1;
        const long long j_lim = (N - W) + i_last;  // last usable key
        const long long b_lim = j_lim / kTB + 1;
        if (b1 > b_lim) b1 = b_lim;
    }
    for (long long b = b0; b < b1; ++b) {
        __syncthreads();
        load_tile<D>(sm.Ks, k + bh * N * D, b * kTB, N);
        load_tile<D>(sm.Vs, v + bh * N * D, b * kTB, N);
        __syncthreads();
        tile_p_ds<D>(sm.Qs, sm.dOs, sm.Ks, sm.Vs, sm.lse_s, sm.delta_s, sm.Ps, sm.dSs, i0, b * kTB, N, W, causal, scale);
        __syncthreads();
#pragma unroll 4
        for (int j = 0; j < kTB; ++j) {
            const float ds = sm.dSs[io][j];
#pragma unroll
            for (int m = 0; m < D / 8; ++m) acc[m] = fmaf(ds, sm.Ks[j][co + 8 * m], acc[m]);
        }
    }
    if (i0 + io < W && b1 > b0) {
#pragma unroll
        for (int m = 0; m < D / 8; ++m) atomicAdd(&dq_acc[(bh * W + i0 + io) * D + co + 8 * m], acc[m]);
    }
}

__global__ void bwd_round_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, long long n) {
    const long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (x < n) dst[x] = __float2bfloat16_rn(src[x]);
}

template <int D>
int launch_d(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
             void* dq, void* dk, void* dv, int B, int H, int N, int W, int causal, float* ws, int num_sms, cudaStream_t st) {
    const long long bh = (long long)B * H, rows = bh * W;
    float* delta = ws;                                  // [B*H*W]
    float* dq_acc = ws + ((rows + 3) / 4) * 4;          // [B*H*W*D], 16-byte aligned
    const float scale = 1.f / sqrtf((float)D);
    const size_t smem = sizeof(BwdSmem<D>);
    static cudaError_t attr_err = [] {
        cudaError_t e = cudaFuncSetAttribute(bwd_dkdv_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(BwdSmem<D>));
        if (e == cudaSuccess) e = cudaFuncSetAttribute(bwd_dq_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(BwdSmem<D>));
        return e;
    }();
    TLIN_CUDA_CHECK(attr_err);
    if (bh > 65535) return TLIN_ERR_UNSUPPORTED;        // grid.y
    const auto* qp = (const __nv_bfloat16*)q;
    const auto* kp = (const __nv_bfloat16*)k;
    const auto* vp = (const __nv_bfloat16*)v;
    const auto* dop = (const __nv_bfloat16*)dout;
    bwd_delta_kernel<D><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>((const __nv_bfloat16*)out, dop, delta, rows);
    TLIN_CUDA_CHECK(cudaGetLastError());
    TLIN_CUDA_CHECK(cudaMemsetAsync(dq_acc, 0, (size_t)rows * D * sizeof(float), st));
    const long long key_blocks = ((long long)N + kTB - 1) / kTB, q_tiles = ((long long)W + kTB - 1) / kTB;
    bwd_dkdv_kernel<D><<<dim3((unsigned)key_blocks, (unsigned)bh), kBwdThreads, smem, st>>>(
        qp, kp, vp, dop, lse, delta, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, N, W, causal, scale);
    TLIN_CUDA_CHECK(cudaGetLastError());
    // slices of the key range for dq: enough CTAs for two waves, never more than 65535 (grid.z) or than key blocks
    long long splits = (2LL * num_sms + q_tiles * bh - 1) / (q_tiles * bh);
    if (splits < 1) splits = 1;
    if (splits > key_blocks) splits = key_blocks;
    if (splits > 65535) splits = 65535;
    const int blocks_per_split = (int)((key_blocks + splits - 1) / splits);
    splits = (key_blocks + blocks_per_split - 1) / blocks_per_split;
    bwd_dq_kernel<D><<<dim3((unsigned)q_tiles, (unsigned)bh, (unsigned)splits), kBwdThreads, smem, st>>>(
        qp, kp, vp, dop, lse, delta, dq_acc, N, W, causal, scale, blocks_per_split);
    TLIN_CUDA_CHECK(cudaGetLastError());
    bwd_round_kernel<<<(unsigned)((rows * D + 255) / 256), 256, 0, st>>>(dq_acc, (__nv_bfloat16*)dq, rows * D);
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch(4);
    return TLIN_OK;
}

}  // namespace

size_t bwd_workspace_bytes(long long B, long long H, long long W, int d) {
    const long long rows = B * H * W;
    return (size_t)((((rows + 3) / 4) * 4 + rows * d) * (long long)sizeof(float));
}

int launch_bwd_simt(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
                    void* dq, void* dk, void* dv, int B, int H, int N, int W, int d, int causal, float* ws, int num_sms,
                    cudaStream_t st) {
    if ((long long)N > 0x7fffffffLL / 4 * 4 || (long long)B * H * W * d > (1LL << 40)) return TLIN_ERR_UNSUPPORTED;
    if (((long long)N + kTB - 1) / kTB > 0x7fffffffLL) return TLIN_ERR_UNSUPPORTED;
    if (d == 128) return launch_d<128>(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, causal, ws, num_sms, st);
    if (d == 64) return launch_d<64>(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, causal, ws, num_sms, st);
    return TLIN_ERR_UNSUPPORTED;
}

}  // namespace tlin
