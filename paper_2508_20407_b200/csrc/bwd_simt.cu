// Backward pass of the attention layer on the CUDA cores (fp32 arithmetic; bf16 or fp32 tensors; any head size the
// CUDA-core forward takes): the chain rule applied to the Section 3 attention formula with the window mask.  Training
// runs every layer as a forward and a backward pass ("cache miss" throughout, Section 4.1); the paper gives no separate
// algorithm for the gradient.
//
//   p_ij  = exp(s_ij - lse_i),  s_ij = q_i.k_j / sqrt(d)      (lse saved by the forward, so no second softmax pass)
//   delta_i = dout_i . out_i   ( = sum_j p_ij dp_ij )
//   dv_j  = sum_i p_ij dout_i          dp_ij = dout_i . v_j          ds_ij = p_ij (dp_ij - delta_i) / sqrt(d)
//   dq_i  = sum_j ds_ij k_j            dk_j  = sum_i ds_ij q_i
//
// Three kernels.  delta: one warp per query row.  dk/dv: one CTA per block of 32 keys of a (b,h), looping over the
// query tiles that can see it; every dk/dv element has one owner, so nothing is atomic.  dq: one CTA per tile of 32
// query rows and per slice of the key range; the slices add their partial dq into an fp32 buffer in the workspace
// (cleared first), which a last kernel rounds to the output type.
//
// This is the fp32 path and the path for head sizes other than 64 and 128 (the counterpart of fwd_simt.cu); it is
// not a roofline target.
#include "tlin_internal.h"
#include <math_constants.h>

namespace tlin {
namespace {

constexpr int kTB = 32;                 // query rows per tile and keys per block
constexpr int kBwdThreads = 256;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ void from_f(__nv_bfloat16& dst, float x) { dst = __float2bfloat16_rn(x); }
__device__ __forceinline__ void from_f(float& dst, float x) { dst = x; }

// rows [r0, r0+32) of a [rows_total, d] matrix into padded fp32 shared memory (row stride d+1); rows beyond
// rows_total become 0
template <typename T>
__device__ __forceinline__ void load_tile(float* dst, const T* src, long long r0, long long rows_total, int d) {
    for (int x = threadIdx.x; x < kTB * d; x += kBwdThreads) {
        const int r = x / d, c = x - r * d;
        dst[r * (d + 1) + c] = r0 + r < rows_total ? to_f(src[(r0 + r) * d + c]) : 0.f;
    }
}

// delta_i = dout_i . out_i, one warp per row
template <typename T>
__global__ void __launch_bounds__(256)
bwd_delta_kernel(const T* __restrict__ out, const T* __restrict__ dout, float* __restrict__ delta, long long rows, int d) {
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int lane = threadIdx.x & 31;
    float acc = 0.f;
    for (int c = lane; c < d; c += 32) acc = fmaf(to_f(out[row * d + c]), to_f(dout[row * d + c]), acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) delta[row] = acc;
}

// shared memory of the two tile kernels: four [32][d+1] tiles, P and dS as [32][33], lse and delta of the rows
struct BwdSmem {
    float *Qs, *dOs, *Ks, *Vs, *Ps, *dSs, *lse_s, *delta_s;
    __device__ BwdSmem(float* base, int d) {
        const int tile = kTB * (d + 1);
        Qs = base;
        dOs = Qs + tile;
        Ks = dOs + tile;
        Vs = Ks + tile;
        Ps = Vs + tile;
        dSs = Ps + kTB * (kTB + 1);
        lse_s = dSs + kTB * (kTB + 1);
        delta_s = lse_s + kTB;
    }
};
size_t bwd_smem_bytes(int d) { return sizeof(float) * (4 * kTB * (d + 1) + 2 * kTB * (kTB + 1) + 2 * kTB); }

// Scores, probabilities and ds of one 32 x 32 (query, key) tile, written to Ps / dSs (both [row][key]).
// Thread t handles key j = t % 32 and rows i = t / 32 + 8 m: the row operands are warp-uniform (broadcast), the key
// operands hit 32 different banks thanks to the padding.
__device__ __forceinline__ void tile_p_ds(const BwdSmem& sm, int d, long long i0, long long j0, long long N, long long W,
                                          int causal, float scale) {
    const int j = threadIdx.x & 31, ib = threadIdx.x >> 5, ld = d + 1;
    float s[4] = {0.f, 0.f, 0.f, 0.f}, dp[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
    for (int c = 0; c < d; ++c) {
        const float kc = sm.Ks[j * ld + c], vc = sm.Vs[j * ld + c];
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            s[m] = fmaf(sm.Qs[(ib + 8 * m) * ld + c], kc, s[m]);
            dp[m] = fmaf(sm.dOs[(ib + 8 * m) * ld + c], vc, dp[m]);
        }
    }
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        const int il = ib + 8 * m;
        const long long i = i0 + il, jj = j0 + j;
        const bool ok = i < W && jj < N && (!causal || jj <= (N - W) + i);
        const float p = ok ? exp2f((s[m] * scale - sm.lse_s[il]) * kLog2e) : 0.f;
        sm.Ps[il * (kTB + 1) + j] = p;
        sm.dSs[il * (kTB + 1) + j] = p * (dp[m] - sm.delta_s[il]) * scale;
    }
}

// MAXM: columns per thread (thread t owns columns t % 8 + 8 m, m < MAXM, below d)
template <typename T, int MAXM>
__global__ void __launch_bounds__(kBwdThreads)
bwd_dkdv_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, const T* __restrict__ dout,
                const float* __restrict__ lse, const float* __restrict__ delta, T* __restrict__ dk, T* __restrict__ dv,
                long long N, long long W, int d, int causal, float scale) {
    extern __shared__ __align__(16) float smem_f[];
    const BwdSmem sm(smem_f, d);
    const int ld = d + 1;
    const long long bh = blockIdx.y, j0 = (long long)blockIdx.x * kTB;
    const T* qb = q + bh * W * d;
    const T* dob = dout + bh * W * d;
    load_tile(sm.Ks, k + bh * N * d, j0, N, d);
    load_tile(sm.Vs, v + bh * N * d, j0, N, d);
    const int jo = threadIdx.x >> 3, co = threadIdx.x & 7;      // owned key and first owned column
    float acc_dk[MAXM], acc_dv[MAXM];
#pragma unroll
    for (int m = 0; m < MAXM; ++m) acc_dk[m] = acc_dv[m] = 0.f;
    // the first query row that may use a key of this block (window rule j <= N-W+i)
    long long i_first = 0;
    if (causal) {
        i_first = j0 - (N - W);
        if (i_first < 0) i_first = 0;
    }
    for (long long i0 = (i_first / kTB) * kTB; i0 < W; i0 += kTB) {
        __syncthreads();
        load_tile(sm.Qs, qb, i0, W, d);
        load_tile(sm.dOs, dob, i0, W, d);
        if (threadIdx.x < kTB) {
            const long long i = i0 + threadIdx.x;
            sm.lse_s[threadIdx.x] = i < W ? lse[bh * W + i] : 0.f;
            sm.delta_s[threadIdx.x] = i < W ? delta[bh * W + i] : 0.f;
        }
        __syncthreads();
        tile_p_ds(sm, d, i0, j0, N, W, causal, scale);
        __syncthreads();
#pragma unroll 4
        for (int i = 0; i < kTB; ++i) {
            const float p = sm.Ps[i * (kTB + 1) + jo], ds = sm.dSs[i * (kTB + 1) + jo];
#pragma unroll
            for (int m = 0; m < MAXM; ++m) {
                const int c = co + 8 * m;
                if (c < d) {
                    acc_dv[m] = fmaf(p, sm.dOs[i * ld + c], acc_dv[m]);
                    acc_dk[m] = fmaf(ds, sm.Qs[i * ld + c], acc_dk[m]);
                }
            }
        }
    }
    if (j0 + jo < N) {
#pragma unroll
        for (int m = 0; m < MAXM; ++m) {
            const int c = co + 8 * m;
            if (c < d) {
                from_f(dk[(bh * N + j0 + jo) * d + c], acc_dk[m]);
                from_f(dv[(bh * N + j0 + jo) * d + c], acc_dv[m]);
            }
        }
    }
}

template <typename T, int MAXM>
__global__ void __launch_bounds__(kBwdThreads)
bwd_dq_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, const T* __restrict__ dout,
              const float* __restrict__ lse, const float* __restrict__ delta, float* __restrict__ dq_acc,
              long long N, long long W, int d, int causal, float scale, int blocks_per_split) {
    extern __shared__ __align__(16) float smem_f[];
    const BwdSmem sm(smem_f, d);
    const int ld = d + 1;
    const long long bh = blockIdx.y, i0 = (long long)blockIdx.x * kTB;
    load_tile(sm.Qs, q + bh * W * d, i0, W, d);
    load_tile(sm.dOs, dout + bh * W * d, i0, W, d);
    if (threadIdx.x < kTB) {
        const long long i = i0 + threadIdx.x;
        sm.lse_s[threadIdx.x] = i < W ? lse[bh * W + i] : 0.f;
        sm.delta_s[threadIdx.x] = i < W ? delta[bh * W + i] : 0.f;
    }
    const int io = threadIdx.x >> 3, co = threadIdx.x & 7;      // owned row and first owned column
    float acc[MAXM];
#pragma unroll
    for (int m = 0; m < MAXM; ++m) acc[m] = 0.f;
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
        load_tile(sm.Ks, k + bh * N * d, b * kTB, N, d);
        load_tile(sm.Vs, v + bh * N * d, b * kTB, N, d);
        __syncthreads();
        tile_p_ds(sm, d, i0, b * kTB, N, W, causal, scale);
        __syncthreads();
#pragma unroll 4
        for (int j = 0; j < kTB; ++j) {
            const float ds = sm.dSs[io * (kTB + 1) + j];
#pragma unroll
            for (int m = 0; m < MAXM; ++m) {
                const int c = co + 8 * m;
                if (c < d) acc[m] = fmaf(ds, sm.Ks[j * ld + c], acc[m]);
            }
        }
    }
    if (i0 + io < W && b1 > b0) {
#pragma unroll
        for (int m = 0; m < MAXM; ++m) {
            const int c = co + 8 * m;
            if (c < d) atomicAdd(&dq_acc[(bh * W + i0 + io) * d + c], acc[m]);
        }
    }
}

template <typename T>
__global__ void bwd_round_kernel(const float* __restrict__ src, T* __restrict__ dst, long long n) {
    const long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (x < n) from_f(dst[x], src[x]);
}

template <typename T, int MAXM>
int launch_t(const T* q, const T* k, const T* v, const T* out, const float* lse, const T* dout, T* dq, T* dk, T* dv,
             int B, int H, int N, int W, int d, int causal, float* ws, int num_sms, cudaStream_t st) {
    const long long bh = (long long)B * H, rows = bh * W;
    float* delta = ws;                                  // [B*H*W]
    float* dq_acc = ws + ((rows + 3) / 4) * 4;          // [B*H*W*d], 16-byte aligned
    const float scale = 1.f / sqrtf((float)d);
    const size_t smem = bwd_smem_bytes(d);
    cudaError_t e = cudaFuncSetAttribute(bwd_dkdv_kernel<T, MAXM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bwd_smem_bytes(8 * MAXM));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(bwd_dq_kernel<T, MAXM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bwd_smem_bytes(8 * MAXM));
    TLIN_CUDA_CHECK(e);
    if (bh > 65535) return TLIN_ERR_UNSUPPORTED;        // grid.y
    bwd_delta_kernel<T><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(out, dout, delta, rows, d);
    TLIN_CUDA_CHECK(cudaGetLastError());
    TLIN_CUDA_CHECK(cudaMemsetAsync(dq_acc, 0, (size_t)rows * d * sizeof(float), st));
    const long long key_blocks = ((long long)N + kTB - 1) / kTB, q_tiles = ((long long)W + kTB - 1) / kTB;
    bwd_dkdv_kernel<T, MAXM><<<dim3((unsigned)key_blocks, (unsigned)bh), kBwdThreads, smem, st>>>(
        q, k, v, dout, lse, delta, dk, dv, N, W, d, causal, scale);
    TLIN_CUDA_CHECK(cudaGetLastError());
    // slices of the key range for dq: enough CTAs for two waves, never more than 65535 (grid.z) or than key blocks
    long long splits = (2LL * num_sms + q_tiles * bh - 1) / (q_tiles * bh);
    if (splits < 1) splits = 1;
    if (splits > key_blocks) splits = key_blocks;
    if (splits > 65535) splits = 65535;
    const int blocks_per_split = (int)((key_blocks + splits - 1) / splits);
    splits = (key_blocks + blocks_per_split - 1) / blocks_per_split;
    bwd_dq_kernel<T, MAXM><<<dim3((unsigned)q_tiles, (unsigned)bh, (unsigned)splits), kBwdThreads, smem, st>>>(
        q, k, v, dout, lse, delta, dq_acc, N, W, d, causal, scale, blocks_per_split);
    TLIN_CUDA_CHECK(cudaGetLastError());
    bwd_round_kernel<T><<<(unsigned)((rows * d + 255) / 256), 256, 0, st>>>(dq_acc, dq, rows * d);
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch(4);
    return TLIN_OK;
}

template <typename T>
int launch_any(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
               void* dq, void* dk, void* dv, int B, int H, int N, int W, int d, int causal, float* ws, int num_sms,
               cudaStream_t st) {
    if ((long long)B * H * W * d > (1LL << 40) || (long long)N > 0x7fffffffLL - kTB) return TLIN_ERR_UNSUPPORTED;
    const T *qt = (const T*)q, *kt = (const T*)k, *vt = (const T*)v, *ot = (const T*)out, *dot = (const T*)dout;
    if (d <= 64) return launch_t<T, 8>(qt, kt, vt, ot, lse, dot, (T*)dq, (T*)dk, (T*)dv, B, H, N, W, d, causal, ws, num_sms, st);
    if (d <= 128) return launch_t<T, 16>(qt, kt, vt, ot, lse, dot, (T*)dq, (T*)dk, (T*)dv, B, H, N, W, d, causal, ws, num_sms, st);
    if (d <= 256) return launch_t<T, 32>(qt, kt, vt, ot, lse, dot, (T*)dq, (T*)dk, (T*)dv, B, H, N, W, d, causal, ws, num_sms, st);
    return TLIN_ERR_UNSUPPORTED;
}

}  // namespace

size_t bwd_workspace_bytes(long long B, long long H, long long W, int d) {
    const long long rows = B * H * W;
    return (size_t)((((rows + 3) / 4) * 4 + rows * d) * (long long)sizeof(float));
}

int launch_bwd_simt(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
                    void* dq, void* dk, void* dv, int B, int H, int N, int W, int d, int causal, int is_f32, float* ws,
                    int num_sms, cudaStream_t st) {
    if (is_f32) return launch_any<float>(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, d, causal, ws, num_sms, st);
    return launch_any<__nv_bfloat16>(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, d, causal, ws, num_sms, st);
}

}  // namespace tlin
