// Exact merge of two attention results over disjoint key sets (the split-K combine, exposed):
//   lse = log(e^lse_a + e^lse_b),  out = (e^lse_a out_a + e^lse_b out_b) / e^lse.
// Not in the paper; it follows from the softmax in the Section 3 attention formula being a ratio of
// sums over keys.  An lse of -inf marks an empty side.
#include "tlin_internal.h"
#include <math_constants.h>

namespace tlin {
namespace {

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float x) { *p = x; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

template <typename T>
__global__ void merge_pair_kernel(const T* oa, const float* la, const T* ob, const float* lb,
                                  T* out, float* lse, int64_t rows, int d) {
    const int64_t total = rows * d;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = idx / d;
        const float a = la[r], b = lb[r];
        const float m = fmaxf(a, b);
        float o;
        if (m == -CUDART_INF_F) {
            o = 0.f;
        } else {
            const float wa = expf(a - m), wb = expf(b - m);
            const float z = wa + wb;
            o = (wa * ldf(oa + idx) + wb * ldf(ob + idx)) / z;
        }
        // lse may alias lse_a: it is written by a second kernel, after every read of lse_a here.
        stf(out + idx, o);
    }
}

__global__ void merge_lse_rows_kernel(const float* la, const float* lb, float* lse, int64_t rows) {
    for (int64_t r = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; r < rows; r += (int64_t)gridDim.x * blockDim.x) {
        const float a = la[r], b = lb[r];
        const float m = fmaxf(a, b);
        lse[r] = m == -CUDART_INF_F ? -CUDART_INF_F : m + logf(expf(a - m) + expf(b - m));
    }
}

template <typename T>
int launch(const T* oa, const float* la, const T* ob, const float* lb, T* out, float* lse,
           int64_t rows, int d, cudaStream_t st) {
    if (rows == 0) return TLIN_OK;
    const int64_t total = rows * d;
    const int threads = 256;
    int64_t blocks = (total + threads - 1) / threads;
    if (blocks > 148 * 16) blocks = 148 * 16;
    merge_pair_kernel<T><<<(unsigned)blocks, threads, 0, st>>>(oa, la, ob, lb, out, lse, rows, d);
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch();
    if (lse != nullptr) {
        int64_t b2 = (rows + threads - 1) / threads;
        if (b2 > 148 * 16) b2 = 148 * 16;
        merge_lse_rows_kernel<<<(unsigned)b2, threads, 0, st>>>(la, lb, lse, rows);
        TLIN_CUDA_CHECK(cudaGetLastError());
        count_launch();
    }
    return TLIN_OK;
}

}  // namespace

int launch_merge_pair_bf16(const void* oa, const float* la, const void* ob, const float* lb,
                           void* out, float* lse, int64_t rows, int d, cudaStream_t st) {
    return launch<__nv_bfloat16>((const __nv_bfloat16*)oa, la, (const __nv_bfloat16*)ob, lb, (__nv_bfloat16*)out, lse, rows, d, st);
}
int launch_merge_pair_f32(const float* oa, const float* la, const float* ob, const float* lb,
                          float* out, float* lse, int64_t rows, int d, cudaStream_t st) {
    return launch<float>(oa, la, ob, lb, out, lse, rows, d, st);
}

}  // namespace tlin
