// Pieces shared by the tensor-core kernels (forward and backward): the work schedule of a CTA as a list of
// segments, and the host-side TMA tensor-map construction.  Parameter structs passed to the templates here carry
// the fields total_units, n_groups, q_tiles, key_tiles, schedule, N, W, causal.
#pragma once
#include "tlin_internal.h"
#include "sm100_ptx.cuh"
#include <mutex>

namespace tlin {
namespace tc {

using namespace ptx;

constexpr int kQTile = 128;                 // rows per Q tile (one TMEM lane per row)
constexpr int kTileM = 2 * kQTile;          // query rows per CTA

// Work of one CTA as a list of segments: a (b,h), a pair of Q tiles (256 query rows) and a range of key tiles.
// Schedule 0: CTA = (group, q-tile pair); the group's unit range [u, u1) over (b,h,key tile) is cut at the (b,h)
// borders.  Schedule 1: the units are whole (b,h,q-tile pair) problems and a CTA takes a contiguous run of them.
struct Segment { int bh, qt, t_begin, t_end, prob; };    // prob: index into the problem table of a batched launch (else 0)

// The first unit of every group comes from the host as a launch parameter (GroupStarts, in the constant bank).
struct SegmentWalker {
    long long u, u1;
    int T, q_tiles, qt_fixed, schedule;
    template <class P>
    __device__ SegmentWalker(const P& p, const GroupStarts& starts) : T(p.key_tiles), q_tiles(p.q_tiles), schedule(p.schedule) {
        const int g = schedule == 0 ? (int)(blockIdx.x / p.q_tiles) : (int)blockIdx.x;
        qt_fixed = schedule == 0 ? (int)(blockIdx.x - g * p.q_tiles) : 0;
        u = starts.u[g];
        u1 = starts.u[g + 1];
    }
    __device__ bool next(Segment& s) {
        if (u >= u1) return false;
        s.prob = 0;
        if (schedule != 0) {
            s.bh = (int)(u / q_tiles);
            s.qt = (int)(u - (long long)s.bh * q_tiles);
            s.t_begin = 0;
            s.t_end = T;
            ++u;
            return true;
        }
        s.qt = qt_fixed;
        s.bh = (int)(u / T);
        s.t_begin = (int)(u - (long long)s.bh * T);
        const long long left = u1 - u;
        s.t_end = (int)((long long)s.t_begin + left < (long long)T ? (long long)s.t_begin + left : (long long)T);
        u += s.t_end - s.t_begin;
        return true;
    }
};

__device__ __forceinline__ void commit_elected(uint64_t* bar) {
    if (elect_one()) tc_commit(bar);
}

// Number of key tiles Q tile `i` of this CTA may use at all (0 if the tile lies beyond W).
template <class P>
__device__ __forceinline__ int tiles_allowed(const P& p, int row0, int i) {
    const int r_first = row0 + i * kQTile;
    if (r_first >= p.W) return 0;
    if (!p.causal) return p.key_tiles;
    const long long r_end = r_first + kQTile < p.W ? r_first + kQTile : p.W;     // one past the last row
    const long long keys = (long long)p.N - p.W + r_end;                        // keys visible to the last row
    return (int)((keys + kTileN - 1) / kTileN);
}
__device__ __forceinline__ int seg_count(const Segment& s, int allowed) {
    const int e = s.t_end < allowed ? s.t_end : allowed;
    return e > s.t_begin ? e - s.t_begin : 0;
}

// ---------------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(f);
    });
    return fn;
}

// [BH, rows, D] bf16, box = 64 elements x box_rows rows x 1, 128-byte swizzle, zero fill outside.  rows_alloc > rows: only
// the first `rows` rows of every (b,h) block of rows_alloc rows are visible (the rest reads as zero fill).
inline int make_map(CUtensorMap* m, const void* ptr, int D, long long rows, long long bh, int box_rows = kQTile, long long rows_alloc = 0) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return TLIN_ERR_CUDA;
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)rows, (cuuint64_t)bh};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)(rows_alloc > 0 ? rows_alloc : rows) * D * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t es[3] = {1, 1, 1};
    const CUresult rc = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS) {
        fprintf(stderr, "libtlin: cuTensorMapEncodeTiled failed (%d)\n", (int)rc);
        return TLIN_ERR_CUDA;
    }
    return TLIN_OK;
}


}  // namespace tc
}  // namespace tlin
