// Internal declarations shared by the translation units of libtlin (never installed).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stdio.h>
#include <mutex>
#include "../../include/tlin.h"

namespace tlin {

constexpr int kDefaultSMs = 148;       // B200
constexpr int kTileN = 128;            // keys per tile on the tensor path
constexpr int kSimtRows = 8;           // query rows per CTA on the CUDA-core path
constexpr int kSimtKeys = 32;          // keys per staged tile on the CUDA-core path
constexpr int kDecodeMaxSplits = 64;   // upper bound on CTAs per (b,h) in the decode step
constexpr int kDecodeMinKeys = 256;    // do not split the cache finer than this
constexpr int kDecodeCtasPerSM = 2;

struct Workspace { void* ptr; size_t bytes; };
Workspace workspace();
int* status_word();                    // device address of the error word (bounded waits report here)
void count_launch(int n = 1);
void reset_launches();                 // every compute entry point starts its count at zero
int current_device_slot();             // index of the current device in per-device tables (-1: beyond them)
int forward_impl();

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) holds for the device that is current when it is called, so a kernel
// that needs more than 48 KB asks once per device.  `done` is a table of 64 flags owned by the caller (one per kernel).
template <class Kernel>
inline cudaError_t allow_dynamic_smem(Kernel kernel, int bytes, bool (&done)[64]) {
    static std::mutex mu;
    const int dev = current_device_slot();
    if (dev < 0) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lk(mu);
    if (done[dev]) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) done[dev] = true;
    return e;
}

// Work sharing of the tensor-core forward and dQ kernels.  The host works out the first unit of every group and passes the
// table to the kernel as a launch parameter (the CTAs only index it).
// Schedule 0 (units = (b,h,key tile)) and unmasked schedule 1 (units = (b,h,256-row query tile pair) problems, all of one
// cost): equal counts, group g starts at floor(g * units / groups).  Schedule 1 with the window rule: problem qt may use
// ceil((N-W+min(W,256(qt+1)))/128) key tiles; its cost is that number plus 3 (starting and finishing a problem, the masked steps on the diagonal and the step the
// pair's second tile runs alone: measured 2.6 key-tile times), and, when there
// are at least three problems per group, the groups take contiguous runs of problems by cost: every group starting where the
// cost before it reaches its share of the total, and, for problems of 10 key-tile times or more on average, moved as little
// as needed to make the costliest run as cheap as contiguous runs allow (with fewer than three problems per group the
// indivisible problems dominate and equal counts do as well).
constexpr int kMaxGroups = 192;        // groups never exceed the SM count (148 on B200); the planner clamps to this
struct GroupStarts { long long u[kMaxGroups + 1]; };   // u[g] = first unit of group g, u[n_groups] = total_units
inline long long fwd_problem_cost(int N, int W, int key_tiles, int qt) {
    long long rows_end = (long long)(qt + 1) * 256;
    if (rows_end > W) rows_end = W;
    long long tiles = ((long long)N - W + rows_end + 127) / 128;
    if (tiles > key_tiles) tiles = key_tiles;
    return tiles + 3;
}
// fills starts->u[0 .. plan.n_groups]; plan.n_groups <= kMaxGroups
void fwd_group_starts(const tlin_fwd_plan& plan, GroupStarts* starts);

// Work sharing of the tensor-core dK/dV kernel (host and device use the same arithmetic).  Units are (b,h,key tile) in that
// order, key tiles of 128 keys, query tiles of 128 rows; with the window rule key tile t is visited by the query tiles from
// floor(max(0, 128 t - (N-W)) / 128) on, so the last key tiles of a (b,h) cost fewer steps, down to one.  Share c of G starts at
// the smallest unit u such that the steps of the units before it reach c/G of all steps.
__host__ __device__ inline long long bwd_first_unit_of_share(int N, int W, int causal, long long total_units, int key_tiles,
                                                            unsigned c, unsigned G) {
    const int T = key_tiles, Qt = (W + 127) / 128;
    if (c >= G) return total_units;
    if (!causal) return (long long)(((unsigned long long)c * (unsigned long long)total_units) / G);
    auto steps_of = [&](long long t) {
        const long long f = t * 128 - ((long long)N - W);
        return (long long)Qt - (f <= 0 ? 0 : f / 128);
    };
    long long t_full = ((long long)N - W) / 128 + 1;                 // tiles [0, t_full) visit every query tile
    if (t_full > T) t_full = T;
    long long per_bh = t_full * Qt;
    for (long long t = t_full; t < T; ++t) per_bh += steps_of(t);
    const long long n_bh = total_units / T;
    const unsigned long long target = ((unsigned long long)c * (unsigned long long)(per_bh * n_bh)) / G;
    const long long bh = (long long)(target / (unsigned long long)per_bh);
    const long long rem = (long long)(target - (unsigned long long)bh * (unsigned long long)per_bh);   // steps into this (b,h)
    long long t;
    if (rem <= t_full * Qt) {
        t = (rem + Qt - 1) / Qt;                                      // smallest t with t * Qt >= rem
    } else {
        long long cum = t_full * Qt;
        t = t_full;
        while (t < T && cum < rem) {
            cum += steps_of(t);
            ++t;
        }
    }
    return bh * T + t;
}

// Batched forward (a table of small problems in one launch).  Units are whole (problem, b*h, 256-row query tile pair)
// problems in table order; a CTA takes a contiguous run of them, the runs balanced by cost (allowed key tiles + 3 under the window rule, + 2 without) with
// the costliest run as cheap as contiguous runs allow.  prefix[x] = cost of the first x units (prefix.size() = units + 1);
// fills starts[0 .. n_ctas], every CTA non-empty (n_ctas <= units).
constexpr int kMaxBatch = 24;          // problems per launch of the batched kernel (its table travels as a launch parameter)
void balanced_run_starts(const long long* prefix, long long units, int n_ctas, long long* starts);

#define TLIN_CUDA_CHECK(expr)                                                              \
    do {                                                                                   \
        cudaError_t e__ = (expr);                                                          \
        if (e__ != cudaSuccess) {                                                          \
            fprintf(stderr, "libtlin: %s failed: %s (%s:%d)\n", #expr,                     \
                    cudaGetErrorString(e__), __FILE__, __LINE__);                          \
            return TLIN_ERR_CUDA;                                                          \
        }                                                                                  \
    } while (0)

// ---- launchers (one per kernel family); all validate nothing: api.cu has done it ----------
int launch_fwd_simt_bf16(const void* q, const void* k, const void* v, void* out, float* lse,
                         int B, int H, int N, int W, int d, int causal, long long kv_rows_alloc, cudaStream_t st);
int launch_fwd_simt_f32(const float* q, const float* k, const float* v, float* out, float* lse,
                        int B, int H, int N, int W, int d, int causal, long long kv_rows_alloc, cudaStream_t st);
int launch_fwd_tc(const void* q, const void* k, const void* v, void* out, float* lse,
                  int B, int H, int N, int W, int d, int causal, const tlin_fwd_plan& plan,
                  float* ws, long long kv_rows_alloc, cudaStream_t st);   // kv_rows_alloc: rows per (b,h) of k, v (0 = N)
int launch_fwd_tc_batched(const tlin_problem* problems, int n, int d, const long long* starts, int n_ctas, cudaStream_t st);
int launch_decode(const void* q_new, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                  void* out, float* lse, int B, int H, int Ncap, int pos, const int* pos_per_seq, int d,
                  const tlin_decode_plan& plan, float* ws, cudaStream_t st);
int launch_bwd_simt(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
                    void* dq, void* dk, void* dv, int B, int H, int N, int W, int d, int causal, int is_f32, float* ws,
                    int num_sms, cudaStream_t st);
size_t bwd_workspace_bytes(long long B, long long H, long long W, int d);
int launch_bwd_tc(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
                  void* dq, void* dk, void* dv, int B, int H, int N, int W, int d, int causal, const tlin_fwd_plan& plan,
                  float* ws, int num_sms, cudaStream_t st);
size_t bwd_tc_workspace_bytes(long long B, long long H, long long W, int d, const tlin_fwd_plan& plan);
// dK, dV and dQ in one tensor-core kernel (d = 128): scores computed once, dQ summed in an fp32 buffer of the workspace
int launch_bwd_fused(const void* q, const void* k, const void* v, const void* out, const float* lse, const void* dout,
                     void* dq, void* dk, void* dv, int B, int H, int N, int W, int d, int causal, float* ws, int num_sms, cudaStream_t st);
size_t bwd_fused_workspace_bytes(long long B, long long H, long long W, int d);
int backward_impl();
int decode_table_max_problems();
int launch_decode_table(const tlin_decode_problem* problems, int n, int d, cudaStream_t st);
int launch_decode_fp8(const void* q_new, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                      const float* k_scale, const float* v_scale, void* out, float* lse, int B, int H, int Ncap, int pos,
                      int d, const tlin_decode_plan& plan, float* ws, cudaStream_t st);
int launch_merge_pair_bf16(const void* oa, const float* la, const void* ob, const float* lb,
                           void* out, float* lse, int64_t rows, int d, cudaStream_t st);
int launch_merge_pair_f32(const float* oa, const float* la, const float* ob, const float* lb,
                          float* out, float* lse, int64_t rows, int d, cudaStream_t st);

}  // namespace tlin
