// C-ABI of libtlin: argument validation, planning, dispatch.  Every check runs on the host before
// any launch; no exception leaves this file.
#include "tlin_internal.h"
#include <atomic>
#include <mutex>
#include <stdlib.h>

namespace tlin {

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_mu;
Workspace g_ws[kMaxDevices] = {};          // one registered workspace per device (indexed by the current device)
std::atomic<int> g_impl{0};
std::atomic<int> g_bwd_impl{0};
thread_local int t_launches = 0;
__device__ int g_status_word = 0;

struct DevInfo { int checked; int major; int sms; };
DevInfo g_dev[kMaxDevices] = {};

int device_info(int* sms) {
    int dev = 0;
    TLIN_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return TLIN_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_mu);
    DevInfo& di = g_dev[dev];
    if (!di.checked) {
        TLIN_CUDA_CHECK(cudaDeviceGetAttribute(&di.major, cudaDevAttrComputeCapabilityMajor, dev));
        TLIN_CUDA_CHECK(cudaDeviceGetAttribute(&di.sms, cudaDevAttrMultiProcessorCount, dev));
        di.checked = 1;
    }
    if (di.major != 10) return TLIN_ERR_ARCH;
    *sms = di.sms;
    return TLIN_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// TLIN_LOG=1 in the environment: every compute call prints the plan it chose to stderr.
bool log_plans() {
    static const bool on = [] {
        const char* e = getenv("TLIN_LOG");
        return e != nullptr && e[0] != '\0' && e[0] != '0';
    }();
    return on;
}
void log_fwd_plan(const char* what, int B, int H, int N, int W, int d, int causal, const tlin_fwd_plan& p) {
    fprintf(stderr, "libtlin: %s B=%d H=%d N=%d W=%d d=%d causal_window=%d -> %s, schedule %d, tile %dx%d, q_tiles %d, key_tiles %d, "
                    "groups %d, ctas %d, units %lld, workspace %lld bytes%s\n",
            what, B, H, N, W, d, causal, p.tensor_path ? "tensor cores" : "CUDA cores", p.schedule, p.tile_m, p.tile_n, p.q_tiles,
            p.key_tiles, p.n_groups, p.n_ctas, (long long)p.total_units, (long long)p.workspace_bytes,
            p.uses_workspace ? " (split, merged by a second kernel)" : "");
}
void log_decode_plan(const char* what, int B, int H, int Ncap, int pos, int d, const tlin_decode_plan& p) {
    fprintf(stderr, "libtlin: %s B=%d H=%d Ncap=%d pos=%d d=%d -> %d splits of %d keys, %d ctas, workspace %lld bytes\n",
            what, B, H, Ncap, pos, d, p.splits, p.keys_per_split, p.n_ctas, (long long)p.workspace_bytes);
}
}  // namespace

// Index of the current device in the per-device tables; 0 where no device can be asked (registering a workspace is
// host bookkeeping and works without one); -1 beyond the tables.
int current_device_slot() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return dev >= 0 && dev < 64 ? dev : -1;
}
Workspace workspace() {
    const int dev = current_device_slot();
    if (dev < 0) return Workspace{nullptr, 0};
    std::lock_guard<std::mutex> lk(g_mu);
    return g_ws[dev];
}
void reset_launches() { t_launches = 0; }
int* status_word() {
    int* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_status_word) != cudaSuccess) return nullptr;
    return p;
}
void count_launch(int n) { t_launches += n; }
int forward_impl() { return g_impl.load(); }
int backward_impl() { return g_bwd_impl.load(); }

}  // namespace tlin

using namespace tlin;

static int forward_common(const void* q, const void* k, const void* v, void* out, float* lse,
                          int B, int H, int N, int W, int d, int causal_window, int is_f32, cudaStream_t st,
                          long long kv_rows_alloc = 0) {
    t_launches = 0;
    if (!q || !k || !v || !out) return TLIN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || N <= 0 || W <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    if (causal_window != 0 && causal_window != 1) return TLIN_ERR_INVALID_ARG;
    if (causal_window && N < W) return TLIN_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return TLIN_ERR_INVALID_ARG;
    if (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)) return TLIN_ERR_INVALID_ARG;
    int sms = 0;
    // shape support is decided before the device is looked at, so that it can be tested without one
    tlin_fwd_plan plan;
    int rc = tlin_plan_forward(B, H, N, W, d, causal_window, is_f32, 0, &plan);
    if (rc != TLIN_OK) return rc;
    rc = device_info(&sms);
    if (rc != TLIN_OK) return rc;
    rc = tlin_plan_forward(B, H, N, W, d, causal_window, is_f32, sms, &plan);
    if (rc != TLIN_OK) return rc;
    if (log_plans()) log_fwd_plan(is_f32 ? "forward (fp32)" : "forward", B, H, N, W, d, causal_window, plan);
    if (is_f32)
        return launch_fwd_simt_f32((const float*)q, (const float*)k, (const float*)v, (float*)out, lse, B, H, N, W, d, causal_window,
                                   kv_rows_alloc, st);
    if (!plan.tensor_path)
        return launch_fwd_simt_bf16(q, k, v, out, lse, B, H, N, W, d, causal_window, kv_rows_alloc, st);
    float* ws = nullptr;
    if (plan.uses_workspace) {
        const Workspace w = workspace();
        if (!w.ptr || w.bytes < (size_t)plan.workspace_bytes) return TLIN_ERR_WORKSPACE;
        ws = (float*)w.ptr;
    }
    return launch_fwd_tc(q, k, v, out, lse, B, H, N, W, d, causal_window, plan, ws, kv_rows_alloc, st);
}

extern "C" int tlin_attn_forward(const void* q, const void* k, const void* v, void* out, float* lse,
                                 int B, int H, int N, int W, int d, int causal_window, tlin_stream_t stream) {
    return forward_common(q, k, v, out, lse, B, H, N, W, d, causal_window, 0, (cudaStream_t)stream);
}

extern "C" int tlin_attn_forward_prefixes(const void* q, const void* k, const void* v, void* out, float* lse,
                                          int B, int H, int L, int W, int d, int C, const int32_t* n_keys,
                                          int causal_window, tlin_stream_t stream) {
    if (!n_keys || C <= 0 || L <= 0 || B <= 0 || H <= 0 || W <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    if (causal_window != 0 && causal_window != 1) return TLIN_ERR_INVALID_ARG;
    for (int c = 0; c < C; ++c)      // every chunk is checked before the first one is launched
        if (n_keys[c] <= 0 || n_keys[c] > L || (causal_window && n_keys[c] < W)) return TLIN_ERR_INVALID_ARG;
    const size_t q_chunk = (size_t)B * H * W * d * 2, lse_chunk = (size_t)B * H * W;
    // Enough whole (chunk, b*h, query tile) problems to fill the SMs: all chunks as one table launch (keys never split, so no
    // workspace).  Fewer: one launch per chunk, each free to split its key range.
    if ((d == 64 || d == 128) && forward_impl() != 1 && C <= kMaxBatch && (long long)B * H <= 0x7fffffffLL) {
        int sms = 0;
        if (device_info(&sms) == TLIN_OK && (long long)C * B * H * ((W + 255) / 256) >= 2LL * sms) {
            tlin_problem tbl[kMaxBatch];
            for (int c = 0; c < C; ++c) {
                tbl[c].q = (const char*)q + c * q_chunk; tbl[c].k = k; tbl[c].v = v;
                tbl[c].out = (char*)out + c * q_chunk; tbl[c].lse = lse ? lse + c * lse_chunk : nullptr;
                tbl[c].BH = B * H; tbl[c].n_keys = n_keys[c]; tbl[c].kv_rows = n_keys[c] == L ? 0 : L;
                tbl[c].n_queries = W; tbl[c].causal_window = causal_window; tbl[c].reserved = 0;
            }
            return tlin_attn_forward_batched(tbl, C, d, stream);
        }
    }
    int total = 0;                 // a chunked call counts the launches of all its chunks
    for (int c = 0; c < C; ++c) {
        const int rc = forward_common((const char*)q + c * q_chunk, k, v, (char*)out + c * q_chunk, lse ? lse + c * lse_chunk : nullptr,
                                      B, H, n_keys[c], W, d, causal_window, 0, (cudaStream_t)stream, L);
        if (rc != TLIN_OK) return rc;
        total += t_launches;
    }
    t_launches = total;
    return TLIN_OK;
}

extern "C" int tlin_attn_forward_cache(const void* q, const void* k_cache, const void* v_cache, void* out, float* lse,
                                       int B, int H, int Ncap, int n_keys, int W, int d, int causal_window, tlin_stream_t stream) {
    if (Ncap <= 0 || n_keys <= 0 || n_keys > Ncap) return TLIN_ERR_INVALID_ARG;
    // the first n_keys rows of every (b,h) block of Ncap rows, read in place (row stride of the cache, nothing copied)
    return forward_common(q, k_cache, v_cache, out, lse, B, H, n_keys, W, d, causal_window, 0, (cudaStream_t)stream, Ncap);
}

extern "C" int tlin_attn_forward_batched(const tlin_problem* problems, int n_problems, int d, tlin_stream_t stream) {
    t_launches = 0;
    if (!problems || n_problems <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return TLIN_ERR_UNSUPPORTED;
    // every problem of every chunk is checked before the first launch
    int64_t starts[kMaxGroups + 1];
    int32_t n_ctas = 0;
    for (int first = 0; first < n_problems; first += kMaxBatch) {
        const int n = n_problems - first < kMaxBatch ? n_problems - first : kMaxBatch;
        const int rc = tlin_plan_batched(problems + first, n, 0, starts, &n_ctas);
        if (rc != TLIN_OK) return rc;
    }
    int sms = 0;
    int rc = device_info(&sms);
    if (rc != TLIN_OK) return rc;
    for (int first = 0; first < n_problems; first += kMaxBatch) {
        const int n = n_problems - first < kMaxBatch ? n_problems - first : kMaxBatch;
        rc = tlin_plan_batched(problems + first, n, sms, starts, &n_ctas);
        if (rc != TLIN_OK) return rc;
        if (log_plans())
            fprintf(stderr, "libtlin: batched forward, problems %d..%d of %d, d=%d -> %lld units on %d ctas\n", first, first + n - 1,
                    n_problems, d, (long long)starts[n_ctas], n_ctas);
        long long st[kMaxGroups + 1];
        for (int g = 0; g <= n_ctas; ++g) st[g] = starts[g];
        rc = launch_fwd_tc_batched(problems + first, n, d, st, n_ctas, (cudaStream_t)stream);
        if (rc != TLIN_OK) return rc;
    }
    return TLIN_OK;
}

extern "C" size_t tlin_workspace_bytes_forward_prefixes(int B, int H, int W, int d, int C, const int32_t* n_keys, int causal_window) {
    size_t need = 0;
    if (!n_keys) return 0;
    for (int c = 0; c < C; ++c) {
        const size_t b = tlin_workspace_bytes_forward(B, H, n_keys[c], W, d, causal_window);
        if (b > need) need = b;
    }
    return need;
}

extern "C" int tlin_attn_forward_f32(const float* q, const float* k, const float* v, float* out, float* lse,
                                     int B, int H, int N, int W, int d, int causal_window, tlin_stream_t stream) {
    return forward_common(q, k, v, out, lse, B, H, N, W, d, causal_window, 1, (cudaStream_t)stream);
}

extern "C" int tlin_attn_forward_host(const void* q_h, const void* k_h, const void* v_h, void* out_h, float* lse_h,
                                      void* q_d, void* k_d, void* v_d, void* out_d, float* lse_d,
                                      int B, int H, int N, int W, int d, int causal_window, tlin_stream_t stream) {
    if (!q_h || !k_h || !v_h || !out_h || !q_d || !k_d || !v_d || !out_d) return TLIN_ERR_INVALID_ARG;
    if (lse_h && !lse_d) return TLIN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || N <= 0 || W <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t qb = (size_t)B * H * W * d * 2, kb = (size_t)B * H * N * d * 2;
    TLIN_CUDA_CHECK(cudaMemcpyAsync(q_d, q_h, qb, cudaMemcpyHostToDevice, st));
    TLIN_CUDA_CHECK(cudaMemcpyAsync(k_d, k_h, kb, cudaMemcpyHostToDevice, st));
    TLIN_CUDA_CHECK(cudaMemcpyAsync(v_d, v_h, kb, cudaMemcpyHostToDevice, st));
    const int rc = forward_common(q_d, k_d, v_d, out_d, lse_d, B, H, N, W, d, causal_window, 0, st);
    if (rc != TLIN_OK) return rc;
    TLIN_CUDA_CHECK(cudaMemcpyAsync(out_h, out_d, qb, cudaMemcpyDeviceToHost, st));
    if (lse_h) TLIN_CUDA_CHECK(cudaMemcpyAsync(lse_h, lse_d, (size_t)B * H * W * sizeof(float), cudaMemcpyDeviceToHost, st));
    return TLIN_OK;
}

// Which arrangement of the tensor-core backward a bf16 call with these sizes gets.  The one-kernel arrangement pays for its
// two saved matrix products with fp32 reductions into a B*H*ceil(W/128)*128*d*4-byte dQ buffer.  Measured against the two
// kernels it is 2 to 13 % faster while that buffer is at most 64 MiB and level with them beyond (its CTAs take the key
// tiles in turn, so the rows being added to stay in L2 at any size); beyond 64 MiB the bitwise repeatable two kernels run.
extern "C" int tlin_backward_arrangement(int B, int H, int N, int W, int d) {
    if (B <= 0 || H <= 0 || N <= 0 || W <= 0) return TLIN_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return TLIN_ERR_UNSUPPORTED;
    if (d != 128) return 1;
    const int mode = backward_impl();
    if (mode != 0) return mode;
    const long long wpad = ((long long)W + 127) / 128 * 128;
    const long long dq32 = (long long)B * H * wpad * d * 4;
    return dq32 <= (64LL << 20) ? 2 : 1;
}

static int backward_common(const void* q, const void* k, const void* v, const void* out, const float* lse,
                           const void* dout, void* dq, void* dk, void* dv,
                           int B, int H, int N, int W, int d, int causal_window, int is_f32, cudaStream_t st) {
    t_launches = 0;
    if (!q || !k || !v || !out || !lse || !dout || !dq || !dk || !dv) return TLIN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || N <= 0 || W <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    if (causal_window != 0 && causal_window != 1) return TLIN_ERR_INVALID_ARG;
    if (causal_window && N < W) return TLIN_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(dout) ||
        !aligned16(dq) || !aligned16(dk) || !aligned16(dv)) return TLIN_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(lse) & 3u) return TLIN_ERR_INVALID_ARG;
    if (is_f32 ? (d % 4 != 0 || d > 256) : (d % 8 != 0 || d > 256)) return TLIN_ERR_UNSUPPORTED;
    int sms = 0;
    int rc = device_info(&sms);
    if (rc != TLIN_OK) return rc;
    const Workspace w = workspace();
    const bool tc = !is_f32 && (d == 64 || d == 128) && forward_impl() != 1;
    if (!tc) {
        if (!w.ptr || w.bytes < bwd_workspace_bytes(B, H, W, d)) return TLIN_ERR_WORKSPACE;
        return launch_bwd_simt(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, d, causal_window, is_f32, (float*)w.ptr, sms, st);
    }
    if (tlin_backward_arrangement(B, H, N, W, d) == 2) {
        if (!w.ptr || w.bytes < bwd_fused_workspace_bytes(B, H, W, d)) return TLIN_ERR_WORKSPACE;
        return launch_bwd_fused(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, d, causal_window, (float*)w.ptr, sms, st);
    }
    tlin_fwd_plan plan;
    rc = tlin_plan_forward(B, H, N, W, d, causal_window, 0, sms, &plan);   // the dQ kernel follows the forward's plan
    if (rc != TLIN_OK) return rc;
    if (log_plans()) log_fwd_plan("backward (dQ kernel follows this plan)", B, H, N, W, d, causal_window, plan);
    if (!w.ptr || w.bytes < bwd_tc_workspace_bytes(B, H, W, d, plan)) return TLIN_ERR_WORKSPACE;
    return launch_bwd_tc(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, d, causal_window, plan, (float*)w.ptr, sms, st);
}

extern "C" int tlin_attn_backward(const void* q, const void* k, const void* v, const void* out, const float* lse,
                                  const void* dout, void* dq, void* dk, void* dv,
                                  int B, int H, int N, int W, int d, int causal_window, tlin_stream_t stream) {
    return backward_common(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, d, causal_window, 0, (cudaStream_t)stream);
}

extern "C" int tlin_attn_backward_f32(const float* q, const float* k, const float* v, const float* out, const float* lse,
                                      const float* dout, float* dq, float* dk, float* dv,
                                      int B, int H, int N, int W, int d, int causal_window, tlin_stream_t stream) {
    return backward_common(q, k, v, out, lse, dout, dq, dk, dv, B, H, N, W, d, causal_window, 1, (cudaStream_t)stream);
}

extern "C" size_t tlin_workspace_bytes_backward(int B, int H, int N, int W, int d) {
    if (B <= 0 || H <= 0 || N <= 0 || W <= 0 || d <= 0) return 0;
    size_t need = bwd_workspace_bytes(B, H, W, d);                 // CUDA-core path
    for (int causal = 0; causal < 2; ++causal) {
        tlin_fwd_plan plan;
        if (causal && N < W) continue;
        if (tlin_plan_forward(B, H, N, W, d, causal, 0, 0, &plan) != TLIN_OK || !plan.tensor_path) continue;
        const size_t t = bwd_tc_workspace_bytes(B, H, W, d, plan);
        if (t > need) need = t;
    }
    if (d == 128) {
        const size_t t = bwd_fused_workspace_bytes(B, H, W, d);
        if (t > need) need = t;
    }
    return need;
}

extern "C" int tlin_decode_step(const void* q_new, const void* k_new, const void* v_new,
                                void* k_cache, void* v_cache, void* out, float* lse,
                                int B, int H, int Ncap, int pos, int d, tlin_stream_t stream) {
    t_launches = 0;
    if (!q_new || !k_new || !v_new || !k_cache || !v_cache || !out) return TLIN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || Ncap <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    if (pos < 0 || pos >= Ncap) return TLIN_ERR_INVALID_ARG;
    if (!aligned16(q_new) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) ||
        !aligned16(v_cache) || !aligned16(out)) return TLIN_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return TLIN_ERR_UNSUPPORTED;
    int sms = 0;
    int rc = device_info(&sms);
    if (rc != TLIN_OK) return rc;
    tlin_decode_plan plan;
    rc = tlin_plan_decode(B, H, pos + 1, d, sms, &plan);
    if (rc != TLIN_OK) return rc;
    if (log_plans()) log_decode_plan("decode", B, H, Ncap, pos, d, plan);
    const Workspace w = workspace();
    if (!w.ptr || w.bytes < (size_t)plan.workspace_bytes) return TLIN_ERR_WORKSPACE;
    return launch_decode(q_new, k_new, v_new, k_cache, v_cache, out, lse, B, H, Ncap, pos, nullptr, d, plan,
                         (float*)w.ptr, (cudaStream_t)stream);
}

extern "C" int tlin_decode_step_batched(const tlin_decode_problem* problems, int n_problems, int d, tlin_stream_t stream) {
    t_launches = 0;
    if (!problems || n_problems <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return TLIN_ERR_UNSUPPORTED;
    for (int i = 0; i < n_problems; ++i) {          // every problem is checked before the first launch
        const tlin_decode_problem& pb = problems[i];
        if (!pb.q_new || !pb.k_cache || !pb.v_cache || !pb.out) return TLIN_ERR_INVALID_ARG;
        if ((pb.k_new == nullptr) != (pb.v_new == nullptr)) return TLIN_ERR_INVALID_ARG;
        if (pb.BH <= 0 || pb.Ncap <= 0) return TLIN_ERR_INVALID_ARG;
        if (pb.k_new ? (pb.pos < 0 || pb.pos >= pb.Ncap) : (pb.pos < 1 || pb.pos > pb.Ncap)) return TLIN_ERR_INVALID_ARG;
        if (!aligned16(pb.q_new) || !aligned16(pb.k_new) || !aligned16(pb.v_new) || !aligned16(pb.k_cache) ||
            !aligned16(pb.v_cache) || !aligned16(pb.out)) return TLIN_ERR_INVALID_ARG;
        if (pb.lse && (reinterpret_cast<uintptr_t>(pb.lse) & 3u)) return TLIN_ERR_INVALID_ARG;
    }
    int sms = 0;
    int rc = device_info(&sms);
    if (rc != TLIN_OK) return rc;
    const int per = decode_table_max_problems();
    for (int first = 0; first < n_problems; first += per) {
        const int n = n_problems - first < per ? n_problems - first : per;
        rc = launch_decode_table(problems + first, n, d, (cudaStream_t)stream);
        if (rc != TLIN_OK) return rc;
    }
    return TLIN_OK;
}

extern "C" int tlin_decode_step_fp8(const void* q_new, const void* k_new, const void* v_new,
                                    void* k_cache, void* v_cache, const float* k_scale, const float* v_scale,
                                    void* out, float* lse, int B, int H, int Ncap, int pos, int d, tlin_stream_t stream) {
    t_launches = 0;
    if (!q_new || !k_new || !v_new || !k_cache || !v_cache || !k_scale || !v_scale || !out) return TLIN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || Ncap <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    if (pos < 0 || pos >= Ncap) return TLIN_ERR_INVALID_ARG;
    if (!aligned16(q_new) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) ||
        !aligned16(v_cache) || !aligned16(out) || (reinterpret_cast<uintptr_t>(k_scale) & 3u) ||
        (reinterpret_cast<uintptr_t>(v_scale) & 3u)) return TLIN_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return TLIN_ERR_UNSUPPORTED;
    int sms = 0;
    int rc = device_info(&sms);
    if (rc != TLIN_OK) return rc;
    tlin_decode_plan plan;
    rc = tlin_plan_decode(B, H, pos + 1, d, sms, &plan);
    if (rc != TLIN_OK) return rc;
    const Workspace w = workspace();
    if (!w.ptr || w.bytes < (size_t)plan.workspace_bytes) return TLIN_ERR_WORKSPACE;
    return launch_decode_fp8(q_new, k_new, v_new, k_cache, v_cache, k_scale, v_scale, out, lse, B, H, Ncap, pos, d, plan,
                             (float*)w.ptr, (cudaStream_t)stream);
}

extern "C" int tlin_decode_step_ragged(const void* q_new, const void* k_new, const void* v_new,
                                       void* k_cache, void* v_cache, void* out, float* lse,
                                       int B, int H, int Ncap, const int32_t* pos, int max_pos, int d, tlin_stream_t stream) {
    t_launches = 0;
    if (!q_new || !k_new || !v_new || !k_cache || !v_cache || !out || !pos) return TLIN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || Ncap <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    if (max_pos < 0 || max_pos >= Ncap) return TLIN_ERR_INVALID_ARG;
    if (!aligned16(q_new) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) ||
        !aligned16(v_cache) || !aligned16(out) || (reinterpret_cast<uintptr_t>(pos) & 3u)) return TLIN_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return TLIN_ERR_UNSUPPORTED;
    int sms = 0;
    int rc = device_info(&sms);
    if (rc != TLIN_OK) return rc;
    tlin_decode_plan plan;
    rc = tlin_plan_decode(B, H, max_pos + 1, d, sms, &plan);      // the longest sequence decides the split
    if (rc != TLIN_OK) return rc;
    const Workspace w = workspace();
    if (!w.ptr || w.bytes < (size_t)plan.workspace_bytes) return TLIN_ERR_WORKSPACE;
    // the kernel checks every entry against max_pos (and Ncap) and reports a bad one through the status word
    return launch_decode(q_new, k_new, v_new, k_cache, v_cache, out, lse, B, H, Ncap, max_pos, pos, d, plan,
                         (float*)w.ptr, (cudaStream_t)stream);
}

extern "C" int tlin_decode_step_host(const void* q_new_h, const void* k_new_h, const void* v_new_h, void* out_h, float* lse_h,
                                     void* q_new_d, void* k_new_d, void* v_new_d, void* out_d, float* lse_d,
                                     void* k_cache, void* v_cache,
                                     int B, int H, int Ncap, int pos, int d, tlin_stream_t stream) {
    if (!q_new_h || !k_new_h || !v_new_h || !out_h || !q_new_d || !k_new_d || !v_new_d || !out_d) return TLIN_ERR_INVALID_ARG;
    if (lse_h && !lse_d) return TLIN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t nb = (size_t)B * H * d * 2;
    TLIN_CUDA_CHECK(cudaMemcpyAsync(q_new_d, q_new_h, nb, cudaMemcpyHostToDevice, st));
    TLIN_CUDA_CHECK(cudaMemcpyAsync(k_new_d, k_new_h, nb, cudaMemcpyHostToDevice, st));
    TLIN_CUDA_CHECK(cudaMemcpyAsync(v_new_d, v_new_h, nb, cudaMemcpyHostToDevice, st));
    const int rc = tlin_decode_step(q_new_d, k_new_d, v_new_d, k_cache, v_cache, out_d, lse_d, B, H, Ncap, pos, d, stream);
    if (rc != TLIN_OK) return rc;
    TLIN_CUDA_CHECK(cudaMemcpyAsync(out_h, out_d, nb, cudaMemcpyDeviceToHost, st));
    if (lse_h) TLIN_CUDA_CHECK(cudaMemcpyAsync(lse_h, lse_d, (size_t)B * H * sizeof(float), cudaMemcpyDeviceToHost, st));
    return TLIN_OK;
}

static int merge_common(const void* oa, const float* la, const void* ob, const float* lb, void* out, float* lse,
                        int64_t rows, int d, int is_f32, cudaStream_t st) {
    t_launches = 0;
    if (!oa || !la || !ob || !lb || !out) return TLIN_ERR_INVALID_ARG;
    if (rows < 0 || d <= 0) return TLIN_ERR_INVALID_ARG;
    int sms = 0;
    const int rc = device_info(&sms);
    if (rc != TLIN_OK) return rc;
    return is_f32 ? launch_merge_pair_f32((const float*)oa, la, (const float*)ob, lb, (float*)out, lse, rows, d, st)
                  : launch_merge_pair_bf16(oa, la, ob, lb, out, lse, rows, d, st);
}

extern "C" int tlin_merge_lse(const void* out_a, const float* lse_a, const void* out_b, const float* lse_b,
                              void* out, float* lse, int64_t rows, int d, tlin_stream_t stream) {
    return merge_common(out_a, lse_a, out_b, lse_b, out, lse, rows, d, 0, (cudaStream_t)stream);
}
extern "C" int tlin_merge_lse_f32(const float* out_a, const float* lse_a, const float* out_b, const float* lse_b,
                                  float* out, float* lse, int64_t rows, int d, tlin_stream_t stream) {
    return merge_common(out_a, lse_a, out_b, lse_b, out, lse, rows, d, 1, (cudaStream_t)stream);
}

extern "C" int tlin_set_workspace(void* dev_ptr, size_t bytes) {
    if ((dev_ptr == nullptr) != (bytes == 0)) return TLIN_ERR_INVALID_ARG;
    if (!aligned16(dev_ptr)) return TLIN_ERR_INVALID_ARG;
    const int dev = current_device_slot();
    if (dev < 0) return TLIN_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_mu);
    g_ws[dev].ptr = dev_ptr;
    g_ws[dev].bytes = bytes;
    return TLIN_OK;
}

extern "C" int tlin_get_status(tlin_stream_t stream) {
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return TLIN_ERR_CUDA;
    int* p = status_word();
    if (!p) return TLIN_ERR_CUDA;
    int h = 0;
    if (cudaMemcpy(&h, p, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return TLIN_ERR_CUDA;
    if (h != 0) {
        const int zero = 0;
        if (cudaMemcpy(p, &zero, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return TLIN_ERR_CUDA;
    }
    return h;
}

extern "C" const char* tlin_status_string(int status) {
    switch (status) {
        case TLIN_OK: return "ok";
        case TLIN_ERR_INVALID_ARG: return "invalid argument";
        case TLIN_ERR_UNSUPPORTED: return "unsupported shape";
        case TLIN_ERR_WORKSPACE: return "workspace missing or too small";
        case TLIN_ERR_CUDA: return "CUDA call failed";
        case TLIN_ERR_TIMEOUT: return "device-side wait timed out";
        case TLIN_ERR_ARCH: return "device is not compute capability 10.x";
        default: return "unknown status";
    }
}

extern "C" const char* tlin_version(void) { return "libtlin 0.1 (sm_100a)"; }

extern "C" int tlin_set_forward_impl(int impl) {
    if (impl < 0 || impl > 2) return TLIN_ERR_INVALID_ARG;
    return g_impl.exchange(impl);
}

extern "C" int tlin_set_backward_impl(int impl) {
    if (impl < 0 || impl > 2) return TLIN_ERR_INVALID_ARG;
    return g_bwd_impl.exchange(impl);
}

extern "C" int tlin_last_launch_count(void) { return t_launches; }
