/*
 * libtlin -- exact-softmax attention of TLinFormer's connectivity for NVIDIA B200 (sm_100a).
 *
 * Paper: "Rethinking Transformer Connectivity: TLinFormer, A Path to Exact, Full
 * Context-Aware Linear Attention" (arXiv 2508.20407).  The library covers the part of the
 * method whose cost grows with the sequence length N: a bounded set of W queries attending
 * over all N keys/values with the exact softmax (Section 3, attention formula; "Focused
 * Attention", "Cross Attention"), causal attention inside the generation window (Section 3,
 * "Causal Attention"), and the cached single-token step (Appendix A, "Cache Hit").
 *
 * Conventions for every entry point
 *   - Plain C ABI.  Unless a parameter is marked HOST, data pointers are DEVICE pointers,
 *     borrowed for the duration of the call; the caller owns and frees every buffer.
 *   - Tensors are dense, row-major, innermost dimension d, and 16-byte aligned.
 *   - Calls that take a stream are asynchronous on it.  Nothing here allocates or frees
 *     device memory; split-K scratch comes from the buffer given to tlin_set_workspace.
 *   - Return value: TLIN_OK (0) or a negative tlin_status.  Argument errors are found on the
 *     host before anything is launched.  No C++ exception crosses the boundary.
 *   - bf16 entry points: bfloat16 inputs, fp32 accumulation, bfloat16 output rounded to
 *     nearest even, fp32 log-sum-exp.  *_f32 entry points: fp32 throughout.
 *   - lse is the natural logarithm of the row's sum of exp(score), scores already scaled by
 *     1/sqrt(d).  (The paper has no such output; it is what makes partial results mergeable.)
 */
#ifndef TLIN_H
#define TLIN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Opaque CUDA stream handle (a cudaStream_t passed as a pointer; NULL = default stream). */
typedef void* tlin_stream_t;

typedef enum {
    TLIN_OK = 0,
    TLIN_ERR_INVALID_ARG = -1, /* null or misaligned pointer, non-positive size, N < W with a causal window, bad pos */
    TLIN_ERR_UNSUPPORTED = -2, /* head dimension outside what the path supports */
    TLIN_ERR_WORKSPACE = -3,   /* workspace missing or smaller than tlin_workspace_bytes_* says */
    TLIN_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed; the message is printed to stderr */
    TLIN_ERR_TIMEOUT = -5,     /* a bounded device-side wait ran out (reported by tlin_get_status) */
    TLIN_ERR_ARCH = -6         /* the current device is not compute capability 10.x */
} tlin_status;

/* ------------------------------------------------------------------------------------------
 * Forward pass ("cache miss", Section 4.1): out = softmax(q k^T / sqrt(d)) v per (b,h).
 *   q   [B,H,W,d]   W query rows: the summary queries of focused attention, or the generation window
 *   k,v [B,H,N,d]   all N keys / values
 *   out [B,H,W,d]   lse [B,H,W] (fp32; may be NULL)
 * causal_window = 0  every query uses all N keys (Section 3, "Focused Attention"/"Cross Attention").
 * causal_window = 1  the queries are the LAST W positions of the N-long sequence; query i uses key j
 *                    iff j <= N-W+i: the history is unmasked and the window is causal (Section 3,
 *                    "Causal Attention", j <= i, aligned to the end).  One softmax runs over the
 *                    union of both key sets.  Requires N >= W.
 * bf16 path: d in {64,128} runs on the tensor cores; any other d that is a multiple of 8 up to 256
 * runs on the CUDA-core kernel.  f32 path: d a multiple of 4 up to 256 (covers the paper's d = 36).
 * Uses the workspace when the plan splits the key range (see tlin_workspace_bytes_forward).
 */
int tlin_attn_forward(const void* q, const void* k, const void* v, void* out, float* lse,
                      int B, int H, int N, int W, int d, int causal_window, tlin_stream_t stream);

int tlin_attn_forward_f32(const float* q, const float* k, const float* v, float* out, float* lse,
                          int B, int H, int N, int W, int d, int causal_window, tlin_stream_t stream);

/* Chunk-scheduled forward for sliding-window training (Section 5.1: the window slides by W_og and every chunk attends to
 * all the chunks before it): C problems over ONE key/value tensor, problem c using its first n_keys[c] rows.
 *   q   [C,B,H,W,d]   the W queries of each chunk        k,v [B,H,L,d]   shared; n_keys[c] <= L (HOST array of C ints)
 *   out [C,B,H,W,d]   lse [C,B,H,W] (may be NULL)
 * causal_window as in tlin_attn_forward, applied per chunk with N = n_keys[c] (with n_keys[c] = (c+1)*W and
 * causal_window = 1 chunk c is the c-th window of the training pass).  k and v are read in place (row stride L); nothing is
 * copied.  When the chunks hold enough whole (chunk, b*h, 256-row query tile) problems to fill the SMs (at least two per SM,
 * C <= 24, d in {64,128}) they are issued as ONE launch (the table form of tlin_attn_forward_batched); otherwise as C
 * launches of the forward kernel on `stream`, each with its own plan and free to split its key range.
 * bf16, head sizes as for tlin_attn_forward.  Workspace: tlin_workspace_bytes_forward_prefixes (the largest of the
 * chunks' needs).  tlin_attn_forward_batched runs such a list, and any other, as one launch. */
int tlin_attn_forward_prefixes(const void* q, const void* k, const void* v, void* out, float* lse,
                               int B, int H, int L, int W, int d, int C, const int32_t* n_keys,
                               int causal_window, tlin_stream_t stream);

/* Cache-miss forward over a decode cache, in place.  Section 4.1 ("Cache Miss") names two inference cases that
 * recompute from scratch: the first token, and "the first new token immediately after the historical context window
 * has been updated (i.e., slided)"; Section 5.2: the history cache stays static only while the window does not slide.
 * After W_og cached steps (tlin_decode_step) the window is full, its rows become history, and the layers that look at
 * the history run again over what the cache now holds:
 *   k_cache, v_cache [B,H,Ncap,d] bf16 as in tlin_decode_step; the call uses rows [0, n_keys) of every (b,h)
 *   (0 < n_keys <= Ncap) through the cache's own row stride.  Nothing is copied, rows >= n_keys are not read, the
 *   caches are not written.
 *   q [B,H,W,d], out, lse, causal_window, head sizes, workspace and errors: as tlin_attn_forward with N = n_keys
 *   (causal_window = 0: summary queries over the new history, Section 3 "Focused Attention"; causal_window = 1: the
 *   last W cached positions as a window, which reproduces what the W decode steps returned).
 * The caller keeps the position count and decides when a window is full; tlin_decode_step continues on the same
 * buffers afterwards. */
int tlin_attn_forward_cache(const void* q, const void* k_cache, const void* v_cache, void* out, float* lse,
                            int B, int H, int Ncap, int n_keys, int W, int d, int causal_window, tlin_stream_t stream);

/* A table of attention problems as ONE launch.  Besides the two N-proportional attentions, a block holds layers whose
 * cost does not grow with N (Appendix A: H self-attention layers over the W_oh summary tokens, cost H*D*W_oh^2, and per
 * generation layer a cross-attention to them plus the causal window, (H+1)*D*W_og*W_oh + (H+2)*D*W_og^2).  Each is a
 * small problem on which a launch of its own spends a large share of its time starting and finishing; problems that do
 * not depend on each other (context layer i and generation layer i both read C_{i-1}; the layers of different
 * requests; the chunks of a sliding-window training pass, Section 5.1, with arbitrary prefix lengths) go into one
 * table and one launch.  Every problem is computed exactly as tlin_attn_forward would compute it.
 *   problems: HOST array of n_problems entries (1 <= n_problems); the pointers inside are DEVICE pointers.
 *   All problems share the head size d (64 or 128: tensor-core path only) and are bf16.
 *   kv_rows: rows per (b,h) of the k, v allocation when it is larger than n_keys (a key prefix read in place, as in
 *   tlin_attn_forward_prefixes / tlin_attn_forward_cache), else 0.  Problems may share k and v.
 * The CTAs take contiguous runs of whole (problem, b*h, 256-row query tile) units, balanced by the key tiles each unit
 * has to visit; keys are never split, so no workspace is used and the result does not depend on the table's neighbours.
 * Long-context problems with few query rows (W <= 1024 over tens of thousands of keys) are better served by
 * tlin_attn_forward, which splits the key range.  Tables of more than 24 problems are issued as several launches. */
typedef struct {
    const void* q;          /* [BH, n_queries, d] */
    const void* k;          /* [BH, kv_rows or n_keys, d] */
    const void* v;
    void* out;              /* [BH, n_queries, d] */
    float* lse;             /* [BH, n_queries] or NULL */
    int32_t BH;             /* number of (batch, head) pairs of this problem */
    int32_t n_keys;         /* N */
    int32_t kv_rows;        /* 0, or rows per (b,h) of the k/v allocation (>= n_keys) */
    int32_t n_queries;      /* W */
    int32_t causal_window;  /* as in tlin_attn_forward; requires n_keys >= n_queries */
    int32_t reserved;       /* 0 */
} tlin_problem;
int tlin_attn_forward_batched(const tlin_problem* problems, int n_problems, int d, tlin_stream_t stream);
/* The split of a table's units among the CTAs of one launch (n_problems <= 24): starts[c] = first unit of CTA c,
 * starts[*n_ctas] = number of units; unit order = problem, then b*h, then query tile pair.  starts has room for
 * num_sms + 1 entries (num_sms <= 0: 148).  Pure host arithmetic. */
int tlin_plan_batched(const tlin_problem* problems, int n_problems, int num_sms, int64_t* starts, int32_t* n_ctas);

/* Same as tlin_attn_forward with HOST input/output buffers (ideally pinned).  *_h are HOST
 * pointers; *_d are DEVICE staging buffers of the same shapes, supplied by the caller.  Copies
 * q,k,v host->device, runs the forward, copies out (and lse if lse_h != NULL) device->host, all on
 * `stream`; the caller synchronises the stream before reading out_h. */
int tlin_attn_forward_host(const void* q_h, const void* k_h, const void* v_h, void* out_h, float* lse_h,
                           void* q_d, void* k_d, void* v_d, void* out_d, float* lse_d,
                           int B, int H, int N, int W, int d, int causal_window, tlin_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * Cached decode step ("cache hit", Section 4.2 and Appendix A: only the newest token takes part;
 * the history cache stays static, Section 5.2).
 *   k_cache,v_cache [B,H,Ncap,d] bf16, rows [0,pos) valid on entry
 *   q_new,k_new,v_new [B,H,1,d] bf16;  out [B,H,1,d] bf16;  lse [B,H] fp32 (may be NULL)
 * Copies k_new,v_new bit-for-bit into row `pos` of the caches, then attends q_new over rows
 * [0,pos] (its own row included).  Rows above pos are not touched.  The caller advances pos.
 * Equals row t of the forward over the final sequence with causal_window = 1.
 * d in {64,128}.  Needs the workspace (tlin_workspace_bytes_decode).  0 <= pos < Ncap.
 */
int tlin_decode_step(const void* q_new, const void* k_new, const void* v_new,
                     void* k_cache, void* v_cache, void* out, float* lse,
                     int B, int H, int Ncap, int pos, int d, tlin_stream_t stream);

/* Cached decode step for a batch whose sequences have different lengths (the paper decodes one sequence at a
 * time, Section 6.3; a served batch holds windows at different offsets, so this is the same cache-hit step,
 * Appendix A, with one cache length per sequence).
 *   pos [B] int32 in DEVICE memory: sequence b has pos[b] valid rows on entry; its new row goes to row pos[b]
 *   and its query attends over rows [0, pos[b]].  Reading the positions on the device lets the caller advance
 *   them there, without a host round trip per token.
 *   max_pos: a HOST-side upper bound of every pos[b] (0 <= max_pos < Ncap); it sizes the split of the key range.
 * An entry outside [0, min(max_pos, Ncap-1)] cannot be seen by the host: the kernel leaves that sequence's cache
 * untouched, writes zeros for it, and tlin_get_status reports TLIN_ERR_INVALID_ARG.
 * Everything else as tlin_decode_step. */
int tlin_decode_step_ragged(const void* q_new, const void* k_new, const void* v_new,
                            void* k_cache, void* v_cache, void* out, float* lse,
                            int B, int H, int Ncap, const int32_t* pos, int max_pos, int d, tlin_stream_t stream);

/* A table of cached decode steps as ONE launch.  In a cache-hit step (Appendix A) the N-proportional term is the new
 * token against the history, served by tlin_decode_step; what remains are short rows: per generation layer the new
 * token against the W_oh cached summary tokens C_i, (H+1)*D*W_oh in all, and against the window so far.  For one
 * token the layers follow one another, but the rows of different sequences, of different requests, or of layers whose
 * inputs are ready are independent; each is a launch-bound problem of its own shape, and a table runs them in one
 * launch: one CTA per (problem, b*h), the whole key range, the result written directly (no split, no workspace).
 *   problems: HOST array; pointers inside are DEVICE pointers, bf16, layouts as in tlin_decode_step with B*H = BH.
 *   pos: valid cache rows on entry.  With k_new, v_new given the new row is copied to row pos (bit-exact) and the
 *   query attends over rows [0, pos]; with k_new = v_new = NULL nothing is written and the query attends over rows
 *   [0, pos) (a cross-attention to a finished cache; pos >= 1).  0 <= pos < Ncap (pos <= Ncap without append).
 *   d in {64,128}.  Meant for short caches: a long one keeps a single CTA per (b*h) busy for its whole length.
 * Tables of more than 48 problems are issued as several launches. */
typedef struct {
    const void* q_new;      /* [BH,1,d] */
    const void* k_new;      /* [BH,1,d] or NULL */
    const void* v_new;      /* [BH,1,d] or NULL (together with k_new) */
    void* k_cache;          /* [BH,Ncap,d] */
    void* v_cache;
    void* out;              /* [BH,1,d] */
    float* lse;             /* [BH] or NULL */
    int32_t BH, Ncap, pos, reserved;
} tlin_decode_problem;
int tlin_decode_step_batched(const tlin_decode_problem* problems, int n_problems, int d, tlin_stream_t stream);

/* tlin_decode_step over an 8-bit cache (not in the paper; it halves the cache memory of Section 5.2 and the bytes a step
 * streams).  k_cache, v_cache [B,H,Ncap,d] hold one byte per element: E4M3 codes of the 8-bit floating point format
 * (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities, largest finite value 448); the value of an element
 * is decode(code) * scale, with k_scale, v_scale [B*H] fp32 in DEVICE memory (one scale per (b,h), chosen by the caller,
 * positive and finite).  q_new, k_new, v_new, out are bf16 as in tlin_decode_step.  The new rows are stored at row `pos` as
 * encode(x / scale): fp32 division, round to nearest with ties to the even code, magnitudes beyond 448 saturate.  The new
 * query then attends to the decoded rows [0, pos], its own included.  d in {64,128}; workspace and errors as for
 * tlin_decode_step. */
int tlin_decode_step_fp8(const void* q_new, const void* k_new, const void* v_new,
                         void* k_cache, void* v_cache, const float* k_scale, const float* v_scale,
                         void* out, float* lse, int B, int H, int Ncap, int pos, int d, tlin_stream_t stream);

/* tlin_decode_step with HOST q/k/v_new and out/lse (the caches stay on the device).  *_d are
 * DEVICE staging buffers ([B,H,1,d] each, lse_d [B,H]). */
int tlin_decode_step_host(const void* q_new_h, const void* k_new_h, const void* v_new_h, void* out_h, float* lse_h,
                          void* q_new_d, void* k_new_d, void* v_new_d, void* out_d, float* lse_d,
                          void* k_cache, void* v_cache,
                          int B, int H, int Ncap, int pos, int d, tlin_stream_t stream);

/* tlin_decode_step for callers that cannot allocate device memory (the paper has no counterpart:
 * this is a packaging variant of the same step).  A library embedded in someone else's memory pool,
 * a worker that may only use buffers handed to it, or code that runs while allocation is off limits
 * has no way to create the split-K workspace that tlin_decode_step wants.  This entry point keeps
 * that scratch in an array compiled into the library (8 454 144 bytes, held on every GPU that loads
 * libtlin until the process exits) and ignores tlin_set_workspace.  It calls no cudaMalloc/cudaFree
 * and no allocating library routine.  Arguments, results and errors are those of tlin_decode_step,
 * plus: shapes with B*H*(d+1)*256 bytes > 8 454 144 (more than 256 (b,h) pairs at d = 128, 508 at
 * d = 64) are rejected with TLIN_ERR_WORKSPACE and a message on stderr.
 * The first call on each device looks up the array's device address (once, with that device
 * current); make that first call outside any stream capture.
 * All calls on a device share the one array.  Every partial slot a call reads was written by the same
 * call, so nothing has to be cleared between calls and stale contents are harmless, but two calls that
 * overlap on the GPU (different streams) race on it: serialise them. */
int tlin_decode_step_static(const void* q_new, const void* k_new, const void* v_new,
                            void* k_cache, void* v_cache, void* out, float* lse,
                            int B, int H, int Ncap, int pos, int d, tlin_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * Backward pass of tlin_attn_forward (bf16 in and out, fp32 arithmetic).  Training runs every layer
 * as a full forward and backward pass ("cache miss" everywhere, Section 4.1); the paper states no
 * gradient algorithm, so this is the chain rule applied to the Section 3 attention formula with the
 * same window rule:  p = exp(q k^T / sqrt(d) - lse),  dv = p^T dout,  dp = dout v^T,
 * ds = p * (dp - rowsum(dout * out)) / sqrt(d),  dq = ds k,  dk = ds^T q.
 *   q, out, dout, dq [B,H,W,d]   k, v, dk, dv [B,H,N,d]   lse [B,H,W] fp32   (all DEVICE, 16-byte aligned)
 * out and lse are what tlin_attn_forward returned for the same q, k, v and causal_window (lse is
 * required here); dout is the loss gradient with respect to out; the loss must not depend on lse.
 * dq, dk, dv are overwritten (keys that no query may use get zeros).
 * bf16: d in {64,128} runs on the tensor cores (two kernels that recompute p, no atomics, bitwise repeatable; or one kernel
 * at d = 128 with dq summed by fp32 reductions, which small calls get by default: tlin_set_backward_impl); any other
 * d that is a multiple of 8 up to 256 runs on the CUDA-core kernels (dq summed with fp32 atomics).  f32: d a multiple
 * of 4 up to 256 (covers the paper's d = 36), CUDA-core kernels.
 * Needs a workspace of tlin_workspace_bytes_backward bytes (row sums, partial or accumulated dq in fp32).
 * Errors as for tlin_attn_forward.
 */
int tlin_attn_backward(const void* q, const void* k, const void* v, const void* out, const float* lse,
                       const void* dout, void* dq, void* dk, void* dv,
                       int B, int H, int N, int W, int d, int causal_window, tlin_stream_t stream);
int tlin_attn_backward_f32(const float* q, const float* k, const float* v, const float* out, const float* lse,
                           const float* dout, float* dq, float* dk, float* dv,
                           int B, int H, int N, int W, int d, int causal_window, tlin_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * Exact merge of two results over DISJOINT key sets for the same queries (not in the paper; it is
 * the split-K combine, exposed so that "history" and "window" attention may also be computed
 * separately and joined): lse = log(e^lse_a + e^lse_b), out = (e^lse_a out_a + e^lse_b out_b)/e^lse.
 * An lse of -inf marks an empty side.  out_* [rows,d] bf16 (or fp32 for _f32), lse_* [rows] fp32.
 * out/lse may alias out_a/lse_a.
 */
int tlin_merge_lse(const void* out_a, const float* lse_a, const void* out_b, const float* lse_b,
                   void* out, float* lse, int64_t rows, int d, tlin_stream_t stream);
int tlin_merge_lse_f32(const float* out_a, const float* lse_a, const float* out_b, const float* lse_b,
                       float* out, float* lse, int64_t rows, int d, tlin_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * Workspace.  Split-K partial results live in one caller-owned device buffer per device:
 * tlin_set_workspace registers it for the device that is current at the call (one buffer per device and
 * process), borrowed until replaced; compute calls use the buffer of their current device.  Calls on
 * different streams that both need the workspace must not overlap.  The *_bytes functions are pure host
 * arithmetic.  With TLIN_LOG=1 in the environment every compute call prints the plan it chose to stderr.
 */
size_t tlin_workspace_bytes_forward(int B, int H, int N, int W, int d, int causal_window);
size_t tlin_workspace_bytes_decode(int B, int H, int Ncap, int d);
size_t tlin_workspace_bytes_forward_prefixes(int B, int H, int W, int d, int C, const int32_t* n_keys, int causal_window);
size_t tlin_workspace_bytes_backward(int B, int H, int N, int W, int d);
int tlin_set_workspace(void* dev_ptr, size_t bytes);

/* ------------------------------------------------------------------------------------------
 * Host-side planning (pure integer arithmetic; callable without a GPU).  The paper is silent on
 * scheduling; its integer shadow is the cost model of Section 4 / Appendix A: the allowed
 * (query,key) pairs of a call number W*N without a mask and W*(N-W) + W*(W+1)/2 with the window.
 */
typedef struct {
    int32_t tile_m;        /* query rows per CTA                                             */
    int32_t tile_n;        /* keys per tile                                                  */
    int32_t q_tiles;       /* ceil(W / tile_m): CTAs that share one key range                */
    int32_t key_tiles;     /* ceil(N / tile_n) per (b,h)                                     */
    int32_t n_groups;      /* group g owns units [start(g), start(g+1)); see `schedule`       */
    int32_t n_ctas;        /* schedule 0: n_groups * q_tiles; schedule 1: n_groups            */
    int64_t total_units;   /* schedule 0: B*H*key_tiles, unit u = (bh = u / key_tiles, tile = u % key_tiles);
                              schedule 1: B*H*q_tiles,  unit u = (bh = u / q_tiles,  q tile = u % q_tiles) */
    int32_t uses_workspace;/* 1 if any (b,h) is split between groups                         */
    int32_t tensor_path;   /* 1 = tcgen05 kernel, 0 = CUDA-core kernel                       */
    int64_t workspace_bytes;
    int32_t schedule;      /* 0: a group of q_tiles CTAs streams a range of (b,h,key tile) units, the key range of
                              a (b,h) may be split between groups (few query rows, long context: Section 3,
                              focused attention and the generation window);
                              1: every CTA works through whole (b,h,query tile) problems, keys never split
                              (many query rows, short context: the restoring cross-attention of Section 3) */
    int32_t causal_window; /* the call's mask, N and W: the group boundaries of schedule 1 depend on them              */
    int32_t n_keys;
    int32_t n_queries;
} tlin_fwd_plan;

typedef struct {
    int32_t splits;        /* CTAs per (b,h)                                                 */
    int32_t keys_per_split;/* split s covers keys [s*keys_per_split, min(L, (s+1)*keys_per_split)) */
    int32_t n_ctas;
    int64_t workspace_bytes;
} tlin_decode_plan;

/* num_sms <= 0 means "use the value of the B200 (148)". */
int tlin_plan_forward(int B, int H, int N, int W, int d, int causal_window, int is_f32, int num_sms, tlin_fwd_plan* plan);
int tlin_plan_decode(int B, int H, int L, int d, int num_sms, tlin_decode_plan* plan);
/* Work sharing of the tensor-core dK/dV kernel of tlin_attn_backward: its units are (b,h,128-key tile) in that order and
 * CTA `share` of `n_shares` starts at the unit returned here (share = n_shares gives the unit count B*H*ceil(N/128)).  The
 * shares are balanced by the number of 128-row query tiles each key tile has to visit, which under the window rule falls
 * towards the end of a (b,h).  -1 on bad arguments. */
int64_t tlin_plan_backward_share_start(int B, int H, int N, int W, int causal_window, int share, int n_shares);
/* First unit of group g.  floor(g * total_units / n_groups), except under schedule 1 with the window rule: there a
 * (b,h,query tile) problem costs the key tiles its rows may use (+3 for starting and finishing it and for its masked steps), which grows with the
 * query tile, and when there are at least three problems per group the groups take contiguous runs of problems whose
 * costliest run is as cheap as contiguous runs allow (long problems) and which stay close to equal shares of the cost. */
int64_t tlin_plan_group_start(const tlin_fwd_plan* plan, int g);
/* Mask predicate: may query i (0 <= i < W) use key j?  1 or 0. */
int tlin_allowed(int64_t i, int64_t j, int64_t N, int64_t W, int causal_window);
/* Class of key tile `kt` for query tile `qt`: 0 = no allowed pair (skipped), 1 = every in-range pair
 * allowed and the tile lies fully inside [0,N), 2 = mixed (masked element by element). */
int tlin_tile_class(int64_t N, int64_t W, int causal_window, int tile_m, int tile_n, int qt, int kt);

/* ------------------------------------------------------------------------------------------
 * Status and options.
 */
/* Synchronises `stream`, then returns and clears the device-side error word of the current device:
 *   TLIN_OK               nothing was reported since the last call;
 *   TLIN_ERR_TIMEOUT      a bounded device-side wait of a tensor-core kernel ran out (the CTA drained and left);
 *   TLIN_ERR_INVALID_ARG  tlin_decode_step_ragged met a pos[b] outside its bounds (only the kernel can see it);
 *   TLIN_ERR_CUDA         a backward tensor-core kernel found its shared-memory layout unusable and did no work,
 *                         or the stream / a copy reported an error.
 * When several kernels reported, the last writer's code is returned. */
int tlin_get_status(tlin_stream_t stream);
/* Diagnostic (not in the paper): launches one tiny kernel that waits, with the bounded wait of the tensor-core
 * kernels, on a barrier nothing ever signals.  The wait gives up after `limit_cycles` SM clocks (1 .. 2e9) and the
 * kernel reports TLIN_ERR_TIMEOUT through tlin_get_status, which is how a stalled attention kernel would end.
 * waited_cycles: DEVICE pointer to one int64 receiving the clocks the kernel spent waiting, or NULL.
 * Nothing faults or hangs; the library stays usable. */
int tlin_debug_wait_expires(long long limit_cycles, long long* waited_cycles, tlin_stream_t stream);
const char* tlin_status_string(int status);
const char* tlin_version(void);
/* Which kernel serves tlin_attn_forward: 0 = automatic, 1 = always the CUDA-core kernel,
 * 2 = tensor-core kernel (TLIN_ERR_UNSUPPORTED if the shape does not allow it).  tlin_attn_backward follows the same
 * switch (1 = CUDA-core kernels for every head size).  Returns the old value. */
int tlin_set_forward_impl(int impl);
/* How the tensor-core kernels of tlin_attn_backward (bf16, d = 64 or 128) are arranged; the chain rule of the Section 3
 * attention formula is the same in both (the paper gives no gradient algorithm of its own):
 *   1 = two kernels, dK/dV and then dQ, each recomputing the scores: seven matrix products per (query, key) pair, no atomics,
 *       bitwise repeatable;
 *   2 = one kernel (d = 128 only; d = 64 keeps the two kernels): scores computed once, five matrix products per pair; the dQ
 *       contribution of every (128-key, 64-query) block is added to an fp32 buffer in the workspace by reductions in L2 and
 *       rounded to bf16 at the end, so dQ repeats only up to the order of those fp32 additions (dK, dV stay bitwise
 *       repeatable); needs B*H*ceil(W/128)*128*(d+2)*4 bytes of workspace, which tlin_workspace_bytes_backward includes;
 *   0 (the default) = the library chooses: arrangement 2 at d = 128 while that fp32 dQ buffer is at most 64 MiB (2 to 13 %
 *       faster on B200), arrangement 1 otherwise (beyond that size the two are level: the reductions, not the matrix
 *       products, bound arrangement 2).
 * Set 1 where bitwise repeatable gradients are needed.  Returns the old value; TLIN_ERR_INVALID_ARG for another argument.
 * tlin_backward_arrangement: the arrangement (1 or 2) a call with these sizes gets under the current setting; host-only. */
int tlin_set_backward_impl(int impl);
int tlin_backward_arrangement(int B, int H, int N, int W, int d);
/* Number of kernels launched by the last tlin_* compute call on this thread. */
int tlin_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TLIN_H */
