/*
 * CPU oracle for the TLinFormer attention hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 statement of what the GPU library must compute.  It is
 * used by the tests, by the smoke check and by the benchmark's CPU-baseline
 * leg, never by the product path, and it shares no code, header, table or
 * helper with the CUDA sources.
 *
 * What it follows (paper: "Rethinking Transformer Connectivity: TLinFormer"):
 *   - Section 3, the attention formula  softmax(Q K^T / sqrt(d_k)) V.  The
 *     method is exact (no approximation), so the oracle is that definition
 *     written out: every row's scores are materialised, the maximum is taken,
 *     the exponentials are summed, and the values are averaged.  Two passes, no
 *     tiling, no running maximum.
 *   - Section 3, "Causal Attention": query i may use keys j <= i.  When the W
 *     queries are the last W positions of an N-long sequence (history followed
 *     by the generation window, Fig. "ideal connection"), query i sits at
 *     absolute position N-W+i, hence the rule j <= N-W+i.
 *   - Section 3, "Focused Attention" / "Cross Attention": a few queries over all
 *     keys, unmasked (causal_window = 0).
 *   - Appendix A, "Cache Hit": in a cached step only the newest token takes
 *     part; it attends to every cached row including its own.
 *   - Section 4.1: training is a forward and a backward pass through every
 *     layer.  The paper states no gradient algorithm; tlin_ref_attn_backward
 *     is the chain rule of the formula above written out row by row (pinned by
 *     central differences of the forward, a library autograd and closed forms).
 *
 * Every function is pinned by tests that do not call it to produce their
 * expectation (closed forms, brute force with an explicit probability matrix,
 * a textbook library routine, invariants); no function here is "parity
 * unpinned".
 *
 * Element types: 0 = bfloat16 bit patterns (uint16_t), 1 = IEEE float.
 * Inputs are widened exactly to double.  Outputs are double.
 * Threads: rows are independent; an OpenMP parallel-for hands them out.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { TLIN_REF_BF16 = 0, TLIN_REF_F32 = 1, TLIN_REF_F64 = 2 /* internal: values already widened */ };

static double widen(const void *base, int elem_type, int64_t idx)
{
    if (elem_type == TLIN_REF_BF16) {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    if (elem_type == TLIN_REF_F64) return ((const double *)base)[idx];
    return (double)((const float *)base)[idx];
}

int tlin_ref_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Mask predicate (Section 3, causal rule, aligned to the end of the sequence). */
int tlin_ref_allowed(int64_t i, int64_t j, int64_t N, int64_t W, int causal_window)
{
    if (j < 0 || j >= N) return 0;
    if (causal_window) return j <= (N - W) + i;
    return 1;
}

/*
 * One query row against key/value rows [0, N): the attention formula of
 * Section 3 with the mask above.  scores is caller scratch of N doubles.
 */
static void attend_row(const void *q, const void *k, const void *v, int elem_type,
                       int64_t qoff, int64_t kvoff, int64_t i, int64_t N, int64_t W, int d,
                       int causal_window, double *scores, double *out_row, double *lse_out)
{
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    double m = -INFINITY;
    for (int64_t j = 0; j < N; ++j) {
        if (!tlin_ref_allowed(i, j, N, W, causal_window)) { scores[j] = -INFINITY; continue; }
        double s = 0.0;
        for (int c = 0; c < d; ++c)
            s += widen(q, elem_type, qoff + c) * widen(k, elem_type, kvoff + j * d + c);
        s *= inv_sqrt_d;
        scores[j] = s;
        if (s > m) m = s;
    }
    double l = 0.0;
    for (int c = 0; c < d; ++c) out_row[c] = 0.0;
    for (int64_t j = 0; j < N; ++j) {
        if (scores[j] == -INFINITY) continue;
        double p = exp(scores[j] - m);
        l += p;
        for (int c = 0; c < d; ++c) out_row[c] += p * widen(v, elem_type, kvoff + j * d + c);
    }
    for (int c = 0; c < d; ++c) out_row[c] /= l;
    *lse_out = m + log(l);
}

/*
 * q:[B,H,W,d]  k,v:[B,H,N,d]  ->  out:[B,H,W,d] (double)  lse:[B,H,W] (double)
 * causal_window = 0: every query sees all N keys.
 * causal_window = 1: query i sees key j iff j <= N-W+i; requires N >= W.
 * Returns 0, or -1 on a bad argument.
 */
int tlin_ref_attn_forward(const void *q, const void *k, const void *v, int elem_type,
                          double *out, double *lse,
                          int B, int H, int64_t N, int64_t W, int d, int causal_window)
{
    if (!q || !k || !v || !out || !lse) return -1;
    if (B <= 0 || H <= 0 || N <= 0 || W <= 0 || d <= 0) return -1;
    if (causal_window && N < W) return -1;
    if (elem_type != TLIN_REF_BF16 && elem_type != TLIN_REF_F32) return -1;
    const int64_t rows = (int64_t)B * H * W;
    int failed = 0;
#pragma omp parallel
    {
        double *scores = (double *)malloc((size_t)N * sizeof(double));
        if (!scores) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (int64_t r = 0; r < rows; ++r) {
            if (!scores) continue;
            const int64_t bh = r / W, i = r % W;
            attend_row(q, k, v, elem_type, (bh * W + i) * d, bh * N * d, i, N, W, d,
                       causal_window, scores, out + r * d, lse + r);
        }
        free(scores);
    }
    return failed ? -2 : 0;
}

/*
 * One cached decode step (Appendix A, "Cache Hit"; Section 5.2, static history
 * cache).  k_cache,v_cache:[B,H,Ncap,d] hold `pos` valid rows.  The new key and
 * value ([B,H,1,d]) are copied verbatim into row `pos`, then the new query
 * attends to rows [0, pos] (its own row included, causal rule j <= i).
 * The caches are modified in place.  out:[B,H,1,d], lse:[B,H].
 */
int tlin_ref_decode_step(const void *q_new, const void *k_new, const void *v_new,
                         void *k_cache, void *v_cache, int elem_type,
                         double *out, double *lse,
                         int B, int H, int64_t Ncap, int64_t pos, int d)
{
    if (!q_new || !k_new || !v_new || !k_cache || !v_cache || !out || !lse) return -1;
    if (B <= 0 || H <= 0 || d <= 0 || Ncap <= 0 || pos < 0 || pos >= Ncap) return -1;
    if (elem_type != TLIN_REF_BF16 && elem_type != TLIN_REF_F32) return -1;
    const size_t esz = elem_type == TLIN_REF_BF16 ? 2 : 4;
    const int64_t L = pos + 1;
    int failed = 0;
#pragma omp parallel
    {
        double *scores = (double *)malloc((size_t)L * sizeof(double));
        if (!scores) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int64_t bh = 0; bh < (int64_t)B * H; ++bh) {
            if (!scores) continue;
            char *kc = (char *)k_cache + (size_t)(bh * Ncap) * d * esz;
            char *vc = (char *)v_cache + (size_t)(bh * Ncap) * d * esz;
            memcpy(kc + (size_t)pos * d * esz, (const char *)k_new + (size_t)bh * d * esz, (size_t)d * esz);
            memcpy(vc + (size_t)pos * d * esz, (const char *)v_new + (size_t)bh * d * esz, (size_t)d * esz);
            /* a single unmasked query over the L rows now valid */
            attend_row(q_new, kc, vc, elem_type, bh * d, 0, 0, L, 1, d, 0, scores, out + bh * d, lse + bh);
        }
        free(scores);
    }
    return failed ? -2 : 0;
}

/*
 * 8-bit floating point, E4M3 (the "FN" variant of the OCP 8-bit floating point
 * specification): 1 sign bit, 4 exponent bits with bias 7, 3 mantissa bits; no
 * infinities; S.1111.111 is NaN; the largest finite value is S.1111.110 = 448;
 * exponent field 0 holds the subnormals m * 2^-9.  Not in the paper: it is the
 * storage format of the optional 8-bit key/value cache.
 */
double tlin_ref_e4m3_decode(uint8_t code)
{
    const int sign = code >> 7, e = (code >> 3) & 15, m = code & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m, -9);
    else v = ldexp(1.0 + m / 8.0, e - 7);
    return sign ? -v : v;
}

/* Nearest finite code, ties to the code with an even mantissa, magnitudes beyond 448 saturate; NaN -> 0x7f. */
uint8_t tlin_ref_e4m3_encode(float x)
{
    if (x != x) return 0x7f;
    const uint8_t sign = signbit(x) ? 0x80 : 0x00;
    const double a = fabs((double)x);
    int best = 0;
    double best_err = INFINITY;
    for (int c = 0; c <= 0x7e; ++c) {          /* the 127 finite non-negative codes, in increasing order of value */
        const double err = fabs(tlin_ref_e4m3_decode((uint8_t)c) - a);
        if (err < best_err || (err == best_err && (c & 1) == 0)) { best_err = err; best = c; }
    }
    return (uint8_t)(sign | best);
}

/*
 * The cached decode step over an 8-bit cache.  k_cache,v_cache:[B,H,Ncap,d] bytes (E4M3 codes); the value of
 * an element is decode(code) * scale, with one fp32 scale per (b,h) for keys and one for values.  The new key
 * and value rows (bf16) are stored as encode(x / scale), the division carried out in fp32 (the precision in
 * which the kernel takes the same decision); the new query (bf16) then attends to the decoded rows [0, pos],
 * its own included.  out:[B,H,1,d], lse:[B,H].
 */
int tlin_ref_decode_step_fp8(const uint16_t *q_new, const uint16_t *k_new, const uint16_t *v_new,
                             uint8_t *k_cache, uint8_t *v_cache, const float *k_scale, const float *v_scale,
                             double *out, double *lse, int B, int H, int64_t Ncap, int64_t pos, int d)
{
    if (!q_new || !k_new || !v_new || !k_cache || !v_cache || !k_scale || !v_scale || !out || !lse) return -1;
    if (B <= 0 || H <= 0 || d <= 0 || Ncap <= 0 || pos < 0 || pos >= Ncap) return -1;
    const int64_t L = pos + 1;
    int failed = 0;
#pragma omp parallel
    {
        double *scores = (double *)malloc((size_t)L * sizeof(double));
        double *kd = (double *)malloc((size_t)L * d * sizeof(double));
        double *vd = (double *)malloc((size_t)L * d * sizeof(double));
        double *qd = (double *)malloc((size_t)d * sizeof(double));
        if (!scores || !kd || !vd || !qd) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int64_t bh = 0; bh < (int64_t)B * H; ++bh) {
            if (!scores || !kd || !vd || !qd) continue;
            uint8_t *kc = k_cache + (size_t)(bh * Ncap) * d, *vc = v_cache + (size_t)(bh * Ncap) * d;
            for (int c = 0; c < d; ++c) {
                const float kx = (float)widen(k_new, TLIN_REF_BF16, bh * d + c) / k_scale[bh];
                const float vx = (float)widen(v_new, TLIN_REF_BF16, bh * d + c) / v_scale[bh];
                kc[(size_t)pos * d + c] = tlin_ref_e4m3_encode(kx);
                vc[(size_t)pos * d + c] = tlin_ref_e4m3_encode(vx);
                qd[c] = widen(q_new, TLIN_REF_BF16, bh * d + c);
            }
            for (int64_t j = 0; j < L; ++j)
                for (int c = 0; c < d; ++c) {
                    kd[j * d + c] = tlin_ref_e4m3_decode(kc[(size_t)j * d + c]) * (double)k_scale[bh];
                    vd[j * d + c] = tlin_ref_e4m3_decode(vc[(size_t)j * d + c]) * (double)v_scale[bh];
                }
            attend_row(qd, kd, vd, TLIN_REF_F64, 0, 0, 0, L, 1, d, 0, scores, out + bh * d, lse + bh);
        }
        free(scores); free(kd); free(vd); free(qd);
    }
    return failed ? -2 : 0;
}

/*
 * Exact combination of two attention results over disjoint key sets A and B for
 * the same queries: with z = exp(lse), softmax over A u B weights each side by
 * z_a/(z_a+z_b) and z_b/(z_a+z_b).  lse = -inf marks an empty side.
 * out_a,out_b,out:[rows,d]  lse_a,lse_b,lse:[rows], all double.
 */
int tlin_ref_merge_lse(const double *out_a, const double *lse_a, const double *out_b, const double *lse_b,
                       double *out, double *lse, int64_t rows, int d)
{
    if (!out_a || !lse_a || !out_b || !lse_b || !out || !lse || rows < 0 || d <= 0) return -1;
    for (int64_t r = 0; r < rows; ++r) {
        const double la = lse_a[r], lb = lse_b[r];
        const double m = la > lb ? la : lb;
        if (m == -INFINITY) {
            lse[r] = -INFINITY;
            for (int c = 0; c < d; ++c) out[r * d + c] = 0.0;
            continue;
        }
        const double wa = exp(la - m), wb = exp(lb - m);
        const double z = wa + wb;
        lse[r] = m + log(z);
        for (int c = 0; c < d; ++c) out[r * d + c] = (wa * out_a[r * d + c] + wb * out_b[r * d + c]) / z;
    }
    return 0;
}

/*
 * Gradient of the forward above (training runs the same attention as a forward and a backward pass; Section 4.1
 * counts training as "cache miss" throughout).  The paper gives no formula of its own: this is the chain rule
 * applied to the attention formula of Section 3, written out row by row with the probabilities materialised.
 * For a loss L with dout = dL/dout (dL/dlse taken as zero):
 *     p_ij  = softmax_j(s_ij),  s_ij = q_i.k_j / sqrt(d)   over the allowed j
 *     dv_j  = sum_i p_ij dout_i
 *     dp_ij = dout_i . v_j
 *     ds_ij = p_ij (dp_ij - sum_j' p_ij' dp_ij')
 *     dq_i  = sum_j ds_ij k_j / sqrt(d)      dk_j = sum_i ds_ij q_i / sqrt(d)
 * q,dout:[B,H,W,d]  k,v:[B,H,N,d] (elem_type as above)  ->  dq:[B,H,W,d]  dk,dv:[B,H,N,d] (double).
 * (b,h) pairs are independent and handed out to threads; inside one the rows run in order.
 */
int tlin_ref_attn_backward(const void *q, const void *k, const void *v, const void *dout, int elem_type,
                           double *dq, double *dk, double *dv,
                           int B, int H, int64_t N, int64_t W, int d, int causal_window)
{
    if (!q || !k || !v || !dout || !dq || !dk || !dv) return -1;
    if (B <= 0 || H <= 0 || N <= 0 || W <= 0 || d <= 0) return -1;
    if (causal_window && N < W) return -1;
    if (elem_type != TLIN_REF_BF16 && elem_type != TLIN_REF_F32) return -1;
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t bh = 0; bh < (int64_t)B * H; ++bh) {
        double *p = (double *)malloc((size_t)N * sizeof(double));
        double *dp = (double *)malloc((size_t)N * sizeof(double));
        if (!p || !dp) {
#pragma omp atomic write
            failed = 1;
            free(p);
            free(dp);
            continue;
        }
        const int64_t qbase = bh * W * d, kbase = bh * N * d;
        for (int64_t x = 0; x < N * d; ++x) { dk[kbase + x] = 0.0; dv[kbase + x] = 0.0; }
        for (int64_t i = 0; i < W; ++i) {
            /* probabilities of row i */
            double m = -INFINITY;
            for (int64_t j = 0; j < N; ++j) {
                if (!tlin_ref_allowed(i, j, N, W, causal_window)) { p[j] = -INFINITY; continue; }
                double s = 0.0;
                for (int c = 0; c < d; ++c)
                    s += widen(q, elem_type, qbase + i * d + c) * widen(k, elem_type, kbase + j * d + c);
                p[j] = s * inv_sqrt_d;
                if (p[j] > m) m = p[j];
            }
            double l = 0.0;
            for (int64_t j = 0; j < N; ++j) {
                p[j] = (p[j] == -INFINITY) ? 0.0 : exp(p[j] - m);
                l += p[j];
            }
            double delta = 0.0;
            for (int64_t j = 0; j < N; ++j) {
                p[j] /= l;
                double t = 0.0;
                for (int c = 0; c < d; ++c)
                    t += widen(dout, elem_type, qbase + i * d + c) * widen(v, elem_type, kbase + j * d + c);
                dp[j] = t;
                delta += p[j] * t;
            }
            for (int c = 0; c < d; ++c) dq[qbase + i * d + c] = 0.0;
            for (int64_t j = 0; j < N; ++j) {
                if (p[j] == 0.0) continue;
                const double ds = p[j] * (dp[j] - delta) * inv_sqrt_d;
                for (int c = 0; c < d; ++c) {
                    dq[qbase + i * d + c] += ds * widen(k, elem_type, kbase + j * d + c);
                    dk[kbase + j * d + c] += ds * widen(q, elem_type, qbase + i * d + c);
                    dv[kbase + j * d + c] += p[j] * widen(dout, elem_type, qbase + i * d + c);
                }
            }
        }
        free(p);
        free(dp);
    }
    return failed ? -2 : 0;
}
