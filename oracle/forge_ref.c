/*
 * forge_ref.c -- CPU oracle for fused scaled-dot-product attention and the fused
 * Linear + bias + tanh-GELU.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of what
 * the fused patterns compute.  It is used by the tests, by the smoke check and by
 * the benchmark's CPU-baseline leg; the product (the CUDA library) never links,
 * loads or calls it, and shares no code, header, table or helper with it.
 *
 * What it follows:
 *   - attention: the unfused chain  Q.K^T -> scale -> [mask] -> softmax -> .V
 *     (Eq. 8) whose result the fused operator must preserve, i.e.
 *     softmax(scale * Q K^T) V (Eq. 9) with the mask applied as exclusion of
 *     keys before the softmax.  Grouped-query heads: query head h reads KV head
 *     h / (Hq / Hkv).
 *   - decode: the same definition with one query row per (batch, head) over the
 *     first lens[b] rows of a KV cache.  The number of splits is not part of the
 *     definition (the split/combine is an identity in exact arithmetic).
 *   - linear: y = gelu_tanh(x W + b) for W stored [K, N] (Listing 6 / Eq. 11:
 *     matmul, element-wise bias add, activation, one dispatch).
 *
 * There is no blocking, fusion, online rescaling or reordering here: scores for a
 * row are all computed, the maximum is taken, exponentials are normalised, and
 * the weighted sum over V is formed, in that order.  OpenMP, when enabled, only
 * distributes independent (batch, head) pairs or output rows over threads.
 *
 * Layouts (row-major, last index fastest):
 *   q, out : [B, Hq, Sq, D]     k, v : [B, Hkv, Skv, D]     lens : int32 [B]
 *   probs  : [B, Hq, Sq, Skv]
 *   x : [M, K]   w : [K, N]   b : [N]   y : [M, N]
 *
 * mask_kind: 0 none, 1 causal, 2 key padding (key j valid iff j < lens[b]),
 *            3 causal and key padding.
 * Causal alignment when Sq != Skv is bottom-right: query i sees keys
 * j <= i + (Skv - Sq).  lens[b] is clamped to [0, Skv].  A row with no allowed
 * key produces zeros (and an all-zero probability row).
 *
 * Additive bias (the optional mask node of Eq. 8 as a tensor): bias [B, Hb, Sq, Skv]
 * with Hb = 1 (shared by all heads) or Hb = Hq is added to the scaled scores before
 * the softmax: s = scale * q.k + bias.  A bias of -infinity excludes the key, like
 * the mask kinds do; the mask kinds still apply on top.
 *
 * Every function returns 0 on success, 1 on an invalid argument.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

static int kv_limit(int mask_kind, const int32_t *lens, int b, int Skv)
{
    int n = Skv;
    if (mask_kind & 2) {
        n = lens[b];
        if (n < 0) n = 0;
        if (n > Skv) n = Skv;
    }
    return n;
}

/* 1 if key j is visible to query i under the mask. */
static int allowed(int mask_kind, int i, int j, int Sq, int Skv, int kvlen)
{
    if (j >= kvlen) return 0;
    if ((mask_kind & 1) && j > i + (Skv - Sq)) return 0;
    return 1;
}

static int check_attn_args(const void *q, const void *k, const void *v, const void *out,
                           int B, int Hq, int Hkv, int Sq, int Skv, int D,
                           int mask_kind, const int32_t *lens)
{
    if (!q || !k || !v || !out) return 1;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Skv <= 0 || D <= 0) return 1;
    if (Hq % Hkv != 0) return 1;
    if (mask_kind < 0 || mask_kind > 3) return 1;
    if ((mask_kind & 2) && !lens) return 1;
    return 0;
}

/*
 * One attention row (Eq. 9 restricted to the allowed keys).  p has room for Skv
 * doubles and receives the probabilities (exact 0.0 where masked).
 */
static void attn_row(const double *qrow, const double *kmat, const double *vmat, double *orow,
                     double *p, int i, int Sq, int Skv, int D, int mask_kind, int kvlen, double scale,
                     const double *bias_row)
{
    double m = -INFINITY;
    int any = 0;
    for (int j = 0; j < Skv; ++j) {
        if (!allowed(mask_kind, i, j, Sq, Skv, kvlen) || (bias_row && bias_row[j] == -INFINITY)) {
            p[j] = -INFINITY;  /* marks an excluded key until the probabilities are written */
            continue;
        }
        double s = 0.0;
        for (int d = 0; d < D; ++d) s += qrow[d] * kmat[(size_t)j * D + d];
        s *= scale;
        if (bias_row) s += bias_row[j];
        p[j] = s;
        if (!any || s > m) m = s;
        any = 1;
    }
    for (int d = 0; d < D; ++d) orow[d] = 0.0;
    if (!any) {
        for (int j = 0; j < Skv; ++j) p[j] = 0.0;
        return;
    }

    double denom = 0.0;
    for (int j = 0; j < Skv; ++j) {
        if (p[j] == -INFINITY) continue;
        p[j] = exp(p[j] - m);
        denom += p[j];
    }
    for (int j = 0; j < Skv; ++j) {
        if (p[j] == -INFINITY) { p[j] = 0.0; continue; }
        p[j] /= denom;
        for (int d = 0; d < D; ++d) orow[d] += p[j] * vmat[(size_t)j * D + d];
    }
}

static int attn_impl(const double *q, const double *k, const double *v, double *out, double *probs,
                     int B, int Hq, int Hkv, int Sq, int Skv, int D,
                     int mask_kind, const int32_t *lens, double scale, const double *bias, int Hb)
{
    if (check_attn_args(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens)) return 1;
    if (bias && Hb != 1 && Hb != Hq) return 1;
    const int G = Hq / Hkv;
    int failed = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hq; ++h) {
            const int kvh = h / G;
            const int kvlen = kv_limit(mask_kind, lens, b, Skv);
            const double *kmat = k + ((size_t)b * Hkv + kvh) * (size_t)Skv * D;
            const double *vmat = v + ((size_t)b * Hkv + kvh) * (size_t)Skv * D;
            double *scratch = probs ? NULL : (double *)malloc(sizeof(double) * (size_t)Skv);
            if (!probs && !scratch) { failed = 1; continue; }
            for (int i = 0; i < Sq; ++i) {
                size_t row = ((size_t)b * Hq + h) * (size_t)Sq + i;
                double *p = probs ? probs + row * (size_t)Skv : scratch;
                const double *bias_row = bias ? bias + (((size_t)b * Hb + (Hb == 1 ? 0 : h)) * (size_t)Sq + i) * (size_t)Skv : NULL;
                attn_row(q + row * D, kmat, vmat, out + row * D, p, i, Sq, Skv, D, mask_kind, kvlen, scale, bias_row);
            }
            free(scratch);
        }
    }
    return failed;
}

/* Fused attention result (Eq. 8 / Eq. 9). */
int forge_ref_attn(const double *q, const double *k, const double *v, double *out,
                   int B, int Hq, int Hkv, int Sq, int Skv, int D,
                   int mask_kind, const int32_t *lens, double scale)
{
    return attn_impl(q, k, v, out, NULL, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, NULL, 0);
}

/* Same, and also returns the probability matrix softmax(mask(scale Q K^T)) that the
 * unfused chain of Eq. 8 would have materialised.  For small shapes. */
int forge_ref_attn_probs(const double *q, const double *k, const double *v, double *out, double *probs,
                         int B, int Hq, int Hkv, int Sq, int Skv, int D,
                         int mask_kind, const int32_t *lens, double scale)
{
    if (!probs) return 1;
    return attn_impl(q, k, v, out, probs, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, NULL, 0);
}

/* Fused attention with an additive bias tensor [B, Hb, Sq, Skv] on the scaled scores (Eq. 8 with its
 * optional mask node as a tensor).  probs may be NULL. */
int forge_ref_attn_bias(const double *q, const double *k, const double *v, double *out, double *probs,
                        int B, int Hq, int Hkv, int Sq, int Skv, int D,
                        int mask_kind, const int32_t *lens, double scale, const double *bias, int Hb)
{
    if (!bias) return 1;
    return attn_impl(q, k, v, out, probs, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, bias, Hb);
}

/*
 * Decode step: q, out [B, Hq, D]; caches [B, Hkv, Smax, D]; sequence b attends its
 * first lens[b] cached rows.  This is Eq. 9 with a single query row per head.
 */
int forge_ref_attn_decode(const double *q, const double *k_cache, const double *v_cache, double *out,
                          int B, int Hq, int Hkv, int Smax, int D, const int32_t *lens, double scale)
{
    if (!lens) return 1;
    return attn_impl(q, k_cache, v_cache, out, NULL, B, Hq, Hkv, 1, Smax, D, 2, lens, scale, NULL, 0);
}

/* tanh form of GELU: 0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3))). */
double forge_ref_gelu_tanh(double z)
{
    const double c = sqrt(2.0 / M_PI);
    return 0.5 * z * (1.0 + tanh(c * (z + 0.044715 * z * z * z)));
}

/* y[m, n] = gelu_tanh(b[n] + sum_k x[m, k] w[k, n])  (Listing 6 / Eq. 11). */
int forge_ref_linear_bias_gelu(const double *x, const double *w, const double *b, double *y,
                               int M, int N, int K)
{
    if (!x || !w || !b || !y || M <= 0 || N <= 0 || K <= 0) return 1;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int kk = 0; kk < K; ++kk) acc += x[(size_t)m * K + kk] * w[(size_t)kk * N + n];
            y[(size_t)m * N + n] = forge_ref_gelu_tanh(acc + b[n]);
        }
    }
    return 0;
}

/*
 * The other patterns the operator-fusion pass produces (Section 4.3 "Pass 5": linear+relu, linear+gelu,
 * linear+silu, and mm+add, a residual addition after a raw matrix multiply):
 *     y[m, n] = act(b[n] + sum_k x[m, k] W(k, n)) + r[m, n]
 * act: 0 tanh-GELU, 1 erf-GELU (0.5 z (1 + erf(z / sqrt 2))), 2 ReLU, 3 SiLU (z / (1 + e^-z)), 4 identity.
 * w_layout: 0 = w stored [K, N]; 1 = w stored [N, K], the [out, in] layout of the listing's Linear.
 * b (length N) and r ([M, N]) may be NULL and then contribute nothing.
 */
int forge_ref_linear_act(const double *x, const double *w, const double *b, const double *r, double *y,
                         int M, int N, int K, int act, int w_layout)
{
    if (!x || !w || !y || M <= 0 || N <= 0 || K <= 0) return 1;
    if (act < 0 || act > 4 || w_layout < 0 || w_layout > 1) return 1;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            double z = 0.0;
            for (int kk = 0; kk < K; ++kk) {
                const double wkn = w_layout == 0 ? w[(size_t)kk * N + n] : w[(size_t)n * K + kk];
                z += x[(size_t)m * K + kk] * wkn;
            }
            if (b) z += b[n];
            double a;
            switch (act) {
            case 0: a = forge_ref_gelu_tanh(z); break;
            case 1: a = 0.5 * z * (1.0 + erf(z / sqrt(2.0))); break;
            case 2: a = z > 0.0 ? z : 0.0; break;
            case 3: a = z / (1.0 + exp(-z)); break;
            default: a = z; break;
            }
            if (r) a += r[(size_t)m * N + n];
            y[(size_t)m * N + n] = a;
        }
    }
    return 0;
}

/* Number of OpenMP threads the loops above will use (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int forge_ref_num_threads(void) { return omp_get_max_threads(); }
#else
int forge_ref_num_threads(void) { return 1; }
#endif

/*
 * Gated MLP input (SwiGLU, the form the 1B-8B decoder models of the evaluation use; the operator-fusion
 * pass's linear+silu pattern followed by the element-wise product with a second projection):
 *     y[m, n] = silu(sum_k x[m, k] wg(k, n)) * (sum_k x[m, k] wu(k, n)),   silu(z) = z / (1 + exp(-z))
 * wg, wu stored [K, N] (w_layout 0) or [N, K] (w_layout 1).
 */
int forge_ref_linear_swiglu(const double *x, const double *wg, const double *wu, double *y,
                            int M, int N, int K, int w_layout)
{
    if (!x || !wg || !wu || !y || M <= 0 || N <= 0 || K <= 0) return 1;
    if (w_layout < 0 || w_layout > 1) return 1;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            double gate = 0.0, up = 0.0;
            for (int kk = 0; kk < K; ++kk) {
                const size_t wi = w_layout == 0 ? (size_t)kk * N + n : (size_t)n * K + kk;
                gate += x[(size_t)m * K + kk] * wg[wi];
                up += x[(size_t)m * K + kk] * wu[wi];
            }
            y[(size_t)m * N + n] = gate / (1.0 + exp(-gate)) * up;
        }
    }
    return 0;
}

/*
 * Weight-only int8 linear (the W-int8 / A-fp16 setting of the evaluation's largest model): symmetric
 * per-output-channel quantisation, w(k, n) = scale[n] * wq[n, k] with wq integers in [-128, 127]:
 *     y[m, n] = act(scale[n] * sum_k x[m, k] wq[n, k] + b[n]) + r[m, n]
 * wq is stored [N, K] (given here as doubles holding the integers); b and r may be NULL; act as in
 * forge_ref_linear_act.
 */
int forge_ref_linear_w8(const double *x, const double *wq, const double *scale, const double *b, const double *r,
                        double *y, int M, int N, int K, int act)
{
    if (!x || !wq || !scale || !y || M <= 0 || N <= 0 || K <= 0) return 1;
    if (act < 0 || act > 4) return 1;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            double z = 0.0;
            for (int kk = 0; kk < K; ++kk) z += x[(size_t)m * K + kk] * wq[(size_t)n * K + kk];
            z *= scale[n];
            if (b) z += b[n];
            double a;
            switch (act) {
            case 0: a = forge_ref_gelu_tanh(z); break;
            case 1: a = 0.5 * z * (1.0 + erf(z / sqrt(2.0))); break;
            case 2: a = z > 0.0 ? z : 0.0; break;
            case 3: a = z / (1.0 + exp(-z)); break;
            default: a = z; break;
            }
            if (r) a += r[(size_t)m * N + n];
            y[(size_t)m * N + n] = a;
        }
    }
    return 0;
}
