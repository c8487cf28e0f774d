/*
 * CPU oracle for the A/F decode-layer hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64 restatement of what one decoder-layer decode step computes
 * when it is split into an Attention side and an FFN side (the A/F split of the
 * paper's Section 4.3: the Attention group sends its outputs to the FFN group,
 * which returns the hidden states).  The paper delegates the operators'
 * arithmetic to the serving engine it builds on, so each function below is the
 * textbook definition of the operator, written as straight loops:
 *
 *   - decode attention: one query per sequence over its whole paged KV cache
 *     (the operator Sections 1-2 call memory-bound on KV-cache reads);
 *   - dense SwiGLU FFN and top-k mixture-of-experts FFN (the operator Section 1
 *     calls memory-bound at small batch, compute-bound at large batch; the two
 *     model families of Section 6.1);
 *   - the layer step = attention -> output projection -> FFN, which by
 *     definition does not depend on how the batch is cut into microbatches
 *     (Section 4.3, Eq. 2 changes the schedule, not the result);
 *   - Eq. 2 itself (the pipeline latency model).
 *
 * No online softmax, no KV splitting, no permutation, no blocking: the CUDA
 * library reorganises these computations, the oracle does not.  Inputs are the
 * same bf16 bit patterns the GPU reads, widened exactly to double on the fly.
 * Nothing here is shared with, or imported by, the CUDA library; only tests,
 * the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Every function is pinned by CPU tests against closed forms, hand-computed
 * cases, invariants and brute force (tests/test_oracle_pins.py).
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC (no -ffast-math: sums run in the
 * written order).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_API __attribute__((visibility("default")))

ORACLE_API int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

ORACLE_API void oracle_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* bf16 bit pattern -> double, exact. */
static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ------------------------------------------------------------------------- */
/* Attention: one query against n keys/values, all in double.                */
/*   s_j = scale * <q, k_j>;  p = softmax(s);  o = sum_j p_j v_j;             */
/*   lse = max_j s_j + ln sum_j exp(s_j - max).                               */
/* keys, vals: [n][D] row-major.  n >= 1.                                     */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_attn_one_query_f64(const double* q, const double* keys, const double* vals,
                                          int n, int D, double scale, double* out, double* lse) {
    double* s = (double*)malloc(sizeof(double) * (size_t)n);
    double m = -INFINITY;
    for (int j = 0; j < n; ++j) {
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += q[d] * keys[(size_t)j * D + d];
        s[j] = scale * acc;
        if (s[j] > m) m = s[j];
    }
    double denom = 0.0;
    for (int j = 0; j < n; ++j) denom += exp(s[j] - m);
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    for (int j = 0; j < n; ++j) {
        double p = exp(s[j] - m) / denom;
        for (int d = 0; d < D; ++d) out[d] += p * vals[(size_t)j * D + d];
    }
    if (lse) *lse = m + log(denom);
    free(s);
}

/* ------------------------------------------------------------------------- */
/* Paged grouped-query decode attention on bf16 inputs.                      */
/*   q            bf16 [B][Hq][D]                                             */
/*   k_cache,v_cache bf16 [num_pages][Hkv][P][D]   (P = page_size)            */
/*   page_table   i32  [B][max_pages]; token j of sequence b lives in page     */
/*                page_table[b][j / P], slot j % P                             */
/*   seq_lens     i32  [B], each >= 1 (counts the token being decoded)         */
/* Query head h reads KV head h / (Hq/Hkv).  No mask, no positional term.      */
/*   out  f64 [B][Hq][D],  lse f64 [B][Hq] (may be NULL)                       */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_attn_decode(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                                   const int32_t* page_table, int max_pages, const int32_t* seq_lens,
                                   int B, int Hq, int Hkv, int D, int P, double scale,
                                   double* out, double* lse) {
    const int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hq; ++h) {
            const int n = seq_lens[b];
            const int g = h / G;
            double* keys = (double*)malloc(sizeof(double) * (size_t)n * D);
            double* vals = (double*)malloc(sizeof(double) * (size_t)n * D);
            double* qd = (double*)malloc(sizeof(double) * (size_t)D);
            for (int d = 0; d < D; ++d) qd[d] = bf16_to_f64(q[((size_t)b * Hq + h) * D + d]);
            for (int j = 0; j < n; ++j) {
                const int64_t page = page_table[(size_t)b * max_pages + j / P];
                const int slot = j % P;
                const size_t base = (((size_t)page * Hkv + g) * P + slot) * (size_t)D;
                for (int d = 0; d < D; ++d) {
                    keys[(size_t)j * D + d] = bf16_to_f64(k_cache[base + d]);
                    vals[(size_t)j * D + d] = bf16_to_f64(v_cache[base + d]);
                }
            }
            oracle_attn_one_query_f64(qd, keys, vals, n, D, scale,
                                      out + ((size_t)b * Hq + h) * D,
                                      lse ? lse + (size_t)b * Hq + h : NULL);
            free(keys); free(vals); free(qd);
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Linear map y[t][n] = sum_k x[t][k] * w[n][k]; x f64 [T][K], w bf16 [N][K].  */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_linear(const double* x, const uint16_t* w, int T, int K, int N, double* y) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int t = 0; t < T; ++t) {
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            const uint16_t* wr = w + (size_t)n * K;
            const double* xr = x + (size_t)t * K;
            for (int k = 0; k < K; ++k) acc += xr[k] * bf16_to_f64(wr[k]);
            y[(size_t)t * N + n] = acc;
        }
    }
}

static inline double silu(double z) { return z / (1.0 + exp(-z)); }

ORACLE_API double oracle_silu(double z) { return silu(z); }

/* ------------------------------------------------------------------------- */
/* Dense SwiGLU FFN:  y_t = W_d ( silu(W_g x_t) .* (W_u x_t) ).              */
/*   x f64 [T][H]; w_gate,w_up bf16 [I][H]; w_down bf16 [H][I]; y f64 [T][H]. */
/* The intermediate h is kept in double (no bf16 rounding).                   */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_ffn_dense_f64x(const double* x, const uint16_t* w_gate, const uint16_t* w_up,
                                      const uint16_t* w_down, int T, int H, int I, double* y) {
    double* h = (double*)malloc(sizeof(double) * (size_t)T * I);
#pragma omp parallel for collapse(2) schedule(static)
    for (int t = 0; t < T; ++t) {
        for (int i = 0; i < I; ++i) {
            double g = 0.0, u = 0.0;
            const double* xr = x + (size_t)t * H;
            for (int k = 0; k < H; ++k) {
                g += bf16_to_f64(w_gate[(size_t)i * H + k]) * xr[k];
                u += bf16_to_f64(w_up[(size_t)i * H + k]) * xr[k];
            }
            h[(size_t)t * I + i] = silu(g) * u;
        }
    }
    oracle_linear(h, w_down, T, I, H, y);
    free(h);
}

static double* widen_bf16(const uint16_t* a, size_t n) {
    double* d = (double*)malloc(sizeof(double) * n);
    for (size_t i = 0; i < n; ++i) d[i] = bf16_to_f64(a[i]);
    return d;
}

ORACLE_API void oracle_ffn_dense(const uint16_t* x, const uint16_t* w_gate, const uint16_t* w_up,
                                 const uint16_t* w_down, int T, int H, int I, double* y) {
    double* xd = widen_bf16(x, (size_t)T * H);
    oracle_ffn_dense_f64x(xd, w_gate, w_up, w_down, T, H, I, y);
    free(xd);
}

/* ------------------------------------------------------------------------- */
/* Top-k routing on fp32 logits [T][E].                                      */
/* Selection: k times, take the largest logit among the experts not yet       */
/* taken; among equal logits the lowest expert index wins.  idx[t][k] is in    */
/* descending-logit order.  A NaN logit never wins a comparison.               */
/* Gates: softmax over the K selected logits (the softmax over all E followed  */
/* by renormalising over the selected K cancels to the same thing).            */
/*   idx i32 [T][K]; gate f64 [T][K].                                          */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_moe_route(const float* logits, int T, int E, int K, int32_t* idx, double* gate) {
    for (int t = 0; t < T; ++t) {
        const float* l = logits + (size_t)t * E;
        for (int k = 0; k < K; ++k) {
            int best = -1;
            for (int e = 0; e < E; ++e) {
                int taken = 0;
                for (int kk = 0; kk < k; ++kk) if (idx[(size_t)t * K + kk] == e) taken = 1;
                if (taken) continue;
                if (best < 0) { best = e; continue; }
                /* strict '>' keeps the lowest index on ties; NaN compares false */
                if (l[e] > l[best] || (l[best] != l[best] && l[e] == l[e])) best = e;
            }
            idx[(size_t)t * K + k] = best;
        }
        double l0 = (double)l[idx[(size_t)t * K]];
        double denom = 0.0;
        for (int k = 0; k < K; ++k) denom += exp((double)l[idx[(size_t)t * K + k]] - l0);
        for (int k = 0; k < K; ++k)
            gate[(size_t)t * K + k] = exp((double)l[idx[(size_t)t * K + k]] - l0) / denom;
    }
}

/* ------------------------------------------------------------------------- */
/* Token permutation implied by the routing: counts per expert, exclusive     */
/* scan, and the position of assignment (t,k) in the expert-sorted order,      */
/* ties inside an expert broken by (t,k) lexicographic order.                  */
/*   counts i32 [E]; offsets i32 [E+1]; pos i32 [T][K].                        */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_moe_permute(const int32_t* idx, int T, int E, int K,
                                   int32_t* counts, int32_t* offsets, int32_t* pos) {
    for (int e = 0; e < E; ++e) counts[e] = 0;
    for (int i = 0; i < T * K; ++i) counts[idx[i]] += 1;
    offsets[0] = 0;
    for (int e = 0; e < E; ++e) offsets[e + 1] = offsets[e] + counts[e];
    for (int i = 0; i < T * K; ++i) {
        int rank = 0;
        for (int j = 0; j < i; ++j) if (idx[j] == idx[i]) rank += 1;
        pos[i] = offsets[idx[i]] + rank;
    }
}

/* ------------------------------------------------------------------------- */
/* Mixture-of-experts FFN: y_t = sum_k gate[t][k] * FFN_{idx[t][k]}(x_t).     */
/*   x f64 [T][H]; logits fp32 [T][E];                                         */
/*   w_gate,w_up bf16 [E][I][H]; w_down bf16 [E][H][I]; y f64 [T][H].          */
/* Optional outputs idx_out [T][K], gate_out [T][K] (NULL to skip).            */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_ffn_moe_f64x(const double* x, const float* logits,
                                    const uint16_t* w_gate, const uint16_t* w_up, const uint16_t* w_down,
                                    int T, int H, int I, int E, int K, double* y,
                                    int32_t* idx_out, double* gate_out) {
    int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)T * K);
    double* gate = (double*)malloc(sizeof(double) * (size_t)T * K);
    double* ye = (double*)malloc(sizeof(double) * (size_t)H);
    oracle_moe_route(logits, T, E, K, idx, gate);
    for (int t = 0; t < T; ++t) {
        for (int n = 0; n < H; ++n) y[(size_t)t * H + n] = 0.0;
        for (int k = 0; k < K; ++k) {
            const int e = idx[(size_t)t * K + k];
            oracle_ffn_dense_f64x(x + (size_t)t * H, w_gate + (size_t)e * I * H, w_up + (size_t)e * I * H,
                                  w_down + (size_t)e * H * I, 1, H, I, ye);
            for (int n = 0; n < H; ++n) y[(size_t)t * H + n] += gate[(size_t)t * K + k] * ye[n];
        }
    }
    if (idx_out) memcpy(idx_out, idx, sizeof(int32_t) * (size_t)T * K);
    if (gate_out) memcpy(gate_out, gate, sizeof(double) * (size_t)T * K);
    free(idx); free(gate); free(ye);
}

ORACLE_API void oracle_ffn_moe(const uint16_t* x, const float* logits,
                               const uint16_t* w_gate, const uint16_t* w_up, const uint16_t* w_down,
                               int T, int H, int I, int E, int K, double* y,
                               int32_t* idx_out, double* gate_out) {
    double* xd = widen_bf16(x, (size_t)T * H);
    oracle_ffn_moe_f64x(xd, logits, w_gate, w_up, w_down, T, H, I, E, K, y, idx_out, gate_out);
    free(xd);
}

/* Router logits from activations: l[t][e] = <x_t, w_router[e]>, in double. */
ORACLE_API void oracle_router_logits(const double* x, const uint16_t* w_router, int T, int H, int E, double* l) {
    oracle_linear(x, w_router, T, H, E, l);
}

/* ------------------------------------------------------------------------- */
/* One decoder-layer decode step, A side then F side, all in double:          */
/*   a = attention(q, kv)            [B][Hq*D]                                 */
/*   x = a W_o^T  (or x = a when w_o is NULL and Hq*D == H)                    */
/*   y = dense FFN(x)  (E == 0)   or   MoE FFN(x, logits)  (E > 0)             */
/* The boundary tensors a and x are not rounded.  attn_out may be NULL.        */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_layer_step(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                                  const int32_t* page_table, int max_pages, const int32_t* seq_lens,
                                  int B, int Hq, int Hkv, int D, int P, double scale,
                                  const uint16_t* w_o, int H, int I, int E, int K,
                                  const uint16_t* w_gate, const uint16_t* w_up, const uint16_t* w_down,
                                  const float* logits, double* attn_out, double* y) {
    const int A = Hq * D;
    double* a = attn_out ? attn_out : (double*)malloc(sizeof(double) * (size_t)B * A);
    oracle_attn_decode(q, k_cache, v_cache, page_table, max_pages, seq_lens, B, Hq, Hkv, D, P, scale, a, NULL);
    double* x = a;
    if (w_o) {
        x = (double*)malloc(sizeof(double) * (size_t)B * H);
        oracle_linear(a, w_o, B, A, H, x);
    }
    if (E == 0) oracle_ffn_dense_f64x(x, w_gate, w_up, w_down, B, H, I, y);
    else oracle_ffn_moe_f64x(x, logits, w_gate, w_up, w_down, B, H, I, E, K, y, NULL, NULL);
    if (w_o) free(x);
    if (!attn_out) free(a);
}

/* ------------------------------------------------------------------------- */
/* Eq. 2: layer time of the interleaved A/F pipeline with microbatch depth M.  */
/*   M = 1 : t_A + t_F + t_comm;   M >= 2 : max(t_A, t_F) + t_comm / M.        */
/* ------------------------------------------------------------------------- */
ORACLE_API double oracle_eq2_layer_time(double t_a, double t_f, double t_comm, int M) {
    if (M <= 1) return t_a + t_f + t_comm;
    return (t_a > t_f ? t_a : t_f) + t_comm / (double)M;
}

/* ========================================================================= */
/* The rest of the decoder layer around the A/F hot path (the Attention       */
/* group's own operators and the residual stream), so that whole layers can   */
/* be chained as in the interleaved pipeline of Section 4.3 (A of layer l+1   */
/* starts from what F of layer l returns).  The paper leaves these operators   */
/* to the two model families it serves (Section 6.1); what follows is their    */
/* public definition: pre-norm residual blocks, RMS normalisation, rotary      */
/* position embedding in the rotate-half convention, optional per-head         */
/* normalisation of queries and keys, K/V of the decoded token appended to     */
/* the paged cache in the cache's storage type (bf16).                         */
/* ========================================================================= */

/* double -> bf16 bit pattern, round to nearest even, one rounding. */
static uint16_t f64_to_bf16(double d) {
    if (d != d) return 0x7fc0;
    const uint16_t sign = signbit(d) ? 0x8000 : 0;
    const double a = fabs(d);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7f80);
    int e;
    (void)frexp(a, &e);                 /* a = m * 2^e, m in [0.5, 1) */
    int qe = e - 8;                     /* quantum 2^qe leaves 8 significant bits */
    if (e - 1 < -126) qe = -126 - 7;    /* subnormal range: fixed quantum */
    const double r = ldexp(nearbyint(ldexp(a, -qe)), qe);   /* default rounding mode: to nearest even */
    const float f = (float)r;           /* exact: r has at most 8 significant bits */
    if (isinf(f) || r > 3.3895313892515355e38) return (uint16_t)(sign | 0x7f80);
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return (uint16_t)(sign | (u >> 16));
}

ORACLE_API uint16_t oracle_f64_to_bf16(double d) { return f64_to_bf16(d); }

/* ------------------------------------------------------------------------- */
/* RMS normalisation over the last axis:                                      */
/*   y[t][i] = x[t][i] / sqrt( (1/H) sum_j x[t][j]^2 + eps ) * w[i].           */
/*   x f64 [T][H]; w bf16 [H] (NULL = all ones); y f64 [T][H].                 */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_rmsnorm(const double* x, const uint16_t* w, int T, int H, double eps, double* y) {
    for (int t = 0; t < T; ++t) {
        double ss = 0.0;
        for (int j = 0; j < H; ++j) ss += x[(size_t)t * H + j] * x[(size_t)t * H + j];
        const double r = 1.0 / sqrt(ss / (double)H + eps);
        for (int i = 0; i < H; ++i)
            y[(size_t)t * H + i] = x[(size_t)t * H + i] * r * (w ? bf16_to_f64(w[i]) : 1.0);
    }
}

/* ------------------------------------------------------------------------- */
/* Rotary position embedding, rotate-half convention, on one head vector:     */
/*   for i < D/2:  angle_i = pos * theta^(-2i/D)                               */
/*     out[i]       = v[i] cos(angle_i) - v[i + D/2] sin(angle_i)              */
/*     out[i + D/2] = v[i + D/2] cos(angle_i) + v[i] sin(angle_i)              */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_rope(const double* v, int D, double pos, double theta, double* out) {
    const int half = D / 2;
    for (int i = 0; i < half; ++i) {
        const double ang = pos * pow(theta, -2.0 * (double)i / (double)D);
        const double c = cos(ang), s = sin(ang);
        const double a = v[i], b = v[i + half];
        out[i] = a * c - b * s;
        out[i + half] = b * c + a * s;
    }
}

/* Paged GQA decode attention with the queries given in double ([B][Hq][D]). */
ORACLE_API void oracle_attn_decode_f64q(const double* q, const uint16_t* k_cache, const uint16_t* v_cache,
                                        const int32_t* page_table, int max_pages, const int32_t* seq_lens,
                                        int B, int Hq, int Hkv, int D, int P, double scale,
                                        double* out, double* lse) {
    const int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hq; ++h) {
            const int n = seq_lens[b];
            const int g = h / G;
            double* keys = (double*)malloc(sizeof(double) * (size_t)n * D);
            double* vals = (double*)malloc(sizeof(double) * (size_t)n * D);
            for (int j = 0; j < n; ++j) {
                const int64_t page = page_table[(size_t)b * max_pages + j / P];
                const size_t base = (((size_t)page * Hkv + g) * P + (size_t)(j % P)) * (size_t)D;
                for (int d = 0; d < D; ++d) {
                    keys[(size_t)j * D + d] = bf16_to_f64(k_cache[base + d]);
                    vals[(size_t)j * D + d] = bf16_to_f64(v_cache[base + d]);
                }
            }
            oracle_attn_one_query_f64(q + ((size_t)b * Hq + h) * D, keys, vals, n, D, scale,
                                      out + ((size_t)b * Hq + h) * D, lse ? lse + (size_t)b * Hq + h : NULL);
            free(keys); free(vals);
        }
    }
}

/* ------------------------------------------------------------------------- */
/* The Attention group's work before the attention operator, for the token    */
/* being decoded (position seq_lens[b] - 1 of sequence b):                     */
/*   xn  = rmsnorm(x, w_ln)                                                    */
/*   qkv = xn W_qkv^T, rows of W_qkv ordered [Hq query heads | Hkv key heads   */
/*         | Hkv value heads], D rows per head                                 */
/*   q_h = rope(norm_q(qkv_h), pos),  k_g = rope(norm_k(qkv_{Hq+g}), pos)      */
/*         (norm_* = RMS normalisation over the D entries of the head with      */
/*          weights w_qn / w_kn; skipped when the pointer is NULL)             */
/*   cache[page_table[b][pos / P]][g][pos % P] = bf16(k_g), bf16(v_g)          */
/* q_out f64 [B][Hq][D].  The caches are updated in place.                     */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_qkv_rope_append(const double* x, const uint16_t* w_ln, const uint16_t* w_qkv,
                                       const uint16_t* w_qn, const uint16_t* w_kn, double eps, double theta,
                                       uint16_t* k_cache, uint16_t* v_cache,
                                       const int32_t* page_table, int max_pages, const int32_t* seq_lens,
                                       int B, int H, int Hq, int Hkv, int D, int P, double* q_out) {
    const int N = (Hq + 2 * Hkv) * D;
    double* xn = (double*)malloc(sizeof(double) * (size_t)B * H);
    double* qkv = (double*)malloc(sizeof(double) * (size_t)B * N);
    double* tmp = (double*)malloc(sizeof(double) * (size_t)D);
    double* rot = (double*)malloc(sizeof(double) * (size_t)D);
    oracle_rmsnorm(x, w_ln, B, H, eps, xn);
    oracle_linear(xn, w_qkv, B, H, N, qkv);
    for (int b = 0; b < B; ++b) {
        const int pos = seq_lens[b] - 1;
        const int64_t page = page_table[(size_t)b * max_pages + pos / P];
        for (int h = 0; h < Hq; ++h) {
            const double* v = qkv + (size_t)b * N + (size_t)h * D;
            if (w_qn) { oracle_rmsnorm(v, w_qn, 1, D, eps, tmp); v = tmp; }
            oracle_rope(v, D, (double)pos, theta, q_out + ((size_t)b * Hq + h) * D);
        }
        for (int g = 0; g < Hkv; ++g) {
            const size_t base = (((size_t)page * Hkv + g) * P + (size_t)(pos % P)) * (size_t)D;
            const double* kk = qkv + (size_t)b * N + (size_t)(Hq + g) * D;
            const double* vv = qkv + (size_t)b * N + (size_t)(Hq + Hkv + g) * D;
            if (w_kn) { oracle_rmsnorm(kk, w_kn, 1, D, eps, tmp); kk = tmp; }
            oracle_rope(kk, D, (double)pos, theta, rot);
            for (int d = 0; d < D; ++d) {
                k_cache[base + d] = f64_to_bf16(rot[d]);
                v_cache[base + d] = f64_to_bf16(vv[d]);
            }
        }
    }
    free(xn); free(qkv); free(tmp); free(rot);
}

/* ------------------------------------------------------------------------- */
/* One whole pre-norm decoder layer, decode step, in double:                  */
/*   A group:  q, cache append  (oracle_qkv_rope_append on x with w_ln_attn)   */
/*             a  = attention(q, cache)                                        */
/*             h1 = x + a W_o^T                  (what A sends to F)           */
/*   F group:  out = h1 + FFN(rmsnorm(h1, w_ln_ffn))  (what F returns)          */
/* FFN = dense SwiGLU (E == 0) or top-K mixture of experts with router         */
/* logits = rmsnorm(h1) W_r^T (or the given logits when w_router is NULL).     */
/* No intermediate is rounded except the cache entries (bf16 storage).         */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_decoder_layer(const double* x, const uint16_t* w_ln_attn, const uint16_t* w_qkv,
                                     const uint16_t* w_qn, const uint16_t* w_kn, double eps, double theta,
                                     uint16_t* k_cache, uint16_t* v_cache,
                                     const int32_t* page_table, int max_pages, const int32_t* seq_lens,
                                     int B, int H, int Hq, int Hkv, int D, int P, double scale,
                                     const uint16_t* w_o, const uint16_t* w_ln_ffn, int I, int E, int K,
                                     const uint16_t* w_gate, const uint16_t* w_up, const uint16_t* w_down,
                                     const uint16_t* w_router, const float* logits,
                                     double* q_out, double* h1_out, double* out) {
    const int A = Hq * D;
    double* q = q_out ? q_out : (double*)malloc(sizeof(double) * (size_t)B * A);
    double* a = (double*)malloc(sizeof(double) * (size_t)B * A);
    double* h1 = h1_out ? h1_out : (double*)malloc(sizeof(double) * (size_t)B * H);
    double* xn = (double*)malloc(sizeof(double) * (size_t)B * H);
    double* f = (double*)malloc(sizeof(double) * (size_t)B * H);
    oracle_qkv_rope_append(x, w_ln_attn, w_qkv, w_qn, w_kn, eps, theta, k_cache, v_cache, page_table, max_pages,
                           seq_lens, B, H, Hq, Hkv, D, P, q);
    oracle_attn_decode_f64q(q, k_cache, v_cache, page_table, max_pages, seq_lens, B, Hq, Hkv, D, P, scale, a, NULL);
    oracle_linear(a, w_o, B, A, H, h1);
    for (size_t i = 0; i < (size_t)B * H; ++i) h1[i] += x[i];
    oracle_rmsnorm(h1, w_ln_ffn, B, H, eps, xn);
    if (E == 0) {
        oracle_ffn_dense_f64x(xn, w_gate, w_up, w_down, B, H, I, f);
    } else if (w_router) {
        double* ld = (double*)malloc(sizeof(double) * (size_t)B * E);
        float* lf = (float*)malloc(sizeof(float) * (size_t)B * E);
        oracle_router_logits(xn, w_router, B, H, E, ld);
        for (size_t i = 0; i < (size_t)B * E; ++i) lf[i] = (float)ld[i];   /* routing takes fp32 logits */
        oracle_ffn_moe_f64x(xn, lf, w_gate, w_up, w_down, B, H, I, E, K, f, NULL, NULL);
        free(ld); free(lf);
    } else {
        oracle_ffn_moe_f64x(xn, logits, w_gate, w_up, w_down, B, H, I, E, K, f, NULL, NULL);
    }
    for (size_t i = 0; i < (size_t)B * H; ++i) out[i] = h1[i] + f[i];
    if (!q_out) free(q);
    if (!h1_out) free(h1);
    free(a); free(xn); free(f);
}

/* ------------------------------------------------------------------------- */
/* Prefill (causal) attention over the paged cache, the attention operator of  */
/* the prefill phase (the paper's PA pool).  Sequence b has n = seq_lens[b]     */
/* cached tokens of which the last m = q_offsets[b+1] - q_offsets[b] are the    */
/* ones being prefilled; query i (0 <= i < m) sits at position n - m + i and    */
/* attends to the cached tokens 0 .. n - m + i (itself included), nothing       */
/* later:                                                                       */
/*   s_j = scale * <q_i, k_j>, p = softmax over j <= pos_i, o_i = sum_j p_j v_j */
/*   q bf16 [T][Hq][D] (T = q_offsets[B], queries of sequence b at rows          */
/*   q_offsets[b] ..); caches, page table as for decode; out f64 [T][Hq][D].     */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_attn_prefill(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                                    const int32_t* page_table, int max_pages, const int32_t* seq_lens,
                                    const int32_t* q_offsets, int B, int Hq, int Hkv, int D, int P, double scale,
                                    double* out) {
    const int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const int n = seq_lens[b];
        const int m = q_offsets[b + 1] - q_offsets[b];
        double* keys = (double*)malloc(sizeof(double) * (size_t)n * D);
        double* vals = (double*)malloc(sizeof(double) * (size_t)n * D);
        double* qd = (double*)malloc(sizeof(double) * (size_t)D);
        for (int g = 0; g < Hkv; ++g) {
            for (int j = 0; j < n; ++j) {
                const int64_t page = page_table[(size_t)b * max_pages + j / P];
                const size_t base = (((size_t)page * Hkv + g) * P + (size_t)(j % P)) * (size_t)D;
                for (int d = 0; d < D; ++d) {
                    keys[(size_t)j * D + d] = bf16_to_f64(k_cache[base + d]);
                    vals[(size_t)j * D + d] = bf16_to_f64(v_cache[base + d]);
                }
            }
            for (int i = 0; i < m; ++i) {
                const int visible = n - m + i + 1;          /* keys 0 .. pos_i */
                const size_t row = (size_t)q_offsets[b] + i;
                for (int hh = 0; hh < G; ++hh) {
                    const int h = g * G + hh;
                    for (int d = 0; d < D; ++d) qd[d] = bf16_to_f64(q[(row * Hq + h) * D + d]);
                    oracle_attn_one_query_f64(qd, keys, vals, visible, D, scale, out + (row * Hq + h) * D, NULL);
                }
            }
        }
        free(keys); free(vals); free(qd);
    }
}

/* ------------------------------------------------------------------------- */
/* The same with the queries in double (the layer oracle does not round q).    */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_attn_prefill_f64q(const double* q, const uint16_t* k_cache, const uint16_t* v_cache,
                                         const int32_t* page_table, int max_pages, const int32_t* seq_lens,
                                         const int32_t* q_offsets, int B, int Hq, int Hkv, int D, int P, double scale,
                                         double* out) {
    const int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const int n = seq_lens[b];
        const int m = q_offsets[b + 1] - q_offsets[b];
        double* keys = (double*)malloc(sizeof(double) * (size_t)n * D);
        double* vals = (double*)malloc(sizeof(double) * (size_t)n * D);
        for (int g = 0; g < Hkv; ++g) {
            for (int j = 0; j < n; ++j) {
                const int64_t page = page_table[(size_t)b * max_pages + j / P];
                const size_t base = (((size_t)page * Hkv + g) * P + (size_t)(j % P)) * (size_t)D;
                for (int d = 0; d < D; ++d) {
                    keys[(size_t)j * D + d] = bf16_to_f64(k_cache[base + d]);
                    vals[(size_t)j * D + d] = bf16_to_f64(v_cache[base + d]);
                }
            }
            for (int i = 0; i < m; ++i) {
                const int visible = n - m + i + 1;          /* keys 0 .. pos_i */
                const size_t row = (size_t)q_offsets[b] + i;
                for (int hh = 0; hh < G; ++hh) {
                    const int h = g * G + hh;
                    oracle_attn_one_query_f64(q + (row * Hq + h) * D, keys, vals, visible, D, scale,
                                              out + (row * Hq + h) * D, NULL);
                }
            }
        }
        free(keys); free(vals);
    }
}

/* ------------------------------------------------------------------------- */
/* The Attention group's work before the attention operator for the tokens    */
/* being prefilled: row q_offsets[b] + i of x is token i of the last            */
/* m = q_offsets[b+1] - q_offsets[b] tokens of sequence b and sits at position  */
/* pos = seq_lens[b] - m + i.  Per row exactly what oracle_qkv_rope_append      */
/* does for its one token: rmsnorm, QKV projection, head norms, rotary          */
/* embedding at pos, K and V rounded to bf16 into the cache slot of pos.        */
/* q_out f64 [T][Hq][D].                                                        */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_qkv_rope_append_prefill(const double* x, const uint16_t* w_ln, const uint16_t* w_qkv,
                                               const uint16_t* w_qn, const uint16_t* w_kn, double eps, double theta,
                                               uint16_t* k_cache, uint16_t* v_cache,
                                               const int32_t* page_table, int max_pages, const int32_t* seq_lens,
                                               const int32_t* q_offsets, int B, int H, int Hq, int Hkv, int D, int P,
                                               double* q_out) {
    const int N = (Hq + 2 * Hkv) * D;
    const int T = q_offsets[B];
    double* xn = (double*)malloc(sizeof(double) * (size_t)T * H);
    double* qkv = (double*)malloc(sizeof(double) * (size_t)T * N);
    double* tmp = (double*)malloc(sizeof(double) * (size_t)D);
    double* rot = (double*)malloc(sizeof(double) * (size_t)D);
    oracle_rmsnorm(x, w_ln, T, H, eps, xn);
    oracle_linear(xn, w_qkv, T, H, N, qkv);
    for (int b = 0; b < B; ++b) {
        const int m = q_offsets[b + 1] - q_offsets[b];
        for (int i = 0; i < m; ++i) {
            const size_t r = (size_t)q_offsets[b] + i;
            const int pos = seq_lens[b] - m + i;
            const int64_t page = page_table[(size_t)b * max_pages + pos / P];
            for (int h = 0; h < Hq; ++h) {
                const double* v = qkv + r * N + (size_t)h * D;
                if (w_qn) { oracle_rmsnorm(v, w_qn, 1, D, eps, tmp); v = tmp; }
                oracle_rope(v, D, (double)pos, theta, q_out + (r * Hq + h) * D);
            }
            for (int g = 0; g < Hkv; ++g) {
                const size_t base = (((size_t)page * Hkv + g) * P + (size_t)(pos % P)) * (size_t)D;
                const double* kk = qkv + r * N + (size_t)(Hq + g) * D;
                const double* vv = qkv + r * N + (size_t)(Hq + Hkv + g) * D;
                if (w_kn) { oracle_rmsnorm(kk, w_kn, 1, D, eps, tmp); kk = tmp; }
                oracle_rope(kk, D, (double)pos, theta, rot);
                for (int d = 0; d < D; ++d) {
                    k_cache[base + d] = f64_to_bf16(rot[d]);
                    v_cache[base + d] = f64_to_bf16(vv[d]);
                }
            }
        }
    }
    free(xn); free(qkv); free(tmp); free(rot);
}

/* ------------------------------------------------------------------------- */
/* One whole pre-norm decoder layer over the tokens being prefilled (the       */
/* paper's PA and PF groups): the decode layer's arithmetic row by row, with    */
/* causal attention over the cache that now also holds the rows' own K / V.     */
/*   x, h1_out, out f64 [T][H], T = q_offsets[B]; logits f32 [T][E] when given. */
/* ------------------------------------------------------------------------- */
ORACLE_API void oracle_prefill_layer(const double* x, const uint16_t* w_ln_attn, const uint16_t* w_qkv,
                                     const uint16_t* w_qn, const uint16_t* w_kn, double eps, double theta,
                                     uint16_t* k_cache, uint16_t* v_cache,
                                     const int32_t* page_table, int max_pages, const int32_t* seq_lens,
                                     const int32_t* q_offsets, int B, int H, int Hq, int Hkv, int D, int P, double scale,
                                     const uint16_t* w_o, const uint16_t* w_ln_ffn, int I, int E, int K,
                                     const uint16_t* w_gate, const uint16_t* w_up, const uint16_t* w_down,
                                     const uint16_t* w_router, const float* logits,
                                     double* q_out, double* h1_out, double* out) {
    const int A = Hq * D;
    const int T = q_offsets[B];
    double* q = q_out ? q_out : (double*)malloc(sizeof(double) * (size_t)T * A);
    double* a = (double*)malloc(sizeof(double) * (size_t)T * A);
    double* h1 = h1_out ? h1_out : (double*)malloc(sizeof(double) * (size_t)T * H);
    double* xn = (double*)malloc(sizeof(double) * (size_t)T * H);
    double* f = (double*)malloc(sizeof(double) * (size_t)T * H);
    oracle_qkv_rope_append_prefill(x, w_ln_attn, w_qkv, w_qn, w_kn, eps, theta, k_cache, v_cache, page_table, max_pages,
                                   seq_lens, q_offsets, B, H, Hq, Hkv, D, P, q);
    oracle_attn_prefill_f64q(q, k_cache, v_cache, page_table, max_pages, seq_lens, q_offsets, B, Hq, Hkv, D, P, scale, a);
    oracle_linear(a, w_o, T, A, H, h1);
    for (size_t i = 0; i < (size_t)T * H; ++i) h1[i] += x[i];
    oracle_rmsnorm(h1, w_ln_ffn, T, H, eps, xn);
    if (E == 0) {
        oracle_ffn_dense_f64x(xn, w_gate, w_up, w_down, T, H, I, f);
    } else if (w_router) {
        double* ld = (double*)malloc(sizeof(double) * (size_t)T * E);
        float* lf = (float*)malloc(sizeof(float) * (size_t)T * E);
        oracle_router_logits(xn, w_router, T, H, E, ld);
        for (size_t i = 0; i < (size_t)T * E; ++i) lf[i] = (float)ld[i];   /* routing takes fp32 logits */
        oracle_ffn_moe_f64x(xn, lf, w_gate, w_up, w_down, T, H, I, E, K, f, NULL, NULL);
        free(ld); free(lf);
    } else {
        oracle_ffn_moe_f64x(xn, logits, w_gate, w_up, w_down, T, H, I, E, K, f, NULL, NULL);
    }
    for (size_t i = 0; i < (size_t)T * H; ++i) out[i] = h1[i] + f[i];
    if (!q_out) free(q);
    if (!h1_out) free(h1);
    free(a); free(xn); free(f);
}
