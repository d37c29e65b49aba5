/*
 * G-KV oracle: a plain, slow, fp64 CPU statement of the decode-time KV-cache eviction step
 * and of the decode attention over the compressed cache.
 *
 * THIS IS TEST INFRASTRUCTURE. It exists to define what the CUDA library must compute and to be
 * timed as a reported CPU baseline. It shares no code with the CUDA path, the CUDA path never
 * calls it, and nothing in the product may import, link or execute it.
 *
 * Every function takes one step of the method, in the paper's order and notation:
 *   Section 3 ("Preliminary"): the unified eviction framework, Eq. 1 (window attention A),
 *       the max-reduce over the query heads of a KV head (A'), Eq. 2 (local score S);
 *   Section 5 ("Training-Free KV Cache Compression with Global Attention"): max-normalisation
 *       of S, the three global-score forms Eq. 3 (max), Eq. 4 (average), Eq. 5 (summation), the
 *       rule for rows without history, the first-step rule, and the recording of F for the
 *       next step;
 *   Appendix on combining the global score with other methods: the redundancy score (normalised
 *       keys, thresholded cosine similarity, column sums, softmax, max-normalisation) and
 *       F' = lambda F - (1 - lambda) R' (gkvo_redundancy, gkvo_combine; its threshold, recent-token
 *       count and epsilon are not in the paper and are parameters); the StreamingLLM baseline of Section 6.1 as a
 *       score-free selection (gkvo_streaming_select).
 * Inputs are the exact bits the GPU consumes: bf16 as uint16 (widened exactly to double) and
 * fp32 score state (widened exactly to double). All arithmetic is double. No blocking, fusion or
 * reordering beyond what the text states.
 *
 * Parity pins (tests/test_oracle_pins.py): every function below is pinned. The accuracy effect of
 * the method on a language model (pass@1 etc.) is "parity unpinned": it needs models and benchmark
 * items that are not available; only a qualitative planted-key survival test stands in for it.
 *
 * Notation: h_q query heads, h_kv KV heads, g = h_q / h_kv, head dimension d, cache length l,
 * window w, budget b, n_c = l - w candidates, n_h leading rows that carry history, C = row
 * capacity (stride) of one head's cache. Query head i reads KV head i / g.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { GKVO_MAX = 0, GKVO_MEAN = 1, GKVO_SUM = 2, GKVO_LOCAL = 3 };

/* bf16 -> double: a bf16 is the top 16 bits of an IEEE fp32; the widening is exact. */
static double bf16_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int gkvo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------------------------
 * Eq. 1: A[i,k,:] = softmax(Q[i,k,:] . K[j,:,:]^T / sqrt(d)) for window row k of query head i,
 * j = i / g.  Q is [h_q][w][d], oldest window row first; K is [h_kv][C][d] with l valid rows.
 * The softmax of window row k runs over the keys that token could see when it was decoded:
 * t <= l - w + k (row l-w+k is that token's own key). A is 0 on the other keys.
 * With causal = 0 the softmax runs over all l keys (used only by pins).
 * A is [h_q][w][l].
 * ------------------------------------------------------------------------------------------ */
void gkvo_window_attention(const uint16_t* Q, const uint16_t* K, int h_q, int h_kv, int w, int l,
                           int C, int d, int causal, double* A) {
    const int g = h_q / h_kv;
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    double* z = (double*)malloc(sizeof(double) * (size_t)l);
    for (int i = 0; i < h_q; ++i) {
        const int j = i / g;
        for (int k = 0; k < w; ++k) {
            const uint16_t* q = Q + ((size_t)i * w + k) * d;
            const int n_vis = causal ? (l - w + k + 1) : l; /* number of visible keys */
            double m = -INFINITY;
            for (int t = 0; t < n_vis; ++t) {
                const uint16_t* key = K + ((size_t)j * C + t) * d;
                double dot = 0.0;
                for (int c = 0; c < d; ++c) dot += bf16_to_double(q[c]) * bf16_to_double(key[c]);
                z[t] = dot * inv_sqrt_d;
                if (z[t] > m) m = z[t];
            }
            double Z = 0.0;
            for (int t = 0; t < n_vis; ++t) Z += exp(z[t] - m);
            double* a = A + ((size_t)i * w + k) * l;
            for (int t = 0; t < n_vis; ++t) a[t] = exp(z[t] - m) / Z;
            for (int t = n_vis; t < l; ++t) a[t] = 0.0;
        }
    }
    free(z);
}

/* Section 3: A'[j,k,t] = max over the query heads i of KV head j of A[i,k,t].  [h_kv][w][l]. */
void gkvo_group_max(const double* A, int h_q, int h_kv, int w, int l, double* Ap) {
    const int g = h_q / h_kv;
    for (int j = 0; j < h_kv; ++j)
        for (int k = 0; k < w; ++k)
            for (int t = 0; t < l; ++t) {
                double best = A[((size_t)(j * g) * w + k) * l + t];
                for (int i = j * g + 1; i < (j + 1) * g; ++i) {
                    const double a = A[((size_t)i * w + k) * l + t];
                    if (a > best) best = a;
                }
                Ap[((size_t)j * w + k) * l + t] = best;
            }
}

/* Eq. 2: S[j,t] = (1/w) sum_k A'[j,k,t].  [h_kv][l]. */
void gkvo_window_mean(const double* Ap, int h_kv, int w, int l, double* S) {
    for (int j = 0; j < h_kv; ++j)
        for (int t = 0; t < l; ++t) {
            double sum = 0.0;
            for (int k = 0; k < w; ++k) sum += Ap[((size_t)j * w + k) * l + t];
            S[(size_t)j * l + t] = sum / (double)w;
        }
}

/* Section 5: S_hat[j,t] = S[j,t] / max_{t' < n_c} S[j,t'].  The window rows are always kept and
 * never compete, so the maximum and the output cover the n_c = l - w candidates only.
 * S has row stride ldS; S_hat is [h_kv][n_c]. A zero maximum gives S_hat = 0. */
void gkvo_max_normalise(const double* S, int h_kv, int ldS, int n_c, double* Shat) {
    for (int j = 0; j < h_kv; ++j) {
        double M = 0.0;
        for (int t = 0; t < n_c; ++t)
            if (S[(size_t)j * ldS + t] > M) M = S[(size_t)j * ldS + t];
        for (int t = 0; t < n_c; ++t)
            Shat[(size_t)j * n_c + t] = (M > 0.0) ? S[(size_t)j * ldS + t] / M : 0.0;
    }
}

/* Eq. 3 / Eq. 4 / Eq. 5 for the rows t < n_h that carry history F_prev (fp32 state, row stride
 * C); F = S_hat for the rows n_h <= t < n_c, for the first compression (n_h = 0) and for the
 * local-score-only mode.  F is [h_kv][n_c]. */
void gkvo_global_merge(const double* Shat, const float* F_prev, int h_kv, int n_c, int n_h, int C,
                       double alpha, int mode, double* F) {
    for (int j = 0; j < h_kv; ++j)
        for (int t = 0; t < n_c; ++t) {
            const double s = Shat[(size_t)j * n_c + t];
            double f = s;
            if (t < n_h && mode != GKVO_LOCAL) {
                const double fp = (double)F_prev[(size_t)j * C + t];
                if (mode == GKVO_MAX) f = (alpha * fp > s) ? alpha * fp : s;
                else if (mode == GKVO_MEAN) f = alpha * fp + (1.0 - alpha) * s;
                else f = alpha * fp + s; /* GKVO_SUM */
            }
            F[(size_t)j * n_c + t] = f;
        }
}

/* Section 3 / Section 5: per KV head keep the b-w candidates with the largest F (equal scores:
 * the lower position wins), listed in ascending position, followed by the w window rows
 * n_c .. l-1.  kept is [h_kv][b].  Requires l > b (otherwise nothing is evicted). */
typedef struct { double f; int t; } gkvo_cand;
static int cand_cmp(const void* pa, const void* pb) {
    const gkvo_cand* a = (const gkvo_cand*)pa;
    const gkvo_cand* b = (const gkvo_cand*)pb;
    if (a->f > b->f) return -1;
    if (a->f < b->f) return 1;
    return (a->t > b->t) - (a->t < b->t);
}
static int int_cmp(const void* pa, const void* pb) {
    const int a = *(const int*)pa, b = *(const int*)pb;
    return (a > b) - (a < b);
}
void gkvo_select(const double* F, int h_kv, int n_c, int l, int b, int w, int32_t* kept) {
    const int n_keep = b - w;
    gkvo_cand* cand = (gkvo_cand*)malloc(sizeof(gkvo_cand) * (size_t)n_c);
    for (int j = 0; j < h_kv; ++j) {
        for (int t = 0; t < n_c; ++t) { cand[t].f = F[(size_t)j * n_c + t]; cand[t].t = t; }
        qsort(cand, (size_t)n_c, sizeof(gkvo_cand), cand_cmp); /* full sort: F desc, t asc */
        int32_t* out = kept + (size_t)j * b;
        for (int r = 0; r < n_keep; ++r) out[r] = cand[r].t;
        qsort(out, (size_t)n_keep, sizeof(int32_t), int_cmp);
        for (int r = 0; r < w; ++r) out[n_keep + r] = l - w + r;
    }
    free(cand);
}

/* Section 5 ("retained ... recorded for use in the next compression step"): gather rows by kept.
 * K, V [h_kv][C][d] bf16 bits and pos [h_kv][C] are compacted to rows 0..b-1 of the outputs
 * (same strides); F_state[j][r] = F[j][kept[r]] for r < b-w (fp32 row stride C; the window rows
 * carry no recorded score). Outputs are separate buffers; rows >= b are not written. */
void gkvo_compact(const uint16_t* K, const uint16_t* V, const int32_t* pos, const double* F,
                  const int32_t* kept, int h_kv, int C, int d, int n_c, int b, int w,
                  uint16_t* K_out, uint16_t* V_out, int32_t* pos_out, double* F_state) {
    for (int j = 0; j < h_kv; ++j)
        for (int r = 0; r < b; ++r) {
            const int src = kept[(size_t)j * b + r];
            memcpy(K_out + ((size_t)j * C + r) * d, K + ((size_t)j * C + src) * d, sizeof(uint16_t) * (size_t)d);
            memcpy(V_out + ((size_t)j * C + r) * d, V + ((size_t)j * C + src) * d, sizeof(uint16_t) * (size_t)d);
            if (pos) pos_out[(size_t)j * C + r] = pos[(size_t)j * C + src];
            if (r < b - w) F_state[(size_t)j * C + r] = F[(size_t)j * n_c + src];
        }
}

/* ------------------------------------------------------------------------------------------
 * One eviction step for one sequence of one layer, steps in the paper's order.
 *   S_in  : NULL -> the local score is computed from Q_win and K (Eq. 1, group max, Eq. 2);
 *           else [h_kv][C] fp32 accumulated window sums (sum over the w decode steps of the
 *           group max of that step's attention row); S = S_in / w. Both are the same quantity.
 * Outputs (any may be NULL): S [h_kv][l], Shat [h_kv][n_c], F [h_kv][n_c], kept [h_kv][b],
 * K_out/V_out/pos_out/F_state as in gkvo_compact.
 * Returns the new length (b), or l unchanged when l <= b (nothing evicted, nothing written).
 * ------------------------------------------------------------------------------------------ */
int gkvo_evict_step(const uint16_t* Q_win, const float* S_in, const uint16_t* K, const uint16_t* V,
                    const int32_t* pos, const float* F_prev, int h_q, int h_kv, int d, int C, int l,
                    int n_h, int b, int w, double alpha, int mode, double* S_out, double* Shat_out,
                    double* F_out, int32_t* kept_out, uint16_t* K_out, uint16_t* V_out,
                    int32_t* pos_out, double* F_state) {
    if (l <= b) return l;
    const int n_c = l - w;
    double* S = (double*)malloc(sizeof(double) * (size_t)h_kv * l);
    if (S_in == NULL) {
        double* A = (double*)malloc(sizeof(double) * (size_t)h_q * w * l);
        double* Ap = (double*)malloc(sizeof(double) * (size_t)h_kv * w * l);
        gkvo_window_attention(Q_win, K, h_q, h_kv, w, l, C, d, 1, A);
        gkvo_group_max(A, h_q, h_kv, w, l, Ap);
        gkvo_window_mean(Ap, h_kv, w, l, S);
        free(A); free(Ap);
    } else {
        for (int j = 0; j < h_kv; ++j)
            for (int t = 0; t < l; ++t) S[(size_t)j * l + t] = (double)S_in[(size_t)j * C + t] / (double)w;
    }
    double* Shat = (double*)malloc(sizeof(double) * (size_t)h_kv * n_c);
    double* F = (double*)malloc(sizeof(double) * (size_t)h_kv * n_c);
    int32_t* kept = (int32_t*)malloc(sizeof(int32_t) * (size_t)h_kv * b);
    gkvo_max_normalise(S, h_kv, l, n_c, Shat);
    gkvo_global_merge(Shat, F_prev, h_kv, n_c, n_h, C, alpha, mode, F);
    gkvo_select(F, h_kv, n_c, l, b, w, kept);
    if (K_out && V_out && F_state)
        gkvo_compact(K, V, pos, F, kept, h_kv, C, d, n_c, b, w, K_out, V_out, pos_out, F_state);
    if (S_out) memcpy(S_out, S, sizeof(double) * (size_t)h_kv * l);
    if (Shat_out) memcpy(Shat_out, Shat, sizeof(double) * (size_t)h_kv * n_c);
    if (F_out) memcpy(F_out, F, sizeof(double) * (size_t)h_kv * n_c);
    if (kept_out) memcpy(kept_out, kept, sizeof(int32_t) * (size_t)h_kv * b);
    free(S); free(Shat); free(F); free(kept);
    return b;
}

/* The same step for n_seq independent sequences (one layer each entry), run in parallel across
 * sequences only. Per-sequence strides are in elements. Only the kept lists and F_state are
 * returned; used for the timed CPU baseline and for batch parity. */
void gkvo_evict_batch(int n_seq, const uint16_t* Q_win, const float* S_in, const uint16_t* K,
                      const uint16_t* V, const float* F_prev, int h_q, int h_kv, int d, int C, int l,
                      int n_h, int b, int w, double alpha, int mode, int32_t* kept_out,
                      uint16_t* K_out, uint16_t* V_out, double* F_state) {
    const size_t kv_stride = (size_t)h_kv * C * d, f_stride = (size_t)h_kv * C;
    const size_t q_stride = (size_t)h_q * w * d;
#pragma omp parallel for schedule(dynamic, 1)
    for (int n = 0; n < n_seq; ++n) {
        gkvo_evict_step(Q_win ? Q_win + n * q_stride : NULL, S_in ? S_in + n * f_stride : NULL,
                        K + n * kv_stride, V + n * kv_stride, NULL, F_prev + n * f_stride, h_q, h_kv,
                        d, C, l, n_h, b, w, alpha, mode, NULL, NULL, NULL,
                        kept_out ? kept_out + (size_t)n * h_kv * b : NULL,
                        K_out ? K_out + n * kv_stride : NULL, V_out ? V_out + n * kv_stride : NULL,
                        NULL, F_state ? F_state + n * f_stride : NULL);
    }
}

/* ------------------------------------------------------------------------------------------
 * Decode attention for one sequence of one layer over a cache of n keys (the current token's key
 * and value already appended, n = len + 1): for query head i, p = softmax_t(q_i . K[j,t] / sqrt(d))
 * over t < n and out_i = sum_t p[t] V[j,t,:].  q [h_q][d], K,V [h_kv][C][d] bf16 bits.
 * out [h_q][d] double; p_out (may be NULL) [h_q][n] double.
 * If Sacc != NULL (fp64 [h_kv][C]): Sacc[j,t] += max over the heads of KV head j of p_i[t],
 * i.e. this token's row of the group max A' that Eq. 2 averages over the window.
 * ------------------------------------------------------------------------------------------ */
void gkvo_decode_attention(const uint16_t* q, const uint16_t* K, const uint16_t* V, int h_q, int h_kv,
                           int d, int C, int n, double* out, double* p_out, double* Sacc) {
    const int g = h_q / h_kv;
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    double* p = (double*)malloc(sizeof(double) * (size_t)h_q * n);
    for (int i = 0; i < h_q; ++i) {
        const int j = i / g;
        double* pi = p + (size_t)i * n;
        double m = -INFINITY;
        for (int t = 0; t < n; ++t) {
            const uint16_t* key = K + ((size_t)j * C + t) * d;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += bf16_to_double(q[(size_t)i * d + c]) * bf16_to_double(key[c]);
            pi[t] = dot * inv_sqrt_d;
            if (pi[t] > m) m = pi[t];
        }
        double Z = 0.0;
        for (int t = 0; t < n; ++t) Z += exp(pi[t] - m);
        for (int t = 0; t < n; ++t) pi[t] = exp(pi[t] - m) / Z;
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int t = 0; t < n; ++t) acc += pi[t] * bf16_to_double(V[((size_t)j * C + t) * d + c]);
            out[(size_t)i * d + c] = acc;
        }
    }
    if (Sacc)
        for (int j = 0; j < h_kv; ++j)
            for (int t = 0; t < n; ++t) {
                double best = p[(size_t)(j * g) * n + t];
                for (int i = j * g + 1; i < (j + 1) * g; ++i)
                    if (p[(size_t)i * n + t] > best) best = p[(size_t)i * n + t];
                Sacc[(size_t)j * C + t] += best;
            }
    if (p_out) memcpy(p_out, p, sizeof(double) * (size_t)h_q * n);
    free(p);
}

/* Decode attention for n_seq independent sequences in parallel across sequences (timed CPU
 * baseline and batch parity). q [n_seq][h_q][d], caches [n_seq][h_kv][C][d], out [n_seq][h_q][d]. */
void gkvo_decode_batch(int n_seq, const uint16_t* q, const uint16_t* K, const uint16_t* V, int h_q,
                       int h_kv, int d, int C, int n, double* out, double* Sacc) {
    const size_t kv_stride = (size_t)h_kv * C * d;
#pragma omp parallel for schedule(dynamic, 1)
    for (int s = 0; s < n_seq; ++s)
        gkvo_decode_attention(q + (size_t)s * h_q * d, K + s * kv_stride, V + s * kv_stride, h_q, h_kv, d,
                              C, n, out + (size_t)s * h_q * d, NULL,
                              Sacc ? Sacc + (size_t)s * h_kv * C : NULL);
}

/* ------------------------------------------------------------------------------------------
 * Appendix "combining the global score with other methods": the redundancy score (of R-KV, as the
 * paper restates it) and its combination with the global score.
 *
 *   Kbar[j,t,:] = K[j,t,:] / (||K[j,t,:]||_2 + eps)                 (normalised key states)
 *   Cm[j]       = Kbar[j] Kbar[j]^T                                  (cosine similarity, l x l)
 *   C'[j,k,t]   = 0 where Cm[j,k,t] < tau, and in the columns t of the `recent` most recent tokens
 *                 (t >= l - recent); Cm elsewhere                    (thresholded similarity)
 *   cbar[j,t]   = sum_k C'[j,k,t]                                    (redundancy level of token t)
 *   R[j,t]      = softmax_t(cbar[j,:])                               (redundancy score)
 *   Rn[j,t]     = R[j,t] / max_t R[j,t]                              (normalised, as the global score is)
 *   Fsel[j,t]   = lambda F[j,t] - (1 - lambda) Rn[j,t]               (the score the selection runs on)
 *
 * The paper gives no value for tau, for the number of recent tokens or for eps (it defers to the
 * R-KV paper): they are parameters here. Reading taken for "those corresponding to the most recent
 * tokens": the COLUMNS of the recent tokens are zeroed, so a recent token is never rated redundant,
 * while its row still counts as a witness of the redundancy of older tokens. The diagonal is not
 * special-cased (the text does not): every kept column carries its own ~1.
 * band (optional, [h_kv][l] int32) counts, per column, the entries whose similarity lies within
 * band_width of tau: a comparison in lower precision may flip exactly those.
 * ------------------------------------------------------------------------------------------ */
void gkvo_redundancy(const uint16_t* K, int h_kv, int C, int d, int l, double tau, int recent, double eps,
                     double* cbar, double* R, double* Rn, int32_t* band, double band_width) {
    double* Kbar = (double*)malloc(sizeof(double) * (size_t)l * d);
    for (int j = 0; j < h_kv; ++j) {
        for (int t = 0; t < l; ++t) {
            const uint16_t* row = K + ((size_t)j * C + t) * d;
            double ss = 0.0;
            for (int c = 0; c < d; ++c) { const double x = bf16_to_double(row[c]); ss += x * x; }
            const double inv = 1.0 / (sqrt(ss) + eps);
            for (int c = 0; c < d; ++c) Kbar[(size_t)t * d + c] = bf16_to_double(row[c]) * inv;
        }
        double* cb = cbar + (size_t)j * l;
        for (int t = 0; t < l; ++t) {
            double sum = 0.0;
            int near = 0;
            for (int k = 0; k < l; ++k) {
                double dot = 0.0;
                for (int c = 0; c < d; ++c) dot += Kbar[(size_t)k * d + c] * Kbar[(size_t)t * d + c];
                if (fabs(dot - tau) < band_width) ++near;
                const int masked = (dot < tau) || (t >= l - recent);
                sum += masked ? 0.0 : dot;
            }
            cb[t] = sum;
            if (band) band[(size_t)j * l + t] = near;
        }
        double m = cb[0];
        for (int t = 1; t < l; ++t) if (cb[t] > m) m = cb[t];
        double Z = 0.0;
        for (int t = 0; t < l; ++t) Z += exp(cb[t] - m);
        double rmax = 0.0;
        for (int t = 0; t < l; ++t) {
            R[(size_t)j * l + t] = exp(cb[t] - m) / Z;
            if (R[(size_t)j * l + t] > rmax) rmax = R[(size_t)j * l + t];
        }
        for (int t = 0; t < l; ++t) Rn[(size_t)j * l + t] = R[(size_t)j * l + t] / rmax;
    }
    free(Kbar);
}

/* Fsel = lambda F - (1 - lambda) Rn over the n_c candidates. F [h_kv][n_c], Rn [h_kv][l]. */
void gkvo_combine(const double* F, const double* Rn, int h_kv, int n_c, int l, double lambda, double* Fsel) {
    for (int j = 0; j < h_kv; ++j)
        for (int t = 0; t < n_c; ++t)
            Fsel[(size_t)j * n_c + t] = lambda * F[(size_t)j * n_c + t] - (1.0 - lambda) * Rn[(size_t)j * l + t];
}

/* The eviction step with the redundancy term: as gkvo_evict_step up to the global score F; the
 * top-(b-w) selection runs on Fsel; the score recorded for the next step is F itself (Section 5
 * records F_t; the redundancy term only steers the selection). Extra outputs (may be NULL):
 * cbar_out, Rn_out [h_kv][l], Fsel_out [h_kv][n_c], band_out [h_kv][l]. */
int gkvo_evict_step_redundancy(const uint16_t* Q_win, const float* S_in, const uint16_t* K, const uint16_t* V,
                               const int32_t* pos, const float* F_prev, int h_q, int h_kv, int d, int C, int l,
                               int n_h, int b, int w, double alpha, int mode, double lambda, double tau,
                               int recent, double eps, double band_width, double* F_out, double* cbar_out,
                               double* Rn_out, double* Fsel_out, int32_t* band_out, int32_t* kept_out,
                               uint16_t* K_out, uint16_t* V_out, int32_t* pos_out, double* F_state) {
    if (l <= b) return l;
    const int n_c = l - w;
    double* F = (double*)malloc(sizeof(double) * (size_t)h_kv * n_c);
    gkvo_evict_step(Q_win, S_in, K, V, pos, F_prev, h_q, h_kv, d, C, l, n_h, b, w, alpha, mode, NULL, NULL, F,
                    NULL, NULL, NULL, NULL, NULL);
    double* cbar = (double*)malloc(sizeof(double) * (size_t)h_kv * l);
    double* R = (double*)malloc(sizeof(double) * (size_t)h_kv * l);
    double* Rn = (double*)malloc(sizeof(double) * (size_t)h_kv * l);
    double* Fsel = (double*)malloc(sizeof(double) * (size_t)h_kv * n_c);
    int32_t* kept = (int32_t*)malloc(sizeof(int32_t) * (size_t)h_kv * b);
    gkvo_redundancy(K, h_kv, C, d, l, tau, recent, eps, cbar, R, Rn, band_out, band_width);
    gkvo_combine(F, Rn, h_kv, n_c, l, lambda, Fsel);
    gkvo_select(Fsel, h_kv, n_c, l, b, w, kept);
    if (K_out && V_out && F_state)
        gkvo_compact(K, V, pos, F, kept, h_kv, C, d, n_c, b, w, K_out, V_out, pos_out, F_state);
    if (F_out) memcpy(F_out, F, sizeof(double) * (size_t)h_kv * n_c);
    if (cbar_out) memcpy(cbar_out, cbar, sizeof(double) * (size_t)h_kv * l);
    if (Rn_out) memcpy(Rn_out, Rn, sizeof(double) * (size_t)h_kv * l);
    if (Fsel_out) memcpy(Fsel_out, Fsel, sizeof(double) * (size_t)h_kv * n_c);
    if (kept_out) memcpy(kept_out, kept, sizeof(int32_t) * (size_t)h_kv * b);
    free(F); free(cbar); free(R); free(Rn); free(Fsel); free(kept);
    return b;
}

/* StreamingLLM policy (the sink-plus-recent baseline the paper compares with: related work on decoding-time eviction,
 * baselines of the experimental setup, Section 6.1), as a degenerate selection on the same framework: no score; the
 * first n_sink rows of the cache (the attention sinks) and the most recent b - n_sink rows are kept, in ascending
 * position. kept [h_kv][b] (every head the same list). Requires l > b and 0 <= n_sink <= b. */
void gkvo_streaming_select(int h_kv, int l, int b, int n_sink, int32_t* kept) {
    for (int j = 0; j < h_kv; ++j) {
        int r = 0;
        for (int t = 0; t < l; ++t)
            if (t < n_sink || t >= l - (b - n_sink)) kept[(size_t)j * b + r++] = t;
    }
}

/* One compression step under that policy: the kept rows are gathered like in gkvo_evict_step; no score exists, so the
 * recorded score state of the kept rows is 0. Returns the new length (b), or l when l <= b (nothing evicted). */
int gkvo_evict_step_streaming(const uint16_t* K, const uint16_t* V, const int32_t* pos, int h_kv, int d, int C, int l,
                              int b, int w, int n_sink, int32_t* kept_out, uint16_t* K_out, uint16_t* V_out,
                              int32_t* pos_out, double* F_state) {
    if (l <= b) return l;
    const int n_c = l - w;
    int32_t* kept = (int32_t*)malloc(sizeof(int32_t) * (size_t)h_kv * b);
    double* F = (double*)calloc((size_t)h_kv * n_c, sizeof(double));
    gkvo_streaming_select(h_kv, l, b, n_sink, kept);
    if (K_out && V_out && F_state) gkvo_compact(K, V, pos, F, kept, h_kv, C, d, n_c, b, w, K_out, V_out, pos_out, F_state);
    if (kept_out) memcpy(kept_out, kept, sizeof(int32_t) * (size_t)h_kv * b);
    free(kept); free(F);
    return b;
}

/* Eviction log of one step: the tokens that are NOT in kept, in ascending cache position, reported by their
 * original position pos[j][t] (or by t itself when pos is NULL). kept [h_kv][b] as gkvo_select returns it,
 * out [h_kv][l - b]. This is the information the paper's sparse-training recipes record per compression
 * step to rebuild the attention mask of a compressed rollout. */
void gkvo_evicted(const int32_t* kept, const int32_t* pos, int h_kv, int C, int l, int b, int32_t* out) {
    unsigned char* in_kept = (unsigned char*)malloc((size_t)l);
    for (int j = 0; j < h_kv; ++j) {
        memset(in_kept, 0, (size_t)l);
        for (int r = 0; r < b; ++r) in_kept[kept[(size_t)j * b + r]] = 1;
        int e = 0;
        for (int t = 0; t < l; ++t)
            if (!in_kept[t]) out[(size_t)j * (l - b) + e++] = pos ? pos[(size_t)j * C + t] : t;
    }
    free(in_kept);
}

/* Appendix on combining the global score with other methods, SnapKV: a sequence-wise max-pooling of the
 * score before the selection ("it suffices to replace the local score utilized by SnapKV with the global
 * score"). out[j][t] = max of X[j][t'] over |t' - t| <= kernel / 2 within 0..n-1 (kernel odd; the window is
 * clipped at the ends, which equals padding with -inf). The paper does not give the kernel size: parameter. */
void gkvo_maxpool(const double* X, int h_kv, int n, int kernel, double* out) {
    const int half = kernel / 2;
    for (int j = 0; j < h_kv; ++j)
        for (int t = 0; t < n; ++t) {
            double m = -INFINITY;
            for (int u = t - half; u <= t + half; ++u)
                if (u >= 0 && u < n && X[(size_t)j * n + u] > m) m = X[(size_t)j * n + u];
            out[(size_t)j * n + t] = m;
        }
}

/* The eviction step with every optional term: F as in gkvo_evict_step; P = maxpool(F) when kernel > 1
 * (else F); Fsel = lambda P - (1 - lambda) Rn when use_redundancy (else P); top-(b-w) on Fsel; F itself is
 * what is recorded. Outputs may be NULL. */
int gkvo_evict_step_full(const uint16_t* Q_win, const float* S_in, const uint16_t* K, const uint16_t* V,
                         const int32_t* pos, const float* F_prev, int h_q, int h_kv, int d, int C, int l, int n_h,
                         int b, int w, double alpha, int mode, int pool_kernel, int use_redundancy, double lambda,
                         double tau, int recent, double eps, double* F_out, double* Fsel_out, int32_t* kept_out,
                         uint16_t* K_out, uint16_t* V_out, int32_t* pos_out, double* F_state) {
    if (l <= b) return l;
    const int n_c = l - w;
    double* F = (double*)malloc(sizeof(double) * (size_t)h_kv * n_c);
    double* P = (double*)malloc(sizeof(double) * (size_t)h_kv * n_c);
    double* Fsel = (double*)malloc(sizeof(double) * (size_t)h_kv * n_c);
    int32_t* kept = (int32_t*)malloc(sizeof(int32_t) * (size_t)h_kv * b);
    gkvo_evict_step(Q_win, S_in, K, V, pos, F_prev, h_q, h_kv, d, C, l, n_h, b, w, alpha, mode, NULL, NULL, F,
                    NULL, NULL, NULL, NULL, NULL);
    if (pool_kernel > 1) gkvo_maxpool(F, h_kv, n_c, pool_kernel, P);
    else memcpy(P, F, sizeof(double) * (size_t)h_kv * n_c);
    if (use_redundancy) {
        double* cbar = (double*)malloc(sizeof(double) * (size_t)h_kv * l);
        double* R = (double*)malloc(sizeof(double) * (size_t)h_kv * l);
        double* Rn = (double*)malloc(sizeof(double) * (size_t)h_kv * l);
        gkvo_redundancy(K, h_kv, C, d, l, tau, recent, eps, cbar, R, Rn, NULL, 0.0);
        gkvo_combine(P, Rn, h_kv, n_c, l, lambda, Fsel);
        free(cbar); free(R); free(Rn);
    } else {
        memcpy(Fsel, P, sizeof(double) * (size_t)h_kv * n_c);
    }
    gkvo_select(Fsel, h_kv, n_c, l, b, w, kept);
    if (K_out && V_out && F_state)
        gkvo_compact(K, V, pos, F, kept, h_kv, C, d, n_c, b, w, K_out, V_out, pos_out, F_state);
    if (F_out) memcpy(F_out, F, sizeof(double) * (size_t)h_kv * n_c);
    if (Fsel_out) memcpy(Fsel_out, Fsel, sizeof(double) * (size_t)h_kv * n_c);
    if (kept_out) memcpy(kept_out, kept, sizeof(int32_t) * (size_t)h_kv * b);
    free(F); free(P); free(Fsel); free(kept);
    return b;
}
