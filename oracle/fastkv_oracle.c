/*
 * FastKV token-saliency selection path -- CPU oracle (TEST INFRASTRUCTURE ONLY).
 *
 * A plain, slow, fp64 restatement of what the path computes, written from the
 * paper's definitions so that it can be checked against them by eye.  It is
 * used only by the tests, the smoke check and the bench's cpu_baseline leg;
 * the CUDA library never calls it and shares no code with it.
 *
 * Inputs are bf16 bit patterns (uint16); widening bf16 -> fp64 is exact, so
 * every result here is the exact-arithmetic definition up to fp64 rounding.
 *
 * Notation follows the paper: N_I = L prompt tokens, N_obs = w window tokens,
 * H query heads, Hkv key/value groups of G = H / Hkv heads, Att_l the causal
 * softmax attention matrix of one layer.
 *
 * Readings taken where the paper is silent or ambiguous (each listed in the
 * design notes of this repository):
 *   - the window is exactly the last w query positions t_j = L-w+j, j=0..w-1
 *     (Eq. 1 prints the bound of the sum as N_obs; the text says "window tokens");
 *   - window / group / head aggregation are sums, not means (ranking-neutral);
 *   - Pooling in Eq. 1 is a stride-1, same-length 1-D pool over offsets
 *     m in [-p/2, p/2]: AVG pads with zeros and divides by p; MAX ignores
 *     out-of-range offsets;
 *   - selection ranks by (score descending, index ascending); with
 *     force_window the last w positions are always kept and are not ranked
 *     (Section 4.2: window tokens are always in the propagated set).
 *
 * Parity pins (tests/test_oracle_*.py): full LxL causal attention through a
 * library softmax, the uniform-attention and single-planted-key closed forms,
 * row-sum / shift / permutation invariants, pooling identities, selection
 * against a brute-force ranking, gather against numpy indexing, decode and prefill attention
 * against a library softmax-attention and closed forms.  Nothing
 * numeric from the paper's own implementation exists to compare against, so
 * parity with that implementation is unpinned; parity with the definitions
 * above is pinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_POOL_AVG 0
#define ORACLE_POOL_MAX 1
#define ORACLE_GROUP_THEN_POOL 0
#define ORACLE_POOL_THEN_GROUP 1

static double bf16_to_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/*
 * Eq. 1, inner term: A[h, i] = sum_{j<w} Att_l[h, t_j, i] with t_j = L-w+j.
 *
 * Att_l[h, t, .] is the causal softmax row of query position t of head h:
 * logits scale * <Q[t,h,:], K[i, h/G, :]> for i <= t, nothing for i > t.
 *
 * q holds query rows for positions q_first_pos, q_first_pos+1, ...: pass the
 * full [L, H, d] tensor with q_first_pos = 0, or only the last w rows with
 * q_first_pos = L-w.  k is [L, Hkv, d].  Both are dense, row-major, bf16 bits.
 * A is [H, L] fp64.
 */
int oracle_window_attention(const uint16_t* q, int64_t q_first_pos, const uint16_t* k,
                            int64_t L, int H, int Hkv, int d, int w, double scale, double* A) {
    if (L < w || w < 1 || H % Hkv != 0 || q_first_pos > L - w) return 1;
    const int G = H / Hkv;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = 0; h < H; ++h) {
        const int g = h / G;
        double* s = (double*)malloc((size_t)L * sizeof(double));
        if (!s) { failed = 1; continue; }
        for (int64_t i = 0; i < L; ++i) A[(int64_t)h * L + i] = 0.0;
        for (int j = 0; j < w; ++j) {
            const int64_t t = L - w + j;                       /* query position */
            const uint16_t* qrow = q + ((t - q_first_pos) * H + h) * (int64_t)d;
            double smax = -INFINITY;
            for (int64_t i = 0; i <= t; ++i) {                 /* causal: keys 0..t */
                const uint16_t* krow = k + (i * Hkv + g) * (int64_t)d;
                double acc = 0.0;
                for (int c = 0; c < d; ++c) acc += bf16_to_f64(qrow[c]) * bf16_to_f64(krow[c]);
                s[i] = scale * acc;
                if (s[i] > smax) smax = s[i];
            }
            double denom = 0.0;
            for (int64_t i = 0; i <= t; ++i) denom += exp(s[i] - smax);
            for (int64_t i = 0; i <= t; ++i) A[(int64_t)h * L + i] += exp(s[i] - smax) / denom;
        }
        free(s);
    }
    return failed;
}

/*
 * Brute force used only to pin oracle_window_attention on small L: build the
 * whole causal attention matrix Att_l[h] (all L query rows) and read its last
 * w rows.  q must be the full [L, H, d] tensor.  att (optional) receives the
 * [H, L, L] matrix.
 */
int oracle_full_attention_window(const uint16_t* q, const uint16_t* k, int64_t L, int H, int Hkv,
                                 int d, int w, double scale, double* A, double* att) {
    if (L < w || H % Hkv != 0) return 1;
    const int G = H / Hkv;
    double* row = (double*)malloc((size_t)L * sizeof(double));
    if (!row) return 1;
    for (int h = 0; h < H; ++h) {
        const int g = h / G;
        for (int64_t i = 0; i < L; ++i) A[(int64_t)h * L + i] = 0.0;
        for (int64_t t = 0; t < L; ++t) {
            double smax = -INFINITY, denom = 0.0;
            for (int64_t i = 0; i < L; ++i) {
                double acc = 0.0;
                for (int c = 0; c < d; ++c)
                    acc += bf16_to_f64(q[(t * H + h) * (int64_t)d + c]) *
                           bf16_to_f64(k[(i * Hkv + g) * (int64_t)d + c]);
                row[i] = (i <= t) ? scale * acc : -INFINITY;
                if (row[i] > smax) smax = row[i];
            }
            for (int64_t i = 0; i < L; ++i) denom += exp(row[i] - smax);
            for (int64_t i = 0; i < L; ++i) {
                const double p = exp(row[i] - smax) / denom;
                if (att) att[((int64_t)h * L + t) * L + i] = p;
                if (t >= L - w) A[(int64_t)h * L + i] += p;
            }
        }
    }
    free(row);
    return 0;
}

/*
 * "Pooling" of Eq. 1 over the sequence axis, one row at a time:
 *   AVG: out[i] = (1/p) * sum_{m=-p/2}^{p/2} in[i+m], terms outside [0,L) are 0;
 *   MAX: out[i] = max over the in-range part of the same offsets.
 * in/out are [rows, L]; p is odd.
 */
int oracle_pool1d(const double* in, int64_t rows, int64_t L, int p, int mode, double* out) {
    if (p < 1 || (p & 1) == 0) return 1;
    const int r = p / 2;
    for (int64_t row = 0; row < rows; ++row) {
        const double* x = in + row * L;
        double* y = out + row * L;
        for (int64_t i = 0; i < L; ++i) {
            if (mode == ORACLE_POOL_AVG) {
                double acc = 0.0;
                for (int m = -r; m <= r; ++m)
                    if (i + m >= 0 && i + m < L) acc += x[i + m];
                y[i] = acc / (double)p;
            } else {
                double best = -INFINITY;
                for (int m = -r; m <= r; ++m)
                    if (i + m >= 0 && i + m < L && x[i + m] > best) best = x[i + m];
                y[i] = best;
            }
        }
    }
    return 0;
}

/*
 * Saliency scores of one layer for one sequence.
 *   GROUP_THEN_POOL: a[g] = sum_{h in g} A[h];  S_kv[g] = Pool(a[g])
 *   POOL_THEN_GROUP: S_h = Pool(A[h]) (Eq. 1);  S_kv[g] = sum_{h in g} S_h
 *                    (App. B.1: group-wise score from the head-wise ones)
 *   S_tsp = sum_g S_kv[g]   (Eq. 2, as a sum over all heads)
 * S_kv is [Hkv, L], S_tsp is [L] (may be NULL), A_out is [H, L] (may be NULL).
 */
int oracle_scores(const uint16_t* q, int64_t q_first_pos, const uint16_t* k, int64_t L, int H,
                  int Hkv, int d, int w, double scale, int pool_kernel, int pool_mode,
                  int agg_order, double* S_kv, double* S_tsp, double* A_out) {
    const int G = H / Hkv;
    double* A = (double*)malloc((size_t)H * L * sizeof(double));
    double* tmp = (double*)malloc((size_t)H * L * sizeof(double));
    if (!A || !tmp) { free(A); free(tmp); return 1; }
    int rc = oracle_window_attention(q, q_first_pos, k, L, H, Hkv, d, w, scale, A);
    if (rc == 0) {
        if (A_out) memcpy(A_out, A, (size_t)H * L * sizeof(double));
        if (agg_order == ORACLE_GROUP_THEN_POOL) {
            for (int g = 0; g < Hkv; ++g)
                for (int64_t i = 0; i < L; ++i) {
                    double acc = 0.0;
                    for (int h = g * G; h < (g + 1) * G; ++h) acc += A[(int64_t)h * L + i];
                    tmp[(int64_t)g * L + i] = acc;
                }
            rc = oracle_pool1d(tmp, Hkv, L, pool_kernel, pool_mode, S_kv);
        } else {
            rc = oracle_pool1d(A, H, L, pool_kernel, pool_mode, tmp);
            for (int g = 0; g < Hkv && rc == 0; ++g)
                for (int64_t i = 0; i < L; ++i) {
                    double acc = 0.0;
                    for (int h = g * G; h < (g + 1) * G; ++h) acc += tmp[(int64_t)h * L + i];
                    S_kv[(int64_t)g * L + i] = acc;
                }
        }
        if (rc == 0 && S_tsp)
            for (int64_t i = 0; i < L; ++i) {
                double acc = 0.0;
                for (int g = 0; g < Hkv; ++g) acc += S_kv[(int64_t)g * L + i];
                S_tsp[i] = acc;
            }
    }
    free(A);
    free(tmp);
    return rc;
}

typedef struct { double score; int64_t index; } ranked_t;

static int by_score_desc_then_index_asc(const void* pa, const void* pb) {
    const ranked_t* a = (const ranked_t*)pa;
    const ranked_t* b = (const ranked_t*)pb;
    if (a->score > b->score) return -1;
    if (a->score < b->score) return 1;
    return (a->index > b->index) - (a->index < b->index);
}

static int by_index_asc(const void* pa, const void* pb) {
    const int64_t a = *(const int64_t*)pa, b = *(const int64_t*)pb;
    return (a > b) - (a < b);
}

/*
 * Top-k token selection (KVCompress / HiddenCompress of App. B.1).
 *   force_window = 1: rank the prefix [0, L-w) only, keep its best k-w
 *     positions, always add the w window positions;  |idx| = k.
 *   force_window = 0: rank all of [0, L), keep the best k.
 * Ranking is a full sort by (score descending, index ascending).  idx comes
 * out ascending.  tau (optional) = score of the last ranked position kept
 * (+inf when none is ranked in).
 */
int oracle_select(const double* S, int64_t L, int64_t k, int w, int force_window,
                  int64_t* idx, double* tau) {
    const int64_t n_cand = force_window ? L - w : L;
    const int64_t k_sel = force_window ? k - w : k;
    if (n_cand < 0 || k_sel < 0 || k_sel > n_cand || k > L) return 1;
    ranked_t* r = (ranked_t*)malloc((size_t)(n_cand > 0 ? n_cand : 1) * sizeof(ranked_t));
    if (!r) return 1;
    for (int64_t i = 0; i < n_cand; ++i) { r[i].score = S[i]; r[i].index = i; }
    qsort(r, (size_t)n_cand, sizeof(ranked_t), by_score_desc_then_index_asc);
    int64_t n = 0;
    for (int64_t j = 0; j < k_sel; ++j) idx[n++] = r[j].index;
    if (tau) *tau = k_sel > 0 ? r[k_sel - 1].score : INFINITY;
    if (force_window)
        for (int64_t i = L - w; i < L; ++i) idx[n++] = i;
    qsort(idx, (size_t)n, sizeof(int64_t), by_index_asc);
    free(r);
    return 0;
}

/*
 * Compaction (Alg. 1, C <- update(K, V); reduced hidden states x): copy rows.
 * dst row j = src row idx[j]; rows are row_bytes long, src rows are
 * src_stride_bytes apart, dst rows are dense.
 */
int oracle_gather_rows(const uint8_t* src, int64_t src_stride_bytes, int64_t row_bytes,
                       const int64_t* idx, int64_t n, uint8_t* dst) {
    for (int64_t j = 0; j < n; ++j)
        memcpy(dst + j * row_bytes, src + idx[j] * src_stride_bytes, (size_t)row_bytes);
    return 0;
}

/*
 * Decoding over the compressed cache (the stage the retained KV of Alg. 1 exists for; Sec. 3, Sec. 5.3):
 * one new query token attends to the k retained entries of its KV group.
 *   out[h, :] = sum_j softmax_j(scale * <q[h], K[h/G, j]>) * V[h/G, j, :],   j = 0..k-1
 * q is [H, d], k_cache and v_cache are [Hkv, k, d] (bf16 bits, dense), out is [H, d] fp64, lse (optional)
 * is the natural-log sum of exponentials of each head's logits.
 */
int oracle_decode_attention(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache, int64_t k,
                            int H, int Hkv, int d, double scale, double* out, double* lse) {
    if (k < 1 || H % Hkv != 0) return 1;
    const int G = H / Hkv;
    double* s = (double*)malloc((size_t)k * sizeof(double));
    if (!s) return 1;
    for (int h = 0; h < H; ++h) {
        const int g = h / G;
        double smax = -INFINITY;
        for (int64_t j = 0; j < k; ++j) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c)
                acc += bf16_to_f64(q[(int64_t)h * d + c]) * bf16_to_f64(k_cache[((int64_t)g * k + j) * d + c]);
            s[j] = scale * acc;
            if (s[j] > smax) smax = s[j];
        }
        double denom = 0.0;
        for (int64_t j = 0; j < k; ++j) denom += exp(s[j] - smax);
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int64_t j = 0; j < k; ++j)
                acc += exp(s[j] - smax) / denom * bf16_to_f64(v_cache[((int64_t)g * k + j) * d + c]);
            out[(int64_t)h * d + c] = acc;
        }
        if (lse) lse[h] = smax + log(denom);
    }
    free(s);
    return 0;
}

/*
 * The layer's own attention (Alg. 1: X <- layer_l(X) produces Att_l; Sec. 4.2: the saliency scores are read
 * off that same matrix): the output of causal softmax attention for every query position,
 *   O[t, h, :] = sum_{i <= t} Att_l[h, t, i] * V[i, h/G, :],
 *   Att_l[h, t, i] = exp(s_i - max_i' s_i') / sum_i' exp(s_i' - max), s_i = scale * <Q[t,h,:], K[i,h/G,:]>, i <= t.
 * q is [L, H, d], k and v are [L, Hkv, d] (bf16 bits, dense); O is [L, H, d] fp64.
 */
int oracle_prefill_attention(const uint16_t* q, const uint16_t* k, const uint16_t* v, int64_t L, int H, int Hkv,
                             int d, double scale, double* O) {
    if (L < 1 || H % Hkv != 0) return 1;
    const int G = H / Hkv;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = 0; h < H; ++h) {
        const int g = h / G;
        double* s = (double*)malloc((size_t)L * sizeof(double));
        if (!s) { failed = 1; continue; }
        for (int64_t t = 0; t < L; ++t) {
            const uint16_t* qrow = q + (t * H + h) * (int64_t)d;
            double smax = -INFINITY;
            for (int64_t i = 0; i <= t; ++i) {                 /* causal: keys 0..t */
                const uint16_t* krow = k + (i * Hkv + g) * (int64_t)d;
                double acc = 0.0;
                for (int c = 0; c < d; ++c) acc += bf16_to_f64(qrow[c]) * bf16_to_f64(krow[c]);
                s[i] = scale * acc;
                if (s[i] > smax) smax = s[i];
            }
            double denom = 0.0;
            for (int64_t i = 0; i <= t; ++i) denom += exp(s[i] - smax);
            double* out = O + (t * H + h) * (int64_t)d;
            for (int c = 0; c < d; ++c) out[c] = 0.0;
            for (int64_t i = 0; i <= t; ++i) {
                const double p = exp(s[i] - smax) / denom;
                const uint16_t* vrow = v + (i * Hkv + g) * (int64_t)d;
                for (int c = 0; c < d; ++c) out[c] += p * bf16_to_f64(vrow[c]);
            }
        }
        free(s);
    }
    return failed;
}

int oracle_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
