/*
 * CPU oracle for prob-sparse multi-head self-attention (forward).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, double-precision
 * statement of what the method computes.  It exists so that the CUDA library
 * can be checked against something written independently from the paper; it
 * shares no code, header, table or helper with the CUDA sources and the
 * library never calls it.
 *
 * Every function follows one passage of the paper (arXiv 2106.09236):
 *   Sec. 3.1  the projections Q = X W_q, K = X W_k, V = X W_v
 *   Eq. 6-8   dense scaled dot-product attention and its per-query form
 *   Eq. 9-10  the KL-motivated sparsity measure  M = LSE - mean
 *   Eq. 11    its sampled approximation          M~ = max - mean over K~
 *   Eq. 12    the piecewise output (attention for I_sparse, cheap value else)
 *   Sec. 3.2  the sample size  L~ = r_sample * ln L  and the top-L_sparse rule
 *   Sec. 2.2 / 3.1  the output matrix that merges the heads after the attention
 *
 * Readings taken where the paper is silent or garbled (kept in one place so a
 * reader can check them):
 *   - Eq. 7 prints the 1/sqrt(d) outside the exponent; Eq. 6 and Eq. 9-11 put
 *     it inside.  Scores are s_ij = q_i . k_j / sqrt(d) everywhere.
 *   - ln is the natural logarithm; counts are rounded up and clamped to
 *     [1, len]:  n(c, len) = min(len, max(1, ceil(c * ln len))).
 *   - K~ is drawn per query, with replacement, by the caller (sample_idx is an
 *     input); a key drawn twice counts twice in the mean of Eq. 11.
 *   - The number of selected queries is u = n(c, len) (the Informer rule the
 *     paper builds on) by default.  r_sparse > 0 selects the paper's own count,
 *     L_sparse = r_sparse * L of Sec. 3.2, per sequence from its own length:
 *     clamp(ceil(r_sparse * len), 1, len) (rounding up, at least one query).
 *     u_override > 0 fixes one count min(u_override, len) for all sequences.
 *   - Selection is per (batch, head); larger M~ first, equal M~ -> the smaller
 *     query index; the index set is reported in ascending order, padded by -1.
 *   - Non-selected valid queries receive mean(V) over valid keys (fill 0, the
 *     value a uniform-attention query would get, Sec. 3.1) or their own value
 *     row v_i (fill 1, Eq. 12 as printed).
 *   - Only a key-padding mask exists: keys and queries at positions >= len_b
 *     are ignored; output rows at those positions are zero.
 *   - M~ is evaluated as (1/U) * sum_j (max - s_j), which is Eq. 11 with the
 *     mean distributed over the max: every term is >= 0, so M~ >= 0 holds
 *     exactly and M~ == 0 exactly for a constant-score query.
 *
 * Layout: Q, K, V are float32 [B][H][T][d] (bf16 test data is widened exactly
 * to float32 by the harness), all arithmetic below is double.
 * sample_idx is int32 [B][T][idx_cols] (idx_per_head == 0, one sample shared by
 * the heads of a sequence) or [B][H][T][idx_cols] (idx_per_head != 0).
 * lengths is int32 [B] or NULL (every sequence has length T).
 *
 * Pins (tests/test_oracle_pins.py): brute force in numpy float64 on tiny
 * shapes, u = len  ==> dense attention, orthogonal-key closed form for M~,
 * max <= LSE <= max + ln U, permutation/shift invariances, planted spikes,
 * padding independence.  Unpinned by design: which of two queries is chosen
 * when their M~ differ by less than the comparison band.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Sec. 3.2: L~ = r_sample ln L (and the same rule for u); ceil, clamp. */
int psattn_oracle_count(double c, int len) {
    if (len <= 0) return 0;
    double x = ceil(c * log((double)len));
    if (x < 1.0) x = 1.0;
    if (x > (double)len) x = (double)len;
    return (int)x;
}

static int seq_len(const int *lengths, int b, int T) {
    int L = lengths ? lengths[b] : T;
    if (L < 0) L = 0;
    if (L > T) L = T;
    return L;
}

static const int *idx_row(const int *sample_idx, int idx_per_head, int H, int T,
                          int idx_cols, int b, int h, int i) {
    size_t r = idx_per_head ? (((size_t)b * H + h) * T + i) : ((size_t)b * T + i);
    return sample_idx + r * (size_t)idx_cols;
}

/* s_ij of Eq. 7 (exponent) / Eq. 11: q_i . k_j / sqrt(d). */
static double score(const float *q, const float *k, int d) {
    double acc = 0.0;
    for (int t = 0; t < d; ++t) acc += (double)q[t] * (double)k[t];
    return acc / sqrt((double)d);
}

/* Eq. 11: M~(q_i, K~) = max_j s_ij - (1/L~) sum_j s_ij over the sampled keys. */
void psattn_oracle_measure(const float *Q, const float *K, int B, int H, int T, int d,
                           const int *lengths, const int *sample_idx, int idx_cols,
                           int idx_per_head, double c, int U_override, double *M) {
    for (int b = 0; b < B; ++b) {
        int L = seq_len(lengths, b, T);
        int U = U_override > 0 ? (U_override < idx_cols ? U_override : idx_cols)
                               : psattn_oracle_count(c, L);
        for (int h = 0; h < H; ++h) {
            const float *Qu = Q + ((size_t)b * H + h) * T * d;
            const float *Ku = K + ((size_t)b * H + h) * T * d;
            double *Mu = M + ((size_t)b * H + h) * T;
            for (int i = 0; i < T; ++i) {
                if (i >= L) { Mu[i] = 0.0; continue; }
                const int *idx = idx_row(sample_idx, idx_per_head, H, T, idx_cols, b, h, i);
                double *s = (double *)malloc(sizeof(double) * (size_t)(U > 0 ? U : 1));
                double mx = -INFINITY;
                for (int j = 0; j < U; ++j) {
                    s[j] = score(Qu + (size_t)i * d, Ku + (size_t)idx[j] * d, d);
                    if (s[j] > mx) mx = s[j];
                }
                double acc = 0.0;
                for (int j = 0; j < U; ++j) acc += mx - s[j];
                Mu[i] = U > 0 ? acc / (double)U : 0.0;
                free(s);
            }
        }
    }
}

/* Eq. 10: M(q_i, K) = ln sum_j exp(s_ij) - (1/L) sum_j s_ij over all valid keys. */
void psattn_oracle_exact_measure(const float *Q, const float *K, int B, int H, int T, int d,
                                 const int *lengths, double *M) {
    for (int b = 0; b < B; ++b) {
        int L = seq_len(lengths, b, T);
        for (int h = 0; h < H; ++h) {
            const float *Qu = Q + ((size_t)b * H + h) * T * d;
            const float *Ku = K + ((size_t)b * H + h) * T * d;
            double *Mu = M + ((size_t)b * H + h) * T;
            for (int i = 0; i < T; ++i) {
                if (i >= L) { Mu[i] = 0.0; continue; }
                double mx = -INFINITY, sum = 0.0, se = 0.0;
                for (int j = 0; j < L; ++j) {
                    double s = score(Qu + (size_t)i * d, Ku + (size_t)j * d, d);
                    if (s > mx) mx = s;
                }
                for (int j = 0; j < L; ++j) {
                    double s = score(Qu + (size_t)i * d, Ku + (size_t)j * d, d);
                    se += exp(s - mx);
                    sum += s;
                }
                Mu[i] = (mx + log(se)) - sum / (double)L;
            }
        }
    }
}

/* Sec. 3.2: how many queries of a sequence of `len` valid positions are selected.
 * r_sparse > 0: L_sparse = r_sparse * L, rounded up, in [1, len]. */
int psattn_oracle_selected_count(double c, int u_override, double r_sparse, int len) {
    if (len <= 0) return 0;
    if (r_sparse > 0.0) {
        double x = ceil(r_sparse * (double)len);
        if (x < 1.0) x = 1.0;
        if (x > (double)len) x = (double)len;
        return (int)x;
    }
    if (u_override > 0) return u_override < len ? u_override : len;
    return psattn_oracle_count(c, len);
}

/* Sec. 3.2: I_sparse = indices of the top-u queries by M~, per (batch, head). */
void psattn_oracle_select(const double *M, int B, int H, int T, const int *lengths,
                          double c, int u_override, double r_sparse, int *sel_idx, int u_max) {
    for (int b = 0; b < B; ++b) {
        int L = seq_len(lengths, b, T);
        int u = psattn_oracle_selected_count(c, u_override, r_sparse, L);
        if (u > u_max) u = u_max;
        for (int h = 0; h < H; ++h) {
            const double *Mu = M + ((size_t)b * H + h) * T;
            int *out = sel_idx + ((size_t)b * H + h) * u_max;
            char *taken = (char *)calloc((size_t)(T > 0 ? T : 1), 1);
            for (int r = 0; r < u; ++r) {           /* u passes of "take the best left" */
                int best = -1;
                for (int i = 0; i < L; ++i) {
                    if (taken[i]) continue;
                    if (best < 0 || Mu[i] > Mu[best]) best = i;   /* strict > keeps the lower index */
                }
                taken[best] = 1;
            }
            int n = 0;
            for (int i = 0; i < L; ++i) if (taken[i]) out[n++] = i;
            for (; n < u_max; ++n) out[n] = -1;
            free(taken);
        }
    }
}

/* Sec. 3.1: a uniform-attention query receives the plain average of the values. */
void psattn_oracle_mean_v(const float *V, int B, int H, int T, int d, const int *lengths,
                          double *vbar) {
    for (int b = 0; b < B; ++b) {
        int L = seq_len(lengths, b, T);
        for (int h = 0; h < H; ++h) {
            const float *Vu = V + ((size_t)b * H + h) * T * d;
            double *out = vbar + ((size_t)b * H + h) * d;
            for (int t = 0; t < d; ++t) {
                double acc = 0.0;
                for (int j = 0; j < L; ++j) acc += (double)Vu[(size_t)j * d + t];
                out[t] = L > 0 ? acc / (double)L : 0.0;
            }
        }
    }
}

/* Eq. 7-8: SA(q_i, K, V) = sum_j p(k_j | q_i) v_j,  p = softmax_j(s_ij), j < len. */
void psattn_oracle_attend_row(const float *Q, const float *K, const float *V, int H, int T,
                              int d, int len, int b, int h, int i, double *out) {
    const float *Qu = Q + ((size_t)b * H + h) * T * d;
    const float *Ku = K + ((size_t)b * H + h) * T * d;
    const float *Vu = V + ((size_t)b * H + h) * T * d;
    double *p = (double *)malloc(sizeof(double) * (size_t)(len > 0 ? len : 1));
    double mx = -INFINITY, den = 0.0;
    for (int j = 0; j < len; ++j) {
        p[j] = score(Qu + (size_t)i * d, Ku + (size_t)j * d, d);
        if (p[j] > mx) mx = p[j];
    }
    for (int j = 0; j < len; ++j) { p[j] = exp(p[j] - mx); den += p[j]; }
    for (int t = 0; t < d; ++t) {
        double acc = 0.0;
        for (int j = 0; j < len; ++j) acc += (p[j] / den) * (double)Vu[(size_t)j * d + t];
        out[t] = acc;
    }
    free(p);
}

/*
 * The whole path for one batch: Eq. 11 -> top-u -> Eq. 12.
 *   O        double [B][H][T][d]
 *   M        double [B][H][T]            (may be NULL)
 *   sel_idx  int32  [B][H][u_max]        ascending, -1 padded
 *   sel_in   if non-NULL, a given index set (same layout) replaces the
 *            measure and the selection: the cross-layer reuse of Sec. 4.4.
 *   r_sparse > 0: the paper's count L_sparse = r_sparse * L per sequence (Sec. 3.2).
 *   fill     0: mean(V) over valid keys;  1: the query's own value row.
 *   nthreads OpenMP threads over (batch, head) units for the timed run; the
 *            arithmetic per unit is the same single-threaded code.
 */
void psattn_oracle_forward(const float *Q, const float *K, const float *V, int B, int H,
                           int T, int d, const int *lengths, const int *sample_idx,
                           int idx_cols, int idx_per_head, double c, int u_override,
                           double r_sparse, int U_override, int fill, const int *sel_in, double *O,
                           double *M, int *sel_idx, int u_max, int nthreads) {
    size_t units = (size_t)B * H;
    double *Mloc = M ? M : (double *)malloc(sizeof(double) * units * (size_t)T);
    if (!sel_in) {
        /* measure and selection, unit by unit so that threads can split them */
#ifdef _OPENMP
#pragma omp parallel for num_threads(nthreads > 0 ? nthreads : 1) schedule(dynamic, 1)
#endif
        for (long un = 0; un < (long)units; ++un) {
            int b = (int)(un / H), h = (int)(un % H);
            const int *len1 = lengths ? lengths + b : NULL;
            const int *idx1 = sample_idx + (idx_per_head ? (size_t)un * T * idx_cols
                                                         : (size_t)b * T * idx_cols);
            psattn_oracle_measure(Q + un * (size_t)T * d, K + un * (size_t)T * d, 1, 1, T, d,
                                  len1, idx1, idx_cols, 1, c, U_override,
                                  Mloc + un * (size_t)T);
            psattn_oracle_select(Mloc + un * (size_t)T, 1, 1, T, len1, c, u_override, r_sparse,
                                 sel_idx + un * (size_t)u_max, u_max);
        }
    } else {
        memcpy(sel_idx, sel_in, sizeof(int) * units * (size_t)u_max);
        if (M) memset(M, 0, sizeof(double) * units * (size_t)T);
    }
#ifdef _OPENMP
#pragma omp parallel for num_threads(nthreads > 0 ? nthreads : 1) schedule(dynamic, 1)
#endif
    for (long un = 0; un < (long)units; ++un) {
        int b = (int)(un / H), h = (int)(un % H);
        int L = seq_len(lengths, b, T);
        const int *sel = sel_idx + un * (size_t)u_max;
        double *Ou = O + un * (size_t)T * d;
        double vbar[4096];
        double *vb = d <= 4096 ? vbar : (double *)malloc(sizeof(double) * (size_t)d);
        const int *len1 = lengths ? lengths + b : NULL;
        psattn_oracle_mean_v(V + un * (size_t)T * d, 1, 1, T, d, len1, vb);
        for (int i = 0; i < T; ++i) {
            double *o = Ou + (size_t)i * d;
            if (i >= L) { for (int t = 0; t < d; ++t) o[t] = 0.0; continue; }
            int chosen = 0;
            for (int r = 0; r < u_max; ++r) if (sel[r] == i) chosen = 1;
            if (chosen) {
                psattn_oracle_attend_row(Q, K, V, H, T, d, L, b, h, i, o);      /* Eq. 12, top */
            } else if (fill == 1) {
                const float *vi = V + (un * (size_t)T + i) * d;                /* Eq. 12, else */
                for (int t = 0; t < d; ++t) o[t] = (double)vi[t];
            } else {
                for (int t = 0; t < d; ++t) o[t] = vb[t];
            }
        }
        if (vb != vbar) free(vb);
    }
    if (!M) free(Mloc);
}

/* Eq. 6: softmax(Q K^T / sqrt(d)) V for every valid query (the dense comparator). */
void psattn_oracle_dense(const float *Q, const float *K, const float *V, int B, int H, int T,
                         int d, const int *lengths, double *O, int nthreads) {
    size_t units = (size_t)B * H;
#ifdef _OPENMP
#pragma omp parallel for num_threads(nthreads > 0 ? nthreads : 1) schedule(dynamic, 1)
#endif
    for (long un = 0; un < (long)units; ++un) {
        int b = (int)(un / H), h = (int)(un % H);
        int L = seq_len(lengths, b, T);
        for (int i = 0; i < T; ++i) {
            double *o = O + (un * (size_t)T + i) * d;
            if (i < L) psattn_oracle_attend_row(Q, K, V, H, T, d, L, b, h, i, o);
            else for (int t = 0; t < d; ++t) o[t] = 0.0;
        }
    }
}

/*
 * Sec. 3.1: the projections that precede the attention, Q = X W_q, K = X W_k, V = X W_v,
 * one (d_x x d) matrix per head and per role.
 *   X   float  [B][T][d_x]
 *   Wt  float  [3][H*d][d_x]   role r (0 = q, 1 = k, 2 = v), row h*d + e holds column e of
 *                              head h's matrix: Wt[r][h*d + e][x] = W_r^h[x][e]
 *   out double [3][B][H][T][d] out[r][b][h][t][e] = sum_x X[b][t][x] * W_r^h[x][e]
 * Rows at positions >= len_b are zero (the attention never reads them).
 */
void psattn_oracle_project_qkv(const float *X, const float *Wt, int B, int T, int dx, int H,
                               int d, const int *lengths, double *out, int nthreads) {
    size_t plane = (size_t)B * H * T * d;
#ifdef _OPENMP
#pragma omp parallel for num_threads(nthreads > 0 ? nthreads : 1) schedule(static)
#endif
    for (long bt = 0; bt < (long)B * T; ++bt) {
        int b = (int)(bt / T), t = (int)(bt % T);
        int L = seq_len(lengths, b, T);
        const float *x = X + (size_t)bt * dx;
        for (int r = 0; r < 3; ++r)
            for (int h = 0; h < H; ++h)
                for (int e = 0; e < d; ++e) {
                    const float *w = Wt + ((size_t)r * H * d + (size_t)h * d + e) * dx;
                    double acc = 0.0;
                    if (t < L)
                        for (int k = 0; k < dx; ++k) acc += (double)x[k] * (double)w[k];
                    out[r * plane + (((size_t)b * H + h) * T + t) * d + e] = acc;
                }
    }
}

/*
 * The output side of the attention module (Sec. 2.2, Eq. 5 places MHSA inside the Conformer block;
 * Sec. 3.1 defines its heads): the heads' outputs are concatenated and multiplied by one output matrix,
 *   Y[b][t][n] = sum_h sum_e O[b][h][t][e] * W_o[h*d + e][n],
 * i.e. head h contributes O[b][h][t][:] times its own (d x d_y) block of W_o.
 *   O    float  [B][H][T][d]    the attention output (Eq. 12)
 *   Wot  float  [d_y][H*d]      W_o stored transposed: Wot[n][h*d + e] = W_o[h*d + e][n]
 *   Y    double [B][T][d_y]     rows at positions >= len_b are zero
 */
void psattn_oracle_project_out(const float *O, const float *Wot, int B, int H, int T, int d, int dy,
                               const int *lengths, double *Y, int nthreads) {
#ifdef _OPENMP
#pragma omp parallel for num_threads(nthreads > 0 ? nthreads : 1) schedule(static)
#endif
    for (long bt = 0; bt < (long)B * T; ++bt) {
        int b = (int)(bt / T), t = (int)(bt % T);
        int L = seq_len(lengths, b, T);
        for (int n = 0; n < dy; ++n) {
            double acc = 0.0;
            if (t < L)
                for (int h = 0; h < H; ++h) {
                    const float *o = O + (((size_t)b * H + h) * T + t) * d;
                    const float *w = Wot + (size_t)n * H * d + (size_t)h * d;
                    for (int e = 0; e < d; ++e) acc += (double)o[e] * (double)w[e];
                }
            Y[(size_t)bt * dy + n] = acc;
        }
    }
}

int psattn_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
