/*
 * TEST INFRASTRUCTURE -- not part of the product path.
 *
 * Plain fp64 CPU statement of Gram-threshold representative-token selection,
 * written from the paper's definitions.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it; the CUDA library never does, and
 * shares no code, header, table or helper with this file.
 *
 * Everything is the definition written out: rows are normalised, dot products
 * are plain k-loops, maxima are plain loops over the index sets the paper
 * names.  The only parallelism is an OpenMP "for" over independent output
 * rows; there is no blocking, no fusion, no reordering of the method's steps.
 *
 * Readings of the paper taken here (each is also a flag-free default of the
 * CUDA library):
 *   - Definition 1 is read literally: gamma_t is the maximum over ALL earlier
 *     tokens s < t (not only earlier representatives), with |.| applied.
 *   - strict "<" against 1 - tau^2; the maximum over an empty set is 0.
 *   - a zero-norm row normalises to the zero vector.
 *   - Algorithm 1 line 4: the maximum runs over all inherited representatives
 *     earlier in token order, valid or not (no update inside the loop).
 *   - Algorithm 1 line 8: the maximum runs over all valid representatives,
 *     earlier or later than t; `causal` != 0 restricts it to s < t (the
 *     variant for which Proposition 3's proof goes through).
 *   - tokens removed at line 5 are not re-examined as additions (line 6 uses
 *     the complement of the inherited set).
 *   - Eq. 2 (attention on the representative set) is taken as printed: every
 *     representative attends to every representative; `causal` != 0 restricts
 *     row i to the representatives at or before it in token order (what a
 *     causal language model's attention would keep).
 *
 * Pinned by tests/test_oracle_*.py (worked examples, closed forms, brute
 * force, invariants, an independent numpy statement, label-level prediction).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int ada_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void ada_oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Section 2.1: Xhat = D^-1 X, D = diag(||x_t||).  norm[t] = ||x_t||_2. */
void ada_oracle_normalize(const double* X, int64_t T, int64_t d,
                          double* Xhat, double* norm) {
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const double* x = X + t * d;
        double ss = 0.0;
        for (int64_t k = 0; k < d; ++k) ss += x[k] * x[k];
        double n = sqrt(ss);
        if (norm) norm[t] = n;
        double* y = Xhat + t * d;
        if (n > 0.0) {
            for (int64_t k = 0; k < d; ++k) y[k] = x[k] / n;
        } else {
            for (int64_t k = 0; k < d; ++k) y[k] = 0.0;
        }
    }
}

static double dot(const double* a, const double* b, int64_t d) {
    double s = 0.0;
    /* summation order is free at fp64 against the tolerances checked */
#pragma omp simd reduction(+ : s)
    for (int64_t k = 0; k < d; ++k) s += a[k] * b[k];
    return s;
}

/* Definition 1: gamma_t = max_{s<t} |G_st| for the listed rows only
 * (rows == NULL: all T rows).  Xhat is already normalised. */
static void gamma_lower(const double* Xhat, int64_t T, int64_t d,
                        const int32_t* rows, int64_t nrows, double* gamma) {
    int64_t n = rows ? nrows : T;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n; ++i) {
        int64_t t = rows ? rows[i] : i;
        const double* xt = Xhat + t * d;
        double g = 0.0;
        for (int64_t s = 0; s < t; ++s) {
            double c = fabs(dot(Xhat + s * d, xt, d));
            if (c > g) g = c;
        }
        gamma[i] = g;
    }
}

/* Definition 1 in full: gamma[T], rep[<=T] ascending, returns r. */
int64_t ada_oracle_full(const double* X, int64_t T, int64_t d, double tau,
                        double* gamma, int32_t* rep) {
    double* Xhat = (double*)malloc(sizeof(double) * (size_t)T * (size_t)d);
    if (!Xhat) return -1;
    ada_oracle_normalize(X, T, d, Xhat, NULL);
    gamma_lower(Xhat, T, d, NULL, T, gamma);
    const double thr = 1.0 - tau * tau;
    int64_t r = 0;
    for (int64_t t = 0; t < T; ++t)
        if (gamma[t] < thr) rep[r++] = (int32_t)t;
    free(Xhat);
    return r;
}

/* gamma_t of Definition 1 for a sample of rows (for checks at sizes where the
 * whole T x T triangle is too slow on a CPU). */
int ada_oracle_full_rows(const double* X, int64_t T, int64_t d,
                         const int32_t* rows, int64_t nrows, double* gamma) {
    double* Xhat = (double*)malloc(sizeof(double) * (size_t)T * (size_t)d);
    if (!Xhat) return -1;
    ada_oracle_normalize(X, T, d, Xhat, NULL);
    gamma_lower(Xhat, T, d, rows, nrows, gamma);
    free(Xhat);
    return 0;
}

/*
 * Algorithm 1 (Cascade Token Selection), lines 1-11.
 *
 *   rep_in[r]      inherited set R^(l), strictly ascending token indices
 *   causal         0: line 8 as printed; 1: restrict line 8 to s < t
 *   force_valid    NULL, or r flags that REPLACE line 5's decision (used by
 *                  tests to continue from a valid-set that differs only by
 *                  tokens inside the tolerance band)
 *   only_rows      NULL, or a list of non-representative tokens: lines 6-9 are
 *                  then evaluated for these tokens only (sampling at large T);
 *                  rep_out/add then cover only valid reps + sampled additions
 * outputs
 *   gamma_rep[r]   line 4, by position in rep_in
 *   gamma_cross[T] line 8, by token index; 0 for inherited reps / unsampled
 *   rep_out, add, rem  ascending; counts in n_out[0..2]
 */
int ada_oracle_cascade(const double* X, int64_t T, int64_t d, double tau,
                       const int32_t* rep_in, int64_t r, int causal,
                       const uint8_t* force_valid,
                       const int32_t* only_rows, int64_t n_only,
                       double* gamma_rep, double* gamma_cross,
                       int32_t* rep_out, int32_t* add, int32_t* rem,
                       int64_t* n_out) {
    const double thr = 1.0 - tau * tau;
    double* Xhat = (double*)malloc(sizeof(double) * (size_t)T * (size_t)d);
    uint8_t* is_rep = (uint8_t*)calloc((size_t)T, 1);
    uint8_t* valid = (uint8_t*)calloc((size_t)(r > 0 ? r : 1), 1);
    uint8_t* is_new = (uint8_t*)calloc((size_t)T, 1);
    uint8_t* is_valid_tok = (uint8_t*)calloc((size_t)T, 1);
    if (!Xhat || !is_rep || !valid || !is_new || !is_valid_tok) return -1;

    /* line 1 */
    ada_oracle_normalize(X, T, d, Xhat, NULL);
    /* line 2: the inherited rows are Xhat[rep_in[i]] */
    for (int64_t i = 0; i < r; ++i) is_rep[rep_in[i]] = 1;

    /* lines 3-4: r x r Gram among inherited reps, max over earlier ones */
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < r; ++i) {
        const double* xi = Xhat + (int64_t)rep_in[i] * d;
        double g = 0.0;
        for (int64_t j = 0; j < i; ++j) {
            double c = fabs(dot(Xhat + (int64_t)rep_in[j] * d, xi, d));
            if (c > g) g = c;
        }
        gamma_rep[i] = g;
    }
    /* line 5 */
    int64_t n_rem = 0;
    for (int64_t i = 0; i < r; ++i) {
        valid[i] = force_valid ? (force_valid[i] != 0) : (gamma_rep[i] < thr);
        if (valid[i]) is_valid_tok[rep_in[i]] = 1;
        else rem[n_rem++] = rep_in[i];
    }

    /* lines 6-8: cross-Gram of non-reps against valid reps, row max */
    for (int64_t t = 0; t < T; ++t) gamma_cross[t] = 0.0;
    int64_t n_rows = only_rows ? n_only : T;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t q = 0; q < n_rows; ++q) {
        int64_t t = only_rows ? only_rows[q] : q;
        if (is_rep[t]) continue;
        const double* xt = Xhat + t * d;
        double g = 0.0;
        for (int64_t i = 0; i < r; ++i) {
            if (!valid[i]) continue;
            int64_t s = rep_in[i];
            if (causal && s >= t) continue;
            double c = fabs(dot(Xhat + s * d, xt, d));
            if (c > g) g = c;
        }
        gamma_cross[t] = g;
        /* line 9 */
        is_new[t] = (g < thr);
    }

    /* lines 10-11: union, ascending */
    int64_t n_rep = 0, n_add = 0;
    for (int64_t t = 0; t < T; ++t) {
        if (is_new[t]) add[n_add++] = (int32_t)t;
        if (is_new[t] || is_valid_tok[t]) rep_out[n_rep++] = (int32_t)t;
    }
    n_out[0] = n_rep;
    n_out[1] = n_add;
    n_out[2] = n_rem;
    free(Xhat); free(is_rep); free(valid); free(is_new); free(is_valid_tok);
    return 0;
}

/* Section 2.3: the attention output of a redundant token is taken from its nearest
 * representative, s* = argmax_{s in R} |G_ts|.  For every token t: nearest[t] = s*
 * (lowest index on exact ties), gamma_near[t] = |G_{t s*}|; a representative is its own
 * nearest representative (gamma_near = |G_tt|: 1, or 0 for a zero row); an empty R gives -1. */
int ada_oracle_nearest(const double* X, int64_t T, int64_t d, const int32_t* rep, int64_t r,
                       int32_t* nearest, double* gamma_near) {
    double* Xhat = (double*)malloc(sizeof(double) * (size_t)T * (size_t)d);
    uint8_t* is_rep = (uint8_t*)calloc((size_t)T, 1);
    if (!Xhat || !is_rep) return -1;
    ada_oracle_normalize(X, T, d, Xhat, NULL);
    for (int64_t i = 0; i < r; ++i) is_rep[rep[i]] = 1;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t t = 0; t < T; ++t) {
        const double* xt = Xhat + t * d;
        if (is_rep[t]) {
            nearest[t] = (int32_t)t;
            gamma_near[t] = fabs(dot(xt, xt, d));
            continue;
        }
        int32_t best = -1;
        double g = -1.0;
        for (int64_t i = 0; i < r; ++i) {           /* ascending s: strict > keeps the lowest index */
            double c = fabs(dot(Xhat + (int64_t)rep[i] * d, xt, d));
            if (c > g) { g = c; best = rep[i]; }
        }
        nearest[t] = best;
        gamma_near[t] = best >= 0 ? g : 0.0;
    }
    free(Xhat); free(is_rep);
    return 0;
}

/* Eq. (4)/(5): Gram operation counts.  full: T^2 d.  cascade: r^2 d + (T-r) r d
 * with r the inherited count. */
uint64_t ada_oracle_op_count(int cascade, int64_t T, int64_t d, int64_t r) {
    uint64_t t = (uint64_t)T, dd = (uint64_t)d, rr = (uint64_t)r;
    if (!cascade) return t * t * dd;
    return rr * rr * dd + (t - rr) * rr * dd;
}

/* Eq. (1): |A n B| / |A u B| for ascending index lists; 1 when both are empty. */
double ada_oracle_jaccard(const int32_t* a, int64_t na, const int32_t* b, int64_t nb) {
    int64_t i = 0, j = 0, inter = 0;
    while (i < na && j < nb) {
        if (a[i] == b[j]) { ++inter; ++i; ++j; }
        else if (a[i] < b[j]) ++i;
        else ++j;
    }
    int64_t uni = na + nb - inter;
    return uni == 0 ? 1.0 : (double)inter / (double)uni;
}

/* Section 8.1 (adaptive threshold across depth): the paper proposes to set tau^(l+1) from the
 * turnover of layer l -- a stable set (low turnover) tolerates a tighter threshold (larger tau:
 * fewer representatives), an evolving one needs a looser threshold -- and gives no formula.
 * Reading taken: a clipped proportional step toward a target turnover,
 *     tau' = min(tau_max, max(tau_min, tau + gain * (target - rho))),
 * with tau' = clip(tau) when rho is undefined (empty inherited set).  Each operation is one
 * rounded fp64 operation, in this order. */
double ada_oracle_tau_update(double tau, double rho, double target, double gain, double tau_min,
                             double tau_max) {
    double t = tau;
    if (rho == rho) {
        const double diff = target - rho;
        const double step = gain * diff;
        t = tau + step;
    }
    if (t < tau_min) t = tau_min;
    if (t > tau_max) t = tau_max;
    return t;
}

/* Eq. (6): (|additions| + |removals|) / |R^(l)|; NaN when the set is empty. */
double ada_oracle_turnover(int64_t n_add, int64_t n_rem, int64_t r) {
    if (r == 0) return NAN;
    return (double)(n_add + n_rem) / (double)r;
}

/*
 * Attention on the representative set (Section 2.3, Eq. 2) for one sequence of T tokens
 * and h heads.  Q, K, V: [T][h][d_h].  For head j, with rho_0 < ... < rho_{r-1} the
 * representatives:
 *     S_ik   = q_{rho_i} . k_{rho_k} / sqrt(d_h)
 *     P_i.   = softmax over k of S_i.          (causal: only k <= i)
 *     A_i    = sum_k P_ik v_{rho_k}
 * out[rho_i][j][:] = A_i; and, when `nearest` is given, a token t outside the set takes
 * the output of its nearest representative: out[t][j][:] = out[nearest[t]][j][:]
 * (Section 2.3).  Rows that receive nothing are set to 0.  Returns 0.
 */
int ada_oracle_attention_reps(const double* Q, const double* K, const double* V, int64_t T,
                              int64_t h, int64_t d_h, const int32_t* rep, int64_t r,
                              const int32_t* nearest, int causal, double* out) {
    const int64_t row = h * d_h;
    memset(out, 0, (size_t)(T * row) * sizeof(double));
    const double scale = 1.0 / sqrt((double)d_h);
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t ij = 0; ij < r * h; ++ij) {
        const int64_t i = ij / h, j = ij % h;
        const double* q = Q + (int64_t)rep[i] * row + j * d_h;
        double* p = (double*)malloc((size_t)(r > 0 ? r : 1) * sizeof(double));
        const int64_t kmax = causal ? i + 1 : r;
        double m = -INFINITY;
        for (int64_t k = 0; k < kmax; ++k) {
            const double* kk = K + (int64_t)rep[k] * row + j * d_h;
            double s = 0.0;
            for (int64_t c = 0; c < d_h; ++c) s += q[c] * kk[c];
            p[k] = s * scale;
            if (p[k] > m) m = p[k];
        }
        double z = 0.0;
        for (int64_t k = 0; k < kmax; ++k) { p[k] = exp(p[k] - m); z += p[k]; }
        double* o = out + (int64_t)rep[i] * row + j * d_h;
        for (int64_t k = 0; k < kmax; ++k) {
            const double w = p[k] / z;
            const double* v = V + (int64_t)rep[k] * row + j * d_h;
            for (int64_t c = 0; c < d_h; ++c) o[c] += w * v[c];
        }
        free(p);
    }
    if (nearest != NULL) {
        /* representatives map to themselves; -1 (empty set) leaves the row at 0 */
#pragma omp parallel for schedule(static)
        for (int64_t t = 0; t < T; ++t) {
            const int32_t s = nearest[t];
            if (s >= 0 && s != t) memcpy(out + t * row, out + (int64_t)s * row, (size_t)row * sizeof(double));
        }
    }
    return 0;
}
