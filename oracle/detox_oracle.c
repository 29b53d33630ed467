/*
 * CPU oracle for the DETOX parameter-server aggregation path (arXiv 1907.12205).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the aggregation computes.
 * It is used by the tests, by the smoke check and by the benchmark's CPU-baseline leg.  It shares no
 * code with the CUDA library and the CUDA library never calls it.
 *
 * Conventions: every input row is fp32, read as given; every sum is carried in fp64 and rounded to
 * fp32 once at the end; all pointers are host pointers; `ld` is a row stride in elements.
 *
 * Pin status (tests/test_oracle_pins.py):
 *   vote, hier_mean, coord_median, sqdist : pinned (paper invariants, closed forms, brute force).
 *   krum scores / multikrum / bulyan      : the paper cites these aggregators (Section 4, "Improved
 *     speed"; Appendix B.1) without restating them; they are pinned to brute-force subset
 *     definitions on tiny inputs and to their f = 0 / beta = 1 / d = 1 reductions.  Beyond those
 *     cases: parity unpinned (this file is the definition).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Total order on fp32 bit patterns used wherever values are ranked:
 * -NaN < -Inf < ... < -0 < +0 < ... < +Inf < +NaN.  (A convention: the paper does not rank specials.) */
static uint32_t order_key(float v) {
    uint32_t u;
    memcpy(&u, &v, 4);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

static int cmp_u32(const void* a, const void* b) {
    uint32_t x = *(const uint32_t*)a, y = *(const uint32_t*)b;
    return (x > y) - (x < y);
}

static float key_to_float(uint32_t k) {
    uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    float v;
    memcpy(&v, &u, 4);
    return v;
}

/* ---------------------------------------------------------------------------------------------
 * Filtering step (Section 3; Algorithm 1, "Filtering step"): z_j = maj{ g_i : i in A_j }, and 0 when
 * no value is sent by more than half of the group.  Two members agree when all d words are bitwise
 * equal.  winner[j] is the lowest worker id of the winning class, or -1.
 * ------------------------------------------------------------------------------------------- */
int oracle_vote(const float* X, int64_t ld, int n, int r, int64_t d, const int32_t* members,
                float* Z, int64_t ldz, int32_t* winner) {
    if (r < 1 || n % r != 0) return 1;
    int G = n / r;
#pragma omp parallel for schedule(dynamic, 1)
    for (int j = 0; j < G; ++j) {
        const int32_t* A = members + (int64_t)j * r;
        int32_t win = -1;
        for (int a = 0; a < r && win < 0; ++a) {
            int votes = 0;
            int32_t lowest = A[a];
            for (int b = 0; b < r; ++b) {
                if (memcmp(X + (int64_t)A[a] * ld, X + (int64_t)A[b] * ld, (size_t)d * 4) == 0) {
                    ++votes;
                    if (A[b] < lowest) lowest = A[b];
                }
            }
            if (2 * votes > r) win = lowest;
        }
        winner[j] = win;
        if (Z) {
            if (win >= 0)
                memcpy(Z + (int64_t)j * ldz, X + (int64_t)win * ld, (size_t)d * 4);
            else
                memset(Z + (int64_t)j * ldz, 0, (size_t)d * 4);
        }
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * A_0 = mean of each vote group (Algorithm 2, step 3, with A_0 the mean as in Section 4):
 * M[s] = (1/|Z_s|) * sum_{j in Z_s} z_j.
 * ------------------------------------------------------------------------------------------- */
int oracle_hier_mean(const float* Z, int64_t ldz, int G, int64_t d, const int32_t* set_offsets,
                     const int32_t* set_members, int S, float* M, int64_t ldm) {
    (void)G;
    for (int s = 0; s < S; ++s) {
        int b = set_offsets[s], e = set_offsets[s + 1];
        if (e <= b) return 1;
#pragma omp parallel for schedule(static)
        for (int64_t c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int t = b; t < e; ++t) acc += (double)Z[(int64_t)set_members[t] * ldz + c];
            M[(int64_t)s * ldm + c] = (float)(acc / (double)(e - b));
        }
    }
    return 0;
}

/* Mean of the listed rows (the averaging step of Multi-Krum; also eq. (1)'s plain mean). */
int oracle_mean_rows(const float* X, int64_t ld, int64_t d, const int32_t* rows, int k, float* out) {
    if (k < 1) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t c = 0; c < d; ++c) {
        double acc = 0.0;
        for (int t = 0; t < k; ++t) acc += (double)X[(int64_t)rows[t] * ld + c];
        out[c] = (float)(acc / (double)k);
    }
    return 0;
}

/* Median of m ranked keys: the middle one; for an even count the fp32 average of the two middle values. */
static float median_of_sorted_keys(const uint32_t* k, int m) {
    if (m & 1) return key_to_float(k[m / 2]);
    float lo = key_to_float(k[m / 2 - 1]), hi = key_to_float(k[m / 2]);
    return (lo + hi) * 0.5f;
}

/* ---------------------------------------------------------------------------------------------
 * Coordinate-wise median (Section 4; Appendix B.1): out[c] = median_i X[rows[i], c].
 * rows == NULL means rows 0..m-1.
 * ------------------------------------------------------------------------------------------- */
int oracle_coord_median(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, float* out) {
    if (m < 1) return 1;
#pragma omp parallel
    {
        uint32_t* k = (uint32_t*)malloc((size_t)m * sizeof(uint32_t));
#pragma omp for schedule(static)
        for (int64_t c = 0; c < d; ++c) {
            for (int i = 0; i < m; ++i) k[i] = order_key(X[(int64_t)(rows ? rows[i] : i) * ld + c]);
            qsort(k, (size_t)m, sizeof(uint32_t), cmp_u32);
            out[c] = median_of_sorted_keys(k, m);
        }
        free(k);
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Pairwise squared Euclidean distances (the O(p^2 d) work of Section 4, "Improved speed"):
 * D[i][j] = sum_c (x_ic - x_jc)^2, computed once per unordered pair and mirrored; D[i][i] = 0.
 * ------------------------------------------------------------------------------------------- */
int oracle_sqdist(const float* X, int64_t ld, int m, int64_t d, double* D) {
    int64_t npairs = (int64_t)m * (m - 1) / 2;
    for (int i = 0; i < m; ++i) D[(int64_t)i * m + i] = 0.0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t p = 0; p < npairs; ++p) {
        /* unrank p -> (i, j), i < j */
        int i = 0;
        int64_t rem = p;
        while (rem >= m - 1 - i) { rem -= m - 1 - i; ++i; }
        int j = i + 1 + (int)rem;
        const float* a = X + (int64_t)i * ld;
        const float* b = X + (int64_t)j * ld;
        double acc = 0.0;
        for (int64_t c = 0; c < d; ++c) {
            double t = (double)a[c] - (double)b[c];
            acc += t * t;
        }
        D[(int64_t)i * m + j] = acc;
        D[(int64_t)j * m + i] = acc;
    }
    return 0;
}

static int cmp_f64(const void* a, const void* b) {
    double x = *(const double*)a, y = *(const double*)b;
    return (x > y) - (x < y);
}

/* Number of neighbours entering a Krum score among `alive` candidates with tolerance f:
 * alive - f - 2 as in Krum, but never fewer than one neighbour while another candidate exists. */
static int krum_neighbours(int alive, int f) {
    int nb = alive - f - 2;
    if (nb < 1) nb = 1;
    if (nb > alive - 1) nb = alive - 1;
    return nb;
}

/* ---------------------------------------------------------------------------------------------
 * Krum score: for every candidate i, the sum of its nb smallest squared distances to the other
 * candidates, added in ascending order.  Rows with alive[i] == 0 neither score nor count as
 * neighbours; their score is +infinity.  alive == NULL means all rows.
 * ------------------------------------------------------------------------------------------- */
int oracle_krum_scores(const double* D, int m, const uint8_t* alive, int f, double* score) {
    int cnt = 0;
    for (int i = 0; i < m; ++i) cnt += alive ? (alive[i] != 0) : 1;
    int nb = krum_neighbours(cnt, f);
    double* tmp = (double*)malloc((size_t)(m > 0 ? m : 1) * sizeof(double));
    for (int i = 0; i < m; ++i) {
        if (alive && !alive[i]) { score[i] = INFINITY; continue; }
        int k = 0;
        for (int j = 0; j < m; ++j)
            if (j != i && (!alive || alive[j])) tmp[k++] = D[(int64_t)i * m + j];
        qsort(tmp, (size_t)k, sizeof(double), cmp_f64);
        double s = 0.0;
        for (int t = 0; t < nb && t < k; ++t) s += tmp[t];
        score[i] = s;
    }
    free(tmp);
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Multi-Krum: score all m rows once, keep the m_sel rows of smallest score (equal scores: the lower
 * index first), report them in ascending index order and average them.
 * D_out (m*m) and scores (m) may be NULL.
 * ------------------------------------------------------------------------------------------- */
int oracle_multikrum(const float* X, int64_t ld, int m, int64_t d, int f, int m_sel, float* out,
                     int32_t* sel, double* scores, double* D_out) {
    if (m < 1 || m_sel < 1 || m_sel > m || f < 0) return 1;
    double* D = D_out ? D_out : (double*)malloc((size_t)m * m * sizeof(double));
    double* sc = scores ? scores : (double*)malloc((size_t)m * sizeof(double));
    oracle_sqdist(X, ld, m, d, D);
    oracle_krum_scores(D, m, NULL, f, sc);
    uint8_t* taken = (uint8_t*)calloc((size_t)m, 1);
    for (int t = 0; t < m_sel; ++t) {
        int best = -1;
        for (int i = 0; i < m; ++i)
            if (!taken[i] && (best < 0 || sc[i] < sc[best])) best = i;
        taken[best] = 1;
    }
    int32_t* rows = (int32_t*)malloc((size_t)m_sel * sizeof(int32_t));
    int k = 0;
    for (int i = 0; i < m; ++i)
        if (taken[i]) rows[k++] = i;
    if (sel) memcpy(sel, rows, (size_t)m_sel * sizeof(int32_t));
    if (out) oracle_mean_rows(X, ld, d, rows, m_sel, out);
    free(rows);
    free(taken);
    if (!scores) free(sc);
    if (!D_out) free(D);
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Bulyan, first stage: theta = m - 2f rounds of Krum on the shrinking candidate set.  Each round
 * scores the remaining candidates against each other (distances are never recomputed), moves the
 * one of smallest score (equal scores: the lower index) to the selection, and drops it.
 * sel receives the theta indices in the order they were chosen.
 * ------------------------------------------------------------------------------------------- */
int oracle_bulyan_select(const double* D, int m, int f, int32_t* sel) {
    int theta = m - 2 * f;
    if (theta < 1) return 1;
    uint8_t* alive = (uint8_t*)malloc((size_t)m);
    double* sc = (double*)malloc((size_t)m * sizeof(double));
    memset(alive, 1, (size_t)m);
    for (int t = 0; t < theta; ++t) {
        oracle_krum_scores(D, m, alive, f, sc);
        int best = -1;
        for (int i = 0; i < m; ++i)
            if (alive[i] && (best < 0 || sc[i] < sc[best])) best = i;
        sel[t] = best;
        alive[best] = 0;
    }
    free(sc);
    free(alive);
    return 0;
}

typedef struct { float dist; uint32_t key; } dist_key;

static int cmp_dist_key(const void* a, const void* b) {
    const dist_key* x = (const dist_key*)a;
    const dist_key* y = (const dist_key*)b;
    if (x->dist != y->dist) return (x->dist > y->dist) - (x->dist < y->dist);
    return (x->key > y->key) - (x->key < y->key);
}

/* ---------------------------------------------------------------------------------------------
 * Bulyan, second stage: per coordinate, take the median of the theta selected values and average
 * the beta values closest to it.  Closeness is |v - median| evaluated in fp32 (so that the choice is
 * the same decision on any fp32 machine); equally close values: the smaller value first.
 * ------------------------------------------------------------------------------------------- */
int oracle_trimmed_around_median(const float* X, int64_t ld, int64_t d, const int32_t* rows, int theta,
                                 int beta, float* out) {
    if (theta < 1 || beta < 1 || beta > theta) return 1;
#pragma omp parallel
    {
        uint32_t* k = (uint32_t*)malloc((size_t)theta * sizeof(uint32_t));
        dist_key* dk = (dist_key*)malloc((size_t)theta * sizeof(dist_key));
#pragma omp for schedule(static)
        for (int64_t c = 0; c < d; ++c) {
            for (int i = 0; i < theta; ++i) k[i] = order_key(X[(int64_t)(rows ? rows[i] : i) * ld + c]);
            qsort(k, (size_t)theta, sizeof(uint32_t), cmp_u32);
            float med = median_of_sorted_keys(k, theta);
            for (int i = 0; i < theta; ++i) {
                float v = key_to_float(k[i]);
                dk[i].dist = fabsf(v - med);
                dk[i].key = k[i];
            }
            qsort(dk, (size_t)theta, sizeof(dist_key), cmp_dist_key);
            double acc = 0.0;
            for (int i = 0; i < beta; ++i) acc += (double)key_to_float(dk[i].key);
            out[c] = (float)(acc / (double)beta);
        }
        free(dk);
        free(k);
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Coordinate-wise alpha-trimmed mean (Section 4, Theorem 4): drop the `trim` smallest and `trim`
 * largest of the m values of a coordinate, average the rest.
 * ------------------------------------------------------------------------------------------- */
int oracle_trimmed_mean(const float* X, int64_t ld, int m, int64_t d, int trim, float* out) {
    if (trim < 0 || m - 2 * trim < 1) return 1;
#pragma omp parallel
    {
        uint32_t* k = (uint32_t*)malloc((size_t)m * sizeof(uint32_t));
#pragma omp for schedule(static)
        for (int64_t c = 0; c < d; ++c) {
            for (int i = 0; i < m; ++i) k[i] = order_key(X[(int64_t)i * ld + c]);
            qsort(k, (size_t)m, sizeof(uint32_t), cmp_u32);
            double acc = 0.0;
            for (int i = trim; i < m - trim; ++i) acc += (double)key_to_float(k[i]);
            out[c] = (float)(acc / (double)(m - 2 * trim));
        }
        free(k);
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Geometric median by Weiszfeld's iteration (Section 4, Theorem 4 names the aggregator; the
 * iteration is the textbook one): y_0 = mean; y <- sum_j w_j x_j / sum_j w_j with
 * w_j = 1 / max(||x_j - y||, eps), `iters` times.  Everything in fp64; rounded to fp32 at the end.
 * ------------------------------------------------------------------------------------------- */
int oracle_geometric_median(const float* X, int64_t ld, int m, int64_t d, int iters, double eps, float* out) {
    if (m < 1 || iters < 0 || !(eps > 0.0)) return 1;
    double* y = (double*)malloc((size_t)d * sizeof(double));
    double* w = (double*)malloc((size_t)m * sizeof(double));
    for (int j = 0; j < m; ++j) w[j] = 1.0;
    for (int t = 0; t <= iters; ++t) {
        double tot = 0.0;
        for (int j = 0; j < m; ++j) tot += w[j];
#pragma omp parallel for schedule(static)
        for (int64_t c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int j = 0; j < m; ++j) acc += w[j] * (double)X[(int64_t)j * ld + c];
            y[c] = acc / tot;
        }
        if (t == iters) break;
        for (int j = 0; j < m; ++j) {
            double dist2 = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : dist2)
            for (int64_t c = 0; c < d; ++c) {
                const double diff = (double)X[(int64_t)j * ld + c] - y[c];
                dist2 += diff * diff;
            }
            const double dist = sqrt(dist2);
            w[j] = 1.0 / (dist > eps ? dist : eps);
        }
    }
    for (int64_t c = 0; c < d; ++c) out[c] = (float)y[c];
    free(w);
    free(y);
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Coordinate-wise sign majority (signSGD with majority vote; Section 5.2, setup 4):
 * out[c] = sign(sum_i sign(x_ic)); sign(0) = sign(NaN) = 0.  rows == NULL means rows 0..m-1.
 * ------------------------------------------------------------------------------------------- */
int oracle_sign_majority(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, float* out) {
    if (m < 1) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t c = 0; c < d; ++c) {
        long votes = 0;
        for (int i = 0; i < m; ++i) {
            const float v = X[(int64_t)(rows ? rows[i] : i) * ld + c];
            votes += (v > 0.0f) - (v < 0.0f);
        }
        out[c] = (float)((votes > 0) - (votes < 0));
    }
    return 0;
}

/* Bulyan = first stage on all m rows with tolerance f, then the second stage with beta = theta - 2f. */
int oracle_bulyan(const float* X, int64_t ld, int m, int64_t d, int f, float* out, int32_t* sel,
                  double* D_out) {
    int theta = m - 2 * f, beta = theta - 2 * f;
    if (f < 0 || beta < 1) return 1;
    double* D = D_out ? D_out : (double*)malloc((size_t)m * m * sizeof(double));
    int32_t* s = sel ? sel : (int32_t*)malloc((size_t)theta * sizeof(int32_t));
    oracle_sqdist(X, ld, m, d, D);
    oracle_bulyan_select(D, m, f, s);
    int rc = out ? oracle_trimmed_around_median(X, ld, d, s, theta, beta, out) : 0;
    if (!sel) free(s);
    if (!D_out) free(D);
    return rc;
}
