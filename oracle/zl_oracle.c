/*
 * CPU oracle for the ZipLine barrier-selection search (test infrastructure).
 *
 * Plain, slow, single-threaded C.  It exists to check the CUDA library and to
 * be timed as a CPU baseline; the product never calls it and it shares no
 * code with the CUDA path.
 *
 * Problem (paper, Section III "The Problem"): n workers, worker p has R
 * predicted iteration end timestamps e^p_1 <= ... <= e^p_R (row p of the
 * n x R matrix M of Section IV).  Pick one element per row to form Z;
 * d_Z = max(Z) - min(Z); Z* = argmin d_Z.  The barrier is max(Z*).
 *
 * Objectives
 *   ZLO_RANGE  d_Z = max(Z) - min(Z)             (the paper's objective function)
 *   ZLO_SUM    d_Z = sum_p (max(Z) - z_p)        (total wait of all workers)
 *
 * Result convention, shared by every function below so that they can be
 * compared bit for bit:
 *   wait    = min over all R^n choices of d_Z
 *   barrier = the smallest max(Z) among the minimisers (of equal minima the
 *             first one found wins: Fig. 3's caption; strict '<' in Algorithm 2)
 *   idx[p]  = the largest 0-based index i with M[p][i] <= barrier
 *             (a worker that finishes exactly at the barrier does not wait;
 *             this is the lexicographically largest minimiser with that barrier)
 *
 * Functions
 *   zlo_enumerate     all R^n combinations (Section IV "Naive search")
 *   zlo_sweep         sort Omega, one left-to-right pass keeping the latest
 *                     element of every worker, O(n) evaluation at every
 *                     position with all workers present (Section IV "ZipLine")
 *   zlo_sweep_window  the same pass with the minimum of Z kept by a two-pointer
 *                     window / the sum of Z kept incrementally; for sizes where
 *                     the O(n) evaluation is too slow
 *   zlo_alg2          Algorithm 2 step by step (drop min(Z), refill until |Z|=n)
 *   zlo_trace         per-position intermediates of the pass, for kernel tests
 *   zlo_gridscan      Algorithm 1 (GridScan) and its rotation over all rows (FullGridScan): the paper's baselines
 *   zlo_predict       phase 1 of ZipLine: R future end timestamps per worker from its most recent interval
 *
 * Return codes: 0 ok, -1 bad argument, -2 a row is not non-decreasing,
 * -3 the objective does not fit int64, -4 out of memory.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ZLO_RANGE = 0, ZLO_SUM = 1 };

typedef struct { int64_t t; int32_t p, i; } zlo_elem;
typedef __int128 i128;

static int check_rows(const int64_t *M, int n, int R) {
    for (int p = 0; p < n; ++p)
        for (int i = 1; i < R; ++i)
            if (M[(size_t)p * R + i] < M[(size_t)p * R + i - 1]) return -2;
    return 0;
}

static int cmp_elem(const void *a, const void *b) {
    const zlo_elem *x = (const zlo_elem *)a, *y = (const zlo_elem *)b;
    if (x->t != y->t) return x->t < y->t ? -1 : 1;
    if (x->p != y->p) return x->p < y->p ? -1 : 1;
    return (x->i > y->i) - (x->i < y->i);
}

/* Omega: all n*R elements, ascending by (timestamp, worker, iteration). */
static zlo_elem *build_omega(const int64_t *M, int n, int R) {
    size_t N = (size_t)n * R;
    zlo_elem *om = (zlo_elem *)malloc(N * sizeof(zlo_elem));
    if (!om) return NULL;
    for (int p = 0; p < n; ++p)
        for (int i = 0; i < R; ++i) {
            zlo_elem e = { M[(size_t)p * R + i], p, i };
            om[(size_t)p * R + i] = e;
        }
    qsort(om, N, sizeof(zlo_elem), cmp_elem);
    return om;
}

/* idx[p] = (number of elements of row p that are <= barrier) - 1 */
static void recover_idx(const int64_t *M, int n, int R, int64_t barrier, int32_t *idx) {
    for (int p = 0; p < n; ++p) {
        int c = 0;
        while (c < R && M[(size_t)p * R + c] <= barrier) ++c;
        idx[p] = c - 1;
    }
}

/* ---------------------------------------------------------------- naive search */
int zlo_enumerate(const int64_t *M, int n, int R, int objective,
                  int64_t *wait, int64_t *barrier, int32_t *idx) {
    if (!M || n < 1 || R < 1 || !wait || !barrier || !idx) return -1;
    if (objective != ZLO_RANGE && objective != ZLO_SUM) return -1;
    int rc = check_rows(M, n, R);
    if (rc) return rc;
    int32_t *j = (int32_t *)calloc((size_t)n, sizeof(int32_t));
    if (!j) return -4;
    int have = 0;
    i128 best_d = 0;
    int64_t best_max = 0;
    for (;;) {
        int64_t mx = M[j[0]], mn = M[j[0]];
        for (int p = 1; p < n; ++p) {
            int64_t v = M[(size_t)p * R + j[p]];
            if (v > mx) mx = v;
            if (v < mn) mn = v;
        }
        i128 d;
        if (objective == ZLO_RANGE) d = (i128)mx - mn;
        else { d = 0; for (int p = 0; p < n; ++p) d += (i128)mx - M[(size_t)p * R + j[p]]; }
        int better = 0;
        if (!have) better = 1;
        else if (d != best_d) better = d < best_d;
        else if (mx != best_max) better = mx < best_max;
        else {                                   /* same d, same barrier: larger indices win */
            for (int p = 0; p < n; ++p)
                if (j[p] != idx[p]) { better = j[p] > idx[p]; break; }
        }
        if (better) { have = 1; best_d = d; best_max = mx; memcpy(idx, j, (size_t)n * sizeof(int32_t)); }
        int p = n - 1;                           /* odometer */
        while (p >= 0 && ++j[p] == R) j[p--] = 0;
        if (p < 0) break;
    }
    free(j);
    if (best_d > (i128)INT64_MAX) return -3;
    *wait = (int64_t)best_d;
    *barrier = best_max;
    return 0;
}

/* ------------------------------------------------- one pass over sorted Omega */
int zlo_sweep(const int64_t *M, int n, int R, int objective,
              int64_t *wait, int64_t *barrier, int32_t *idx) {
    if (!M || n < 1 || R < 1 || !wait || !barrier || !idx) return -1;
    if (objective != ZLO_RANGE && objective != ZLO_SUM) return -1;
    int rc = check_rows(M, n, R);
    if (rc) return rc;
    size_t N = (size_t)n * R;
    zlo_elem *om = build_omega(M, n, R);
    int64_t *last = (int64_t *)malloc((size_t)n * sizeof(int64_t));
    char *seen = (char *)calloc((size_t)n, 1);
    if (!om || !last || !seen) { free(om); free(last); free(seen); return -4; }
    int cnt = 0, have = 0;
    i128 best = 0;
    int64_t best_t = 0;
    for (size_t k = 0; k < N; ++k) {
        int p = om[k].p;
        if (!seen[p]) { seen[p] = 1; ++cnt; }
        last[p] = om[k].t;                       /* the worker's older element leaves Z */
        if (cnt < n) continue;
        int64_t t = om[k].t;                     /* newest element = max(Z) */
        i128 d;
        if (objective == ZLO_RANGE) {
            int64_t mn = last[0];
            for (int q = 1; q < n; ++q) if (last[q] < mn) mn = last[q];
            d = (i128)t - mn;
        } else {
            d = 0;
            for (int q = 0; q < n; ++q) d += (i128)t - last[q];
        }
        if (!have || d < best) { have = 1; best = d; best_t = t; }
    }
    free(om); free(last); free(seen);
    if (best > (i128)INT64_MAX) return -3;
    *wait = (int64_t)best;
    *barrier = best_t;
    recover_idx(M, n, R, best_t, idx);
    return 0;
}

/* Same pass; min(Z) is the left end of the shortest suffix window of the
 * positions seen so far that still holds every worker, sum(Z) is updated by
 * the difference between a worker's new and old element. */
int zlo_sweep_window(const int64_t *M, int n, int R, int objective,
                     int64_t *wait, int64_t *barrier, int32_t *idx) {
    if (!M || n < 1 || R < 1 || !wait || !barrier || !idx) return -1;
    if (objective != ZLO_RANGE && objective != ZLO_SUM) return -1;
    int rc = check_rows(M, n, R);
    if (rc) return rc;
    size_t N = (size_t)n * R;
    zlo_elem *om = build_omega(M, n, R);
    int64_t *last = (int64_t *)malloc((size_t)n * sizeof(int64_t));
    int32_t *inwin = (int32_t *)calloc((size_t)n, sizeof(int32_t));
    if (!om || !last || !inwin) { free(om); free(last); free(inwin); return -4; }
    int cnt = 0, have = 0;
    size_t left = 0;
    i128 best = 0, sum = 0;
    int64_t best_t = 0;
    for (size_t k = 0; k < N; ++k) {
        int p = om[k].p;
        if (inwin[p] == 0) { ++cnt; sum += om[k].t; }
        else sum += (i128)om[k].t - last[p];
        last[p] = om[k].t;
        ++inwin[p];
        while (inwin[om[left].p] > 1) { --inwin[om[left].p]; ++left; }
        if (cnt < n) continue;
        int64_t t = om[k].t;
        i128 d = (objective == ZLO_RANGE) ? (i128)t - om[left].t : (i128)n * t - sum;
        if (!have || d < best) { have = 1; best = d; best_t = t; }
    }
    free(om); free(last); free(inwin);
    if (best > (i128)INT64_MAX) return -3;
    *wait = (int64_t)best;
    *barrier = best_t;
    recover_idx(M, n, R, best_t, idx);
    return 0;
}

/* ------------------------------------------------------- Algorithm 2, as printed
 * Z is kept as one slot per worker (in[p], zt[p], zi[p]).  "min(Z)" is the
 * element of Z that entered first among those with the smallest timestamp.
 * If Omega runs out while Z is being refilled the search stops and the
 * incomplete Z is not evaluated (the listing has no test for that case).
 * Only the RANGE objective: the listing computes max(Z) - min(Z).
 * idx_alg2[p] is the element of Z* itself (it can be an earlier element than
 * idx of the other functions when workers tie at the barrier). */
int zlo_alg2(const int64_t *M, int n, int R,
             int64_t *wait, int64_t *barrier, int32_t *idx_alg2) {
    if (!M || n < 1 || R < 1 || !wait || !barrier || !idx_alg2) return -1;
    int rc = check_rows(M, n, R);
    if (rc) return rc;
    size_t N = (size_t)n * R, pos = 0;
    zlo_elem *om = build_omega(M, n, R);
    int64_t *zt = (int64_t *)malloc((size_t)n * sizeof(int64_t));
    int32_t *zi = (int32_t *)malloc((size_t)n * sizeof(int32_t));
    size_t *zpos = (size_t *)malloc((size_t)n * sizeof(size_t));
    char *in = (char *)calloc((size_t)n, 1);
    if (!om || !zt || !zi || !zpos || !in) { free(om); free(zt); free(zi); free(zpos); free(in); return -4; }
    int size = 0;
#define ADD_LEFTMOST() do { zlo_elem w = om[pos]; if (!in[w.p]) { in[w.p] = 1; ++size; } \
                            zt[w.p] = w.t; zi[w.p] = w.i; zpos[w.p] = pos; ++pos; } while (0)
#define EVAL(mx, mn) do { mx = INT64_MIN; mn = INT64_MAX; \
        for (int q = 0; q < n; ++q) { if (zt[q] > mx) mx = zt[q]; if (zt[q] < mn) mn = zt[q]; } } while (0)
    while (size < n) ADD_LEFTMOST();             /* N >= n and every worker occurs: terminates */
    int64_t mx, mn;
    EVAL(mx, mn);
    int64_t best = mx - mn, best_t = mx;
    for (int q = 0; q < n; ++q) idx_alg2[q] = zi[q];
    while (pos < N) {
        int drop = 0;                            /* remove min(Z): oldest position */
        for (int q = 1; q < n; ++q) if (zpos[q] < zpos[drop]) drop = q;
        in[drop] = 0; --size;
        while (size < n && pos < N) ADD_LEFTMOST();
        if (size < n) break;
        EVAL(mx, mn);
        if (mx - mn < best) {
            best = mx - mn; best_t = mx;
            for (int q = 0; q < n; ++q) idx_alg2[q] = zi[q];
        }
    }
#undef ADD_LEFTMOST
#undef EVAL
    free(om); free(zt); free(zi); free(zpos); free(in);
    *wait = best;
    *barrier = best_t;
    return 0;
}

/* ----------------------------------------------------------------------- trace
 * Per position k of Omega (order: timestamp, worker, iteration), N = n*R:
 *   om_t, om_p, om_i  the element
 *   delta[k]  = e^p_i - e^p_{i-1}   (e^p_1 itself for the first element of a row)
 *   first[k]  = 1 if it is the first element of its row
 *   S[k]      = inclusive prefix sum of delta  = sum over started workers of their latest element
 *   cnt[k]    = inclusive prefix sum of first  = workers present in Z
 *   next[k]   = e^p_{i+1}, INT64_MAX for the last element of a row
 *   PM[k]     = max of next over positions < k  (INT64_MIN at k = 0)
 *   d_range[k]= max(om_t[k], t0, PM[k]) - om_t[k] with t0 = max_p e^p_1; INT64_MAX if that max is INT64_MAX.
 *               This is d_Z of the best Z whose smallest element is position k.
 *   w_sum[k]  = n*om_t[k] - S[k] if cnt[k] == n, else INT64_MAX
 * Any output pointer may be NULL. */
int zlo_trace(const int64_t *M, int n, int R,
              int64_t *om_t, int32_t *om_p, int32_t *om_i,
              int64_t *delta, int32_t *first, int64_t *S, int32_t *cnt,
              int64_t *next, int64_t *PM, int64_t *d_range, int64_t *w_sum) {
    if (!M || n < 1 || R < 1) return -1;
    int rc = check_rows(M, n, R);
    if (rc) return rc;
    size_t N = (size_t)n * R;
    zlo_elem *om = build_omega(M, n, R);
    if (!om) return -4;
    int64_t t0 = M[0];
    for (int p = 1; p < n; ++p) if (M[(size_t)p * R] > t0) t0 = M[(size_t)p * R];
    i128 s = 0;
    int c = 0;
    int64_t pm = INT64_MIN;
    for (size_t k = 0; k < N; ++k) {
        zlo_elem e = om[k];
        const int64_t *row = M + (size_t)e.p * R;
        int64_t dl = e.i == 0 ? e.t : e.t - row[e.i - 1];
        int64_t nx = e.i == R - 1 ? INT64_MAX : row[e.i + 1];
        s += dl;
        c += e.i == 0;
        if (s > (i128)INT64_MAX) { free(om); return -3; }
        if (om_t) om_t[k] = e.t;
        if (om_p) om_p[k] = e.p;
        if (om_i) om_i[k] = e.i;
        if (delta) delta[k] = dl;
        if (first) first[k] = e.i == 0;
        if (S) S[k] = (int64_t)s;
        if (cnt) cnt[k] = c;
        if (next) next[k] = nx;
        if (PM) PM[k] = pm;
        if (d_range) {
            int64_t g = e.t;
            if (t0 > g) g = t0;
            if (pm > g) g = pm;
            d_range[k] = g == INT64_MAX ? INT64_MAX : g - e.t;
        }
        if (w_sum) {
            i128 w = (i128)n * e.t - s;
            if (c == n && w > (i128)INT64_MAX) { free(om); return -3; }
            w_sum[k] = c == n ? (int64_t)w : INT64_MAX;
        }
        if (nx > pm) pm = nx;
    }
    free(om);
    return 0;
}

/* ---------------------------------------------------------------------- predictor
 * Phase 1 of ZipLine (Introduction; Section II, first property; Section III): the future iteration
 * intervals of a worker are predicted from its most recent interval under the stable-environment
 * assumption.  The paper gives no formula; the reading taken is constant-interval extrapolation:
 *   e^p_i = last[p] + i * interval[p],  i = 1..R
 * last[p] = the worker's latest observed end timestamp, interval[p] >= 0 its most recent interval.
 * out is [n][R].  Returns -1 on bad arguments, -3 if a value would reach 2^62. */
int zlo_predict(const int64_t *last, const int64_t *interval, int n, int R, int64_t *out) {
    if (!last || !interval || !out || n < 1 || R < 1) return -1;
    const i128 limit = (i128)1 << 62;
    for (int p = 0; p < n; ++p) {
        if (last[p] < 0 || interval[p] < 0) return -1;
        for (int i = 1; i <= R; ++i) {
            i128 v = (i128)last[p] + (i128)i * interval[p];
            if (v >= limit) return -3;
            out[(size_t)p * R + (i - 1)] = (int64_t)v;
        }
    }
    return 0;
}

/* ------------------------------------------------------- Algorithm 1 (GridScan) / FullGridScan
 * GridScan (Section IV, Algorithm 1): the designated row is the one with the earliest first element
 * (the lowest-numbered such row).  For every point e of the designated row, Z holds e and, from every
 * other row, the point at the shortest distance |M[p][i] - e|; d_Z = max(Z) - min(Z); the first Z with
 * a strictly smaller d_Z is kept.  FullGridScan (same section) designates every row in turn, rows in
 * order, keeping the strict minimum over all n*R candidates.
 * Readings: between two points of a row at equal distance the earlier one is taken; among equal points
 * of a row the one with the lowest index.  Heuristics: wait >= the optimum of the search above.
 * idx[p] = index of the element of Z* in row p; barrier = max(Z*). */
int zlo_gridscan(const int64_t *M, int n, int R, int full, int64_t *wait, int64_t *barrier, int32_t *idx) {
    if (!M || n < 1 || R < 1 || !wait || !barrier || !idx) return -1;
    int rc = check_rows(M, n, R);
    if (rc) return rc;
    int32_t *z = (int32_t *)malloc((size_t)n * sizeof(int32_t));
    if (!z) return -4;
    int pb = 0;
    for (int p = 1; p < n; ++p) if (M[(size_t)p * R] < M[(size_t)pb * R]) pb = p;
    int have = 0;
    int64_t best = 0, best_max = 0;
    for (int q = full ? 0 : pb; q < (full ? n : pb + 1); ++q) {
        for (int j = 0; j < R; ++j) {
            const int64_t e = M[(size_t)q * R + j];
            int64_t mx = e, mn = e;
            for (int p = 0; p < n; ++p) {
                if (p == q) { z[p] = j; continue; }
                int bi = 0;
                int64_t bd = INT64_MAX;
                for (int i = 0; i < R; ++i) {                     /* shortest distance; earlier point on ties */
                    int64_t v = M[(size_t)p * R + i];
                    int64_t dist = v > e ? v - e : e - v;
                    if (dist < bd) { bd = dist; bi = i; }
                }
                z[p] = bi;
                int64_t v = M[(size_t)p * R + bi];
                if (v > mx) mx = v;
                if (v < mn) mn = v;
            }
            if (!have || mx - mn < best) {
                have = 1; best = mx - mn; best_max = mx;
                memcpy(idx, z, (size_t)n * sizeof(int32_t));
            }
        }
    }
    free(z);
    *wait = best;
    *barrier = best_max;
    return 0;
}
