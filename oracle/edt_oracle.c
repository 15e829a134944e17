/*
 * CPU oracle for the exact Euclidean distance transform (EDT).
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the test-suite, the smoke check and the
 * CPU-baseline leg of the benchmark may call this library.  It shares no code, header,
 * table or helper with the CUDA library and does not know that library exists.
 *
 * What it computes (paper, Section 2.1 "Covered transforms", paragraph "Distance transforms":
 * every foreground element is labelled with its distance to the nearest background element;
 * Section 2.3.2 "Distance-transform kernels": nearest-background indices on request):
 *
 *   for every image (b, c) of a contiguous row-major (B, C, n_0 .. n_{d-1}) uint8 mask, with
 *   Z = { z : mask[b, c, z] == 0 } and per-axis sampling w_k > 0,
 *
 *       sq(x)   = min over z in Z of  sum_k ( w_k * (x_k - z_k) )^2
 *       dist(x) = sqrt(sq(x))
 *       idx(x)  = some z in Z attaining the minimum
 *
 *   Z empty  ->  sq = +inf (INT64_MAX in the integer output), dist = +inf, every index
 *   component = -1, decided per image.
 *
 * Two routines:
 *
 *   edt_oracle_brute  the definition written out: every voxel against every background voxel.
 *                     Quadratic; tiny inputs only.
 *   edt_oracle_sep    the same minimum rewritten as nested per-axis minima.  Because the summand
 *                     separates per axis,
 *                         g_{-1}(x) = 0 if x in Z else +inf
 *                         g_k(x)    = min_j [ g_{k-1}(x with x_k := j) + (w_k (x_k - j))^2 ]
 *                     taken over the axes in any order, ends at sq(x) (the separable formulation of
 *                     Section 2.3.2).  Each inner minimum is an exhaustive scan of the line -- no
 *                     envelope logic.  The scan walks outward from x_k in both directions and stops
 *                     once (w_k * delta)^2 >= best: no farther j can give a smaller value, so the
 *                     result is still the exhaustive minimum.
 *
 * Arithmetic: when every w_k == 1.0 the squared distances are int64 and exact; otherwise they are
 * float64.  Distances are float64 sqrt of those.
 *
 * Pins (tests, CPU only): brute force is checked against hand-computed fixtures, closed forms
 * (single background voxel, half-space masks) and SciPy called as a black box; edt_oracle_sep is
 * checked against brute force on small inputs of every rank and against invariants (axis
 * permutation / flip, 1-Lipschitz neighbours, monotonicity, batch independence).
 * The choice among equidistant background voxels is deliberately unpinned: any minimiser is valid.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define EDT_ORACLE_MAX_DIMS 8

enum { EDT_ORACLE_OK = 0, EDT_ORACLE_BAD_ARG = 1, EDT_ORACLE_NO_MEM = 2 };

static int unit_sampling(int ndim, const double* sampling) {
    if (!sampling) return 1;
    for (int k = 0; k < ndim; ++k)
        if (sampling[k] != 1.0) return 0;
    return 1;
}

static int check_args(const uint8_t* mask, int ndim, const int64_t* shape, const double* sampling) {
    if (!mask || !shape || ndim < 1 || ndim > EDT_ORACLE_MAX_DIMS) return EDT_ORACLE_BAD_ARG;
    for (int k = 0; k < ndim + 2; ++k)
        if (shape[k] < 0) return EDT_ORACLE_BAD_ARG;
    if (sampling)
        for (int k = 0; k < ndim; ++k)
            if (!(sampling[k] > 0.0) || isinf(sampling[k])) return EDT_ORACLE_BAD_ARG;
    return EDT_ORACLE_OK;
}

/* Row-major decode of a linear spatial index into coordinates. */
static void decode(int64_t lin, int ndim, const int64_t* n, int64_t* coord) {
    for (int k = ndim - 1; k >= 0; --k) {
        coord[k] = lin % n[k];
        lin /= n[k];
    }
}

/*
 * Writes the outputs of one image from its per-voxel squared distance and site.
 * site[x] = linear spatial index of the chosen background voxel, or -1.
 */
static void write_image_outputs(int64_t V, int ndim, const int64_t* n, int is_unit, const int64_t* sq_i,
                                const double* sq_f, const int64_t* site, double* out_dist, int64_t* out_sq,
                                int64_t* out_idx) {
    int64_t coord[EDT_ORACLE_MAX_DIMS];
    for (int64_t x = 0; x < V; ++x) {
        int none = site[x] < 0;
        if (out_dist) out_dist[x] = none ? INFINITY : sqrt(is_unit ? (double)sq_i[x] : sq_f[x]);
        if (out_sq) out_sq[x] = none ? INT64_MAX : sq_i[x];
        if (out_idx) {
            if (none) {
                for (int k = 0; k < ndim; ++k) out_idx[(int64_t)k * V + x] = -1;
            } else {
                decode(site[x], ndim, n, coord);
                for (int k = 0; k < ndim; ++k) out_idx[(int64_t)k * V + x] = coord[k];
            }
        }
    }
}

/*
 * The definition, literally.  Outputs (each may be NULL):
 *   out_dist  float64 (B, C, n...)       distance
 *   out_sq    int64   (B, C, n...)       exact squared distance; only meaningful for unit sampling
 *                                        (left untouched otherwise)
 *   out_sqf   float64 (B, C, n...)       squared distance as float64 (both modes)
 *   out_idx   int64   (B, C, ndim, n...) coordinates of the chosen background voxel
 * Ties: the background voxel met first in row-major order wins.
 */
int edt_oracle_brute(const uint8_t* mask, int ndim, const int64_t* shape, const double* sampling, double* out_dist,
                     int64_t* out_sq, double* out_sqf, int64_t* out_idx) {
    int rc = check_args(mask, ndim, shape, sampling);
    if (rc) return rc;
    const int64_t* n = shape + 2;
    int64_t images = shape[0] * shape[1], V = 1;
    for (int k = 0; k < ndim; ++k) V *= n[k];
    if (images == 0 || V == 0) return EDT_ORACLE_OK;
    int is_unit = unit_sampling(ndim, sampling);
    double w[EDT_ORACLE_MAX_DIMS];
    for (int k = 0; k < ndim; ++k) w[k] = sampling ? sampling[k] : 1.0;

    int64_t* zlist = (int64_t*)malloc(sizeof(int64_t) * (size_t)V * (size_t)ndim);
    int64_t* sq_i = (int64_t*)malloc(sizeof(int64_t) * (size_t)V);
    double* sq_f = (double*)malloc(sizeof(double) * (size_t)V);
    int64_t* site = (int64_t*)malloc(sizeof(int64_t) * (size_t)V);
    if (!zlist || !sq_i || !sq_f || !site) {
        free(zlist); free(sq_i); free(sq_f); free(site);
        return EDT_ORACLE_NO_MEM;
    }
    for (int64_t img = 0; img < images; ++img) {
        const uint8_t* m = mask + img * V;
        int64_t nz = 0;
        for (int64_t x = 0; x < V; ++x)
            if (m[x] == 0) {
                decode(x, ndim, n, zlist + nz * ndim);
                ++nz;
            }
        /* linear indices of background voxels, in the same order as zlist */
        int64_t* zl = (int64_t*)malloc(sizeof(int64_t) * (size_t)(nz > 0 ? nz : 1));
        if (!zl) { free(zlist); free(sq_i); free(sq_f); free(site); return EDT_ORACLE_NO_MEM; }
        {
            int64_t t = 0;
            for (int64_t x = 0; x < V; ++x)
                if (m[x] == 0) zl[t++] = x;
        }
        for (int64_t x = 0; x < V; ++x) {
            int64_t cx[EDT_ORACLE_MAX_DIMS];
            decode(x, ndim, n, cx);
            int64_t best_i = INT64_MAX, best_site = -1;
            double best_f = INFINITY;
            for (int64_t t = 0; t < nz; ++t) {
                const int64_t* z = zlist + t * ndim;
                if (is_unit) {
                    int64_t s = 0;
                    for (int k = 0; k < ndim; ++k) {
                        int64_t d = cx[k] - z[k];
                        s += d * d;
                    }
                    if (s < best_i) { best_i = s; best_site = zl[t]; }
                } else {
                    double s = 0.0;
                    for (int k = 0; k < ndim; ++k) {
                        double d = w[k] * (double)(cx[k] - z[k]);
                        s += d * d;
                    }
                    if (s < best_f) { best_f = s; best_site = zl[t]; }
                }
            }
            sq_i[x] = best_i;
            sq_f[x] = is_unit ? (best_site < 0 ? INFINITY : (double)best_i) : best_f;
            site[x] = best_site;
        }
        free(zl);
        write_image_outputs(V, ndim, n, is_unit, sq_i, sq_f, site, out_dist ? out_dist + img * V : NULL,
                            (out_sq && is_unit) ? out_sq + img * V : NULL,
                            out_idx ? out_idx + img * V * ndim : NULL);
        if (out_sqf) memcpy(out_sqf + img * V, sq_f, sizeof(double) * (size_t)V);
    }
    free(zlist); free(sq_i); free(sq_f); free(site);
    return EDT_ORACLE_OK;
}

/*
 * One nested minimum along spatial axis `axis` of one image, in place on (g, site).
 * The image is viewed as (outer, n_axis, inner) with strides (n_axis*inner, inner, 1).
 * is_unit: g_i is used (INT64_MAX = +inf, never entering arithmetic); else g_f (IEEE +inf).
 */
static int sep_axis_pass(int64_t V, int ndim, const int64_t* n, int axis, double w, int is_unit, int64_t* g_i,
                         double* g_f, int64_t* site) {
    int64_t len = n[axis], inner = 1;
    for (int k = axis + 1; k < ndim; ++k) inner *= n[k];
    int64_t outer = V / (len * inner);
    int64_t lines = outer * inner;
    int failed = 0;
#pragma omp parallel
    {
        int64_t* tmp_i = (int64_t*)malloc(sizeof(int64_t) * (size_t)len);
        double* tmp_f = (double*)malloc(sizeof(double) * (size_t)len);
        int64_t* tmp_s = (int64_t*)malloc(sizeof(int64_t) * (size_t)len);
        if (!tmp_i || !tmp_f || !tmp_s) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(static)
            for (int64_t line = 0; line < lines; ++line) {
                int64_t o = line / inner, r = line % inner;
                int64_t base = o * len * inner + r;
                for (int64_t i = 0; i < len; ++i) {
                    int64_t p = base + i * inner;
                    int64_t best_s = site[p];
                    if (is_unit) {
                        int64_t best = g_i[p]; /* j = i term: + 0 */
                        for (int64_t delta = 1; delta < len; ++delta) {
                            int64_t add = delta * delta; /* (1 * delta)^2 */
                            if (add >= best) break;      /* no farther j can be smaller */
                            int64_t jl = i - delta, jr = i + delta;
                            if (jl < 0 && jr >= len) break;
                            if (jl >= 0) {
                                int64_t q = base + jl * inner;
                                if (g_i[q] != INT64_MAX && g_i[q] + add < best) { best = g_i[q] + add; best_s = site[q]; }
                            }
                            if (jr < len) {
                                int64_t q = base + jr * inner;
                                if (g_i[q] != INT64_MAX && g_i[q] + add < best) { best = g_i[q] + add; best_s = site[q]; }
                            }
                        }
                        tmp_i[i] = best;
                    } else {
                        double best = g_f[p];
                        for (int64_t delta = 1; delta < len; ++delta) {
                            double t = w * (double)delta;
                            double add = t * t;
                            if (add >= best) break;
                            int64_t jl = i - delta, jr = i + delta;
                            if (jl < 0 && jr >= len) break;
                            if (jl >= 0) {
                                int64_t q = base + jl * inner;
                                if (g_f[q] + add < best) { best = g_f[q] + add; best_s = site[q]; }
                            }
                            if (jr < len) {
                                int64_t q = base + jr * inner;
                                if (g_f[q] + add < best) { best = g_f[q] + add; best_s = site[q]; }
                            }
                        }
                        tmp_f[i] = best;
                    }
                    tmp_s[i] = best_s;
                }
                for (int64_t i = 0; i < len; ++i) {
                    int64_t p = base + i * inner;
                    if (is_unit) g_i[p] = tmp_i[i]; else g_f[p] = tmp_f[i];
                    site[p] = tmp_s[i];
                }
            }
        }
        free(tmp_i); free(tmp_f); free(tmp_s);
    }
    return failed ? EDT_ORACLE_NO_MEM : EDT_ORACLE_OK;
}

/*
 * Nested per-axis minima over the spatial axes listed in `axes` (naxes entries, each axis at most
 * once), in that order.  With all ndim axes listed (axes == NULL means 0, 1, .. ndim-1) the result is
 * the distance transform; with a subset it is the intermediate g after those axes, which lets a
 * single pass of another implementation be checked on its own.
 *
 * Outputs (each may be NULL):
 *   out_dist float64 (B,C,n...)        sqrt of the value below
 *   out_sq   int64   (B,C,n...)        g as int64, unit sampling only (INT64_MAX = +inf)
 *   out_sqf  float64 (B,C,n...)        g as float64 (+inf where no site)
 *   out_idx  int64   (B,C,ndim,n...)   coordinates of the carried site (-1 where none)
 * Ties: a candidate replaces the current best only when strictly smaller; at equal delta the
 * lower j is examined first.
 */
int edt_oracle_sep_axes(const uint8_t* mask, int ndim, const int64_t* shape, const double* sampling, const int* axes,
                        int naxes, double* out_dist, int64_t* out_sq, double* out_sqf, int64_t* out_idx) {
    int rc = check_args(mask, ndim, shape, sampling);
    if (rc) return rc;
    int order[EDT_ORACLE_MAX_DIMS], seen[EDT_ORACLE_MAX_DIMS] = {0};
    if (!axes) {
        naxes = ndim;
        for (int k = 0; k < ndim; ++k) order[k] = k;
    } else {
        if (naxes < 0 || naxes > ndim) return EDT_ORACLE_BAD_ARG;
        for (int k = 0; k < naxes; ++k) {
            if (axes[k] < 0 || axes[k] >= ndim || seen[axes[k]]) return EDT_ORACLE_BAD_ARG;
            seen[axes[k]] = 1;
            order[k] = axes[k];
        }
    }
    const int64_t* n = shape + 2;
    int64_t images = shape[0] * shape[1], V = 1;
    for (int k = 0; k < ndim; ++k) V *= n[k];
    if (images == 0 || V == 0) return EDT_ORACLE_OK;
    int is_unit = unit_sampling(ndim, sampling);

    int64_t* g_i = is_unit ? (int64_t*)malloc(sizeof(int64_t) * (size_t)V) : NULL;
    double* g_f = (double*)malloc(sizeof(double) * (size_t)V);
    int64_t* site = (int64_t*)malloc(sizeof(int64_t) * (size_t)V);
    if ((is_unit && !g_i) || !g_f || !site) {
        free(g_i); free(g_f); free(site);
        return EDT_ORACLE_NO_MEM;
    }
    for (int64_t img = 0; img < images; ++img) {
        const uint8_t* m = mask + img * V;
        for (int64_t x = 0; x < V; ++x) { /* g_{-1} */
            int bg = (m[x] == 0);
            if (is_unit) g_i[x] = bg ? 0 : INT64_MAX; else g_f[x] = bg ? 0.0 : INFINITY;
            site[x] = bg ? x : -1;
        }
        for (int t = 0; t < naxes; ++t) {
            int a = order[t];
            rc = sep_axis_pass(V, ndim, n, a, sampling ? sampling[a] : 1.0, is_unit, g_i, g_f, site);
            if (rc) { free(g_i); free(g_f); free(site); return rc; }
        }
        if (is_unit)
            for (int64_t x = 0; x < V; ++x) g_f[x] = (g_i[x] == INT64_MAX) ? INFINITY : (double)g_i[x];
        write_image_outputs(V, ndim, n, is_unit, g_i, g_f, site, out_dist ? out_dist + img * V : NULL,
                            (out_sq && is_unit) ? out_sq + img * V : NULL,
                            out_idx ? out_idx + img * V * ndim : NULL);
        if (out_sqf) memcpy(out_sqf + img * V, g_f, sizeof(double) * (size_t)V);
    }
    free(g_i); free(g_f); free(site);
    return EDT_ORACLE_OK;
}

/* The full transform: nested minima over every axis. */
int edt_oracle_sep(const uint8_t* mask, int ndim, const int64_t* shape, const double* sampling, double* out_dist,
                   int64_t* out_sq, double* out_sqf, int64_t* out_idx) {
    return edt_oracle_sep_axes(mask, ndim, shape, sampling, NULL, 0, out_dist, out_sq, out_sqf, out_idx);
}

/* Threads the per-line loops will use (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int edt_oracle_threads(void) { return omp_get_max_threads(); }
void edt_oracle_set_threads(int t) { if (t > 0) omp_set_num_threads(t); }
#else
int edt_oracle_threads(void) { return 1; }
void edt_oracle_set_threads(int t) { (void)t; }
#endif
