/*
 * sna_oracle.c — fp64 CPU oracle for spherical neighborhood attention.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA library is
 * checked against.  It shares no code, header, table or constant with the CUDA path and must never
 * be linked, imported or called by it.  Only the tests, the smoke check and the CPU-baseline /
 * reference legs of the benchmark may use it.
 *
 * Everything is double precision.  There is no blocking, fusion or reordering beyond what the
 * definitions state; OpenMP only distributes independent outer iterations (output points, or
 * independent batch*head slices for the scatter in the backward pass).
 *
 * What each routine follows (paper = "Attention on the Sphere", arXiv 2505.11157):
 *   - sphere parametrisation x(theta, phi)                : App. A.1, first equation
 *   - quadrature rule sum_i u(x_i) w_i                    : Eq. (quadrature), Sec. 3.2; App. A.1
 *   - geodesic disc D(x) = {x' : d(x,x') <= theta_cutoff} : Eq. (s2_neighborhood_attention)
 *   - indicator table 1[h,h',w'] built at output lon 0    : App. B.3 (text after the DISCO equation)
 *   - forward                                             : App. B.3, Eq. (s2_attention_discrete_detailed)
 *   - gradients                                           : App. B.4 (quotient rule / softmax identity)
 *   - global attention as softmax with bias log(w)        : App. B.1 Eq. (s2_attention_discrete), App. B.2
 *
 * Readings taken where the paper is silent (all listed again in the design notes):
 *   - equiangular grid includes both poles, theta_h = pi*h/(nlat-1), Clenshaw-Curtis weights;
 *   - the grid App. A.1 itself prints (theta_i = pi*i/nlat, i = 0..nlat-1: north pole in, south pole out, point
 *     weights 2 pi^2/(nlat nlon) sin(theta_i)) is the third grid, "equiangular trapezoid": its weights are the
 *     composite trapezoid rule in theta and sum to 4 pi only approximately; its pole ring has weight zero, so
 *     those points are members of a disc but contribute nothing, and an output point whose whole disc has
 *     weight zero has no defined result (0/0) and is reported as an empty neighborhood;
 *   - "Gaussian grid" = Gauss-Legendre nodes in cos(theta), ordered north to south;
 *   - point weight w_{h'} = (latitude weight) * 2*pi/nlon_in, so the weights sum to 4*pi;
 *   - different resolutions: input column = (w' + w*ps) mod nlon_in with ps = nlon_in/nlon_out;
 *   - ties on the disc boundary count as inside: member iff d <= theta_cutoff + 1e-10, and a pair
 *     with 1e-12 < |d - theta_cutoff| < 1e-8 is reported as ambiguous instead of being decided by
 *     rounding; theta_cutoff >= pi selects every point;
 *   - scale 1/sqrt(C) with C the per-head channel count, in forward and backward;
 *   - batch and heads are one flat leading dimension N of independent problems.
 *
 * Array layouts (all contiguous, channels last):
 *   q, out, dout, dq : [N][nlat_out][nlon_out][C]      k, v, dk, dv : [N][nlat_in][nlon_in][C]
 *
 * Parity status: every routine here is pinned by the CPU tests (closed-form weights, polynomial
 * exactness, library Gauss-Legendre nodes, hand-derived tiny tables, softmax invariants, roll
 * equivariance, the theta_cutoff = pi limit against a library dense attention, finite differences).
 * Nothing is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_INVALID 1
#define ORACLE_ERR_AMBIGUOUS_TIE 2
#define ORACLE_ERR_EMPTY_NEIGHBORHOOD 3
#define ORACLE_ERR_CAPACITY 4

#define GRID_EQUIANGULAR 0
#define GRID_LEGENDRE_GAUSS 1
#define GRID_EQUIANGULAR_TRAPEZOID 2

static const double PI = 3.14159265358979323846264338327950288;

int sna_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Legendre polynomial P_n(x) and its derivative by the three-term recurrence. */
static void legendre_pn(int n, double x, double *p, double *dp) {
    double p0 = 1.0, p1 = x;
    if (n == 0) { *p = 1.0; *dp = 0.0; return; }
    for (int l = 2; l <= n; ++l) {
        double p2 = ((2.0 * l - 1.0) * x * p1 - (l - 1.0) * p0) / l;
        p0 = p1; p1 = p2;
    }
    *p = p1;
    *dp = n * (x * p1 - p0) / (x * x - 1.0);
}

/* Gauss-Legendre nodes x_h (descending, so colatitude ascends) and weights on [-1, 1]. */
static void gauss_legendre(int n, double *x, double *w) {
    for (int i = 0; i < n; ++i) {
        double z = cos(PI * (i + 0.75) / (n + 0.5));
        for (int it = 0; it < 100; ++it) {
            double p, dp;
            legendre_pn(n, z, &p, &dp);
            double dz = p / dp;
            z -= dz;
            if (fabs(dz) < 1e-16) break;
        }
        double p, dp;
        legendre_pn(n, z, &p, &dp);
        x[i] = z;
        w[i] = 2.0 / ((1.0 - z * z) * dp * dp);
    }
}

/* Colatitudes theta_h, h = 0 (north) ... nlat-1 (south).  App. A.1. */
int sna_oracle_colatitudes(int grid, int nlat, double *theta) {
    if (nlat < 2 || !theta) return ORACLE_ERR_INVALID;
    if (grid == GRID_EQUIANGULAR) {
        for (int h = 0; h < nlat; ++h) theta[h] = PI * h / (nlat - 1);
        return ORACLE_OK;
    }
    if (grid == GRID_EQUIANGULAR_TRAPEZOID) {   /* Eq. (latlon_grid) */
        for (int h = 0; h < nlat; ++h) theta[h] = PI * h / nlat;
        return ORACLE_OK;
    }
    if (grid == GRID_LEGENDRE_GAUSS) {
        double *x = (double *)malloc(sizeof(double) * nlat * 2);
        if (!x) return ORACLE_ERR_INVALID;
        gauss_legendre(nlat, x, x + nlat);
        for (int h = 0; h < nlat; ++h) theta[h] = acos(x[h]);
        free(x);
        return ORACLE_OK;
    }
    return ORACLE_ERR_INVALID;
}

/* Latitude quadrature weights for int_{-1}^{1} f(cos theta) d(cos theta); they sum to 2 (the trapezoid
 * grid's to (pi/nlat) cot(pi/(2 nlat)) = 2 - pi^2/(6 nlat^2) + ...). */
int sna_oracle_latitude_weights(int grid, int nlat, double *wlat) {
    if (nlat < 2 || !wlat) return ORACLE_ERR_INVALID;
    if (grid == GRID_EQUIANGULAR) {
        /* Clenshaw-Curtis on nlat-1 intervals. */
        int n = nlat - 1;
        for (int h = 0; h < nlat; ++h) {
            double th = PI * h / n;
            double s = 1.0;
            for (int k = 1; k <= n / 2; ++k) {
                double b = (2 * k == n) ? 1.0 : 2.0;
                s -= b / (4.0 * k * k - 1.0) * cos(2.0 * k * th);
            }
            double c = (h == 0 || h == n) ? 1.0 : 2.0;
            wlat[h] = c / n * s;
        }
        return ORACLE_OK;
    }
    if (grid == GRID_EQUIANGULAR_TRAPEZOID) {
        /* Eq. (latlon_quad_weights): q_ij = 2 pi^2/(nlat nlon) sin(theta_i) = wlat_i * 2 pi/nlon. */
        for (int h = 0; h < nlat; ++h) wlat[h] = PI / nlat * sin(PI * h / nlat);
        return ORACLE_OK;
    }
    if (grid == GRID_LEGENDRE_GAUSS) {
        double *x = (double *)malloc(sizeof(double) * nlat);
        if (!x) return ORACLE_ERR_INVALID;
        gauss_legendre(nlat, x, wlat);
        free(x);
        return ORACLE_OK;
    }
    return ORACLE_ERR_INVALID;
}

/* Per-point quadrature weight of input ring h': omega[h'] = wlat[h'] * 2*pi/nlon.  Eq. (quadrature). */
int sna_oracle_quad_weights(int grid, int nlat, int nlon, double *omega) {
    int rc = sna_oracle_latitude_weights(grid, nlat, omega);
    if (rc) return rc;
    if (nlon < 1) return ORACLE_ERR_INVALID;
    for (int h = 0; h < nlat; ++h) omega[h] *= 2.0 * PI / nlon;
    return ORACLE_OK;
}

/*
 * Neighborhood table by brute force: for every output latitude h (at output longitude 0) and every
 * input point (h', w'), the geodesic distance is arccos of the dot product of the two unit vectors.
 * Entries are emitted h' ascending, then w' ascending.  Call with capacity = 0 to get the count.
 */
int sna_oracle_neighborhood(int grid_in, int nlat_in, int nlon_in, int grid_out, int nlat_out,
                            double theta_cutoff, int64_t *row_ptr, int32_t *lat_in, int32_t *lon_off,
                            int64_t capacity, int64_t *nnz_out) {
    if (nlat_in < 2 || nlat_out < 2 || nlon_in < 1 || !(theta_cutoff > 0.0) || !nnz_out) return ORACLE_ERR_INVALID;
    double *th_in = (double *)malloc(sizeof(double) * nlat_in);
    double *th_out = (double *)malloc(sizeof(double) * nlat_out);
    double *w_in = (double *)malloc(sizeof(double) * nlat_in);
    int rc = sna_oracle_colatitudes(grid_in, nlat_in, th_in);
    if (!rc) rc = sna_oracle_colatitudes(grid_out, nlat_out, th_out);
    if (!rc) rc = sna_oracle_latitude_weights(grid_in, nlat_in, w_in);
    if (rc) { free(th_in); free(th_out); free(w_in); return rc; }
    const int everything = theta_cutoff >= PI;
    int64_t n = 0;
    int status = ORACLE_OK;
    for (int h = 0; h < nlat_out; ++h) {
        if (row_ptr) row_ptr[h] = n;
        const double xo[3] = { sin(th_out[h]), 0.0, cos(th_out[h]) };
        int64_t weighted = 0;   /* members with a non-zero quadrature weight */
        for (int hp = 0; hp < nlat_in; ++hp) {
            for (int wp = 0; wp < nlon_in; ++wp) {
                int member;
                if (everything) {
                    member = 1;
                } else {
                    double phi = 2.0 * PI * wp / nlon_in;
                    double xi[3] = { sin(th_in[hp]) * cos(phi), sin(th_in[hp]) * sin(phi), cos(th_in[hp]) };
                    double dot = xo[0] * xi[0] + xo[1] * xi[1] + xo[2] * xi[2];
                    if (dot > 1.0) dot = 1.0;
                    if (dot < -1.0) dot = -1.0;
                    double d = acos(dot);
                    double gap = fabs(d - theta_cutoff);
                    if (gap > 1e-12 && gap < 1e-8) status = ORACLE_ERR_AMBIGUOUS_TIE;
                    member = d <= theta_cutoff + 1e-10;
                }
                if (member) {
                    if (n < capacity && lat_in && lon_off) { lat_in[n] = hp; lon_off[n] = wp; }
                    ++n;
                    if (w_in[hp] > 0.0) ++weighted;
                }
            }
        }
        if (weighted == 0 && status == ORACLE_OK) status = ORACLE_ERR_EMPTY_NEIGHBORHOOD;
    }
    if (row_ptr) row_ptr[nlat_out] = n;
    *nnz_out = n;
    free(th_in); free(th_out); free(w_in);
    if (status) return status;
    if (capacity > 0 && n > capacity) return ORACLE_ERR_CAPACITY;
    return ORACLE_OK;
}

/* ---- one output point: the definition, written out -------------------------------------------- */

typedef struct {
    int nlat_in, nlon_in, nlat_out, nlon_out, C;
    const int64_t *row_ptr; const int32_t *lat_in; const int32_t *lon_off;
    const double *omega;
} geom_t;

static inline const double *in_point(const geom_t *g, const double *base, int n, int hp, int col) {
    return base + (((int64_t)n * g->nlat_in + hp) * g->nlon_in + col) * g->C;
}
static inline int64_t out_index(const geom_t *g, int n, int h, int w) {
    return (((int64_t)n * g->nlat_out + h) * g->nlon_out + w) * g->C;
}
static inline int in_column(const geom_t *g, int off, int w) {
    int ps = g->nlon_in / g->nlon_out;
    return (int)(((int64_t)off + (int64_t)w * ps) % g->nlon_in);
}

/* max_j s_ij and Z_i = sum_j exp(s_ij - max) * omega_j for output point i = (n, h, w). */
static void point_stats(const geom_t *g, const double *q, const double *k, int n, int h, int w,
                        double *smax, double *Z) {
    const double scale = 1.0 / sqrt((double)g->C);
    const double *qi = q + out_index(g, n, h, w);
    double m = -INFINITY;
    for (int64_t e = g->row_ptr[h]; e < g->row_ptr[h + 1]; ++e) {
        const double *kj = in_point(g, k, n, g->lat_in[e], in_column(g, g->lon_off[e], w));
        double s = 0.0;
        for (int c = 0; c < g->C; ++c) s += qi[c] * kj[c];
        s *= scale;
        if (s > m) m = s;
    }
    double z = 0.0;
    for (int64_t e = g->row_ptr[h]; e < g->row_ptr[h + 1]; ++e) {
        const double *kj = in_point(g, k, n, g->lat_in[e], in_column(g, g->lon_off[e], w));
        double s = 0.0;
        for (int c = 0; c < g->C; ++c) s += qi[c] * kj[c];
        s *= scale;
        z += exp(s - m) * g->omega[g->lat_in[e]];
    }
    *smax = m; *Z = z;
}

/* y_i = sum_j alpha_ij v_j / sum_j alpha_ij, alpha_ij = exp(s_ij) omega_j.  Eq. (s2_attention_discrete_detailed). */
static void point_forward(const geom_t *g, const double *q, const double *k, const double *v,
                          int n, int h, int w, double *y, double *lse) {
    const double scale = 1.0 / sqrt((double)g->C);
    const double *qi = q + out_index(g, n, h, w);
    double m, Z;
    point_stats(g, q, k, n, h, w, &m, &Z);
    for (int c = 0; c < g->C; ++c) y[c] = 0.0;
    for (int64_t e = g->row_ptr[h]; e < g->row_ptr[h + 1]; ++e) {
        int hp = g->lat_in[e], col = in_column(g, g->lon_off[e], w);
        const double *kj = in_point(g, k, n, hp, col);
        const double *vj = in_point(g, v, n, hp, col);
        double s = 0.0;
        for (int c = 0; c < g->C; ++c) s += qi[c] * kj[c];
        double a = exp(s * scale - m) * g->omega[hp];
        for (int c = 0; c < g->C; ++c) y[c] += a * vj[c];
    }
    for (int c = 0; c < g->C; ++c) y[c] /= Z;
    if (lse) *lse = m + log(Z);
}

int sna_oracle_forward(int nlat_in, int nlon_in, int nlat_out, int nlon_out,
                       const int64_t *row_ptr, const int32_t *lat_in, const int32_t *lon_off,
                       const double *omega, int N, int C,
                       const double *q, const double *k, const double *v, double *out, double *lse) {
    if (nlon_out < 1 || nlon_in % nlon_out != 0 || N < 1 || C < 1) return ORACLE_ERR_INVALID;
    geom_t g = { nlat_in, nlon_in, nlat_out, nlon_out, C, row_ptr, lat_in, lon_off, omega };
    int64_t npts = (int64_t)N * nlat_out * nlon_out;
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t i = 0; i < npts; ++i) {
        int w = (int)(i % nlon_out);
        int h = (int)((i / nlon_out) % nlat_out);
        int n = (int)(i / ((int64_t)nlon_out * nlat_out));
        point_forward(&g, q, k, v, n, h, w, out + i * C, lse ? lse + i : NULL);
    }
    return ORACLE_OK;
}

/* Forward at selected output points pts[3*p + {0,1,2}] = (n, h, w). */
int sna_oracle_forward_points(int nlat_in, int nlon_in, int nlat_out, int nlon_out,
                              const int64_t *row_ptr, const int32_t *lat_in, const int32_t *lon_off,
                              const double *omega, int N, int C,
                              const double *q, const double *k, const double *v,
                              int64_t npts, const int32_t *pts, double *out) {
    if (nlon_out < 1 || nlon_in % nlon_out != 0 || N < 1 || C < 1) return ORACLE_ERR_INVALID;
    geom_t g = { nlat_in, nlon_in, nlat_out, nlon_out, C, row_ptr, lat_in, lon_off, omega };
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t p = 0; p < npts; ++p)
        point_forward(&g, q, k, v, pts[3 * p], pts[3 * p + 1], pts[3 * p + 2], out + p * C, NULL);
    return ORACLE_OK;
}

/*
 * Backward, App. B.4 with the outer sums restored:
 *   p_ij = alpha_ij / sum_l alpha_il,  t_ij = dy_i . v_j,  D_i = sum_j p_ij t_ij,
 *   ds_ij = p_ij (t_ij - D_i),
 *   dq_i  = scale * sum_j ds_ij k_j,   dk_j += scale * ds_ij q_i,   dv_j += p_ij dy_i.
 * dk and dv are scattered with plain "+=" inside each batch*head slice n.
 */
static void point_backward(const geom_t *g, const double *q, const double *k, const double *v,
                           const double *dout, int n, int h, int w,
                           double *dq_i, double *dk, double *dv) {
    const int C = g->C;
    const double scale = 1.0 / sqrt((double)C);
    const int64_t oi = out_index(g, n, h, w);
    const double *qi = q + oi, *dyi = dout + oi;
    double m, Z;
    point_stats(g, q, k, n, h, w, &m, &Z);
    double D = 0.0;
    for (int64_t e = g->row_ptr[h]; e < g->row_ptr[h + 1]; ++e) {
        int hp = g->lat_in[e], col = in_column(g, g->lon_off[e], w);
        const double *kj = in_point(g, k, n, hp, col), *vj = in_point(g, v, n, hp, col);
        double s = 0.0, t = 0.0;
        for (int c = 0; c < C; ++c) { s += qi[c] * kj[c]; t += dyi[c] * vj[c]; }
        double p = exp(s * scale - m) * g->omega[hp] / Z;
        D += p * t;
    }
    if (dq_i) for (int c = 0; c < C; ++c) dq_i[c] = 0.0;
    for (int64_t e = g->row_ptr[h]; e < g->row_ptr[h + 1]; ++e) {
        int hp = g->lat_in[e], col = in_column(g, g->lon_off[e], w);
        const double *kj = in_point(g, k, n, hp, col), *vj = in_point(g, v, n, hp, col);
        double s = 0.0, t = 0.0;
        for (int c = 0; c < C; ++c) { s += qi[c] * kj[c]; t += dyi[c] * vj[c]; }
        double p = exp(s * scale - m) * g->omega[hp] / Z;
        double ds = p * (t - D);
        if (dq_i) for (int c = 0; c < C; ++c) dq_i[c] += scale * ds * kj[c];
        if (dk) {
            double *dkj = dk + (kj - k);
            for (int c = 0; c < C; ++c) dkj[c] += scale * ds * qi[c];
        }
        if (dv) {
            double *dvj = dv + (vj - v);
            for (int c = 0; c < C; ++c) dvj[c] += p * dyi[c];
        }
    }
}

int sna_oracle_backward(int nlat_in, int nlon_in, int nlat_out, int nlon_out,
                        const int64_t *row_ptr, const int32_t *lat_in, const int32_t *lon_off,
                        const double *omega, int N, int C,
                        const double *q, const double *k, const double *v, const double *dout,
                        double *dq, double *dk, double *dv) {
    if (nlon_out < 1 || nlon_in % nlon_out != 0 || N < 1 || C < 1) return ORACLE_ERR_INVALID;
    geom_t g = { nlat_in, nlon_in, nlat_out, nlon_out, C, row_ptr, lat_in, lon_off, omega };
    memset(dk, 0, sizeof(double) * (size_t)N * nlat_in * nlon_in * C);
    memset(dv, 0, sizeof(double) * (size_t)N * nlat_in * nlon_in * C);
    /* slices n are independent problems; inside a slice the scatter is serial */
#pragma omp parallel for schedule(dynamic, 1)
    for (int n = 0; n < N; ++n)
        for (int h = 0; h < nlat_out; ++h)
            for (int w = 0; w < nlon_out; ++w)
                point_backward(&g, q, k, v, dout, n, h, w, dq + out_index(&g, n, h, w), dk, dv);
    return ORACLE_OK;
}

/* dq at selected output points (n, h, w). */
int sna_oracle_dq_points(int nlat_in, int nlon_in, int nlat_out, int nlon_out,
                         const int64_t *row_ptr, const int32_t *lat_in, const int32_t *lon_off,
                         const double *omega, int N, int C,
                         const double *q, const double *k, const double *v, const double *dout,
                         int64_t npts, const int32_t *pts, double *dq) {
    if (nlon_out < 1 || nlon_in % nlon_out != 0 || N < 1 || C < 1) return ORACLE_ERR_INVALID;
    geom_t g = { nlat_in, nlon_in, nlat_out, nlon_out, C, row_ptr, lat_in, lon_off, omega };
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t p = 0; p < npts; ++p)
        point_backward(&g, q, k, v, dout, pts[3 * p], pts[3 * p + 1], pts[3 * p + 2], dq + p * C, NULL, NULL);
    return ORACLE_OK;
}

/*
 * dk and dv at selected input points (n, h', w'): every output point whose disc contains the input
 * point is visited (found by scanning the whole table), its softmax is evaluated in full, and its
 * single contribution to this input point is added.
 */
int sna_oracle_dkdv_points(int nlat_in, int nlon_in, int nlat_out, int nlon_out,
                           const int64_t *row_ptr, const int32_t *lat_in, const int32_t *lon_off,
                           const double *omega, int N, int C,
                           const double *q, const double *k, const double *v, const double *dout,
                           int64_t npts, const int32_t *pts, double *dk, double *dv) {
    if (nlon_out < 1 || nlon_in % nlon_out != 0 || N < 1 || C < 1) return ORACLE_ERR_INVALID;
    geom_t g = { nlat_in, nlon_in, nlat_out, nlon_out, C, row_ptr, lat_in, lon_off, omega };
    const double scale = 1.0 / sqrt((double)C);
    const int ps = nlon_in / nlon_out;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t p = 0; p < npts; ++p) {
        int n = pts[3 * p], hp = pts[3 * p + 1], wp = pts[3 * p + 2];
        const double *kj = in_point(&g, k, n, hp, wp), *vj = in_point(&g, v, n, hp, wp);
        double *dkj = dk + p * C, *dvj = dv + p * C;
        for (int c = 0; c < C; ++c) { dkj[c] = 0.0; dvj[c] = 0.0; }
        for (int h = 0; h < nlat_out; ++h) {
            for (int64_t e = row_ptr[h]; e < row_ptr[h + 1]; ++e) {
                if (lat_in[e] != hp) continue;
                int shift = ((wp - lon_off[e]) % nlon_in + nlon_in) % nlon_in;  /* = w*ps */
                if (shift % ps != 0) continue;
                int w = shift / ps;
                /* output point i = (n, h, w) has this input point in its disc */
                const int64_t oi = out_index(&g, n, h, w);
                const double *qi = q + oi, *dyi = dout + oi;
                double m, Z;
                point_stats(&g, q, k, n, h, w, &m, &Z);
                double D = 0.0;
                for (int64_t f = row_ptr[h]; f < row_ptr[h + 1]; ++f) {
                    int hq = lat_in[f], col = in_column(&g, lon_off[f], w);
                    const double *kl = in_point(&g, k, n, hq, col), *vl = in_point(&g, v, n, hq, col);
                    double s = 0.0, t = 0.0;
                    for (int c = 0; c < C; ++c) { s += qi[c] * kl[c]; t += dyi[c] * vl[c]; }
                    D += exp(s * scale - m) * omega[hq] / Z * t;
                }
                double s = 0.0, t = 0.0;
                for (int c = 0; c < C; ++c) { s += qi[c] * kj[c]; t += dyi[c] * vj[c]; }
                double pij = exp(s * scale - m) * omega[hp] / Z;
                double ds = pij * (t - D);
                for (int c = 0; c < C; ++c) { dkj[c] += scale * ds * qi[c]; dvj[c] += pij * dyi[c]; }
            }
        }
    }
    return ORACLE_OK;
}

/*
 * Dense quadrature-weighted attention over ALL input points (no table): the discrete global
 * attention, i.e. softmax of s_ij + log(w_j).  App. B.1 Eq. (s2_attention_discrete), App. B.2.
 *   q, out [N][Mout][C];  k, v [N][Min][C];  wpt [Min] per-point weights.
 */
int sna_oracle_dense_forward(int N, int64_t Mout, int64_t Min, int C, const double *wpt,
                             const double *q, const double *k, const double *v, double *out) {
    if (N < 1 || C < 1 || Mout < 1 || Min < 1) return ORACLE_ERR_INVALID;
    const double scale = 1.0 / sqrt((double)C);
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t i = 0; i < (int64_t)N * Mout; ++i) {
        int n = (int)(i / Mout);
        const double *qi = q + i * C;
        const double *kn = k + (int64_t)n * Min * C, *vn = v + (int64_t)n * Min * C;
        double *lg = (double *)malloc(sizeof(double) * Min);
        double m = -INFINITY;
        for (int64_t j = 0; j < Min; ++j) {
            double s = 0.0;
            for (int c = 0; c < C; ++c) s += qi[c] * kn[j * C + c];
            lg[j] = s * scale + log(wpt[j]);
            if (lg[j] > m) m = lg[j];
        }
        double Z = 0.0;
        for (int64_t j = 0; j < Min; ++j) { lg[j] = exp(lg[j] - m); Z += lg[j]; }
        double *y = out + i * C;
        for (int c = 0; c < C; ++c) y[c] = 0.0;
        for (int64_t j = 0; j < Min; ++j)
            for (int c = 0; c < C; ++c) y[c] += lg[j] / Z * vn[j * C + c];
        free(lg);
    }
    return ORACLE_OK;
}
