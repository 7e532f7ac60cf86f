/*
 * gart_oracle.c -- float64 CPU oracle for ray-traced Gaussian rendering and its
 * analytic backward pass.
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, by-the-definition
 * implementation used only to check the CUDA library and to serve as the timed
 * CPU baseline of the benchmark.  It shares no code, header, table or constant
 * with the CUDA path and must never be reached from the product path.
 *
 * Everything is computed in double precision.  Inputs are double arrays (the
 * callers widen their fp32 scene arrays exactly).
 *
 * What each part follows (3DGART paper):
 *   - Gaussian density, covariance Sigma = R S S^T R^T ........ Sec. 3.1, Eq. 1-2
 *   - ray, local space o_g, d_g, maximum-response distance ... Sec. 3.2, Eq. 3-5
 *   - front-to-back compositing, T_i, alpha_i ................ Sec. 3.3, Eq. 6-8
 *   - clamping radius alpha_c, alpha_min ..................... Sec. 3.4, Eq. 9-10
 *   - perspective-correct screen-space AABB .................. Sec. 4.2, Eq. 11-14
 *   - tile / primitive pair lists, tile offsets .............. Sec. 4.3 ("Reverse Tile Mapping")
 *   - gradients w.r.t. mean, scale, quaternion, opacity, SH .. Sec. 4.4 (the sums the
 *     primitive-centric pass re-associates; 11 + 3K words per Gaussian,
 *     59 at SH degree 3)
 *
 * Pins (see tests/test_oracle_*.py): brute-force ellipsoid projection and the
 * textbook tangent-line bound of a sphere for the AABB; golden-section search
 * for the maximum-response point; the closed-form render of one isotropic
 * Gaussian; T_final = prod(1 - alpha_i) and the partition-of-unity invariant;
 * a two-Gaussian closed form with permutation invariance; Unsoeld's theorem and
 * numerical orthonormality for the SH table; central finite differences for
 * every gradient word; translation invariance (sum of dL/dmu = -dL/do); the per-hit
 * intermediate-buffer entries against the opacity and SH gradients they must reproduce
 * (dL/dsigma = sum <g, entry.xyz> / sigma, dL/dsh = sum Y w g on unclamped channels).
 *
 * Readings of the paper used here (the paper is silent or ambiguous):
 *   - pinhole camera, pixel centres at +0.5, unit ray directions;
 *   - T' rows are in pixel units (viewport folded in), the AABB selects pixels
 *     whose CENTRE lies inside [p - h, p + h];
 *   - a Gaussian is culled if sigma <= alpha_min or if its alpha_c-ellipsoid lies
 *     entirely at depth <= near; it is "front" if the ellipsoid lies entirely
 *     at depth >= near, otherwise it "straddles" and its rectangle is the whole
 *     image unless its bounding sphere is outside one of the four side planes;
 *   - a ray hits a Gaussian iff alpha >= alpha_min and t* > 0; by default no early
 *     termination, no alpha clamp, no hit cap (each is an option, off unless set);
 *   - hits are ordered by (t*, id); colour is max(0, 0.5 + sum_k Y_k(d) sh_k)
 *     with d the unit ray direction; background colour multiplies T_final;
 *   - gradients are with respect to the given (activated) parameters; the
 *     quaternion enters through the polynomial rotation formula without
 *     normalisation.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_MAX_K 16

typedef struct {
    int32_t width, height;
    double fx, fy, cx, cy;
    double w2c[12]; /* row-major [R | t] */
} orc_camera;

typedef struct {
    int64_t n;
    int32_t sh_degree;
    const double *mean;    /* [n,3] */
    const double *scale;   /* [n,3] */
    const double *quat;    /* [n,4] w,x,y,z */
    const double *opacity; /* [n] */
    const double *sh;      /* [n,K,3] */
} orc_scene;

typedef struct {
    double alpha_min;
    double near_z;
    double bg[3];
    int64_t max_hits; /* 0: every hit is composited (the paper's setting).  m > 0: only the first m hits of a ray in
                         (t*, id) order, the cap on ray-primitive intersections that the paper lists among the
                         compromises of 3DGRT (comparison with prior work); later hits weigh nothing */
    double t_min;     /* 0: off.  > 0: early termination, the other usual shortcut of such tracers: a ray ends before the
                         first hit whose transmittance in front, T_i, is below t_min; that hit and all later ones weigh
                         nothing (T_final is the transmittance reached) */
    double alpha_max; /* >= 1: off.  < 1: a hit's alpha is min(sigma rho, alpha_max); where the clamp is active alpha is a
                         constant, so the hit passes no gradient to opacity, mean, scale or rotation (its colour still
                         gets one) */
    int64_t kernel_degree; /* k of the response rho = exp(-D^k / 2), D the Mahalanobis distance of the ray's closest point
                         (Eq. 4 is k = 2, the paper's benchmark setting, Sec. 5.2; 0 means 2).  An even k > 2 is a "narrow"
                         kernel, the last of the compromises the paper lists for 3DGRT (Sec. 5.5): flatter top, faster
                         fall-off, and a clamping radius alpha_c = (2 ln(sigma / alpha_min))^(1/k) in place of Eq. 9-10's
                         square root.  The maximum-response point along a ray does not depend on k */
} orc_config;

static int kernel_degree_of(const orc_config *cfg) { return cfg->kernel_degree > 0 ? (int)cfg->kernel_degree : 2; }

/* ------------------------------------------------------------------ threads */
int orc_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
void orc_set_threads(int t) {
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* ------------------------------------------------------------------ small math */
/* Rotation matrix of a quaternion (w,x,y,z), polynomial form, row-major. */
static void quat_to_R(const double *q, double *R) {
    const double w = q[0], x = q[1], y = q[2], z = q[3];
    R[0] = 1.0 - 2.0 * (y * y + z * z); R[1] = 2.0 * (x * y - w * z);       R[2] = 2.0 * (x * z + w * y);
    R[3] = 2.0 * (x * y + w * z);       R[4] = 1.0 - 2.0 * (x * x + z * z); R[5] = 2.0 * (y * z - w * x);
    R[6] = 2.0 * (x * z - w * y);       R[7] = 2.0 * (y * z + w * x);       R[8] = 1.0 - 2.0 * (x * x + y * y);
}

/* Real spherical harmonics up to degree 3 of a unit vector; index k = l(l+1)+m. */
void orc_sh_basis(const double *d, double *Y) {
    const double x = d[0], y = d[1], z = d[2];
    const double pi = 3.14159265358979323846;
    const double xx = x * x, yy = y * y, zz = z * z;
    Y[0] = 1.0 / (2.0 * sqrt(pi));
    const double c1 = sqrt(3.0) / (2.0 * sqrt(pi));
    Y[1] = -c1 * y; Y[2] = c1 * z; Y[3] = -c1 * x;
    const double a2 = sqrt(15.0) / (2.0 * sqrt(pi));
    const double b2 = sqrt(5.0) / (4.0 * sqrt(pi));
    const double c2 = sqrt(15.0) / (4.0 * sqrt(pi));
    Y[4] = a2 * x * y;
    Y[5] = -a2 * y * z;
    Y[6] = b2 * (2.0 * zz - xx - yy);
    Y[7] = -a2 * x * z;
    Y[8] = c2 * (xx - yy);
    const double e3 = sqrt(35.0 / (2.0 * pi)) / 4.0;
    const double f3 = sqrt(105.0) / (2.0 * sqrt(pi));
    const double g3 = sqrt(21.0 / (2.0 * pi)) / 4.0;
    const double h3 = sqrt(7.0) / (4.0 * sqrt(pi));
    const double k3 = sqrt(105.0) / (4.0 * sqrt(pi));
    Y[9]  = -e3 * y * (3.0 * xx - yy);
    Y[10] = f3 * x * y * z;
    Y[11] = -g3 * y * (4.0 * zz - xx - yy);
    Y[12] = h3 * z * (2.0 * zz - 3.0 * xx - 3.0 * yy);
    Y[13] = -g3 * x * (4.0 * zz - xx - yy);
    Y[14] = k3 * z * (xx - yy);
    Y[15] = -e3 * x * (xx - 3.0 * yy);
}

/* Camera origin o = -R^T t and unit world direction of pixel (x,y). */
static void cam_origin(const orc_camera *c, double *o) {
    const double *M = c->w2c;
    for (int j = 0; j < 3; ++j) o[j] = -(M[0 + j] * M[3] + M[4 + j] * M[7] + M[8 + j] * M[11]);
}
static void cam_ray_dir(const orc_camera *c, int x, int y, double *d) {
    const double *M = c->w2c;
    const double dc[3] = {(x + 0.5 - c->cx) / c->fx, (y + 0.5 - c->cy) / c->fy, 1.0};
    double w[3];
    for (int j = 0; j < 3; ++j) w[j] = M[0 + j] * dc[0] + M[4 + j] * dc[1] + M[8 + j] * dc[2];
    const double inv = 1.0 / sqrt(w[0] * w[0] + w[1] * w[1] + w[2] * w[2]);
    d[0] = w[0] * inv; d[1] = w[1] * inv; d[2] = w[2] * inv;
}
void orc_ray(const orc_camera *c, int x, int y, double *o, double *d) {
    cam_origin(c, o);
    cam_ray_dir(c, x, y, d);
}

/* ------------------------------------------------------------------ bounds (Eq. 9-14) */
/* Per Gaussian geometry in camera space. Returns class: 0 culled, 1 front, 2 straddle. */
typedef struct {
    int cls;
    double alpha_c;
    double Ac[9];  /* R_w2c R S alpha_c */
    double mu_c[3];
    double ez;
    double radius; /* alpha_c * max(s) */
    double cls_margin;
} gauss_geom;

static void gauss_geometry(const orc_scene *s, int64_t i, const orc_camera *cam, const orc_config *cfg, gauss_geom *g) {
    const double sigma = s->opacity[i];
    g->cls = 0; g->cls_margin = fabs(sigma - cfg->alpha_min);
    if (!(sigma > cfg->alpha_min)) return;
    g->alpha_c = pow(2.0 * log(sigma / cfg->alpha_min), 1.0 / kernel_degree_of(cfg));   /* Eq. 9-10 for exp(-D^k / 2) */
    double R[9];
    quat_to_R(s->quat + 4 * i, R);
    const double *sc = s->scale + 3 * i;
    const double *M = cam->w2c;
    double A[9];
    for (int r = 0; r < 3; ++r) for (int c = 0; c < 3; ++c) A[3 * r + c] = R[3 * r + c] * sc[c] * g->alpha_c;
    for (int r = 0; r < 3; ++r) for (int c = 0; c < 3; ++c)
        g->Ac[3 * r + c] = M[4 * r + 0] * A[0 + c] + M[4 * r + 1] * A[3 + c] + M[4 * r + 2] * A[6 + c];
    const double *mu = s->mean + 3 * i;
    for (int r = 0; r < 3; ++r) g->mu_c[r] = M[4 * r + 0] * mu[0] + M[4 * r + 1] * mu[1] + M[4 * r + 2] * mu[2] + M[4 * r + 3];
    g->ez = sqrt(g->Ac[6] * g->Ac[6] + g->Ac[7] * g->Ac[7] + g->Ac[8] * g->Ac[8]);
    double smax = sc[0] > sc[1] ? sc[0] : sc[1];
    if (sc[2] > smax) smax = sc[2];
    g->radius = g->alpha_c * smax;
    const double zfar = g->mu_c[2] + g->ez, znear = g->mu_c[2] - g->ez;
    double m = fabs(zfar - cfg->near_z);
    if (fabs(znear - cfg->near_z) < m) m = fabs(znear - cfg->near_z);
    if (g->cls_margin > m) g->cls_margin = m;
    if (zfar <= cfg->near_z) { g->cls = 0; return; }
    g->cls = (znear >= cfg->near_z) ? 1 : 2;
}

static double frac_margin(double v) { /* distance of v to the nearest integer */
    return fabs(v - nearbyint(v));
}

/*
 * Screen-space rectangles (inclusive pixel ranges x0..x1, y0..y1 of pixel centres)
 * for all Gaussians.  rect = (0,0,-1,-1) when no pixel is selected.
 * cls: 0 culled by rule, 1 front, 2 straddle.  margin[i]: smallest distance of any
 * decision of Gaussian i to its decision boundary (class tests in scene units,
 * rectangle edges in pixels); may be NULL.
 */
void orc_bounds(const orc_scene *s, const orc_camera *cam, const orc_config *cfg,
                int32_t *rect, uint8_t *cls, double *margin) {
    const int W = cam->width, H = cam->height;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < s->n; ++i) {
        gauss_geom g;
        gauss_geometry(s, i, cam, cfg, &g);
        int32_t *r = rect + 4 * i;
        r[0] = 0; r[1] = 0; r[2] = -1; r[3] = -1;
        cls[i] = (uint8_t)g.cls;
        double mg = g.cls_margin;
        if (g.cls == 1) {
            /* rows of T' in pixel units: x, y, w (Eq. 11) */
            double Tx[4], Ty[4], Tw[4];
            for (int c = 0; c < 3; ++c) {
                Tx[c] = cam->fx * g.Ac[0 + c] + cam->cx * g.Ac[6 + c];
                Ty[c] = cam->fy * g.Ac[3 + c] + cam->cy * g.Ac[6 + c];
                Tw[c] = g.Ac[6 + c];
            }
            Tx[3] = cam->fx * g.mu_c[0] + cam->cx * g.mu_c[2];
            Ty[3] = cam->fy * g.mu_c[1] + cam->cy * g.mu_c[2];
            Tw[3] = g.mu_c[2];
            const double v[4] = {1.0, 1.0, 1.0, -1.0};
            double sden = 0.0, px = 0.0, py = 0.0, qx = 0.0, qy = 0.0;
            for (int c = 0; c < 4; ++c) sden += v[c] * Tw[c] * Tw[c];        /* Eq. 13 */
            for (int c = 0; c < 4; ++c) {
                const double f = v[c] / sden;
                px += f * Tx[c] * Tw[c]; py += f * Ty[c] * Tw[c];            /* Eq. 14 */
                qx += f * Tx[c] * Tx[c]; qy += f * Ty[c] * Ty[c];
            }
            double hx2 = px * px - qx, hy2 = py * py - qy;
            const double hx = sqrt(hx2 > 0.0 ? hx2 : 0.0), hy = sqrt(hy2 > 0.0 ? hy2 : 0.0);
            const double lo_x = px - hx - 0.5, hi_x = px + hx - 0.5;          /* Eq. 12, pixel centres */
            const double lo_y = py - hy - 0.5, hi_y = py + hy - 0.5;
            double cx0 = ceil(lo_x), cx1 = floor(hi_x), cy0 = ceil(lo_y), cy1 = floor(hi_y);
            double e;
            e = frac_margin(lo_x); if (e < mg) mg = e;
            e = frac_margin(hi_x); if (e < mg) mg = e;
            e = frac_margin(lo_y); if (e < mg) mg = e;
            e = frac_margin(hi_y); if (e < mg) mg = e;
            if (cx0 < 0.0) cx0 = 0.0;
            if (cy0 < 0.0) cy0 = 0.0;
            if (cx1 > W - 1) cx1 = W - 1;
            if (cy1 > H - 1) cy1 = H - 1;
            if (cx1 >= cx0 && cy1 >= cy0) {
                r[0] = (int32_t)cx0; r[1] = (int32_t)cy0; r[2] = (int32_t)cx1; r[3] = (int32_t)cy1;
            }
        } else if (g.cls == 2) {
            /* bounding sphere against the four side planes through the camera origin */
            const double nrm[4][3] = {
                {cam->fx, 0.0, cam->cx}, {-cam->fx, 0.0, W - cam->cx},
                {0.0, cam->fy, cam->cy}, {0.0, -cam->fy, H - cam->cy}};
            int outside = 0;
            for (int p = 0; p < 4; ++p) {
                const double len = sqrt(nrm[p][0] * nrm[p][0] + nrm[p][1] * nrm[p][1] + nrm[p][2] * nrm[p][2]);
                const double dist = (nrm[p][0] * g.mu_c[0] + nrm[p][1] * g.mu_c[1] + nrm[p][2] * g.mu_c[2]) / len;
                if (dist < -g.radius) outside = 1;
                const double e = fabs(dist + g.radius);
                if (e < mg) mg = e;
            }
            if (!outside) { r[0] = 0; r[1] = 0; r[2] = W - 1; r[3] = H - 1; }
        }
        if (margin) margin[i] = mg;
    }
}

/* ------------------------------------------------------------------ tile map (Sec. 4.3) */
/*
 * Tile lists from rectangles: tile t = ty * tiles_x + tx lists, in ascending id,
 * every Gaussian whose rectangle overlaps it.  tile_off has tiles_x*tiles_y + 1
 * entries.  Call with pair_gid == NULL to obtain the number of pairs (return
 * value) and tile_off only.  *slots receives sum of rectangle areas (Eq. 15 with
 * lambda_s = 1, in entries).
 */
int64_t orc_tile_map(int64_t n, const int32_t *rect, int width, int height, int ts,
                     uint32_t *tile_off, uint32_t *pair_gid, int64_t *slots) {
    const int tiles_x = (width + ts - 1) / ts, tiles_y = (height + ts - 1) / ts;
    const int64_t T = (int64_t)tiles_x * tiles_y;
    int64_t *cnt = (int64_t *)calloc((size_t)T + 1, sizeof(int64_t));
    int64_t S = 0;
    for (int64_t i = 0; i < n; ++i) {
        const int32_t *r = rect + 4 * i;
        if (r[2] < r[0] || r[3] < r[1]) continue;
        S += (int64_t)(r[2] - r[0] + 1) * (r[3] - r[1] + 1);
        for (int ty = r[1] / ts; ty <= r[3] / ts; ++ty)
            for (int tx = r[0] / ts; tx <= r[2] / ts; ++tx) cnt[(int64_t)ty * tiles_x + tx]++;
    }
    int64_t run = 0;
    for (int64_t t = 0; t < T; ++t) { tile_off[t] = (uint32_t)run; run += cnt[t]; cnt[t] = tile_off[t]; }
    tile_off[T] = (uint32_t)run;
    if (slots) *slots = S;
    if (pair_gid) {
        for (int64_t i = 0; i < n; ++i) {
            const int32_t *r = rect + 4 * i;
            if (r[2] < r[0] || r[3] < r[1]) continue;
            for (int ty = r[1] / ts; ty <= r[3] / ts; ++ty)
                for (int tx = r[0] / ts; tx <= r[2] / ts; ++tx) pair_gid[cnt[(int64_t)ty * tiles_x + tx]++] = (uint32_t)i;
        }
    }
    free(cnt);
    return run;
}

/* ------------------------------------------------------------------ view: hits, compositing, backward */
typedef struct {
    orc_scene sc;
    orc_camera cam;
    orc_config cfg;
    int K;
    int64_t n_rays;
    uint64_t *ray_off; /* [n_rays + 1] */
    uint32_t *gid;     /* [H] */
    double *t;         /* [H] maximum-response distance */
    double *alpha;     /* [H] */
    double *T;         /* [H] transmittance before the hit (after composite) */
    double *Rs;        /* [H,3] colour composited behind the hit (after composite) */
    double *col;       /* [H,3] clamped colour of the hit */
    uint8_t *pos;      /* [H] bit c set if raw colour channel c > 0 */
    double *ae;        /* [H] alpha as composited: min(alpha, alpha_max) (after composite) */
    uint8_t *clamped;  /* [H] 1 where the clamp is active */
    double *kap;       /* [H] kappa_i = sum over the composited hits j in front of i of alpha_j / (1 - alpha_j) */
    double *Bk;        /* [H,3] conditioning of the colour behind the hit (see orc_view_lt_entries) */
    double *ray_margin; /* [n_rays, 2] the same two margins per ray */
    double margin_t, margin_a; /* smallest |ln(T_i / t_min)| and |ln(alpha / alpha_max)| met by composite (decision margins) */
    int composited;
} orc_view;

orc_view *orc_view_create(const orc_scene *s, const orc_camera *cam, const orc_config *cfg) {
    orc_view *v = (orc_view *)calloc(1, sizeof(orc_view));
    v->sc = *s; v->cam = *cam; v->cfg = *cfg;
    v->K = (s->sh_degree + 1) * (s->sh_degree + 1);
    v->n_rays = (int64_t)cam->width * cam->height;
    return v;
}
static void view_free_hits(orc_view *v) {
    free(v->ray_off); free(v->gid); free(v->t); free(v->alpha); free(v->T); free(v->Rs); free(v->col); free(v->pos);
    free(v->ae); free(v->clamped); free(v->kap); free(v->Bk); free(v->ray_margin);
    v->ray_margin = NULL;
    v->ray_off = NULL; v->gid = NULL; v->t = v->alpha = v->T = v->Rs = v->col = NULL; v->pos = NULL;
    v->ae = v->kap = v->Bk = NULL; v->clamped = NULL;
    v->composited = 0;
}
void orc_view_destroy(orc_view *v) {
    if (!v) return;
    view_free_hits(v);
    free(v);
}

/* W = S^-1 R^T and o_g = W (o - mu) for Gaussian i (Eq. 5). */
static void gauss_local(const orc_scene *s, int64_t i, const double *o, double *Wm, double *og) {
    double R[9];
    quat_to_R(s->quat + 4 * i, R);
    const double *sc = s->scale + 3 * i, *mu = s->mean + 3 * i;
    for (int k = 0; k < 3; ++k) for (int j = 0; j < 3; ++j) Wm[3 * k + j] = R[3 * j + k] / sc[k];
    const double p[3] = {o[0] - mu[0], o[1] - mu[1], o[2] - mu[2]};
    for (int k = 0; k < 3; ++k) og[k] = Wm[3 * k] * p[0] + Wm[3 * k + 1] * p[1] + Wm[3 * k + 2] * p[2];
}

/* Response of Gaussian (Wm, og, sigma) along unit direction d: t*, alpha, x_g (Eq. 4, 5, 8). */
static void ray_response(const double *Wm, const double *og, double sigma, const double *d, int kdeg,
                         double *tstar, double *alpha, double *xg) {
    double dg[3];
    for (int k = 0; k < 3; ++k) dg[k] = Wm[3 * k] * d[0] + Wm[3 * k + 1] * d[1] + Wm[3 * k + 2] * d[2];
    const double a = dg[0] * dg[0] + dg[1] * dg[1] + dg[2] * dg[2];
    const double b = og[0] * dg[0] + og[1] * dg[1] + og[2] * dg[2];
    const double ts = -b / a;
    double x[3];
    for (int k = 0; k < 3; ++k) x[k] = og[k] + ts * dg[k];
    const double D2 = x[0] * x[0] + x[1] * x[1] + x[2] * x[2];
    *tstar = ts;
    *alpha = sigma * exp(-0.5 * pow(D2, 0.5 * kdeg));   /* Eq. 4 at k = 2 */
    if (xg) { xg[0] = x[0]; xg[1] = x[1]; xg[2] = x[2]; }
}

/* alpha and t* of (ray, Gaussian) without any threshold; out = {alpha, t*}. */
void orc_view_eval_pair(const orc_view *v, int64_t ray, int64_t gid, double *out) {
    double o[3], d[3], Wm[9], og[3];
    cam_origin(&v->cam, o);
    cam_ray_dir(&v->cam, (int)(ray % v->cam.width), (int)(ray / v->cam.width), d);
    gauss_local(&v->sc, gid, o, Wm, og);
    ray_response(Wm, og, v->sc.opacity[gid], d, kernel_degree_of(&v->cfg), &out[1], &out[0], NULL);
}

/*
 * Candidate pixel range of Gaussian i.  mode 0: whole image (true brute force).
 * mode 1: bounding sphere (mu, alpha_c * max s) projected with the tangent-angle
 * form, padded by one pixel; whole image when the sphere reaches depth <= near.
 * Independent of the Eq. 11-14 rectangle.
 */
static void candidate_range(const orc_view *v, const gauss_geom *g, int mode, int *x0, int *y0, int *x1, int *y1) {
    const int W = v->cam.width, H = v->cam.height;
    *x0 = 0; *y0 = 0; *x1 = W - 1; *y1 = H - 1;
    if (mode == 0) return;
    const double X = g->mu_c[0], Y = g->mu_c[1], Z = g->mu_c[2], r = g->radius;
    if (Z - r <= v->cfg.near_z || Z - r <= 0.0) return;
    {
        const double th = atan2(X, Z), ph = asin(r / sqrt(X * X + Z * Z));
        const double lo = v->cam.fx * tan(th - ph) + v->cam.cx - 0.5, hi = v->cam.fx * tan(th + ph) + v->cam.cx - 0.5;
        const double a = floor(lo) - 1.0, b = ceil(hi) + 1.0;
        if (a > *x0) *x0 = a > W ? W : (int)a;
        if (b < *x1) *x1 = b < -1.0 ? -1 : (int)b;
    }
    {
        const double th = atan2(Y, Z), ph = asin(r / sqrt(Y * Y + Z * Z));
        const double lo = v->cam.fy * tan(th - ph) + v->cam.cy - 0.5, hi = v->cam.fy * tan(th + ph) + v->cam.cy - 0.5;
        const double a = floor(lo) - 1.0, b = ceil(hi) + 1.0;
        if (a > *y0) *y0 = a > H ? H : (int)a;
        if (b < *y1) *y1 = b < -1.0 ? -1 : (int)b;
    }
}

typedef struct { double t; uint32_t gid; double alpha; } hit_rec;
static int hit_cmp(const void *a, const void *b) {
    const hit_rec *p = (const hit_rec *)a, *q = (const hit_rec *)b;
    if (p->t < q->t) return -1;
    if (p->t > q->t) return 1;
    return (p->gid > q->gid) - (p->gid < q->gid);
}

/*
 * Find, for every requested ray, all hits (alpha >= alpha_min and t* > 0) among the
 * Gaussians not culled by rule, ordered by (t*, id).  pixel_mask (may be NULL)
 * selects rays: only pixels with a non-zero mask byte are processed.  mode as in
 * candidate_range.  Returns the number of hits.
 */
int64_t orc_view_find_hits(orc_view *v, int mode, const uint8_t *pixel_mask) {
    view_free_hits(v);
    const int W = v->cam.width;
    const int64_t NR = v->n_rays;
    double o[3];
    cam_origin(&v->cam, o);
    uint64_t *cnt = (uint64_t *)calloc((size_t)NR + 1, sizeof(uint64_t));
    /* per image row the span of requested pixels (hi < lo: none), so that a sparse request does not walk the whole image
     * for every Gaussian; the rays visited and what is computed for them are the same */
    const int Hh = v->cam.height;
    int *row_lo = (int *)malloc((size_t)Hh * sizeof(int)), *row_hi = (int *)malloc((size_t)Hh * sizeof(int));
    for (int y = 0; y < Hh; ++y) {
        row_lo[y] = 0; row_hi[y] = W - 1;
        if (pixel_mask) {
            int lo = W, hi = -1;
            for (int x = 0; x < W; ++x) if (pixel_mask[(int64_t)y * W + x]) { if (x < lo) lo = x; hi = x; }
            row_lo[y] = lo; row_hi[y] = hi;
        }
    }
    for (int pass = 0; pass < 2; ++pass) {
#pragma omp parallel for schedule(dynamic, 256)
        for (int64_t i = 0; i < v->sc.n; ++i) {
            gauss_geom g;
            gauss_geometry(&v->sc, i, &v->cam, &v->cfg, &g);
            if (g.cls == 0) continue;
            int x0, y0, x1, y1;
            candidate_range(v, &g, mode, &x0, &y0, &x1, &y1);
            if (x1 < x0 || y1 < y0) continue;
            double Wm[9], og[3];
            gauss_local(&v->sc, i, o, Wm, og);
            const double sigma = v->sc.opacity[i];
            for (int y = y0; y <= y1; ++y) for (int x = (x0 > row_lo[y] ? x0 : row_lo[y]); x <= (x1 < row_hi[y] ? x1 : row_hi[y]); ++x) {
                const int64_t ray = (int64_t)y * W + x;
                if (pixel_mask && !pixel_mask[ray]) continue;
                double d[3], ts, al;
                cam_ray_dir(&v->cam, x, y, d);
                ray_response(Wm, og, sigma, d, kernel_degree_of(&v->cfg), &ts, &al, NULL);
                if (!(al >= v->cfg.alpha_min && ts > 0.0)) continue;
                if (pass == 0) {
#pragma omp atomic
                    cnt[ray]++;
                } else {
                    uint64_t slot;
#pragma omp atomic capture
                    slot = cnt[ray]++;
                    v->gid[slot] = (uint32_t)i; v->t[slot] = ts; v->alpha[slot] = al;
                }
            }
        }
        if (pass == 0) {
            v->ray_off = (uint64_t *)malloc(((size_t)NR + 1) * sizeof(uint64_t));
            uint64_t run = 0;
            for (int64_t r = 0; r < NR; ++r) { v->ray_off[r] = run; run += cnt[r]; cnt[r] = v->ray_off[r]; }
            v->ray_off[NR] = run;
            v->gid = (uint32_t *)malloc((size_t)(run + 1) * sizeof(uint32_t));
            v->t = (double *)malloc((size_t)(run + 1) * sizeof(double));
            v->alpha = (double *)malloc((size_t)(run + 1) * sizeof(double));
        }
    }
    free(cnt); free(row_lo); free(row_hi);
    /* order every ray's hits by (t*, id) */
#pragma omp parallel
    {
        hit_rec *buf = NULL; size_t cap = 0;
#pragma omp for schedule(dynamic, 64)
        for (int64_t r = 0; r < NR; ++r) {
            const uint64_t b = v->ray_off[r], e = v->ray_off[r + 1];
            const size_t m = (size_t)(e - b);
            if (m < 2) continue;
            if (m > cap) { cap = 2 * m; buf = (hit_rec *)realloc(buf, cap * sizeof(hit_rec)); }
            for (size_t j = 0; j < m; ++j) { buf[j].t = v->t[b + j]; buf[j].gid = v->gid[b + j]; buf[j].alpha = v->alpha[b + j]; }
            qsort(buf, m, sizeof(hit_rec), hit_cmp);
            for (size_t j = 0; j < m; ++j) { v->t[b + j] = buf[j].t; v->gid[b + j] = buf[j].gid; v->alpha[b + j] = buf[j].alpha; }
        }
        free(buf);
    }
    return (int64_t)v->ray_off[NR];
}

/*
 * Impose hit lists (replay): ray r's hits are gid[ray_off[r] .. ray_off[r+1]) in the
 * given order; alpha and t* are evaluated for exactly those pairs, no threshold.
 */
void orc_view_set_hits(orc_view *v, const uint64_t *ray_off, const uint32_t *gid) {
    view_free_hits(v);
    const int64_t NR = v->n_rays;
    const uint64_t Hn = ray_off[NR];
    v->ray_off = (uint64_t *)malloc(((size_t)NR + 1) * sizeof(uint64_t));
    memcpy(v->ray_off, ray_off, ((size_t)NR + 1) * sizeof(uint64_t));
    v->gid = (uint32_t *)malloc((size_t)(Hn + 1) * sizeof(uint32_t));
    memcpy(v->gid, gid, (size_t)Hn * sizeof(uint32_t));
    v->t = (double *)malloc((size_t)(Hn + 1) * sizeof(double));
    v->alpha = (double *)malloc((size_t)(Hn + 1) * sizeof(double));
    double o[3];
    cam_origin(&v->cam, o);
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t r = 0; r < NR; ++r) {
        if (ray_off[r] == ray_off[r + 1]) continue;
        double d[3];
        cam_ray_dir(&v->cam, (int)(r % v->cam.width), (int)(r / v->cam.width), d);
        for (uint64_t h = ray_off[r]; h < ray_off[r + 1]; ++h) {
            double Wm[9], og[3];
            gauss_local(&v->sc, gid[h], o, Wm, og);
            ray_response(Wm, og, v->sc.opacity[gid[h]], d, kernel_degree_of(&v->cfg), &v->t[h], &v->alpha[h], NULL);
        }
    }
}

int64_t orc_view_num_hits(const orc_view *v) { return v->ray_off ? (int64_t)v->ray_off[v->n_rays] : 0; }

/* Copy out the hit lists; any pointer may be NULL. */
void orc_view_get_hits(const orc_view *v, uint64_t *ray_off, uint32_t *gid, double *t, double *alpha) {
    const uint64_t Hn = v->ray_off[v->n_rays];
    if (ray_off) memcpy(ray_off, v->ray_off, ((size_t)v->n_rays + 1) * sizeof(uint64_t));
    if (gid) memcpy(gid, v->gid, (size_t)Hn * sizeof(uint32_t));
    if (t) memcpy(t, v->t, (size_t)Hn * sizeof(double));
    if (alpha) memcpy(alpha, v->alpha, (size_t)Hn * sizeof(double));
}

/*
 * Front-to-back compositing (Eq. 6-8) of the current hit lists.
 * color [n_rays,3], t_final [n_rays], hit_count [n_rays] (any may be NULL).
 * Also keeps, per hit, T_i, the clamped colour and the colour composited behind
 * the hit (summed back to front), which the backward pass needs.
 * With a hit cap (cfg.max_hits > 0) the ray ends after its first max_hits hits: the hits behind keep their
 * place in the lists but get T_i = 0, so they add nothing to the colour, to T_final or to any gradient.
 * Early termination (cfg.t_min > 0) ends the ray the same way before the first hit with T_i < t_min; the clamp
 * (cfg.alpha_max < 1) composites min(alpha, alpha_max).
 * Also kept per hit, for the error analysis of single-precision evaluations: kappa_i, the sum of alpha_j / (1 - alpha_j)
 * over the composited hits in front (a relative error eps of every alpha_j moves ln T_i by at most eps kappa_i).
 */
void orc_view_composite(orc_view *v, double *color, double *t_final, uint32_t *hit_count) {
    const int64_t NR = v->n_rays;
    const uint64_t Hn = v->ray_off[NR];
    const int K = v->K;
    if (!v->T) {
        v->T = (double *)malloc((size_t)(Hn + 1) * sizeof(double));
        v->Rs = (double *)malloc((size_t)(Hn + 1) * 3 * sizeof(double));
        v->col = (double *)malloc((size_t)(Hn + 1) * 3 * sizeof(double));
        v->pos = (uint8_t *)malloc((size_t)(Hn + 1));
        v->ae = (double *)malloc((size_t)(Hn + 1) * sizeof(double));
        v->clamped = (uint8_t *)malloc((size_t)(Hn + 1));
        v->kap = (double *)malloc((size_t)(Hn + 1) * sizeof(double));
        v->Bk = (double *)malloc((size_t)(Hn + 1) * 3 * sizeof(double));
        v->ray_margin = (double *)malloc((size_t)(NR + 1) * 2 * sizeof(double));
    }
    const double t_min = v->cfg.t_min, a_max = v->cfg.alpha_max;
    double margin_t = INFINITY, margin_a = INFINITY;
#pragma omp parallel for schedule(dynamic, 64) reduction(min : margin_t, margin_a)
    for (int64_t r = 0; r < NR; ++r) {
        const uint64_t b = v->ray_off[r], e = v->ray_off[r + 1];
        double C[3] = {0, 0, 0}, T = 1.0, kappa = 0.0, rm_t = INFINITY, rm_a = INFINITY;
        int ended = 0;
        if (e > b) {
            double d[3], Y[ORC_MAX_K];
            cam_ray_dir(&v->cam, (int)(r % v->cam.width), (int)(r / v->cam.width), d);
            orc_sh_basis(d, Y);
            for (uint64_t h = b; h < e; ++h) {
                const double *sh = v->sc.sh + (size_t)v->gid[h] * K * 3;
                if (!ended && t_min > 0.0) {
                    if (fabs(log(T / t_min)) < rm_t) rm_t = fabs(log(T / t_min));
                    if (T < t_min) ended = 1;
                }
                const int capped = ended || (v->cfg.max_hits > 0 && h - b >= (uint64_t)v->cfg.max_hits);
                const double al = v->alpha[h] > a_max ? a_max : v->alpha[h];
                v->ae[h] = al;
                v->clamped[h] = v->alpha[h] > a_max;
                if (a_max < 1.0 && !capped && fabs(log(v->alpha[h] / a_max)) < rm_a) rm_a = fabs(log(v->alpha[h] / a_max));
                uint8_t pm = 0;
                for (int c = 0; c < 3; ++c) {
                    double raw = 0.5;
                    for (int k = 0; k < K; ++k) raw += Y[k] * sh[3 * k + c];
                    if (raw > 0.0) pm |= (uint8_t)(1u << c);
                    v->col[3 * h + c] = raw > 0.0 ? raw : 0.0;
                    if (!capped) C[c] += T * al * v->col[3 * h + c];
                }
                v->pos[h] = pm;
                v->T[h] = capped ? 0.0 : T;
                v->kap[h] = kappa;
                if (!capped) { T *= (1.0 - al); kappa += al / (1.0 - al); }
            }
        }
        double Rb[3] = {T * v->cfg.bg[0], T * v->cfg.bg[1], T * v->cfg.bg[2]};
        double Bk[3] = {kappa * fabs(Rb[0]), kappa * fabs(Rb[1]), kappa * fabs(Rb[2])};
        for (int c = 0; c < 3; ++c) C[c] += Rb[c];
        for (uint64_t h = e; h-- > b;) {
            const int capped = v->T[h] == 0.0;   /* (not composited: behind a cap or behind the end of the ray) */
            for (int c = 0; c < 3; ++c) {
                v->Rs[3 * h + c] = capped ? 0.0 : Rb[c];   /* nothing lies behind a hit that is not composited */
                v->Bk[3 * h + c] = capped ? 0.0 : Bk[c];
                Rb[c] += v->T[h] * v->ae[h] * v->col[3 * h + c];
                Bk[c] += (1.0 + v->kap[h]) * v->T[h] * v->ae[h] * v->col[3 * h + c];
            }
        }
        if (color) { color[3 * r] = C[0]; color[3 * r + 1] = C[1]; color[3 * r + 2] = C[2]; }
        if (t_final) t_final[r] = T;
        if (hit_count) hit_count[r] = (uint32_t)(e - b);
        v->ray_margin[2 * r] = rm_t; v->ray_margin[2 * r + 1] = rm_a;
        if (rm_t < margin_t) margin_t = rm_t;
        if (rm_a < margin_a) margin_a = rm_a;
    }
    v->margin_t = margin_t; v->margin_a = margin_a;
    v->composited = 1;
}

/* Smallest margins of the two floating-point decisions that the options add: out[0] = min |ln(T_i / t_min)| over the
 * termination tests made, out[1] = min |ln(alpha / alpha_max)| over the composited hits (infinity where an option is off). */
void orc_view_margins(const orc_view *v, double *out) { out[0] = v->margin_t; out[1] = v->margin_a; }

/* The same two margins for every ray: out [n_rays, 2] (infinity where the ray met no such decision). */
int orc_view_ray_margins(const orc_view *v, double *out) {
    if (!v->composited) return 1;
    memcpy(out, v->ray_margin, (size_t)v->cam.width * v->cam.height * 2 * sizeof(double));
    return 0;
}

/*
 * What the compact intermediate buffer (Sec. 4.3-4.4) has to hold per hit for the primitive-centric
 * backward, in the reading where the forward stores the derivative of the pixel colour instead of
 * (T, alpha, colour): from Eq. 6-8, with c the clamped colour of hit i, w = T_i alpha_i and B the colour
 * composited behind the hit (background included),
 *     alpha_i dC/dalpha_i = w c - alpha_i / (1 - alpha_i) B.
 * entry [H,4] receives that vector and w; flags [H] bit ch is set where colour channel ch is not
 * clamped (its SH gradient is w g_ch Y_k, zero otherwise).  Hit order = the view's lists.
 * Where the alpha clamp is active alpha_i is a constant: the vector part, which only ever multiplies the derivative
 * of alpha_i with respect to a parameter, is zero by definition; w = T_i alpha_max.
 * cond [H,4] (may be NULL): how far a relative error eps of every alpha on the ray (what single precision leaves of
 * alpha = sigma exp(-D^2 / 2)) can move each word, to first order, divided by eps.  With a_j = alpha_j / (1 - alpha_j)
 * and kappa_i = sum of a_j over the composited hits in front: T_i moves by kappa_i eps (relative), w_i by
 * (1 + kappa_i) eps, alpha_i / (1 - alpha_i) by (1 + a_i) eps, and B, a sum of w_j c_j behind and T_final bg, by
 * sum (1 + kappa_j) w_j c_j + kappa_end T_final |bg| =: Bk.  Hence
 *     cond[3] = (1 + kappa_i) w,   cond[c] = (1 + kappa_i) |w c_c| + alpha / (1 - alpha) ((1 + a_i) |B_c| + Bk_c).
 * Returns 0, or -1 if the view was not composited.
 */
int orc_view_lt_entries(const orc_view *v, double *entry, uint8_t *flags, double *cond) {
    if (!v->composited) return -1;
    const uint64_t Hn = v->ray_off[v->n_rays];
    for (uint64_t h = 0; h < Hn; ++h) {
        const double al = v->ae[h], w = v->T[h] * al, r = al / (1.0 - al);
        for (int c = 0; c < 3; ++c) {
            entry[4 * h + c] = v->clamped[h] ? 0.0 : w * v->col[3 * h + c] - r * v->Rs[3 * h + c];
            if (cond) cond[4 * h + c] = v->clamped[h] ? 0.0 : (1.0 + v->kap[h]) * fabs(w * v->col[3 * h + c])
                                                               + r * ((1.0 + r) * fabs(v->Rs[3 * h + c]) + v->Bk[3 * h + c]);
        }
        entry[4 * h + 3] = w;
        if (cond) cond[4 * h + 3] = (1.0 + v->kap[h]) * w;
        if (flags) flags[h] = v->pos[h];
    }
    return 0;
}

/*
 * Analytic backward of L = sum_rays <g_ray, C_ray> for the current (composited) hit lists.
 * dL_dC [n_rays,3].  grad [n, 11+3K] doubles: d mean(3), d scale(3), d quat(4), d opacity(1),
 * d sh(K*3, coefficient-major); fully overwritten.  grad_abs (may be NULL) receives, in
 * the same layout, the sum of absolute values of the per-hit contributions (the
 * conditioning of each sum).  grad_abs_elem (may be NULL) is the same with every hit's
 * contribution split further into its three colour channels: words 0..10 are linear in
 * alpha dL/dalpha = sum_c g_c (T alpha col_c - alpha Rs_c / (1 - alpha)), and the scale takes
 * sum_c |g_c (...)_c| in its place.  It bounds what a relative perturbation of the four
 * per-hit quantities (those three terms and T alpha) can do to a gradient word.
 * grad_abs_terms (may be NULL) splits once more: each channel's term is itself the difference of T alpha col_c and
 * alpha Rs_c / (1 - alpha), which nearly cancel where a hit has the colour of what lies behind it, and the scale
 * takes the sum of the two magnitudes: the mass of the products that any evaluation of Eq. 6-8 has to form.
 * grad_cond (may be NULL): per gradient word, how far a relative error eps of every alpha (single-precision
 * evaluation) can move it through the transmittances, divided by eps: the sum over the word's hits of the hit's
 * sensitivity to its entry times the entry's conditioning `cond` of orc_view_lt_entries.  A hit behind nearly opaque
 * ones (kappa in the hundreds) carries that factor however the sums are ordered.
 * Returns 0, or -1 if the view was not composited.
 */
int orc_view_backward(orc_view *v, const double *dL_dC, double *grad, double *grad_abs, double *grad_abs_elem,
                      double *grad_abs_terms, double *grad_cond) {
    if (!v->composited) return -1;
    const int K = v->K, G = 11 + 3 * K;
    const int64_t NR = v->n_rays;
    memset(grad, 0, (size_t)v->sc.n * G * sizeof(double));
    if (grad_abs) memset(grad_abs, 0, (size_t)v->sc.n * G * sizeof(double));
    if (grad_abs_elem) memset(grad_abs_elem, 0, (size_t)v->sc.n * G * sizeof(double));
    if (grad_abs_terms) memset(grad_abs_terms, 0, (size_t)v->sc.n * G * sizeof(double));
    if (grad_cond) memset(grad_cond, 0, (size_t)v->sc.n * G * sizeof(double));
    double o[3];
    cam_origin(&v->cam, o);
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t r = 0; r < NR; ++r) {
        const uint64_t b = v->ray_off[r], e = v->ray_off[r + 1];
        if (e == b) continue;
        double d[3], Y[ORC_MAX_K];
        cam_ray_dir(&v->cam, (int)(r % v->cam.width), (int)(r / v->cam.width), d);
        orc_sh_basis(d, Y);
        const double *g = dL_dC + 3 * r;
        for (uint64_t h = b; h < e; ++h) {
            const int64_t i = v->gid[h];
            const double al = v->ae[h], T = v->T[h];
            double contrib[11 + 3 * ORC_MAX_K];
            /* colour -> SH */
            for (int k = 0; k < K; ++k) for (int c = 0; c < 3; ++c)
                contrib[11 + 3 * k + c] = ((v->pos[h] >> c) & 1) ? Y[k] * T * al * g[c] : 0.0;
            /* alpha */
            double dalpha = 0.0, dalpha_abs = 0.0, dalpha_terms = 0.0, dalpha_cond = 0.0;
            for (int c = 0; c < 3 && !v->clamped[h]; ++c) {   /* (a clamped alpha is a constant: no gradient through it) */
                const double term = g[c] * (T * v->col[3 * h + c] - v->Rs[3 * h + c] / (1.0 - al));
                dalpha += term;
                dalpha_abs += fabs(term);
                dalpha_terms += fabs(g[c]) * (fabs(T * v->col[3 * h + c]) + fabs(v->Rs[3 * h + c] / (1.0 - al)));
                /* conditioning of alpha dL/dalpha = sum_c g_c entry_c, per unit of alpha (see orc_view_lt_entries) */
                dalpha_cond += fabs(g[c]) * ((1.0 + v->kap[h]) * fabs(T * v->col[3 * h + c])
                                             + ((1.0 + al / (1.0 - al)) * fabs(v->Rs[3 * h + c]) + v->Bk[3 * h + c]) / (1.0 - al));
            }
            const double sigma = v->sc.opacity[i];
            const double rho = al / sigma;
            contrib[10] = dalpha * rho;
            /* geometry */
            double Wm[9], og[3], ts, a2, xg[3];
            gauss_local(&v->sc, i, o, Wm, og);
            const int kdeg = kernel_degree_of(&v->cfg);
            ray_response(Wm, og, sigma, d, kdeg, &ts, &a2, xg);
            /* dL / d(D^2) with alpha = sigma exp(-(D^2)^(k/2) / 2): d alpha / d(D^2) = -alpha (k/4) (D^2)^(k/2 - 1), i.e.
             * -alpha / 2 at k = 2; d(D^2)/dt* = 0 at the maximum */
            const double D2 = xg[0] * xg[0] + xg[1] * xg[1] + xg[2] * xg[2];
            const double Gd = -0.25 * kdeg * pow(D2, 0.5 * kdeg - 1.0) * al * dalpha;
            const double *mu = v->sc.mean + 3 * i, *sc = v->sc.scale + 3 * i, *q = v->sc.quat + 4 * i;
            const double xw[3] = {o[0] + ts * d[0] - mu[0], o[1] + ts * d[1] - mu[1], o[2] + ts * d[2] - mu[2]};
            for (int j = 0; j < 3; ++j)
                contrib[j] = -2.0 * Gd * (Wm[0 + j] * xg[0] + Wm[3 + j] * xg[1] + Wm[6 + j] * xg[2]);
            for (int k = 0; k < 3; ++k) contrib[3 + k] = -2.0 * Gd * xg[k] * xg[k] / sc[k];
            double dR[9];
            for (int j = 0; j < 3; ++j) for (int k = 0; k < 3; ++k) dR[3 * j + k] = 2.0 * Gd * xw[j] * xg[k] / sc[k];
            const double w = q[0], x = q[1], y = q[2], z = q[3];
            /* chain rule through the polynomial rotation formula */
            contrib[6] = 2.0 * (-z * dR[1] + y * dR[2] + z * dR[3] - x * dR[5] - y * dR[6] + x * dR[7]);
            contrib[7] = 2.0 * (y * dR[1] + z * dR[2] + y * dR[3] - 2.0 * x * dR[4] - w * dR[5] + z * dR[6] + w * dR[7] - 2.0 * x * dR[8]);
            contrib[8] = 2.0 * (-2.0 * y * dR[0] + x * dR[1] + w * dR[2] + x * dR[3] + z * dR[5] - w * dR[6] + z * dR[7] - 2.0 * y * dR[8]);
            contrib[9] = 2.0 * (-2.0 * z * dR[0] - w * dR[1] + x * dR[2] + w * dR[3] - 2.0 * z * dR[4] + y * dR[5] + x * dR[6] + y * dR[7]);
            double *gi = grad + (size_t)i * G;
            for (int k = 0; k < G; ++k) {
                if (contrib[k] != 0.0) {
#pragma omp atomic
                    gi[k] += contrib[k];
                }
            }
            if (grad_abs) {
                double *ga = grad_abs + (size_t)i * G;
                for (int k = 0; k < G; ++k) {
                    if (contrib[k] != 0.0) {
#pragma omp atomic
                        ga[k] += fabs(contrib[k]);
                    }
                }
            }
            if (grad_abs_terms) {
                double *gt = grad_abs_terms + (size_t)i * G;
                const double split = dalpha != 0.0 ? dalpha_terms / fabs(dalpha) : 0.0;   /* >= 1 */
                for (int k = 0; k < G; ++k) {
                    if (contrib[k] != 0.0) {
                        const double a = fabs(contrib[k]) * (k < 11 ? split : 1.0);
#pragma omp atomic
                        gt[k] += a;
                    }
                }
            }
            if (grad_cond) {
                double *gc = grad_cond + (size_t)i * G;
                const double split = dalpha != 0.0 ? dalpha_cond / fabs(dalpha) : 0.0;
                for (int k = 0; k < G; ++k) {
                    if (contrib[k] != 0.0) {
                        const double a = fabs(contrib[k]) * (k < 11 ? split : 1.0 + v->kap[h]);
#pragma omp atomic
                        gc[k] += a;
                    }
                }
            }
            if (grad_abs_elem) {
                double *ge = grad_abs_elem + (size_t)i * G;
                const double split = dalpha != 0.0 ? dalpha_abs / fabs(dalpha) : 0.0;   /* >= 1 */
                for (int k = 0; k < G; ++k) {
                    if (contrib[k] != 0.0) {
                        const double a = fabs(contrib[k]) * (k < 11 ? split : 1.0);
#pragma omp atomic
                        ge[k] += a;
                    }
                }
            }
        }
    }
    return 0;
}
