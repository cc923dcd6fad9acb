/*
 * flashbev_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of the Sampling-VT operator (paper Eq. 1,
 * Sec. 3.1) evaluated in the loop order of the fused algorithm (Algorithm 2):
 * for every BEV cell, for every height bin z, for every camera n: voxel centre
 * -> projection -> validity mask M_n -> bilinear sample f_n -> per-z camera
 * reduction -> sum over z.  Nothing here is blocked, fused, vectorised or
 * reordered beyond that; the only concession to run time is an OpenMP
 * "parallel for" over BEV cells, which Sec. 3.2.2 states are independent.
 *
 * Only the tests, the smoke check and the bench's CPU-baseline leg may call
 * this file.  It shares no source, header, table or helper with the CUDA
 * library and neither includes the other.
 *
 * Conventions (each one is a reading of the paper or of the operator's
 * interface statement; they are listed with their justification in the design
 * notes):
 *   - voxel centres are BIN centres on all three axes:
 *       x_w = x_min + (ix + 1/2) (x_max - x_min) / X        (Sec. 4.1: [-50,50] m
 *       at 0.5 m <-> X = 200, [-5,5] m at 1.25 m <-> Z = 8: bins, not linspace)
 *   - the 4x4 matrix maps homogeneous metres to (u d, v d, d) in full-resolution
 *     image pixels; only rows 0..2 are read
 *   - M_n = 1 iff d > 0.1 and the sample lies strictly inside the feature map
 *     under grid_sample(align_corners=False) conventions:
 *       fx = u Wf / Wimg - 1/2,  fy = v Hf / Himg - 1/2,
 *       -1/2 < fx < Wf - 1/2,   -1/2 < fy < Hf - 1/2
 *   - f_n is bilinear interpolation with zero padding: a tap outside
 *     [0,Wf-1] x [0,Hf-1] contributes 0, the sample still counts in den_z
 *   - reduce = 0 (SUM):                out = sum_z sum_n M f
 *     reduce = 1 (MEAN_OVER_VALID):    out = (sum_z sum_n M f) / max(1, sum_z sum_n M)
 *     reduce = 2 (CAMERA_MEAN_Z_SUM):  out = sum_z [ sum_n M f / max(1, sum_n M) ]   (Eq. 1)
 *
 * Parity pins (tests/, CPU only): constant and affine feature maps (closed
 * forms), camera permutation, linearity, z-split additivity, grid-subset
 * invariance, a hand-computed one-sample case, an orthographic special case
 * against a library bilinear resampler, the Alg. 1 (tensorised) order written
 * independently in numpy, and the identities that tie the three reduce modes
 * together.  Which normalisation the interface's "mean_over_valid" means is a
 * reading, not something the paper fixes: for reduce = 1 parity is pinned to
 * that reading only ("parity unpinned" with respect to the paper).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_DEPTH_MIN 0.1    /* metres; interface statement: camera depth > 0.1 m */
#define ORACLE_BORDER_EPS 1e-3  /* feature px (image borders) / metres (depth plane) */

int flashbev_oracle_version(void) { return 1; }

int flashbev_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * features  : host, float32 [B][N][Hf][Wf][C]  (bf16 workloads pass the bf16-rounded
 *             values, which are exact in float32; everything is widened to double)
 * lidar2img : host, float32 [B][N][4][4] row-major
 * out       : host, double  [B][X][Y][C]
 * count     : host, int32   [B][X][Y]   sum over z,n of M_n                 (may be NULL)
 * flagged   : host, int32   [B][X][Y]   samples within ORACLE_BORDER_EPS of a
 *                                        validity border                    (may be NULL)
 * sumw      : host, double  [B][X][Y]   sum over valid samples of the in-bounds
 *                                        bilinear weight mass               (may be NULL)
 * interior  : host, uint8   [B][X][Y]   1 iff every valid sample has all four taps
 *                                        inside the map                     (may be NULL)
 * nzbins    : host, int32   [B][X][Y]   number of z bins with den_z > 0     (may be NULL)
 * nthreads  : OpenMP threads over cells (<= 0: library default)
 * returns 0, or -1 on a bad argument, -2 if out of memory.
 */
int flashbev_oracle_sampling_vt(const float *features, const float *lidar2img,
                                int B, int N, int C, int Hf, int Wf, int Himg, int Wimg,
                                double x_min, double x_max, double y_min, double y_max,
                                double z_min, double z_max, int X, int Y, int Z, int reduce,
                                double *out, int32_t *count, int32_t *flagged, double *sumw,
                                uint8_t *interior, int32_t *nzbins, int nthreads)
{
    if (!features || !lidar2img || !out) return -1;
    if (B <= 0 || N <= 0 || C <= 0 || Hf <= 0 || Wf <= 0 || Himg <= 0 || Wimg <= 0) return -1;
    if (X <= 0 || Y <= 0 || Z <= 0 || reduce < 0 || reduce > 2) return -1;
    if (!(x_max > x_min) || !(y_max > y_min) || !(z_max > z_min)) return -1;

    const double sx = (double)Wf / (double)Wimg; /* image px -> feature px */
    const double sy = (double)Hf / (double)Himg;
    const long long cells = (long long)B * X * Y;
    int oom = 0;
#ifdef _OPENMP
    if (nthreads <= 0) nthreads = omp_get_max_threads();
#else
    nthreads = 1;
#endif

#pragma omp parallel num_threads(nthreads)
    {
        double *acc = (double *)malloc(sizeof(double) * (size_t)C);
        double *num = (double *)malloc(sizeof(double) * (size_t)C);
        if (!acc || !num) {
#pragma omp atomic write
            oom = 1;
        }
#pragma omp barrier
        if (!oom) {
#pragma omp for schedule(dynamic, 16)
            for (long long cell = 0; cell < cells; ++cell) {
                const int b = (int)(cell / ((long long)X * Y));
                const int ix = (int)((cell / Y) % X);
                const int iy = (int)(cell % Y);
                /* voxel centre (Alg. 2 "compute voxel center"): bin centres */
                const double xw = x_min + ((double)ix + 0.5) * (x_max - x_min) / (double)X;
                const double yw = y_min + ((double)iy + 0.5) * (y_max - y_min) / (double)Y;

                for (int c = 0; c < C; ++c) acc[c] = 0.0;
                int32_t cnt = 0, flg = 0, nzb = 0;
                double sw = 0.0;
                int inter = 1;

                for (int k = 0; k < Z; ++k) { /* z outer, n inner: Alg. 2 */
                    const double zw = z_min + ((double)k + 0.5) * (z_max - z_min) / (double)Z;
                    for (int c = 0; c < C; ++c) num[c] = 0.0;
                    int den = 0;

                    for (int n = 0; n < N; ++n) {
                        const float *M = lidar2img + ((size_t)b * N + n) * 16;
                        /* projection: rows 0..2 of M times (x_w, y_w, z_w, 1) */
                        const double p0 = (double)M[0] * xw + (double)M[1] * yw + (double)M[2] * zw + (double)M[3];
                        const double p1 = (double)M[4] * xw + (double)M[5] * yw + (double)M[6] * zw + (double)M[7];
                        const double d = (double)M[8] * xw + (double)M[9] * yw + (double)M[10] * zw + (double)M[11];

                        /* M_n, first half: positive depth (also rejects NaN) */
                        const int in_front = (d > ORACLE_DEPTH_MIN);
                        if (!in_front && !(d > ORACLE_DEPTH_MIN - ORACLE_BORDER_EPS)) continue;
                        /* here d > 0.099, so the perspective division is well defined */

                        const double u = p0 / d; /* image pixels */
                        const double v = p1 / d;
                        const double fx = u * sx - 0.5; /* feature pixels, align_corners=False */
                        const double fy = v * sy - 0.5;

                        /* signed distances to the four image borders (feature px) and to
                           the depth plane (m); the smallest one decides validity */
                        const double mx0 = fx + 0.5, mx1 = ((double)Wf - 0.5) - fx;
                        const double my0 = fy + 0.5, my1 = ((double)Hf - 0.5) - fy;
                        const double md = d - ORACLE_DEPTH_MIN;
                        const int in_img = (mx0 > 0.0) && (mx1 > 0.0) && (my0 > 0.0) && (my1 > 0.0);
                        if (isfinite(fx) && isfinite(fy)) {
                            double m = md;
                            if (mx0 < m) m = mx0;
                            if (mx1 < m) m = mx1;
                            if (my0 < m) m = my0;
                            if (my1 < m) m = my1;
                            /* border sample: its validity may legitimately differ between
                               two correct implementations; reported, excluded from parity */
                            if (fabs(m) < ORACLE_BORDER_EPS) flg += 1;
                        }
                        if (!in_front || !in_img) continue; /* M_n = 0 */

                        /* bilinear sample f_n with zero padding */
                        const double x0f = floor(fx), y0f = floor(fy);
                        const int x0 = (int)x0f, y0 = (int)y0f;
                        const double tx = fx - x0f, ty = fy - y0f;
                        const float *Fn = features + ((size_t)b * N + n) * (size_t)Hf * Wf * C;
                        double wsum = 0.0;
                        int all_in = 1;
                        for (int dy = 0; dy < 2; ++dy) {
                            for (int dx = 0; dx < 2; ++dx) {
                                const int xi = x0 + dx, yi = y0 + dy;
                                const double w = (dx ? tx : 1.0 - tx) * (dy ? ty : 1.0 - ty);
                                if (xi < 0 || xi > Wf - 1 || yi < 0 || yi > Hf - 1) {
                                    all_in = 0;
                                    continue;
                                }
                                const float *t = Fn + ((size_t)yi * Wf + xi) * C;
                                for (int c = 0; c < C; ++c) num[c] += w * (double)t[c];
                                wsum += w;
                            }
                        }
                        den += 1;
                        sw += wsum;
                        if (!all_in) inter = 0;
                    }

                    cnt += den;
                    if (den > 0) nzb += 1;
                    if (reduce == 2) {
                        const double dz = (double)(den > 1 ? den : 1); /* g_z = num_z / max(1, den_z) */
                        for (int c = 0; c < C; ++c) acc[c] += num[c] / dz;
                    } else {
                        for (int c = 0; c < C; ++c) acc[c] += num[c];
                    }
                }

                double *o = out + (size_t)cell * C;
                if (reduce == 1) {
                    const double dn = (double)(cnt > 1 ? cnt : 1);
                    for (int c = 0; c < C; ++c) o[c] = acc[c] / dn;
                } else {
                    for (int c = 0; c < C; ++c) o[c] = acc[c];
                }
                if (count) count[cell] = cnt;
                if (flagged) flagged[cell] = flg;
                if (sumw) sumw[cell] = sw;
                if (interior) interior[cell] = (uint8_t)inter;
                if (nzbins) nzbins[cell] = nzb;
            }
        }
        free(acc);
        free(num);
    }
    return oom ? -2 : 0;
}


/* ------------------------------------------------------------------------------------------
 * Backward of the operator with respect to the features (the paper reports it in Tables 2 and 4
 * but prints no algorithm).  The forward map is linear in the features -- masks and weights do
 * not depend on them -- so its gradient is the transpose of that linear map, written out:
 *
 *   grad_features[b,n,yt,xt,c] = sum over cells, z and taps landing on (yt,xt) of
 *                                coeff(cell,z) * w_tap * grad_out[b,ix,iy,c]
 *   coeff = 1                                   (SUM)
 *         = 1 / max(1, sum_z sum_n M_n)         (MEAN_OVER_VALID; the whole cell's count)
 *         = 1 / max(1, sum_n M_n(z))            (CAMERA_MEAN_Z_SUM, Eq. 1)
 *
 * Plain loops in fp64; OpenMP over the (b, n) camera maps, each of which is written by one thread
 * only (every thread re-derives the validity of all cameras for the normalisations).
 * Pinned in tests by the adjoint identity <forward(F), G> = <F, backward(G)> against the forward
 * oracle above, by a hand-computed sample and by structural checks.
 */
static int oracle_project(const float *M, double xw, double yw, double zw, double sx, double sy, int Hf, int Wf,
                          double *fx, double *fy)
{
    const double p0 = (double)M[0] * xw + (double)M[1] * yw + (double)M[2] * zw + (double)M[3];
    const double p1 = (double)M[4] * xw + (double)M[5] * yw + (double)M[6] * zw + (double)M[7];
    const double d = (double)M[8] * xw + (double)M[9] * yw + (double)M[10] * zw + (double)M[11];
    if (!(d > ORACLE_DEPTH_MIN)) return 0;
    *fx = (p0 / d) * sx - 0.5;
    *fy = (p1 / d) * sy - 0.5;
    return (*fx > -0.5) && (*fx < (double)Wf - 0.5) && (*fy > -0.5) && (*fy < (double)Hf - 0.5);
}

/*
 * grad_out      : host, double [B][X][Y][C]
 * grad_features : host, double [B][N][Hf][Wf][C]   (overwritten)
 * returns 0, or -1 on a bad argument.
 */
int flashbev_oracle_sampling_vt_backward(const double *grad_out, const float *lidar2img, int B, int N, int C, int Hf,
                                         int Wf, int Himg, int Wimg, double x_min, double x_max, double y_min,
                                         double y_max, double z_min, double z_max, int X, int Y, int Z, int reduce,
                                         double *grad_features, int nthreads)
{
    if (!grad_out || !lidar2img || !grad_features) return -1;
    if (B <= 0 || N <= 0 || C <= 0 || Hf <= 0 || Wf <= 0 || Himg <= 0 || Wimg <= 0) return -1;
    if (X <= 0 || Y <= 0 || Z <= 0 || reduce < 0 || reduce > 2) return -1;
    if (!(x_max > x_min) || !(y_max > y_min) || !(z_max > z_min)) return -1;
    const double sx = (double)Wf / (double)Wimg, sy = (double)Hf / (double)Himg;
#ifdef _OPENMP
    if (nthreads <= 0) nthreads = omp_get_max_threads();
#else
    nthreads = 1;
#endif
#pragma omp parallel for schedule(dynamic, 1) num_threads(nthreads)
    for (int bn = 0; bn < B * N; ++bn) {
        const int b = bn / N, n = bn % N;
        double *Gn = grad_features + (size_t)bn * Hf * Wf * C;
        for (size_t i = 0; i < (size_t)Hf * Wf * C; ++i) Gn[i] = 0.0;
        const float *Mb = lidar2img + (size_t)b * N * 16;
        for (int ix = 0; ix < X; ++ix) {
            for (int iy = 0; iy < Y; ++iy) {
                const double xw = x_min + ((double)ix + 0.5) * (x_max - x_min) / (double)X;
                const double yw = y_min + ((double)iy + 0.5) * (y_max - y_min) / (double)Y;
                const double *go = grad_out + (((size_t)b * X + ix) * Y + iy) * C;
                int count = 0; /* valid samples of the whole cell (MEAN_OVER_VALID) */
                if (reduce == 1) {
                    for (int k = 0; k < Z; ++k) {
                        const double zw = z_min + ((double)k + 0.5) * (z_max - z_min) / (double)Z;
                        for (int m = 0; m < N; ++m) {
                            double fx, fy;
                            count += oracle_project(Mb + m * 16, xw, yw, zw, sx, sy, Hf, Wf, &fx, &fy);
                        }
                    }
                }
                for (int k = 0; k < Z; ++k) {
                    const double zw = z_min + ((double)k + 0.5) * (z_max - z_min) / (double)Z;
                    double fx, fy;
                    if (!oracle_project(Mb + n * 16, xw, yw, zw, sx, sy, Hf, Wf, &fx, &fy)) continue;
                    double coeff = 1.0;
                    if (reduce == 1) {
                        coeff = 1.0 / (double)(count > 1 ? count : 1);
                    } else if (reduce == 2) {
                        int den = 0; /* cameras that see this height bin */
                        for (int m = 0; m < N; ++m) {
                            double gx, gy;
                            den += oracle_project(Mb + m * 16, xw, yw, zw, sx, sy, Hf, Wf, &gx, &gy);
                        }
                        coeff = 1.0 / (double)(den > 1 ? den : 1);
                    }
                    const double x0f = floor(fx), y0f = floor(fy);
                    const int x0 = (int)x0f, y0 = (int)y0f;
                    const double tx = fx - x0f, ty = fy - y0f;
                    for (int dy = 0; dy < 2; ++dy) {
                        for (int dx = 0; dx < 2; ++dx) {
                            const int xi = x0 + dx, yi = y0 + dy;
                            if (xi < 0 || xi > Wf - 1 || yi < 0 || yi > Hf - 1) continue; /* zero padding */
                            const double w = coeff * (dx ? tx : 1.0 - tx) * (dy ? ty : 1.0 - ty);
                            double *t = Gn + ((size_t)yi * Wf + xi) * C;
                            for (int c = 0; c < C; ++c) t[c] += w * go[c];
                        }
                    }
                }
            }
        }
    }
    return 0;
}


/* ------------------------------------------------------------------------------------------
 * FlashSCA: spatial cross-attention with on-the-fly projection (paper Sec. 4.4, "Cross-framework
 * applicability").  The paper states the idea only; the operator is the deformable-attention view
 * transformation of BEVFormer, restated here:
 *
 *   every BEV query q = (ix, iy) owns Zref reference heights (bin centres of [z_min, z_max]);
 *   reference k is projected into camera n exactly as in the Sampling-VT operator; it is VALID iff
 *   depth > 0.1 and the pixel lies strictly inside the image; (ru, rv) = (u / Wimg, v / Himg);
 *   camera n is HIT by q iff at least one of its references is valid;
 *   for every hit camera, head h, level l and point p (which uses reference k = p mod Zref):
 *       pixel position in level l:  px = ru W_l + dx - 1/2,  py = rv H_l + dy - 1/2
 *       ((dx, dy) = offsets[b,q,h,l,p], in texels of level l; align_corners = False),
 *       s = bilinear sample of value level l of camera n, channels of head h, zero padding,
 *       and the point contributes  A[b,q,h,l,p] * s  if its reference is valid (this reading
 *       masks per reference; the original masks per camera only);
 *   out[b,q,h,:] = (sum over hit cameras, levels, points) / max(1, number of hit cameras).
 *
 * value   : host float32 [B][N][T][heads*Dh], T = sum_l H_l W_l texels, levels concatenated
 * level_hw: host int32 [L][2] = (H_l, W_l)
 * offsets : host float32 [B][Q][heads][L][P][2];  weights: host float32 [B][Q][heads][L][P]
 * out     : host double [B][Q][heads*Dh];  hits / flagged: host int32 [B][Q] (may be NULL)
 * Q = X*Y with q = ix*Y + iy.  Returns 0, or -1 on a bad argument.
 */
int flashbev_oracle_sca(const float *value, const int32_t *level_hw, const float *lidar2img, const float *offsets,
                        const float *weights, int B, int N, int heads, int Dh, int L, int P, int Himg, int Wimg,
                        double x_min, double x_max, double y_min, double y_max, double z_min, double z_max, int X,
                        int Y, int Zref, double *out, int32_t *hits, int32_t *flagged, int nthreads)
{
    if (!value || !level_hw || !lidar2img || !offsets || !weights || !out) return -1;
    if (B <= 0 || N <= 0 || heads <= 0 || Dh <= 0 || L <= 0 || P <= 0 || Himg <= 0 || Wimg <= 0) return -1;
    if (X <= 0 || Y <= 0 || Zref <= 0 || N > 64 || Zref > 64) return -1;
    if (!(x_max > x_min) || !(y_max > y_min) || !(z_max > z_min)) return -1;
    const int D = heads * Dh, Q = X * Y;
    long long T = 0;
    for (int l = 0; l < L; ++l) {
        if (level_hw[2 * l] <= 0 || level_hw[2 * l + 1] <= 0) return -1;
        T += (long long)level_hw[2 * l] * level_hw[2 * l + 1];
    }
#ifdef _OPENMP
    if (nthreads <= 0) nthreads = omp_get_max_threads();
#else
    nthreads = 1;
#endif
#pragma omp parallel for schedule(dynamic, 16) num_threads(nthreads)
    for (long long bq = 0; bq < (long long)B * Q; ++bq) {
        const int b = (int)(bq / Q), q = (int)(bq % Q);
        const int ix = q / Y, iy = q % Y;
        const double xw = x_min + ((double)ix + 0.5) * (x_max - x_min) / (double)X;
        const double yw = y_min + ((double)iy + 0.5) * (y_max - y_min) / (double)Y;
        double ru[64][64], rv[64][64]; /* [n][k] */
        int valid[64][64], hit[64], nhit = 0, flg = 0;
        for (int n = 0; n < N; ++n) {
            const float *M = lidar2img + ((size_t)b * N + n) * 16;
            hit[n] = 0;
            for (int k = 0; k < Zref; ++k) {
                const double zw = z_min + ((double)k + 0.5) * (z_max - z_min) / (double)Zref;
                const double p0 = (double)M[0] * xw + (double)M[1] * yw + (double)M[2] * zw + (double)M[3];
                const double p1 = (double)M[4] * xw + (double)M[5] * yw + (double)M[6] * zw + (double)M[7];
                const double d = (double)M[8] * xw + (double)M[9] * yw + (double)M[10] * zw + (double)M[11];
                valid[n][k] = 0;
                ru[n][k] = rv[n][k] = 0.0;
                if (!(d > ORACLE_DEPTH_MIN - ORACLE_BORDER_EPS)) continue;
                const double u = p0 / d, v = p1 / d;
                if (isfinite(u) && isfinite(v)) { /* smallest signed margin: image px, depth m */
                    double m = d - ORACLE_DEPTH_MIN;
                    if (u < m) m = u;
                    if ((double)Wimg - u < m) m = (double)Wimg - u;
                    if (v < m) m = v;
                    if ((double)Himg - v < m) m = (double)Himg - v;
                    if (fabs(m) < ORACLE_BORDER_EPS) flg += 1;
                }
                if (d > ORACLE_DEPTH_MIN && u > 0.0 && u < (double)Wimg && v > 0.0 && v < (double)Himg) {
                    valid[n][k] = 1;
                    ru[n][k] = u / (double)Wimg;
                    rv[n][k] = v / (double)Himg;
                    hit[n] = 1;
                }
            }
            nhit += hit[n];
        }
        double *o = out + (size_t)bq * D;
        for (int c = 0; c < D; ++c) o[c] = 0.0;
        for (int n = 0; n < N; ++n) {
            if (!hit[n]) continue;
            const float *Vn = value + ((size_t)b * N + n) * (size_t)T * D;
            for (int h = 0; h < heads; ++h) {
                long long lvl0 = 0;
                for (int l = 0; l < L; ++l) {
                    const int Hl = level_hw[2 * l], Wl = level_hw[2 * l + 1];
                    for (int p = 0; p < P; ++p) {
                        const int k = p % Zref;
                        if (!valid[n][k]) continue;
                        const size_t sidx = ((((size_t)b * Q + q) * heads + h) * L + l) * P + p;
                        const double A = (double)weights[sidx];
                        const double px = ru[n][k] * (double)Wl + (double)offsets[2 * sidx] - 0.5;
                        const double py = rv[n][k] * (double)Hl + (double)offsets[2 * sidx + 1] - 0.5;
                        const double x0f = floor(px), y0f = floor(py);
                        const double tx = px - x0f, ty = py - y0f;
                        for (int dy = 0; dy < 2; ++dy) {
                            for (int dx = 0; dx < 2; ++dx) {
                                const double xi = x0f + dx, yi = y0f + dy;
                                if (!(xi >= 0.0 && xi <= (double)(Wl - 1) && yi >= 0.0 && yi <= (double)(Hl - 1))) continue;
                                const double w = A * (dx ? tx : 1.0 - tx) * (dy ? ty : 1.0 - ty);
                                const float *t = Vn + ((size_t)lvl0 + (size_t)yi * Wl + (size_t)xi) * D + (size_t)h * Dh;
                                for (int e = 0; e < Dh; ++e) o[h * Dh + e] += w * (double)t[e];
                            }
                        }
                    }
                    lvl0 += (long long)Hl * Wl;
                }
            }
        }
        const double g = 1.0 / (double)(nhit > 1 ? nhit : 1);
        for (int c = 0; c < D; ++c) o[c] *= g;
        if (hits) hits[bq] = nhit;
        if (flagged) flagged[bq] = flg;
    }
    return 0;
}
