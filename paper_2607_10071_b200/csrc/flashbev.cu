// Fused Sampling-VT for B200 (sm_100a): kernels and the C ABI declared in flashbev.h.
//
// Two kernels compute the same operator (paper Eq. 1, fused as in Algorithm 2):
//
//   vt_per_output_kernel  one thread per (cell, channel group); every thread recomputes the
//                         projection of every (z, n) itself.  This is the work decomposition
//                         Algorithm 2 describes; it is kept as the generic path (any C, any
//                         alignment) and as the baseline the tiled kernel is measured against.
//
//   vt_tiled_kernel       a CTA owns a small tile of BEV cells.  The channel-independent part
//                         (voxel centre, projection, validity, bilinear weights, per-z camera
//                         count) is evaluated ONCE per (cell, camera, height) by "walker" threads
//                         in fp64 and turned into a compact list of row records in shared
//                         memory; successive heights that land on the same texel rows are merged
//                         into one record before any feature is touched.  Channel lanes then walk
//                         the list with 128-bit loads and fp32 FMAs.  Nothing but the output is
//                         written to global memory.
//
// Geometry (projection, validity, floor, fractions) is fp64, weights and accumulation fp32.
#include "flashbev.h"

#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr double kDepthMin = 0.1;   // metres: a sample needs camera depth > 0.1 m
constexpr int kThreads = 256;       // tiled kernel: 8 warps
constexpr int kWarps = kThreads / 32;
constexpr int kRecordSlots = 128;   // list records per warp (shared by the warp's cells)
constexpr int kWalkerCap = 2048;    // walker descriptors per CTA and height chunk
constexpr int kMaxCams = 64;

struct KParams {
    const void *feat;
    const float *l2i;
    float *out;
    int32_t *count_out;
    int B, N, C, Hf, Wf, X, Y, Z, reduce;
    double sx, sy;              // image px -> feature px
    double x_min, dx, y_min, dy, z_min, dz;
    // tiled kernel only
    int vecs;                   // 16-byte vectors per texel (C * elem / 16)
    int g;                      // lanes per cell
    int cpw;                    // cells per warp
    int wx, wy, Wx, Wy;         // cells per warp block, warp blocks per CTA tile (x, y)
    int tiles_x, tiles_y;
    int zc;                     // height bins per chunk (multiple of 4 unless == Z)
    int walk;                   // height bins per walker
    int lcap;                   // records per cell list
};

// ------------------------------------------------------------------------------------------
// shared geometry helpers

// 1/d for d > 0.1: single-precision seed refined twice in fp64 (relative error ~1e-16).
__device__ __forceinline__ double fast_rcp(double d)
{
    double r = (double)__frcp_rn((float)d);
    double e = fma(-d, r, 1.0);
    r = fma(r, e, r);
    e = fma(-d, r, 1.0);
    return fma(r, e, r);
}

struct Sample {
    int x0, y0;
    float tx, ty;
};

// One candidate sample.  ps0/ps1 are rows 0/1 of the projection already multiplied by the
// image->feature scale, d is row 2.  Returns M_n; fills the bilinear corner and fractions.
__device__ __forceinline__ bool project_sample(double ps0, double ps1, double d, double wlim, double hlim,
                                               Sample &s)
{
    if (!(d > kDepthMin)) return false;  // also rejects NaN
    const double r = fast_rcp(d);
    const double fx = fma(ps0, r, -0.5);  // grid_sample(align_corners=False) texel coordinates
    const double fy = fma(ps1, r, -0.5);
    if (!(fx > -0.5 && fx < wlim && fy > -0.5 && fy < hlim)) return false;
    const double flx = floor(fx), fly = floor(fy);
    s.x0 = (int)flx;
    s.y0 = (int)fly;
    s.tx = (float)(fx - flx);
    s.ty = (float)(fy - fly);
    return true;
}

__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8])
{
    f[0] = __uint_as_float(v.x << 16);
    f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16);
    f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16);
    f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16);
    f[7] = __uint_as_float(v.w & 0xffff0000u);
}

__device__ __forceinline__ float load_elem(const float *p) { return __ldg(p); }
__device__ __forceinline__ float load_elem(const uint16_t *p)
{
    return __uint_as_float(((uint32_t)__ldg(p)) << 16);
}

// ------------------------------------------------------------------------------------------
// Kernel 1: one thread per (cell, group of VEC channels).  T = float or uint16_t (bf16 bits).

template <typename T, int VEC>
__global__ void __launch_bounds__(256) vt_per_output_kernel(const KParams p)
{
    const int groups = (p.C + VEC - 1) / VEC;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long cell = gid / groups;
    if (cell >= (long long)p.B * p.X * p.Y) return;
    const int c0 = (int)(gid % groups) * VEC;
    const int b = (int)(cell / ((long long)p.X * p.Y));
    const int ix = (int)((cell / p.Y) % p.X);
    const int iy = (int)(cell % p.Y);
    const double xw = p.x_min + ((double)ix + 0.5) * p.dx;
    const double yw = p.y_min + ((double)iy + 0.5) * p.dy;
    const double wlim = (double)p.Wf - 0.5, hlim = (double)p.Hf - 0.5;
    const T *feat = static_cast<const T *>(p.feat);

    float acc[VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) acc[i] = 0.f;
    int count = 0;

    for (int k = 0; k < p.Z; ++k) {
        const double zw = p.z_min + ((double)k + 0.5) * p.dz;
        float num[VEC];
#pragma unroll
        for (int i = 0; i < VEC; ++i) num[i] = 0.f;
        int den = 0;
        for (int n = 0; n < p.N; ++n) {
            const float *M = p.l2i + ((size_t)b * p.N + n) * 16;
            const double p0 = fma((double)M[2], zw, fma((double)M[1], yw, fma((double)M[0], xw, (double)M[3])));
            const double p1 = fma((double)M[6], zw, fma((double)M[5], yw, fma((double)M[4], xw, (double)M[7])));
            const double d = fma((double)M[10], zw, fma((double)M[9], yw, fma((double)M[8], xw, (double)M[11])));
            Sample s;
            if (!project_sample(p0 * p.sx, p1 * p.sy, d, wlim, hlim, s)) continue;
            den += 1;
            const T *fn = feat + ((size_t)b * p.N + n) * (size_t)p.Hf * p.Wf * p.C;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int xi = s.x0 + (t & 1), yi = s.y0 + (t >> 1);
                if (xi < 0 || xi > p.Wf - 1 || yi < 0 || yi > p.Hf - 1) continue;  // zero padding
                const float w = ((t & 1) ? s.tx : 1.f - s.tx) * ((t >> 1) ? s.ty : 1.f - s.ty);
                const T *tp = fn + ((size_t)yi * p.Wf + xi) * p.C + c0;
                if (VEC == 1) {
                    num[0] = fmaf(w, load_elem(tp), num[0]);
                } else if (sizeof(T) == 4) {
                    const float4 v = __ldg(reinterpret_cast<const float4 *>(tp));
                    num[0] = fmaf(w, v.x, num[0]);
                    num[1 % VEC] = fmaf(w, v.y, num[1 % VEC]);
                    num[2 % VEC] = fmaf(w, v.z, num[2 % VEC]);
                    num[3 % VEC] = fmaf(w, v.w, num[3 % VEC]);
                } else {
                    float f[8];
                    unpack8(__ldg(reinterpret_cast<const uint4 *>(tp)), f);
#pragma unroll
                    for (int i = 0; i < 8; ++i) num[i % VEC] = fmaf(w, f[i], num[i % VEC]);
                }
            }
        }
        count += den;
        if (p.reduce == FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM) {
            const float g = 1.f / (float)(den > 1 ? den : 1);  // g_z = num_z / max(1, den_z)
#pragma unroll
            for (int i = 0; i < VEC; ++i) acc[i] = fmaf(num[i], g, acc[i]);
        } else {
#pragma unroll
            for (int i = 0; i < VEC; ++i) acc[i] += num[i];
        }
    }
    if (p.reduce == FLASHBEV_REDUCE_MEAN_OVER_VALID) {
        const float g = 1.f / (float)(count > 1 ? count : 1);
#pragma unroll
        for (int i = 0; i < VEC; ++i) acc[i] *= g;
    }
    float *o = p.out + (size_t)cell * p.C + c0;
    if (VEC == 1) {
        o[0] = acc[0];
    } else {
#pragma unroll
        for (int i = 0; i < VEC; i += 4)
            __stcs(reinterpret_cast<float4 *>(o + i),
                   make_float4(acc[i], acc[(i + 1) % VEC], acc[(i + 2) % VEC], acc[(i + 3) % VEC]));
    }
    if (p.count_out && c0 == 0) p.count_out[cell] = count;
}

// ------------------------------------------------------------------------------------------
// Kernel 2: tiled.  Shared-memory layout (dynamic):
//   double  mats[N][12]          rows 0..2 of lidar2img[b][n], rows 0/1 pre-scaled to feature px
//   float4  lists[warps][kRecordSlots + cpw]   per cell: lcap records (+1 pad) {vector offset, wL, wR, -}
//   uint32  walkers[kWalkerCap]  packed (cell, camera, first bin in chunk, bins - 1)
//   uint32  den[cells * zc / 4]  per (cell, z) camera counts, one byte each (Eq. 1 mode only)
//   int     list_count[cells], cell_count[cells], n_walkers

struct TileSmem {
    double *mats;
    float4 *lists;
    uint32_t *walkers;
    uint32_t *den;
    int *list_count;
    int *cell_count;
    int *n_walkers;
};

__host__ __device__ inline size_t tile_smem_bytes(int N, int cells, int cpw, int zc)
{
    size_t s = (size_t)N * 12 * sizeof(double);
    s += (size_t)kWarps * (kRecordSlots + cpw) * sizeof(float4);
    s += (size_t)kWalkerCap * sizeof(uint32_t);
    s += (size_t)((cells * zc + 3) / 4) * sizeof(uint32_t);
    s += (size_t)(2 * cells + 4) * sizeof(int);
    return s;
}

__device__ __forceinline__ TileSmem carve(unsigned char *base, int N, int cells, int cpw, int zc)
{
    TileSmem t;
    t.mats = reinterpret_cast<double *>(base);
    base += (size_t)N * 12 * sizeof(double);
    t.lists = reinterpret_cast<float4 *>(base);
    base += (size_t)kWarps * (kRecordSlots + cpw) * sizeof(float4);
    t.walkers = reinterpret_cast<uint32_t *>(base);
    base += (size_t)kWalkerCap * sizeof(uint32_t);
    t.den = reinterpret_cast<uint32_t *>(base);
    base += (size_t)((cells * zc + 3) / 4) * sizeof(uint32_t);
    t.list_count = reinterpret_cast<int *>(base);
    t.cell_count = t.list_count + cells;
    t.n_walkers = t.cell_count + cells;
    return t;
}

// Position of local cell c inside the CTA tile (warp-major, so a warp's cells are adjacent).
__device__ __forceinline__ void cell_xy(const KParams &p, int c, int &lx, int &ly)
{
    const int w = c / p.cpw, j = c - w * p.cpw;
    const int jx = j / p.wy, jy = j - jx * p.wy;
    const int wxi = w / p.Wy, wyi = w - wxi * p.Wy;
    lx = wxi * p.wx + jx;
    ly = wyi * p.wy + jy;
}

// Geometry of one (cell, camera) column: row_i(z) = A_i + B_i * z_w, with B_i read from smem.
struct Column {
    double a0, a1, a2;
};

__device__ __forceinline__ Column make_column(const double *m, double xw, double yw)
{
    Column c;
    c.a0 = fma(m[1], yw, fma(m[0], xw, m[3]));
    c.a1 = fma(m[5], yw, fma(m[4], xw, m[7]));
    c.a2 = fma(m[9], yw, fma(m[8], xw, m[11]));
    return c;
}

template <int V, bool BF16>
__global__ void __launch_bounds__(kThreads) vt_tiled_kernel(const KParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int EPV = BF16 ? 8 : 4;  // channels per 16-byte vector
    const int cells = kWarps * p.cpw;
    const TileSmem sm = carve(smem_raw, p.N, cells, p.cpw, p.zc);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // ---- which tile
    const int tpb = p.tiles_x * p.tiles_y;
    const int b = blockIdx.x / tpb;
    const int trem = blockIdx.x - b * tpb;
    const int tile_x = trem / p.tiles_y, tile_y = trem - tile_x * p.tiles_y;
    const int tx = p.Wx * p.wx, ty = p.Wy * p.wy;
    const int ix0 = tile_x * tx, iy0 = tile_y * ty;
    const double wlim = (double)p.Wf - 0.5, hlim = (double)p.Hf - 0.5;

    // ---- stage the camera matrices of this batch element (a1)
    for (int i = tid; i < p.N * 12; i += kThreads) {
        const int n = i / 12, e = i - n * 12;
        double v = (double)__ldg(p.l2i + ((size_t)b * p.N + n) * 16 + e);
        if (e < 4) v *= p.sx;
        else if (e < 8) v *= p.sy;
        sm.mats[i] = v;
    }
    for (int i = tid; i < cells; i += kThreads) sm.cell_count[i] = 0;

    // ---- gather role of this lane
    const int cg = lane / p.g, gl = lane - cg * p.g;
    const int my_cell = warp * p.cpw + cg;  // valid if cg < cpw
    int mlx = 0, mly = 0;
    if (cg < p.cpw) cell_xy(p, my_cell, mlx, mly);
    const int vec0 = blockIdx.y * (p.g * V) + gl;  // first channel vector of this lane
    const bool lane_on = (cg < p.cpw) && (ix0 + mlx < p.X) && (iy0 + mly < p.Y);
    const uint4 *featb = static_cast<const uint4 *>(p.feat) + (size_t)b * p.N * p.Hf * p.Wf * p.vecs;
    const float4 *my_list = sm.lists + warp * (kRecordSlots + p.cpw) + (cg < p.cpw ? cg : 0) * (p.lcap + 1);

    float acc[V][EPV];
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < EPV; ++e) acc[v][e] = 0.f;

    for (int kc0 = 0; kc0 < p.Z; kc0 += p.zc) {
        const int kc1 = min(p.Z, kc0 + p.zc);  // chunk [kc0, kc1)
        if (tid == 0) *sm.n_walkers = 0;
        if (p.reduce == FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM)
            for (int i = tid; i < (cells * p.zc + 3) / 4; i += kThreads) sm.den[i] = 0u;
        __syncthreads();

        // ---- phase A: per (cell, camera) column, a conservative interval of height bins that can
        // be valid (every validity condition is linear in z once d > 0), split into walkers
        for (int pr = tid; pr < cells * p.N; pr += kThreads) {
            const int c = pr / p.N, n = pr - c * p.N;
            int lx, ly;
            cell_xy(p, c, lx, ly);
            if (ix0 + lx >= p.X || iy0 + ly >= p.Y) continue;
            const double xw = p.x_min + ((double)(ix0 + lx) + 0.5) * p.dx;
            const double yw = p.y_min + ((double)(iy0 + ly) + 0.5) * p.dy;
            const double *m = sm.mats + n * 12;
            const Column col = make_column(m, xw, yw);
            const double zc0 = p.z_min + 0.5 * p.dz;  // centre of bin 0; z_w(k) = zc0 + k dz
            // conditions alpha + beta * k > 0 (k real): depth, left, right, top, bottom
            const double al[5] = {col.a2 + m[10] * zc0 - kDepthMin, col.a0 + m[2] * zc0,
                                  (double)p.Wf * (col.a2 + m[10] * zc0) - (col.a0 + m[2] * zc0),
                                  col.a1 + m[6] * zc0, (double)p.Hf * (col.a2 + m[10] * zc0) - (col.a1 + m[6] * zc0)};
            const double be[5] = {m[10] * p.dz, m[2] * p.dz, ((double)p.Wf * m[10] - m[2]) * p.dz, m[6] * p.dz,
                                  ((double)p.Hf * m[10] - m[6]) * p.dz};
            float lo = (float)kc0 - 1.f, hi = (float)kc1;
            bool empty = false;
#pragma unroll
            for (int i = 0; i < 5; ++i) {
                const float a = (float)al[i], bb = (float)be[i];
                if (bb > 0.f) lo = fmaxf(lo, -a / bb);       // k > -a/b
                else if (bb < 0.f) hi = fminf(hi, -a / bb);  // k < -a/b
                else if (a <= 0.f) empty = true;             // independent of z (NaN: keep)
            }
            if (empty) continue;
            // widen by a guard far above the float error; every bin is re-tested exactly later
            const float guard = 0.05f + 1e-5f * (float)p.Z;
            int klo = (int)floorf(fminf(fmaxf(lo - guard, (float)kc0 - 1.f), (float)kc1)) + 1;
            int khi = (int)ceilf(fmaxf(fminf(hi + guard, (float)kc1), (float)kc0 - 1.f)) - 1;
            klo = max(klo, kc0);
            khi = min(khi, kc1 - 1);
            if (klo > khi) continue;
            const int nw = (khi - klo + p.walk) / p.walk;
            const int base = atomicAdd(sm.n_walkers, nw);
            for (int i = 0; i < nw; ++i) {
                const int k0 = klo + i * p.walk, k1 = min(khi, k0 + p.walk - 1);
                if (base + i < kWalkerCap)
                    sm.walkers[base + i] = (uint32_t)c | ((uint32_t)n << 8) | ((uint32_t)(k0 - kc0) << 14) |
                                           ((uint32_t)(k1 - k0) << 23);
            }
        }
        __syncthreads();
        const int n_walkers = min(*sm.n_walkers, kWalkerCap);

        // ---- Eq. 1 mode: den_z = sum_n M_n for every (cell, z) of the chunk, before any weight
        if (p.reduce == FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM) {
            for (int wi = tid; wi < n_walkers; wi += kThreads) {
                const uint32_t wd = sm.walkers[wi];
                const int c = wd & 0xff, n = (wd >> 8) & 0x3f, k0 = kc0 + ((wd >> 14) & 0x1ff), k1 = k0 + (wd >> 23);
                int lx, ly;
                cell_xy(p, c, lx, ly);
                const double xw = p.x_min + ((double)(ix0 + lx) + 0.5) * p.dx;
                const double yw = p.y_min + ((double)(iy0 + ly) + 0.5) * p.dy;
                const double *m = sm.mats + n * 12;
                const Column col = make_column(m, xw, yw);
                for (int k = k0; k <= k1; ++k) {
                    const double zw = p.z_min + ((double)k + 0.5) * p.dz;
                    Sample s;
                    if (project_sample(fma(m[2], zw, col.a0), fma(m[6], zw, col.a1), fma(m[10], zw, col.a2), wlim,
                                       hlim, s)) {
                        const int di = c * p.zc + (k - kc0);
                        atomicAdd(&sm.den[di >> 2], 1u << (8 * (di & 3)));
                    }
                }
            }
            __syncthreads();
        }

        // ---- walkers in batches of one per thread; each batch: walk -> gather, repeated while a
        // walker had to stop because its cell's list was full
        for (int wb = 0; wb < n_walkers; wb += kThreads) {
            const int wi = wb + tid;
            bool done = wi >= n_walkers;
            int wc = 0, wn = 0, k = 0, kend = -1, vcount = 0;
            Column col = {0.0, 0.0, 0.0};
            const double *m = sm.mats;
            if (!done) {
                const uint32_t wd = sm.walkers[wi];
                wc = wd & 0xff;
                wn = (wd >> 8) & 0x3f;
                k = kc0 + ((wd >> 14) & 0x1ff);
                kend = k + (int)(wd >> 23);
                int lx, ly;
                cell_xy(p, wc, lx, ly);
                const double xw = p.x_min + ((double)(ix0 + lx) + 0.5) * p.dx;
                const double yw = p.y_min + ((double)(iy0 + ly) + 0.5) * p.dy;
                m = sm.mats + wn * 12;
                col = make_column(m, xw, yw);
            }
            // open pair of texel rows (oy, oy+1) at column ox with merged weights
            bool open = false, flushed = false;
            int ox = 0, oy = 0;
            float uL = 0.f, uR = 0.f, lL = 0.f, lR = 0.f;
            float4 *wlist = sm.lists + (wc / p.cpw) * (kRecordSlots + p.cpw) + (wc % p.cpw) * (p.lcap + 1);

            while (true) {
                for (int i = tid; i < cells; i += kThreads) sm.list_count[i] = 0;
                __syncthreads();

                while (!done) {
                    // what does the next step want to emit?
                    Sample s;
                    bool valid = false;
                    float scale = 1.f;
                    int close_u = 0, close_l = 0;  // close upper / lower open row
                    if (k <= kend) {
                        const double zw = p.z_min + ((double)k + 0.5) * p.dz;
                        valid = project_sample(fma(m[2], zw, col.a0), fma(m[6], zw, col.a1), fma(m[10], zw, col.a2),
                                               wlim, hlim, s);
                        if (!valid) {
                            ++k;
                            continue;
                        }
                        if (open) {
                            if (s.x0 == ox && s.y0 == oy) {
                            } else if (s.x0 == ox && s.y0 == oy + 1) close_u = 1;
                            else if (s.x0 == ox && s.y0 == oy - 1) close_l = 1;
                            else close_u = close_l = 1;
                        }
                    } else {
                        if (!open || flushed) {
                            done = true;
                            break;
                        }
                        close_u = close_l = 1;
                    }
                    // records to write: rows inside the map with a non-zero weight
                    const float cuL = (ox >= 0) ? uL : 0.f, cuR = (ox + 1 <= p.Wf - 1) ? uR : 0.f;
                    const float clL = (ox >= 0) ? lL : 0.f, clR = (ox + 1 <= p.Wf - 1) ? lR : 0.f;
                    const bool emit_u = close_u && oy >= 0 && oy <= p.Hf - 1 && (cuL != 0.f || cuR != 0.f);
                    const bool emit_l = close_l && oy + 1 >= 0 && oy + 1 <= p.Hf - 1 && (clL != 0.f || clR != 0.f);
                    const int need = (int)emit_u + (int)emit_l;
                    if (need) {
                        const int slot = atomicAdd(&sm.list_count[wc], need);
                        if (slot + need > p.lcap) {  // list full: null any slot we hold, retry next round
                            if (slot < p.lcap) wlist[slot] = make_float4(0.f, 0.f, 0.f, 0.f);
                            break;
                        }
                        int sl = slot;
                        if (emit_u) {
                            const int off = ((wn * p.Hf + oy) * p.Wf + ox) * p.vecs;
                            wlist[sl++] = make_float4(__int_as_float(off), cuL, cuR, 0.f);
                        }
                        if (emit_l) {
                            const int off = ((wn * p.Hf + oy + 1) * p.Wf + ox) * p.vecs;
                            wlist[sl] = make_float4(__int_as_float(off), clL, clR, 0.f);
                        }
                    }
                    if (k > kend) {
                        flushed = true;
                        done = true;
                        break;
                    }
                    // commit the sample
                    if (p.reduce == FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM) {
                        const int di = wc * p.zc + (k - kc0);
                        const uint32_t dn = (sm.den[di >> 2] >> (8 * (di & 3))) & 0xffu;
                        scale = 1.f / (float)(dn > 1u ? dn : 1u);
                    }
                    const float wx1 = s.tx, wx0 = 1.f - s.tx;
                    const float wy1 = s.ty * scale, wy0 = (1.f - s.ty) * scale;
                    const float w00 = wx0 * wy0, w01 = wx1 * wy0, w10 = wx0 * wy1, w11 = wx1 * wy1;
                    if (open && close_u && !close_l) {  // moved one row down
                        uL = lL + w00, uR = lR + w01, lL = w10, lR = w11;
                    } else if (open && close_l && !close_u) {  // moved one row up
                        lL = uL + w10, lR = uR + w11, uL = w00, uR = w01;
                    } else if (open && !close_u && !close_l) {
                        uL += w00, uR += w01, lL += w10, lR += w11;
                    } else {
                        uL = w00, uR = w01, lL = w10, lR = w11;
                    }
                    open = true;
                    ox = s.x0;
                    oy = s.y0;
                    ++vcount;
                    ++k;
                }
                __syncthreads();

                // ---- gather (a7): channel lanes walk their cell's records
                {
                    const int nrec = lane_on ? min(sm.list_count[my_cell], p.lcap) : 0;
                    const int maxn = __reduce_max_sync(0xffffffffu, nrec);
                    for (int j = 0; j < maxn; j += 2) {
                        float4 r[2];
                        r[0] = (j < nrec) ? my_list[j] : make_float4(0.f, 0.f, 0.f, 0.f);
                        r[1] = (j + 1 < nrec) ? my_list[j + 1] : make_float4(0.f, 0.f, 0.f, 0.f);
                        uint4 tl[2][V], tr[2][V];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const uint4 *base = featb + __float_as_int(r[u].x);
#pragma unroll
                            for (int v = 0; v < V; ++v) {
                                const int vi = vec0 + v * p.g;
                                tl[u][v] = make_uint4(0u, 0u, 0u, 0u);
                                tr[u][v] = make_uint4(0u, 0u, 0u, 0u);
                                if (vi < p.vecs) {
                                    if (r[u].y != 0.f) tl[u][v] = __ldg(base + vi);
                                    if (r[u].z != 0.f) tr[u][v] = __ldg(base + p.vecs + vi);
                                }
                            }
                        }
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
#pragma unroll
                            for (int v = 0; v < V; ++v) {
                                if (BF16) {
                                    float fl[8], fr[8];
                                    unpack8(tl[u][v], fl);
                                    unpack8(tr[u][v], fr);
#pragma unroll
                                    for (int e = 0; e < 8; ++e) {
                                        acc[v][e % EPV] = fmaf(r[u].y, fl[e], acc[v][e % EPV]);
                                        acc[v][e % EPV] = fmaf(r[u].z, fr[e], acc[v][e % EPV]);
                                    }
                                } else {
                                    const float fl[4] = {__uint_as_float(tl[u][v].x), __uint_as_float(tl[u][v].y),
                                                         __uint_as_float(tl[u][v].z), __uint_as_float(tl[u][v].w)};
                                    const float fr[4] = {__uint_as_float(tr[u][v].x), __uint_as_float(tr[u][v].y),
                                                         __uint_as_float(tr[u][v].z), __uint_as_float(tr[u][v].w)};
#pragma unroll
                                    for (int e = 0; e < 4; ++e) {
                                        acc[v][e] = fmaf(r[u].y, fl[e], acc[v][e]);
                                        acc[v][e] = fmaf(r[u].z, fr[e], acc[v][e]);
                                    }
                                }
                            }
                        }
                    }
                }
                if (!__syncthreads_or(!done)) break;
            }
            if (wi < n_walkers && vcount) atomicAdd(&sm.cell_count[wc], vcount);
        }
        __syncthreads();
    }

    // ---- epilogue (a8): one store per output vector
    if (lane_on) {
        const int count = sm.cell_count[my_cell];
        const float g = (p.reduce == FLASHBEV_REDUCE_MEAN_OVER_VALID) ? 1.f / (float)(count > 1 ? count : 1) : 1.f;
        const size_t cell = ((size_t)b * p.X + (ix0 + mlx)) * p.Y + (iy0 + mly);
        float *o = p.out + cell * p.C;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int vi = vec0 + v * p.g;
            if (vi < p.vecs) {
#pragma unroll
                for (int e = 0; e < EPV; e += 4)
                    __stcs(reinterpret_cast<float4 *>(o + (size_t)vi * EPV + e),
                           make_float4(acc[v][e] * g, acc[v][e + 1] * g, acc[v][e + 2] * g, acc[v][e + 3] * g));
            }
        }
        if (p.count_out && gl == 0 && blockIdx.y == 0) p.count_out[cell] = count;
    }
}

// ------------------------------------------------------------------------------------------
// host side

thread_local int t_last_launches = 0;
thread_local const char *t_last_kernel = "none";

bool params_ok(const flashbev_vt_params *p, flashbev_status &st)
{
    st = FLASHBEV_INVALID_ARG;
    if (!p || p->struct_size < sizeof(flashbev_vt_params)) return false;
    if (!p->features || !p->lidar2img || !p->out) return false;
    if (p->B <= 0 || p->N <= 0 || p->C <= 0 || p->feat_h <= 0 || p->feat_w <= 0 || p->img_h <= 0 || p->img_w <= 0)
        return false;
    if (p->X <= 0 || p->Y <= 0 || p->Z <= 0) return false;
    if (!(p->x_max > p->x_min) || !(p->y_max > p->y_min) || !(p->z_max > p->z_min)) return false;
    if (!(p->x_max - p->x_min < 1e300) || !(p->y_max - p->y_min < 1e300) || !(p->z_max - p->z_min < 1e300))
        return false;  // rejects inf / NaN ranges
    if (p->feat_dtype != FLASHBEV_F32 && p->feat_dtype != FLASHBEV_BF16) return false;
    if (p->layout != FLASHBEV_NHWC && p->layout != FLASHBEV_NCHW) return false;
    if (p->reduce < 0 || p->reduce > 2) return false;
    if (p->out_dtype != FLASHBEV_F32 && p->out_dtype != FLASHBEV_BF16) return false;
    if (p->kernel < 0 || p->kernel > 2) return false;
    st = FLASHBEV_UNSUPPORTED;
    if (p->layout != FLASHBEV_NHWC || p->out_dtype != FLASHBEV_F32) return false;
    if (p->N > kMaxCams) return false;
    const size_t elem = p->feat_dtype == FLASHBEV_F32 ? 4 : 2;
    const double cam_bytes = (double)p->N * p->feat_h * p->feat_w * p->C * (double)elem;
    if (cam_bytes >= 34359738368.0) return false;                          // 2^35
    if ((double)p->B * p->X * p->Y >= 2147483648.0) return false;          // 2^31
    if ((double)p->B * p->X * p->Y * p->C >= 9.0e15) return false;
    st = FLASHBEV_OK;
    return true;
}

flashbev_status check_alignment(const flashbev_vt_params *p)
{
    const size_t elem = p->feat_dtype == FLASHBEV_F32 ? 4 : 2;
    if (((uintptr_t)p->features % elem) || ((uintptr_t)p->out % 4) || ((uintptr_t)p->lidar2img % 4)) return FLASHBEV_MISALIGNED;
    if (p->valid_count_out && ((uintptr_t)p->valid_count_out % 4)) return FLASHBEV_MISALIGNED;
    return FLASHBEV_OK;
}

KParams base_params(const flashbev_vt_params *p)
{
    KParams k = {};
    k.feat = p->features;
    k.l2i = p->lidar2img;
    k.out = static_cast<float *>(p->out);
    k.count_out = p->valid_count_out;
    k.B = p->B, k.N = p->N, k.C = p->C, k.Hf = p->feat_h, k.Wf = p->feat_w;
    k.X = p->X, k.Y = p->Y, k.Z = p->Z, k.reduce = p->reduce;
    k.sx = (double)p->feat_w / (double)p->img_w;
    k.sy = (double)p->feat_h / (double)p->img_h;
    k.x_min = p->x_min, k.dx = (p->x_max - p->x_min) / (double)p->X;
    k.y_min = p->y_min, k.dy = (p->y_max - p->y_min) / (double)p->Y;
    k.z_min = p->z_min, k.dz = (p->z_max - p->z_min) / (double)p->Z;
    return k;
}

flashbev_status launch_per_output(const flashbev_vt_params *p, cudaStream_t stream)
{
    const KParams k = base_params(p);
    const bool bf16 = p->feat_dtype == FLASHBEV_BF16;
    const int vec = bf16 ? 8 : 4;
    const bool vec_ok = (p->C % vec == 0) && ((uintptr_t)p->features % 16 == 0) && ((uintptr_t)p->out % 16 == 0);
    const int per_thread = vec_ok ? vec : 1;
    const long long threads = (long long)p->B * p->X * p->Y * ((p->C + per_thread - 1) / per_thread);
    const long long blocks = (threads + 255) / 256;
    if (blocks > 2147483647LL) return FLASHBEV_UNSUPPORTED;
    const dim3 grid((unsigned)blocks), block(256);
    if (bf16 && vec_ok) {
        vt_per_output_kernel<uint16_t, 8><<<grid, block, 0, stream>>>(k);
        t_last_kernel = "per_output_bf16x8";
    } else if (bf16) {
        vt_per_output_kernel<uint16_t, 1><<<grid, block, 0, stream>>>(k);
        t_last_kernel = "per_output_bf16x1";
    } else if (vec_ok) {
        vt_per_output_kernel<float, 4><<<grid, block, 0, stream>>>(k);
        t_last_kernel = "per_output_f32x4";
    } else {
        vt_per_output_kernel<float, 1><<<grid, block, 0, stream>>>(k);
        t_last_kernel = "per_output_f32x1";
    }
    return FLASHBEV_OK;
}

bool tiled_applicable(const flashbev_vt_params *p)
{
    const size_t elem = p->feat_dtype == FLASHBEV_F32 ? 4 : 2;
    if (((size_t)p->C * elem) % 16) return false;
    if (((uintptr_t)p->features % 16) || ((uintptr_t)p->out % 16)) return false;
    const double vecs_total = (double)p->N * p->feat_h * p->feat_w * (double)((size_t)p->C * elem / 16);
    return vecs_total < 2147483648.0;
}

template <int V, bool BF16>
cudaError_t launch_tiled_inst(const KParams &k, dim3 grid, size_t smem, cudaStream_t stream)
{
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(vt_tiled_kernel<V, BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    vt_tiled_kernel<V, BF16><<<grid, dim3(kThreads), smem, stream>>>(k);
    return cudaSuccess;
}

flashbev_status launch_tiled(const flashbev_vt_params *p, cudaStream_t stream)
{
    KParams k = base_params(p);
    const bool bf16 = p->feat_dtype == FLASHBEV_BF16;
    const int elem = bf16 ? 2 : 4;
    k.vecs = p->C * elem / 16;

    // channel mapping: V vectors per lane, g lanes per cell
    int V = p->tune[0], g = p->tune[1];
    if (!(V == 1 || V == 2 || V == 4) || g < 1 || g > 32) V = 0, g = 0;
    if (!V) {
        if (k.vecs <= 8) V = 1, g = k.vecs;
        else if (k.vecs <= 16) V = (k.vecs % 2 == 0) ? 2 : 1, g = (k.vecs + V - 1) / V;
        else if (k.vecs <= 64) V = 2, g = (k.vecs + 1) / 2;
        else V = 4, g = (k.vecs + 3) / 4;
        if (g > 32) g = 32;
    }
    k.g = g;
    k.cpw = 32 / g;
    if (k.cpw > 8) k.cpw = 8;
    // warp block (wx x wy cells) and CTA arrangement (Wx x Wy warps): near-square tiles
    k.wy = (k.cpw % 2 == 0) ? 2 : (k.cpw == 3 ? 3 : 1);
    if (k.cpw == 8) k.wy = 4;
    if (k.cpw == 6) k.wy = 3;
    k.wx = k.cpw / k.wy;
    k.cpw = k.wx * k.wy;
    k.Wx = (k.wx >= k.wy) ? 2 : 4;
    k.Wy = kWarps / k.Wx;
    const int tx = k.Wx * k.wx, ty = k.Wy * k.wy, cells = kWarps * k.cpw;
    k.tiles_x = (p->X + tx - 1) / tx;
    k.tiles_y = (p->Y + ty - 1) / ty;
    k.lcap = kRecordSlots / k.cpw;
    k.walk = (p->tune[2] >= 1 && p->tune[2] <= 64) ? p->tune[2] : 8;
    // height chunk: all walkers of a chunk must fit the descriptor array
    int per_pair = kWalkerCap / (cells * p->N);
    if (per_pair < 1) return FLASHBEV_UNSUPPORTED;
    int zc = per_pair * k.walk;
    if (zc > 256) zc = 256;
    if (zc >= p->Z) zc = p->Z;
    else zc = (zc / 4) * 4 > 0 ? (zc / 4) * 4 : zc;
    k.zc = zc;

    const long long tiles = (long long)p->B * k.tiles_x * k.tiles_y;
    const int cblocks = (k.vecs + g * V - 1) / (g * V);
    if (tiles > 2147483647LL || cblocks > 65535) return FLASHBEV_UNSUPPORTED;
    const dim3 grid((unsigned)tiles, (unsigned)cblocks);
    const size_t smem = tile_smem_bytes(p->N, cells, k.cpw, k.zc);
    cudaError_t e;
    static const char *const names[2][3] = {{"tiled_f32_v1", "tiled_f32_v2", "tiled_f32_v4"},
                                            {"tiled_bf16_v1", "tiled_bf16_v2", "tiled_bf16_v4"}};
    if (bf16) {
        if (V == 1) e = launch_tiled_inst<1, true>(k, grid, smem, stream);
        else if (V == 2) e = launch_tiled_inst<2, true>(k, grid, smem, stream);
        else e = launch_tiled_inst<4, true>(k, grid, smem, stream);
    } else {
        if (V == 1) e = launch_tiled_inst<1, false>(k, grid, smem, stream);
        else if (V == 2) e = launch_tiled_inst<2, false>(k, grid, smem, stream);
        else e = launch_tiled_inst<4, false>(k, grid, smem, stream);
    }
    t_last_kernel = names[bf16 ? 1 : 0][V == 1 ? 0 : (V == 2 ? 1 : 2)];
    return e == cudaSuccess ? FLASHBEV_OK : FLASHBEV_CUDA_ERROR;
}

flashbev_status run_device(const flashbev_vt_params *p, cudaStream_t stream)
{
    flashbev_status st;
    const bool tiled = p->kernel == FLASHBEV_KERNEL_TILED || (p->kernel == FLASHBEV_KERNEL_AUTO && tiled_applicable(p));
    if (tiled && !tiled_applicable(p)) return FLASHBEV_UNSUPPORTED;
    st = tiled ? launch_tiled(p, stream) : launch_per_output(p, stream);
    if (st != FLASHBEV_OK) return st;
    if (cudaGetLastError() != cudaSuccess) return FLASHBEV_CUDA_ERROR;
    t_last_launches = 1;
    return FLASHBEV_OK;
}

struct StagingLayout {
    size_t feat_off, mat_off, out_off, cnt_off, total;
};

StagingLayout staging_layout(const flashbev_vt_params *p)
{
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    const size_t elem = p->feat_dtype == FLASHBEV_F32 ? 4 : 2;
    StagingLayout s;
    s.feat_off = 0;
    s.mat_off = up((size_t)p->B * p->N * p->feat_h * p->feat_w * p->C * elem);
    s.out_off = s.mat_off + up((size_t)p->B * p->N * 64);
    s.cnt_off = s.out_off + up((size_t)p->B * p->X * p->Y * p->C * 4);
    s.total = s.cnt_off + (p->valid_count_out ? up((size_t)p->B * p->X * p->Y * 4) : 0);
    return s;
}

}  // namespace

extern "C" {

flashbev_status flashbev_sampling_vt(const flashbev_vt_params *p, void *stream)
{
    flashbev_status st;
    if (!params_ok(p, st)) return st;
    if ((st = check_alignment(p)) != FLASHBEV_OK) return st;
    return run_device(p, static_cast<cudaStream_t>(stream));
}

size_t flashbev_workspace_bytes(const flashbev_vt_params *p)
{
    (void)p;
    return 0;
}

size_t flashbev_host_staging_bytes(const flashbev_vt_params *p)
{
    flashbev_status st;
    if (!params_ok(p, st)) return 0;
    return staging_layout(p).total;
}

flashbev_status flashbev_sampling_vt_host(const flashbev_vt_params *p, void *d_staging, size_t staging_bytes,
                                          void *stream_)
{
    flashbev_status st;
    if (!params_ok(p, st)) return st;
    if (!d_staging) return FLASHBEV_INVALID_ARG;
    if ((uintptr_t)d_staging % 256) return FLASHBEV_MISALIGNED;
    const StagingLayout L = staging_layout(p);
    if (staging_bytes < L.total) return FLASHBEV_TOO_SMALL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    unsigned char *base = static_cast<unsigned char *>(d_staging);
    flashbev_vt_params d = *p;
    d.features = base + L.feat_off;
    d.lidar2img = reinterpret_cast<const float *>(base + L.mat_off);
    d.out = base + L.out_off;
    d.valid_count_out = p->valid_count_out ? reinterpret_cast<int32_t *>(base + L.cnt_off) : nullptr;
    const size_t feat_bytes =
        (size_t)p->B * p->N * p->feat_h * p->feat_w * p->C * (p->feat_dtype == FLASHBEV_F32 ? 4 : 2);
    if (cudaMemcpyAsync(base + L.feat_off, p->features, feat_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(base + L.mat_off, p->lidar2img, (size_t)p->B * p->N * 64, cudaMemcpyHostToDevice, stream) !=
            cudaSuccess) {
        cudaGetLastError();
        return FLASHBEV_CUDA_ERROR;
    }
    if ((st = run_device(&d, stream)) != FLASHBEV_OK) return st;
    if (cudaMemcpyAsync(p->out, base + L.out_off, (size_t)p->B * p->X * p->Y * p->C * 4, cudaMemcpyDeviceToHost, stream) !=
            cudaSuccess ||
        (p->valid_count_out && cudaMemcpyAsync(p->valid_count_out, base + L.cnt_off, (size_t)p->B * p->X * p->Y * 4,
                                               cudaMemcpyDeviceToHost, stream) != cudaSuccess)) {
        cudaGetLastError();
        return FLASHBEV_CUDA_ERROR;
    }
    return FLASHBEV_OK;
}

int flashbev_last_launch_count(void) { return t_last_launches; }
const char *flashbev_last_kernel_name(void) { return t_last_kernel; }

const char *flashbev_status_string(int status)
{
    switch (status) {
        case FLASHBEV_OK: return "ok";
        case FLASHBEV_INVALID_ARG: return "invalid argument";
        case FLASHBEV_UNSUPPORTED: return "unsupported configuration";
        case FLASHBEV_MISALIGNED: return "misaligned pointer";
        case FLASHBEV_CUDA_ERROR: return "CUDA error";
        case FLASHBEV_TOO_SMALL: return "staging buffer too small";
        default: return "unknown status";
    }
}

int flashbev_version(void) { return FLASHBEV_VERSION; }

}  // extern "C"
