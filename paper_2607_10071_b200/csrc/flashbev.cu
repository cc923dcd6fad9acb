// Fused Sampling-VT for B200 (sm_100a): kernels and the C ABI declared in flashbev.h.
//
// Two kernels compute the same operator (paper Eq. 1, fused as in Algorithm 2); a third, at the end of the
// kernel part, is the fused spatial cross-attention of Sec. 4.4:
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
//                         the list with 128- or 256-bit loads and fp32 FMAs.  Nothing but the output is
//                         written to global memory.
//
// Geometry (projection, validity, floor, fractions) is fp64, weights and accumulation fp32.
#include "flashbev.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <mutex>

namespace {

constexpr double kDepthMin = 0.1;   // metres: a sample needs camera depth > 0.1 m
constexpr int kMaxCams = 64;

struct KParams {
    const void *feat;
    const float *l2i;
    float *out;
    int32_t *count_out;
    const float *gout;          // backward: gradient of the output [B][X][Y][C]
    float *gfeat;               // backward: gradient of the features [B][N][Hf][Wf][C], fp32, pre-zeroed
    int B, N, C, Hf, Wf, X, Y, Z, reduce;
    int out_bf16;               // store the output as bfloat16 (round to nearest even) instead of float32
    int out_nchw;               // tiled kernel: scalar stores with the strides below (planar output, or ragged channels-last rows)
    int out_c;                  // ... channels of the output (the kernel's C may be padded)
    size_t out_bs, out_cells, out_chs;  // ... element strides of batch element, cell and channel
    int pdl;                    // host only: launch the forward with programmatic stream serialization
    int accumulate;             // add the result to the fp32 output instead of overwriting it (multi-resolution levels)
    double sx, sy;              // image px -> feature px
    double x_min, dx, y_min, dy, z_min, dz;
    // tiled kernel only
    int vecs;                   // 16-byte vectors per texel (C * elem / 16)
    int g;                      // lanes per cell
    int cpw;                    // cells per sub-block (= wx * wy <= 8): the cells one gather pass covers
    int wx, wy;                 // sub-block size in cells (x, y)
    int sbx, sby, sbn;          // sub-blocks per super-block (x, y, total)
    int ct;                     // cells per super-block (<= 32)
    float inv_n;                // 1 / N
    int blocks_x, blocks_y;     // super-blocks per batch element
    int band, reps;             // super-block order: bands of `band` rows; super-blocks per warp
    int nbands, centre_out;     // number of bands; visit them from the middle of the grid outwards
    int total_sbs;              // super-blocks in visiting order (bands * band * blocks_y)
    int whole_tasks;            // super-blocks (in visiting order) taken whole by one warp; the rest go one sub-block per warp
    int walk, walk_shift;       // height bins (or texel rows) per run: a power of two, 2 walk <= slots
    int inv_g;                  // ceil(65536 / g)
    int slots;                  // record slots per warp
    int colcap;                 // column descriptors per warp (>= cpw * N)
    int wcap;                   // runs per warp (= column descriptors per warp * ceil(Z / walk))
    int den_bytes;              // bytes of the per-(cell, height) camera counts per warp (Eq. 1 mode, else 0)
    int rstep;                  // distance (16-byte vectors) from a record's first tap to its second: vecs, or 0 on 1-texel-wide maps
    int nvec_cam;               // N * Hf * Wf * vecs: vectors of one batch element's feature maps (bounds-checked build)
    int wide;                   // host side: use the instance with adjacent channel vectors and 256-bit loads
    unsigned *err;              // bounds-checked build: device word that counts out-of-range indices (may be null)
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

// Index guard.  In the bounds-checked build (-DFLASHBEV_DEBUG_BOUNDS) every computed shared-memory slot, record
// offset and output index of the tiled kernel goes through this: an index outside [0, n) is counted into the
// caller's device word and replaced by 0, so the access that follows stays in range.  In the normal build it
// is the identity and costs nothing.
#ifdef FLASHBEV_DEBUG_BOUNDS
__device__ __forceinline__ int fb_idx(long long i, long long n, unsigned *err)
{
    if (i < 0 || i >= n) {
        if (err) atomicAdd(err, 1u);
        return 0;
    }
    return (int)i;
}
__device__ __forceinline__ size_t fb_idx64(size_t i, size_t n, unsigned *err)
{
    if (i >= n) {
        if (err) atomicAdd(err, 1u);
        return 0;
    }
    return i;
}
#define FB_IDX(i, n, err) fb_idx((long long)(i), (long long)(n), (err))
#define FB_IDX64(i, n, err) fb_idx64((size_t)(i), (size_t)(n), (err))
#else
#define FB_IDX(i, n, err) (i)
#define FB_IDX64(i, n, err) (i)
#endif

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

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo)) |
           ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi)) << 16);
}

__device__ __forceinline__ float load_elem(const float *p) { return __ldg(p); }
__device__ __forceinline__ float load_elem(const uint16_t *p)
{
    return __uint_as_float(((uint32_t)__ldg(p)) << 16);
}

// ------------------------------------------------------------------------------------------
// Kernel 1: one thread per (cell, group of VEC channels).  T = float or uint16_t (bf16 bits).
// SCALAR: the group's channels are loaded and stored one by one (any channel count, any alignment; the last group may
// be short); otherwise as one 16-byte vector.

template <typename T, int VEC, bool SCALAR = false>
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
                if (SCALAR) {
#pragma unroll
                    for (int i = 0; i < VEC; ++i)
                        if (c0 + i < p.C) num[i] = fmaf(w, load_elem(tp + i), num[i]);
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
            const float g = 1.f / (float)(den > 1 ? den : 1);  // mean over the cameras that see this height
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
    if (p.out_bf16) {
        uint16_t *o = reinterpret_cast<uint16_t *>(p.out) + (size_t)cell * p.C + c0;
        if (SCALAR) {
#pragma unroll
            for (int i = 0; i < VEC; ++i)
                if (c0 + i < p.C) o[i] = __bfloat16_as_ushort(__float2bfloat16_rn(acc[i]));
        } else {
#pragma unroll
            for (int i = 0; i < VEC; i += 4)
                *reinterpret_cast<uint2 *>(o + i) = make_uint2(pack_bf16x2(acc[i], acc[(i + 1) % VEC]),
                                                               pack_bf16x2(acc[(i + 2) % VEC], acc[(i + 3) % VEC]));
        }
    } else {
        float *o = p.out + (size_t)cell * p.C + c0;
        if (p.accumulate) {
#pragma unroll
            for (int i = 0; i < VEC; ++i)
                if (!SCALAR || c0 + i < p.C) acc[i] += o[i];
        }
        if (SCALAR) {
#pragma unroll
            for (int i = 0; i < VEC; ++i)
                if (c0 + i < p.C) o[i] = acc[i];
        } else {
#pragma unroll
            for (int i = 0; i < VEC; i += 4)
                __stcs(reinterpret_cast<float4 *>(o + i),
                       make_float4(acc[i], acc[(i + 1) % VEC], acc[(i + 2) % VEC], acc[(i + 3) % VEC]));
        }
    }
    if (p.count_out && c0 == 0) p.count_out[cell] = count;
}

// Kernel 1b: the same per-output decomposition for channel-planar tensors, features
// [B][N][C][Hf][Wf] and out [B][C][X][Y] (the layout the paper's own kernel works on, Sec. 4.1:
// C x Hf x Wf per camera).  One thread per (b, x, y, group of CH channels): the projection of a sample is shared by
// the CH channel planes a thread reads.  Threads are ordered with iy fastest so that stores and the taps of
// neighbouring cells coalesce.  Needs no scratch memory.
template <typename T, int CH>
__global__ void __launch_bounds__(256) vt_per_output_nchw_kernel(const KParams p)
{
    const int groups = (p.C + CH - 1) / CH;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= (long long)p.B * groups * p.X * p.Y) return;
    const int iy = (int)(gid % p.Y);
    const int ix = (int)((gid / p.Y) % p.X);
    const int c0 = (int)((gid / ((long long)p.X * p.Y)) % groups) * CH;
    const int b = (int)(gid / ((long long)p.X * p.Y * groups));
    const double xw = p.x_min + ((double)ix + 0.5) * p.dx;
    const double yw = p.y_min + ((double)iy + 0.5) * p.dy;
    const double wlim = (double)p.Wf - 0.5, hlim = (double)p.Hf - 0.5;
    const T *feat = static_cast<const T *>(p.feat);
    const size_t plane_elems = (size_t)p.Hf * p.Wf;
    float acc[CH];
#pragma unroll
    for (int j = 0; j < CH; ++j) acc[j] = 0.f;
    int count = 0;
    for (int k = 0; k < p.Z; ++k) {
        const double zw = p.z_min + ((double)k + 0.5) * p.dz;
        float num[CH];
#pragma unroll
        for (int j = 0; j < CH; ++j) num[j] = 0.f;
        int den = 0;
        for (int n = 0; n < p.N; ++n) {
            const float *M = p.l2i + ((size_t)b * p.N + n) * 16;
            const double p0 = fma((double)M[2], zw, fma((double)M[1], yw, fma((double)M[0], xw, (double)M[3])));
            const double p1 = fma((double)M[6], zw, fma((double)M[5], yw, fma((double)M[4], xw, (double)M[7])));
            const double d = fma((double)M[10], zw, fma((double)M[9], yw, fma((double)M[8], xw, (double)M[11])));
            Sample s;
            if (!project_sample(p0 * p.sx, p1 * p.sy, d, wlim, hlim, s)) continue;
            den += 1;
            const T *plane = feat + (((size_t)b * p.N + n) * p.C + c0) * plane_elems;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int xi = s.x0 + (t & 1), yi = s.y0 + (t >> 1);
                if (xi < 0 || xi > p.Wf - 1 || yi < 0 || yi > p.Hf - 1) continue;  // zero padding
                const float w = ((t & 1) ? s.tx : 1.f - s.tx) * ((t >> 1) ? s.ty : 1.f - s.ty);
                const T *tap = plane + (size_t)yi * p.Wf + xi;
#pragma unroll
                for (int j = 0; j < CH; ++j)
                    if (c0 + j < p.C) num[j] = fmaf(w, load_elem(tap + j * plane_elems), num[j]);
            }
        }
        count += den;
        const float inv = 1.f / (float)(den > 1 ? den : 1);
#pragma unroll
        for (int j = 0; j < CH; ++j) {
            if (p.reduce == FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM) acc[j] = fmaf(num[j], inv, acc[j]);
            else acc[j] += num[j];
        }
    }
    const float gn = p.reduce == FLASHBEV_REDUCE_MEAN_OVER_VALID ? 1.f / (float)(count > 1 ? count : 1) : 1.f;
    const size_t plane_out = (size_t)p.X * p.Y;
    const size_t o0 = ((size_t)b * p.C + c0) * plane_out + (size_t)ix * p.Y + iy;
#pragma unroll
    for (int j = 0; j < CH; ++j) {
        if (c0 + j >= p.C) break;
        float v = acc[j];
        if (p.reduce == FLASHBEV_REDUCE_MEAN_OVER_VALID) v *= gn;
        const size_t o = o0 + j * plane_out;
        if (p.out_bf16) reinterpret_cast<uint16_t *>(p.out)[o] = __bfloat16_as_ushort(__float2bfloat16_rn(v));
        else p.out[o] = p.accumulate ? v + p.out[o] : v;
    }
    if (p.count_out && c0 == 0) p.count_out[((size_t)b * p.X + ix) * p.Y + iy] = count;
}

// ------------------------------------------------------------------------------------------
// Kernel 2: tiled (forward and backward), see vt_tiled.cuh
#include "vt_tiled.cuh"

// ------------------------------------------------------------------------------------------
// Kernel 3: FlashSCA -- spatial cross-attention with on-the-fly projection (paper Sec. 4.4).  One warp per
// BEV query, three phases, all warp-local:
//   1. the lanes project the query's Zref reference heights into all cameras (fp64, the validity rule of
//      the Sampling-VT operator) and keep the normalised image positions and a per-camera visibility mask
//      in shared memory;
//   2. for every camera that sees the query, the lanes turn (head, level, point) triples -- read with
//      coalesced streaming loads in the order the offsets and weights are stored -- into tap records
//      {4 value indices, 4 weights} in shared memory: attention weight x bilinear weight, out-of-map taps
//      clamped to an in-map address with weight 0 (zero padding without predicates);
//   3. the lanes of a head (head_dim / 4 lanes, 16 bytes of the head's channels each) walk the head's
//      records: four 128-bit loads and packed fp32 FMAs per record.
// No per-camera, BEV-shaped tensor (reference points, masks, sampling locations) ever exists in memory.

constexpr int kScaMaxLevels = 8;
constexpr int kScaMaxChunkPoints = 32;  // sampling points per chunk (bit mask of visible points)

struct ScaParams {
    const uint4 *value;    // [B][N][T][16-byte vectors of the D channels], float32 or bfloat16
    const float *l2i;
    const float2 *offsets; // [B][Q][heads][L][P]
    const float *weights;  // [B][Q][heads][L][P]
    float4 *out;           // [B][Q][D / 4], float32
    int32_t *hits_out;
    int B, N, heads, Dh, L, P, X, Y, Zref, Himg, Wimg;
    int lph, hp;           // lanes per head, heads per pass
    int Pc, pitch;         // points per chunk; records per head in shared memory (L * Pc + 1)
    long long T;           // texels per camera (all levels)
    double x_min, dx, y_min, dy, z_min, dz;
    int Hl[kScaMaxLevels], Wl[kScaMaxLevels], lvl0[kScaMaxLevels];
};

// Shared memory of one warp: reference points, visibility masks, tap records (16 + 16 bytes each), the
// texel positions of the references of one camera (16 bytes per height x level) and two staging buffers
// for the (offset, weight) pairs of a chunk (8 + 4 bytes per head x level x point).
__host__ __device__ inline size_t sca_warp_smem(int N, int Zref, int heads, int pitch, int items, int L)
{
    return (size_t)N * Zref * sizeof(double2) + (((size_t)N * sizeof(uint32_t) + 15) & ~(size_t)15) +
           (size_t)heads * pitch * 32 + (size_t)Zref * L * 16 + 2 * (((size_t)items * 12 + 15) & ~(size_t)15);
}

__device__ __forceinline__ void cp_async_4(void *dst, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_8(void *dst, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// EVEN: every lane has a head in every pass (heads = V * heads per pass, 32 lanes all used)
template <int V, bool EVEN, bool BF16>
__global__ void __launch_bounds__(128, V <= 2 ? 5 : 3) sca_kernel(const ScaParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int max_items = p.heads * p.L * p.Pc;

    // ---- per-CTA table: item i = (head * L + level) * Pc + point  ->  head | level | point | point % Zref
    uint32_t *dec = reinterpret_cast<uint32_t *>(smem_raw);
    for (int i = threadIdx.x; i < max_items; i += blockDim.x) {
        const int hl = i / p.Pc, j = i - hl * p.Pc;
        const int h = hl / p.L, l = hl - h * p.L;
        dec[i] = ((uint32_t)h << 24) | ((uint32_t)l << 16) | ((uint32_t)(j % p.Zref) << 8) | (uint32_t)j;
    }
    __syncthreads();

    const unsigned Q = (unsigned)(p.X * p.Y);
    const unsigned gq = blockIdx.x * 4u + (unsigned)warp;  // query index over the batch (< 2^31, checked by the host)
    if (gq >= (unsigned)p.B * Q) return;
    const unsigned b = gq / Q, q = gq - b * Q;
    const int ix = (int)(q / (unsigned)p.Y), iy = (int)(q - (unsigned)ix * (unsigned)p.Y);
    const int nref = p.N * p.Zref;
    const int cap = p.heads * p.pitch;
    const size_t stage_bytes = ((size_t)max_items * 12 + 15) & ~(size_t)15;
    unsigned char *mine = smem_raw + (((size_t)max_items * 4 + 15) & ~(size_t)15) +
                          warp * sca_warp_smem(p.N, p.Zref, p.heads, p.pitch, max_items, p.L);
    double2 *ref = reinterpret_cast<double2 *>(mine);
    uint32_t *vm = reinterpret_cast<uint32_t *>(mine + (size_t)nref * sizeof(double2));
    uint4 *rec_i = reinterpret_cast<uint4 *>(mine + (size_t)nref * sizeof(double2) + (((size_t)p.N * 4 + 15) & ~(size_t)15));
    float4 *rec_w = reinterpret_cast<float4 *>(rec_i + cap);
    int4 *base_tab = reinterpret_cast<int4 *>(rec_w + cap);                       // [Zref][L]: texel position of a reference
    unsigned char *stage = reinterpret_cast<unsigned char *>(base_tab + p.Zref * p.L);  // [2][offsets | weights]

    const size_t qrow = ((size_t)b * Q + q) * (size_t)(p.heads * p.L);  // first (head, level) row of the query
    // asynchronous copy of one chunk's offsets and weights into item order
    const auto stage_chunk = [&](int pt0, int buf) {
        const int npc = min(p.Pc, p.P - pt0);
        float2 *so = reinterpret_cast<float2 *>(stage + buf * stage_bytes);
        float *sw = reinterpret_cast<float *>(so + max_items);
        for (int i = lane; i < max_items; i += 32) {
            const uint32_t t = dec[i];
            const int j = (int)(t & 0xffu);
            if (j >= npc) continue;
            const size_t sidx = (qrow + (t >> 24) * p.L + ((t >> 16) & 0xffu)) * p.P + pt0 + j;
            cp_async_8(so + i, p.offsets + sidx);
            cp_async_4(sw + i, p.weights + sidx);
        }
        cp_async_commit();
    };
    stage_chunk(0, 0);

    // ---- phase 1: reference points, (camera, height) pairs over the lanes
    for (int n = lane; n < p.N; n += 32) vm[n] = 0u;
    __syncwarp();
    const double xw = p.x_min + ((double)ix + 0.5) * p.dx, yw = p.y_min + ((double)iy + 0.5) * p.dy;
    for (int pr = lane; pr < nref; pr += 32) {
        const int n = pr / p.Zref, k = pr - n * p.Zref;
        const float *M = p.l2i + ((size_t)b * p.N + n) * 16;
        const double zw = p.z_min + ((double)k + 0.5) * p.dz;
        const double p0 = fma((double)__ldg(M + 2), zw, fma((double)__ldg(M + 1), yw, fma((double)__ldg(M), xw, (double)__ldg(M + 3))));
        const double p1 = fma((double)__ldg(M + 6), zw, fma((double)__ldg(M + 5), yw, fma((double)__ldg(M + 4), xw, (double)__ldg(M + 7))));
        const double d = fma((double)__ldg(M + 10), zw, fma((double)__ldg(M + 9), yw, fma((double)__ldg(M + 8), xw, (double)__ldg(M + 11))));
        const double r = fast_rcp(d);  // d <= 0 or NaN: every test below fails
        const double u = p0 * r, v = p1 * r;
        const bool ok = (d > kDepthMin) & (u > 0.0) & (u < (double)p.Wimg) & (v > 0.0) & (v < (double)p.Himg);
        ref[pr] = make_double2(u / (double)p.Wimg, v / (double)p.Himg);
        if (ok) atomicOr(&vm[n], 1u << k);
    }
    __syncwarp();
    int hits = 0;
    for (int n0 = 0; n0 < p.N; n0 += 32)
        hits += __popc(__ballot_sync(FULL, n0 + lane < p.N && vm[min(n0 + lane, p.N - 1)] != 0u));

    // ---- lanes -> (head, 16-byte slice of the head's channels)
    const int hsub = lane / p.lph, e4 = lane - hsub * p.lph;
    constexpr int PV = BF16 ? 4 : 2;  // channel pairs per 16-byte vector
    float2 acc[V][PV];
    bool on[V];
    int hrow[V];  // first record of the lane's head
#pragma unroll
    for (int v = 0; v < V; ++v) {
#pragma unroll
        for (int e = 0; e < PV; ++e) acc[v][e] = make_float2(0.f, 0.f);
        const int h = v * p.hp + hsub;
        on[v] = EVEN || (hsub < p.hp && h < p.heads);
        hrow[v] = (on[v] ? h : 0) * p.pitch;
    }
    const int D4 = p.heads * p.lph;  // 16-byte vectors per texel
    const int nbase = p.Zref * p.L;

    for (int pt0 = 0, c = 0; pt0 < p.P; pt0 += p.Pc, ++c) {
        const int npc = min(p.Pc, p.P - pt0);
        // the next chunk's offsets and weights travel while this one is worked on
        if (pt0 + p.Pc < p.P) {
            stage_chunk(pt0 + p.Pc, (c + 1) & 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncwarp();
        const float2 *so = reinterpret_cast<const float2 *>(stage + (c & 1) * stage_bytes);
        const float *sw = reinterpret_cast<const float *>(so + max_items);
        const int k0 = pt0 % p.Zref;
        const int klane = (pt0 + lane) % p.Zref;  // reference height of the chunk's point `lane`
        for (int n = 0; n < p.N; ++n) {
            const uint32_t mask = vm[n];
            if (mask == 0u) continue;  // warp-uniform: the camera does not see this query
            // visible points of the chunk: the reference height a point belongs to must be seen
            const uint32_t vis = __ballot_sync(FULL, lane < npc && ((mask >> klane) & 1u));
            if (vis == 0u) continue;
            const uint4 *vcam = p.value + ((size_t)b * p.N + n) * (size_t)p.T * D4 + e4;
            __syncwarp();  // the previous records and reference positions have been consumed
            // texel position of every visible reference on every level: integer part and fraction
            for (int e = lane; e < nbase; e += 32) {
                const int k = e / p.L, l = e - k * p.L;
                if (!((mask >> k) & 1u)) continue;
                const double2 rf = ref[n * p.Zref + k];  // inside (0, 1)^2
                const double bx = fma(rf.x, (double)p.Wl[l], -0.5), by = fma(rf.y, (double)p.Hl[l], -0.5);
                const double fbx = floor(bx), fby = floor(by);
                base_tab[e] = make_int4((int)fbx, (int)fby, __float_as_int((float)(bx - fbx)), __float_as_int((float)(by - fby)));
            }
            __syncwarp();
            // ---- phase 2: tap records, one (head, level, point) per lane and step
            for (int i = lane; i < max_items; i += 32) {
                const uint32_t t = dec[i];
                const int j = (int)(t & 0xffu);
                if (j >= npc || !((vis >> j) & 1u)) continue;
                const int h = (int)(t >> 24), l = (int)((t >> 16) & 0xffu);
                int k = (int)((t >> 8) & 0xffu) + k0;
                k = k >= p.Zref ? k - p.Zref : k;
                const float a = sw[i];
                const float2 of = so[i];
                const int4 bs = base_tab[k * p.L + l];
                const int Hl = p.Hl[l], Wl = p.Wl[l];
                // position = integer base + (fraction + offset); absurd offsets are clamped, their taps are all outside
                const float sx = fminf(fmaxf(__int_as_float(bs.z) + of.x, -65536.f), 65536.f);
                const float sy = fminf(fmaxf(__int_as_float(bs.w) + of.y, -65536.f), 65536.f);
                const float flx = floorf(sx), fly = floorf(sy);
                const float tx = sx - flx, ty = sy - fly;
                const int x0 = bs.x + (int)flx, y0 = bs.y + (int)fly;
                const bool inx0 = (unsigned)x0 < (unsigned)Wl, inx1 = (unsigned)(x0 + 1) < (unsigned)Wl;
                const bool iny0 = (unsigned)y0 < (unsigned)Hl, iny1 = (unsigned)(y0 + 1) < (unsigned)Hl;
                const int xa = min(max(x0, 0), Wl - 1), xb = min(max(x0 + 1, 0), Wl - 1);
                const int ya = min(max(y0, 0), Hl - 1), yb = min(max(y0 + 1, 0), Hl - 1);
                const float wx0 = a * (1.f - tx), wx1 = a * tx;
                float4 w;
                w.x = inx0 && iny0 ? wx0 * (1.f - ty) : 0.f;
                w.y = inx1 && iny0 ? wx1 * (1.f - ty) : 0.f;
                w.z = inx0 && iny1 ? wx0 * ty : 0.f;
                w.w = inx1 && iny1 ? wx1 * ty : 0.f;
                const uint32_t hoff = (uint32_t)(h * p.lph);
                const uint32_t ra = (uint32_t)(p.lvl0[l] + ya * Wl), rb = (uint32_t)(p.lvl0[l] + yb * Wl);
                uint4 ti;
                ti.x = (ra + xa) * D4 + hoff;
                ti.y = (ra + xb) * D4 + hoff;
                ti.z = (rb + xa) * D4 + hoff;
                ti.w = (rb + xb) * D4 + hoff;
                rec_i[i + h] = ti;  // = head * pitch + level * Pc + point
                rec_w[i + h] = w;
            }
            __syncwarp();
            // ---- phase 3: gather, every lane over the records of its heads
            for (int l = 0; l < p.L; ++l) {
                for (uint32_t m = vis; m; m &= m - 1u) {
                    const int slot = l * p.Pc + __ffs(m) - 1;
                    uint4 ti[V];
                    float4 tw[V];
                    uint4 s[V][4];
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        ti[v] = rec_i[hrow[v] + slot];
                        tw[v] = rec_w[hrow[v] + slot];
                    }
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        if (!on[v]) continue;
                        s[v][0] = __ldg(vcam + ti[v].x);
                        s[v][1] = __ldg(vcam + ti[v].y);
                        s[v][2] = __ldg(vcam + ti[v].z);
                        s[v][3] = __ldg(vcam + ti[v].w);
                    }
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        if (!on[v]) continue;
                        fma_vec<BF16>(acc[v], s[v][0], make_float2(tw[v].x, tw[v].x));
                        fma_vec<BF16>(acc[v], s[v][1], make_float2(tw[v].y, tw[v].y));
                        fma_vec<BF16>(acc[v], s[v][2], make_float2(tw[v].z, tw[v].z));
                        fma_vec<BF16>(acc[v], s[v][3], make_float2(tw[v].w, tw[v].w));
                    }
                }
            }
        }
    }
    const float g = 1.f / (float)(hits > 1 ? hits : 1);
#pragma unroll
    for (int v = 0; v < V; ++v) {
        if (!on[v]) continue;
        // the lane's 16-byte vector of values is PV / 2 float4 of output
        float4 *o = p.out + (((size_t)b * Q + q) * D4 + (v * p.hp + hsub) * p.lph + e4) * (PV / 2);
#pragma unroll
        for (int e = 0; e < PV; e += 2)
            __stcs(o + e / 2, make_float4(acc[v][e].x * g, acc[v][e].y * g, acc[v][e + 1].x * g, acc[v][e + 1].y * g));
    }
    if (p.hits_out && lane == 0) p.hits_out[gq] = hits;
}

// ------------------------------------------------------------------------------------------
// Channel-planar features [planes][C][HW] -> channels last [planes][HW][C] (T: 2- or 4-byte elements), through a
// padded shared-memory tile: reads run along HW, writes along C.
template <typename T>
__global__ void __launch_bounds__(256) nchw_to_nhwc_kernel(const T *__restrict__ in, T *__restrict__ out, int C, int HW)
{
    __shared__ T tile[32][33];
    const size_t plane = (size_t)blockIdx.z * C * HW;
    const int hw0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int c = c0 + j, hw = hw0 + threadIdx.x;
        if (c < C && hw < HW) tile[j][threadIdx.x] = in[plane + (size_t)c * HW + hw];
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int hw = hw0 + j, c = c0 + threadIdx.x;
        if (c < C && hw < HW) out[plane + (size_t)hw * C + c] = tile[threadIdx.x][j];
    }
}

// Channels-last rows of C elements -> rows of Cpad >= C elements, the tail zero (T: 2- or 4-byte elements).
template <typename T>
__global__ void __launch_bounds__(256) pad_channels_kernel(const T *__restrict__ in, T *__restrict__ out, long long rows, int C, int Cpad)
{
    const long long total = rows * Cpad;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / Cpad;
        const int c = (int)(i - r * Cpad);
        out[i] = c < C ? in[r * C + c] : T(0);
    }
}

// ------------------------------------------------------------------------------------------
// host side

thread_local int t_last_launches = 0;
thread_local const char *t_last_kernel = "none";

// The optional device word of the bounds-checked build (absent in structs of callers built against an older header).
unsigned *debug_word(const flashbev_vt_params *p)
{
    return p->struct_size >= sizeof(flashbev_vt_params) ? p->debug_error_word : nullptr;
}

// A full-size copy of a caller's struct, which may be shorter (older header): missing fields are zero.
flashbev_vt_params copy_params(const flashbev_vt_params *p)
{
    flashbev_vt_params c;
    memset(&c, 0, sizeof(c));
    memcpy(&c, p, std::min(p->struct_size, sizeof(c)));
    c.struct_size = sizeof(c);
    return c;
}

bool params_ok(const flashbev_vt_params *p, flashbev_status &st)
{
    st = FLASHBEV_INVALID_ARG;
    if (!p || p->struct_size < offsetof(flashbev_vt_params, debug_error_word)) return false;  // (older headers end there)
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
    const size_t oelem = p->out_dtype == FLASHBEV_F32 ? 4 : 2;
    if (((uintptr_t)p->features % elem) || ((uintptr_t)p->out % oelem) || ((uintptr_t)p->lidar2img % 4)) return FLASHBEV_MISALIGNED;
    if (p->valid_count_out && ((uintptr_t)p->valid_count_out % 4)) return FLASHBEV_MISALIGNED;
    if (debug_word(p) && ((uintptr_t)debug_word(p) % 4)) return FLASHBEV_MISALIGNED;
    return FLASHBEV_OK;
}

KParams base_params(const flashbev_vt_params *p, bool accumulate = false)
{
    KParams k = {};
    k.accumulate = accumulate;
    k.feat = p->features;
    k.l2i = p->lidar2img;
    k.out = static_cast<float *>(p->out);
    k.count_out = p->valid_count_out;
    k.B = p->B, k.N = p->N, k.C = p->C, k.Hf = p->feat_h, k.Wf = p->feat_w;
    k.X = p->X, k.Y = p->Y, k.Z = p->Z, k.reduce = p->reduce;
    k.out_bf16 = p->out_dtype == FLASHBEV_BF16;
    k.err = debug_word(p);
    k.sx = (double)p->feat_w / (double)p->img_w;
    k.sy = (double)p->feat_h / (double)p->img_h;
    k.x_min = p->x_min, k.dx = (p->x_max - p->x_min) / (double)p->X;
    k.y_min = p->y_min, k.dy = (p->y_max - p->y_min) / (double)p->Y;
    k.z_min = p->z_min, k.dz = (p->z_max - p->z_min) / (double)p->Z;
    return k;
}

flashbev_status launch_per_output(const flashbev_vt_params *p, cudaStream_t stream, bool accumulate = false)
{
    const KParams k = base_params(p, accumulate);
    const bool bf16 = p->feat_dtype == FLASHBEV_BF16;
    if (p->layout == FLASHBEV_NCHW) {
        constexpr int CH = 8;  // channel planes per thread
        const long long threads = (long long)p->B * ((p->C + CH - 1) / CH) * p->X * p->Y;
        const long long blocks = (threads + 255) / 256;
        if (blocks > 2147483647LL) return FLASHBEV_UNSUPPORTED;
        if (bf16) vt_per_output_nchw_kernel<uint16_t, CH><<<dim3((unsigned)blocks), dim3(256), 0, stream>>>(k);
        else vt_per_output_nchw_kernel<float, CH><<<dim3((unsigned)blocks), dim3(256), 0, stream>>>(k);
        t_last_kernel = bf16 ? "per_output_nchw_bf16" : "per_output_nchw_f32";
        return FLASHBEV_OK;
    }
    const int vec = bf16 ? 8 : 4;
    const bool vec_ok = (p->C % vec == 0) && ((uintptr_t)p->features % 16 == 0) && ((uintptr_t)p->out % 16 == 0);
    constexpr int kScalarGroup = 4;  // channels per thread when they are loaded one by one
    const int per_thread = vec_ok ? vec : kScalarGroup;
    const long long threads = (long long)p->B * p->X * p->Y * ((p->C + per_thread - 1) / per_thread);
    const long long blocks = (threads + 255) / 256;
    if (blocks > 2147483647LL) return FLASHBEV_UNSUPPORTED;
    const dim3 grid((unsigned)blocks), block(256);
    if (bf16 && vec_ok) {
        vt_per_output_kernel<uint16_t, 8><<<grid, block, 0, stream>>>(k);
        t_last_kernel = "per_output_bf16x8";
    } else if (bf16) {
        vt_per_output_kernel<uint16_t, kScalarGroup, true><<<grid, block, 0, stream>>>(k);
        t_last_kernel = "per_output_bf16x1";
    } else if (vec_ok) {
        vt_per_output_kernel<float, 4><<<grid, block, 0, stream>>>(k);
        t_last_kernel = "per_output_f32x4";
    } else {
        vt_per_output_kernel<float, kScalarGroup, true><<<grid, block, 0, stream>>>(k);
        t_last_kernel = "per_output_f32x1";
    }
    return FLASHBEV_OK;
}

// Number of SMs of the current device (cached per device; 148 on a B200).
int sm_count()
{
    static std::atomic<int> cached[64];  // 0: not asked yet (concurrent callers may both ask: same answer)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return 148;
    }
    int n = cached[dev].load(std::memory_order_relaxed);
    if (!n) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            n = 148;
        }
        cached[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

// Shapes the tiled kernel serves (whatever the layout): channel rows of whole 16-byte vectors, bounded Z and map size.
bool tiled_shape_ok(const flashbev_vt_params *p)
{
    const size_t elem = p->feat_dtype == FLASHBEV_F32 ? 4 : 2;
    if (((size_t)p->C * elem) % 16) return false;
    if (p->Z > 32767) return false;  // a column's interval of height bins is kept in two 16-bit fields
    if (p->reduce == FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM && p->Z > 16384) return false;  // per-height camera counts on chip
    const double vecs_total = (double)p->N * p->feat_h * p->feat_w * (double)((size_t)p->C * elem / 16);
    return vecs_total < 2147483648.0;
}

bool tiled_applicable(const flashbev_vt_params *p)
{
    if (p->layout != FLASHBEV_NHWC) return false;
    if (((uintptr_t)p->features % 16) || ((uintptr_t)p->out % 16)) return false;
    return tiled_shape_ok(p);
}

// Bytes of the channels-last copy of NCHW features (0: the shape cannot take the tiled kernel).
size_t nchw_copy_bytes(const flashbev_vt_params *p)
{
    if (p->layout != FLASHBEV_NCHW || !tiled_shape_ok(p)) return 0;
    return (size_t)p->B * p->N * p->feat_h * p->feat_w * p->C * (p->feat_dtype == FLASHBEV_F32 ? 4 : 2);
}

// NCHW tensors with a workspace that holds the channels-last copy: transposing copy, then the tiled kernel.
bool nchw_tiled_applicable(const flashbev_vt_params *p)
{
    if (p->struct_size < sizeof(flashbev_vt_params) || !p->workspace) return false;
    const size_t need = nchw_copy_bytes(p);
    return need && p->workspace_bytes >= need && (uintptr_t)p->workspace % 16 == 0 &&
           (long long)p->B * p->N <= 65535 && (p->C + 31) / 32 <= 65535;
}

// Channels-last tensors whose rows are not whole 16-byte vectors: channels rounded up to the next whole vector.
int padded_channels(const flashbev_vt_params *p)
{
    const int vec = p->feat_dtype == FLASHBEV_F32 ? 4 : 8;
    return (p->C + vec - 1) / vec * vec;
}

// Bytes of the padded copy of such features (0: not that case, or the padded shape cannot take the tiled kernel).
size_t pad_copy_bytes(const flashbev_vt_params *p)
{
    const size_t elem = p->feat_dtype == FLASHBEV_F32 ? 4 : 2;
    if (p->layout != FLASHBEV_NHWC || ((size_t)p->C * elem) % 16 == 0) return 0;
    flashbev_vt_params q = copy_params(p);
    q.C = padded_channels(p);
    if (!tiled_shape_ok(&q)) return 0;
    return (size_t)p->B * p->N * p->feat_h * p->feat_w * q.C * elem;
}

bool padded_tiled_applicable(const flashbev_vt_params *p)
{
    if (p->struct_size < sizeof(flashbev_vt_params) || !p->workspace) return false;
    const size_t need = pad_copy_bytes(p);
    return need && p->workspace_bytes >= need && (uintptr_t)p->workspace % 16 == 0;
}

template <int V, bool BF16, int WARPS, bool BWD, bool WIDE = false, bool PLANAR = false>
cudaError_t launch_tiled_inst(const KParams &k, dim3 grid, size_t smem, cudaStream_t stream)
{
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(vt_tiled_kernel<V, BF16, WARPS, BWD, WIDE, PLANAR>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    if (!BWD && k.pdl) {
        // forward launches may overlap their start with the end of the kernel before them in the stream (the kernel
        // waits for that kernel's completion before it reads or writes global memory)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = grid, cfg.blockDim = dim3(WARPS * 32), cfg.dynamicSmemBytes = smem, cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr, cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, vt_tiled_kernel<V, BF16, WARPS, BWD, WIDE, PLANAR>, k);
    }
    vt_tiled_kernel<V, BF16, WARPS, BWD, WIDE, PLANAR><<<grid, dim3(WARPS * 32), smem, stream>>>(k);
    return cudaSuccess;
}

template <int V, bool BF16>
cudaError_t launch_tiled_warps(int warps, const KParams &k, dim3 grid, size_t smem, cudaStream_t stream)
{
    switch (warps) {
        case 1: return launch_tiled_inst<V, BF16, 1, false>(k, grid, smem, stream);
        case 2: return launch_tiled_inst<V, BF16, 2, false>(k, grid, smem, stream);
        case 8: return launch_tiled_inst<V, BF16, 8, false>(k, grid, smem, stream);
        default:
            if (k.out_nchw) {  // (planar output: instances for 4 warps per CTA only)
                if (V >= 2 && k.wide) return launch_tiled_inst<V, BF16, 4, false, (V >= 2), true>(k, grid, smem, stream);
                return launch_tiled_inst<V, BF16, 4, false, false, true>(k, grid, smem, stream);
            }
            if (V >= 2 && k.wide) return launch_tiled_inst<V, BF16, 4, false, (V >= 2)>(k, grid, smem, stream);
            return launch_tiled_inst<V, BF16, 4, false>(k, grid, smem, stream);
    }
}

// Chooses the channel mapping, super-block shape, run length, list size and grid of the tiled kernel.
flashbev_status configure_tiled(const flashbev_vt_params *p, KParams &k, int &V, int &warps, dim3 &grid, size_t &smem,
                                bool accumulate = false)
{
    k = base_params(p, accumulate);
    const bool bf16 = p->feat_dtype == FLASHBEV_BF16;
    const int elem = bf16 ? 2 : 4;
    const bool eq1 = p->reduce == FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM;
    k.vecs = p->C * elem / 16;
    k.rstep = p->feat_w > 1 ? k.vecs : 0;
    k.nvec_cam = p->N * p->feat_h * p->feat_w * k.vecs;  // < 2^31: tiled_applicable
    k.inv_n = 1.0f / (float)p->N;

    // channel mapping: V vectors per lane, g lanes per cell
    V = p->tune[0];
    int g = p->tune[1];
    if (!(V == 1 || V == 2 || V == 4) || g < 1 || g > 32) V = 0, g = 0;
    if (!V) {
        // (measured) up to 8 vectors per texel: one per lane; up to 32: two adjacent ones per lane; beyond: four.
        if (k.vecs <= 8) V = 1, g = k.vecs;
        else if (k.vecs <= 32) V = (k.vecs % 2 == 0 || k.vecs > 16) ? 2 : 1, g = (k.vecs + V - 1) / V;
        else V = 4, g = (k.vecs + 3) / 4;
        if (g > 32) g = 32;
    }
    warps = p->tune[3] & 0xf;
    if (!(warps == 1 || warps == 2 || warps == 4 || warps == 8)) warps = 4;
    k.g = g;
    k.inv_g = (65536 + g - 1) / g;
    int cpw = std::min(32 / g, kMaxCpw);
    cpw = std::min(cpw, std::max(1, kColCapMax / p->N));  // a sub-block's candidate columns fit the descriptor table
    // sub-block of wx x wy cells, near-square, y (the contiguous output axis) the longer side
    k.wy = (cpw % 2 == 0) ? 2 : (cpw == 3 ? 3 : 1);
    if (cpw == 8) k.wy = 4;
    if (cpw == 6) k.wy = 3;
    if (cpw == 5 || cpw == 7) k.wy = cpw;
    k.wx = cpw / k.wy;
    k.cpw = k.wx * k.wy;

    // record slots per warp and bins per run (a run writes at most two records per bin)
    const int slots_tune = (p->tune[3] >> 20) & 0xff;
    k.slots = slots_tune ? std::max(64, slots_tune * 16) : 512;
    // a run is at most `walk` height bins, or `walk` texel rows of a column that moves at most two rows per bin
    const int units = std::max(p->Z, std::min(p->feat_h, 2 * p->Z + 2));  // per column at most
    k.walk = (p->tune[2] >= 1 && p->tune[2] <= 256) ? p->tune[2] : 16;
    // (the rounds of a sub-block whose records exceed the slots need 2 walk (cells + 1) <= slots)
    k.walk = std::max(1, std::min(k.walk, std::min(units, k.slots / (2 * (k.cpw + 1)))));
    k.colcap = std::max(32, (k.cpw * p->N + 7) / 8 * 8);
    for (k.walk_shift = 0; (2 << k.walk_shift) <= k.walk; ++k.walk_shift) {}
    k.walk = 1 << k.walk_shift;
    int runs = (units + k.walk - 1) / k.walk;
    while (k.colcap * runs > 2048 && 2 * k.walk <= std::min(256, k.slots / (2 * (k.cpw + 1)))) {  // keep the run table small: longer runs
        k.walk *= 2, k.walk_shift += 1;
        runs = (units + k.walk - 1) / k.walk;
    }

    // super-block: about as many cells as fill the record slots in one round (a cell writes roughly 0.7 Z + 8
    // records on surround rigs), so that the walkers of a round keep most lanes busy
    int sbx = (p->tune[3] >> 4) & 0xf, sby = (p->tune[3] >> 8) & 0xf;
    auto fits = [&](int nx, int ny) {
        const int ct = nx * ny * k.cpw;
        if (ct > kMaxCt || ct * p->N > 512) return false;
        if (eq1 && (long long)ct * p->Z > 16384) return false;
        return true;
    };
    if (sbx < 1 || sby < 1 || !fits(sbx, sby)) {
        // (from sweeps) about 10-16 cells per warp -- enough columns to keep the geometry lanes busy -- but fewer if
        // that leaves the SMs less than three rounds of warps, never more than the record slots hold in four rounds
        // (a cell writes roughly 1.2 Z + 12 records on surround rigs; rounds hold whole sub-blocks, and columns of
        // 32-256 bins gain more from full geometry lanes than they lose to further rounds: 20-30 % measured) and
        // never fewer warps than the SMs can hold.
        static const int shapes[][2] = {{1, 1}, {1, 2}, {2, 2}, {2, 3}, {2, 4}, {3, 3}, {3, 4}, {4, 4}};
        const long long cells = (long long)p->B * p->X * p->Y, warp_slots = (long long)sm_count() * 20;
        double want = std::min(16.0, std::max(10.0, (double)cells / (3.0 * warp_slots)));
        want = std::min(want, (double)cells / warp_slots);
        const double rounds = p->Z <= 5 * p->feat_h ? 4.0 : 1.0;  // (very tall columns: the walkers dominate, one round is better)
        want = std::min(want, rounds * k.slots / (1.2 * std::min(p->Z, 2 * p->feat_h) + 12.0));
        sbx = sby = 1;
        double best = 1e30;
        for (const auto &sh : shapes) {
            const int ct = sh[0] * sh[1] * k.cpw;
            if (!fits(sh[0], sh[1])) break;
            const double miss = ct > want ? ct - want : want - ct;
            if (miss < best) best = miss, sbx = sh[0], sby = sh[1];
        }
    }
    if (!fits(sbx, sby)) return FLASHBEV_UNSUPPORTED;
    k.sbx = sbx, k.sby = sby, k.sbn = sbx * sby;
    k.ct = k.sbn * k.cpw;
    k.blocks_x = (p->X + sbx * k.wx - 1) / (sbx * k.wx);
    k.blocks_y = (p->Y + sby * k.wy - 1) / (sby * k.wy);
    { const int bc = (p->tune[3] >> 18) & 3; k.band = bc == 1 ? 1 : (bc == 2 ? 4 : (bc == 3 ? 8 : 2)); }
    k.reps = (p->tune[3] >> 12) & 0xf;
    if (k.reps < 1) k.reps = 1;
    k.wcap = k.colcap * runs;
    k.den_bytes = eq1 ? (int)align16((size_t)k.ct * p->Z) : 0;

    const long long bands = (k.blocks_x + k.band - 1) / k.band;
    k.nbands = (int)bands;
    k.centre_out = !((p->tune[3] >> 28) & 1);
    const long long sbs = bands * k.band * k.blocks_y;  // super-blocks in visiting order (those past the grid's edge do nothing)
    // the tail of the order is split into single sub-blocks: about one warp's worth per resident warp slot
    // (0 = default: one short task per resident warp slot when a super-block has four or more sub-blocks)
    static const double tail_factor[8] = {-1.0, 0.0, 0.25, 0.5, 1.0, 1.5, 2.0, 3.0};
    double tf = tail_factor[((unsigned)p->tune[3] >> 29) & 7];
    if (tf < 0.0) tf = k.sbn >= 4 ? 1.0 : 0.0;
    long long tail = k.sbn > 1 ? std::min<long long>(sbs, (long long)(sm_count() * 20 * tf) / k.sbn) : 0;
    if (k.reps > 1) tail = 0;
    k.total_sbs = (int)sbs;
    k.whole_tasks = (int)(sbs - tail);
    const long long ids = (sbs - tail) + tail * k.sbn;
    const long long ctas = (ids + (long long)warps * k.reps - 1) / ((long long)warps * k.reps);
    const int cblocks = (k.vecs + g * V - 1) / (g * V);
    if (ctas > 2147483647LL || ids + (long long)warps * k.reps >= 2147483647LL || cblocks > 65535 || p->B > 65535)
        return FLASHBEV_UNSUPPORTED;  // (task ids are 32-bit in the kernel)
    grid = dim3((unsigned)ctas, (unsigned)cblocks, (unsigned)p->B);
    // adjacent vectors and 256-bit loads: half the load instructions (bf16 features are issue-bound), and whole
    // texels per cell where the strided 16-byte segments of a cell would not cover whole 128-byte lines
    k.wide = warps == 4 && (V == 2 || (V == 4 && (p->tune[3] & 0x20000))) && k.vecs % V == 0 && (uintptr_t)p->features % 32 == 0 &&
             (bf16 || (g * 16) % 128 != 0 || (p->tune[3] & 0x20000)) && !(p->tune[3] & 0x10000);
    smem = align16(cta_table_bytes(p->N)) +
           (size_t)warps * warp_smem_layout(nullptr, nullptr, k.slots, k.colcap, k.wcap, k.ct, k.ct * p->N, k.den_bytes);
    if (smem > 200 * 1024) return FLASHBEV_UNSUPPORTED;
    return FLASHBEV_OK;
}

// scalar_out: 0 vector stores into channels-last rows; 1 planar output [B][C][X][Y]; 2 channels-last rows of out_c
// channels (the kernel's own C is padded)
flashbev_status launch_tiled(const flashbev_vt_params *p, cudaStream_t stream, bool accumulate = false, int scalar_out = 0,
                             int out_c = 0)
{
    KParams k;
    int V, warps;
    dim3 grid;
    size_t smem;
    const flashbev_status st = configure_tiled(p, k, V, warps, grid, smem, accumulate);
    if (st != FLASHBEV_OK) return st;
    k.out_nchw = scalar_out != 0;
    {
        const size_t plane = (size_t)p->X * p->Y;
        if (scalar_out == 1) k.out_c = p->C, k.out_bs = plane * p->C, k.out_cells = 1, k.out_chs = plane;
        if (scalar_out == 2) k.out_c = out_c, k.out_bs = plane * out_c, k.out_cells = out_c, k.out_chs = 1;
    }
    k.pdl = getenv("FLASHBEV_NO_PDL") ? 0 : 1;
    const bool bf16 = p->feat_dtype == FLASHBEV_BF16;
    cudaError_t e;
    static const char *const names[2][3] = {{"tiled_f32_v1", "tiled_f32_v2", "tiled_f32_v4"},
                                            {"tiled_bf16_v1", "tiled_bf16_v2", "tiled_bf16_v4"}};
    if (bf16) {
        if (V == 1) e = launch_tiled_warps<1, true>(warps, k, grid, smem, stream);
        else if (V == 2) e = launch_tiled_warps<2, true>(warps, k, grid, smem, stream);
        else e = launch_tiled_warps<4, true>(warps, k, grid, smem, stream);
    } else {
        if (V == 1) e = launch_tiled_warps<1, false>(warps, k, grid, smem, stream);
        else if (V == 2) e = launch_tiled_warps<2, false>(warps, k, grid, smem, stream);
        else e = launch_tiled_warps<4, false>(warps, k, grid, smem, stream);
    }
    t_last_kernel = names[bf16 ? 1 : 0][V == 1 ? 0 : (V == 2 ? 1 : 2)];
    return e == cudaSuccess ? FLASHBEV_OK : FLASHBEV_CUDA_ERROR;
}

// NCHW tensors on the tiled kernel: features -> channels-last copy in the workspace, output written planar.
flashbev_status launch_nchw_tiled(const flashbev_vt_params *p, cudaStream_t stream, bool accumulate)
{
    flashbev_vt_params q = *p;
    q.features = p->workspace;
    q.layout = FLASHBEV_NHWC;
    q.tune[3] = (q.tune[3] & ~0xf) | 4;  // the planar-output instances are built for 4 warps per CTA
    {   // configure first: nothing is enqueued for a shape the tiled kernel cannot take
        KParams k;
        int V, warps;
        dim3 grid;
        size_t smem;
        const flashbev_status st = configure_tiled(&q, k, V, warps, grid, smem, accumulate);
        if (st != FLASHBEV_OK) return st;
    }
    const int HW = p->feat_h * p->feat_w;
    const dim3 grid((unsigned)((HW + 31) / 32), (unsigned)((p->C + 31) / 32), (unsigned)(p->B * p->N)), block(32, 8);
    if (p->feat_dtype == FLASHBEV_BF16)
        nchw_to_nhwc_kernel<uint16_t><<<grid, block, 0, stream>>>(static_cast<const uint16_t *>(p->features),
                                                                  static_cast<uint16_t *>(p->workspace), p->C, HW);
    else
        nchw_to_nhwc_kernel<float><<<grid, block, 0, stream>>>(static_cast<const float *>(p->features),
                                                               static_cast<float *>(p->workspace), p->C, HW);
    if (cudaGetLastError() != cudaSuccess) return FLASHBEV_CUDA_ERROR;
    const flashbev_status st = launch_tiled(&q, stream, accumulate, 1);
    if (st == FLASHBEV_OK) t_last_kernel = p->feat_dtype == FLASHBEV_BF16 ? "tiled_bf16_nchw" : "tiled_f32_nchw";
    return st;
}

// Ragged channels-last tensors on the tiled kernel: features -> zero-padded copy in the workspace, output written
// one channel at a time into the caller's rows.
flashbev_status launch_padded_tiled(const flashbev_vt_params *p, cudaStream_t stream, bool accumulate)
{
    flashbev_vt_params q = *p;
    q.features = p->workspace;
    q.C = padded_channels(p);
    q.tune[3] = (q.tune[3] & ~0xf) | 4;  // the scalar-store instances are built for 4 warps per CTA
    {
        KParams k;
        int V, warps;
        dim3 grid;
        size_t smem;
        const flashbev_status st = configure_tiled(&q, k, V, warps, grid, smem, accumulate);
        if (st != FLASHBEV_OK) return st;
    }
    const long long rows = (long long)p->B * p->N * p->feat_h * p->feat_w;
    const unsigned blocks = (unsigned)std::min<long long>((rows * q.C + 255) / 256, 148LL * 32);
    if (p->feat_dtype == FLASHBEV_BF16)
        pad_channels_kernel<uint16_t><<<blocks, 256, 0, stream>>>(static_cast<const uint16_t *>(p->features),
                                                                  static_cast<uint16_t *>(p->workspace), rows, p->C, q.C);
    else
        pad_channels_kernel<float><<<blocks, 256, 0, stream>>>(static_cast<const float *>(p->features),
                                                               static_cast<float *>(p->workspace), rows, p->C, q.C);
    if (cudaGetLastError() != cudaSuccess) return FLASHBEV_CUDA_ERROR;
    const flashbev_status st = launch_tiled(&q, stream, accumulate, 2, p->C);
    if (st == FLASHBEV_OK) t_last_kernel = p->feat_dtype == FLASHBEV_BF16 ? "tiled_bf16_padded" : "tiled_f32_padded";
    return st;
}

flashbev_status run_device(const flashbev_vt_params *p, cudaStream_t stream, bool accumulate = false)
{
    flashbev_status st;
    if (p->layout == FLASHBEV_NHWC && p->kernel != FLASHBEV_KERNEL_PER_OUTPUT && padded_tiled_applicable(p)) {
        st = launch_padded_tiled(p, stream, accumulate);
        if (st == FLASHBEV_OK) {
            if (cudaGetLastError() != cudaSuccess) return FLASHBEV_CUDA_ERROR;
            t_last_launches = 2;
            return FLASHBEV_OK;
        }
        if (!(st == FLASHBEV_UNSUPPORTED && p->kernel == FLASHBEV_KERNEL_AUTO)) return st;
    }
    if (p->layout == FLASHBEV_NCHW) {
        const bool can = nchw_tiled_applicable(p);
        if (p->kernel == FLASHBEV_KERNEL_TILED && !can) return FLASHBEV_UNSUPPORTED;
        if (can && p->kernel != FLASHBEV_KERNEL_PER_OUTPUT) {
            st = launch_nchw_tiled(p, stream, accumulate);
            if (st == FLASHBEV_OK) {
                if (cudaGetLastError() != cudaSuccess) return FLASHBEV_CUDA_ERROR;
                t_last_launches = 2;
                return FLASHBEV_OK;
            }
            if (!(st == FLASHBEV_UNSUPPORTED && p->kernel == FLASHBEV_KERNEL_AUTO)) return st;
        }
        if ((st = launch_per_output(p, stream, accumulate)) != FLASHBEV_OK) return st;
        if (cudaGetLastError() != cudaSuccess) return FLASHBEV_CUDA_ERROR;
        t_last_launches = 1;
        return FLASHBEV_OK;
    }
    const bool tiled = p->kernel == FLASHBEV_KERNEL_TILED || (p->kernel == FLASHBEV_KERNEL_AUTO && tiled_applicable(p));
    if (tiled && !tiled_applicable(p)) return FLASHBEV_UNSUPPORTED;
    st = tiled ? launch_tiled(p, stream, accumulate) : launch_per_output(p, stream, accumulate);
    // AUTO: shapes the tiled kernel cannot be configured for (nothing was launched) go to the generic kernel
    if (tiled && st == FLASHBEV_UNSUPPORTED && p->kernel == FLASHBEV_KERNEL_AUTO) st = launch_per_output(p, stream, accumulate);
    if (st != FLASHBEV_OK) return st;
    if (cudaGetLastError() != cudaSuccess) return FLASHBEV_CUDA_ERROR;
    t_last_launches = 1;
    return FLASHBEV_OK;
}

struct StagingLayout {
    size_t feat_off, mat_off, out_off, cnt_off, total;
    size_t ws_off, ws_bytes, total_with_ws;  // NCHW tensors: room for the channels-last copy behind the rest (optional)
};

// False if the staging area of this problem would not fit 2^62 bytes (the byte counts below would wrap).
bool staging_layout(const flashbev_vt_params *p, StagingLayout &s)
{
    const size_t elem = p->feat_dtype == FLASHBEV_F32 ? 4 : 2;
    const double feat = (double)p->B * p->N * p->feat_h * p->feat_w * p->C * (double)elem;
    const double out = (double)p->B * p->X * p->Y * p->C * 4.0;
    if (!(feat + out + (double)p->B * p->N * 64.0 + (double)p->B * p->X * p->Y * 4.0 < 4.0e18)) return false;
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    s.feat_off = 0;
    s.mat_off = up((size_t)p->B * p->N * p->feat_h * p->feat_w * p->C * elem);
    s.out_off = s.mat_off + up((size_t)p->B * p->N * 64);
    s.cnt_off = s.out_off + up((size_t)p->B * p->X * p->Y * p->C * (p->out_dtype == FLASHBEV_F32 ? 4 : 2));
    s.total = s.cnt_off + (p->valid_count_out ? up((size_t)p->B * p->X * p->Y * 4) : 0);
    s.ws_off = s.total, s.ws_bytes = p->layout == FLASHBEV_NCHW ? nchw_copy_bytes(p) : pad_copy_bytes(p);
    s.total_with_ws = s.total + up(s.ws_bytes);
    return true;
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
    flashbev_status st;
    if (!params_ok(p, st)) return 0;
    return p->layout == FLASHBEV_NCHW ? nchw_copy_bytes(p) : pad_copy_bytes(p);
}

size_t flashbev_host_staging_bytes(const flashbev_vt_params *p)
{
    flashbev_status st;
    if (!params_ok(p, st)) return 0;
    StagingLayout L;
    return staging_layout(p, L) ? L.total_with_ws : 0;
}

flashbev_status flashbev_sampling_vt_host(const flashbev_vt_params *p, void *d_staging, size_t staging_bytes,
                                          void *stream_)
{
    flashbev_status st;
    if (!params_ok(p, st)) return st;
    if (!d_staging) return FLASHBEV_INVALID_ARG;
    if ((uintptr_t)d_staging % 256) return FLASHBEV_MISALIGNED;
    StagingLayout L;
    if (!staging_layout(p, L)) return FLASHBEV_UNSUPPORTED;
    if (staging_bytes < L.total) return FLASHBEV_TOO_SMALL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    unsigned char *base = static_cast<unsigned char *>(d_staging);
    flashbev_vt_params d = copy_params(p);
    d.features = base + L.feat_off;
    d.lidar2img = reinterpret_cast<const float *>(base + L.mat_off);
    d.out = base + L.out_off;
    d.valid_count_out = p->valid_count_out ? reinterpret_cast<int32_t *>(base + L.cnt_off) : nullptr;
    d.workspace = nullptr, d.workspace_bytes = 0;
    if (L.ws_bytes && staging_bytes >= L.total_with_ws) d.workspace = base + L.ws_off, d.workspace_bytes = L.ws_bytes;
    const size_t feat_bytes =
        (size_t)p->B * p->N * p->feat_h * p->feat_w * p->C * (p->feat_dtype == FLASHBEV_F32 ? 4 : 2);
    if (cudaMemcpyAsync(base + L.feat_off, p->features, feat_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(base + L.mat_off, p->lidar2img, (size_t)p->B * p->N * 64, cudaMemcpyHostToDevice, stream) !=
            cudaSuccess) {
        cudaGetLastError();
        return FLASHBEV_CUDA_ERROR;
    }
    if ((st = run_device(&d, stream)) != FLASHBEV_OK) return st;
    if (cudaMemcpyAsync(p->out, base + L.out_off, (size_t)p->B * p->X * p->Y * p->C * (p->out_dtype == FLASHBEV_F32 ? 4 : 2),
                        cudaMemcpyDeviceToHost, stream) !=
            cudaSuccess ||
        (p->valid_count_out && cudaMemcpyAsync(p->valid_count_out, base + L.cnt_off, (size_t)p->B * p->X * p->Y * 4,
                                               cudaMemcpyDeviceToHost, stream) != cudaSuccess)) {
        cudaGetLastError();
        return FLASHBEV_CUDA_ERROR;
    }
    return FLASHBEV_OK;
}

// ---- backward --------------------------------------------------------------------------------
flashbev_status flashbev_sampling_vt_backward(const flashbev_vt_backward_params *q, void *stream_)
{
    if (!q || q->struct_size < offsetof(flashbev_vt_backward_params, debug_error_word)) return FLASHBEV_INVALID_ARG;
    if (!q->grad_out || !q->grad_features) return FLASHBEV_INVALID_ARG;
    // same geometry description as the forward: validate it through the forward's checks
    flashbev_vt_params p = {};
    p.struct_size = sizeof(p);
    p.features = q->grad_features;
    p.feat_dtype = FLASHBEV_F32;
    p.layout = FLASHBEV_NHWC;
    p.lidar2img = q->lidar2img;
    p.B = q->B, p.N = q->N, p.C = q->C, p.feat_h = q->feat_h, p.feat_w = q->feat_w, p.img_h = q->img_h, p.img_w = q->img_w;
    p.x_min = q->x_min, p.x_max = q->x_max, p.y_min = q->y_min, p.y_max = q->y_max, p.z_min = q->z_min, p.z_max = q->z_max;
    p.X = q->X, p.Y = q->Y, p.Z = q->Z, p.reduce = q->reduce;
    p.out = const_cast<float *>(q->grad_out);
    p.out_dtype = FLASHBEV_F32;
    p.kernel = FLASHBEV_KERNEL_TILED;
    for (int i = 0; i < 4; ++i) p.tune[i] = q->tune[i];
    p.debug_error_word = q->struct_size >= sizeof(flashbev_vt_backward_params) ? q->debug_error_word : nullptr;
    flashbev_status st;
    if (!params_ok(&p, st)) return st;
    if (((uintptr_t)q->grad_out % 16) || ((uintptr_t)q->grad_features % 16) || ((uintptr_t)q->lidar2img % 4))
        return FLASHBEV_MISALIGNED;
    if (q->C % 4 || !tiled_applicable(&p)) return FLASHBEV_UNSUPPORTED;
    KParams k;
    int V, warps;
    dim3 grid;
    size_t smem;
    p.tune[3] = (p.tune[3] & ~0xf) | 4;  // the backward instances are built for 4 warps per CTA
    // (measured) the scatter is bound by reductions on hot L2 sectors: small blocks in single-row bands spread them
    // best (7-9 % over the forward's defaults)
    if ((long long)p.B * p.X * p.Y >= 16384) {  // (small grids: the forward's defaults)
        if (!(p.tune[3] & 0xff0)) p.tune[3] |= (1 << 4) | (2 << 8);
        if (!(p.tune[3] & 0xc0000)) p.tune[3] |= 0x40000;
    }
    if ((st = configure_tiled(&p, k, V, warps, grid, smem)) != FLASHBEV_OK) return st;
    k.feat = nullptr, k.out = nullptr, k.count_out = nullptr;
    k.gout = q->grad_out, k.gfeat = q->grad_features;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const size_t bytes = (size_t)q->B * q->N * q->feat_h * q->feat_w * q->C * sizeof(float);
    if (cudaMemsetAsync(q->grad_features, 0, bytes, stream) != cudaSuccess) {
        cudaGetLastError();
        return FLASHBEV_CUDA_ERROR;
    }
    cudaError_t e;
    if (V == 1) e = launch_tiled_inst<1, false, 4, true>(k, grid, smem, stream);
    else if (V == 2) e = launch_tiled_inst<2, false, 4, true>(k, grid, smem, stream);
    else e = launch_tiled_inst<4, false, 4, true>(k, grid, smem, stream);
    if (e != cudaSuccess || cudaGetLastError() != cudaSuccess) return FLASHBEV_CUDA_ERROR;
    t_last_launches = 1;
    t_last_kernel = V == 1 ? "tiled_bwd_v1" : (V == 2 ? "tiled_bwd_v2" : "tiled_bwd_v4");
    return FLASHBEV_OK;
}

// ---- multi-resolution gathering: one launch per pyramid level, levels after the first add to the output
flashbev_status flashbev_sampling_vt_multires(const flashbev_vt_multires_params *q, void *stream)
{
    if (!q || q->struct_size < sizeof(flashbev_vt_multires_params) || !q->base || !q->features || !q->feat_hw)
        return FLASHBEV_INVALID_ARG;
    if (q->levels < 1 || q->levels > FLASHBEV_MAX_LEVELS) return FLASHBEV_INVALID_ARG;
    if (q->base->struct_size < offsetof(flashbev_vt_params, debug_error_word)) return FLASHBEV_INVALID_ARG;
    flashbev_vt_params lv[FLASHBEV_MAX_LEVELS];
    flashbev_status st;
    for (int l = 0; l < q->levels; ++l) {  // every level is checked before anything is enqueued
        lv[l] = copy_params(q->base);
        lv[l].features = q->features[l];
        lv[l].feat_h = q->feat_hw[2 * l], lv[l].feat_w = q->feat_hw[2 * l + 1];
        if (l > 0) lv[l].valid_count_out = nullptr;
        if (!params_ok(&lv[l], st)) return st;
        if (lv[l].out_dtype != FLASHBEV_F32) return FLASHBEV_UNSUPPORTED;
        if ((st = check_alignment(&lv[l])) != FLASHBEV_OK) return st;
        const bool tiled = lv[l].kernel == FLASHBEV_KERNEL_TILED;
        if (tiled && !tiled_applicable(&lv[l])) return FLASHBEV_UNSUPPORTED;
    }
    for (int l = 0; l < q->levels; ++l)
        if ((st = run_device(&lv[l], static_cast<cudaStream_t>(stream), l > 0)) != FLASHBEV_OK) return st;
    t_last_launches = q->levels;
    return FLASHBEV_OK;
}

// ---- FlashSCA ---------------------------------------------------------------------------------
flashbev_status flashbev_sca(const flashbev_sca_params *q, void *stream_)
{
    if (!q || q->struct_size < sizeof(flashbev_sca_params)) return FLASHBEV_INVALID_ARG;
    if (!q->value || !q->level_hw || !q->lidar2img || !q->offsets || !q->weights || !q->out) return FLASHBEV_INVALID_ARG;
    if (q->B <= 0 || q->N <= 0 || q->heads <= 0 || q->head_dim <= 0 || q->L <= 0 || q->P <= 0) return FLASHBEV_INVALID_ARG;
    if (q->img_h <= 0 || q->img_w <= 0 || q->X <= 0 || q->Y <= 0 || q->Zref <= 0) return FLASHBEV_INVALID_ARG;
    if (!(q->x_max > q->x_min) || !(q->y_max > q->y_min) || !(q->z_max > q->z_min)) return FLASHBEV_INVALID_ARG;
    if (!(q->x_max - q->x_min < 1e300) || !(q->y_max - q->y_min < 1e300) || !(q->z_max - q->z_min < 1e300))
        return FLASHBEV_INVALID_ARG;
    if (q->value_dtype != FLASHBEV_F32 && q->value_dtype != FLASHBEV_BF16) return FLASHBEV_INVALID_ARG;
    ScaParams k = {};
    long long T = 0;
    for (int l = 0; l < q->L && l < kScaMaxLevels; ++l) {
        const int Hl = q->level_hw[2 * l], Wl = q->level_hw[2 * l + 1];
        if (Hl <= 0 || Wl <= 0) return FLASHBEV_INVALID_ARG;
        k.Hl[l] = Hl, k.Wl[l] = Wl, k.lvl0[l] = (int)T;
        T += (long long)Hl * Wl;
    }
    const bool bf16 = q->value_dtype == FLASHBEV_BF16;
    const int epv = bf16 ? 8 : 4;  // elements per 16-byte vector
    if (q->L > kScaMaxLevels || q->N > kMaxCams || q->Zref > 32) return FLASHBEV_UNSUPPORTED;
    if (q->head_dim % epv || q->head_dim > 128 || (long long)q->N * q->Zref > 1024) return FLASHBEV_UNSUPPORTED;
    if (T >= 2147483647LL || (double)q->B * q->X * q->Y >= 2147483648.0) return FLASHBEV_UNSUPPORTED;
    if (((uintptr_t)q->value % 16) || ((uintptr_t)q->out % 16) || ((uintptr_t)q->offsets % 8) ||
        ((uintptr_t)q->weights % 4) || ((uintptr_t)q->lidar2img % 4) || (q->hits_out && ((uintptr_t)q->hits_out % 4)))
        return FLASHBEV_MISALIGNED;
    k.lph = q->head_dim / epv;
    k.hp = 32 / k.lph;
    const int V = (q->heads + k.hp - 1) / k.hp;
    if (V > 4) return FLASHBEV_UNSUPPORTED;
    k.value = static_cast<const uint4 *>(q->value);
    k.l2i = q->lidar2img;
    k.offsets = reinterpret_cast<const float2 *>(q->offsets);
    k.weights = q->weights;
    k.out = reinterpret_cast<float4 *>(q->out);
    k.hits_out = q->hits_out;
    k.B = q->B, k.N = q->N, k.heads = q->heads, k.Dh = q->head_dim, k.L = q->L, k.P = q->P;
    k.X = q->X, k.Y = q->Y, k.Zref = q->Zref, k.Himg = q->img_h, k.Wimg = q->img_w, k.T = T;
    k.x_min = q->x_min, k.dx = (q->x_max - q->x_min) / (double)q->X;
    k.y_min = q->y_min, k.dy = (q->y_max - q->y_min) / (double)q->Y;
    k.z_min = q->z_min, k.dz = (q->z_max - q->z_min) / (double)q->Zref;
    const long long queries = (long long)q->B * q->X * q->Y;
    const long long blocks = (queries + 3) / 4;
    if (blocks > 2147483647LL) return FLASHBEV_UNSUPPORTED;
    if ((double)T * q->heads * k.lph >= 2147483648.0) return FLASHBEV_UNSUPPORTED;  // 32-bit value indices in the records
    if (q->chunk_records < 0) return FLASHBEV_INVALID_ARG;
    const int chunk_records = q->chunk_records > 0 ? q->chunk_records : 128;
    k.Pc = std::max(1, std::min(std::min(q->P, kScaMaxChunkPoints), chunk_records / (q->heads * q->L)));
    k.pitch = q->L * k.Pc + 1;  // odd pitch: the heads of a warp read different shared-memory banks
    const int items = q->heads * q->L * k.Pc;
    const size_t smem = (((size_t)items * 4 + 15) & ~(size_t)15) + 4 * sca_warp_smem(q->N, q->Zref, q->heads, k.pitch, items, q->L);
    if (smem > 200 * 1024) return FLASHBEV_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    auto launch = [&](auto kern) -> cudaError_t {
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        kern<<<dim3((unsigned)blocks), dim3(128), smem, stream>>>(k);
        return cudaSuccess;
    };
    cudaError_t e;
    const bool even = k.hp * k.lph == 32 && q->heads == V * k.hp;
    if (bf16) {
        if (V == 1) e = even ? launch(sca_kernel<1, true, true>) : launch(sca_kernel<1, false, true>);
        else if (V == 2) e = even ? launch(sca_kernel<2, true, true>) : launch(sca_kernel<2, false, true>);
        else return FLASHBEV_UNSUPPORTED;
    } else {
        if (V == 1) e = even ? launch(sca_kernel<1, true, false>) : launch(sca_kernel<1, false, false>);
        else if (V == 2) e = even ? launch(sca_kernel<2, true, false>) : launch(sca_kernel<2, false, false>);
        else if (V == 3) e = even ? launch(sca_kernel<3, true, false>) : launch(sca_kernel<3, false, false>);
        else e = even ? launch(sca_kernel<4, true, false>) : launch(sca_kernel<4, false, false>);
    }
    if (e != cudaSuccess || cudaGetLastError() != cudaSuccess) return FLASHBEV_CUDA_ERROR;
    t_last_launches = 1;
    t_last_kernel = bf16 ? "sca_bf16" : "sca_f32";
    return FLASHBEV_OK;
}

// ---- allocation-free host entry point -------------------------------------------------------
// The staging area lives in the library image.  In host code the array's name is only a handle:
// the address the GPU understands has to be asked for, per device, with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_staging[FLASHBEV_STATIC_STAGING_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_ptr[kMaxDevices];  // device address of g_static_staging on device i, once looked up

// Device address of the built-in staging area on the current device (nullptr on failure).
void *static_staging_address()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return nullptr;
    }
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_staging) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        g_static_ptr[dev] = ptr;
    }
    return g_static_ptr[dev];
}
}  // namespace

flashbev_status flashbev_sampling_vt_host_static(const flashbev_vt_params *p, void *stream)
{
    flashbev_status st;
    if (!params_ok(p, st)) return st;
    StagingLayout L;
    if (!staging_layout(p, L) || L.total > (size_t)FLASHBEV_STATIC_STAGING_BYTES) return FLASHBEV_EXCEEDS_STATIC_STAGING;
    void *staging = static_staging_address();  // first call on this device: symbol look-up
    if (!staging) return FLASHBEV_CUDA_ERROR;
    // From here on this is the caller-staged path with the built-in area as the staging buffer.
    return flashbev_sampling_vt_host(p, staging, (size_t)FLASHBEV_STATIC_STAGING_BYTES, stream);
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
        case FLASHBEV_EXCEEDS_STATIC_STAGING: return "problem exceeds the built-in staging area";
        default: return "unknown status";
    }
}

int flashbev_version(void) { return FLASHBEV_VERSION; }

}  // extern "C"
