// Tiled Sampling-VT kernel (forward and backward) for B200 (sm_100a).  Included by flashbev.cu inside its
// anonymous namespace, after the shared helpers (KParams, fast_rcp, kDepthMin, FB_IDX, pack_bf16x2).
//
// A WARP owns a super-block of up to 32 adjacent BEV cells (sbn sub-blocks of cpw <= 8 cells) and works through
// it alone (__syncwarp only; the CTA shares nothing but the per-batch-element tables staged once at kernel
// start).  Everything that does not depend on the channel is computed once per (cell, camera, height) and
// turned into a compact list of "row records" in shared memory before a single feature is read (paper Sec. 3.3:
// the projection, validity test and bilinear weights of Algorithm 2, hoisted out of the channel dimension):
//
//   1a. candidates  one lane per (cell, camera): the five validity conditions are linear in the height once the
//                   depth is positive, so a column whose two end bins both fail the same condition (widened by a
//                   texel) has no valid bin.  About 4/5 of the candidates end here; the rest are compacted.
//   1b. columns     one lane per surviving column: the valid bins form ONE interval; it comes in closed form
//                   (float, conservative) and its two ends are confirmed with the exact fp64 test.  A camera
//                   without pitch or roll sees the column under one texel column (x0, tx constant) with fy affine
//                   in the bin index: then the texel rows the column touches, and so the number of records it
//                   will write, follow in closed form.  Columns are cut into runs of at most `walk` bins; a
//                   prefix sum over the record counts gives every run its place in the list, so the records of a
//                   cell are contiguous, their order is fixed and no atomics are needed.  The valid-sample count
//                   of a cell and the per-height camera counts of Eq. 1 follow from the intervals alone.
//   2.  walkers     one lane per run: successive bins that land on the same texel rows are merged into one
//                   record {left tap, right tap, wL, wR} per row.  Affine columns cost one fp64 FMA and a floor
//                   per bin; the others are projected bin by bin in fp64 (their records are counted by a first
//                   sweep of the same walker).
//   3.  gather      one sub-block at a time: g lanes per cell, V 16-byte channel vectors per lane; per record two
//                   128- or 256-bit loads per vector and packed fp32 FMAs into register accumulators.  Runs that
//                   do not fit the record slots are taken in several rounds; the accumulators of the sub-block
//                   stay in registers, so every output vector is written exactly once, with a streaming store.
// The backward instance replaces step 3 by the transpose: fp32 vector reductions of w * grad_out into the
// feature gradient.
//
// Shared memory (dynamic):
//   CTA  : double mats[N][12]   rows 0..2 of lidar2img[b][n], rows 0/1 pre-scaled to feature texels
//          float  slope[N][5]   d/dk of the five validity conditions
//          int    camfast[N]    1: the camera's depth and horizontal texel coordinate do not depend on height
//          int    celltab[32]   position of cell c inside a super-block: lx | ly << 8
//   warp : int     roff[slots]     row records of the current round: vector index of the first tap (the second follows
//          float2  rw[slots]       `rstep` vectors later) and the two weights
//          ColDesc col[ccap]       columns of the current segment, (cell, camera) order
//          uint32  wk[wcap]        runs: column | first bin << 8 | (bins - 1) << 24
//          int     woff[wcap + 1]  records before run w
//          int     colw[ccap + 1]  runs before column j
//          uint16  cand[ct * N]    surviving candidates: cell | camera << 8
//          double2 cellxy[32], int cfirst[33], int cnt[32]
//          uint8   den[ct * Z]     cameras per (cell, height bin), Eq. 1 mode only

#ifndef FB_EMIT_INLINE
#define FB_EMIT_INLINE __forceinline__
#endif
#ifndef FB_U_BF16V2
#define FB_U_BF16V2 3
#endif
#ifndef FB_WARPS_PER_SM
#define FB_WARPS_PER_SM 20
#endif

constexpr int kMaxCt = 32;   // cells per super-block
constexpr int kMaxCpw = 8;   // cells per sub-block
constexpr int kColCapMax = 64;  // column descriptors per warp (a sub-block never has more candidates than that)
constexpr int kWalkIlp = 1;  // height bins whose geometry a general walker evaluates independently

struct __align__(16) ColDesc {
    double d0, d1;  // affine: fy(k') = d0 + k' d1 with d1 >= 0 (bins renumbered so that rows ascend); general: a0, a1
    union {
        double d2;  // general: a2  (a_i = row i of the scaled matrix applied to (x_w, y_w, 0, 1))
        struct {
            int offc;   // affine: vector index of the column's first loaded texel at row 0
            float tx;   // affine: horizontal fraction
        } f;
    };
    int kk;    // klo | khi << 16: the valid bins
    int meta;  // cell | camera << 6 | affine << 12 | reversed << 13 | edge << 14 (0 interior, 1 left tap outside, 2 right tap outside)
};
static_assert(sizeof(ColDesc) == 32, "column descriptor is two 16-byte words");

struct WarpSmem {
    int *roff;
    float2 *rw;
    ColDesc *col;
    uint32_t *wk;
    int *woff, *colw, *cfirst, *cnt;
    uint16_t *cand;
    double2 *cellxy;
    unsigned char *den;
};

__host__ __device__ inline size_t align16(size_t v) { return (v + 15) & ~(size_t)15; }

__host__ __device__ inline size_t cta_table_bytes(int N)
{
    return align16((size_t)N * 12 * sizeof(double)) + align16((size_t)N * 5 * sizeof(float)) + align16((size_t)N * sizeof(int)) +
           kMaxCt * sizeof(int);
}

__host__ __device__ inline size_t warp_smem_layout(unsigned char *base, WarpSmem *t, int slots, int colcap, int wcap, int ct, int ncand,
                                                   int den_bytes)
{
    size_t o = 0;
    auto take = [&](size_t bytes) {
        unsigned char *ptr = base ? base + o : nullptr;
        o += align16(bytes);
        return ptr;
    };
    unsigned char *p0 = take((size_t)slots * sizeof(float2));
    unsigned char *p0b = take((size_t)slots * sizeof(int));
    unsigned char *p1 = take((size_t)colcap * sizeof(ColDesc));
    unsigned char *p2 = take((size_t)ct * sizeof(double2));
    unsigned char *p3 = take((size_t)wcap * sizeof(uint32_t));
    unsigned char *p4 = take((size_t)(wcap + 1) * sizeof(int));
    unsigned char *p5 = take((size_t)(colcap + 1) * sizeof(int));
    unsigned char *p6 = take((size_t)(2 * kMaxCt + 1) * sizeof(int));
    unsigned char *p7 = take((size_t)ncand * sizeof(uint16_t));
    unsigned char *p8 = take((size_t)den_bytes);
    if (t) {
        t->rw = reinterpret_cast<float2 *>(p0);
        t->roff = reinterpret_cast<int *>(p0b);
        t->col = reinterpret_cast<ColDesc *>(p1);
        t->cellxy = reinterpret_cast<double2 *>(p2);
        t->wk = reinterpret_cast<uint32_t *>(p3);
        t->woff = reinterpret_cast<int *>(p4);
        t->colw = reinterpret_cast<int *>(p5);
        t->cfirst = reinterpret_cast<int *>(p6);
        t->cnt = t->cfirst + kMaxCt + 1;
        t->cand = reinterpret_cast<uint16_t *>(p7);
        t->den = p8;
    }
    return o;
}

// Horizontal weights of the two texels a record loads (xc, xc + 1, both inside the map): an out-of-map tap
// weighs 0 and the in-map one takes the slot that keeps both addresses loadable.
__device__ __forceinline__ void fold_x(int x0, float tx, int Wf, int &xc, float &cl, float &cr)
{
    if (x0 < 0) {                 // left tap outside: the right tap is texel 0, loaded as the record's first tap
        xc = 0, cl = tx, cr = 0.f;
    } else if (x0 >= Wf - 1) {    // right tap outside
        if (Wf > 1) xc = Wf - 2, cl = 0.f, cr = 1.f - tx;
        else xc = 0, cl = 1.f - tx, cr = 0.f;
    } else {
        xc = x0, cl = 1.f - tx, cr = tx;
    }
}

// acc += w * (channels of one 16-byte vector), two channels per packed fp32 FMA
template <bool BF16>
__device__ __forceinline__ void fma_vec(float2 (&acc)[BF16 ? 4 : 2], const uint4 &t, const float2 w)
{
    if (BF16) {
        acc[0] = __ffma2_rn(make_float2(__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xffff0000u)), w, acc[0]);
        acc[1] = __ffma2_rn(make_float2(__uint_as_float(t.y << 16), __uint_as_float(t.y & 0xffff0000u)), w, acc[1]);
        acc[2 % (BF16 ? 4 : 2)] =
            __ffma2_rn(make_float2(__uint_as_float(t.z << 16), __uint_as_float(t.z & 0xffff0000u)), w, acc[2 % (BF16 ? 4 : 2)]);
        acc[3 % (BF16 ? 4 : 2)] =
            __ffma2_rn(make_float2(__uint_as_float(t.w << 16), __uint_as_float(t.w & 0xffff0000u)), w, acc[3 % (BF16 ? 4 : 2)]);
    } else {
        acc[0] = __ffma2_rn(make_float2(__uint_as_float(t.x), __uint_as_float(t.y)), w, acc[0]);
        acc[1] = __ffma2_rn(make_float2(__uint_as_float(t.z), __uint_as_float(t.w)), w, acc[1]);
    }
}

// Two adjacent 16-byte vectors with one 256-bit load (sm_100: ld.global.v8), 32-byte aligned address.
__device__ __forceinline__ void ldg_pair(const uint4 *ptr, uint4 &a, uint4 &b)
{
    asm("ld.global.nc.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
        : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w)
        : "l"(ptr));
}

// base + 16 * index in one widening multiply-add
__device__ __forceinline__ const uint4 *vec_at(const uint4 *base, unsigned index)
{
    const uint4 *r;
    asm("mad.wide.u32 %0, %1, 16, %2;" : "=l"(r) : "r"(index), "l"(base));
    return r;
}

// shared-memory loads through 32-bit shared-window addresses
__device__ __forceinline__ unsigned lds_u32(unsigned addr)
{
    unsigned v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ float2 lds_f32x2(unsigned addr)
{
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
    return v;
}

// U records of one cell list: two taps each, both always loadable; packed fp32 FMAs into the accumulators.
template <int U, int V, bool BF16, bool WIDE>
__device__ __forceinline__ void gather_records(float2 (&acc)[V][BF16 ? 4 : 2], unsigned loff, unsigned lw, unsigned rstep,
                                               const uint4 *const (&featv)[V])
{
    unsigned ro[U];
    float2 rw[U];
#pragma unroll
    for (int u = 0; u < U; ++u) ro[u] = lds_u32(loff + 4 * u), rw[u] = lds_f32x2(lw + 8 * u);
    uint4 t[U][2][V];
    if (WIDE) {  // the lane's vectors are adjacent: V / 2 loads of 32 bytes per tap
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int v = 0; v + 1 < V; v += 2) {
                ldg_pair(vec_at(featv[v], ro[u]), t[u][0][v], t[u][0][v + 1]);
                ldg_pair(vec_at(featv[v], ro[u] + rstep), t[u][1][v], t[u][1][v + 1]);
            }
    } else {
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int v = 0; v < V; ++v) {
                t[u][0][v] = __ldg(vec_at(featv[v], ro[u]));
                t[u][1][v] = __ldg(vec_at(featv[v], ro[u] + rstep));
            }
    }
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
        for (int v = 0; v < V; ++v) {
            fma_vec<BF16>(acc[v], t[u][0][v], make_float2(rw[u].x, rw[u].x));
            fma_vec<BF16>(acc[v], t[u][1][v], make_float2(rw[u].y, rw[u].y));
        }
}

// Gather of one cell list by its channel lanes: groups of U records, then the rest one by one.
// loff / lw: shared-window addresses of the list's offsets and weights.
template <int V, bool BF16, bool WIDE>
__device__ __forceinline__ void gather_list(float2 (&acc)[V][BF16 ? 4 : 2], unsigned loff, unsigned lw, int nrec, unsigned rstep,
                                            const uint4 *const (&featv)[V])
{
    constexpr int U = V == 1 ? 4 : (V == 2 ? (BF16 ? FB_U_BF16V2 : 2) : 1);
    int j = 0;
    for (; j + U <= nrec; j += U, loff += 4 * U, lw += 8 * U) gather_records<U, V, BF16, WIDE>(acc, loff, lw, rstep, featv);
    if (U > 1)
        for (; j < nrec; ++j, loff += 4, lw += 8) gather_records<1, V, BF16, WIDE>(acc, loff, lw, rstep, featv);
}

// Backward of the gather: every record adds its two weighted taps of the cell's output gradient to the
// feature gradient (the transpose of gather_list).  Vector reductions: texels are shared by cells.
template <int V>
__device__ __forceinline__ void scatter_list(const float4 (&go)[V], const bool (&on)[V], const int *loff, const float2 *lw, int nrec,
                                             int rstep, float4 *const (&gfv)[V])
{
    for (int j = 0; j < nrec; ++j) {
        const int off = loff[j];
        const float wl = lw[j].x, wr = lw[j].y;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            if (!on[v]) continue;  // ragged last channel block
            if (wl != 0.f) atomicAdd(gfv[v] + off, make_float4(go[v].x * wl, go[v].y * wl, go[v].z * wl, go[v].w * wl));
            if (wr != 0.f) atomicAdd(gfv[v] + off + rstep, make_float4(go[v].x * wr, go[v].y * wr, go[v].z * wr, go[v].w * wr));
        }
    }
}

// ---- step 1a: can any height bin of candidate column (cell at xy, camera n) be valid? -------------------------
// Every validity condition is a linear function of the height that must be positive (depth - 0.1; fx + 1/2 and
// Wf - 1/2 - fx times the depth; likewise fy).  If one of them, relaxed by a texel, is negative at the first AND
// the last bin centre it is negative in between: no bin of the column is valid.  NaN compares false: kept.
__device__ __forceinline__ bool column_possible(const KParams &p, const double *m, double2 xy)
{
    const double zl = p.z_min + 0.5 * p.dz, zh = fma((double)(p.Z - 1), p.dz, zl);
    const double a0 = fma(m[1], xy.y, fma(m[0], xy.x, m[3]));
    const double a1 = fma(m[5], xy.y, fma(m[4], xy.x, m[7]));
    const double a2 = fma(m[9], xy.y, fma(m[8], xy.x, m[11]));
    const double dl = fma(m[10], zl, a2), dh = fma(m[10], zh, a2);
    const double ul = fma(m[2], zl, a0), uh = fma(m[2], zh, a0);
    const double vl = fma(m[6], zl, a1), vh = fma(m[6], zh, a1);
    const double wf = (double)p.Wf + 0.5, hf = (double)p.Hf + 0.5;
    bool out = (dl < 0.05) & (dh < 0.05);
    out |= (fma(1.5, dl, ul) < 0.0) & (fma(1.5, dh, uh) < 0.0);   // fx < -3/2 wherever the depth is positive
    out |= (fma(wf, dl, -ul) < 0.0) & (fma(wf, dh, -uh) < 0.0);   // fx > Wf + 1/2
    out |= (fma(1.5, dl, vl) < 0.0) & (fma(1.5, dh, vh) < 0.0);
    out |= (fma(hf, dl, -vl) < 0.0) & (fma(hf, dh, -vh) < 0.0);
    return !out;
}

// ---- step 1b: the interval of valid bins of a column, exactly; affine form for height-independent cameras -----
// Returns the number of valid bins (0: the column drops out) and fills D.
__device__ __forceinline__ int column_build(const KParams &p, const double *mats, const float *slope, const int *camfast,
                                            double2 xy, int c, int n, ColDesc &D)
{
    const double *m = mats + n * 12;
    const float *sl = slope + n * 5;
    const double zc0 = p.z_min + 0.5 * p.dz;  // centre of bin 0; z_w(k) = zc0 + k dz
    const double a0 = fma(m[1], xy.y, fma(m[0], xy.x, m[3]));
    const double a1 = fma(m[5], xy.y, fma(m[4], xy.x, m[7]));
    const double a2 = fma(m[9], xy.y, fma(m[8], xy.x, m[11]));
    D.d0 = a0, D.d1 = a1, D.d2 = a2;
    D.kk = 1;  // klo = 1 > khi = 0: no bins
    D.meta = c | (n << 6);
    if (camfast[n]) {
        // Depth and fx do not depend on the height: one texel column, fy = ay + k sy affine in the bin index k, and
        // the valid bins are those with -1/2 < fy < Hf - 1/2: an interval in closed form, its ends confirmed.
        if (!(a2 > kDepthMin)) return 0;
        const double r = fast_rcp(a2);
        const double fx = fma(a0, r, -0.5);
        const double wl = (double)p.Wf - 0.5, hl = (double)p.Hf - 0.5;
        if (!(fx > -0.5 && fx < wl)) return 0;
        const double ay = fma(fma(m[6], zc0, a1), r, -0.5), sy = m[6] * p.dz * r;
        const double inv = fast_rcp(sy);
        const double ta = (-0.5 - ay) * inv, tb = (hl - ay) * inv;      // fy crosses the two borders at these k
        const double zf = (double)p.Z;
        double tlo = sy > 0.0 ? ta : (sy < 0.0 ? tb : -1.0), thi = sy > 0.0 ? tb : (sy < 0.0 ? ta : zf);
        tlo = fmin(fmax(tlo, -1.0), zf), thi = fmin(fmax(thi, -1.0), zf);  // NaN -> the whole range: every bin is then tested
        int klo = max((int)floor(tlo), 0), khi = min((int)ceil(thi), p.Z - 1);
        auto inside = [&](int k) {
            const double fy = fma((double)k, sy, ay);
            return (fy > -0.5) & (fy < hl);
        };
        while (klo <= khi && !inside(klo)) ++klo;
        while (khi > klo && !inside(khi)) --khi;
        if (klo > khi) return 0;
        const bool rev = sy < 0.0;  // rows ascend with the renumbered bins k' = khi - k
        const double flx = floor(fx);
        const int x0 = (int)flx;
        const int edge = x0 < 0 ? 1 : (x0 >= p.Wf - 1 ? 2 : 0);
        const int xc = edge == 1 ? 0 : (edge == 2 ? max(p.Wf - 2, 0) : x0);
        D.d0 = fma((double)(rev ? khi : klo), sy, ay);
        D.d1 = rev ? -sy : sy;
        D.f.offc = (n * p.Hf * p.Wf + xc) * p.vecs;
        D.f.tx = (float)(fx - flx);
        D.kk = klo | (khi << 16);
        D.meta |= (1 << 12) | ((rev ? 1 : 0) << 13) | (edge << 14);
        return khi - klo + 1;
    }
    // conditions alpha + beta * k > 0 (k real): depth, left, right, top, bottom -> conservative interval
    float lo = -1.f, hi = (float)p.Z;
    bool empty = false;
    auto cond = [&](float a, float bslope) {
        const float t = -a * __frcp_rn(bslope);                  // the condition changes sign at k = t
        lo = bslope > 0.f ? fmaxf(lo, t) : lo;                   // k > -a/b
        hi = bslope < 0.f ? fminf(hi, t) : hi;                   // k < -a/b
        empty |= (bslope == 0.f) & (a <= 0.f);                   // independent of z (NaN: keep, tested exactly below)
    };
    const double d0 = fma(m[10], zc0, a2);
    const double p00 = fma(m[2], zc0, a0);
    const double p10 = fma(m[6], zc0, a1);
    cond((float)(d0 - kDepthMin), sl[0]);
    cond((float)p00, sl[1]);
    cond((float)fma((double)p.Wf, d0, -p00), sl[2]);
    cond((float)p10, sl[3]);
    cond((float)fma((double)p.Hf, d0, -p10), sl[4]);
    if (empty || !(lo < hi)) return 0;
    // widen by a guard far above the float error, then confirm both ends exactly
    const float guard = 0.05f + 1e-5f * (float)p.Z;
    int klo = (int)floorf(fminf(fmaxf(lo - guard, -1.f), (float)p.Z)) + 1;
    int khi = (int)ceilf(fmaxf(fminf(hi + guard, (float)p.Z), -1.f)) - 1;
    klo = max(klo, 0);
    khi = min(khi, p.Z - 1);
    const double wlim = (double)p.Wf - 0.5, hlim = (double)p.Hf - 0.5;
    double fy_at = 0.0;  // fy of the bin tested last
    auto exact = [&](int k) {
        const double zw = fma((double)k, p.dz, zc0);
        const double d = fma(m[10], zw, a2);
        const double r = fast_rcp(d);  // d <= 0 or NaN gives inf / NaN: the tests below fail
        const double fx = fma(fma(m[2], zw, a0), r, -0.5);
        const double fy = fma(fma(m[6], zw, a1), r, -0.5);
        fy_at = fy;
        return (d > kDepthMin) & (fx > -0.5) & (fx < wlim) & (fy > -0.5) & (fy < hlim);
    };
    while (klo <= khi && !exact(klo)) ++klo;
    if (klo > khi) return 0;
    const double fy_lo = fy_at;
    while (khi > klo && !exact(khi)) --khi;
    const bool rev = khi > klo && fy_at < fy_lo;  // rows ascend with the renumbered bins k' = khi - k
    D.kk = klo | (khi << 16);
    D.meta |= (rev ? 1 : 0) << 13;
    return khi - klo + 1;
}

// An affine column with a step of at most two rows per bin touches every texel row from its first bin's row to the
// row below its last bin's row: its records are those rows (inside the map), one each, and a run is a range of
// ROWS.  With larger steps the rows of successive bins never coincide: two records per bin, and a run is a range
// of BINS.  Either way the number of records of a run is known without walking it.
__device__ __forceinline__ bool affine_by_rows(const ColDesc &D) { return D.d1 <= 1.999; }

// Units (rows or bins) of an affine column that its runs are cut from, and the first row it writes.
__device__ __forceinline__ int affine_units(const KParams &p, const ColDesc &D, int nb, int &row_first)
{
    const int r_first = (int)floor(D.d0), r_last = (int)floor(fma((double)(nb - 1), D.d1, D.d0));
    row_first = max(r_first, 0);
    return affine_by_rows(D) ? max(0, min(r_last + 1, p.Hf - 1) - row_first + 1) : nb;
}

// Records of a run of an affine column: [u0, u0 + len) are rows counted from the column's first written row, or bins.
__device__ __forceinline__ int affine_run_records(const ColDesc &D, int len) { return affine_by_rows(D) ? len : 2 * len; }

// ---- step 2: walker of an affine column.  Writes exactly affine_run_records() records. -------------------------
// A run of rows [ra, rb) takes the bins whose upper tap lies in rows ra - 1 .. rb - 1: a row's weight is the (1 - ty)
// of the bins in it plus the ty of the bins in the row above, so every run is complete by itself and neighbouring
// runs share no record.  Bins are taken in order and a row's record is written when the bins have moved past it.
__device__ __forceinline__ void walk_affine(const KParams &p, const WarpSmem &sm, const ColDesc &D, int u0, int len,
                                            int *out_off, float2 *out_w, int cap)
{
    const int meta = D.meta;
    const bool rev = (meta >> 13) & 1;
    const int edge = (meta >> 14) & 3;
    const float tx = D.f.tx;
    float cl = 0.f, cr = 0.f;  // horizontal weights of the two loaded texels (an out-of-map tap weighs 0)
    if (edge == 0) cl = 1.f - tx, cr = tx;
    else if (edge == 1) cl = tx;
    else if (p.Wf > 1) cr = 1.f - tx;
    else cl = 1.f - tx;
    const bool eq1 = p.reduce == FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM;
    const int klo = D.kk & 0xffff, khi = (D.kk >> 16) & 0xffff, nb = khi - klo + 1;
    const unsigned char *den = sm.den + (meta & 63) * p.Z + (rev ? khi : klo);  // den[cell][bin of k' = 0]
    const int dstep = rev ? -1 : 1;
    const int rowv = p.Wf * p.vecs, offc = D.f.offc;
    const double S = D.d1, A = D.d0;

    if (affine_by_rows(D)) {
        len = min(len, cap);  // (never cuts: the run's slots were counted from the same numbers)
#ifdef FLASHBEV_DEBUG_BOUNDS
        (void)FB_IDX((out_off - sm.roff) + len - 1, p.slots, p.err);
#endif
        const int ra = max((int)floor(A), 0) + u0;
        const double inv = (double)__frcp_rn((float)S);
        auto first_bin_at = [&](double rr) {  // smallest k' in [0, nb] with A + k' S >= rr
            double e = ceil((rr - A) * inv);
            e = fmin(fmax(e, 0.0), (double)nb);  // NaN -> 0
            int k = (int)e;
            if (k > 0 && fma((double)(k - 1), S, A) >= rr) --k;
            else if (k < nb && fma((double)k, S, A) < rr) ++k;
            return k;
        };
        const int kb = first_bin_at((double)(ra - 1)), ke = first_bin_at((double)(ra + len));
        // The two rows the current bin touches are kept in registers; a row is written, once, when the bins have
        // left it (its weight is complete then: the (1 - ty) of its own bins and the ty of the bins of the row above).
        int off = FB_IDX(offc + ra * rowv, p.nvec_cam - p.vecs - p.rstep + 1 - (len - 1) * rowv, p.err) - rowv;
        int icur = -1;  // a0: weight of row icur, a1: of row icur + 1 (relative to ra); pw, po, off belong to row icur
        float a0 = 0.f, a1 = 0.f;
        float2 *pw = out_w - 1;
        int *po = out_off - 1;
        double kd = (double)kb;
        const unsigned char *dk = den + kb * dstep;
        for (int k = kb; k < ke; ++k, kd += 1.0, dk += dstep) {
            const double fy = fma(kd, S, A), fl = floor(fy);
            const int i = (int)fl - ra;  // row of the upper tap, relative: -1 .. len - 1, never decreasing
            float ty = (float)(fy - fl), tu = 1.f - ty;
            if (eq1) {
#ifdef FLASHBEV_DEBUG_BOUNDS
                dk = sm.den + FB_IDX(dk - sm.den, p.den_bytes, p.err);
#endif
                const float sc = 1.f / (float)max(1, (int)*dk);
                ty *= sc, tu *= sc;
            }
            if (i != icur) {
                if ((unsigned)icur < (unsigned)len) *pw = make_float2(cl * a0, cr * a0), *po = off;
                a0 = a1, a1 = 0.f, ++icur, ++pw, ++po, off += rowv;
                while (i != icur && icur < len) {  // a row without a bin of its own (steps of more than one row per bin)
                    *pw = make_float2(cl * a0, cr * a0), *po = off;
                    a0 = 0.f, ++icur, ++pw, ++po, off += rowv;
                }
            }
            a0 += tu, a1 += ty;
        }
        if ((unsigned)icur < (unsigned)len) *pw = make_float2(cl * a0, cr * a0), *po = off;
        a0 = a1;
        for (++icur, ++pw, ++po, off += rowv; icur < len; ++icur, ++pw, ++po, off += rowv, a0 = 0.f)
            *pw = make_float2(cl * a0, cr * a0), *po = off;
    } else {
        // rows of successive bins never coincide: two records per bin (a row outside the map: weight 0, clamped)
        len = min(len, cap / 2);
#ifdef FLASHBEV_DEBUG_BOUNDS
        (void)FB_IDX((out_off - sm.roff) + 2 * len - 1, p.slots, p.err);
#endif
        double kd = (double)u0;
        const unsigned char *dk = den + u0 * dstep;
        for (int i = 0; i < len; ++i, kd += 1.0, dk += dstep) {
            const double fy = fma(kd, S, A), fl = floor(fy);
            const int r = (int)fl;
            float ty = (float)(fy - fl), tu = 1.f - ty;
            if (eq1) {
#ifdef FLASHBEV_DEBUG_BOUNDS
                dk = sm.den + FB_IDX(dk - sm.den, p.den_bytes, p.err);
#endif
                const float sc = 1.f / (float)max(1, (int)*dk);
                ty *= sc, tu *= sc;
            }
            if (r < 0) tu = 0.f;
            if (r + 1 > p.Hf - 1) ty = 0.f;
            const int ru = max(r, 0), rl = min(r + 1, p.Hf - 1);
            out_off[2 * i] = FB_IDX(offc + ru * rowv, p.nvec_cam - p.vecs - p.rstep + 1, p.err);
            out_w[2 * i] = make_float2(cl * tu, cr * tu);
            out_off[2 * i + 1] = FB_IDX(offc + rl * rowv, p.nvec_cam - p.vecs - p.rstep + 1, p.err);
            out_w[2 * i + 1] = make_float2(cl * ty, cr * ty);
        }
    }
}

// ---- step 2: walker of a general column (every bin projected in fp64).  COUNT-only or EMIT. ------------------------
template <bool EMIT>
__device__ __forceinline__ int walk_general(const KParams &p, const WarpSmem &sm, const double *mats, const ColDesc &D, int k0,
                                            int len, int *out_off, float2 *out_w, int cap)
{
    const int meta = D.meta;
    const bool rev = (meta >> 13) & 1;
    const int cell = meta & 63, cam = (meta >> 6) & 63;
    const int klo = D.kk & 0xffff, khi = (D.kk >> 16) & 0xffff;
    const int rowv = p.Wf * p.vecs;
    const double *m = mats + cam * 12;
    const double zc0 = p.z_min + 0.5 * p.dz;
    int n = 0;
    bool open = false;
    int ro = 0, xo = 0, xco = 0;  // open rows (ro, ro + 1) at bilinear corner column xo, first loaded texel xco
    float uL = 0.f, uR = 0.f, lL = 0.f, lR = 0.f;
    auto put = [&](int row, float wl, float wr) {
        if (row >= 0 && row <= p.Hf - 1) {
            if (EMIT && n < cap) {
                const int off = FB_IDX((cam * p.Hf * p.Wf + xco) * p.vecs + row * rowv, p.nvec_cam - p.vecs - p.rstep + 1, p.err);
                out_off[n] = off, out_w[n] = make_float2(wl, wr);
            }
            ++n;
        }
    };
    for (int i0 = 0; i0 < len; i0 += kWalkIlp) {
        int r[kWalkIlp], x0[kWalkIlp], xc[kWalkIlp];
        float cl[kWalkIlp], cr[kWalkIlp], ty[kWalkIlp];
#pragma unroll
        for (int i = 0; i < kWalkIlp; ++i) {
            const int kp = k0 + min(i0 + i, len - 1);  // past the end: the last bin again (ignored below)
            const double zw = fma((double)(rev ? khi - kp : klo + kp), p.dz, zc0);
            const double d = fma(m[10], zw, D.d2);
            const double rd = fast_rcp(d);
            const double fx = fma(fma(m[2], zw, D.d0), rd, -0.5);
            const double fy = fma(fma(m[6], zw, D.d1), rd, -0.5);
            const double flx = floor(fx), fly = floor(fy);
            r[i] = (int)fly, x0[i] = (int)flx;
            ty[i] = (float)(fy - fly);
            fold_x(x0[i], (float)(fx - flx), p.Wf, xc[i], cl[i], cr[i]);
        }
#pragma unroll
        for (int i = 0; i < kWalkIlp; ++i) {
            if (i0 + i < len) {
                const bool col_same = open & (x0[i] == xo);
                const bool same = col_same & (r[i] == ro), next = col_same & (r[i] == ro + 1);
                if (!same) {
                    if (open) {
                        put(ro, uL, uR);
                        if (!next) put(ro + 1, lL, lR);
                    }
                    uL = next ? lL : 0.f, uR = next ? lR : 0.f, lL = 0.f, lR = 0.f;
                    ro = r[i], xo = x0[i], xco = xc[i], open = true;
                }
                if (EMIT) {
                    float s = 1.f;
                    if (p.reduce == FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM) {  // Eq. 1: 1 / max(1, cameras that see this height)
                        const int kp = k0 + i0 + i;
                        const unsigned dn = sm.den[FB_IDX(cell * p.Z + (rev ? khi - kp : klo + kp), p.den_bytes, p.err)];
                        s = 1.f / (float)(dn > 1u ? dn : 1u);
                    }
                    const float wy1 = ty[i] * s, wy0 = (1.f - ty[i]) * s;
                    uL = fmaf(cl[i], wy0, uL), uR = fmaf(cr[i], wy0, uR);
                    lL = fmaf(cl[i], wy1, lL), lR = fmaf(cr[i], wy1, lR);
                }
            }
        }
    }
    if (open) {
        put(ro, uL, uR);
        put(ro + 1, lL, lR);
    }
    return n;
}

// The three geometry steps are separate functions (not inlined) so that their fp64-heavy register needs stay out of
// the gather loop's allocation; everything they exchange lives in the warp's shared memory.
struct WarpCtx {
    const double *mats;
    const float *slope;
    const int *camfast;
    unsigned char *warp_base;  // this warp's shared memory
};

__device__ __forceinline__ WarpSmem warp_smem(const KParams &p, unsigned char *warp_base)
{
    WarpSmem sm;
    warp_smem_layout(warp_base, &sm, p.slots, p.colcap, p.wcap, p.ct, p.ct * p.N, p.den_bytes);
    return sm;
}

// ---- step 1a over a super-block: candidates -> survivors, compacted in (cell, camera) order.  Returns their number.
__device__ __forceinline__ int survey_candidates(const KParams &p, WarpCtx cx, unsigned in_mask)
{
    constexpr unsigned FULL = 0xffffffffu;
    const WarpSmem sm = warp_smem(p, cx.warp_base);
    const int lane = threadIdx.x & 31;
    const unsigned lt_mask = (1u << lane) - 1u;
    const int ncand = p.ct * p.N;
    int nsurv = 0;
    for (int p0 = 0; p0 < ncand; p0 += 32) {
        const int pr = p0 + lane;
        const int c = (int)(((float)pr + 0.5f) * p.inv_n), n = pr - c * p.N;
        bool keep = false;
        if (pr < ncand && ((in_mask >> c) & 1u)) keep = column_possible(p, cx.mats + n * 12, sm.cellxy[c]);
        const unsigned bal = __ballot_sync(FULL, keep);
        const int idx = nsurv + __popc(bal & lt_mask);
        if (pr < ncand && n == 0) sm.cfirst[FB_IDX(c, kMaxCt + 1, p.err)] = idx;  // where the cell's columns start
        if (keep) sm.cand[FB_IDX(idx, ncand, p.err)] = (uint16_t)(c | (n << 8));
        nsurv += __popc(bal);
    }
    if (lane == 0) sm.cfirst[p.ct] = nsurv;
    __syncwarp();
    return nsurv;
}

// ---- step 1b over a segment (survivors [jb, jb + ncols), cells [c_lo, c_hi)): exact intervals, runs and their record
// counts (two exclusive scans over the columns), valid samples per cell, Eq. 1 camera counts.  Returns the number of runs.
__device__ __forceinline__ int build_columns(const KParams &p, WarpCtx cx, int jb, int ncols, int c_lo, int c_hi)
{
    constexpr unsigned FULL = 0xffffffffu;
    const WarpSmem sm = warp_smem(p, cx.warp_base);
    const int lane = threadIdx.x & 31;
    int nw = 0, nrec_seg = 0;
    for (int j0 = 0; j0 < ncols; j0 += 32) {
        const int j = j0 + lane;
        ColDesc D;
        int nb = 0;
        if (j < ncols) {
            const int cn = sm.cand[jb + j];
            nb = column_build(p, cx.mats, cx.slope, cx.camfast, sm.cellxy[cn & 0xff], cn & 0xff, cn >> 8, D);
            sm.col[FB_IDX(j, p.colcap, p.err)] = D;
        }
        bool affine = false;
        int units = nb, row_first = 0;  // what the column's runs are cut from: bins, or rows of an affine column
        if (nb > 0) {
            affine = (D.meta >> 12) & 1;
            if (affine) units = affine_units(p, D, nb, row_first);
        }
        const int runs = (units + p.walk - 1) >> p.walk_shift;  // walk is a power of two
        int x = runs;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int y = __shfl_up_sync(FULL, x, off);
            if (lane >= off) x += y;
        }
        const int wbase = nw + x - runs;
        nw += __shfl_sync(FULL, x, 31);
        int mine = 0;  // records of this lane's column
        if (j < ncols) {
            sm.colw[j] = wbase;
            // runs of equal length (17 rows: 9 + 8, not 16 + 1): the walkers of a round finish together
            const int per = runs > 1 ? (units + runs - 1) / runs : units;
            for (int i = 0; i < runs; ++i) {
                const int u0 = i * per, len = min(per, units - u0);
                sm.wk[FB_IDX(wbase + i, p.wcap, p.err)] = (uint32_t)j | ((uint32_t)u0 << 8) | ((uint32_t)(len - 1) << 24);
                sm.woff[FB_IDX(wbase + i, p.wcap + 1, p.err)] = mine;
                mine += affine ? affine_run_records(D, len) : walk_general<false>(p, sm, cx.mats, D, u0, len, nullptr, nullptr, 0);
            }
        }
        int y = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int z = __shfl_up_sync(FULL, y, off);
            if (lane >= off) y += z;
        }
        const int rbase = nrec_seg + y - mine;
        nrec_seg += __shfl_sync(FULL, y, 31);
        if (j < ncols)
            for (int i = 0; i < runs; ++i) sm.woff[wbase + i] += rbase;
    }
    if (lane == 0) sm.colw[ncols] = nw, sm.woff[nw] = nrec_seg;
    __syncwarp();

    // valid samples per cell; Eq. 1: cameras per (cell, height bin) -- the intervals say it all
    if (lane >= c_lo && lane < c_hi) {
        int n = 0;
        for (int j = sm.cfirst[lane] - jb; j < sm.cfirst[lane + 1] - jb; ++j) {
            const int kk = sm.col[j].kk;
            n += max(0, ((kk >> 16) & 0xffff) - (kk & 0xffff) + 1);
        }
        sm.cnt[lane] = n;
    }
    if (p.reduce == FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM) {
        for (int i = c_lo * p.Z + lane; i < c_hi * p.Z; i += 32) {
            const int c = i / p.Z, k = i - c * p.Z;
            int dn = 0;
            for (int j = sm.cfirst[c] - jb; j < sm.cfirst[c + 1] - jb; ++j) {
                const int kk = sm.col[j].kk;
                dn += (k >= (kk & 0xffff) && k <= ((kk >> 16) & 0xffff)) ? 1 : 0;
            }
            sm.den[FB_IDX(i, p.den_bytes, p.err)] = (unsigned char)dn;
        }
    }
    __syncwarp();
    return nw;
}

// ---- step 2: run w is walked by the calling lane; its records go to slots [at, at + its count) ------------------
__device__ __forceinline__ void walk_one(const KParams &p, const WarpSmem &sm, const double *mats, int w, int at)
{
    const uint32_t wd = sm.wk[w];
    const ColDesc D = sm.col[FB_IDX(wd & 0xff, p.colcap, p.err)];
    at = FB_IDX(at, p.slots, p.err);
    if ((D.meta >> 12) & 1) walk_affine(p, sm, D, (wd >> 8) & 0xffff, (wd >> 24) + 1, sm.roff + at, sm.rw + at, p.slots - at);
    else walk_general<true>(p, sm, mats, D, (wd >> 8) & 0xffff, (wd >> 24) + 1, sm.roff + at, sm.rw + at, p.slots - at);
}

// WIDE: a lane's V channel vectors are adjacent (32-byte aligned pairs, 256-bit loads) instead of g apart
// PLANAR: the output is written one channel at a time with the strides in the parameters -- [B][C][X][Y] tensors, or
// channels-last rows that are not whole 16-byte vectors (the features are then a copy in the kernel's own layout);
// instances of their own, so that the vector-store instances do not carry the scalar stores
template <int V, bool BF16, int WARPS, bool BWD, bool WIDE, bool PLANAR = false>
__global__ void __launch_bounds__(WARPS * 32, (V == 4 ? 12 : FB_WARPS_PER_SM) / WARPS)
    vt_tiled_kernel(const KParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int PV = BF16 ? 4 : 2;  // channel pairs per 16-byte vector
    constexpr int THREADS = WARPS * 32;
    constexpr unsigned FULL = 0xffffffffu;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.z;

    double *mats = reinterpret_cast<double *>(smem_raw);
    float *slope = reinterpret_cast<float *>(smem_raw + align16((size_t)p.N * 12 * sizeof(double)));
    int *camfast = reinterpret_cast<int *>(reinterpret_cast<unsigned char *>(slope) + align16((size_t)p.N * 5 * sizeof(float)));
    int *celltab = reinterpret_cast<int *>(reinterpret_cast<unsigned char *>(camfast) + align16((size_t)p.N * sizeof(int)));
    WarpCtx cx;
    cx.mats = mats, cx.slope = slope, cx.camfast = camfast;
    cx.warp_base = smem_raw + align16(cta_table_bytes(p.N)) +
                   warp * warp_smem_layout(nullptr, nullptr, p.slots, p.colcap, p.wcap, p.ct, p.ct * p.N, p.den_bytes);
    const WarpSmem sm = warp_smem(p, cx.warp_base);

    // Programmatic dependent launch: let the next grid of the stream place its CTAs while this one drains, and (as the
    // dependent of the grid before) touch no global memory until that grid has completed and its writes are visible.
    // Both are no-ops for a launch without the attribute.
    if (!BWD) {
        asm volatile("griddepcontrol.launch_dependents;");
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }

    // ---- per-CTA tables: camera matrices (scaled to feature texels), condition slopes, camera class, cell positions
    for (int i = tid; i < p.N * 12; i += THREADS) {
        const int n = i / 12, e = i - n * 12;
        double v = (double)__ldg(p.l2i + ((size_t)b * p.N + n) * 16 + e);
        if (e < 4) v *= p.sx;
        else if (e < 8) v *= p.sy;
        mats[i] = v;
    }
    for (int n = tid; n < p.N; n += THREADS) {
        const float *M = p.l2i + ((size_t)b * p.N + n) * 16;
        const double m2 = (double)__ldg(M + 2) * p.sx, m6 = (double)__ldg(M + 6) * p.sy, m10 = (double)__ldg(M + 10);
        // d/dk of: depth - 0.1, p0s, Wf d - p0s, p1s, Hf d - p1s
        slope[n * 5 + 0] = (float)(m10 * p.dz);
        slope[n * 5 + 1] = (float)(m2 * p.dz);
        slope[n * 5 + 2] = (float)(((double)p.Wf * m10 - m2) * p.dz);
        slope[n * 5 + 3] = (float)(m6 * p.dz);
        slope[n * 5 + 4] = (float)(((double)p.Hf * m10 - m6) * p.dz);
        camfast[n] = (m10 == 0.0 && m2 == 0.0) ? 1 : 0;
    }
    for (int c = tid; c < kMaxCt; c += THREADS) {
        int v = 0;
        if (c < p.ct) {
            const int s = c / p.cpw, j = c - s * p.cpw;  // sub-block, cell inside it
            const int si = s / p.sby, sj = s - si * p.sby;
            const int jx = j / p.wy, jy = j - jx * p.wy;
            v = (si * p.wx + jx) | ((sj * p.wy + jy) << 8);
        }
        celltab[c] = v;
    }
    __syncthreads();  // the only CTA-wide barrier

    // ---- gather role of this lane inside a sub-block
    const int cg = (lane * p.inv_g) >> 16, gl = lane - cg * p.g;  // lane / g
    const bool role = cg < p.cpw;
    constexpr bool kWide = WIDE && V >= 2 && !BWD;
    const int vstep = kWide ? 1 : p.g;  // distance between the lane's channel vectors
    const int vec0 = kWide ? (blockIdx.y * p.g + gl) * V : blockIdx.y * (p.g * V) + gl;  // the lane's first vector
    // channel vectors past the end of the row (ragged last channel block) re-read vector 0, never stored
    const uint4 *featv[V];
    float4 *gfv[V];  // backward: where this lane's channel vectors of a texel's gradient live
    {
        const size_t cam0 = (size_t)b * p.N * p.Hf * p.Wf * p.vecs;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int vi = (vec0 + v * vstep < p.vecs) ? vec0 + v * vstep : 0;
            featv[v] = BWD ? nullptr : static_cast<const uint4 *>(p.feat) + cam0 + vi;
            gfv[v] = BWD ? reinterpret_cast<float4 *>(p.gfeat) + cam0 + vi : nullptr;
        }
    }
    const int out_lane = vec0 * (PV * 2), vstride = vstep * (PV * 2);  // channel of the lane's first vector; channels between its vectors
    bool von[V];                                                         // the lane's v-th vector exists (ragged last channel block)
#pragma unroll
    for (int v = 0; v < V; ++v) von[v] = vec0 + v * vstep < p.vecs;
    const int my_tab = celltab[lane];
    const unsigned roff_s = (unsigned)__cvta_generic_to_shared(sm.roff), rw_s = (unsigned)__cvta_generic_to_shared(sm.rw);

    for (int rep = 0; rep < p.reps; ++rep) {
        // ---- which super-block: ids run along y inside bands of `band` rows of super-blocks
        int id = (blockIdx.x * WARPS + warp) * p.reps + rep;
        // The last super-blocks of the order are handed out one sub-block per warp: short tasks for the end of the
        // grid, when the SMs run out of work one warp at a time.
        int s_begin = 0, s_end = p.sbn;
        if (id >= p.whole_tasks) {
            const int k = id - p.whole_tasks, q = k / p.sbn;
            id = p.whole_tasks + q, s_begin = k - q * p.sbn, s_end = s_begin + 1;
        }
        if (id >= p.total_sbs) continue;  // (padding warps of the last CTA; warp-uniform)
        const int per_band = p.band * p.blocks_y;
        int bandi = id / per_band;
        const int rem = id - bandi * per_band;
        if (p.centre_out) {  // bands from the middle of the grid outwards: the cells around the ego write the most records
            const int half = (bandi + 1) >> 1;
            bandi = ((p.nbands - 1) >> 1) + ((bandi & 1) ? half : -half);
        }
        const int by = rem / p.band, bx = bandi * p.band + (rem - by * p.band);
        if ((unsigned)bx >= (unsigned)p.blocks_x || (unsigned)by >= (unsigned)p.blocks_y) continue;  // past the grid's edge; warp-uniform
        const int ix0 = bx * (p.sbx * p.wx), iy0 = by * (p.sby * p.wy);

        unsigned in_mask;  // bit c: cell c of the super-block is inside the grid
        {
            const int lx = my_tab & 0xff, ly = my_tab >> 8;
            const bool in = (lane >= s_begin * p.cpw) && (lane < s_end * p.cpw) && (ix0 + lx < p.X) && (iy0 + ly < p.Y);
            const double nan = __longlong_as_double(0x7ff8000000000000LL);
            if (lane < p.ct)
                sm.cellxy[lane] = make_double2(in ? p.x_min + ((double)(ix0 + lx) + 0.5) * p.dx : nan,
                                               in ? p.y_min + ((double)(iy0 + ly) + 0.5) * p.dy : nan);
            in_mask = __ballot_sync(FULL, in);
        }
        __syncwarp();
        survey_candidates(p, cx, in_mask);

        // ---- segments: as many sub-blocks as have at most `colcap` surviving columns together (normally all of them)
        for (int s0 = s_begin; s0 < s_end;) {
            const int jb = sm.cfirst[s0 * p.cpw];
            int s1 = s0 + 1;
            while (s1 < s_end && sm.cfirst[min((s1 + 1) * p.cpw, p.ct)] - jb <= p.colcap) ++s1;
            const int ncols = sm.cfirst[min(s1 * p.cpw, p.ct)] - jb;  // <= colcap: a sub-block has at most cpw * N candidates
            const int nw = build_columns(p, cx, jb, ncols, s0 * p.cpw, min(s1 * p.cpw, p.ct));

            // ---- rounds: the runs of as many whole sub-blocks as fit the record slots are walked together (one lane
            // per run), then the sub-blocks are gathered one by one
            int wa = 0, wb = 0;  // the current round holds runs [wa, wb)
            for (int s = s0; s < s1; ++s) {
                const int cell = s * p.cpw + (role ? cg : 0);
                const bool lane_on = role && ((in_mask >> cell) & 1u);
                const int tab = celltab[cell];
                // (lanes without a cell inside the grid never use it)
                const size_t ocell = lane_on ? (size_t)FB_IDX(((size_t)b * p.X + (ix0 + (tab & 0xff))) * p.Y + (iy0 + (tab >> 8)),
                                                              (size_t)p.B * p.X * p.Y, p.err) : 0;
                const int sw_lo = sm.colw[sm.cfirst[s * p.cpw] - jb], sw_hi = sm.colw[sm.cfirst[min((s + 1) * p.cpw, p.ct)] - jb];
                const int cw_lo = sm.colw[sm.cfirst[cell] - jb], cw_hi = sm.colw[sm.cfirst[cell + 1] - jb];  // this lane's cell
                const int sub_records = sm.woff[sw_hi] - sm.woff[sw_lo];
                const bool oversized = sub_records > p.slots;
                if (!oversized && sw_hi > wb) {
                    __syncwarp();
                    wa = sw_lo, wb = sw_hi;
                    for (int s2 = s + 1; s2 < s1; ++s2) {
                        const int hi2 = sm.colw[sm.cfirst[min((s2 + 1) * p.cpw, p.ct)] - jb];
                        if (sm.woff[hi2] - sm.woff[wa] > p.slots) break;
                        wb = hi2;
                    }
                    const int base = sm.woff[wa];
                    for (int w = wa + lane; w < wb; w += 32) walk_one(p, sm, mats, w, sm.woff[w] - base);
                    __syncwarp();
                }

                float2 acc[V][PV];
#pragma unroll
                for (int v = 0; v < V; ++v)
#pragma unroll
                    for (int e = 0; e < PV; ++e) acc[v][e] = make_float2(0.f, 0.f);
                float4 go[V];  // backward: this lane's channel vectors of the cell's output gradient
                bool on[V];
                if (BWD) {
                    const int count = sm.cnt[cell];
                    const float gscale = (p.reduce == FLASHBEV_REDUCE_MEAN_OVER_VALID) ? 1.f / (float)(count > 1 ? count : 1) : 1.f;
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        const int vi = vec0 + v * vstep;
                        go[v] = make_float4(0.f, 0.f, 0.f, 0.f);
                        on[v] = lane_on && vi < p.vecs;
                        if (on[v] && cw_hi > cw_lo) {
                            go[v] = __ldg(reinterpret_cast<const float4 *>(p.gout + ocell * p.C) + vi);
                            go[v].x *= gscale, go[v].y *= gscale, go[v].z *= gscale, go[v].w *= gscale;
                        }
                    }
                }

                if (!oversized) {
                    const int c0 = sm.woff[cw_lo] - sm.woff[wa];
                    const int nrec = lane_on ? sm.woff[cw_hi] - sm.woff[cw_lo] : 0;
                    if (BWD) {
                        if (nrec > 0) scatter_list<V>(go, on, sm.roff + c0, sm.rw + c0, nrec, p.rstep, gfv);
                    } else {
                        gather_list<V, BF16, kWide>(acc, roff_s + 4 * c0, rw_s + 8 * c0, nrec, (unsigned)p.rstep, featv);
                    }
                } else {
                    // A sub-block whose records exceed the slots: several rounds of as many runs as fit, in order; the
                    // accumulators live across the walkers here.
                    int pos = sw_lo;
                    while (pos < sw_hi) {
                        __syncwarp();
                        const int base = sm.woff[pos];
                        int upto = pos;
                        for (int w0 = pos + 1; w0 <= sw_hi; w0 += 32) {
                            const int w = w0 + lane;
                            const bool fits = w <= sw_hi && sm.woff[w] - base <= p.slots;
                            const unsigned bal = __ballot_sync(FULL, fits);
                            upto = w0 - 1 + __popc(bal);
                            if (bal != FULL) break;
                        }
                        if (upto <= pos) upto = pos + 1;  // (cannot happen: one run always fits; never loop without progress)
                        for (int w = pos + lane; w < upto; w += 32) walk_one(p, sm, mats, w, sm.woff[w] - base);
                        __syncwarp();
                        // this lane's cell: its runs inside [pos, upto)
                        const int lw = min(max(cw_lo, pos), upto), hw = min(max(cw_hi, pos), upto);
                        const int c0 = sm.woff[lw] - base;
                        const int nrec = lane_on ? sm.woff[hw] - sm.woff[lw] : 0;
                        if (BWD) {
                            if (nrec > 0) scatter_list<V>(go, on, sm.roff + c0, sm.rw + c0, nrec, p.rstep, gfv);
                        } else {
                            gather_list<V, BF16, kWide>(acc, roff_s + 4 * c0, rw_s + 8 * c0, nrec, (unsigned)p.rstep, featv);
                        }
                        pos = upto;
                    }
                    wa = wb = sw_hi;
                }
                if (BWD) continue;

                // ---- the one store of every output vector
                if (lane_on) {
                    const int count = sm.cnt[cell];
                    if (p.reduce == FLASHBEV_REDUCE_MEAN_OVER_VALID) {
                        const float gn = 1.f / (float)(count > 1 ? count : 1);
#pragma unroll
                        for (int v = 0; v < V; ++v)
#pragma unroll
                            for (int e = 0; e < PV; ++e) acc[v][e].x *= gn, acc[v][e].y *= gn;
                    }
                    float *o = p.out + ocell * p.C + out_lane;  // this lane's first channel of the cell
                    if (PLANAR) {
                        // one scalar per channel: out[b][cell][channel] with the strides of the caller's layout (planar:
                        // the cells of a sub-block are adjacent in y; ragged channels-last rows: channels adjacent)
                        const size_t plane = (size_t)p.X * p.Y;
                        const size_t at = (size_t)b * p.out_bs + (ocell - (size_t)b * plane) * p.out_cells;
#pragma unroll
                        for (int v = 0; v < V; ++v)
                            if (von[v]) {
#pragma unroll
                                for (int e = 0; e < PV; ++e) {
#pragma unroll
                                    for (int hl = 0; hl < 2; ++hl) {
                                        const int ch = out_lane + v * vstride + e * 2 + hl;
                                        if (ch >= p.out_c) continue;  // (padding channels of the copy)
                                        const size_t idx = FB_IDX64(at + (size_t)ch * p.out_chs, (size_t)p.B * p.out_bs, p.err);
                                        float val = hl ? acc[v][e].y : acc[v][e].x;
                                        if (p.out_bf16) {
                                            uint16_t *ob = reinterpret_cast<uint16_t *>(p.out) + idx;
                                            if (p.accumulate) val += __bfloat162float(__ushort_as_bfloat16(*ob));
                                            *ob = __bfloat16_as_ushort(__float2bfloat16_rn(val));
                                        } else {
                                            if (p.accumulate) val += p.out[idx];
                                            __stcs(p.out + idx, val);
                                        }
                                    }
                                }
                            }
                    } else if (!(p.accumulate | p.out_bf16)) {
#pragma unroll
                        for (int v = 0; v < V; ++v)
                            if (von[v]) {
#pragma unroll
                                for (int e = 0; e < PV; e += 2)
                                    __stcs(reinterpret_cast<float4 *>(o + v * vstride + e * 2),
                                           make_float4(acc[v][e].x, acc[v][e].y, acc[v][e + 1].x, acc[v][e + 1].y));
                            }
                    } else {
#pragma unroll
                        for (int v = 0; v < V; ++v)
                            if (von[v]) {
#pragma unroll
                                for (int e = 0; e < PV; e += 2) {
                                    float4 *dst = reinterpret_cast<float4 *>(o + v * vstride + e * 2);
                                    float4 val = make_float4(acc[v][e].x, acc[v][e].y, acc[v][e + 1].x, acc[v][e + 1].y);
                                    if (p.accumulate) {  // multi-resolution levels after the first: `dst` holds the other levels' sum
                                        const float4 prev = *dst;
                                        val.x += prev.x, val.y += prev.y, val.z += prev.z, val.w += prev.w;
                                    }
                                    if (p.out_bf16) {
                                        uint16_t *ob = reinterpret_cast<uint16_t *>(p.out) + ocell * p.C + out_lane;
                                        *reinterpret_cast<uint2 *>(ob + v * vstride + e * 2) =
                                            make_uint2(pack_bf16x2(val.x, val.y), pack_bf16x2(val.z, val.w));
                                    } else {
                                        __stcs(dst, val);
                                    }
                                }
                            }
                    }
                    if (p.count_out && gl == 0 && blockIdx.y == 0) p.count_out[ocell] = count;
                }
            }
            s0 = s1;
        }
        __syncwarp();
    }
}
