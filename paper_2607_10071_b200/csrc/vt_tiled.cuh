// Tiled Sampling-VT kernel (forward and backward) for B200 (sm_100a).  Included by flashbev.cu inside its
// anonymous namespace, after the shared helpers (KParams, fast_rcp, kDepthMin, FB_IDX).
//
// A WARP owns a sub-block of up to 8 adjacent BEV cells and works through it alone (__syncwarp only; the CTA
// shares nothing but the per-batch-element camera tables staged once at kernel start).  Everything that does
// not depend on the channel is computed once per (cell, camera, height) and turned into a compact list of
// "row records" in shared memory before a single feature is read (paper Sec. 3.3: the projection, validity
// test and bilinear weights of Algorithm 2, hoisted out of the channel dimension):
//
//   1. columns   one lane per (cell, camera): the five validity conditions are linear in the height once the
//                depth is positive, so the valid height bins of a column form one interval [klo, khi]; it is
//                found in closed form (float, conservative) and its two ends are confirmed with the exact
//                fp64 test.  The surviving columns are compacted (ballot) into column descriptors.  The cell's
//                valid-sample count and the per-height camera counts of Eq. 1 follow from the intervals alone.
//   2. items     the columns' work is cut into items that the 32 lanes take in order, one item per lane:
//                - a camera without pitch or roll sees a column under one texel column (x0, tx constant) with
//                  fy affine in the bin index; if several bins share a texel row the item is a texel ROW: the
//                  bins that fall into it and their summed weights are arithmetic series (closed form);
//                - otherwise the item is a height BIN; the lane that starts a run of bins on the same texel
//                  rows sums the run (and the lower-row weights of the run just before it, when that run ends
//                  one row above), so successive bins that touch the same row still give one record.
//                Records {left tap, right tap, wL, wR} are written in item order at positions given by a
//                ballot/popc prefix: no atomics, the list of every cell is contiguous and its order fixed.
//   3. gather    g lanes per cell, V 16-byte channel vectors per lane: per record two 128- or 256-bit loads per
//                vector and packed fp32 FMAs into register accumulators.  A list that does not fit its slots is
//                consumed in several rounds; the accumulators stay in registers, so every output vector is
//                written exactly once, with a streaming store.
// The backward instance replaces step 3 by the transpose: fp32 vector reductions of w * grad_out into the
// feature gradient.
//
// Shared memory (dynamic):
//   CTA  : double mats[N][12]   rows 0..2 of lidar2img[b][n], rows 0/1 pre-scaled to feature texels
//          float  slope[N][5]   d/dk of the five validity conditions
//          int    camfast[N]    1: the camera's depth and horizontal texel coordinate do not depend on height
//   warp : int4    rec[slots]    row records of the current round
//          ColDesc col[ncap]     descriptors of the valid columns (ncap = cells * N)
//          double2 cellxy[8]     voxel-centre (x_w, y_w) of the cells (NaN: outside the grid)
//          int     cfirst[9], cstart[8], cend[8], cnt[8]
//          uint8   den[cells * Z]   cameras per (cell, height bin), Eq. 1 mode only

constexpr int kMaxCells = 8;        // cells per warp
constexpr int kKindRows = 0;        // item = texel row of a height-independent column (closed form)
constexpr int kKindBinsFast = 1;    // item = height bin, height-independent column
constexpr int kKindBinsGeneral = 2; // item = height bin, full projection per bin

struct __align__(16) ColDesc {
    double a, s;     // fast: fy(k') = a + k' s, rows ascending with k' (s >= 0); general: a0, a1 (rows 0/1 at z = 0)
    double inv;      // rows: ~1 / s; general: a2 (row 2 at z = 0)
    int offc;        // fast: vector index of the left loadable texel of the column at row 0
    int r0;          // fast: floor(a)
    float cl, cr;    // fast: horizontal weights of the two loadable texels (an out-of-map tap is folded to weight 0)
    int istart;      // first item of the column in the warp's item order
    int nitems;
    int kk;          // klo | khi << 16
    int meta;        // cell | camera << 8 | kind << 16 | reversed << 18 | first column of cell << 19 | last << 20
    int pad0, pad1;
};
static_assert(sizeof(ColDesc) == 64, "column descriptor is four 16-byte words");

struct WarpSmem {
    int4 *rec;
    ColDesc *col;
    double2 *cellxy;
    int *cfirst, *cstart, *cend, *cnt;
    unsigned char *den;
};

__host__ __device__ inline size_t align16(size_t v) { return (v + 15) & ~(size_t)15; }

__host__ __device__ inline size_t cta_table_bytes(int N)
{
    return align16((size_t)N * 12 * sizeof(double)) + align16((size_t)N * 5 * sizeof(float)) + align16((size_t)N * sizeof(int));
}

__host__ __device__ inline size_t warp_smem_layout(unsigned char *base, WarpSmem *t, int slots, int ncap, int den_bytes)
{
    size_t o = 0;
    auto take = [&](size_t bytes) {
        unsigned char *ptr = base ? base + o : nullptr;
        o += align16(bytes);
        return ptr;
    };
    unsigned char *p0 = take((size_t)slots * sizeof(int4));
    unsigned char *p1 = take((size_t)ncap * sizeof(ColDesc));
    unsigned char *p2 = take((size_t)kMaxCells * sizeof(double2));
    unsigned char *p3 = take((size_t)(4 * kMaxCells + 4) * sizeof(int));
    unsigned char *p4 = take((size_t)den_bytes);
    if (t) {
        t->rec = reinterpret_cast<int4 *>(p0);
        t->col = reinterpret_cast<ColDesc *>(p1);
        t->cellxy = reinterpret_cast<double2 *>(p2);
        t->cfirst = reinterpret_cast<int *>(p3);
        t->cstart = t->cfirst + kMaxCells + 1;
        t->cend = t->cstart + kMaxCells;
        t->cnt = t->cend + kMaxCells;
        t->den = p4;
    }
    return o;
}

// One height bin of a column: bilinear corner (x0, y0), vertical fraction, and the horizontal weights of the
// two texels that are actually loaded (xc, xc + 1 with xc inside the map; an out-of-map tap weighs 0).
struct Tap {
    int x0, y0, xc;
    float cl, cr, ty;
};

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

// Gather of one cell list by its channel lanes, U records per iteration.  Every record is two taps of one
// texel row, both always loadable.  Lanes whose list is shorter than the warp's longest repeat their last
// record with weight 0; lanes with no records do nothing.
template <int V, bool BF16, bool WIDE>
__device__ __forceinline__ void gather_list(float2 (&acc)[V][BF16 ? 4 : 2], const int4 *list, int nrec, int maxn,
                                            const uint4 *const (&featv)[V])
{
    constexpr int U = V == 1 ? 4 : (V == 2 ? (BF16 ? 3 : 2) : 1);
    if (nrec <= 0) return;
    const int last = nrec - 1;
    for (int j = 0; j < maxn; j += U) {
        int4 r[U];
#pragma unroll
        for (int u = 0; u < U; ++u) r[u] = list[min(j + u, last)];
        uint4 t[U][2][V];
        if (WIDE) {  // the lane's vectors are adjacent: V / 2 loads of 32 bytes per tap
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int v = 0; v + 1 < V; v += 2) {
                    ldg_pair(featv[v] + r[u].x, t[u][0][v], t[u][0][v + 1]);
                    ldg_pair(featv[v] + r[u].y, t[u][1][v], t[u][1][v + 1]);
                }
        } else {
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    t[u][0][v] = __ldg(featv[v] + r[u].x);
                    t[u][1][v] = __ldg(featv[v] + r[u].y);
                }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const bool has = j + u <= last;
            const float wl = has ? __int_as_float(r[u].z) : 0.f;
            const float wr = has ? __int_as_float(r[u].w) : 0.f;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                fma_vec<BF16>(acc[v], t[u][0][v], make_float2(wl, wl));
                fma_vec<BF16>(acc[v], t[u][1][v], make_float2(wr, wr));
            }
        }
    }
}

// Backward of the gather: every record adds its two weighted taps of the cell's output gradient to the
// feature gradient (the transpose of gather_list).  Vector reductions: texels are shared by cells.
template <int V>
__device__ __forceinline__ void scatter_list(const float4 (&go)[V], const bool (&on)[V], const int4 *list, int nrec,
                                             float4 *const (&gfv)[V])
{
    for (int j = 0; j < nrec; ++j) {
        const int4 r = list[j];
        const float wl = __int_as_float(r.z), wr = __int_as_float(r.w);
#pragma unroll
        for (int v = 0; v < V; ++v) {
            if (!on[v]) continue;  // ragged last channel block
            if (wl != 0.f) atomicAdd(gfv[v] + r.x, make_float4(go[v].x * wl, go[v].y * wl, go[v].z * wl, go[v].w * wl));
            if (wr != 0.f) atomicAdd(gfv[v] + r.y, make_float4(go[v].x * wr, go[v].y * wr, go[v].z * wr, go[v].w * wr));
        }
    }
}

// ---- step 1: one candidate column (cell c, camera n) -----------------------------------------------------
// Returns false if no height bin of the column is valid; otherwise fills the descriptor (all but istart and the
// first / last flags).
__device__ __forceinline__ bool make_column(const KParams &p, const double *mats, const float *slope, const int *camfast,
                                            double2 xy, int c, int n, ColDesc &D)
{
    const double *m = mats + n * 12;
    const float *sl = slope + n * 5;
    const double zc0 = p.z_min + 0.5 * p.dz;  // centre of bin 0; z_w(k) = zc0 + k dz
    const double a0 = fma(m[1], xy.y, fma(m[0], xy.x, m[3]));
    const double a1 = fma(m[5], xy.y, fma(m[4], xy.x, m[7]));
    const double a2 = fma(m[9], xy.y, fma(m[8], xy.x, m[11]));
    const double wlim = (double)p.Wf - 0.5, hlim = (double)p.Hf - 0.5;

    // conditions alpha + beta * k > 0 (k real): depth, left, right, top, bottom -> conservative interval
    float lo = -1.f, hi = (float)p.Z;
    bool empty = false;
    auto cond = [&](float a, float bslope) {
        if (bslope > 0.f) lo = fmaxf(lo, -a * __frcp_rn(bslope));       // k > -a/b
        else if (bslope < 0.f) hi = fminf(hi, -a * __frcp_rn(bslope));  // k < -a/b
        else if (a <= 0.f) empty = true;  // independent of z (NaN: keep, tested exactly below)
    };
    const double d0 = fma(m[10], zc0, a2);
    cond((float)(d0 - kDepthMin), sl[0]);
    if (empty || !(lo < hi)) return false;
    const double p00 = fma(m[2], zc0, a0);
    cond((float)p00, sl[1]);
    cond((float)fma((double)p.Wf, d0, -p00), sl[2]);
    if (empty || !(lo < hi)) return false;
    const double p10 = fma(m[6], zc0, a1);
    cond((float)p10, sl[3]);
    cond((float)fma((double)p.Hf, d0, -p10), sl[4]);
    if (empty) return false;
    // widen by a guard far above the float error, then confirm both ends exactly
    const float guard = 0.05f + 1e-5f * (float)p.Z;
    int klo = (int)floorf(fminf(fmaxf(lo - guard, -1.f), (float)p.Z)) + 1;
    int khi = (int)ceilf(fmaxf(fminf(hi + guard, (float)p.Z), -1.f)) - 1;
    klo = max(klo, 0);
    khi = min(khi, p.Z - 1);
    auto exact = [&](int k) {
        const double zw = fma((double)k, p.dz, zc0);
        const double d = fma(m[10], zw, a2);
        const double r = fast_rcp(d);  // d <= 0 or NaN gives inf / NaN: the tests below fail
        const double fx = fma(fma(m[2], zw, a0), r, -0.5);
        const double fy = fma(fma(m[6], zw, a1), r, -0.5);
        return (d > kDepthMin) & (fx > -0.5) & (fx < wlim) & (fy > -0.5) & (fy < hlim);
    };
    while (klo <= khi && !exact(klo)) ++klo;
    while (khi > klo && !exact(khi)) --khi;
    if (klo > khi) return false;

    const int nb = khi - klo + 1;
    D.kk = klo | (khi << 16);
    D.pad0 = D.pad1 = 0;
    D.istart = 0;
    if (camfast[n]) {
        // depth and fx do not depend on the height: one texel column, fy affine in the bin index
        const double r = fast_rcp(a2);
        const double fx = fma(a0, r, -0.5);
        const double flx = floor(fx);
        int xc;
        fold_x((int)flx, (float)(fx - flx), p.Wf, xc, D.cl, D.cr);
        const double ay = fma(p10, r, -0.5);   // fy of bin 0
        const double sy = m[6] * p.dz * r;     // fy step per bin
        const bool rev = sy < 0.0;
        D.s = rev ? -sy : sy;
        D.a = fma((double)(rev ? khi : klo), sy, ay);
        const double fl0 = floor(D.a);
        const double fln = floor(fma((double)(nb - 1), D.s, D.a));
        const int nrows = (int)(fln - fl0) + 2;
        const bool rows = p.reduce != FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM && nrows < nb && D.s >= 1e-9;
        D.inv = rows ? (double)__frcp_rn((float)D.s) : 0.0;
        D.offc = (n * p.Hf * p.Wf + xc) * p.vecs;
        D.r0 = (int)fl0;
        D.nitems = rows ? nrows : nb;
        D.meta = c | (n << 8) | ((rows ? kKindRows : kKindBinsFast) << 16) | ((rev ? 1 : 0) << 18);
    } else {
        D.a = a0, D.s = a1, D.inv = a2;
        D.offc = 0, D.r0 = 0, D.cl = D.cr = 0.f;
        D.nitems = nb;
        D.meta = c | (n << 8) | (kKindBinsGeneral << 16);
    }
    return true;
}

// ---- step 2: one item -> up to two row records -------------------------------------------------------------
struct ItemOut {
    bool va, vb;
    int4 ra, rb;
};

__device__ __forceinline__ void make_item(const KParams &p, const WarpSmem &sm, const double *mats, const ColDesc &D, int li,
                                          ItemOut &o)
{
    o.va = o.vb = false;
    const int kind = (D.meta >> 16) & 3;
    const int klo = D.kk & 0xffff, khi = D.kk >> 16, nb = khi - klo + 1;
    const int rowv = p.Wf * p.vecs;
    if (kind == kKindRows) {
        // texel row r of a height-independent column: the bins k' with floor(a + k' s) == r are k' in [k1, k2),
        // those of the row above [k0, k1); their (1 - ty) and ty sums are arithmetic series
        const int r = D.r0 + li;
        const double ay = D.a, sy = D.s, inv = D.inv;
        auto first_bin_at = [&](double rr) {  // smallest k' in [0, nb] with a + k' s >= rr
            double e = ceil((rr - ay) * inv);
            e = fmin(fmax(e, 0.0), (double)nb);  // NaN -> 0
            int k = (int)e;
            if (k > 0 && fma((double)(k - 1), sy, ay) >= rr) --k;
            else if (k < nb && fma((double)k, sy, ay) < rr) ++k;
            return k;
        };
        const double rr = (double)r;
        const int k0 = first_bin_at(rr - 1.0), k1 = first_bin_at(rr), k2 = first_bin_at(rr + 1.0);
        const double dm = (double)(k1 - k0), dn = (double)(k2 - k1);
        const double sum_ty_row = fma(dn, ay - rr, sy * (0.5 * dn * (double)(k1 + k2 - 1)));          // over [k1, k2)
        const double sum_ty_above = fma(dm, ay - (rr - 1.0), sy * (0.5 * dm * (double)(k0 + k1 - 1)));  // over [k0, k1)
        const float w = (float)((dn - sum_ty_row) + sum_ty_above);
        if (r >= 0 && r <= p.Hf - 1 && w != 0.f) {
            const int off = FB_IDX(D.offc + r * rowv, p.nvec_cam - p.vecs - p.rstep + 1, p.err);
            o.va = true;
            o.ra = make_int4(off, off + p.rstep, __float_as_int(D.cl * w), __float_as_int(D.cr * w));
        }
        return;
    }

    const bool general = kind == kKindBinsGeneral;
    const bool rev = (D.meta >> 18) & 1;
    const int cell = D.meta & 0xff, cam = (D.meta >> 8) & 0xff;
    const double *m = mats + cam * 12;
    const double zc0 = p.z_min + 0.5 * p.dz;
    auto eval = [&](int kp, Tap &t) {
        if (general) {
            const double zw = fma((double)(klo + kp), p.dz, zc0);
            const double d = fma(m[10], zw, D.inv);
            const double r = fast_rcp(d);
            const double fx = fma(fma(m[2], zw, D.a), r, -0.5);
            const double fy = fma(fma(m[6], zw, D.s), r, -0.5);
            const double flx = floor(fx), fly = floor(fy);
            t.x0 = (int)flx;
            t.y0 = (int)fly;
            t.ty = (float)(fy - fly);
            fold_x(t.x0, (float)(fx - flx), p.Wf, t.xc, t.cl, t.cr);
        } else {
            const double fy = fma((double)kp, D.s, D.a);
            const double fly = floor(fy);
            t.x0 = 0, t.xc = 0;
            t.y0 = (int)fly;
            t.ty = (float)(fy - fly);
            t.cl = D.cl, t.cr = D.cr;
        }
    };
    auto scale = [&](int kp) {  // Eq. 1: 1 / max(1, cameras that see this cell at this height)
        if (p.reduce != FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM) return 1.f;
        const int k = rev ? khi - kp : klo + kp;
        const unsigned dn = sm.den[FB_IDX(cell * p.Z + k, p.den_bytes, p.err)];
        return 1.f / (float)(dn > 1u ? dn : 1u);
    };

    Tap cur, pv;
    eval(li, cur);
    bool head = true;
    if (li > 0) {
        eval(li - 1, pv);
        head = !(pv.x0 == cur.x0 && pv.y0 == cur.y0);
    }
    if (!head) return;  // the lane that starts this run of bins covers it
    float uL = 0.f, uR = 0.f, lL = 0.f, lR = 0.f;
    bool next_continues = false;  // the next run starts on this run's lower row: its record takes our lower weights
    {
        int e = li;
        Tap t = cur;
        while (true) {
            const float s = scale(e);
            const float wy1 = t.ty * s, wy0 = (1.f - t.ty) * s;
            uL = fmaf(t.cl, wy0, uL), uR = fmaf(t.cr, wy0, uR);
            lL = fmaf(t.cl, wy1, lL), lR = fmaf(t.cr, wy1, lR);
            if (++e >= nb) break;
            eval(e, t);
            if (!(t.x0 == cur.x0 && t.y0 == cur.y0)) {
                next_continues = t.x0 == cur.x0 && t.y0 == cur.y0 + 1;
                break;
            }
        }
    }
    if (li > 0 && pv.x0 == cur.x0 && pv.y0 + 1 == cur.y0) {
        // the run before ended one row above: its lower-row weights belong to our upper row
        int b = li - 1;
        Tap t = pv;
        while (true) {
            const float wy1 = t.ty * scale(b);
            uL = fmaf(t.cl, wy1, uL), uR = fmaf(t.cr, wy1, uR);
            if (--b < 0) break;
            eval(b, t);
            if (!(t.x0 == pv.x0 && t.y0 == pv.y0)) break;
        }
    }
    const int offc = general ? (cam * p.Hf * p.Wf + cur.xc) * p.vecs : D.offc;
    const int r = cur.y0;
    if (r >= 0 && r <= p.Hf - 1 && (uL != 0.f || uR != 0.f)) {
        const int off = FB_IDX(offc + r * rowv, p.nvec_cam - p.vecs - p.rstep + 1, p.err);
        o.va = true;
        o.ra = make_int4(off, off + p.rstep, __float_as_int(uL), __float_as_int(uR));
    }
    if (!next_continues && r + 1 >= 0 && r + 1 <= p.Hf - 1 && (lL != 0.f || lR != 0.f)) {
        const int off = FB_IDX(offc + (r + 1) * rowv, p.nvec_cam - p.vecs - p.rstep + 1, p.err);
        o.vb = true;
        o.rb = make_int4(off, off + p.rstep, __float_as_int(lL), __float_as_int(lR));
    }
}

// WIDE: a lane's V channel vectors are adjacent (32-byte aligned pairs, 256-bit loads) instead of g apart
template <int V, bool BF16, int WARPS, bool BWD, bool WIDE>
__global__ void __launch_bounds__(WARPS * 32, (V == 4 ? 12 : 20) / WARPS)
    vt_tiled_kernel(const KParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int PV = BF16 ? 4 : 2;  // channel pairs per 16-byte vector
    constexpr int THREADS = WARPS * 32;
    constexpr unsigned FULL = 0xffffffffu;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned lt_mask = (1u << lane) - 1u;
    const int b = blockIdx.z;

    double *mats = reinterpret_cast<double *>(smem_raw);
    float *slope = reinterpret_cast<float *>(smem_raw + align16((size_t)p.N * 12 * sizeof(double)));
    int *camfast = reinterpret_cast<int *>(smem_raw + align16((size_t)p.N * 12 * sizeof(double)) +
                                           align16((size_t)p.N * 5 * sizeof(float)));
    WarpSmem sm;
    {
        const size_t per_warp = warp_smem_layout(nullptr, nullptr, p.slots, p.ncap, p.den_bytes);
        warp_smem_layout(smem_raw + cta_table_bytes(p.N) + warp * per_warp, &sm, p.slots, p.ncap, p.den_bytes);
    }

    // ---- per-CTA tables: camera matrices (scaled to feature texels), condition slopes, camera class
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
    // every record slot always holds loadable offsets: lanes may read (not use) slots past their list
    for (int i = lane; i < p.slots; i += 32) sm.rec[i] = make_int4(0, 0, 0, 0);
    __syncthreads();  // the only CTA-wide barrier

    // ---- gather role of this lane inside a sub-block
    const int cg = lane / p.g, gl = lane - cg * p.g;
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
    const int ncand = p.cpw * p.N;

    for (int rep = 0; rep < p.reps; ++rep) {
        // ---- which sub-block: ids run along y inside bands of `band` rows of sub-blocks
        const int id = (blockIdx.x * WARPS + warp) * p.reps + rep;
        const int per_band = p.band * p.blocks_y;
        const int bandi = id / per_band, rem = id - bandi * per_band;
        const int by = rem / p.band, bx = bandi * p.band + (rem - by * p.band);
        if (bx >= p.blocks_x) continue;  // warp-uniform
        const int ix0 = bx * p.wx, iy0 = by * p.wy;

        unsigned in_mask;  // bit c: cell c of the sub-block is inside the grid
        {
            const int lx = lane / p.wy, ly = lane - lx * p.wy;
            const bool in = (lane < p.cpw) && (ix0 + lx < p.X) && (iy0 + ly < p.Y);
            if (lane < kMaxCells) {
                const double nan = __longlong_as_double(0x7ff8000000000000LL);
                sm.cellxy[lane] = make_double2(in ? p.x_min + ((double)(ix0 + lx) + 0.5) * p.dx : nan,
                                               in ? p.y_min + ((double)(iy0 + ly) + 0.5) * p.dy : nan);
            }
            in_mask = __ballot_sync(FULL, in);
        }
        __syncwarp();

        // ---- step 1: columns, compacted in (cell, camera) order
        int ncols = 0;
        for (int p0 = 0; p0 < ncand; p0 += 32) {
            const int pr = p0 + lane;
            const int c = pr / p.N, n = pr - c * p.N;
            ColDesc D;
            bool valid = false;
            if (pr < ncand && ((in_mask >> c) & 1u)) valid = make_column(p, mats, slope, camfast, sm.cellxy[c], c, n, D);
            const unsigned bal = __ballot_sync(FULL, valid);
            const int idx = ncols + __popc(bal & lt_mask);
            if (pr < ncand && n == 0) sm.cfirst[FB_IDX(c, kMaxCells + 1, p.err)] = idx;  // where the cell's columns start
            if (valid) sm.col[FB_IDX(idx, p.ncap, p.err)] = D;
            ncols += __popc(bal);
        }
        if (lane == 0) sm.cfirst[p.cpw] = ncols;
        __syncwarp();

        // ---- item offsets of the columns (exclusive scan), first / last column of a cell, valid samples per cell
        int T = 0;
        for (int j0 = 0; j0 < ncols; j0 += 32) {
            const int j = j0 + lane;
            const int ni = j < ncols ? sm.col[j].nitems : 0;
            int x = ni;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int y = __shfl_up_sync(FULL, x, off);
                if (lane >= off) x += y;
            }
            if (j < ncols) {
                const int meta = sm.col[j].meta, c = meta & 0xff;
                sm.col[j].istart = T + x - ni;
                sm.col[j].meta = meta | ((j == sm.cfirst[c]) ? (1 << 19) : 0) | ((j + 1 == sm.cfirst[c + 1]) ? (1 << 20) : 0);
            }
            T += __shfl_sync(FULL, x, 31);
        }
        if (lane < p.cpw) {
            int n = 0;
            for (int j = sm.cfirst[lane]; j < sm.cfirst[lane + 1]; ++j) {
                const int kk = sm.col[j].kk;
                n += (kk >> 16) - (kk & 0xffff) + 1;
            }
            sm.cnt[lane] = n;
        }
        if (p.reduce == FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM) {
            // cameras per (cell, height bin): the columns' intervals say it all
            for (int i = lane; i < p.cpw * p.Z; i += 32) {
                const int c = i / p.Z, k = i - c * p.Z;
                int dn = 0;
                for (int j = sm.cfirst[c]; j < sm.cfirst[c + 1]; ++j) {
                    const int kk = sm.col[j].kk;
                    dn += (k >= (kk & 0xffff) && k <= (kk >> 16)) ? 1 : 0;
                }
                sm.den[FB_IDX(i, p.den_bytes, p.err)] = (unsigned char)dn;
            }
        }
        __syncwarp();

        float2 acc[V][PV];
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int e = 0; e < PV; ++e) acc[v][e] = make_float2(0.f, 0.f);

        const int cell = role ? cg : 0;
        const bool lane_on = role && ((in_mask >> cell) & 1u);
        const int my_lx = cell / p.wy, my_ly = cell - my_lx * p.wy;
        // (lanes without a cell inside the grid never use it)
        const size_t ocell = lane_on ? (size_t)FB_IDX(((size_t)b * p.X + (ix0 + my_lx)) * p.Y + (iy0 + my_ly),
                                                      (size_t)p.B * p.X * p.Y, p.err) : 0;

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
                if (on[v] && T > 0) {
                    go[v] = __ldg(reinterpret_cast<const float4 *>(p.gout + ocell * p.C) + vi);
                    go[v].x *= gscale, go[v].y *= gscale, go[v].z *= gscale, go[v].w *= gscale;
                }
            }
        }

        // ---- rounds: fill the record list from the items in order, then gather it
        int t0 = 0;
        while (t0 < T) {
            if (lane < kMaxCells) sm.cstart[lane] = 0, sm.cend[lane] = 0;
            __syncwarp();
            const int round_first = t0;
            int fill = 0;
            while (t0 < T && fill + 64 <= p.slots) {
                const int t = t0 + lane;
                const int pass_last = min(T, t0 + 32) - 1;
                ItemOut o;
                o.va = o.vb = false;
                int q = 0, li = 0, meta = 0, nitems = 0;
                if (t < T) {
                    int lo = 0, hi = ncols;  // istart[lo] <= t < istart[hi]
                    while (hi - lo > 1) {
                        const int mid = (lo + hi) >> 1;
                        if (sm.col[mid].istart <= t) lo = mid;
                        else hi = mid;
                    }
                    const ColDesc D = sm.col[FB_IDX(lo, p.ncap, p.err)];
                    li = t - D.istart;
                    meta = D.meta, nitems = D.nitems;
                    q = meta & 0xff;
                    make_item(p, sm, mats, D, li, o);
                }
                const unsigned ba = __ballot_sync(FULL, o.va), bb = __ballot_sync(FULL, o.vb);
                const int pos_a = fill + __popc(ba & lt_mask) + __popc(bb & lt_mask);
                const int pos_b = pos_a + (o.va ? 1 : 0);
                if (o.va) sm.rec[FB_IDX(pos_a, p.slots, p.err)] = o.ra;
                if (o.vb) sm.rec[FB_IDX(pos_b, p.slots, p.err)] = o.rb;
                if (t < T) {
                    if ((li == 0 && (meta & (1 << 19))) || t == round_first) sm.cstart[FB_IDX(q, kMaxCells, p.err)] = pos_a;
                    if ((li == nitems - 1 && (meta & (1 << 20))) || t == pass_last)
                        sm.cend[FB_IDX(q, kMaxCells, p.err)] = pos_b + (o.vb ? 1 : 0);
                }
                fill += __popc(ba) + __popc(bb);
                t0 += 32;
                __syncwarp();
            }
            if (t0 > T) t0 = T;

            const int c0 = sm.cstart[cell];
            const int nrec = lane_on ? sm.cend[cell] - c0 : 0;
            if (BWD) {
                if (nrec > 0) scatter_list<V>(go, on, sm.rec + c0, nrec, gfv);
            } else {
                const int maxn = __reduce_max_sync(FULL, nrec);
                gather_list<V, BF16, kWide>(acc, sm.rec + c0, nrec, maxn, featv);
            }
            __syncwarp();
        }
        if (BWD) continue;

        // ---- the one store of every output vector
        if (lane_on) {
            const int count = sm.cnt[cell];
            const float gn = (p.reduce == FLASHBEV_REDUCE_MEAN_OVER_VALID) ? 1.f / (float)(count > 1 ? count : 1) : 1.f;
            float *o = p.out + ocell * p.C;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const int vi = vec0 + v * vstep;
                if (vi < p.vecs) {
#pragma unroll
                    for (int e = 0; e < PV; e += 2) {
                        float4 *dst = reinterpret_cast<float4 *>(o + (size_t)vi * (PV * 2) + e * 2);
                        float4 val = make_float4(acc[v][e].x * gn, acc[v][e].y * gn, acc[v][e + 1].x * gn, acc[v][e + 1].y * gn);
                        if (p.accumulate) {  // multi-resolution levels after the first: `dst` holds the other levels' sum
                            const float4 prev = *dst;
                            val.x += prev.x, val.y += prev.y, val.z += prev.z, val.w += prev.w;
                        }
                        if (p.out_bf16) {
                            uint16_t *ob = reinterpret_cast<uint16_t *>(p.out) + ocell * p.C;
                            *reinterpret_cast<uint2 *>(ob + (size_t)vi * (PV * 2) + e * 2) =
                                make_uint2(pack_bf16x2(val.x, val.y), pack_bf16x2(val.z, val.w));
                        } else {
                            __stcs(dst, val);
                        }
                    }
                }
            }
            if (p.count_out && gl == 0 && blockIdx.y == 0) p.count_out[ocell] = count;
        }
        __syncwarp();
    }
}
