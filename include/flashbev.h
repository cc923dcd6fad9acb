/*
 * flashbev.h -- C ABI of the B200 (sm_100a) fused Sampling-VT library.
 *
 * One operator: the exact sampling-based BEV view transformation of the FlashBEV
 * paper, executed as a single fused gather-reduction (Sec. 3.3, Algorithm 2) so
 * that only the B x X x Y x C output is ever written and no height-dependent
 * intermediate exists.
 *
 * Plain C: pointers and sizes only.  Every pointer in `flashbev_vt_params` is a
 * DEVICE pointer unless the entry point says otherwise.  The caller owns every
 * buffer.  Unless an entry point says otherwise the library allocates nothing,
 * frees nothing, keeps no pointer after return, never synchronises the device,
 * and enqueues its work on the caller's stream.  It is re-entrant and thread safe; the only state it
 * keeps is per host thread (what flashbev_last_launch_count / flashbev_last_kernel_name report) and a
 * per-device cache of the multiprocessor count.
 */
#ifndef FLASHBEV_H_
#define FLASHBEV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FLASHBEV_VERSION 100 /* 0.1.0 */

typedef enum flashbev_status {
    FLASHBEV_OK = 0,
    FLASHBEV_INVALID_ARG = 1,  /* null pointer, non-positive size, empty range, unknown enum, short struct */
    FLASHBEV_UNSUPPORTED = 2,  /* a combination this version does not implement (the tiled kernel on NCHW or
                                  on rows that are not whole 16-byte vectors, sizes beyond the index ranges
                                  stated below) */
    FLASHBEV_MISALIGNED = 3,   /* `out` or `lidar2img` not 4-byte aligned, `features` not element aligned (tensors that are
                                  element- but not 16-byte aligned are served by the per-output kernel under AUTO and
                                  refused with FLASHBEV_UNSUPPORTED under FLASHBEV_KERNEL_TILED) */
    FLASHBEV_CUDA_ERROR = 4,   /* the launch (or a copy of the host entry point) failed; the CUDA error
                                  has been consumed with cudaGetLastError */
    FLASHBEV_TOO_SMALL = 5,    /* a caller-provided staging buffer is smaller than required */
    FLASHBEV_EXCEEDS_STATIC_STAGING = 6 /* flashbev_sampling_vt_host_static: the problem needs more than
                                           FLASHBEV_STATIC_STAGING_BYTES of device staging */
} flashbev_status;

typedef enum flashbev_dtype { FLASHBEV_F32 = 0, FLASHBEV_BF16 = 1 } flashbev_dtype;

/* NHWC: features [B][N][Hf][Wf][C] and out [B][X][Y][C], C contiguous (Algorithm 2 states the
 * output as B x X x Y x C): the fast layout.  NCHW: features [B][N][C][Hf][Wf] and out [B][C][X][Y]
 * (channel planes, as in Sec. 4.1); served by the per-output kernel only. */
typedef enum flashbev_layout { FLASHBEV_NHWC = 0, FLASHBEV_NCHW = 1 } flashbev_layout;

/*
 * Reduction over cameras n and height bins z (M_n = validity mask, f_n = bilinear sample):
 *   SUM               out = sum_z sum_n M_n f_n
 *   MEAN_OVER_VALID   out = (sum_z sum_n M_n f_n) / max(1, sum_z sum_n M_n)
 *   CAMERA_MEAN_Z_SUM out = sum_z [ sum_n M_n f_n / max(1, sum_n M_n) ]      (paper Eq. 1)
 */
typedef enum flashbev_reduce {
    FLASHBEV_REDUCE_SUM = 0,
    FLASHBEV_REDUCE_MEAN_OVER_VALID = 1,
    FLASHBEV_REDUCE_CAMERA_MEAN_Z_SUM = 2
} flashbev_reduce;

/* Kernel selection.  AUTO picks the tiled kernel whenever the channel row is a whole number of
 * 16-byte vectors, `features` and `out` are 16-byte aligned and the shape is one the tiled kernel can
 * be configured for; the per-output kernel (several times slower) otherwise --
 * flashbev_last_kernel_name() tells which one ran. */
typedef enum flashbev_kernel {
    FLASHBEV_KERNEL_AUTO = 0,
    FLASHBEV_KERNEL_PER_OUTPUT = 1, /* one thread per (cell, channel group), geometry recomputed per
                                       thread: the decomposition Algorithm 2 describes */
    FLASHBEV_KERNEL_TILED = 2       /* geometry once per (cell, camera, height) per warp tile, handed to the
                                       channel lanes through shared memory */
} flashbev_kernel;

/*
 * Operator description (Sec. 3.1 for the mathematics, Algorithm 2 for inputs and output).
 *
 * Geometry conventions:
 *   - voxel centres are bin centres: x_w(ix) = x_min + (ix + 1/2)(x_max - x_min)/X, likewise y, z
 *     (Sec. 4.1: [-50,50] m at 0.5 m <-> 200 bins);
 *   - lidar2img[b][n] is a row-major 4x4 float matrix taking homogeneous metres to
 *     (u*d, v*d, d) with (u, v) in full-resolution image pixels; row 3 is never read;
 *   - feature-map coordinates follow grid_sample(align_corners=False):
 *       fx = u * feat_w / img_w - 1/2,  fy = v * feat_h / img_h - 1/2;
 *   - M_n = 1 iff d > 0.1 and -1/2 < fx < feat_w - 1/2 and -1/2 < fy < feat_h - 1/2;
 *   - f_n is bilinear with zero padding; a valid sample counts once whatever number of its
 *     taps is in bounds.
 * Projection, validity, floor and the fractional parts are evaluated in fp64; interpolation
 * weights and accumulation are fp32.  Non-finite matrix entries make the affected samples
 * invalid; they never cause a fault.  The forward result is reproducible bit for bit from run to
 * run (no atomics, fixed summation order for a given launch configuration).
 *
 * Index ranges: N*feat_h*feat_w*C*sizeof(element) < 2^35 and B*X*Y < 2^31, N <= 64,
 * else FLASHBEV_UNSUPPORTED.
 */
typedef struct flashbev_vt_params {
    size_t struct_size;        /* sizeof(flashbev_vt_params) of the caller's header */
    const void *features;      /* [B][N][feat_h][feat_w][C], element type feat_dtype; read only */
    int32_t feat_dtype;        /* flashbev_dtype */
    int32_t layout;            /* flashbev_layout */
    const float *lidar2img;    /* [B][N][4][4] float32; read only */
    int32_t B, N, C;
    int32_t feat_h, feat_w;    /* feature map size (texels) */
    int32_t img_h, img_w;      /* full-resolution image size (pixels) the matrices project to */
    double x_min, x_max;       /* BEV ranges, metres; max > min */
    double y_min, y_max;
    double z_min, z_max;
    int32_t X, Y, Z;           /* number of bins per axis */
    int32_t reduce;            /* flashbev_reduce */
    void *out;                 /* [B][X][Y][C] (NHWC) or [B][C][X][Y] (NCHW), element type out_dtype; every
                                  element is written (cells no camera sees get 0): no pre-zeroing needed */
    int32_t out_dtype;         /* FLASHBEV_F32, or FLASHBEV_BF16: the fp32 result rounded to nearest even once */
    int32_t kernel;            /* flashbev_kernel */
    int32_t *valid_count_out;  /* optional [B][X][Y] int32: sum_z sum_n M_n per cell; NULL to skip */
    int32_t tune[4];           /* launch-geometry hints of the tiled kernel, 0 = library defaults (they never change the
                                  result beyond fp32 summation order).  tune[0]: channel vectors per lane (1,2,4);
                                  tune[1]: lanes per cell; tune[2]: height bins (or texel rows) per geometry run, rounded
                                  down to a power of two; tune[3]: bits 0-3 warps per CTA (1,2,4,8), bits 4-7 / 8-11
                                  sub-blocks per warp in x / y, bits 12-15 super-blocks per warp, bit 16 never / bit 17
                                  always use 256-bit feature loads, bits 18-19 band height of the super-block order
                                  (2,1,4,8), bits 20-27 record slots per warp in units of 16, bit 28 visit the bands in
                                  row order instead of from the middle of the grid outwards, bits 29-31 how many of the
                                  last super-blocks are handed out one sub-block per warp (0 default; 1..7 = 0, 1/4, 1/2,
                                  1, 3/2, 2, 3 short tasks per resident warp slot).  Values that do not fit fall back
                                  to the defaults */
    uint32_t *debug_error_word; /* optional DEVICE word, or NULL.  Only the bounds-checked build of the library
                                  (-DFLASHBEV_DEBUG_BOUNDS) uses it: every shared-memory slot, record offset and
                                  output index the tiled kernel computes is range-checked there; an index out of
                                  range is counted into this word (atomically) and replaced by a safe one, never
                                  dereferenced.  The caller zeroes the word before the call and reads it after
                                  synchronising.  The normal build ignores it.  Callers built against an older
                                  header (struct_size without this field) are accepted. */
    void *workspace;           /* optional DEVICE scratch, 16-byte aligned, or NULL.  Two kinds of tensors use it,
                                  with flashbev_workspace_bytes(p) bytes here: channel-planar (NCHW) features are
                                  first transposed into it (channels last), and channels-last features whose rows
                                  are not whole 16-byte vectors are copied into it with zero-padded rows; the
                                  tiled kernel then runs on the copy and writes the output in the caller's own
                                  layout.  Without it such tensors take the generic per-output kernel (several
                                  times to an order of magnitude slower).  Callers built against a header without
                                  these two fields are accepted. */
    size_t workspace_bytes;    /* size of `workspace` */
} flashbev_vt_params;

/*
 * The operator (Eq. 1; Algorithm 2).  Validates `p` on the host (no CUDA call is made and no
 * device memory is touched when validation fails), then enqueues exactly one kernel on `stream`
 * (two for NCHW tensors with a workspace: a transposing copy first) and returns without waiting
 * (`stream` is a cudaStream_t, passed as void*; NULL = the default stream).
 * Uses no device memory beyond `features`, `lidar2img`, `out`, `valid_count_out` and `workspace`.
 * The tiled kernel is launched with programmatic stream serialization: its thread blocks may be
 * placed on the SMs while the kernel before it in the stream is still draining, and wait there for
 * that kernel's completion before they read or write any global memory -- stream order as seen
 * through memory is unchanged.  The environment variable FLASHBEV_NO_PDL turns this off.
 */
flashbev_status flashbev_sampling_vt(const flashbev_vt_params *p, void *stream);

/* Device scratch the operator can use beyond its inputs and outputs.  0 for channels-last (NHWC)
 * tensors with rows of whole 16-byte vectors (Sec. 3.3.1: all intermediates live in registers / on
 * chip).  For NCHW tensors with such rows: the size of a channels-last copy of the features; for
 * channels-last tensors with other channel counts: the size of a copy with the rows padded to whole
 * vectors.  `workspace` may lend it to the call (optional; see the field). */
size_t flashbev_workspace_bytes(const flashbev_vt_params *p);

/*
 * Same operator for callers whose data lives in HOST memory.  `p->features`, `p->lidar2img`,
 * `p->out` (and `p->valid_count_out` if not NULL) are HOST pointers here (pinned memory makes the
 * copies asynchronous).  `d_staging` is a caller-owned DEVICE buffer of at least
 * flashbev_host_staging_bytes(p) bytes, 256-byte aligned.  Enqueues on `stream`: host->device
 * copies of features and matrices, the kernel, device->host copy of the output; returns without
 * waiting -- synchronise `stream` before reading `out`.  Allocates nothing.
 */
flashbev_status flashbev_sampling_vt_host(const flashbev_vt_params *p, void *d_staging,
                                          size_t staging_bytes, void *stream);
/* 0 if `p` is invalid.  For NCHW tensors the figure includes flashbev_workspace_bytes(p) of scratch for the
 * channels-last copy; a buffer without that last part is accepted and the generic kernel runs. */
size_t flashbev_host_staging_bytes(const flashbev_vt_params *p);

/*
 * Host-buffer variant that needs no device buffer from the caller and never allocates.
 * (The paper has no counterpart: this exists for deployment, not for the method.)
 *
 * Who needs it: callers that are not allowed to create device memory at the point where they call
 * -- an inference-engine plugin that was handed no workspace, a perception loop whose memory budget
 * is frozen after start-up, code running while other streams must not be disturbed (cudaMalloc and
 * cudaFree synchronise the whole device), or a component that simply has no allocator to ask.
 *
 * Same contract as flashbev_sampling_vt_host (all pointers in `p` are HOST pointers, work is
 * enqueued on `stream`, synchronise the stream before reading `out`), except that the device
 * staging area is a fixed array of FLASHBEV_STATIC_STAGING_BYTES bytes that is part of the
 * library image: every GPU on which the library is loaded sets that much memory aside until the
 * process exits, whether this function is used or not.
 *
 *  - A problem whose flashbev_host_staging_bytes(p) (for NCHW tensors: without the optional scratch
 *    part) exceeds FLASHBEV_STATIC_STAGING_BYTES is refused with FLASHBEV_EXCEEDS_STATIC_STAGING
 *    before anything is enqueued.
 *  - The first call on each device looks up the device address of the array (once per device, with
 *    that device current) and remembers it; make that first call outside any stream capture.
 *  - The array is shared by every call and keeps whatever the previous call left in it.  Nothing in
 *    it has to start at zero (inputs are copied over it and the kernel writes every output
 *    element), but two calls whose GPU work overlaps -- different streams, or different host
 *    threads -- race on it: keep calls to this entry point in one stream order per device.
 *  - Calls no cudaMalloc, cudaFree or any other allocating routine.
 */
#define FLASHBEV_STATIC_STAGING_BYTES (32u * 1024u * 1024u)
flashbev_status flashbev_sampling_vt_host_static(const flashbev_vt_params *p, void *stream);

/*
 * Backward of the operator with respect to the features (the paper reports its cost in Tables 2
 * and 4 without printing an algorithm).  The forward is linear in the features, so the gradient is
 * its transpose: grad_features[b,n,y,x,c] = sum over the cells, heights and taps that read texel
 * (y,x) of camera n of  coeff * tap weight * grad_out[b,ix,iy,c],  coeff = 1 (SUM),
 * 1/max(1, valid samples of the cell) (MEAN_OVER_VALID), 1/max(1, cameras seeing that height bin)
 * (CAMERA_MEAN_Z_SUM).  Geometry fields have the meaning they have in flashbev_vt_params.
 *
 * Enqueues on `stream` a memset of `grad_features` to zero and one kernel that scatters with
 * fp32 vector atomics (texels are shared between cells, so the summation order -- and the last
 * bits of the result -- can differ from run to run).  Allocates nothing.  C must be a multiple of
 * 4 and both gradient pointers 16-byte aligned, else FLASHBEV_UNSUPPORTED / FLASHBEV_MISALIGNED.
 */
typedef struct flashbev_vt_backward_params {
    size_t struct_size;        /* sizeof(flashbev_vt_backward_params) of the caller's header */
    const float *grad_out;     /* device, [B][X][Y][C] float32; read only */
    const float *lidar2img;    /* device, [B][N][4][4] float32; read only */
    int32_t B, N, C;
    int32_t feat_h, feat_w;
    int32_t img_h, img_w;
    double x_min, x_max;
    double y_min, y_max;
    double z_min, z_max;
    int32_t X, Y, Z;
    int32_t reduce;            /* flashbev_reduce */
    float *grad_features;      /* device, [B][N][feat_h][feat_w][C] float32; overwritten */
    int32_t tune[4];           /* as in flashbev_vt_params; 0 = defaults */
    uint32_t *debug_error_word; /* as in flashbev_vt_params (bounds-checked build only); callers built against a
                                  header without this field are accepted */
} flashbev_vt_backward_params;

flashbev_status flashbev_sampling_vt_backward(const flashbev_vt_backward_params *p, void *stream);

/*
 * FlashSCA: spatial cross-attention with on-the-fly projection (Sec. 4.4, "Cross-framework
 * applicability"; the paper states the idea, the operator is BEVFormer's deformable-attention view
 * transformation).  Every BEV query q = (ix, iy) has Zref reference heights (bin centres of
 * [z_min, z_max]); reference k is projected into camera n with lidar2img exactly as in
 * flashbev_vt_params and is valid iff depth > 0.1 and the pixel is strictly inside the image.  A
 * camera is hit by the query iff one of its references is valid.  For every hit camera, head h,
 * level l and sampling point p (which uses reference k = p mod Zref, if valid) the value map is
 * sampled bilinearly (align_corners=False, zero padding) at
 *     px = u / img_w * W_l + offsets[..][0] - 1/2,   py = v / img_h * H_l + offsets[..][1] - 1/2
 * and out[b][q][h][:] = sum(weights * sample) / max(1, number of hit cameras).
 * References are projected in fp64, interpolation weights and accumulation are fp32.  One kernel on
 * `stream`; nothing allocated; no per-camera BEV-shaped intermediate is ever stored.
 */
typedef struct flashbev_sca_params {
    size_t struct_size;        /* sizeof(flashbev_sca_params) of the caller's header */
    const void *value;         /* device, [B][N][T][heads][head_dim], T = sum_l H_l*W_l (levels concatenated,
                                  each level row-major); value_dtype, 16-byte aligned */
    int32_t value_dtype;       /* FLASHBEV_F32 or FLASHBEV_BF16 (accumulation and output are float32 either way) */
    int32_t chunk_records;     /* tuning: tap records built per pass over a query (shared memory per warp); 0 = default */
    const int32_t *level_hw;   /* HOST, [L][2] = (H_l, W_l); read during the call only; L <= 8 */
    const float *lidar2img;    /* device, [B][N][4][4] float32 */
    const float *offsets;      /* device, [B][X*Y][heads][L][P][2] float32, in texels of level l */
    const float *weights;      /* device, [B][X*Y][heads][L][P] float32 (normally a softmax over L*P) */
    int32_t B, N, heads, head_dim; /* head_dim a multiple of 4 (float32) or 8 (bfloat16), <= 128; at most
                                      4 (float32) / 2 (bfloat16) passes of 32 lanes over the heads (a head
                                      takes head_dim * element size / 16 lanes): else FLASHBEV_UNSUPPORTED */
    int32_t L, P;
    int32_t img_h, img_w;
    double x_min, x_max;
    double y_min, y_max;
    double z_min, z_max;
    int32_t X, Y, Zref;        /* queries q = ix * Y + iy; Zref <= 32 */
    int32_t reserved2;
    float *out;                /* device, [B][X*Y][heads*head_dim] float32; every element written */
    int32_t *hits_out;         /* optional device [B][X*Y] int32: cameras that see the query */
} flashbev_sca_params;

flashbev_status flashbev_sca(const flashbev_sca_params *p, void *stream);

/* ---- multi-resolution gathering ------------------------------------------------------------
 * The paper names gathering from several feature resolutions as future work (Sec. 5) and gives no
 * formula; the operation built here is the plain sum over the levels of a feature pyramid,
 *
 *     out = sum_l  SamplingVT(features_l; feat_h_l x feat_w_l),
 *
 * every level sampled at the same voxel centres with the same matrices, validity rule, interpolation
 * and reduce mode as the single-level operator (for the two mean modes every level is normalised
 * by itself before the sum).  One launch per level on `stream`; level 0 overwrites `out`, the others
 * add to it, so nothing is allocated and no workspace is needed.
 *
 *   base      all arguments of the single-level call; its `features`, `feat_h`, `feat_w` are ignored.
 *             `out_dtype` must be FLASHBEV_F32 (partial sums are not rounded); `valid_count_out`, if
 *             given, receives the counts of level 0.
 *   levels    number of levels, 1..FLASHBEV_MAX_LEVELS
 *   features  HOST array of `levels` DEVICE pointers, each a tensor of the layout and dtype of `base`
 *             with C channels and its own map size; read during the call only
 *   feat_hw   HOST array [levels][2] = (feat_h_l, feat_w_l); read during the call only
 * Alignment and size rules are those of flashbev_sampling_vt, checked for every level before the
 * first launch.  flashbev_last_launch_count() reports `levels` afterwards. */
#define FLASHBEV_MAX_LEVELS 8
typedef struct flashbev_vt_multires_params {
    size_t struct_size;              /* sizeof(flashbev_vt_multires_params) of the caller's header */
    const flashbev_vt_params *base;  /* HOST */
    int32_t levels;
    int32_t reserved;
    const void *const *features;     /* HOST array of DEVICE pointers */
    const int32_t *feat_hw;          /* HOST, [levels][2] */
} flashbev_vt_multires_params;

flashbev_status flashbev_sampling_vt_multires(const flashbev_vt_multires_params *p, void *stream);

/* Number of kernels the last successful call of flashbev_sampling_vt[_host] on this thread
 * enqueued (always 1), and a short name of the kernel instance it chose (static storage). */
int flashbev_last_launch_count(void);
const char *flashbev_last_kernel_name(void);

const char *flashbev_status_string(int status); /* static storage, never NULL */
int flashbev_version(void);                     /* FLASHBEV_VERSION of the built library */

#ifdef __cplusplus
}
#endif
#endif /* FLASHBEV_H_ */
