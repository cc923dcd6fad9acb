"""Thin ctypes binding of the C ABI in include/flashbev.h.

Argument marshalling only: every step of the operator runs inside the CUDA
library.  PyTorch is used by callers for device memory and streams; this module
needs only integer addresses.  There is no CPU fallback: if the library has not
been built, or the call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libflashbev.so")

OK, INVALID_ARG, UNSUPPORTED, MISALIGNED, CUDA_ERROR, TOO_SMALL = range(6)
EXCEEDS_STATIC_STAGING = 6
STATIC_STAGING_BYTES = 32 * 1024 * 1024
F32, BF16 = 0, 1
NHWC, NCHW = 0, 1
REDUCE_SUM, REDUCE_MEAN_OVER_VALID, REDUCE_CAMERA_MEAN_Z_SUM = 0, 1, 2
KERNEL_AUTO, KERNEL_PER_OUTPUT, KERNEL_TILED = 0, 1, 2


class VtParams(ctypes.Structure):
    """Mirror of ``flashbev_vt_params``."""
    _fields_ = [
        ("struct_size", ctypes.c_size_t),
        ("features", ctypes.c_void_p),
        ("feat_dtype", ctypes.c_int32),
        ("layout", ctypes.c_int32),
        ("lidar2img", ctypes.c_void_p),
        ("B", ctypes.c_int32), ("N", ctypes.c_int32), ("C", ctypes.c_int32),
        ("feat_h", ctypes.c_int32), ("feat_w", ctypes.c_int32),
        ("img_h", ctypes.c_int32), ("img_w", ctypes.c_int32),
        ("x_min", ctypes.c_double), ("x_max", ctypes.c_double),
        ("y_min", ctypes.c_double), ("y_max", ctypes.c_double),
        ("z_min", ctypes.c_double), ("z_max", ctypes.c_double),
        ("X", ctypes.c_int32), ("Y", ctypes.c_int32), ("Z", ctypes.c_int32),
        ("reduce", ctypes.c_int32),
        ("out", ctypes.c_void_p),
        ("out_dtype", ctypes.c_int32),
        ("kernel", ctypes.c_int32),
        ("valid_count_out", ctypes.c_void_p),
        ("tune", ctypes.c_int32 * 4),
        ("debug_error_word", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t),
    ]


class VtBackwardParams(ctypes.Structure):
    """Mirror of ``flashbev_vt_backward_params``."""
    _fields_ = [
        ("struct_size", ctypes.c_size_t),
        ("grad_out", ctypes.c_void_p),
        ("lidar2img", ctypes.c_void_p),
        ("B", ctypes.c_int32), ("N", ctypes.c_int32), ("C", ctypes.c_int32),
        ("feat_h", ctypes.c_int32), ("feat_w", ctypes.c_int32),
        ("img_h", ctypes.c_int32), ("img_w", ctypes.c_int32),
        ("x_min", ctypes.c_double), ("x_max", ctypes.c_double),
        ("y_min", ctypes.c_double), ("y_max", ctypes.c_double),
        ("z_min", ctypes.c_double), ("z_max", ctypes.c_double),
        ("X", ctypes.c_int32), ("Y", ctypes.c_int32), ("Z", ctypes.c_int32),
        ("reduce", ctypes.c_int32),
        ("grad_features", ctypes.c_void_p),
        ("tune", ctypes.c_int32 * 4),
        ("debug_error_word", ctypes.c_void_p),
    ]


class ScaParams(ctypes.Structure):
    """Mirror of ``flashbev_sca_params``."""
    _fields_ = [
        ("struct_size", ctypes.c_size_t),
        ("value", ctypes.c_void_p),
        ("value_dtype", ctypes.c_int32), ("chunk_records", ctypes.c_int32),
        ("level_hw", ctypes.c_void_p),
        ("lidar2img", ctypes.c_void_p),
        ("offsets", ctypes.c_void_p),
        ("weights", ctypes.c_void_p),
        ("B", ctypes.c_int32), ("N", ctypes.c_int32), ("heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("L", ctypes.c_int32), ("P", ctypes.c_int32),
        ("img_h", ctypes.c_int32), ("img_w", ctypes.c_int32),
        ("x_min", ctypes.c_double), ("x_max", ctypes.c_double),
        ("y_min", ctypes.c_double), ("y_max", ctypes.c_double),
        ("z_min", ctypes.c_double), ("z_max", ctypes.c_double),
        ("X", ctypes.c_int32), ("Y", ctypes.c_int32), ("Zref", ctypes.c_int32), ("reserved2", ctypes.c_int32),
        ("out", ctypes.c_void_p),
        ("hits_out", ctypes.c_void_p),
    ]


class VtMultiresParams(ctypes.Structure):
    """ctypes mirror of ``flashbev_vt_multires_params``."""
    _fields_ = [
        ("struct_size", ctypes.c_size_t),
        ("base", ctypes.POINTER(VtParams)),
        ("levels", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("features", ctypes.POINTER(ctypes.c_void_p)),
        ("feat_hw", ctypes.POINTER(ctypes.c_int32)),
    ]


MAX_LEVELS = 8


class FlashBevError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {status_string(status)} (status {status})")
        self.status = status


_lib = None


def _declare(L: ctypes.CDLL) -> ctypes.CDLL:
    """Argument and result types of every entry point of a loaded libflashbev."""
    P = ctypes.POINTER(VtParams)
    L.flashbev_sampling_vt.restype = ctypes.c_int
    L.flashbev_sampling_vt.argtypes = [P, ctypes.c_void_p]
    L.flashbev_sampling_vt_host.restype = ctypes.c_int
    L.flashbev_sampling_vt_host.argtypes = [P, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
    L.flashbev_sampling_vt_host_static.restype = ctypes.c_int
    L.flashbev_sampling_vt_host_static.argtypes = [P, ctypes.c_void_p]
    L.flashbev_sampling_vt_backward.restype = ctypes.c_int
    L.flashbev_sampling_vt_backward.argtypes = [ctypes.POINTER(VtBackwardParams), ctypes.c_void_p]
    L.flashbev_sampling_vt_multires.restype = ctypes.c_int
    L.flashbev_sampling_vt_multires.argtypes = [ctypes.POINTER(VtMultiresParams), ctypes.c_void_p]
    L.flashbev_sca.restype = ctypes.c_int
    L.flashbev_sca.argtypes = [ctypes.POINTER(ScaParams), ctypes.c_void_p]
    L.flashbev_workspace_bytes.restype = ctypes.c_size_t
    L.flashbev_workspace_bytes.argtypes = [P]
    L.flashbev_host_staging_bytes.restype = ctypes.c_size_t
    L.flashbev_host_staging_bytes.argtypes = [P]
    L.flashbev_last_launch_count.restype = ctypes.c_int
    L.flashbev_last_kernel_name.restype = ctypes.c_char_p
    L.flashbev_status_string.restype = ctypes.c_char_p
    L.flashbev_status_string.argtypes = [ctypes.c_int]
    L.flashbev_version.restype = ctypes.c_int
    return L


def load_library(path: str) -> ctypes.CDLL:
    """Load another build of the library (e.g. the bounds-checked one) next to the default one."""
    if not os.path.exists(path):
        raise FileNotFoundError(f"{path} is missing: build it with paper_2607_10071_b200.build (there is no CPU fallback)")
    return _declare(ctypes.CDLL(path))


def lib() -> ctypes.CDLL:
    """Load libflashbev.so (built in-tree by ``paper_2607_10071_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2607_10071_b200.build` "
                "(there is no CPU fallback)")
        _lib = _declare(ctypes.CDLL(LIB_PATH))
    return _lib


def status_string(status: int) -> str:
    return lib().flashbev_status_string(int(status)).decode()


def version() -> int:
    return int(lib().flashbev_version())


def make_params(features_ptr, feat_dtype, lidar2img_ptr, B, N, C, feat_hw, img_hw, bev_range, grid,
                reduce, out_ptr, valid_count_ptr=None, kernel=KERNEL_AUTO, tune=(0, 0, 0, 0),
                layout=NHWC, out_dtype=F32, debug_error_word=None, workspace=None, workspace_bytes=0) -> VtParams:
    p = VtParams()
    p.struct_size = ctypes.sizeof(VtParams)
    p.features, p.feat_dtype, p.layout = features_ptr, feat_dtype, layout
    p.lidar2img = lidar2img_ptr
    p.B, p.N, p.C = B, N, C
    p.feat_h, p.feat_w = feat_hw
    p.img_h, p.img_w = img_hw
    p.x_min, p.x_max, p.y_min, p.y_max, p.z_min, p.z_max = (float(v) for v in bev_range)
    p.X, p.Y, p.Z = grid
    p.reduce = reduce
    p.out, p.out_dtype, p.kernel = out_ptr, out_dtype, kernel
    p.valid_count_out = valid_count_ptr
    p.debug_error_word = debug_error_word
    p.workspace, p.workspace_bytes = workspace, int(workspace_bytes)
    for i, t in enumerate(tune):
        p.tune[i] = int(t)
    return p


def flashbev_sampling_vt(params: VtParams, stream: int | None = None, check: bool = True, library=None) -> int:
    """Enqueue the fused operator on ``stream`` (a raw cudaStream_t value; None/0 = default stream).
    ``library``: another build loaded with ``load_library`` instead of the default one."""
    st = (library or lib()).flashbev_sampling_vt(ctypes.byref(params), ctypes.c_void_p(stream or 0))
    if check and st != OK:
        raise FlashBevError(st, "flashbev_sampling_vt")
    return st


def flashbev_sampling_vt_host(params: VtParams, d_staging: int, staging_bytes: int, stream: int | None = None,
                              check: bool = True) -> int:
    """Host-buffer variant: pointers in ``params`` are host addresses, ``d_staging`` a device buffer."""
    st = lib().flashbev_sampling_vt_host(ctypes.byref(params), ctypes.c_void_p(d_staging),
                                         ctypes.c_size_t(staging_bytes), ctypes.c_void_p(stream or 0))
    if check and st != OK:
        raise FlashBevError(st, "flashbev_sampling_vt_host")
    return st


def flashbev_sampling_vt_host_static(params: VtParams, stream: int | None = None, check: bool = True) -> int:
    """Host-buffer variant for callers that may not allocate device memory: pointers in ``params`` are
    host addresses and the staging area is the fixed STATIC_STAGING_BYTES array inside the library.
    Calls on one device must not overlap on the GPU (they share that array)."""
    st = lib().flashbev_sampling_vt_host_static(ctypes.byref(params), ctypes.c_void_p(stream or 0))
    if check and st != OK:
        raise FlashBevError(st, "flashbev_sampling_vt_host_static")
    return st


def flashbev_sampling_vt_multires(base: VtParams, feature_ptrs, feat_hws, stream: int | None = None,
                                  check: bool = True) -> int:
    """Sum of the operator over the levels of a feature pyramid: ``feature_ptrs`` are device pointers,
    ``feat_hws`` the (feat_h, feat_w) of every level; ``base`` carries everything else."""
    n = len(feature_ptrs)
    q = VtMultiresParams()
    q.struct_size = ctypes.sizeof(VtMultiresParams)
    q.base = ctypes.pointer(base)
    q.levels = n
    ptrs = (ctypes.c_void_p * max(n, 1))(*[int(v) for v in feature_ptrs])
    hw = (ctypes.c_int32 * max(2 * n, 2))(*[int(v) for pair in feat_hws for v in pair])
    q.features = ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p))
    q.feat_hw = ctypes.cast(hw, ctypes.POINTER(ctypes.c_int32))
    st = lib().flashbev_sampling_vt_multires(ctypes.byref(q), ctypes.c_void_p(stream or 0))
    if check and st != OK:
        raise FlashBevError(st, "flashbev_sampling_vt_multires")
    return st


def make_backward_params(grad_out_ptr, lidar2img_ptr, B, N, C, feat_hw, img_hw, bev_range, grid, reduce,
                         grad_features_ptr, tune=(0, 0, 0, 0), debug_error_word=None) -> VtBackwardParams:
    p = VtBackwardParams()
    p.struct_size = ctypes.sizeof(VtBackwardParams)
    p.grad_out, p.lidar2img, p.grad_features = grad_out_ptr, lidar2img_ptr, grad_features_ptr
    p.B, p.N, p.C = B, N, C
    p.feat_h, p.feat_w = feat_hw
    p.img_h, p.img_w = img_hw
    p.x_min, p.x_max, p.y_min, p.y_max, p.z_min, p.z_max = (float(v) for v in bev_range)
    p.X, p.Y, p.Z = grid
    p.reduce = reduce
    for i, t in enumerate(tune):
        p.tune[i] = int(t)
    p.debug_error_word = debug_error_word
    return p


def flashbev_sampling_vt_backward(params: VtBackwardParams, stream: int | None = None, check: bool = True,
                                  library=None) -> int:
    """Enqueue the gradient w.r.t. the features (memset + one scatter kernel) on ``stream``."""
    st = (library or lib()).flashbev_sampling_vt_backward(ctypes.byref(params), ctypes.c_void_p(stream or 0))
    if check and st != OK:
        raise FlashBevError(st, "flashbev_sampling_vt_backward")
    return st


def sampling_vt_backward(grad_out, lidar2img, feat_hw, img_hw, bev_range, grid, reduce=REDUCE_SUM,
                         grad_features=None, tune=(0, 0, 0, 0), stream=None):
    """grad_out: CUDA float32 [B,X,Y,C]; returns CUDA float32 [B,N,Hf,Wf,C] (marshalling only)."""
    import torch

    if not grad_out.is_cuda or grad_out.dtype != torch.float32 or not grad_out.is_contiguous():
        raise ValueError("grad_out must be a contiguous CUDA float32 tensor")
    B, X, Y, C = grad_out.shape
    N = lidar2img.shape[1]
    if grad_features is None:
        grad_features = torch.empty((B, N, feat_hw[0], feat_hw[1], C), dtype=torch.float32, device=grad_out.device)
    p = make_backward_params(grad_out.data_ptr(), lidar2img.data_ptr(), B, N, C, feat_hw, img_hw, bev_range,
                             (X, Y, grid[2]), reduce, grad_features.data_ptr(), tune)
    if stream is None:
        stream = torch.cuda.current_stream(grad_out.device).cuda_stream
    with torch.cuda.device(grad_out.device):
        flashbev_sampling_vt_backward(p, stream)
    return grad_features


def flashbev_sca(params: ScaParams, stream: int | None = None, check: bool = True) -> int:
    """Enqueue the fused spatial cross-attention on ``stream``."""
    st = lib().flashbev_sca(ctypes.byref(params), ctypes.c_void_p(stream or 0))
    if check and st != OK:
        raise FlashBevError(st, "flashbev_sca")
    return st


def sca(value, level_hw, lidar2img, offsets, weights, img_hw, bev_range, grid, out=None, hits=None, stream=None,
        chunk_records=0):
    """value: CUDA float32 or bfloat16 [B,N,T,heads,Dh]; offsets [B,Q,heads,L,P,2]; weights [B,Q,heads,L,P] (CUDA float32).
    level_hw: sequence of (H_l, W_l).  Returns CUDA float32 [B, Q, heads*Dh] (marshalling only)."""
    import numpy as np
    import torch

    for t in (lidar2img, offsets, weights):
        if not t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous():
            raise ValueError("sca needs contiguous CUDA float32 tensors")
    if not value.is_cuda or not value.is_contiguous() or value.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("value must be a contiguous CUDA float32 or bfloat16 tensor")
    B, N, T, heads, Dh = value.shape
    X, Y, Zref = grid
    L, P = weights.shape[3], weights.shape[4]
    lv = np.ascontiguousarray(level_hw, np.int32)
    if out is None:
        out = torch.empty((B, X * Y, heads * Dh), dtype=torch.float32, device=value.device)
    p = ScaParams()
    p.struct_size = ctypes.sizeof(ScaParams)
    p.value, p.chunk_records = value.data_ptr(), int(chunk_records)
    p.value_dtype = F32 if value.dtype == torch.float32 else BF16
    p.level_hw = lv.ctypes.data
    p.lidar2img, p.offsets, p.weights = lidar2img.data_ptr(), offsets.data_ptr(), weights.data_ptr()
    p.B, p.N, p.heads, p.head_dim, p.L, p.P = B, N, heads, Dh, L, P
    p.img_h, p.img_w = img_hw
    p.x_min, p.x_max, p.y_min, p.y_max, p.z_min, p.z_max = (float(v) for v in bev_range)
    p.X, p.Y, p.Zref = X, Y, Zref
    p.out = out.data_ptr()
    p.hits_out = None if hits is None else hits.data_ptr()
    if stream is None:
        stream = torch.cuda.current_stream(value.device).cuda_stream
    with torch.cuda.device(value.device):
        flashbev_sca(p, stream)
    return out


def flashbev_workspace_bytes(params: VtParams) -> int:
    return int(lib().flashbev_workspace_bytes(ctypes.byref(params)))


def flashbev_host_staging_bytes(params: VtParams) -> int:
    return int(lib().flashbev_host_staging_bytes(ctypes.byref(params)))


def flashbev_last_launch_count() -> int:
    return int(lib().flashbev_last_launch_count())


def flashbev_last_kernel_name() -> str:
    return lib().flashbev_last_kernel_name().decode()


# ---------------------------------------------------------------------------------------------
# convenience for torch callers (marshalling only)

def sampling_vt(features, lidar2img, img_hw, bev_range, grid, reduce=REDUCE_SUM, out=None,
                valid_count=None, kernel=KERNEL_AUTO, tune=(0, 0, 0, 0), stream=None, layout=NHWC,
                out_dtype=F32, workspace=True):
    """features: CUDA tensor [B,N,Hf,Wf,C] (NHWC) or [B,N,C,Hf,Wf] (NCHW), float32 or bfloat16,
    contiguous; lidar2img: CUDA float32 [B,N,4,4].  Returns the output tensor [B,X,Y,C] (NHWC) or
    [B,C,X,Y] (NCHW), float32 or bfloat16 per ``out_dtype`` (allocated by torch if ``out`` is None).
    ``workspace``: for NCHW tensors and for channel counts that are not whole 16-byte vectors, lend the call the
    scratch ``flashbev_workspace_bytes`` asks for (a torch allocation, or a uint8 CUDA tensor of the caller's);
    False: none, the generic kernel runs."""
    import torch

    if not features.is_cuda or not lidar2img.is_cuda:
        raise ValueError("sampling_vt needs CUDA tensors; there is no CPU path")
    if not features.is_contiguous() or not lidar2img.is_contiguous():
        raise ValueError("features and lidar2img must be contiguous")
    if features.dtype == torch.float32:
        dt = F32
    elif features.dtype == torch.bfloat16:
        dt = BF16
    else:
        raise ValueError("features must be float32 or bfloat16")
    if lidar2img.dtype != torch.float32:
        raise ValueError("lidar2img must be float32")
    if layout == NHWC:
        B, N, Hf, Wf, C = features.shape
    else:
        B, N, C, Hf, Wf = features.shape
    X, Y, Z = grid
    if out is None:
        out = torch.empty((B, X, Y, C) if layout == NHWC else (B, C, X, Y),
                          dtype=torch.float32 if out_dtype == F32 else torch.bfloat16, device=features.device)
    p = make_params(features.data_ptr(), dt, lidar2img.data_ptr(), B, N, C, (Hf, Wf), img_hw, bev_range,
                    (X, Y, Z), reduce, out.data_ptr(),
                    None if valid_count is None else valid_count.data_ptr(), kernel, tune, layout, out_dtype)
    if workspace is not False and workspace is not None:
        need = flashbev_workspace_bytes(p)
        if need:
            ws = workspace if workspace is not True else torch.empty(need, dtype=torch.uint8, device=features.device)
            p.workspace, p.workspace_bytes = ws.data_ptr(), ws.numel() * ws.element_size()
    if stream is None:
        stream = torch.cuda.current_stream(features.device).cuda_stream
    with torch.cuda.device(features.device):
        flashbev_sampling_vt(p, stream)
    return out


def sampling_vt_multires(features, lidar2img, img_hw, bev_range, grid, reduce=REDUCE_SUM, out=None,
                         valid_count=None, kernel=KERNEL_AUTO, tune=(0, 0, 0, 0), stream=None, layout=NHWC):
    """features: sequence of CUDA tensors, one per pyramid level, each [B,N,Hf_l,Wf_l,C] (NHWC) or
    [B,N,C,Hf_l,Wf_l] (NCHW) of one dtype.  Returns the float32 sum over the levels (marshalling only)."""
    import torch

    f0 = features[0]
    for f in features:
        if not f.is_cuda or not f.is_contiguous() or f.dtype != f0.dtype:
            raise ValueError("every level must be a contiguous CUDA tensor of the same dtype")
    if f0.dtype == torch.float32:
        dt = F32
    elif f0.dtype == torch.bfloat16:
        dt = BF16
    else:
        raise ValueError("features must be float32 or bfloat16")
    if not lidar2img.is_cuda or lidar2img.dtype != torch.float32 or not lidar2img.is_contiguous():
        raise ValueError("lidar2img must be a contiguous CUDA float32 tensor")
    if layout == NHWC:
        B, N, _, _, C = f0.shape
        hws = [(f.shape[2], f.shape[3]) for f in features]
    else:
        B, N, C, _, _ = f0.shape
        hws = [(f.shape[3], f.shape[4]) for f in features]
    X, Y, Z = grid
    if out is None:
        out = torch.empty((B, X, Y, C) if layout == NHWC else (B, C, X, Y), dtype=torch.float32, device=f0.device)
    base = make_params(f0.data_ptr(), dt, lidar2img.data_ptr(), B, N, C, hws[0], img_hw, bev_range, (X, Y, Z),
                       reduce, out.data_ptr(), None if valid_count is None else valid_count.data_ptr(),
                       kernel, tune, layout, F32)
    # planar tensors and ragged channel counts: lend the scratch of the largest level (the levels run one after another)
    need = 0
    for f, hw in zip(features, hws):
        base.features, base.feat_h, base.feat_w = f.data_ptr(), hw[0], hw[1]
        need = max(need, flashbev_workspace_bytes(base))
    base.features, base.feat_h, base.feat_w = f0.data_ptr(), hws[0][0], hws[0][1]
    if need:
        ws = torch.empty(need, dtype=torch.uint8, device=f0.device)
        base.workspace, base.workspace_bytes = ws.data_ptr(), need
    if stream is None:
        stream = torch.cuda.current_stream(f0.device).cuda_stream
    with torch.cuda.device(f0.device):
        flashbev_sampling_vt_multires(base, [f.data_ptr() for f in features], hws, stream)
    return out
