"""ctypes front end of the fp64 CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Builds ``flashbev_oracle.c`` with gcc on first use and exposes ``sampling_vt``.
Only the tests, the smoke check and the bench's CPU-baseline leg may import this
module; it imports nothing from the CUDA package and the CUDA package imports
nothing from here.

The arithmetic lives entirely in the C file (paper Eq. 1 / Algorithm 2); this
module only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "flashbev_oracle.c")
_LIB = os.path.join(_HERE, "libflashbev_oracle.so")

REDUCE_SUM = 0
REDUCE_MEAN_OVER_VALID = 1
REDUCE_CAMERA_MEAN_Z_SUM = 2  # paper Eq. 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (plain gcc, OpenMP over cells, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-std=c99", "-O2", "-fopenmp", "-ffp-contract=off", "-Wall", "-Wextra",
               "-shared", "-fPIC", _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        d, i, p = ctypes.c_double, ctypes.c_int, ctypes.c_void_p
        lib.flashbev_oracle_sampling_vt.restype = i
        lib.flashbev_oracle_sampling_vt.argtypes = (
            [p, p] + [i] * 7 + [d] * 6 + [i] * 4 + [p] * 6 + [i])
        lib.flashbev_oracle_sampling_vt_backward.restype = i
        lib.flashbev_oracle_sampling_vt_backward.argtypes = [p, p] + [i] * 7 + [d] * 6 + [i] * 4 + [p, i]
        lib.flashbev_oracle_sca.restype = i
        lib.flashbev_oracle_sca.argtypes = [p] * 5 + [i] * 8 + [d] * 6 + [i] * 3 + [p] * 3 + [i]
        lib.flashbev_oracle_max_threads.restype = i
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().flashbev_oracle_max_threads())


@dataclass
class OracleResult:
    out: np.ndarray        # float64 [B, X, Y, C]
    count: np.ndarray      # int32   [B, X, Y]  valid samples per cell
    flagged: np.ndarray    # int32   [B, X, Y]  border samples per cell
    sumw: np.ndarray       # float64 [B, X, Y]  in-bounds bilinear weight mass
    interior: np.ndarray   # bool    [B, X, Y]  all taps of all valid samples in bounds
    nzbins: np.ndarray     # int32   [B, X, Y]  height bins seen by at least one camera


def sampling_vt(features, lidar2img, img_hw, bev_range, grid, reduce=REDUCE_SUM, threads=0) -> OracleResult:
    """Run the oracle.

    features : float32 array [B, N, Hf, Wf, C] (bf16 workloads: bf16-rounded values)
    lidar2img: float32 array [B, N, 4, 4]
    img_hw   : (Himg, Wimg)
    bev_range: (x_min, x_max, y_min, y_max, z_min, z_max) in metres
    grid     : (X, Y, Z)
    """
    f = np.ascontiguousarray(features, dtype=np.float32)
    m = np.ascontiguousarray(lidar2img, dtype=np.float32)
    if f.ndim != 5 or m.shape != (f.shape[0], f.shape[1], 4, 4):
        raise ValueError("features must be [B,N,Hf,Wf,C] and lidar2img [B,N,4,4]")
    B, N, Hf, Wf, C = f.shape
    X, Y, Z = (int(v) for v in grid)
    out = np.empty((B, X, Y, C), np.float64)
    count = np.empty((B, X, Y), np.int32)
    flagged = np.empty((B, X, Y), np.int32)
    sumw = np.empty((B, X, Y), np.float64)
    interior = np.empty((B, X, Y), np.uint8)
    nzbins = np.empty((B, X, Y), np.int32)
    rc = _load().flashbev_oracle_sampling_vt(
        f.ctypes.data, m.ctypes.data, B, N, C, Hf, Wf, int(img_hw[0]), int(img_hw[1]),
        *(float(v) for v in bev_range), X, Y, Z, int(reduce),
        out.ctypes.data, count.ctypes.data, flagged.ctypes.data, sumw.ctypes.data,
        interior.ctypes.data, nzbins.ctypes.data, int(threads))
    if rc != 0:
        raise ValueError(f"flashbev_oracle_sampling_vt rejected its arguments (status {rc})")
    return OracleResult(out, count, flagged, sumw, interior.astype(bool), nzbins)


def sampling_vt_backward(grad_out, lidar2img, feat_hw, img_hw, bev_range, grid, reduce=REDUCE_SUM, threads=0):
    """Gradient of the operator with respect to the features (fp64).

    grad_out : float64-convertible array [B, X, Y, C];  lidar2img: float32 [B, N, 4, 4]
    Returns float64 [B, N, Hf, Wf, C].
    """
    g = np.ascontiguousarray(grad_out, dtype=np.float64)
    m = np.ascontiguousarray(lidar2img, dtype=np.float32)
    X, Y, Z = (int(v) for v in grid)
    B, N = m.shape[:2]
    if g.ndim != 4 or g.shape[:3] != (B, X, Y) or m.shape != (B, N, 4, 4):
        raise ValueError("grad_out must be [B,X,Y,C] and lidar2img [B,N,4,4]")
    C = g.shape[3]
    Hf, Wf = (int(v) for v in feat_hw)
    out = np.empty((B, N, Hf, Wf, C), np.float64)
    rc = _load().flashbev_oracle_sampling_vt_backward(
        g.ctypes.data, m.ctypes.data, B, N, C, Hf, Wf, int(img_hw[0]), int(img_hw[1]),
        *(float(v) for v in bev_range), X, Y, Z, int(reduce), out.ctypes.data, int(threads))
    if rc != 0:
        raise ValueError(f"flashbev_oracle_sampling_vt_backward rejected its arguments (status {rc})")
    return out


def sca(value, level_hw, lidar2img, offsets, weights, img_hw, bev_range, grid, threads=0):
    """Spatial cross-attention with on-the-fly projection (fp64).

    value   : float32 [B, N, T, heads, Dh]   (T = sum of H_l * W_l, levels concatenated)
    level_hw: int [L, 2];  lidar2img: float32 [B, N, 4, 4]
    offsets : float32 [B, Q, heads, L, P, 2] (texels of the level);  weights: float32 [B, Q, heads, L, P]
    grid    : (X, Y, Zref), Q = X * Y.   Returns (out float64 [B, Q, heads*Dh], hits int32 [B, Q], flagged int32 [B, Q]).
    """
    v = np.ascontiguousarray(value, np.float32)
    lv = np.ascontiguousarray(level_hw, np.int32)
    m = np.ascontiguousarray(lidar2img, np.float32)
    of = np.ascontiguousarray(offsets, np.float32)
    wt = np.ascontiguousarray(weights, np.float32)
    B, N, T, heads, Dh = v.shape
    X, Y, Zref = (int(t) for t in grid)
    Q = X * Y
    L, P = wt.shape[3], wt.shape[4]
    if lv.shape != (L, 2) or int((lv[:, 0] * lv[:, 1]).sum()) != T or of.shape != (B, Q, heads, L, P, 2) \
            or wt.shape != (B, Q, heads, L, P) or m.shape != (B, N, 4, 4):
        raise ValueError("inconsistent shapes")
    out = np.empty((B, Q, heads * Dh), np.float64)
    hits = np.empty((B, Q), np.int32)
    flagged = np.empty((B, Q), np.int32)
    rc = _load().flashbev_oracle_sca(
        v.ctypes.data, lv.ctypes.data, m.ctypes.data, of.ctypes.data, wt.ctypes.data, B, N, heads, Dh, L, P,
        int(img_hw[0]), int(img_hw[1]), *(float(t) for t in bev_range), X, Y, Zref,
        out.ctypes.data, hits.ctypes.data, flagged.ctypes.data, int(threads))
    if rc != 0:
        raise ValueError(f"flashbev_oracle_sca rejected its arguments (status {rc})")
    return out, hits, flagged


def sampling_vt_multires(features, lidar2img, img_hw, bev_range, grid, reduce=REDUCE_SUM, threads=0) -> OracleResult:
    """Multi-resolution gathering, defined as the plain sum over the pyramid levels of the single-level
    operator (every level normalised by itself in the mean modes).  The paper only names the idea as
    future work; this is the definition the CUDA entry point documents.

    features: sequence of float32 arrays [B, N, Hf_l, Wf_l, C].  count/flagged/interior/nzbins are those of
    level 0, except `flagged`, which is the per-cell maximum over the levels.
    """
    res = [sampling_vt(f, lidar2img, img_hw, bev_range, grid, reduce, threads) for f in features]
    out = res[0].out.copy()
    flagged = res[0].flagged.copy()
    for r in res[1:]:
        out += r.out
        flagged = np.maximum(flagged, r.flagged)
    return OracleResult(out, res[0].count, flagged, res[0].sumw, res[0].interior, res[0].nzbins)
