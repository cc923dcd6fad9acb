"""Seeded synthetic workloads: camera rigs, feature maps and the benchmark shapes.

This module only GENERATES inputs (camera matrices, random feature maps, grid
descriptions).  It contains none of the operator's arithmetic -- no projection of
BEV cells, no validity test, no interpolation -- and is the one module that both
the CUDA path's tests/bench and the CPU oracle's tests draw their inputs from.

The shapes follow the paper's workloads (Sec. 4.1: multi-camera surround rig,
stride-8/stride-4 backbone feature maps, a BEV grid of 0.2-1 m cells, 4-64 height
bins); the values are standard-normal noise standing in for backbone features of a
driving dataset, which is not reproduced here in any form.

Frames: ego frame x forward, y left, z up (metres); camera frame x right, y down,
z forward.  ``lidar2img`` maps homogeneous ego coordinates to (u*d, v*d, d) in
full-resolution image pixels.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Tuple

import numpy as np

REDUCE_SUM = 0
REDUCE_MEAN_OVER_VALID = 1
REDUCE_CAMERA_MEAN_Z_SUM = 2

SEED_ROOT = (2607, 10071)


@dataclass(frozen=True)
class Workload:
    name: str
    index: int                 # seed stream
    B: int
    N: int
    C: int
    dtype: str                 # "f32" | "bf16"
    feat_hw: Tuple[int, int]   # (Hf, Wf)
    img_hw: Tuple[int, int]    # (Himg, Wimg)
    grid: Tuple[int, int, int]           # (X, Y, Z)
    bev_range: Tuple[float, float, float, float, float, float]  # x_min,x_max,y_min,y_max,z_min,z_max
    reduce: int
    fov_deg: float = 70.0
    cam_height: float = 1.6
    yaw_jitter_deg: float = 2.0
    general_pose: bool = False  # random pitch/roll/offset/focal (tests only)
    extra: dict = field(default_factory=dict, compare=False)

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def candidates(self) -> int:
        """B*N*X*Y*Z candidate samples."""
        X, Y, Z = self.grid
        return self.B * self.N * X * Y * Z

    @property
    def sample_channels(self) -> int:
        return self.candidates * self.C

    @property
    def feature_bytes(self) -> int:
        return self.B * self.N * self.feat_hw[0] * self.feat_hw[1] * self.C * self.elem_bytes

    @property
    def matrix_bytes(self) -> int:
        return self.B * self.N * 64

    @property
    def output_bytes(self) -> int:
        X, Y, _ = self.grid
        return self.B * X * Y * self.C * 4

    @property
    def unique_bytes(self) -> int:
        """Minimum bytes any implementation moves: features + matrices + fp32 output."""
        return self.feature_bytes + self.matrix_bytes + self.output_bytes


def _sym(r):  # symmetric x/y range
    return (-r, r, -r, r)


WORKLOADS = {
    "tiny": Workload("tiny", 0, 1, 6, 32, "f32", (16, 44), (128, 352), (50, 50, 4),
                     _sym(25.0) + (-3.0, 1.0), REDUCE_SUM),
    "representative": Workload("representative", 1, 1, 6, 80, "f32", (32, 88), (256, 704), (200, 200, 8),
                               _sym(50.0) + (-5.0, 3.0), REDUCE_SUM),
    "half_taller": Workload("half_taller", 2, 2, 6, 128, "bf16", (32, 88), (256, 704), (200, 200, 16),
                            _sym(50.0) + (-5.0, 3.0), REDUCE_MEAN_OVER_VALID),
    "long_range": Workload("long_range", 3, 1, 6, 128, "bf16", (64, 176), (256, 704), (400, 400, 16),
                           _sym(100.0) + (-5.0, 3.0), REDUCE_SUM),
    "high_res": Workload("high_res", 4, 1, 8, 64, "bf16", (64, 176), (256, 704), (512, 512, 64),
                         _sym(51.2) + (-5.0, 3.0), REDUCE_SUM, fov_deg=60.0),
    # the paper's own reference shape (Sec. 4.1), for context rows only
    "paper_shape": Workload("paper_shape", 5, 1, 6, 128, "f32", (56, 100), (448, 800), (200, 200, 8),
                            _sym(50.0) + (-5.0, 5.0), REDUCE_CAMERA_MEAN_Z_SUM),
}
CONFIG_ORDER = ["tiny", "representative", "half_taller", "long_range", "high_res"]


def get(name: str, **overrides) -> Workload:
    w = WORKLOADS[name]
    return replace(w, **overrides) if overrides else w


def rng_for(index: int, *more: int) -> np.random.Generator:
    return np.random.default_rng(list(SEED_ROOT) + [int(index)] + [int(m) for m in more])


def ring_rig(N, fov_deg, img_hw, yaw_jitter_rad, cam_height=1.6):
    """Surround rig: camera n yawed n*360/N degrees (+ jitter), zero pitch and roll,
    principal point at the image centre, square pixels.

    yaw_jitter_rad: array [B, N].  Returns float32 [B, N, 4, 4].
    """
    Himg, Wimg = img_hw
    jit = np.asarray(yaw_jitter_rad, np.float64)
    B = jit.shape[0]
    f = Wimg / (2.0 * np.tan(np.deg2rad(fov_deg) / 2.0))
    K = np.array([[f, 0.0, Wimg / 2.0], [0.0, f, Himg / 2.0], [0.0, 0.0, 1.0]])
    out = np.zeros((B, N, 4, 4), np.float64)
    t = np.array([0.0, 0.0, cam_height])
    for b in range(B):
        for n in range(N):
            yaw = np.deg2rad(n * 360.0 / N) + jit[b, n]
            right = np.array([np.sin(yaw), -np.cos(yaw), 0.0])
            down = np.array([0.0, 0.0, -1.0])
            fwd = np.array([np.cos(yaw), np.sin(yaw), 0.0])
            R = np.stack([right, down, fwd])
            KR = K @ R
            out[b, n, :3, :3] = KR
            out[b, n, :3, 3] = -KR @ t
            out[b, n, 3, 3] = 1.0
    return out.astype(np.float32)


def _rot(axis, a):
    c, s = np.cos(a), np.sin(a)
    if axis == 0:
        return np.array([[1, 0, 0], [0, c, -s], [0, s, c]])
    if axis == 1:
        return np.array([[c, 0, s], [0, 1, 0], [-s, 0, c]])
    return np.array([[c, -s, 0], [s, c, 0], [0, 0, 1]])


def general_rig(B, N, img_hw, rng, fov_deg=70.0):
    """Test rig with pitch/roll up to +-10 degrees, cameras on a 0.5-1.5 m ring at
    1.2-2.0 m height and a different focal length per camera, so that depth and
    both pixel coordinates vary with height.  Returns float32 [B, N, 4, 4]."""
    Himg, Wimg = img_hw
    out = np.zeros((B, N, 4, 4), np.float64)
    for b in range(B):
        for n in range(N):
            yaw = np.deg2rad(n * 360.0 / N) + rng.uniform(-0.3, 0.3)
            pitch, roll = np.deg2rad(rng.uniform(-10, 10, 2))
            f = Wimg / (2.0 * np.tan(np.deg2rad(fov_deg * rng.uniform(0.8, 1.2)) / 2.0))
            K = np.array([[f, 0.0, Wimg / 2.0 + rng.uniform(-8, 8)],
                          [0.0, f * rng.uniform(0.95, 1.05), Himg / 2.0 + rng.uniform(-8, 8)],
                          [0.0, 0.0, 1.0]])
            base = np.stack([np.array([np.sin(yaw), -np.cos(yaw), 0.0]),
                             np.array([0.0, 0.0, -1.0]),
                             np.array([np.cos(yaw), np.sin(yaw), 0.0])])
            R = _rot(2, roll) @ _rot(0, pitch) @ base
            r = rng.uniform(0.5, 1.5)
            t = np.array([r * np.cos(yaw), r * np.sin(yaw), rng.uniform(1.2, 2.0)])
            KR = K @ R
            out[b, n, :3, :3] = KR
            out[b, n, :3, 3] = -KR @ t
            out[b, n, 3, 3] = 1.0
    return out.astype(np.float32)


def round_to_bf16(x: np.ndarray):
    """Round float32 to bfloat16, ties to even.  Returns (values as float32, uint16 bit patterns)."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = ((u + bias) >> np.uint32(16)).astype(np.uint16)  # finite inputs only
    vals = (r.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return vals, r


@dataclass
class Inputs:
    workload: Workload
    features: np.ndarray        # float32 [B,N,Hf,Wf,C]; for bf16 workloads already bf16-rounded
    features_bf16: np.ndarray | None  # uint16 bit patterns (bf16 workloads) else None
    lidar2img: np.ndarray       # float32 [B,N,4,4]


def make_inputs(w: Workload, stream: int = 0) -> Inputs:
    """Draw one frame of inputs.  ``stream`` selects an independent frame with the same shape."""
    rng = rng_for(w.index, stream) if stream else rng_for(w.index)
    Hf, Wf = w.feat_hw
    if w.general_pose:
        mats = general_rig(w.B, w.N, w.img_hw, rng, w.fov_deg)
    else:
        jit = np.deg2rad(rng.uniform(-w.yaw_jitter_deg, w.yaw_jitter_deg, (w.B, w.N))) \
            if w.yaw_jitter_deg > 0 else np.zeros((w.B, w.N))
        mats = ring_rig(w.N, w.fov_deg, w.img_hw, jit, w.cam_height)
    feats = rng.standard_normal((w.B, w.N, Hf, Wf, w.C), dtype=np.float32)
    bits = None
    if w.dtype == "bf16":
        feats, bits = round_to_bf16(feats)
    return Inputs(w, feats, bits, mats)


def make_sca_inputs(P=8, X=200, Y=200, seed=0):
    """Synthetic inputs of the spatial-cross-attention operator at BEVFormer-base sizes (paper Sec. 4.4:
    N = 6, C = 256, 8 heads, 200 x 200 queries, Zref = 4, L = 4): six-camera ring rig for 928 x 1600 images,
    value maps of strides 8-64, standard-normal values and offsets (2 texels sigma), softmax attention weights."""
    rng = np.random.default_rng(list(SEED_ROOT) + [77, int(seed)])
    img_hw = (928, 1600)
    levels = ((116, 200), (58, 100), (29, 50), (15, 25))
    N, heads, Dh, Zref = 6, 8, 32, 4
    mats = ring_rig(N, 70.0, img_hw, np.deg2rad(rng.uniform(-2, 2, (1, N))))
    T = sum(h * w for h, w in levels)
    value = rng.standard_normal((1, N, T, heads, Dh), dtype=np.float32)
    Q = X * Y
    offsets = rng.standard_normal((1, Q, heads, len(levels), P, 2), dtype=np.float32) * np.float32(2.0)
    logits = rng.standard_normal((1, Q, heads, len(levels) * P), dtype=np.float32)
    e = np.exp(logits - logits.max(-1, keepdims=True))
    weights = (e / e.sum(-1, keepdims=True)).reshape(1, Q, heads, len(levels), P).astype(np.float32)
    return dict(value=value, level_hw=np.array(levels, np.int32), lidar2img=mats, offsets=offsets, weights=weights,
                img_hw=img_hw, bev_range=(-51.2, 51.2, -51.2, 51.2, -5.0, 3.0), grid=(X, Y, Zref))


def make_pyramid_inputs(w: Workload, levels: int = 3, stream: int = 0):
    """A feature pyramid for the multi-resolution variant: level l has the map of `w` halved l times
    (rounded up), the same cameras and channel count, independent standard-normal values.
    Returns (list of Inputs-like feature arrays [B,N,Hf_l,Wf_l,C] float32, list of bf16 bit arrays or None, lidar2img)."""
    base = make_inputs(w, stream)
    rng = rng_for(w.index, 900 + stream)
    feats, bits = [base.features], [base.features_bf16]
    Hf, Wf = w.feat_hw
    for _ in range(1, levels):
        Hf, Wf = (Hf + 1) // 2, (Wf + 1) // 2
        f = rng.standard_normal((w.B, w.N, Hf, Wf, w.C), dtype=np.float32)
        b = None
        if w.dtype == "bf16":
            f, b = round_to_bf16(f)
        feats.append(f)
        bits.append(b)
    return feats, bits, base.lidar2img
