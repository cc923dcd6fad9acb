"""Tensorised Sampling-VT on the GPU with stock PyTorch ops (paper Algorithm 1) -- a COMPARISON baseline.

This is the execution the paper argues against: it materialises the voxel grid, the projected
coordinates, the ``B x N x C x X x Y x Z`` sampled tensor, the mask and the per-height means in HBM
(Sec. 3.2.1).  It exists to put the fused kernel's latency and memory next to the tensorised ones on the
same B200 (Sec. 4.3 reports ~5x / ~37x on an RTX A6000) and as a second, GPU-side cross-check of the
fused kernel.  It is not part of the product path and is never used as a fallback.
"""
from __future__ import annotations

import torch
import torch.nn.functional as F


def sampling_vt_tensorized(features, lidar2img, img_hw, bev_range, grid, reduce=0):
    """features: CUDA float32 [B,N,Hf,Wf,C]; lidar2img: CUDA float32 [B,N,4,4].  Returns float32 [B,X,Y,C].

    Geometry is done in float64 (as the fused kernel does); sampling, masking and the reductions in float32.
    """
    B, N, Hf, Wf, C = features.shape
    Himg, Wimg = img_hw
    X, Y, Z = grid
    x0, x1, y0, y1, z0, z1 = bev_range
    dev = features.device
    f64 = torch.float64
    # step 1: voxel grid (X,Y,Z,4), bin centres
    xs = x0 + (torch.arange(X, device=dev, dtype=f64) + 0.5) * ((x1 - x0) / X)
    ys = y0 + (torch.arange(Y, device=dev, dtype=f64) + 0.5) * ((y1 - y0) / Y)
    zs = z0 + (torch.arange(Z, device=dev, dtype=f64) + 0.5) * ((z1 - z0) / Z)
    gx, gy, gz = torch.meshgrid(xs, ys, zs, indexing="ij")
    vox = torch.stack([gx, gy, gz, torch.ones_like(gx)], dim=-1)
    # step 2: projected coordinates (B,N,X,Y,Z,3)
    proj = torch.einsum("bnij,xyzj->bnxyzi", lidar2img[:, :, :3, :].to(f64), vox)
    depth = proj[..., 2]
    front = depth > 0.1
    safe = torch.where(front, depth, torch.ones_like(depth))
    u, v = proj[..., 0] / safe, proj[..., 1] / safe
    # step 4 (mask from the coordinates)
    mask = front & (u > 0) & (u < Wimg) & (v > 0) & (v < Himg)
    # step 3: Features3D (B,N,C,X,Y,Z)
    gxn = torch.where(mask, 2.0 * u / Wimg - 1.0, torch.full_like(u, -5.0)).to(torch.float32)
    gyn = torch.where(mask, 2.0 * v / Himg - 1.0, torch.full_like(v, -5.0)).to(torch.float32)
    g = torch.stack([gxn, gyn], dim=-1).reshape(B * N, X * Y, Z, 2)
    img = features.reshape(B * N, Hf, Wf, C).permute(0, 3, 1, 2)
    f3d = F.grid_sample(img, g, mode="bilinear", padding_mode="zeros", align_corners=False)
    f3d = f3d.reshape(B, N, C, X, Y, Z) * mask[:, :, None].to(f3d.dtype)
    num = f3d.sum(dim=1)                      # (B,C,X,Y,Z)
    den = mask.sum(dim=1)                     # (B,X,Y,Z)
    if reduce == 2:                           # step 5 + 6 (Eq. 1)
        out = (num / den.clamp(min=1)[:, None]).sum(dim=-1)
    elif reduce == 0:
        out = num.sum(dim=-1)
    else:
        out = num.sum(dim=-1) / den.sum(dim=-1).clamp(min=1)[:, None]
    return out.permute(0, 2, 3, 1).contiguous()
