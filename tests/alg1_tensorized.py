"""Tensorised Sampling-VT (paper Algorithm 1) for tiny grids -- an independent pin of the oracle.

Written in the materialising order of Algorithm 1 (voxel grid -> projected
coordinates -> Features3D -> mask -> valid camera mean -> height sum) with numpy
array operations, and with the bilinear step delegated to a library routine:
``torch.nn.functional.grid_sample`` in float64 on the CPU
(mode="bilinear", padding_mode="zeros", align_corners=False).  It shares no code
with the C oracle (nested scalar loops in fused order) or with the CUDA path.
Memory is O(B N C X Y Z): tests only.
"""
import numpy as np
import torch
import torch.nn.functional as F


def sampling_vt_tensorized(features, lidar2img, img_hw, bev_range, grid, reduce):
    feats = np.asarray(features, np.float64)            # [B,N,Hf,Wf,C]
    P = np.asarray(lidar2img, np.float64)[:, :, :3, :]  # [B,N,3,4]
    B, N, Hf, Wf, C = feats.shape
    Himg, Wimg = img_hw
    X, Y, Z = grid
    x0, x1, y0, y1, z0, z1 = bev_range

    # step 1: voxel grid (B,X,Y,Z,3) of bin centres (homogeneous 4th coordinate appended)
    xs = x0 + (np.arange(X) + 0.5) * ((x1 - x0) / X)
    ys = y0 + (np.arange(Y) + 0.5) * ((y1 - y0) / Y)
    zs = z0 + (np.arange(Z) + 0.5) * ((z1 - z0) / Z)
    vox = np.stack(list(np.meshgrid(xs, ys, zs, indexing="ij")) + [np.ones((X, Y, Z))], axis=-1)

    # step 2: projected coordinates (B,N,X,Y,Z,3)
    proj = np.einsum("bnij,xyzj->bnxyzi", P, vox)
    depth = proj[..., 2]
    front = depth > 0.1
    safe = np.where(front, depth, 1.0)
    u = proj[..., 0] / safe
    v = proj[..., 1] / safe

    # step 4 (mask from the coordinates): inside the image with positive depth
    with np.errstate(invalid="ignore"):
        mask = front & (u > 0.0) & (u < Wimg) & (v > 0.0) & (v < Himg)

    # step 3: Features3D (B,N,C,X,Y,Z) by library bilinear sampling on the normalised grid
    gx = np.where(mask, 2.0 * u / Wimg - 1.0, -5.0)
    gy = np.where(mask, 2.0 * v / Himg - 1.0, -5.0)
    g = torch.from_numpy(np.stack([gx, gy], axis=-1).reshape(B * N, X * Y, Z, 2))
    img = torch.from_numpy(feats.reshape(B * N, Hf, Wf, C)).permute(0, 3, 1, 2).contiguous()
    f3d = F.grid_sample(img, g, mode="bilinear", padding_mode="zeros", align_corners=False)
    f3d = f3d.numpy().reshape(B, N, C, X, Y, Z)
    f3d = f3d * mask[:, :, None]

    num = f3d.sum(axis=1)                 # (B,C,X,Y,Z)
    den = mask.sum(axis=1)                # (B,X,Y,Z)
    count = den.sum(axis=-1)              # (B,X,Y)
    if reduce == 2:      # step 5 + 6: valid camera mean per z, then height sum (Eq. 1)
        out = (num / np.maximum(1, den)[:, None]).sum(axis=-1)
    elif reduce == 0:
        out = num.sum(axis=-1)
    else:
        out = num.sum(axis=-1) / np.maximum(1, count)[:, None]
    return np.ascontiguousarray(out.transpose(0, 2, 3, 1)), count.astype(np.int32), mask
