"""CPU pins of the spatial-cross-attention (FlashSCA) oracle against things other than itself."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from paper_2607_10071_b200 import workloads as wl


def make_case(seed, B=1, N=6, heads=2, Dh=3, levels=((6, 9), (3, 5)), P=4, grid=(5, 4, 2), general=True, rng_xy=6.0,
              bev_range=None, twin=True):
    rng = np.random.default_rng([77, seed])
    img_hw = (levels[0][0] * 8, levels[0][1] * 8)
    mats = wl.general_rig(B, N, img_hw, rng) if general else \
        wl.ring_rig(N, 70.0, img_hw, np.deg2rad(rng.uniform(-3, 3, (B, N))))
    if twin and N > 1:        # the last camera nearly duplicates the first: some queries are seen twice
        mats[:, -1] = mats[:, 0]
        mats[:, -1, 0, 3] += 5.0
    T = sum(h * w for h, w in levels)
    value = rng.standard_normal((B, N, T, heads, Dh)).astype(np.float32)
    Q = grid[0] * grid[1]
    L = len(levels)
    offsets = (rng.standard_normal((B, Q, heads, L, P, 2)) * 1.5).astype(np.float32)
    logits = rng.standard_normal((B, Q, heads, L * P))
    weights = (np.exp(logits) / np.exp(logits).sum(-1, keepdims=True)).reshape(B, Q, heads, L, P).astype(np.float32)
    bev_range = bev_range or (-rng_xy, rng_xy, -rng_xy, rng_xy, -2.0, 2.0)
    return dict(value=value, level_hw=np.array(levels, np.int32), lidar2img=mats, offsets=offsets, weights=weights,
                img_hw=img_hw, bev_range=bev_range, grid=grid)


def sca_tensorized(value, level_hw, lidar2img, offsets, weights, img_hw, bev_range, grid):
    """Per-camera, fully materialised evaluation with a library bilinear sampler (torch grid_sample, float64):
    reference points for all queries -> per-camera masks -> sampling locations [B,Q,heads,L,P,2] per camera ->
    sampled values -> attention-weighted sum -> mean over the cameras that see the query."""
    B, N, T, heads, Dh = value.shape
    X, Y, Zref = grid
    Q = X * Y
    Himg, Wimg = img_hw
    x0, x1, y0, y1, z0, z1 = bev_range
    xs = x0 + (np.arange(X) + 0.5) * ((x1 - x0) / X)
    ys = y0 + (np.arange(Y) + 0.5) * ((y1 - y0) / Y)
    zs = z0 + (np.arange(Zref) + 0.5) * ((z1 - z0) / Zref)
    gx, gy, gz = np.meshgrid(xs, ys, zs, indexing="ij")
    pts = np.stack([gx, gy, gz, np.ones_like(gx)], -1).reshape(Q, Zref, 4)
    cam = np.einsum("bnij,qkj->bnqki", lidar2img.astype(np.float64)[:, :, :3], pts)       # [B,N,Q,Zref,3]
    d = cam[..., 2]
    front = d > 0.1
    safe = np.where(front, d, 1.0)
    u, v = cam[..., 0] / safe, cam[..., 1] / safe
    valid = front & (u > 0) & (u < Wimg) & (v > 0) & (v < Himg)                           # [B,N,Q,Zref]
    hit = valid.any(-1)                                                                     # [B,N,Q]
    L, P = weights.shape[3], weights.shape[4]
    k_of_p = np.arange(P) % Zref
    out = np.zeros((B, Q, heads, Dh))
    lvl0 = 0
    for l, (Hl, Wl) in enumerate(level_hw):
        vl = torch.from_numpy(value[:, :, lvl0:lvl0 + Hl * Wl].astype(np.float64))        # [B,N,HlWl,heads,Dh]
        lvl0 += Hl * Wl
        img = vl.reshape(B, N, Hl, Wl, heads, Dh).permute(0, 1, 4, 5, 2, 3).reshape(B * N * heads, Dh, Hl, Wl)
        ru = (u / Wimg)[..., k_of_p]                                                        # [B,N,Q,P]
        rv = (v / Himg)[..., k_of_p]
        vm = valid[..., k_of_p]
        lx = ru[:, :, :, None, :] + offsets[:, None, :, :, l, :, 0] / Wl                   # [B,N,Q,heads,P]
        ly = rv[:, :, :, None, :] + offsets[:, None, :, :, l, :, 1] / Hl
        g = np.stack([2 * lx - 1, 2 * ly - 1], -1)
        g = np.where(vm[:, :, :, None, :, None], g, -7.0)                                  # invalid -> far outside
        g = torch.from_numpy(g).permute(0, 1, 3, 2, 4, 5).reshape(B * N * heads, Q, P, 2)
        s = F.grid_sample(img, g, mode="bilinear", padding_mode="zeros", align_corners=False)   # [BNh,Dh,Q,P]
        s = s.reshape(B, N, heads, Dh, Q, P).numpy()
        a = weights[:, :, :, l, :].astype(np.float64)                                      # [B,Q,heads,P]
        a = a.transpose(0, 2, 1, 3)[:, None] * vm[:, :, None, :, :]                        # [B,N,heads,Q,P]
        out += np.einsum("bnhdqp,bnhqp->bqhd", s, a)
    nh = hit.sum(1)                                                                         # [B,Q]
    return (out / np.maximum(1, nh)[..., None, None]).reshape(B, Q, heads * Dh), nh.astype(np.int32)


@pytest.mark.parametrize("general", [False, True])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_sca_matches_the_tensorized_evaluation_with_a_library_sampler(oracle, seed, general):
    c = make_case(seed, general=general)
    out, hits, flagged = oracle.sca(**c)
    ref, nh = sca_tensorized(**c)
    assert hits.sum() > 5 and (hits > 1).any()
    assert np.array_equal(hits, nh)
    assert np.allclose(out, ref, rtol=0, atol=1e-11)


def test_sca_single_point_by_hand(oracle):
    # one camera looking along +z of the ego frame (pinhole f=8, centre (6,4)); query centre (1, 0.5), one
    # reference height z=4 -> u = 8, v = 5 of a 12 x 8 image -> (ru, rv) = (2/3, 5/8); level 4 x 6:
    # px = 2/3*6 + 0.25 - 0.5 = 3.75, py = 5/8*4 + 0.5 - 0.5 = 2.5 -> taps (3,2) .125 (4,2) .375 (3,3) .125 (4,3) .375
    M = np.zeros((1, 1, 4, 4), np.float32)
    M[0, 0, 0] = [8, 0, 6, 0]
    M[0, 0, 1] = [0, 8, 4, 0]
    M[0, 0, 2] = [0, 0, 1, 0]
    y, x = np.meshgrid(np.arange(4), np.arange(6), indexing="ij")
    value = (10.0 * y + x).astype(np.float32).reshape(1, 1, 24, 1, 1)
    out, hits, _ = oracle.sca(value, np.array([[4, 6]]), M, np.array([0.25, 0.5], np.float32).reshape(1, 1, 1, 1, 1, 2),
                              np.array([0.5], np.float32).reshape(1, 1, 1, 1, 1), (8, 12), (0, 2, 0, 1, 3, 5), (1, 1, 1))
    expect = 0.5 * (.125 * 23 + .375 * 24 + .125 * 33 + .375 * 34)
    assert hits[0, 0] == 1 and out[0, 0, 0] == pytest.approx(expect, abs=1e-12)


def test_sca_reduces_to_sampling_vt_for_one_camera_zero_offsets(oracle):
    """N = 1, one level, P = Zref, zero offsets, unit weights: the attention is the plain sum over the heights of
    the bilinear samples -- the SUM-mode Sampling-VT of the same feature map (pinned separately)."""
    c = make_case(5, N=1, heads=1, Dh=4, levels=((6, 9),), P=3, grid=(6, 5, 3), general=False,
                  bev_range=(3.0, 15.0, -6.0, 6.0, -1.0, 3.0))
    c["offsets"][:] = 0
    c["weights"][:] = 1
    out, hits, _ = oracle.sca(**c)
    feats = c["value"].reshape(1, 1, 6, 9, 4)
    vt = oracle.sampling_vt(feats, c["lidar2img"], c["img_hw"], c["bev_range"], c["grid"], 0)
    assert vt.count.sum() > 10
    assert np.allclose(out.reshape(1, 6, 5, 4), vt.out, rtol=0, atol=1e-12)
    assert np.array_equal(hits.reshape(1, 6, 5), (vt.count > 0).astype(np.int32))


def test_sca_invariants(oracle):
    c = make_case(9, N=4, general=True)
    out, hits, _ = oracle.sca(**c)
    # camera permutation
    perm = [2, 0, 3, 1]
    c2 = dict(c, value=c["value"][:, perm], lidar2img=c["lidar2img"][:, perm])
    out2, hits2, _ = oracle.sca(**c2)
    assert np.array_equal(hits, hits2) and np.allclose(out, out2, rtol=1e-12, atol=1e-13)
    # linear in the value tensor
    rng = np.random.default_rng(1)
    v2 = (np.round(rng.standard_normal(c["value"].shape) * 16) / 16).astype(np.float32)
    v1 = (np.round(c["value"] * 16) / 16).astype(np.float32)
    o1 = oracle.sca(**dict(c, value=v1))[0]
    o2 = oracle.sca(**dict(c, value=v2))[0]
    o3 = oracle.sca(**dict(c, value=(2 * v1 + 0.5 * v2).astype(np.float32)))[0]
    assert np.allclose(o3, 2 * o1 + 0.5 * o2, rtol=0, atol=1e-12)
    # queries nobody sees give exactly zero; a constant map with weights summing to one per head gives the constant
    assert np.all(out[hits == 0] == 0.0)
    cc = make_case(11, N=1, general=False, rng_xy=3.0, levels=((16, 24),), P=2, grid=(3, 3, 2))
    cc["value"][:] = 2.5
    cc["offsets"][:] *= 0.1
    o, h, _ = oracle.sca(**cc)
    seen_fully = h == 1
    assert seen_fully.any()
