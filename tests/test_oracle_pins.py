"""CPU-only pins of the fp64 oracle against things other than itself.

Each test names the fact it pins.  The paper prints no worked input->output
example, so value-level pins are: hand-computed single samples, closed forms on
orthographic rigs, the tensorised order (Algorithm 1) with a library bilinear
sampler, and invariants of Eq. 1.
"""
import os

import numpy as np
import pytest

from paper_2607_10071_b200 import workloads as wl
from tests import alg1_tensorized

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SUM, MEAN, EQ1 = 0, 1, 2


def ortho(su, tu, sv, tv, gu=0.0, gv=0.0, depth=1.0):
    """d == depth, u = (su*x + gu*z + tu), v = (sv*y + gv*z + tv)  (image px)."""
    M = np.zeros((4, 4), np.float32)
    M[0] = [su * depth, 0, gu * depth, tu * depth]
    M[1] = [0, sv * depth, gv * depth, tv * depth]
    M[2] = [0, 0, 0, depth]
    M[3, 3] = 1
    return M


def pinhole(f, cx, cy):
    """Ego axes == camera axes (x right, y down, z forward)."""
    M = np.zeros((4, 4), np.float32)
    M[0] = [f, 0, cx, 0]
    M[1] = [0, f, cy, 0]
    M[2] = [0, 0, 1, 0]
    M[3, 3] = 1
    return M


def ramp(Hf, Wf):
    """F[y, x, 0] = 10 y + x ; F[y, x, 1] = 1."""
    y, x = np.meshgrid(np.arange(Hf), np.arange(Wf), indexing="ij")
    return np.stack([10.0 * y + x, np.ones_like(x, float)], -1).astype(np.float32)[None, None]


# ---------------------------------------------------------------- hand-computed samples

def test_single_sample_orthographic_by_hand(oracle):
    # image 8x12, map 4x6 (scale 1/2).  u = 5.5 -> fx = 2.25 ; v = 4 -> fy = 1.5
    # taps (x,y): (2,1) .375  (3,1) .125  (2,2) .375  (3,2) .125 ; F = 10y + x
    # => .375*12 + .125*13 + .375*22 + .125*23 = 17.25
    M = ortho(1.0, 5.5, 1.0, 4.0)[None, None]
    r = oracle.sampling_vt(ramp(4, 6), M, (8, 12), (-1, 1, -1, 1, 0, 2), (1, 1, 1), SUM)
    assert r.out[0, 0, 0, 0] == pytest.approx(17.25, abs=1e-12)
    assert r.out[0, 0, 0, 1] == pytest.approx(1.0, abs=1e-12)
    assert r.count[0, 0, 0] == 1 and r.interior[0, 0, 0] and r.flagged[0, 0, 0] == 0


def test_single_sample_perspective_by_hand(oracle):
    # voxel centre (1, 0.5, 4) -> u = 8*1/4 + 6 = 8, v = 8*0.5/4 + 4 = 5
    # fx = 8/2 - .5 = 3.5, fy = 5/2 - .5 = 2 -> taps (3,2) .5 and (4,2) .5 -> 23.5
    M = pinhole(8.0, 6.0, 4.0)[None, None]
    r = oracle.sampling_vt(ramp(4, 6), M, (8, 12), (0, 2, 0, 1, 3, 5), (1, 1, 1), EQ1)
    assert r.out[0, 0, 0, 0] == pytest.approx(23.5, abs=1e-12)
    assert r.count[0, 0, 0] == 1


def test_axes_are_not_transposed(oracle):
    # 2x3 cells: only x moves u, only y moves v.  cell (ix,iy) centre = (ix+.5, iy+.5)
    # u = 2x + 1 -> fx = x ; v = 2y + 1 -> fy = y  => out = 10*(iy+.5) + (ix+.5)
    M = ortho(2.0, 1.0, 2.0, 1.0)[None, None]
    r = oracle.sampling_vt(ramp(4, 6), M, (8, 12), (0, 2, 0, 3, 0, 1), (2, 3, 1), SUM)
    for ix in range(2):
        for iy in range(3):
            assert r.out[0, ix, iy, 0] == pytest.approx(10 * (iy + .5) + (ix + .5), abs=1e-12)


def test_zero_padding_rim_by_hand(oracle):
    # u = 0.5 -> fx = -0.25 : x0 = -1, tx = .75 -> only texel x=0 with weight .75
    # v = 4   -> fy = 1.5   : rows 1, 2 with .5 each.   F = 10y + x -> .75*(.5*10 + .5*20) = 11.25
    M = ortho(1.0, 0.5, 1.0, 4.0)[None, None]
    r = oracle.sampling_vt(ramp(4, 6), M, (8, 12), (-1, 1, -1, 1, 0, 2), (1, 1, 1), SUM)
    assert r.out[0, 0, 0, 0] == pytest.approx(11.25, abs=1e-12)
    assert r.out[0, 0, 0, 1] == pytest.approx(0.75, abs=1e-12)      # weight mass
    assert r.sumw[0, 0, 0] == pytest.approx(0.75, abs=1e-12)
    assert r.count[0, 0, 0] == 1 and not r.interior[0, 0, 0]      # the sample still counts
    # bottom-right rim: u = 11.9 -> fx = 5.45 (x0 = 5, x=6 is outside), v = 7.8 -> fy = 3.4
    M = ortho(1.0, 11.9, 1.0, 7.8)[None, None]
    r = oracle.sampling_vt(ramp(4, 6), M, (8, 12), (-1, 1, -1, 1, 0, 2), (1, 1, 1), MEAN)
    assert r.out[0, 0, 0, 1] == pytest.approx(0.55 * 0.6, abs=1e-6)
    assert r.out[0, 0, 0, 0] == pytest.approx(0.55 * 0.6 * 35.0, abs=1e-4)


@pytest.mark.parametrize("u,v,d,valid", [
    (0.02, 4.0, 1.0, True), (-0.02, 4.0, 1.0, False),     # left border u = 0
    (11.98, 4.0, 1.0, True), (12.02, 4.0, 1.0, False),    # right border u = Wimg
    (6.0, 0.02, 1.0, True), (6.0, -0.02, 1.0, False),     # top
    (6.0, 7.98, 1.0, True), (6.0, 8.02, 1.0, False),      # bottom
    (6.0, 4.0, 0.2, True), (6.0, 4.0, 0.05, False),       # depth plane 0.1 m
    (6.0, 4.0, -1.0, False),                              # behind the camera
])
def test_validity_rules(oracle, u, v, d, valid):
    M = ortho(0.0, u, 0.0, v, depth=d)[None, None]
    r = oracle.sampling_vt(ramp(4, 6), M, (8, 12), (-1, 1, -1, 1, 0, 2), (1, 1, 1), SUM)
    assert r.count[0, 0, 0] == int(valid)
    if not valid:
        assert np.all(r.out == 0.0)


def test_border_flags(oracle):
    def run(u, v, d=1.0):
        M = ortho(0.0, u, 0.0, v, depth=d)[None, None]
        return oracle.sampling_vt(ramp(4, 6), M, (8, 12), (-1, 1, -1, 1, 0, 2), (1, 1, 1), SUM)
    assert run(0.001, 4.0).flagged[0, 0, 0] == 1          # 5e-4 feature px inside the left border
    assert run(-0.001, 4.0).flagged[0, 0, 0] == 1         # 5e-4 outside
    assert run(0.01, 4.0).flagged[0, 0, 0] == 0           # 5e-3 inside
    assert run(6.0, 4.0, 0.1004).flagged[0, 0, 0] == 1    # grazing the depth plane, inside the image
    assert run(6.0, 4.0, 0.0996).flagged[0, 0, 0] == 1
    assert run(600.0, 4.0, 0.1004).flagged[0, 0, 0] == 0  # grazing it, but far outside the image
    assert run(0.001, -50.0).flagged[0, 0, 0] == 0        # grazing u = 0, but far outside in v


def test_non_finite_matrix_is_invalid_not_fatal(oracle):
    M = ortho(1.0, 5.5, 1.0, 4.0)[None, None].copy()
    for bad in (np.nan, np.inf, -np.inf):
        for idx in ((0, 3), (2, 3), (1, 1)):
            Mb = M.copy()
            Mb[0, 0][idx] = bad
            r = oracle.sampling_vt(ramp(4, 6), Mb, (8, 12), (-1, 1, -1, 1, 0, 2), (1, 1, 1), SUM)
            assert np.all(np.isfinite(r.out))


# ---------------------------------------------------------------- the paper's grid convention

def test_bin_convention_matches_paper_grid():
    """Sec. 4.1 fixes ranges, resolutions and bin counts together; only bin centres fit."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "paper_grid_convention.txt"))
            if l.strip() and not l.startswith("#")]
    for axis, lo, hi, res, n in rows:
        lo, hi, res, n = float(lo), float(hi), float(res), int(n)
        assert (hi - lo) / n == pytest.approx(res)          # bins: n cells of size res
        assert (hi - lo) / (n - 1) != pytest.approx(res)    # an endpoint-inclusive linspace would not


def test_voxel_centres_are_bin_centres(oracle):
    """Read the voxel coordinates back through an orthographic camera and an affine map."""
    rows = {l.split()[0]: l.split()[1:] for l in open(os.path.join(GOLDEN, "paper_grid_convention.txt"))
            if l.strip() and not l.startswith("#")}
    lo, hi, res, n = float(rows["x"][0]), float(rows["x"][1]), float(rows["x"][2]), int(rows["x"][3])
    zlo, zhi, zres, nz = float(rows["z"][0]), float(rows["z"][1]), float(rows["z"][2]), int(rows["z"][3])
    Wf, Hf = 256, 4
    # fx = x + 100, fy = (z + 5)/4  -> F = x-texel index reproduces the coordinate
    M = np.zeros((1, 1, 4, 4), np.float32)
    M[0, 0, 0] = [1, 0, 0, 100.5]
    M[0, 0, 1] = [0, 0, 0.25, 1.25 + 0.5]
    M[0, 0, 2] = [0, 0, 0, 1]
    y, x = np.meshgrid(np.arange(Hf), np.arange(Wf), indexing="ij")
    feats = np.stack([x, y], -1).astype(np.float32)[None, None]
    r = oracle.sampling_vt(feats, M, (Hf, Wf), (lo, hi, -1, 1, zlo, zhi), (n, 1, nz), MEAN)
    xs = r.out[0, :, 0, 0] - 100.0
    assert xs[0] == pytest.approx(lo + res / 2, abs=1e-9)       # -49.75, not -50
    assert xs[-1] == pytest.approx(hi - res / 2, abs=1e-9)
    assert np.allclose(np.diff(xs), res, atol=1e-9)
    # mean over the Z bins of fy = (z+5)/4 is the mean of the bin centres
    zc = zlo + (np.arange(nz) + 0.5) * zres
    assert r.out[0, 0, 0, 1] == pytest.approx(np.mean((zc + 5) / 4), abs=1e-9)
    assert np.all(r.count == nz)


# ---------------------------------------------------------------- closed forms

def _ortho_rig(N):
    # camera n: fx = 1 + 0.5 x + 0.1 n + 0.25 z ; fy = 0.5 + 0.25 y + 0.05 n  (all interior for the grid below)
    Ms = []
    for n in range(N):
        su, tu, gu = 2 * 0.5, 2 * (1 + 0.1 * n + 0.5), 2 * 0.25
        sv, tv = 2 * 0.25, 2 * (0.5 + 0.05 * n + 0.5)
        Ms.append(ortho(su, tu, sv, tv, gu=gu, depth=1.0 + n))
    return np.stack(Ms)[None]


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
def test_constant_map_closed_form(oracle, reduce):
    N, Z, X, Y, C = 3, 4, 6, 5, 3
    kappa = np.array([2.0, -1.5, 0.25])
    feats = np.broadcast_to(kappa.astype(np.float32), (1, N, 8, 16, C)).copy()
    r = oracle.sampling_vt(feats, _ortho_rig(N), (16, 32), (0, 6, 0, 5, 0, 4), (X, Y, Z), reduce)
    assert np.all(r.count == N * Z) and np.all(r.interior)
    expect = {SUM: kappa * N * Z, MEAN: kappa, EQ1: kappa * Z}[reduce]
    assert np.allclose(r.out, expect, rtol=0, atol=1e-12)


def test_affine_map_closed_form(oracle):
    """Bilinear interpolation reproduces affine functions: out = sum of projected coordinates."""
    N, Z, X, Y = 3, 4, 6, 5
    a, b, g = np.array([1.0, 0.0, -2.0]), np.array([0.0, 1.0, 0.5]), np.array([0.0, 0.0, 3.0])
    y, x = np.meshgrid(np.arange(8), np.arange(16), indexing="ij")
    F1 = (a * x[..., None] + b * y[..., None] + g).astype(np.float32)
    feats = np.broadcast_to(F1, (1, N, 8, 16, 3)).copy()
    r = oracle.sampling_vt(feats, _ortho_rig(N), (16, 32), (0, 6, 0, 5, 0, 4), (X, Y, Z), SUM)
    xs, ys, zs = np.arange(X) + 0.5, np.arange(Y) + 0.5, np.arange(Z) + 0.5
    n = np.arange(N)
    fx = (1 + 0.5 * xs[:, None, None] + 0.1 * n[None, None, :] + 0.25 * zs[None, :, None]).sum((1, 2))  # [X]
    fy = (0.5 + 0.25 * ys[:, None] + 0.05 * n[None, :]).sum(1) * Z                                       # [Y]
    expect = a * fx[:, None, None] + b * fy[None, :, None] + g * (N * Z)
    assert np.allclose(r.out[0], expect, rtol=0, atol=1e-5)   # matrices are float32: coordinates carry 1e-7


# ---------------------------------------------------------------- Algorithm 1 order with a library sampler

def _tiny_case(seed, general, N=3, C=3, Hf=5, Wf=7, grid=(6, 5, 3)):
    w = wl.Workload("t", 100 + seed, 2, N, C, "f32", (Hf, Wf), (Hf * 8, Wf * 8), grid,
                    (-6.0, 6.0, -6.0, 6.0, -2.0, 2.5), 0, general_pose=general, yaw_jitter_deg=5.0)
    return wl.make_inputs(w)


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
@pytest.mark.parametrize("general", [False, True])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_matches_tensorized_order_with_library_bilinear(oracle, reduce, general, seed):
    inp = _tiny_case(seed, general)
    w = inp.workload
    r = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, reduce)
    ref, cnt, _ = alg1_tensorized.sampling_vt_tensorized(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, reduce)
    assert r.count.sum() > 20          # the case is not vacuous
    assert np.array_equal(r.count, cnt)
    assert np.allclose(r.out, ref, rtol=0, atol=1e-11)


def test_tiny_workload_counts_match_tensorized_geometry(oracle):
    """Validity totals of the benchmark's smallest rig from independent array code."""
    w = wl.get("tiny", C=2)
    inp = wl.make_inputs(w)
    r = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, SUM)
    ref, cnt, _ = alg1_tensorized.sampling_vt_tensorized(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, SUM)
    assert np.array_equal(r.count, cnt)
    assert 8000 < r.count.sum() < 11000      # about 16 % of 60 000 candidates on this rig
    assert np.allclose(r.out, ref, rtol=0, atol=1e-11)


def zero_jitter_totals():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "zero_jitter_valid_totals.txt")) if l.strip() and not l.startswith("#")]
    return {r[0]: (int(r[1]), int(r[2])) for r in rows}


@pytest.mark.parametrize("name", ["tiny", "representative", "half_taller"])
def test_valid_sample_totals_of_the_benchmark_rigs_without_jitter(oracle, name):
    """Geometry + validity at full grid size: the totals of an independent enumeration (a handful of samples
    within 1e-3 px of a border may fall either way; the oracle flags those)."""
    cand, valid = zero_jitter_totals()[name]
    w = wl.get(name, yaw_jitter_deg=0.0, C=4 if wl.get(name).dtype == "f32" else 8)
    inp = wl.make_inputs(w)
    r = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, SUM)
    assert w.candidates == cand
    assert abs(int(r.count.sum()) - valid) <= int(r.flagged.sum())
    assert r.flagged.sum() <= 1e-4 * cand


def test_height_bins_seen_by_hand(oracle):
    """nzbins counts the height bins seen by at least one camera; count adds the cameras up.
    One cell, three bins z = 0.5, 1.5, 2.5, image 8 x 12, map 4 x 6, orthographic cameras (depth 1):
      A: u = 20 z - 15 = -5, 15, 35 -> always outside 0 < u < 12: sees no bin;
      B: u = 6, v = 2 z + 1 = 2, 4, 6 -> sees all three;
      C: u = 6, v = 4 z - 1 = 1, 5, 9 -> sees bins 0 and 1 (9 > 8).
    So count = 5 and nzbins = 3."""
    A = ortho(0.0, -15.0, 0.0, 1.0, gu=20.0, gv=2.0)
    Bm = ortho(0.0, 6.0, 0.0, 1.0, gv=2.0)
    Cm = ortho(0.0, 6.0, 0.0, -1.0, gv=4.0)
    M = np.stack([A, Bm, Cm])[None]
    F = np.ones((1, 3, 4, 6, 1), np.float32)
    r = oracle.sampling_vt(F, M, (8, 12), (0, 1, 0, 1, 0, 3), (1, 1, 3), SUM)
    assert r.count[0, 0, 0] == 5 and r.nzbins[0, 0, 0] == 3
    # constant map, all samples interior: SUM = count, Eq. 1 = bins seen, MEAN = 1
    assert r.out[0, 0, 0, 0] == pytest.approx(5.0, abs=1e-12)
    e = oracle.sampling_vt(F, M, (8, 12), (0, 1, 0, 1, 0, 3), (1, 1, 3), EQ1)
    assert e.out[0, 0, 0, 0] == pytest.approx(3.0, abs=1e-12)
    # drop camera B: bins 0 and 1 are seen once, bin 2 never
    r2 = oracle.sampling_vt(F[:, [0, 2]], M[:, [0, 2]], (8, 12), (0, 1, 0, 1, 0, 3), (1, 1, 3), SUM)
    assert r2.count[0, 0, 0] == 2 and r2.nzbins[0, 0, 0] == 2


# ---------------------------------------------------------------- invariants of Eq. 1

@pytest.fixture(scope="module")
def case():
    return _tiny_case(7, True, N=6, C=5, Hf=6, Wf=9, grid=(7, 6, 4))


def _run(oracle, inp, reduce, feats=None, mats=None, rng_=None, grid=None):
    w = inp.workload
    return oracle.sampling_vt(inp.features if feats is None else feats,
                              inp.lidar2img if mats is None else mats,
                              w.img_hw, rng_ or w.bev_range, grid or w.grid, reduce)


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
def test_camera_permutation_invariance(oracle, case, reduce):
    perm = [2, 0, 3, 1, 5, 4]
    a = _run(oracle, case, reduce)
    b = _run(oracle, case, reduce, feats=case.features[:, perm], mats=case.lidar2img[:, perm])
    assert np.array_equal(a.count, b.count)
    assert np.allclose(a.out, b.out, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
def test_linearity_in_features(oracle, case, reduce):
    rng = np.random.default_rng(5)
    # multiples of 1/16 keep 2*F1 + F2/2 exact in float32: only the fp64 summation order differs
    F1 = (np.round(case.features * 16) / 16).astype(np.float32)
    F2 = (np.round(rng.standard_normal(case.features.shape) * 16) / 16).astype(np.float32)
    mix = (2.0 * F1 + 0.5 * F2).astype(np.float32)
    a, b, c = (_run(oracle, case, reduce, feats=F1), _run(oracle, case, reduce, feats=F2),
               _run(oracle, case, reduce, feats=mix))
    assert np.allclose(c.out, 2.0 * a.out + 0.5 * b.out, rtol=0, atol=1e-12)


def test_z_split_additivity(oracle, case):
    x0, x1, y0, y1, z0, z1 = case.workload.bev_range
    zm = 0.5 * (z0 + z1)
    X, Y, Z = case.workload.grid
    full = _run(oracle, case, SUM)
    lo = _run(oracle, case, SUM, rng_=(x0, x1, y0, y1, z0, zm), grid=(X, Y, Z // 2))
    hi = _run(oracle, case, SUM, rng_=(x0, x1, y0, y1, zm, z1), grid=(X, Y, Z // 2))
    assert np.array_equal(full.count, lo.count + hi.count)
    assert np.allclose(full.out, lo.out + hi.out, rtol=0, atol=1e-12)


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
def test_grid_subset_invariance(oracle, case, reduce):
    """No cross-cell dependency (Sec. 3.2.2): a sub-rectangle reproduces its cells."""
    x0, x1, y0, y1, z0, z1 = case.workload.bev_range
    X, Y, Z = case.workload.grid
    dx, dy = (x1 - x0) / X, (y1 - y0) / Y
    full = _run(oracle, case, reduce)
    sub = _run(oracle, case, reduce, rng_=(x0 + 2 * dx, x0 + 5 * dx, y0 + 1 * dy, y0 + 4 * dy, z0, z1), grid=(3, 3, Z))
    assert np.allclose(sub.out, full.out[:, 2:5, 1:4], rtol=0, atol=1e-11)
    assert np.array_equal(sub.count, full.count[:, 2:5, 1:4])


def test_batch_elements_are_independent(oracle, case):
    a = _run(oracle, case, EQ1)
    b = _run(oracle, case, EQ1, feats=case.features[1:], mats=case.lidar2img[1:])
    assert np.array_equal(a.out[1:], b.out)


def test_unseen_cells_are_exactly_zero(oracle):
    w = wl.get("tiny", C=4)
    inp = wl.make_inputs(w)
    for reduce in (SUM, MEAN, EQ1):
        r = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, reduce)
        assert (r.count == 0).sum() > 10
        assert np.all(r.out[r.count == 0] == 0.0)       # max(1, den) in Eq. 1


def test_reduce_mode_identities(oracle, case):
    s, m, e = (_run(oracle, case, k) for k in (SUM, MEAN, EQ1))
    # MEAN = SUM / max(1,count)
    assert np.allclose(m.out, s.out / np.maximum(1, s.count)[..., None], rtol=0, atol=1e-13)
    # one height bin: Eq. 1 is the valid mean
    x0, x1, y0, y1, z0, z1 = case.workload.bev_range
    X, Y, _ = case.workload.grid
    m1 = _run(oracle, case, MEAN, grid=(X, Y, 1))
    e1 = _run(oracle, case, EQ1, grid=(X, Y, 1))
    assert np.allclose(m1.out, e1.out, rtol=0, atol=1e-13)
    # a single camera: den_z <= 1 everywhere, so Eq. 1 equals the plain sum
    s1 = _run(oracle, case, SUM, feats=case.features[:, :1], mats=case.lidar2img[:, :1])
    e1 = _run(oracle, case, EQ1, feats=case.features[:, :1], mats=case.lidar2img[:, :1])
    assert np.array_equal(s1.out, e1.out)
    # two identical cameras: Eq. 1 is unchanged, the plain sum doubles
    f2, m2 = np.repeat(case.features[:, :1], 2, 1), np.repeat(case.lidar2img[:, :1], 2, 1)
    e2 = _run(oracle, case, EQ1, feats=f2, mats=m2)
    s2 = _run(oracle, case, SUM, feats=f2, mats=m2)
    assert np.allclose(e2.out, e1.out, rtol=0, atol=1e-13)
    assert np.allclose(s2.out, 2 * s1.out, rtol=0, atol=1e-13)
    # on the 6-camera rig some height bins are seen twice, and there the modes differ
    assert np.any(s.count > s.nzbins)
    assert not np.allclose(s.out, e.out)
    same = s.count == s.nzbins             # cells whose bins are each seen at most once
    assert np.array_equal(s.out[same], e.out[same])


def test_bf16_rounding_of_inputs_is_ties_to_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.1415927], np.float32)
    vals, bits = wl.round_to_bf16(x)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    assert vals[0] == 1.0 and vals[1] == 1.0 and vals[2] == 1.015625 and vals[3] == -2.5
    assert abs(vals[4] - 3.140625) < 1e-9
    import torch
    t = torch.from_numpy(x).to(torch.bfloat16).view(torch.uint16).numpy()
    assert np.array_equal(t, bits)


def test_rejects_bad_arguments(oracle):
    f = np.zeros((1, 1, 2, 2, 1), np.float32)
    M = np.zeros((1, 1, 4, 4), np.float32)
    with pytest.raises(ValueError):
        oracle.sampling_vt(f, M, (4, 4), (1, -1, -1, 1, 0, 1), (1, 1, 1), SUM)   # x_max <= x_min
    with pytest.raises(ValueError):
        oracle.sampling_vt(f, M, (4, 4), (-1, 1, -1, 1, 0, 1), (1, 1, 1), 7)     # unknown reduce


# ---------------------------------------------------------------- backward oracle (gradient w.r.t. features)

@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
@pytest.mark.parametrize("general", [False, True])
def test_backward_is_the_adjoint_of_the_forward(oracle, reduce, general):
    """<forward(F), G> == <F, backward(G)> for arbitrary F, G fixes the backward completely
    (the forward is linear in F), so every pin of the forward oracle carries over."""
    inp = _tiny_case(3, general, N=6, C=4, Hf=6, Wf=9, grid=(7, 6, 5))
    w = inp.workload
    rng = np.random.default_rng(11)
    for trial in range(3):
        F = rng.standard_normal(inp.features.shape).astype(np.float32)
        G = rng.standard_normal((w.B,) + tuple(w.grid[:2]) + (w.C,))
        out = oracle.sampling_vt(F, inp.lidar2img, w.img_hw, w.bev_range, w.grid, reduce).out
        gF = oracle.sampling_vt_backward(G, inp.lidar2img, w.feat_hw, w.img_hw, w.bev_range, w.grid, reduce)
        lhs, rhs = float((out * G).sum()), float((F.astype(np.float64) * gF).sum())
        assert np.abs(out).sum() > 10.0 and np.abs(gF).sum() > 10.0      # not vacuous
        assert lhs == pytest.approx(rhs, rel=1e-12, abs=1e-12)


def test_backward_single_sample_by_hand(oracle):
    # the orthographic sample of test_single_sample_orthographic_by_hand: taps (2,1) .375 (3,1) .125 (2,2) .375 (3,2) .125
    M = ortho(1.0, 5.5, 1.0, 4.0)[None, None]
    G = np.array([2.0, -1.0]).reshape(1, 1, 1, 2)
    g = oracle.sampling_vt_backward(G, M, (4, 6), (8, 12), (-1, 1, -1, 1, 0, 2), (1, 1, 1), SUM)
    expect = np.zeros((4, 6))
    expect[1, 2], expect[1, 3], expect[2, 2], expect[2, 3] = .375, .125, .375, .125
    assert np.allclose(g[0, 0, :, :, 0], 2.0 * expect, atol=1e-12)
    assert np.allclose(g[0, 0, :, :, 1], -1.0 * expect, atol=1e-12)


def test_backward_normalisations_and_untouched_texels(oracle):
    inp = _tiny_case(4, False, N=6, C=2, Hf=6, Wf=9, grid=(7, 6, 4))
    w = inp.workload
    G = np.ones((w.B,) + tuple(w.grid[:2]) + (w.C,))
    fwd = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, SUM)
    gs = oracle.sampling_vt_backward(G, inp.lidar2img, w.feat_hw, w.img_hw, w.bev_range, w.grid, SUM)
    gm = oracle.sampling_vt_backward(G, inp.lidar2img, w.feat_hw, w.img_hw, w.bev_range, w.grid, MEAN)
    ge = oracle.sampling_vt_backward(G, inp.lidar2img, w.feat_hw, w.img_hw, w.bev_range, w.grid, EQ1)
    # with G == 1 the gradient sums the weights: total mass = in-bounds weight mass of the forward
    assert gs.sum() / w.C == pytest.approx(fwd.sumw.sum(), rel=1e-12)
    assert np.all(gs >= 0) and np.all(gm <= gs + 1e-15) and np.all(ge <= gs + 1e-15)
    assert (gs == 0).any()                       # texels nobody samples get exactly zero
    # pre-scaling G by 1/max(1,count) turns the SUM backward into the MEAN backward
    Gs = G / np.maximum(1, fwd.count)[..., None]
    assert np.allclose(oracle.sampling_vt_backward(Gs, inp.lidar2img, w.feat_hw, w.img_hw, w.bev_range, w.grid, SUM),
                       gm, rtol=0, atol=1e-13)


def test_oracle_has_not_drifted_from_its_committed_outputs(oracle):
    """Regression guard (not a correctness pin): values written by tests/golden/make_oracle_regression.py."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_oracle_regression", os.path.join(GOLDEN, "make_oracle_regression.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    want = [l.split() for l in open(os.path.join(GOLDEN, "oracle_regression.txt")) if not l.startswith("#")]
    got = mod.rows()
    assert len(want) == len(got) == 15
    for wrow, grow in zip(want, got):
        assert [int(v) for v in wrow[:5]] == list(grow[:5])
        assert float(wrow[5]) == pytest.approx(grow[5], rel=1e-13, abs=1e-13)
