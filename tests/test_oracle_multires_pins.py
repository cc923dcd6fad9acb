"""Pins of the oracle's multi-resolution sum: it must be the sum over levels of the single-level operator,
checked against properties that do not go through the function under test."""
import numpy as np
import pytest

from paper_2607_10071_b200 import workloads as wl
from tests import alg1_tensorized

SUM, MEAN, EQ1 = 0, 1, 2


def _case(seed, levels=3):
    w = wl.Workload("mr", 5000 + seed, 1, 6, 3, "f32", (12, 20), (96, 160), (9, 8, 5),
                    (-12.0, 12.0, -12.0, 12.0, -3.0, 2.0), 0, general_pose=True)
    feats, _, mats = wl.make_pyramid_inputs(w, levels)
    return w, feats, mats


def test_one_level_is_the_single_level_operator(oracle):
    w, feats, mats = _case(0, 1)
    a = oracle.sampling_vt_multires(feats, mats, w.img_hw, w.bev_range, w.grid, EQ1)
    b = oracle.sampling_vt(feats[0], mats, w.img_hw, w.bev_range, w.grid, EQ1)
    assert a.count.sum() > 20
    assert np.array_equal(a.out, b.out) and np.array_equal(a.count, b.count)


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
def test_two_levels_of_one_size_equal_one_level_of_their_sum(oracle, reduce):
    """The operator is linear in the features: levels of equal size can be added before sampling."""
    w, feats, mats = _case(1, 1)
    rng = np.random.default_rng(3)
    f1 = (rng.integers(-64, 64, feats[0].shape) / 16.0).astype(np.float32)   # exactly representable
    f2 = (rng.integers(-64, 64, feats[0].shape) / 16.0).astype(np.float32)
    a = oracle.sampling_vt_multires([f1, f2], mats, w.img_hw, w.bev_range, w.grid, reduce)
    b = oracle.sampling_vt(f1 + f2, mats, w.img_hw, w.bev_range, w.grid, reduce)
    assert np.abs(b.out).max() > 0.5
    assert np.allclose(a.out, b.out, rtol=0, atol=1e-12)


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
def test_pyramid_matches_array_code_with_library_bilinear(oracle, reduce):
    """Every level evaluated by the tensorised order with the library sampler, summed here."""
    w, feats, mats = _case(2, 3)
    assert [f.shape[2:4] for f in feats] == [(12, 20), (6, 10), (3, 5)]
    a = oracle.sampling_vt_multires(feats, mats, w.img_hw, w.bev_range, w.grid, reduce)
    ref = 0.0
    for f in feats:
        r, cnt, _ = alg1_tensorized.sampling_vt_tensorized(f, mats, w.img_hw, w.bev_range, w.grid, reduce)
        assert np.array_equal(cnt, a.count)      # validity does not depend on the level
        ref = ref + r
    assert a.count.sum() > 20
    assert np.allclose(a.out, ref, rtol=0, atol=1e-11)


def test_a_constant_pyramid_sums_the_levels(oracle):
    """Interior cells of constant maps: every level returns its constant times the valid count."""
    w, feats, mats = _case(3, 3)
    consts = [1.0, -0.5, 0.25]
    const_feats = [np.full_like(f, c) for f, c in zip(feats, consts)]
    a = oracle.sampling_vt_multires(const_feats, mats, w.img_hw, w.bev_range, w.grid, SUM)
    per_level = [oracle.sampling_vt(f, mats, w.img_hw, w.bev_range, w.grid, SUM) for f in const_feats]
    inner = per_level[0].interior & per_level[1].interior & per_level[2].interior & (a.count > 0)
    assert inner.sum() > 5
    expect = a.count[inner] * sum(consts)
    assert np.allclose(a.out[inner][:, 0], expect, rtol=0, atol=1e-9)
