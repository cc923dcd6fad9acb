"""GPU parity of the backward pass (gradient w.r.t. the features) against the fp64 oracle.

Tolerance: the kernel accumulates with fp32 atomics in an order that changes from run to run, so the
comparison is a relative one: relative L2 <= 2e-6 and max-abs <= 4e-6 * max|reference| (a texel
collects up to a few thousand fp32 contributions; their rounding errors add like 6e-8 * sqrt(n)).
"""
import numpy as np
import pytest
from hypothesis import HealthCheck, given, settings, strategies as st

from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import workloads as wl

pytestmark = pytest.mark.gpu
SUM, MEAN, EQ1 = 0, 1, 2


def run_backward(w, lidar2img, G, reduce, tune=(0, 0, 0, 0)):
    import torch
    dev = torch.device("cuda:0")
    g = torch.from_numpy(np.ascontiguousarray(G, np.float32)).to(dev)
    m = torch.from_numpy(lidar2img).to(dev)
    gf = torch.full((w.B, w.N, w.feat_hw[0], w.feat_hw[1], w.C), float("nan"), dtype=torch.float32, device=dev)
    fb.sampling_vt_backward(g, m, w.feat_hw, w.img_hw, w.bev_range, w.grid, reduce, grad_features=gf, tune=tune)
    name = fb.flashbev_last_kernel_name()
    torch.cuda.synchronize()
    return gf.cpu().numpy(), name


def check(oracle, w, lidar2img, reduce, seed=0, tune=(0, 0, 0, 0)):
    rng = np.random.default_rng(seed)
    G = rng.standard_normal((w.B,) + tuple(w.grid[:2]) + (w.C,)).astype(np.float32)
    ref = oracle.sampling_vt_backward(G, lidar2img, w.feat_hw, w.img_hw, w.bev_range, w.grid, reduce)
    got, name = run_backward(w, lidar2img, G, reduce, tune)
    assert name.startswith("tiled_bwd")
    assert np.all(np.isfinite(got)), "unwritten or non-finite gradient"
    err = np.abs(got - ref)
    rel = np.sqrt((err ** 2).sum() / max(1e-300, (ref ** 2).sum()))
    scale = np.abs(ref).max()
    msg = f"{w.name} reduce={reduce} {name}: rel_l2={rel:.2e} max_abs={err.max():.2e} max|ref|={scale:.2f}"
    assert rel <= 2e-6, msg
    assert err.max() <= 4e-6 * max(1.0, scale), msg
    assert np.all(got[ref == 0.0] == 0.0), msg          # texels nobody samples stay exactly zero
    return msg


@pytest.mark.parametrize("name", ["tiny", "representative"])
@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
def test_backward_benchmark_shapes(oracle, name, reduce):
    w = wl.get(name)
    inp = wl.make_inputs(w)
    print("\n" + check(oracle, w, inp.lidar2img, reduce))


def test_backward_long_range_shape_fp32(oracle):
    """The largest benchmark grid with 128 fp32 channels: many sub-blocks per warp, 32-vector texels, record
    offsets beyond 2^20 (the forward benchmark uses bf16 there; the backward is fp32 only)."""
    w = wl.get("long_range", dtype="f32")
    inp = wl.make_inputs(w)
    print("\n" + check(oracle, w, inp.lidar2img, SUM))


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
@pytest.mark.parametrize("C", [4, 36, 80, 128, 260])
def test_backward_general_pose_channel_counts(oracle, reduce, C):
    w = wl.Workload(f"bwd{C}", 2000 + C, 2, 6, C, "f32", (12, 20), (96, 160), (21, 19, 5),
                    (-12.0, 12.0, -12.0, 12.0, -3.0, 2.0), 0, general_pose=True)
    inp = wl.make_inputs(w)
    check(oracle, w, inp.lidar2img, reduce, seed=C)


def test_backward_many_heights_and_overlapping_cameras(oracle):
    w = wl.Workload("bwd_overlap", 78, 1, 8, 32, "f32", (24, 40), (192, 320), (12, 10, 96),
                    (8.0, 20.0, -5.0, 5.0, -2.0, 4.0), 0, general_pose=False, yaw_jitter_deg=0.0)
    inp = wl.make_inputs(w)
    inp.lidar2img[:] = inp.lidar2img[:, :1]
    inp.lidar2img[0, :, 0, 3] += np.arange(8, dtype=np.float32) * 3.0
    for reduce in (SUM, MEAN, EQ1):
        check(oracle, w, inp.lidar2img, reduce)
    check(oracle, w, inp.lidar2img, EQ1, tune=(0, 0, 3, 0))


def test_backward_is_the_adjoint_of_the_forward_on_the_gpu():
    import torch
    w = wl.get("representative")
    inp = wl.make_inputs(w)
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(3)
    G = rng.standard_normal((w.B,) + tuple(w.grid[:2]) + (w.C,)).astype(np.float32)
    for reduce in (SUM, MEAN, EQ1):
        out = fb.sampling_vt(torch.from_numpy(inp.features).to(dev), torch.from_numpy(inp.lidar2img).to(dev),
                             w.img_hw, w.bev_range, w.grid, reduce).cpu().numpy().astype(np.float64)
        gF, _ = run_backward(w, inp.lidar2img, G, reduce)
        lhs, rhs = (out * G).sum(), (inp.features.astype(np.float64) * gF).sum()
        assert lhs == pytest.approx(rhs, rel=2e-5), (reduce, lhs, rhs)


def test_backward_rejects_what_it_does_not_support():
    w = wl.get("tiny")
    good = dict(grad_out_ptr=4096, lidar2img_ptr=8192, B=w.B, N=w.N, C=w.C, feat_hw=w.feat_hw, img_hw=w.img_hw,
                bev_range=w.bev_range, grid=w.grid, reduce=0, grad_features_ptr=16384)
    for over, status in ((dict(C=30), fb.UNSUPPORTED), (dict(grad_out_ptr=4100), fb.MISALIGNED),
                         (dict(grad_features_ptr=None), fb.INVALID_ARG), (dict(reduce=5), fb.INVALID_ARG),
                         (dict(grid=(0, 50, 4)), fb.INVALID_ARG)):
        p = fb.make_backward_params(**{**good, **over})
        assert fb.flashbev_sampling_vt_backward(p, None, check=False) == status, over


@st.composite
def backward_cases(draw):
    return dict(
        seed=draw(st.integers(0, 10_000)), C=4 * draw(st.sampled_from([1, 2, 3, 5, 8, 10, 16, 20, 33])),
        B=draw(st.integers(1, 2)), N=draw(st.integers(1, 7)),
        feat=(draw(st.integers(1, 16)), draw(st.integers(1, 20))),
        grid=(draw(st.integers(1, 21)), draw(st.integers(1, 21)), draw(st.sampled_from([1, 2, 5, 8, 16, 40, 97]))),
        general=draw(st.booleans()), rng_xy=draw(st.sampled_from([3.0, 10.0, 40.0])),
        reduce=draw(st.sampled_from([SUM, MEAN, EQ1])),
        walk=draw(st.sampled_from([0, 1, 4, 32])), slots=draw(st.sampled_from([0, 64, 128, 1024])),
        shape=draw(st.sampled_from([0, (1 << 4) | (1 << 8), (2 << 4) | (2 << 8), (4 << 4) | (2 << 8)])))


@settings(max_examples=80, deadline=None, derandomize=True,
          suppress_health_check=[HealthCheck.function_scoped_fixture, HealthCheck.too_slow])
@given(case=backward_cases())
def test_backward_random_problems_match_the_oracle(oracle, case):
    """Random rigs (surround and general pose), shapes, reduce modes and launch-geometry hints against the oracle's
    backward; hints the kernel cannot be configured for are refused on the host."""
    w = wl.Workload("bwd_prop", 7000 + case["seed"], case["B"], case["N"], case["C"], "f32", case["feat"],
                    (case["feat"][0] * 8, case["feat"][1] * 8), case["grid"],
                    (-case["rng_xy"], case["rng_xy"], -case["rng_xy"], case["rng_xy"], -3.0, 2.5), case["reduce"],
                    general_pose=case["general"], yaw_jitter_deg=5.0)
    inp = wl.make_inputs(w)
    tune = (0, 0, case["walk"], case["shape"] | ((case["slots"] // 16) << 20))
    try:
        check(oracle, w, inp.lidar2img, case["reduce"], seed=case["seed"], tune=tune)
    except fb.FlashBevError as e:
        assert e.status == fb.UNSUPPORTED, e
