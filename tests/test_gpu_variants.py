"""Variants of the operator: channel-planar (NCHW) tensors and bfloat16 output."""
import numpy as np
import pytest

from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu
SUM, MEAN, EQ1 = 0, 1, 2


def _cuda_features(inp, layout):
    import torch
    w = inp.workload
    dev = torch.device("cuda:0")
    if w.dtype == "bf16":
        f = torch.from_numpy(inp.features_bf16.view(np.int16)).to(dev).view(torch.bfloat16)
    else:
        f = torch.from_numpy(inp.features).to(dev)
    if layout == fb.NCHW:
        f = f.permute(0, 1, 4, 2, 3).contiguous()
    return f, torch.from_numpy(inp.lidar2img).to(dev)


def _bf16_to_f32(t):
    import torch
    return t.to(torch.float32).cpu().numpy()


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
@pytest.mark.parametrize("dtype,C", [("f32", 5), ("f32", 32), ("f32", 44), ("bf16", 24), ("bf16", 7), ("bf16", 72)])
def test_nchw_tensors(oracle, reduce, dtype, C):
    import torch
    w = wl.Workload(f"nchw{C}", 3000 + C, 2, 5, C, dtype, (10, 14), (80, 112), (17, 13, 6),
                    (-10.0, 10.0, -10.0, 10.0, -3.0, 2.0), 0, general_pose=True)
    inp = wl.make_inputs(w)
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, reduce)
    f, m = _cuda_features(inp, fb.NCHW)
    X, Y, Z = w.grid
    cnt = torch.full((w.B, X, Y), -1, dtype=torch.int32, device=f.device)
    elem = 4 if dtype == "f32" else 2
    for workspace in (True, False):
        cnt.fill_(-1)
        out = fb.sampling_vt(f, m, w.img_hw, w.bev_range, w.grid, reduce, valid_count=cnt, layout=fb.NCHW, workspace=workspace)
        # with the scratch lent, shapes with whole 16-byte channel rows run the tiled kernel on a channels-last copy
        tiled = workspace and (C * elem) % 16 == 0
        assert fb.flashbev_last_kernel_name().startswith("tiled" if tiled else "per_output_nchw")
        assert fb.flashbev_last_kernel_name().endswith("nchw" if tiled else ("bf16" if dtype == "bf16" else "f32"))
        assert fb.flashbev_last_launch_count() == (2 if tiled else 1)
        assert out.shape == (w.B, C, X, Y)
        parity.assert_parity(w, ref, out.permute(0, 2, 3, 1).cpu().numpy(), cnt.cpu().numpy(), "[nchw]", check_fraction=False)


def test_nchw_benchmark_shape(oracle):
    import torch
    w = wl.get("tiny")
    inp = wl.make_inputs(w)
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, EQ1)
    f, m = _cuda_features(inp, fb.NCHW)
    out = fb.sampling_vt(f, m, w.img_hw, w.bev_range, w.grid, EQ1, layout=fb.NCHW)
    assert fb.flashbev_last_kernel_name() == "tiled_f32_nchw"
    parity.assert_parity(w, ref, out.permute(0, 2, 3, 1).cpu().numpy(), None, "[nchw tiny]")
    # the planar result is the channels-last result, bit for bit (same kernel, same order of sums)
    f2, _ = _cuda_features(inp, fb.NHWC)
    out2 = fb.sampling_vt(f2, m, w.img_hw, w.bev_range, w.grid, EQ1)
    assert torch.equal(out.permute(0, 2, 3, 1), out2)


@pytest.mark.parametrize("name", ["representative", "half_taller"])
def test_nchw_benchmark_configurations_on_the_tiled_kernel(oracle, name):
    """Two benchmark configurations as channel-planar tensors (fp32 and bf16 features), against the oracle."""
    import torch
    w = wl.get(name)
    inp = wl.make_inputs(w)
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, w.reduce)
    f, m = _cuda_features(inp, fb.NCHW)
    X, Y, Z = w.grid
    cnt = torch.full((w.B, X, Y), -1, dtype=torch.int32, device=f.device)
    out = fb.sampling_vt(f, m, w.img_hw, w.bev_range, w.grid, w.reduce, valid_count=cnt, layout=fb.NCHW)
    assert fb.flashbev_last_kernel_name().startswith("tiled") and fb.flashbev_last_kernel_name().endswith("nchw")
    parity.assert_parity(w, ref, out.permute(0, 2, 3, 1).cpu().numpy(), cnt.cpu().numpy(), f"[nchw {name}]")


@pytest.mark.parametrize("kernel", [fb.KERNEL_AUTO, fb.KERNEL_PER_OUTPUT])
@pytest.mark.parametrize("name,reduce", [("tiny", SUM), ("representative", EQ1), ("half_taller", MEAN)])
def test_bf16_output_is_the_fp32_result_rounded_once(oracle, kernel, name, reduce):
    """|out - oracle| <= (tolerance of the fp32-output path) + half a bf16 ulp of the value (2^-9 |ref|)."""
    import torch
    w = wl.get(name)
    inp = wl.make_inputs(w)
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, reduce)
    f, m = _cuda_features(inp, fb.NHWC)
    out = fb.sampling_vt(f, m, w.img_hw, w.bev_range, w.grid, reduce, kernel=kernel, out_dtype=fb.BF16)
    assert out.dtype == torch.bfloat16
    got = _bf16_to_f32(out).astype(np.float64)
    keep = ref.flagged == 0
    base = 1e-4 if w.dtype == "f32" else 2e-3 * np.sqrt(np.maximum(1, ref.count))[..., None]
    bound = (base + np.abs(ref.out) * 2.0 ** -8 + 1e-30) * np.ones_like(ref.out)
    err = np.abs(got - ref.out)
    assert np.all(err[keep] <= bound[keep]), float((err / bound)[keep].max())
    # and it is exactly the rounding of the fp32 output of the same kernel
    out32 = fb.sampling_vt(f, m, w.img_hw, w.bev_range, w.grid, reduce, kernel=kernel)
    assert torch.equal(out32.to(torch.bfloat16), out)   # (both kernels: same sums, one rounding at the store)


def test_bf16_output_with_nchw(oracle):
    import torch
    w = wl.Workload("nchw_bf16out", 3100, 1, 4, 6, "f32", (8, 12), (64, 96), (9, 8, 4),
                    (-8.0, 8.0, -8.0, 8.0, -3.0, 2.0), 0, general_pose=True)
    inp = wl.make_inputs(w)
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, SUM)
    f, m = _cuda_features(inp, fb.NCHW)
    out = fb.sampling_vt(f, m, w.img_hw, w.bev_range, w.grid, SUM, layout=fb.NCHW, out_dtype=fb.BF16)
    got = _bf16_to_f32(out.permute(0, 2, 3, 1)).astype(np.float64)
    assert np.all(np.abs(got - ref.out) <= 1e-4 + np.abs(ref.out) * 2.0 ** -8)


@pytest.mark.parametrize("name", ["representative", "half_taller"])
def test_feature_pointer_aligned_to_16_but_not_32_bytes(name):
    """The 256-bit loads need 32-byte alignment; a tensor that starts 16 bytes later takes the 128-bit
    instance and must give the same numbers (every cell adds its taps in the same order)."""
    import torch
    w = wl.get(name)
    inp = wl.make_inputs(w)
    f, m = _cuda_features(inp, fb.NHWC)
    shifted_store = torch.empty(f.numel() + 16 // f.element_size(), dtype=f.dtype, device=f.device)
    shifted = shifted_store[16 // f.element_size():].view(f.shape)
    shifted.copy_(f)
    assert f.data_ptr() % 32 == 0 and shifted.data_ptr() % 32 == 16
    a = fb.sampling_vt(f, m, w.img_hw, w.bev_range, w.grid, w.reduce)
    b = fb.sampling_vt(shifted, m, w.img_hw, w.bev_range, w.grid, w.reduce)
    assert torch.equal(a, b)


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
@pytest.mark.parametrize("dtype,C", [("f32", 1), ("f32", 5), ("f32", 82), ("bf16", 7), ("bf16", 12), ("bf16", 130)])
def test_ragged_channel_counts_on_the_tiled_kernel(oracle, reduce, dtype, C):
    """Channels-last rows that are not whole 16-byte vectors: with the scratch lent the tiled kernel runs on a copy with
    zero-padded rows and writes the caller's ragged rows one channel at a time; without it the generic kernel runs.
    Same oracle either way, and not a byte outside the output rows is touched."""
    import torch
    w = wl.Workload(f"ragged{C}", 3300 + C, 2, 5, C, dtype, (10, 14), (80, 112), (17, 13, 6),
                    (-10.0, 10.0, -10.0, 10.0, -3.0, 2.0), 0, general_pose=True)
    inp = wl.make_inputs(w)
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, reduce)
    f, m = _cuda_features(inp, fb.NHWC)
    X, Y, Z = w.grid
    for workspace in (True, False):
        cnt = torch.full((w.B, X, Y), -1, dtype=torch.int32, device=f.device)
        guard = torch.full((w.B * X * Y * C + 64,), 7.0, device=f.device)
        out = guard[:w.B * X * Y * C].view(w.B, X, Y, C)
        fb.sampling_vt(f, m, w.img_hw, w.bev_range, w.grid, reduce, out=out, valid_count=cnt, workspace=workspace)
        name = fb.flashbev_last_kernel_name()
        assert name == (("tiled_bf16_padded" if dtype == "bf16" else "tiled_f32_padded") if workspace else
                        ("per_output_bf16x1" if dtype == "bf16" else "per_output_f32x1"))
        assert fb.flashbev_last_launch_count() == (2 if workspace else 1)
        assert bool((guard[w.B * X * Y * C:] == 7.0).all())
        parity.assert_parity(w, ref, out.cpu().numpy(), cnt.cpu().numpy(), f"[ragged {name}]", check_fraction=False)
