"""Multi-resolution gathering (sum of the operator over a feature pyramid) against the fp64 oracle."""
import dataclasses

import numpy as np
import pytest

from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu
SUM, MEAN, EQ1 = 0, 1, 2


def _upload(w, feats, bits, mats, layout=fb.NHWC):
    import torch
    dev = torch.device("cuda:0")
    out = []
    for f, b in zip(feats, bits):
        if w.dtype == "bf16":
            t = torch.from_numpy(b.view(np.int16)).to(dev).view(torch.bfloat16)
        else:
            t = torch.from_numpy(f).to(dev)
        if layout == fb.NCHW:
            t = t.permute(0, 1, 4, 2, 3).contiguous()
        out.append(t)
    return out, torch.from_numpy(mats).to(dev)


def _scaled(w, feats, bits, s):
    """Scale the values (a power of two, so bf16 patterns stay valid) to keep |out| within the fp32 budget."""
    feats = [f * np.float32(s) for f in feats]
    if w.dtype == "bf16":
        bits = [wl.round_to_bf16(f)[1] for f in feats]
    return feats, bits


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
@pytest.mark.parametrize("name,levels", [("tiny", 3), ("representative", 3), ("half_taller", 2)])
def test_pyramid_parity(oracle, name, levels, reduce):
    import torch
    w = wl.get(name)
    feats, bits, mats = wl.make_pyramid_inputs(w, levels)
    feats, bits = _scaled(w, feats, bits, 0.25)
    ref = oracle.sampling_vt_multires(feats, mats, w.img_hw, w.bev_range, w.grid, reduce)
    f, m = _upload(w, feats, bits, mats)
    X, Y, Z = w.grid
    out = torch.full((w.B, X, Y, w.C), float("nan"), dtype=torch.float32, device=m.device)
    cnt = torch.full((w.B, X, Y), -1, dtype=torch.int32, device=m.device)
    fb.sampling_vt_multires(f, m, w.img_hw, w.bev_range, w.grid, reduce, out=out, valid_count=cnt)
    assert fb.flashbev_last_launch_count() == levels
    assert fb.flashbev_last_kernel_name().startswith("tiled")
    # coarse levels widen the border band (1e-3 feature px is more image px): the flagged share is per level
    rep = parity.assert_parity(w, ref, out.cpu().numpy(), cnt.cpu().numpy(), f"[multires {name} r{reduce}]",
                               check_fraction=False)
    assert rep.flagged_fraction < levels * parity.MAX_FLAGGED_FRACTION
    print(name, levels, reduce, rep)


@pytest.mark.parametrize("kernel,layout", [(fb.KERNEL_PER_OUTPUT, fb.NHWC), (fb.KERNEL_PER_OUTPUT, fb.NCHW),
                                           (fb.KERNEL_AUTO, fb.NCHW), (fb.KERNEL_AUTO, fb.NHWC)])
@pytest.mark.parametrize("dtype,C", [("f32", 6), ("bf16", 24)])
def test_pyramid_generic_kernels_and_lent_workspace(oracle, kernel, layout, dtype, C):
    """Per-output kernels (odd channel counts, planar tensors) add the levels the same way, and so do the tiled kernel's
    scalar-store instances on the copies in the workspace the wrapper lends (planar tensors, ragged channel counts)."""
    w = wl.Workload(f"mrg{C}", 5100 + C, 2, 5, C, dtype, (11, 15), (88, 120), (13, 11, 6),
                    (-10.0, 10.0, -10.0, 10.0, -3.0, 2.0), 0, general_pose=True)
    feats, bits, mats = wl.make_pyramid_inputs(w, 3)
    ref = oracle.sampling_vt_multires(feats, mats, w.img_hw, w.bev_range, w.grid, EQ1)
    f, m = _upload(w, feats, bits, mats, layout)
    out = fb.sampling_vt_multires(f, m, w.img_hw, w.bev_range, w.grid, EQ1, kernel=kernel, layout=layout)
    whole = (C * (4 if dtype == "f32" else 2)) % 16 == 0
    if kernel == fb.KERNEL_PER_OUTPUT or (layout == fb.NCHW and not whole):
        assert fb.flashbev_last_kernel_name().startswith("per_output")
    elif layout == fb.NCHW:
        assert fb.flashbev_last_kernel_name().endswith("nchw")
    else:
        assert fb.flashbev_last_kernel_name().endswith("padded" if not whole else "v1")
    o = out.permute(0, 2, 3, 1) if layout == fb.NCHW else out
    parity.assert_parity(w, ref, o.cpu().numpy(), None, "[multires generic]", check_fraction=False)


def test_one_level_equals_the_single_level_call_bit_for_bit():
    import torch
    w = wl.get("tiny")
    feats, bits, mats = wl.make_pyramid_inputs(w, 1)
    f, m = _upload(w, feats, bits, mats)
    a = fb.sampling_vt_multires(f, m, w.img_hw, w.bev_range, w.grid, EQ1)
    b = fb.sampling_vt(f[0], m, w.img_hw, w.bev_range, w.grid, EQ1)
    assert torch.equal(a, b)


def test_levels_accumulate_in_order_and_ignore_what_out_held():
    """Level 0 overwrites (a NaN-filled output stays clean); two equal levels give twice one level."""
    import torch
    w = wl.get("tiny")
    feats, bits, mats = wl.make_pyramid_inputs(w, 1)
    f, m = _upload(w, feats, bits, mats)
    X, Y, Z = w.grid
    out = torch.full((w.B, X, Y, w.C), float("nan"), dtype=torch.float32, device=m.device)
    fb.sampling_vt_multires([f[0], f[0]], m, w.img_hw, w.bev_range, w.grid, SUM, out=out)
    first = fb.sampling_vt(f[0], m, w.img_hw, w.bev_range, w.grid, SUM)
    # added levels keep their sums in registers: the configuration with one sub-block per warp
    added = fb.sampling_vt(f[0], m, w.img_hw, w.bev_range, w.grid, SUM, tune=(0, 0, 0, 0x110))
    assert torch.isfinite(out).all()
    assert torch.equal(out, first + added)


def test_rejections():
    import torch
    w = wl.get("tiny")
    feats, bits, mats = wl.make_pyramid_inputs(w, 2)
    f, m = _upload(w, feats, bits, mats)
    X, Y, Z = w.grid
    out = torch.empty((w.B, X, Y, w.C), dtype=torch.float32, device=m.device)
    base = fb.make_params(f[0].data_ptr(), fb.F32, m.data_ptr(), w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range,
                          w.grid, SUM, out.data_ptr())
    hws = [tuple(t.shape[2:4]) for t in f]
    ptrs = [t.data_ptr() for t in f]
    assert fb.flashbev_sampling_vt_multires(base, [], [], check=False) == fb.INVALID_ARG
    assert fb.flashbev_sampling_vt_multires(base, ptrs * 5, hws * 5, check=False) == fb.INVALID_ARG   # 10 levels
    assert fb.flashbev_sampling_vt_multires(base, [ptrs[0], 0], hws, check=False) == fb.INVALID_ARG   # null level
    assert fb.flashbev_sampling_vt_multires(base, ptrs, [hws[0], (0, 5)], check=False) == fb.INVALID_ARG
    assert fb.flashbev_sampling_vt_multires(base, [ptrs[0], ptrs[1] + 2], hws, check=False) == fb.MISALIGNED
    bf = fb.make_params(f[0].data_ptr(), fb.F32, m.data_ptr(), w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range,
                        w.grid, SUM, out.data_ptr(), out_dtype=fb.BF16)
    assert fb.flashbev_sampling_vt_multires(bf, ptrs, hws, check=False) == fb.UNSUPPORTED
    assert fb.flashbev_sampling_vt_multires(base, ptrs, hws, check=False) == fb.OK
    torch.cuda.synchronize()
