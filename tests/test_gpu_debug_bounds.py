"""The bounds-checked build of the CUDA library (-DFLASHBEV_DEBUG_BOUNDS) on a GPU.

No memory checker may run on the shared machines, so the library can be built with its own guard: every
shared-memory slot, record offset and output index the tiled kernel computes goes through a range check that
counts a violation into the caller's ``debug_error_word`` and redirects the access to a safe slot.  These tests
run the benchmark configurations, the many-rounds stress case, odd shapes and the backward pass in that build,
require the word to stay 0 and the results to match the oracle as in the normal build.
"""
import numpy as np
import pytest
from hypothesis import HealthCheck, given, settings, strategies as st

from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import build as fbuild
from paper_2607_10071_b200 import workloads as wl
from tests import parity
from tests.test_gpu_parity import small

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def checked():
    return fb.load_library(fbuild.build(debug_bounds=True))


def run_checked(checked, inp, reduce, tune=(0, 0, 0, 0)):
    import torch
    w = inp.workload
    dev = torch.device("cuda:0")
    if w.dtype == "bf16":
        feats = torch.from_numpy(inp.features_bf16.view(np.int16)).to(dev).view(torch.bfloat16)
    else:
        feats = torch.from_numpy(inp.features).to(dev)
    mats = torch.from_numpy(inp.lidar2img).to(dev)
    X, Y, Z = w.grid
    out = torch.full((w.B, X, Y, w.C), float("nan"), dtype=torch.float32, device=dev)
    cnt = torch.full((w.B, X, Y), -1, dtype=torch.int32, device=dev)
    word = torch.zeros(1, dtype=torch.int32, device=dev)
    p = fb.make_params(feats.data_ptr(), fb.BF16 if w.dtype == "bf16" else fb.F32, mats.data_ptr(), w.B, w.N, w.C,
                       w.feat_hw, w.img_hw, w.bev_range, w.grid, reduce, out.data_ptr(), cnt.data_ptr(), fb.KERNEL_TILED,
                       tune, debug_error_word=word.data_ptr())
    fb.flashbev_sampling_vt(p, torch.cuda.current_stream().cuda_stream, library=checked)
    torch.cuda.synchronize()
    return out.cpu().numpy(), cnt.cpu().numpy(), int(word.item())


@pytest.mark.parametrize("name", wl.CONFIG_ORDER)
def test_benchmark_configurations_make_no_out_of_range_index(oracle, checked, name):
    inp = wl.make_inputs(wl.get(name))
    w = inp.workload
    for reduce in {w.reduce, 2}:
        out, cnt, violations = run_checked(checked, inp, reduce)
        assert violations == 0, f"{name} reduce={reduce}: {violations} out-of-range indices"
        ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, reduce)
        parity.assert_parity(w, ref, out, cnt, f"[bounds-checked build, reduce={reduce}]")


def test_many_rounds_and_odd_shapes_make_no_out_of_range_index(oracle, checked):
    # all cameras overlap: far more records per cell than the slots hold
    w = wl.Workload("overlap", 77, 1, 8, 32, "f32", (24, 40), (192, 320), (12, 10, 96),
                    (8.0, 20.0, -5.0, 5.0, -2.0, 4.0), 0, general_pose=False, yaw_jitter_deg=0.0)
    inp = wl.make_inputs(w)
    inp.lidar2img[:] = inp.lidar2img[:, :1]
    inp.lidar2img[0, :, 0, 3] += np.arange(8, dtype=np.float32) * 3.0
    cases = [(inp, 2, (0, 0, 0, 0)), (inp, 0, (0, 0, 4, 0x04000000)), (inp, 1, (0, 0, 64, 0))]
    for seed, kw in ((1, dict(grid=(1, 1, 1))), (2, dict(grid=(33, 31, 7), C=80)), (3, dict(feat=(1, 1))),
                     (4, dict(feat=(12, 1))), (5, dict(N=33, C=16, grid=(10, 9, 6))), (6, dict(grid=(9, 11, 300), B=1)),
                     (7, dict(C=128, dtype="bf16", general=False, grid=(40, 40, 12), rng_xy=30.0)),
                     (8, dict(C=260)), (9, dict(C=264, dtype="bf16"))):
        cases.append((small(700 + seed, **kw), 2, (0, 0, 0, 0)))
    for case, reduce, tune in cases:
        out, cnt, violations = run_checked(checked, case, reduce, tune)
        assert violations == 0, f"{case.workload.name} {case.workload.grid} reduce={reduce} tune={tune}: {violations}"
        assert np.all(np.isfinite(out))
        assert cnt.min() >= 0


@pytest.mark.parametrize("name", ["half_taller", "paper_shape", "representative"])
def test_launch_geometry_hints_make_no_out_of_range_index(oracle, checked, name):
    """Super-block shapes, tail lengths, orders and warps per CTA that leave padding warps in the last CTA and
    partial super-blocks at the grid's edge."""
    inp = wl.make_inputs(wl.get(name))
    w = inp.workload
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, w.reduce)
    shapes = [0, (1 << 4) | (2 << 8), (2 << 4) | (3 << 8), (3 << 4) | (3 << 8)]
    for shape in shapes:
        for tail in range(8):
            for extra in (0, 1 << 28, 2, 8, 1 << 18):       # default, row-major order, 2 / 8 warps per CTA, single-row bands
                tune = (0, 0, 0, shape | (32 << 20) | (tail << 29) | extra)
                out, cnt, violations = run_checked(checked, inp, w.reduce, tune)
                assert violations == 0, f"{name} tune[3]={tune[3]:#x}: {violations} out-of-range indices"
                assert np.array_equal(cnt[ref.flagged == 0], ref.count[ref.flagged == 0]), hex(tune[3])


@pytest.mark.parametrize("name,C,reduce,tune3", [
    ("tiny", 32, 2, 0), ("tiny", 32, 1, 0), ("representative", 80, 0, 0), ("representative", 24, 2, 0),
    ("representative", 144, 1, 0), ("representative", 80, 0, (2 << 4) | (4 << 8)),
])
def test_backward_makes_no_out_of_range_index(checked, name, C, reduce, tune3):
    """The backward in the checked build: the error word stays 0 and the result equals the normal build's up to the
    order of the atomic sums."""
    import torch
    w = wl.get(name, C=C)
    inp = wl.make_inputs(w)
    dev = torch.device("cuda:0")
    X, Y, Z = w.grid
    go = torch.randn((w.B, X, Y, w.C), generator=torch.Generator().manual_seed(3)).to(dev)
    mats = torch.from_numpy(inp.lidar2img).to(dev)
    ref = fb.sampling_vt_backward(go, mats, w.feat_hw, w.img_hw, w.bev_range, w.grid, reduce)
    gf = torch.empty_like(ref)
    word = torch.zeros(1, dtype=torch.int32, device=dev)
    p = fb.make_backward_params(go.data_ptr(), mats.data_ptr(), w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range, w.grid, reduce,
                                gf.data_ptr(), (0, 0, 0, tune3), debug_error_word=word.data_ptr())
    fb.flashbev_sampling_vt_backward(p, torch.cuda.current_stream().cuda_stream, library=checked)
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    scale = float(ref.abs().max())
    assert float((gf - ref).abs().max()) <= 1e-5 * max(1.0, scale)


@st.composite
def checked_cases(draw):
    dtype = draw(st.sampled_from(["f32", "bf16"]))
    vec = 4 if dtype == "f32" else 8
    return dict(
        seed=draw(st.integers(0, 10_000)), dtype=dtype, C=vec * draw(st.sampled_from([1, 2, 3, 5, 8, 10, 16, 20, 33])),
        B=draw(st.integers(1, 2)), N=draw(st.integers(1, 9)),
        feat=(draw(st.integers(1, 20)), draw(st.integers(1, 24))),
        grid=(draw(st.integers(1, 19)), draw(st.integers(1, 19)), draw(st.sampled_from([1, 2, 5, 8, 16, 40, 97, 200]))),
        general=draw(st.booleans()), rng_xy=draw(st.sampled_from([3.0, 10.0, 40.0])),
        reduce=draw(st.sampled_from([0, 1, 2])),
        walk=draw(st.sampled_from([0, 1, 4, 16, 64])), slots=draw(st.sampled_from([0, 64, 96, 256, 1024])),
        shape=draw(st.sampled_from([0, (1 << 4) | (1 << 8), (2 << 4) | (2 << 8), (4 << 4) | (4 << 8)])),
        tail=draw(st.integers(0, 7)), order=draw(st.sampled_from([0, 1 << 28, 1 << 18, 3 << 18])))


@settings(max_examples=150, deadline=None, derandomize=True,
          suppress_health_check=[HealthCheck.function_scoped_fixture, HealthCheck.too_slow])
@given(case=checked_cases())
def test_random_problems_and_hints_make_no_out_of_range_index(oracle, checked, case):
    """Random rigs (surround and general pose), shapes, dtypes, reduce modes and launch-geometry hints -- small record
    lists that force many rounds, long and short runs, every order of the work -- in the bounds-checked build: no index
    out of range, and the oracle's numbers."""
    w = wl.Workload("checked", 9000 + case["seed"], case["B"], case["N"], case["C"], case["dtype"], case["feat"],
                    (case["feat"][0] * 8, case["feat"][1] * 8), case["grid"],
                    (-case["rng_xy"], case["rng_xy"], -case["rng_xy"], case["rng_xy"], -3.0, 2.5), case["reduce"],
                    general_pose=case["general"], yaw_jitter_deg=5.0)
    inp = wl.make_inputs(w)
    tune = (0, 0, case["walk"], case["shape"] | ((case["slots"] // 16) << 20) | (case["tail"] << 29) | case["order"])
    try:
        out, cnt, violations = run_checked(checked, inp, case["reduce"], tune)
    except fb.FlashBevError as e:  # hints the forced tiled kernel cannot be configured for: refused on the host
        assert e.status == fb.UNSUPPORTED, e
        return
    assert violations == 0, f"{case}: {violations} out-of-range indices"
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, case["reduce"])
    parity.assert_parity(w, ref, out, cnt, f"[checked build {case}]", check_fraction=False, large_outputs=True)


@pytest.mark.parametrize("layout,dtype,C", [(fb.NCHW, "f32", 32), (fb.NCHW, "bf16", 72), (fb.NHWC, "f32", 82), (fb.NHWC, "bf16", 13)])
def test_copies_in_a_lent_workspace_make_no_out_of_range_index(oracle, checked, layout, dtype, C):
    """Planar tensors and ragged channel counts in the checked build: transposed / padded copy in the workspace, scalar
    stores with the caller's strides -- no index out of range, nothing written past the output, the oracle's numbers."""
    import torch
    w = wl.Workload("lent", 8800 + C, 2, 5, C, dtype, (10, 14), (80, 112), (23, 17, 12),
                    (-10.0, 10.0, -10.0, 10.0, -3.0, 2.0), 2, general_pose=False, yaw_jitter_deg=3.0)
    inp = wl.make_inputs(w)
    dev = torch.device("cuda:0")
    if dtype == "bf16":
        f = torch.from_numpy(inp.features_bf16.view(np.int16)).to(dev).view(torch.bfloat16)
    else:
        f = torch.from_numpy(inp.features).to(dev)
    if layout == fb.NCHW:
        f = f.permute(0, 1, 4, 2, 3).contiguous()
    m = torch.from_numpy(inp.lidar2img).to(dev)
    X, Y, Z = w.grid
    n_out = w.B * X * Y * C
    guard = torch.full((n_out + 64,), 7.0, device=dev)
    cnt = torch.full((w.B, X, Y), -1, dtype=torch.int32, device=dev)
    word = torch.zeros(1, dtype=torch.int32, device=dev)
    p = fb.make_params(f.data_ptr(), fb.BF16 if dtype == "bf16" else fb.F32, m.data_ptr(), w.B, w.N, C, w.feat_hw, w.img_hw,
                       w.bev_range, w.grid, 2, guard.data_ptr(), cnt.data_ptr(), layout=layout, debug_error_word=word.data_ptr())
    need = fb.flashbev_workspace_bytes(p)
    assert need > 0
    ws = torch.empty(need, dtype=torch.uint8, device=dev)
    p.workspace, p.workspace_bytes = ws.data_ptr(), need
    fb.flashbev_sampling_vt(p, torch.cuda.current_stream().cuda_stream, library=checked)
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    assert bool((guard[n_out:] == 7.0).all())
    out = guard[:n_out].view((w.B, C, X, Y) if layout == fb.NCHW else (w.B, X, Y, C))
    out = out.permute(0, 2, 3, 1) if layout == fb.NCHW else out
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, 2)
    parity.assert_parity(w, ref, out.cpu().numpy(), cnt.cpu().numpy(), "[lent workspace, checked build]", check_fraction=False)
