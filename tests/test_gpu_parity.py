"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle, element by element."""
import numpy as np
import pytest

from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

SUM, MEAN, EQ1 = 0, 1, 2
_oracle_cache = {}


def oracle_of(oracle, inp, reduce):
    key = (id(inp), reduce)
    if key not in _oracle_cache:
        w = inp.workload
        _oracle_cache[key] = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, reduce)
    return _oracle_cache[key]


@pytest.fixture(scope="module")
def bench_inputs():
    return {name: wl.make_inputs(wl.get(name)) for name in wl.CONFIG_ORDER}


# ---------------------------------------------------------------- the five benchmark configurations, full size

@pytest.mark.parametrize("name", wl.CONFIG_ORDER)
@pytest.mark.parametrize("mode", ["own", "eq1"])
def test_benchmark_config_tiled(oracle, bench_inputs, name, mode):
    inp = bench_inputs[name]
    w = inp.workload
    reduce = w.reduce if mode == "own" else EQ1
    out, cnt, kname = parity.run_gpu(inp, reduce, fb.KERNEL_AUTO)
    assert kname.startswith("tiled")
    rep = parity.assert_parity(w, oracle_of(oracle, inp, reduce), out, cnt, f"[{kname} reduce={reduce}]")
    print(f"\n{name} reduce={reduce} {kname}: {rep}")


@pytest.mark.parametrize("name", wl.CONFIG_ORDER)
def test_benchmark_config_per_output_kernel(oracle, bench_inputs, name):
    inp = bench_inputs[name]
    w = inp.workload
    out, cnt, kname = parity.run_gpu(inp, w.reduce, fb.KERNEL_PER_OUTPUT)
    assert kname.startswith("per_output")
    parity.assert_parity(w, oracle_of(oracle, inp, w.reduce), out, cnt, f"[{kname}]")


def test_half_taller_all_modes(oracle, bench_inputs):
    inp = bench_inputs["half_taller"]
    for reduce in (SUM, MEAN, EQ1):
        out, cnt, kname = parity.run_gpu(inp, reduce)
        parity.assert_parity(inp.workload, oracle_of(oracle, inp, reduce), out, cnt, f"[{kname} reduce={reduce}]")


# ---------------------------------------------------------------- small, odd and degenerate shapes

def small(seed, B=2, N=6, C=32, dtype="f32", feat=(12, 20), grid=(21, 19, 5), general=True, rng_xy=12.0,
          z=(-3.0, 2.0), stride=8, fov=70.0, jitter=5.0):
    w = wl.Workload(f"small{seed}", 1000 + seed, B, N, C, dtype, feat, (feat[0] * stride, feat[1] * stride), grid,
                    (-rng_xy, rng_xy, -rng_xy, rng_xy, z[0], z[1]), 0, general_pose=general, fov_deg=fov,
                    yaw_jitter_deg=jitter)
    return wl.make_inputs(w)


def check_small(oracle, inp, reduce, kernel=fb.KERNEL_AUTO, tune=(0, 0, 0, 0), large_outputs=False):
    w = inp.workload
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, reduce)
    out, cnt, kname = parity.run_gpu(inp, reduce, kernel, tune)
    rep = parity.assert_parity(w, ref, out, cnt, f"[{kname} reduce={reduce} tune={tune}]", check_fraction=False,
                               large_outputs=large_outputs)
    if large_outputs:
        print(f"\n{w.name} {w.grid} reduce={reduce}: max|ref|={np.abs(ref.out).max():.1f} {rep}")
    return ref, out, kname


@pytest.mark.parametrize("reduce", [SUM, MEAN, EQ1])
@pytest.mark.parametrize("kernel", [fb.KERNEL_PER_OUTPUT, fb.KERNEL_TILED])
@pytest.mark.parametrize("dtype,C", [("f32", 32), ("f32", 80), ("f32", 4), ("f32", 36), ("f32", 128), ("f32", 260),
                                     ("bf16", 64), ("bf16", 128), ("bf16", 8), ("bf16", 40), ("bf16", 264)])
def test_channel_counts_general_pose(oracle, reduce, kernel, dtype, C):
    ref, _, _ = check_small(oracle, small(C, C=C, dtype=dtype), reduce, kernel)
    assert ref.count.sum() > 500


@pytest.mark.parametrize("dtype,C", [("f32", 3), ("f32", 1), ("f32", 7), ("bf16", 5), ("bf16", 12)])
def test_channel_counts_without_16_byte_rows(oracle, dtype, C):
    """With the scratch the torch wrapper lends: the tiled kernel on a zero-padded copy; the generic kernel when asked
    for; and the tiled kernel forced on the caller's own rows is refused on the host."""
    inp = small(40 + C, C=C, dtype=dtype)
    _, _, kname = check_small(oracle, inp, EQ1)
    assert kname.startswith("tiled") and kname.endswith("padded")
    _, _, kname = check_small(oracle, inp, EQ1, fb.KERNEL_PER_OUTPUT)
    assert kname.startswith("per_output") and kname.endswith("x1")
    w = inp.workload
    p = fb.make_params(16, fb.F32 if dtype == "f32" else fb.BF16, 16, w.B, w.N, C, w.feat_hw, w.img_hw, w.bev_range,
                       w.grid, 0, 16, kernel=fb.KERNEL_TILED)
    assert fb.flashbev_sampling_vt(p, None, check=False) == fb.UNSUPPORTED


@pytest.mark.parametrize("grid", [(1, 1, 1), (1, 37, 2), (37, 1, 3), (5, 3, 1), (33, 31, 7), (64, 64, 4)])
def test_ragged_and_tiny_grids(oracle, grid):
    for dtype, C in (("f32", 32), ("bf16", 128), ("f32", 80)):
        check_small(oracle, small(grid[0] * 100 + grid[1], C=C, dtype=dtype, grid=grid), EQ1)


@pytest.mark.parametrize("Z", [1, 2, 63, 64, 65, 130, 300])
def test_height_bin_counts_span_several_chunks(oracle, Z):
    inp = small(Z, B=1, C=32, grid=(9, 11, Z), z=(-4.0, 4.0))
    for reduce in (SUM, EQ1):
        check_small(oracle, inp, reduce, large_outputs=True)   # up to hundreds of samples per cell


@pytest.mark.parametrize("N", [1, 2, 7, 16, 33, 64])
def test_camera_counts(oracle, N):
    check_small(oracle, small(N, B=1, N=N, C=16, grid=(10, 9, 6)), EQ1)
    check_small(oracle, small(N, B=1, N=N, C=16, grid=(10, 9, 6)), MEAN)


def test_every_camera_sees_every_cell_many_heights(oracle):
    """All cameras overlap, so a sub-block collects far more records than the slots hold: its runs
    are taken in several rounds while the accumulators stay in registers."""
    w = wl.Workload("overlap", 77, 1, 8, 32, "f32", (24, 40), (192, 320), (12, 10, 96),
                    (8.0, 20.0, -5.0, 5.0, -2.0, 4.0), 0, general_pose=False, yaw_jitter_deg=0.0)
    inp = wl.make_inputs(w)
    inp.lidar2img[:] = inp.lidar2img[:, :1]                 # eight copies of the forward camera
    inp.lidar2img[0, :, 0, 3] += np.arange(8, dtype=np.float32) * 3.0   # shifted by a few pixels each
    for reduce in (SUM, MEAN, EQ1):           # ~770 samples per cell
        ref, _, _ = check_small(oracle, inp, reduce, large_outputs=True)
        assert ref.count.max() > 300
    for walk in (1, 3, 64):
        check_small(oracle, inp, EQ1, tune=(0, 0, walk, 0), large_outputs=True)
    for slots16 in (4, 8, 16):                 # few record slots: sub-blocks whose records take several rounds
        check_small(oracle, inp, SUM, tune=(0, 0, 0, slots16 << 20), large_outputs=True)


@pytest.mark.parametrize("tune", [(1, 8, 0, 0), (2, 4, 0, 0), (4, 2, 0, 0), (1, 4, 0, 0), (2, 2, 2, 0), (4, 1, 5, 0),
                                  (1, 32, 0, 0), (2, 16, 1, 0), (1, 3, 0, 0), (2, 5, 16, 0)])
def test_tuning_knobs_do_not_change_results(oracle, tune):
    check_small(oracle, small(5, C=32, dtype="f32"), EQ1, fb.KERNEL_TILED, tune)
    check_small(oracle, small(6, C=64, dtype="bf16"), SUM, fb.KERNEL_TILED, tune)


def test_no_camera_sees_anything(oracle):
    inp = small(9, B=1, C=32, general=False, rng_xy=4.0)
    inp.lidar2img[:, :, 2, :] = np.array([0.0, 0.0, 0.0, -1.0], np.float32)   # depth -1 m everywhere
    ref, out, _ = check_small(oracle, inp, EQ1)
    assert ref.count.sum() == 0 and np.all(out == 0.0)


def test_non_finite_matrix_entries_invalidate_samples_only(oracle):
    inp = small(10, B=1, C=32)
    inp.lidar2img[0, 1, 0, 2] = np.nan
    inp.lidar2img[0, 2, 2, 3] = np.inf
    inp.lidar2img[0, 3, 1, 1] = -np.inf
    for kernel in (fb.KERNEL_PER_OUTPUT, fb.KERNEL_TILED):
        check_small(oracle, inp, EQ1, kernel)


def test_zero_pitch_ring_rig_small(oracle):
    for dtype, C in (("f32", 32), ("bf16", 64)):
        check_small(oracle, small(11, C=C, dtype=dtype, general=False, grid=(40, 40, 12), rng_xy=30.0), SUM)


def test_steep_columns_and_single_texel_wide_maps(oracle):
    # a 1-texel-wide and a 1-texel-high map: every sample has out-of-range taps
    check_small(oracle, small(12, C=32, feat=(12, 1)), EQ1)
    check_small(oracle, small(13, C=32, feat=(1, 20)), EQ1)
    check_small(oracle, small(14, C=32, feat=(1, 1)), SUM)


def test_batch_elements_use_their_own_cameras_and_features(oracle):
    inp = small(15, B=3, C=32)
    w = inp.workload
    out, _, _ = parity.run_gpu(inp, EQ1)
    one = wl.Inputs(wl.Workload(**{**w.__dict__, "B": 1}), inp.features[2:3].copy(), None, inp.lidar2img[2:3].copy())
    out1, _, _ = parity.run_gpu(one, EQ1)
    assert np.array_equal(out[2:3], out1)


# ---------------------------------------------------------------- properties that hold at any size

def test_repeatable_bit_for_bit(bench_inputs):
    for name, reduce in (("representative", SUM), ("half_taller", EQ1)):
        inp = bench_inputs[name]
        a, _, _ = parity.run_gpu(inp, reduce)
        b, _, _ = parity.run_gpu(inp, reduce)
        assert np.array_equal(a, b)


@pytest.mark.parametrize("name", wl.CONFIG_ORDER)
def test_valid_sample_totals_without_jitter_match_the_independent_enumeration(oracle, name):
    """The kernel's own count output, and the oracle's, against totals counted by independent array code
    (tests/golden/zero_jitter_valid_totals.txt); samples within 1e-3 px of a border may fall either way."""
    import os
    rows = [l.split() for l in open(os.path.join(os.path.dirname(__file__), "golden", "zero_jitter_valid_totals.txt"))
            if l.strip() and not l.startswith("#")]
    cand, valid = {r[0]: (int(r[1]), int(r[2])) for r in rows}[name]
    base = wl.get(name)
    w = wl.get(name, yaw_jitter_deg=0.0, C=4 if base.dtype == "f32" else 8)
    inp = wl.make_inputs(w)
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, SUM)
    slack = int(ref.flagged.sum())
    assert w.candidates == cand and slack <= 1e-4 * cand
    assert abs(int(ref.count.sum()) - valid) <= slack
    _, cnt, kname = parity.run_gpu(inp, SUM, fb.KERNEL_TILED)
    assert abs(int(cnt.astype(np.int64).sum()) - valid) <= slack, kname


def test_both_kernels_agree_closely(bench_inputs):
    inp = bench_inputs["representative"]
    a, ca, _ = parity.run_gpu(inp, EQ1, fb.KERNEL_TILED)
    b, cb, _ = parity.run_gpu(inp, EQ1, fb.KERNEL_PER_OUTPUT)
    assert np.array_equal(ca, cb)
    assert np.abs(a - b).max() < 2e-5


def test_no_device_memory_is_allocated_by_the_call(bench_inputs):
    import torch
    inp = bench_inputs["representative"]
    w = inp.workload
    dev = torch.device("cuda:0")
    feats = torch.from_numpy(inp.features).to(dev)
    mats = torch.from_numpy(inp.lidar2img).to(dev)
    X, Y, Z = w.grid
    out = torch.empty((w.B, X, Y, w.C), dtype=torch.float32, device=dev)
    fb.sampling_vt(feats, mats, w.img_hw, w.bev_range, w.grid, SUM, out=out)   # warm up (module load)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    torch.cuda.reset_peak_memory_stats()
    alloc0 = torch.cuda.max_memory_allocated()
    fb.sampling_vt(feats, mats, w.img_hw, w.bev_range, w.grid, SUM, out=out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert torch.cuda.max_memory_allocated() == alloc0
    assert free1 == free0
    p = fb.make_params(feats.data_ptr(), fb.F32, mats.data_ptr(), w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range,
                       w.grid, SUM, out.data_ptr())
    assert fb.flashbev_workspace_bytes(p) == 0
    assert out.numel() * 4 == w.output_bytes


def test_host_buffer_entry_point(oracle, bench_inputs):
    import torch
    for name in ("tiny", "half_taller"):
        inp = bench_inputs[name]
        w = inp.workload
        X, Y, Z = w.grid
        if w.dtype == "bf16":
            hf = torch.from_numpy(inp.features_bf16.view(np.int16)).pin_memory()
            dt = fb.BF16
        else:
            hf = torch.from_numpy(inp.features).pin_memory()
            dt = fb.F32
        hm = torch.from_numpy(inp.lidar2img).pin_memory()
        hout = torch.full((w.B, X, Y, w.C), float("nan")).pin_memory()
        hcnt = torch.full((w.B, X, Y), -1, dtype=torch.int32).pin_memory()
        p = fb.make_params(hf.data_ptr(), dt, hm.data_ptr(), w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range, w.grid,
                           w.reduce, hout.data_ptr(), hcnt.data_ptr())
        need = fb.flashbev_host_staging_bytes(p)
        assert need >= w.unique_bytes
        staging = torch.empty(need, dtype=torch.uint8, device="cuda:0")
        assert fb.flashbev_sampling_vt_host(p, staging.data_ptr(), need - 1, None, check=False) == fb.TOO_SMALL
        s = torch.cuda.Stream()
        fb.flashbev_sampling_vt_host(p, staging.data_ptr(), need, s.cuda_stream)
        s.synchronize()
        parity.assert_parity(w, oracle_of(oracle, inp, w.reduce), hout.numpy(), hcnt.numpy(), "[host entry]")


def test_host_buffer_entry_point_with_planar_tensors(oracle, bench_inputs):
    """NCHW host tensors: with the whole staging area the channels-last copy is made there and the tiled kernel runs;
    with the area cut down to its compulsory part the generic kernel runs; same numbers either way."""
    import torch
    inp = bench_inputs["tiny"]
    w = inp.workload
    X, Y, Z = w.grid
    hf = torch.from_numpy(np.ascontiguousarray(inp.features.transpose(0, 1, 4, 2, 3))).pin_memory()
    hm = torch.from_numpy(inp.lidar2img).pin_memory()
    ref = oracle_of(oracle, inp, w.reduce)
    full = None
    for cut in (False, True):
        hout = torch.full((w.B, w.C, X, Y), float("nan")).pin_memory()
        p = fb.make_params(hf.data_ptr(), fb.F32, hm.data_ptr(), w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range, w.grid,
                           w.reduce, hout.data_ptr(), layout=fb.NCHW)
        need, ws = fb.flashbev_host_staging_bytes(p), fb.flashbev_workspace_bytes(p)
        assert ws == inp.features.nbytes and need >= w.unique_bytes + ws
        staging = torch.empty(need, dtype=torch.uint8, device="cuda:0")
        s = torch.cuda.Stream()
        fb.flashbev_sampling_vt_host(p, staging.data_ptr(), need - ws if cut else need, s.cuda_stream)
        s.synchronize()
        assert fb.flashbev_last_kernel_name() == ("per_output_nchw_f32" if cut else "tiled_f32_nchw")
        parity.assert_parity(w, ref, hout.permute(0, 2, 3, 1).numpy(), None, "[host entry, planar]")
        full = hout if full is None else full
    assert float((full - hout).abs().max()) <= 1e-5


def test_host_buffer_entry_point_with_ragged_channel_counts(oracle):
    """Host tensors with C = 30 fp32 (120-byte rows): the staging area has room for the padded copy, so the tiled kernel
    runs; cut down to its compulsory part the generic kernel runs."""
    import torch
    w = wl.get("tiny", C=30)
    inp = wl.make_inputs(w)
    X, Y, Z = w.grid
    hf = torch.from_numpy(inp.features).pin_memory()
    hm = torch.from_numpy(inp.lidar2img).pin_memory()
    ref = oracle_of(oracle, inp, w.reduce)
    for cut in (False, True):
        hout = torch.full((w.B, X, Y, w.C), float("nan")).pin_memory()
        hcnt = torch.full((w.B, X, Y), -1, dtype=torch.int32).pin_memory()
        p = fb.make_params(hf.data_ptr(), fb.F32, hm.data_ptr(), w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range, w.grid,
                           w.reduce, hout.data_ptr(), hcnt.data_ptr())
        need, ws = fb.flashbev_host_staging_bytes(p), fb.flashbev_workspace_bytes(p)
        assert ws == inp.features.nbytes // 30 * 32
        staging = torch.empty(need, dtype=torch.uint8, device="cuda:0")
        s = torch.cuda.Stream()
        fb.flashbev_sampling_vt_host(p, staging.data_ptr(), need - ws if cut else need, s.cuda_stream)
        s.synchronize()
        assert fb.flashbev_last_kernel_name() == ("per_output_f32x1" if cut else "tiled_f32_padded")
        parity.assert_parity(w, ref, hout.numpy(), hcnt.numpy(), "[host entry, ragged]")


def test_runs_on_a_caller_stream(oracle, bench_inputs):
    import torch
    inp = bench_inputs["tiny"]
    w = inp.workload
    dev = torch.device("cuda:0")
    feats = torch.from_numpy(inp.features).to(dev)
    mats = torch.from_numpy(inp.lidar2img).to(dev)
    s = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        out = fb.sampling_vt(feats, mats, w.img_hw, w.bev_range, w.grid, SUM)
    s.synchronize()
    assert fb.flashbev_last_launch_count() == 1
    parity.assert_parity(w, oracle_of(oracle, inp, SUM), out.cpu().numpy(), None)


def test_back_to_back_launches_keep_stream_order(bench_inputs):
    """The forward is launched with programmatic stream serialization (its thread blocks may be resident before the
    kernel in front of it has finished).  A second call that reads the first call's output as its feature map must see
    the finished output: same bits as with a synchronisation in between, over many rounds with changing inputs."""
    import torch
    inp = bench_inputs["tiny"]
    w = inp.workload
    dev = torch.device("cuda:0")
    X, Y, Z = w.grid
    mats = torch.from_numpy(inp.lidar2img).to(dev)
    w2 = wl.Workload("chained", 4242, 1, 1, w.C, "f32", (X, Y), (X * 8, Y * 8), (64, 64, 8),
                     (-20.0, 20.0, -20.0, 20.0, -3.0, 3.0), 0, general_pose=False, yaw_jitter_deg=0.0, fov_deg=100.0)
    mats2 = torch.from_numpy(wl.make_inputs(w2).lidar2img).to(dev)
    g = torch.Generator(device=dev).manual_seed(5)
    stream = torch.cuda.Stream(dev)
    for it in range(20):
        feats = torch.randn((w.B, w.N) + tuple(w.feat_hw) + (w.C,), generator=g, device=dev)
        mid = torch.zeros((1, X, Y, w.C), device=dev)
        outs = []
        for synced in (True, False):
            mid.zero_()
            out2 = torch.full((1, 64, 64, w.C), float("nan"), device=dev)
            torch.cuda.synchronize()
            with torch.cuda.stream(stream):
                fb.sampling_vt(feats, mats, w.img_hw, w.bev_range, w.grid, 0, out=mid, stream=stream.cuda_stream)
                if synced:
                    stream.synchronize()
                fb.sampling_vt(mid.view(1, 1, X, Y, w.C), mats2, w2.img_hw, w2.bev_range, w2.grid, 0, out=out2,
                               stream=stream.cuda_stream)
            stream.synchronize()
            outs.append(out2)
        assert torch.equal(outs[0], outs[1]), it
        assert float(outs[0].abs().max()) > 0.0
