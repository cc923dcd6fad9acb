"""The allocation-free host entry point (collected last on purpose: see the file name).

``flashbev_sampling_vt_host_static`` serves callers that cannot hand the library a device buffer
and may not allocate one -- a plugin without workspace, a loop with a frozen memory budget, code
that must not trigger the device-wide synchronisation of cudaMalloc/cudaFree.  Its staging area
is a fixed array inside the library.  The test calls it through the C ABI twice in a row (the
second call finds the first call's data in the shared array) and requires the same output as the
existing caller-staged entry point, which the parity tests check against the oracle.
"""
import numpy as np
import pytest

from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _host_params(w, inp, out, cnt):
    import torch
    if w.dtype == "bf16":
        hf = torch.from_numpy(inp.features_bf16.view(np.int16)).pin_memory()
        dt = fb.BF16
    else:
        hf = torch.from_numpy(inp.features).pin_memory()
        dt = fb.F32
    hm = torch.from_numpy(inp.lidar2img).pin_memory()
    p = fb.make_params(hf.data_ptr(), dt, hm.data_ptr(), w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range, w.grid,
                       w.reduce, out.data_ptr(), cnt.data_ptr())
    return p, (hf, hm)


def test_static_staging_entry_matches_the_caller_staged_one_twice_in_a_row():
    import torch
    stream = torch.cuda.Stream()
    for name, frame in (("representative", 0), ("tiny", 1)):      # second call: other shape, other data
        w = wl.get(name)
        inp = wl.make_inputs(w, stream=frame)
        X, Y, Z = w.grid
        # existing entry point: caller-owned staging buffer
        ref_out = torch.full((w.B, X, Y, w.C), float("nan")).pin_memory()
        ref_cnt = torch.full((w.B, X, Y), -1, dtype=torch.int32).pin_memory()
        p_ref, keep_ref = _host_params(w, inp, ref_out, ref_cnt)
        need = fb.flashbev_host_staging_bytes(p_ref)
        assert 0 < need <= fb.STATIC_STAGING_BYTES
        staging = torch.empty(need, dtype=torch.uint8, device="cuda:0")
        fb.flashbev_sampling_vt_host(p_ref, staging.data_ptr(), need, stream.cuda_stream)
        stream.synchronize()
        # new entry point: no buffer from the caller, nothing allocated
        for attempt in range(2):
            out = torch.full((w.B, X, Y, w.C), float("nan")).pin_memory()
            cnt = torch.full((w.B, X, Y), -1, dtype=torch.int32).pin_memory()
            p, keep = _host_params(w, inp, out, cnt)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            fb.flashbev_sampling_vt_host_static(p, stream.cuda_stream)
            stream.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
            assert np.all(np.isfinite(out.numpy())), f"{name} call {attempt}: unwritten output"
            assert np.array_equal(cnt.numpy(), ref_cnt.numpy()), f"{name} call {attempt}: valid counts differ"
            # same kernel, same inputs, fixed summation order: the two entry points agree bit for bit
            assert np.array_equal(out.numpy(), ref_out.numpy()), f"{name} call {attempt}: outputs differ"


def test_static_staging_entry_refuses_problems_beyond_its_limit_and_bad_arguments():
    w = wl.get("long_range")                       # needs ~99 MB of staging: beyond the 32 MiB array
    p = fb.make_params(4096, fb.BF16, 4096, w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range, w.grid, w.reduce, 4096)
    assert fb.flashbev_host_staging_bytes(p) > fb.STATIC_STAGING_BYTES
    assert fb.flashbev_sampling_vt_host_static(p, None, check=False) == fb.EXCEEDS_STATIC_STAGING
    assert "built-in staging" in fb.status_string(fb.EXCEEDS_STATIC_STAGING)
    p.Z = 0
    assert fb.flashbev_sampling_vt_host_static(p, None, check=False) == fb.INVALID_ARG
