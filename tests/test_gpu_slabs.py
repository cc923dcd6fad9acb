"""Sharding one frame: an X-slab of the BEV grid is an ordinary smaller problem (own x-range and X, output
pointer moved to the slab's first row), so ranks that replicate the features need no exchange.  Two slabs
computed separately must reproduce the single call."""
import numpy as np
import pytest

from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,cut", [("representative", 96), ("tiny", 17), ("long_range", 203)])
def test_two_x_slabs_reproduce_the_whole_frame(oracle, name, cut):
    import torch
    w = wl.get(name)
    assert w.B == 1
    inp = wl.make_inputs(w)
    dev = torch.device("cuda:0")
    if w.dtype == "bf16":
        f = torch.from_numpy(inp.features_bf16.view(np.int16)).to(dev).view(torch.bfloat16)
    else:
        f = torch.from_numpy(inp.features).to(dev)
    m = torch.from_numpy(inp.lidar2img).to(dev)
    X, Y, Z = w.grid
    x_min, x_max = w.bev_range[:2]
    dx = (x_max - x_min) / X
    whole = torch.empty((1, X, Y, w.C), dtype=torch.float32, device=dev)
    cnt_whole = torch.empty((1, X, Y), dtype=torch.int32, device=dev)
    fb.sampling_vt(f, m, w.img_hw, w.bev_range, w.grid, w.reduce, out=whole, valid_count=cnt_whole)
    parts = torch.full_like(whole, float("nan"))
    cnt_parts = torch.full_like(cnt_whole, -1)
    for x0, x1 in ((0, cut), (cut, X)):                      # what rank 0 and rank 1 of two would compute
        rng = (x_min + x0 * dx, x_min + x1 * dx) + tuple(w.bev_range[2:])
        fb.sampling_vt(f, m, w.img_hw, rng, (x1 - x0, Y, Z), w.reduce, out=parts[:, x0:x1], valid_count=cnt_parts[:, x0:x1])
    torch.cuda.synchronize()
    # the slab's cell centres are recomputed from its own x_min: equal up to fp64 rounding, so border samples may flip
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, w.reduce)
    keep = torch.from_numpy(ref.flagged == 0).to(dev)
    assert torch.equal(cnt_parts[keep], cnt_whole[keep])
    diff = (parts - whole).abs()[keep]
    assert float(diff.max()) <= 1e-5, float(diff.max())
