"""The PyTorch tensorised baseline (Algorithm 1 on the GPU) agrees with the fused kernel.

grid_sample interpolates in float32 with float32 grid coordinates, so the baseline itself is only
accurate to ~1e-4 (the paper reports 2.9e-4 between its two implementations, Table 2); the fused kernel is
held to the fp64 oracle elsewhere.
"""
import numpy as np
import pytest

from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,reduce", [("tiny", 0), ("tiny", 2), ("representative", 0), ("representative", 1)])
def test_fused_kernel_matches_the_tensorized_baseline(name, reduce):
    import torch
    from paper_2607_10071_b200 import tensorized_baseline as tb
    w = wl.get(name)
    inp = wl.make_inputs(w)
    dev = torch.device("cuda:0")
    feats = torch.from_numpy(inp.features).to(dev)
    mats = torch.from_numpy(inp.lidar2img).to(dev)
    fused = fb.sampling_vt(feats, mats, w.img_hw, w.bev_range, w.grid, reduce)
    base = tb.sampling_vt_tensorized(feats, mats, w.img_hw, w.bev_range, w.grid, reduce)
    err = (fused - base).abs()
    # a handful of border samples may be classified differently by the float32 grid of grid_sample
    assert float((err > 1e-3).float().mean()) < 1e-3
    assert float(err.median()) < 1e-5
