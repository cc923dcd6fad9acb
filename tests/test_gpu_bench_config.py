"""The launch configuration the benchmark times (several resident frames, one launch per frame, replayed as a
CUDA graph on a side stream) must produce what a direct call produces, and frame 0 must match the oracle."""
import numpy as np
import pytest

import bench
from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["representative", "half_taller", "long_range"])
def test_graph_replay_of_a_benchmark_step(oracle, name):
    import torch
    w = wl.get(name)
    dev = torch.device("cuda:0")
    df = bench.DeviceFrames(w, 3, dev, 0)
    stream = torch.cuda.Stream(dev)
    with torch.cuda.stream(stream):
        assert df.launch_all(stream.cuda_stream) == 3      # module load outside the capture, as in the bench
        torch.cuda.synchronize()
        direct = [o.clone() for o in df.outs]
        for o in df.outs:
            o.fill_(float("nan"))
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            df.launch_all(torch.cuda.current_stream().cuda_stream)
        for o in df.outs:                                    # capture does not execute
            o.fill_(float("nan"))
        graph.replay()
        graph.replay()
        torch.cuda.synchronize()
    for a, b in zip(direct, df.outs):
        assert torch.equal(a, b)
    inp = wl.make_inputs(w)                                  # frame 0 of rank 0 is the seeded base frame
    feats = inp.features
    if w.dtype == "bf16":                                    # the bench converts on the device: same rounding
        assert np.array_equal(df.feats[0].view(torch.int16).cpu().numpy().view(np.uint16), inp.features_bf16)
    ref = oracle.sampling_vt(feats, inp.lidar2img, w.img_hw, w.bev_range, w.grid, w.reduce)
    parity.assert_parity(w, ref, df.outs[0].cpu().numpy(), None, f"[bench frame 0 {name}]")
