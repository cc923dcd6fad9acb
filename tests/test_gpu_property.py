"""Property test: random small rigs, shapes, dtypes and reduce modes -- CUDA path vs the fp64 oracle."""
import numpy as np
import pytest
from hypothesis import HealthCheck, given, settings, strategies as st

from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu


@st.composite
def cases(draw):
    dtype = draw(st.sampled_from(["f32", "bf16"]))
    vec = 4 if dtype == "f32" else 8
    C = vec * draw(st.sampled_from([1, 2, 3, 5, 8, 9, 12, 16, 20, 23, 24, 27, 32, 40, 66])) if draw(st.booleans()) else draw(st.integers(1, 40))
    return dict(
        seed=draw(st.integers(0, 10_000)), dtype=dtype, C=C,
        B=draw(st.integers(1, 2)), N=draw(st.integers(1, 7)),
        feat=(draw(st.integers(1, 14)), draw(st.integers(1, 18))),
        grid=(draw(st.integers(1, 13)), draw(st.integers(1, 13)), draw(st.integers(1, 40))),
        general=draw(st.booleans()), rng_xy=draw(st.sampled_from([3.0, 10.0, 40.0])),
        reduce=draw(st.sampled_from([0, 1, 2])), kernel=draw(st.sampled_from([fb.KERNEL_AUTO, fb.KERNEL_PER_OUTPUT])),
        walk=draw(st.sampled_from([0, 1, 3, 8])))


@settings(max_examples=200, deadline=None, derandomize=True,
          suppress_health_check=[HealthCheck.function_scoped_fixture, HealthCheck.too_slow])
@given(case=cases())
def test_random_small_problems_match_the_oracle(oracle, case):
    w = wl.Workload("prop", 5000 + case["seed"], case["B"], case["N"], case["C"], case["dtype"], case["feat"],
                    (case["feat"][0] * 8, case["feat"][1] * 8), case["grid"],
                    (-case["rng_xy"], case["rng_xy"], -case["rng_xy"], case["rng_xy"], -3.0, 2.5), case["reduce"],
                    general_pose=case["general"], yaw_jitter_deg=5.0)
    inp = wl.make_inputs(w)
    ref = oracle.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, case["reduce"])
    out, cnt, kname = parity.run_gpu(inp, case["reduce"], case["kernel"], (0, 0, case["walk"], 0))
    parity.assert_parity(w, ref, out, cnt, f"[{kname} {case}]", check_fraction=False, large_outputs=True)  # up to ~200 samples per cell
