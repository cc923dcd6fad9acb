"""GPU parity of the fused spatial cross-attention (FlashSCA) against its fp64 oracle.

Gates as for the fp32 Sampling-VT path: max-abs <= 1e-4 and relative L2 <= 1e-6 over the queries
without a reference point within 1e-3 (image px / m) of a validity border; hit counts bit-exact.
"""
import numpy as np
import pytest

from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import workloads as wl
from tests.test_oracle_sca_pins import make_case

pytestmark = pytest.mark.gpu


def run_gpu(c, bf16=False, chunk_records=0):
    import torch
    dev = torch.device("cuda:0")
    t = {k: torch.from_numpy(np.ascontiguousarray(c[k])).to(dev) for k in ("value", "lidar2img", "offsets", "weights")}
    if bf16:  # c["value"] already holds bf16-representable numbers; ship their 16-bit patterns
        bits = wl.round_to_bf16(c["value"])[1]
        t["value"] = torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)
    B = c["value"].shape[0]
    Q = c["grid"][0] * c["grid"][1]
    D = c["value"].shape[3] * c["value"].shape[4]
    out = torch.full((B, Q, D), float("nan"), dtype=torch.float32, device=dev)
    hits = torch.full((B, Q), -1, dtype=torch.int32, device=dev)
    fb.sca(t["value"], c["level_hw"], t["lidar2img"], t["offsets"], t["weights"], c["img_hw"], c["bev_range"], c["grid"],
           out=out, hits=hits, chunk_records=chunk_records)
    assert fb.flashbev_last_kernel_name() == ("sca_bf16" if bf16 else "sca_f32") and fb.flashbev_last_launch_count() == 1
    torch.cuda.synchronize()
    return out.cpu().numpy(), hits.cpu().numpy()


def check(oracle, c, label="", bf16=False, chunk_records=0):
    if bf16:  # the oracle sees the same bf16-rounded values the kernel reads
        c = dict(c, value=wl.round_to_bf16(c["value"])[0])
    ref, rhits, flagged = oracle.sca(**c)
    out, hits = run_gpu(c, bf16, chunk_records)
    assert np.all(np.isfinite(out)), label
    keep = flagged == 0
    assert np.array_equal(hits[keep], rhits[keep]), label
    err = np.abs(out.astype(np.float64) - ref)[keep]
    rel = np.sqrt((err ** 2).sum() / max(1e-300, (ref[keep] ** 2).sum()))
    msg = f"{label}: max_abs={err.max():.2e} rel_l2={rel:.2e} hit_queries={int((rhits > 0).sum())} flagged={int((~keep).sum())}"
    assert err.max() <= 1e-4 and rel <= 1e-6, msg
    assert np.all(out[rhits == 0] == 0.0), msg
    return msg


@pytest.mark.parametrize("general", [False, True])
@pytest.mark.parametrize("heads,Dh", [(2, 4), (8, 32), (4, 8), (1, 128), (3, 12), (16, 16)])
def test_head_shapes(oracle, general, heads, Dh):
    c = make_case(heads * 100 + Dh, B=2, N=6, heads=heads, Dh=Dh, levels=((12, 18), (6, 9), (3, 5)), P=4,
                  grid=(9, 7, 2), general=general, rng_xy=10.0)
    check(oracle, c, f"heads={heads} Dh={Dh}")


@pytest.mark.parametrize("P,Zref,L", [(8, 4, 4), (16, 4, 4), (3, 2, 1), (5, 4, 2), (1, 1, 1), (32, 4, 4)])
def test_point_and_level_counts(oracle, P, Zref, L):
    levels = ((16, 24), (8, 12), (4, 6), (2, 3))[:L]
    c = make_case(P * 10 + Zref, N=6, heads=4, Dh=8, levels=levels, P=P, grid=(8, 9, Zref), rng_xy=12.0)
    check(oracle, c, f"P={P} Zref={Zref} L={L}")


@pytest.mark.parametrize("general", [False, True])
@pytest.mark.parametrize("heads,Dh", [(8, 32), (4, 8), (2, 16), (1, 128), (3, 24), (16, 16), (16, 8), (40, 8)])
def test_bf16_values(oracle, general, heads, Dh):
    """bfloat16 value maps, fp32 accumulation: the only error left is the summation order."""
    c = make_case(heads * 100 + Dh + 7, B=2, N=6, heads=heads, Dh=Dh, levels=((12, 18), (6, 9), (3, 5)), P=4,
                  grid=(9, 7, 2), general=general, rng_xy=10.0)
    check(oracle, c, f"bf16 heads={heads} Dh={Dh}", bf16=True)


def test_bf16_unsupported_shapes():
    import torch
    c = make_case(5, N=2, heads=2, Dh=4, grid=(4, 4, 2))
    dev = torch.device("cuda:0")
    t = {k: torch.from_numpy(np.ascontiguousarray(c[k])).to(dev) for k in ("value", "lidar2img", "offsets", "weights")}
    with pytest.raises(fb.FlashBevError) as e:   # head_dim 4 is half a 16-byte vector of bfloat16
        fb.sca(t["value"].to(torch.bfloat16), c["level_hw"], t["lidar2img"], t["offsets"], t["weights"], c["img_hw"],
               c["bev_range"], c["grid"])
    assert e.value.status == fb.UNSUPPORTED


@pytest.mark.parametrize("P,Zref,records", [(5, 4, 16), (7, 3, 24), (12, 4, 64), (9, 2, 8), (33, 4, 0)])
def test_ragged_point_chunks(oracle, P, Zref, records):
    """Points are processed in chunks of `records / (heads * L)`: last chunks that are shorter, chunks that
    do not start on a multiple of Zref, one point per chunk, and more than 32 points."""
    c = make_case(P * 100 + Zref, N=6, heads=4, Dh=8, levels=((16, 24), (8, 12)), P=P, grid=(8, 9, Zref), rng_xy=12.0)
    check(oracle, c, f"P={P} Zref={Zref} records={records}", chunk_records=records)


def test_non_finite_and_unseen(oracle):
    c = make_case(3, N=4, heads=2, Dh=4, grid=(6, 6, 2))
    c["lidar2img"][0, 1, 0, 2] = np.nan
    c["lidar2img"][0, 2, 0, 3] = np.inf
    check(oracle, c, "non-finite matrices")
    c = make_case(4, N=3, heads=2, Dh=4, grid=(6, 6, 2))
    c["lidar2img"][:, :, 2, :] = np.array([0, 0, 0, -1.0], np.float32)
    ref, rhits, _ = oracle.sca(**c)
    out, hits = run_gpu(c)
    assert rhits.sum() == 0 and np.all(out == 0.0) and np.all(hits == 0)


def test_bevformer_base_shape(oracle):
    """N = 6, C = 256, 8 heads, 200 x 200 queries, Zref = 4, L = 4, P = 8 (the paper's Table 7 setting), ring rig."""
    c = wl.make_sca_inputs(P=8)
    print("\n" + check(oracle, c, "bevformer-base P=8"))
    print(check(oracle, c, "bevformer-base P=8, bf16 values", bf16=True))
