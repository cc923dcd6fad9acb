"""Host-only checks of the C ABI: the library loads, exports what the header declares, the
ctypes mirror matches the C struct, and argument validation happens before any CUDA call."""
import ctypes
import os
import re
import subprocess
import sys

import pytest

from paper_2607_10071_b200 import binding as fb
from paper_2607_10071_b200 import build as fbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "flashbev.h")


@pytest.fixture(scope="module", autouse=True)
def built():
    fbuild.build()


def declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(flashbev_[a-z_0-9]+)\s*\(", src)))


def test_every_declared_symbol_is_exported():
    names = declared_functions()
    assert "flashbev_sampling_vt" in names and len(names) >= 8
    lib = ctypes.CDLL(fb.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in flashbev.h but not exported"


def test_binding_exposes_the_same_names():
    for n in declared_functions():
        assert hasattr(fb, n) or n in ("flashbev_status_string", "flashbev_version"), n
    assert fb.version() == 100
    assert fb.status_string(fb.OK) == "ok" and "unknown" in fb.status_string(99)


@pytest.mark.parametrize("cname,mirror", [("flashbev_vt_params", "VtParams"),
                                          ("flashbev_vt_backward_params", "VtBackwardParams"),
                                          ("flashbev_sca_params", "ScaParams"),
                                          ("flashbev_vt_multires_params", "VtMultiresParams")])
def test_ctypes_struct_matches_the_c_struct(tmp_path, cname, mirror):
    prog = tmp_path / "layout.c"
    cls = getattr(fb, mirror)
    fields = [f[0] for f in cls._fields_]
    body = "\n".join(f'printf("{f} %zu\\n", offsetof({cname}, {f}));' for f in fields)
    prog.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "flashbev.h"\nint main(void){\n'
                    + body + f'\nprintf("sizeof %zu\\n", sizeof({cname}));\nreturn 0;}}\n')
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(prog), "-o", str(exe)],
                   check=True)
    got = dict(l.split() for l in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines())
    for f in fields:
        assert int(got[f]) == getattr(cls, f).offset, f
    assert int(got["sizeof"]) == ctypes.sizeof(cls)


def good_params(**over):
    kw = dict(features_ptr=4096, feat_dtype=fb.F32, lidar2img_ptr=8192, B=1, N=6, C=32, feat_hw=(16, 44),
              img_hw=(128, 352), bev_range=(-25, 25, -25, 25, -3, 1), grid=(50, 50, 4), reduce=0, out_ptr=16384)
    kw.update(over)
    return fb.make_params(**kw)


@pytest.mark.parametrize("over,status", [
    (dict(features_ptr=None), fb.INVALID_ARG),
    (dict(lidar2img_ptr=None), fb.INVALID_ARG),
    (dict(out_ptr=None), fb.INVALID_ARG),
    (dict(B=0), fb.INVALID_ARG), (dict(N=-1), fb.INVALID_ARG), (dict(C=0), fb.INVALID_ARG),
    (dict(feat_hw=(0, 44)), fb.INVALID_ARG), (dict(img_hw=(128, 0)), fb.INVALID_ARG),
    (dict(grid=(50, 0, 4)), fb.INVALID_ARG), (dict(grid=(50, 50, 0)), fb.INVALID_ARG),
    (dict(bev_range=(25, -25, -25, 25, -3, 1)), fb.INVALID_ARG),
    (dict(bev_range=(-25, 25, -25, 25, 1, 1)), fb.INVALID_ARG),
    (dict(bev_range=(-25, float("nan"), -25, 25, -3, 1)), fb.INVALID_ARG),
    (dict(bev_range=(-25, float("inf"), -25, 25, -3, 1)), fb.INVALID_ARG),
    (dict(reduce=3), fb.INVALID_ARG), (dict(feat_dtype=2), fb.INVALID_ARG), (dict(kernel=9), fb.INVALID_ARG),
    (dict(layout=7), fb.INVALID_ARG),
    (dict(layout=fb.NCHW, kernel=fb.KERNEL_TILED), fb.UNSUPPORTED),  # planar tensors on the tiled kernel need a workspace
    (dict(out_dtype=fb.BF16, out_ptr=16385), fb.MISALIGNED),
    (dict(N=65), fb.UNSUPPORTED),
    (dict(B=1 << 20, grid=(1 << 10, 1 << 10, 4)), fb.UNSUPPORTED),
    (dict(features_ptr=4098), fb.MISALIGNED),
    (dict(out_ptr=16386), fb.MISALIGNED),
    (dict(lidar2img_ptr=8194), fb.MISALIGNED),
    (dict(features_ptr=4100, kernel=fb.KERNEL_TILED), fb.UNSUPPORTED),     # tiled kernel needs 16-byte alignment
    (dict(C=30, kernel=fb.KERNEL_TILED), fb.UNSUPPORTED),
])
def test_invalid_arguments_are_rejected_on_the_host(over, status):
    """None of these reach a CUDA call, so they run (and must not crash) on a machine without a GPU."""
    assert fb.flashbev_sampling_vt(good_params(**over), None, check=False) == status


def test_short_struct_and_null_params_are_rejected():
    p = good_params()
    p.struct_size = 8
    assert fb.flashbev_sampling_vt(p, None, check=False) == fb.INVALID_ARG
    assert fb.lib().flashbev_sampling_vt(None, None) == fb.INVALID_ARG
    assert fb.flashbev_host_staging_bytes(p) == 0
    with pytest.raises(fb.FlashBevError):
        fb.flashbev_sampling_vt(p, None)


def test_host_entry_validates_staging():
    p = good_params()
    need = fb.flashbev_host_staging_bytes(p)
    assert need >= 1 * 6 * 16 * 44 * 32 * 4 + 6 * 64 + 50 * 50 * 32 * 4
    assert fb.flashbev_sampling_vt_host(p, None, need, None, check=False) == fb.INVALID_ARG
    assert fb.flashbev_sampling_vt_host(p, 4096 + 8, need, None, check=False) == fb.MISALIGNED
    assert fb.flashbev_sampling_vt_host(p, 4096, need - 1, None, check=False) == fb.TOO_SMALL
    assert fb.flashbev_workspace_bytes(p) == 0


def test_workspace_is_asked_for_planar_tensors_only():
    """Channels-last tensors need no scratch; NCHW tensors may lend the size of a channels-last copy of the features
    (only when the channel rows are whole 16-byte vectors: other shapes take the generic kernel anyway)."""
    assert fb.flashbev_workspace_bytes(good_params()) == 0
    assert fb.flashbev_workspace_bytes(good_params(layout=fb.NCHW)) == 1 * 6 * 16 * 44 * 32 * 4
    assert fb.flashbev_workspace_bytes(good_params(layout=fb.NCHW, C=30)) == 0
    # channels-last rows that are not whole 16-byte vectors: a copy with the rows padded to whole vectors
    assert fb.flashbev_workspace_bytes(good_params(C=30)) == 1 * 6 * 16 * 44 * 32 * 4
    assert fb.flashbev_workspace_bytes(good_params(C=33, feat_dtype=fb.BF16)) == 1 * 6 * 16 * 44 * 40 * 2
    # a workspace that is too small or misaligned is not used: forcing the tiled kernel is refused on the host
    for ws, nbytes in ((8192, 100), (8200, 1 << 30)):
        p = good_params(layout=fb.NCHW, kernel=fb.KERNEL_TILED)
        p.workspace, p.workspace_bytes = ws, nbytes
        assert fb.flashbev_sampling_vt(p, None, check=False) == fb.UNSUPPORTED


def test_multires_arguments_are_validated_on_the_host():
    """Level count, null levels and map sizes are checked before any CUDA call (fake, aligned addresses)."""
    base = good_params()
    hw = [(16, 44), (8, 22)]
    ptrs = [4096, 8192]
    assert fb.flashbev_sampling_vt_multires(base, [], [], None, check=False) == fb.INVALID_ARG
    assert fb.flashbev_sampling_vt_multires(base, ptrs * 5, hw * 5, None, check=False) == fb.INVALID_ARG
    assert fb.flashbev_sampling_vt_multires(base, [4096, 0], hw, None, check=False) == fb.INVALID_ARG
    assert fb.flashbev_sampling_vt_multires(base, ptrs, [(16, 44), (0, 22)], None, check=False) == fb.INVALID_ARG
    assert fb.flashbev_sampling_vt_multires(base, [4096, 8192 + 2], hw, None, check=False) == fb.MISALIGNED
    assert fb.flashbev_sampling_vt_multires(good_params(out_dtype=fb.BF16), ptrs, hw, None, check=False) == fb.UNSUPPORTED
    assert fb.lib().flashbev_sampling_vt_multires(None, None) == fb.INVALID_ARG


def test_sca_arguments_are_validated_on_the_host():
    import numpy as np
    lv = np.array([[4, 6], [2, 3]], np.int32)

    def params(**over):
        p = fb.ScaParams()
        p.struct_size = ctypes.sizeof(fb.ScaParams)
        p.value, p.value_dtype, p.level_hw = 4096, fb.F32, lv.ctypes.data
        p.lidar2img, p.offsets, p.weights, p.out = 8192, 12288, 16384, 20480
        p.B, p.N, p.heads, p.head_dim, p.L, p.P = 1, 2, 2, 8, 2, 4
        p.img_h, p.img_w = 32, 48
        p.x_min, p.x_max, p.y_min, p.y_max, p.z_min, p.z_max = -1, 1, -1, 1, -1, 1
        p.X, p.Y, p.Zref = 3, 3, 2
        for k, v in over.items():
            setattr(p, k, v)
        return p

    for over, status in [(dict(value=None), fb.INVALID_ARG), (dict(heads=0), fb.INVALID_ARG), (dict(P=0), fb.INVALID_ARG),
                         (dict(x_max=-1.0), fb.INVALID_ARG), (dict(value_dtype=7), fb.INVALID_ARG),
                         (dict(chunk_records=-1), fb.INVALID_ARG), (dict(head_dim=6), fb.UNSUPPORTED),
                         (dict(head_dim=132), fb.UNSUPPORTED), (dict(Zref=33), fb.UNSUPPORTED),
                         (dict(value_dtype=fb.BF16, head_dim=4), fb.UNSUPPORTED), (dict(heads=200), fb.UNSUPPORTED),
                         (dict(value=4096 + 4), fb.MISALIGNED), (dict(offsets=12288 + 4), fb.MISALIGNED),
                         (dict(struct_size=8), fb.INVALID_ARG)]:
        assert fb.flashbev_sca(params(**over), None, check=False) == status, over
    assert fb.lib().flashbev_sca(None, None) == fb.INVALID_ARG


def test_product_path_never_imports_the_oracle():
    code = ("import sys; import paper_2607_10071_b200.binding, paper_2607_10071_b200.workloads, "
            "paper_2607_10071_b200.build; "
            "assert not any(m == 'oracle' or m.startswith('oracle.') for m in sys.modules), 'oracle imported'")
    subprocess.run([sys.executable, "-c", code], check=True, cwd=ROOT)
    pat = re.compile(r"^\s*(from|import)\s+oracle\b|flashbev_oracle|oracle/", re.M)
    for fn in ("binding.py", "workloads.py", "build.py", "__init__.py", os.path.join("csrc", "flashbev.cu")):
        assert not pat.search(open(os.path.join(ROOT, "paper_2607_10071_b200", fn)).read()), fn
    assert not pat.search(open(HEADER).read())
