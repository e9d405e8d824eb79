"""CPU-only checks of the boundary: the C-ABI library builds, loads and exports every symbol the
headers declare; entry points that need no device behave; workload and sharding host logic."""
import ctypes
import glob
import os
import re

import numpy as np
import pytest

from paper_2304_11267_b200 import binding as bd
from paper_2304_11267_b200 import build as libbuild
from paper_2304_11267_b200 import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    libbuild.build()
    return bd.load()


def declared_functions():
    names = []
    for header in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))):
        text = open(header).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(sd_(?:attn|geglu|groupnorm|winograd)_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_headers_declare_the_expected_entry_points():
    names = declared_functions()
    for must in ("sd_attn_create", "sd_attn_forward", "sd_attn_destroy"):
        assert must in names
    assert set(names) == set(bd.EXPORTS)


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), "libsd_attn.so does not export %s" % name


def test_entry_points_that_need_no_device(lib):
    assert bd.sd_attn_destroy(None) == bd.OK
    assert bd.status_string(bd.OK) == "ok"
    for code in range(1, 8):
        assert bd.status_string(code) not in ("ok", "unknown status")
    assert bd.status_string(99) == "unknown status"
    # null handle: rejected before anything touches a device
    assert bd.sd_attn_forward(None, 16, 16, 16, 16, 1, 1, 1, 1, 8, 1.0, bd.F16) == bd.ERR_INVALID_VALUE
    assert bd.sd_attn_set_mode(None, bd.MODE_FUSED) == bd.ERR_INVALID_VALUE
    assert bd.sd_attn_last_mode(None) == bd.MODE_AUTO
    assert bd.sd_attn_launch_count(None) == 0


def test_workspace_and_staging_sizes(lib):
    B, H, Nq, Nk, d = 2, 8, 4096, 4096, 40
    rows = B * H * Nq
    need = bd.sd_attn_workspace_bytes(bd.MODE_TWOPASS, B, H, Nq, Nk, d, bd.F16)
    assert need == rows * Nk * 4 + rows * 8                      # A (already 256-aligned) + [L,S]
    assert bd.sd_attn_workspace_bytes(bd.MODE_FUSED, B, H, Nq, Nk, d, bd.F16) == 0
    assert bd.sd_attn_workspace_bytes(bd.MODE_TWOPASS, 1, 1, 3, 77, 40, bd.F16) == 1024 + 24
    st = bd.sd_attn_host_staging_bytes(2, 8, 4096, 77, 40, bd.F16)
    qb = 2 * 8 * 4096 * 40 * 2
    kb = (2 * 8 * 77 * 40 * 2 + 255) // 256 * 256
    assert st == 2 * qb + 2 * kb
    assert bd.sd_attn_host_staging_bytes(0, 8, 4096, 77, 40, bd.F16) == 0


def test_newer_entry_points_reject_bad_arguments_before_touching_a_device(lib):
    """Argument checks come before any CUDA call, so they answer on a machine without a GPU."""
    assert bd.sd_attn_set_layout(None, bd.LAYOUT_BNHD) == bd.ERR_INVALID_VALUE
    assert lib.sd_attn_forward_batch(None, None, 0, bd.F16, None) == bd.ERR_INVALID_VALUE
    # the Winograd convolution: sizes are host arithmetic
    assert bd.sd_winograd_filter_elems(320, 320) == 36 * 320 * 320
    assert bd.sd_winograd_filter_elems(0, 320) == 0
    T = 2 * 16 * 16                                                  # 64 x 64 image, batch 2: 4 x 4 output tiles
    assert bd.sd_winograd_workspace_bytes(2, 64, 64, 320, 320) == 36 * T * 320 * 2 + 36 * T * 320 * 4
    r256 = lambda n: (n + 255) // 256 * 256                        # each plane starts 256-byte aligned
    assert bd.sd_winograd_workspace_bytes(1, 5, 9, 8, 16) == r256(36 * 6 * 8 * 2) + r256(36 * 6 * 16 * 4)   # ragged: 2 x 3 tiles
    assert bd.sd_winograd_workspace_bytes(1, 1, 1, 8, 8) == r256(36 * 8 * 2) + r256(36 * 8 * 4)
    assert bd.sd_winograd_workspace_bytes(1, 0, 8, 8, 8) == 0
    f = bd.sd_winograd_conv3x3_forward
    assert f(256, 256, 0, 256, 256, 1 << 30, 1, 8, 8, 0, 16, 0) == bd.ERR_INVALID_VALUE     # C = 0
    assert f(256, 256, 0, 256, 256, 1 << 30, 1, 8, 8, 12, 16, 0) == bd.ERR_UNSUPPORTED      # C % 8 != 0
    assert f(256, 256, 0, 256, 256, 1 << 30, 0, 8, 8, 16, 16, 0) == bd.OK                   # N = 0: nothing to do
    assert f(0, 256, 0, 256, 256, 1 << 30, 1, 8, 8, 16, 16, 0) == bd.ERR_INVALID_VALUE      # null x
    assert f(264, 256, 0, 256, 256, 1 << 30, 1, 8, 8, 16, 16, 0) == bd.ERR_ALIGNMENT
    assert f(256, 256, 0, 256, 256, 100, 1, 8, 8, 16, 16, 0) == bd.ERR_WORKSPACE            # scratch too small
    assert f(256, 256, 0, 256, 384, 1 << 30, 1, 8, 8, 16, 16, 0) == bd.ERR_WORKSPACE        # scratch not 256-aligned
    assert bd.sd_winograd_transform_filter(0, 256, 16, 16, 0) == bd.ERR_INVALID_VALUE
    assert bd.sd_winograd_transform_filter(256, 256, 12, 16, 0) == bd.ERR_UNSUPPORTED
    # the element-wise and normalisation steps
    assert bd.load().sd_geglu_forward(None, None, 4, 8, bd.F16, None) == bd.ERR_INVALID_VALUE
    assert bd.load().sd_geglu_forward(None, None, 0, 8, bd.F16, None) == bd.OK
    assert bd.load().sd_groupnorm_forward(None, None, None, None, 1, 30, 4, 4, ctypes.c_float(1e-5), bd.F16, None) == bd.ERR_INVALID_VALUE


def test_create_without_a_device_fails_cleanly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    h = ctypes.c_void_p(1234)
    rc = lib.sd_attn_create(ctypes.byref(h))
    assert rc in (bd.ERR_CUDA, bd.ERR_ARCH)
    assert h.value is None


def test_binding_refuses_to_run_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(bd, "_lib", None)
    monkeypatch.setattr(bd, "LIB_PATH", str(tmp_path / "libsd_attn.so"))
    with pytest.raises(FileNotFoundError):
        bd.sd_attn_destroy(None)


# ---------------------------------------------------------------- workloads

def test_workload_shapes_and_flop_counts():
    cfg = workloads.all_configs()
    assert [len(cfg[i]) for i in range(1, 6)] == [1, 2, 4, 32, 3]
    c2 = cfg[2][0]
    assert (c2.B, c2.H, c2.Nq, c2.Nk, c2.d) == (2, 8, 4096, 4096, 40)
    assert c2.flops == 4 * 2 * 8 * 4096 * 4096 * 40 == 42949672960
    assert c2.io_bytes() == 2 * 16 * 40 * 4 * 4096
    total = sum(c.flops for c in cfg[4])
    assert abs(total / 1e9 - 252.10) < 0.05
    kinds = [c.kind for c in cfg[4]]
    assert kinds.count("self") == 16 and kinds.count("cross") == 16
    assert cfg[4][-2].Nq == 64 and cfg[4][-2].d == 160 and cfg[4][-2].kind == "self"
    assert float(c2.scale()) == pytest.approx(1 / np.sqrt(40), rel=1e-7)


def test_inputs_are_deterministic_and_structured():
    call = workloads.config3()[3]
    q1, k1, v1 = workloads.make_inputs(call)
    q2, k2, v2 = workloads.make_inputs(call)
    assert np.array_equal(q1, q2) and np.array_equal(k1, k2) and np.array_equal(v1, v2)
    assert q1.dtype == np.float16 and q1.shape == (2, 8, 64, 160) and k1.shape == (2, 8, 77, 160)
    assert np.array_equal(v1[:, :, 57:], np.broadcast_to(v1[:, :, 57:58], v1[:, :, 57:].shape))
    assert not np.array_equal(k1[:, :, 56], k1[:, :, 57])
    plain, peaked = workloads.config2()
    qp, _, _ = workloads.make_inputs(plain)
    qk, _, _ = workloads.make_inputs(peaked)
    assert 0.97 < qp.astype(np.float64).std() < 1.03
    assert 3.9 < qk.astype(np.float64).std() < 4.1


def test_shard_units_partitions_without_gaps():
    for n in (0, 1, 16, 17, 32):
        for world in (1, 2, 3, 8):
            spans = [workloads.shard_units(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
                assert a1 == b0 and a0 <= a1
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        workloads.shard_units(4, 2, 2)
