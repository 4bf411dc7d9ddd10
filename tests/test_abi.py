"""The C-ABI library builds, loads and exports every symbol the header declares;
argument validation happens on the host before any CUDA call (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2605_06665_b200 import binding as B
from paper_2605_06665_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    builder.build()
    return B.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "unipool.h")).read()
    declared = set(re.findall(r"\b(unipool_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_sizes_are_host_functions(lib):
    cfg = B.make_config(768, 2048, 96, 2, 12, 16384, B.BF16, 1e-6, 2.0)
    cap = B.row_capacity(cfg)
    assert cap % B.ROW_ALIGN == 0 and cap >= 16384 * 2 + 96 * 127
    assert B.workspace_bytes(cfg) > cap * 768 * 2


@pytest.mark.parametrize("field,value,code", [
    ("d_model", 100, -2), ("d_ff", 0, -2), ("pool_size", 513, -2), ("top_k", 9, -2),
    ("top_k", 0, -2), ("dtype", 5, -1), ("n_layers", 0, -1), ("c", 0.0, -1),
])
def test_bad_config_is_refused_before_any_launch(lib, field, value, code):
    cfg = B.make_config(256, 512, 16, 2, 4, 512, B.FP32, 1e-6, 2.0)
    setattr(cfg, field, value)
    handle = ctypes.c_void_p()
    rc = lib.unipool_create(ctypes.byref(handle), ctypes.byref(cfg), None, 0, None)
    assert rc == code and not handle.value
    assert lib.unipool_last_error()
    assert B.workspace_bytes(cfg) == 0


def test_missing_workspace_is_refused(lib):
    cfg = B.make_config(256, 512, 16, 2, 4, 512, B.FP32, 1e-6, 2.0)
    handle = ctypes.c_void_p()
    assert lib.unipool_create(ctypes.byref(handle), ctypes.byref(cfg), None, 0, None) == -3
    assert lib.unipool_create(ctypes.byref(handle), ctypes.byref(cfg), ctypes.c_void_p(256 + 8), 1 << 40, None) == -3
    assert b"aligned" in lib.unipool_last_error()


def test_null_context_is_refused(lib):
    assert lib.unipool_check_status(None, None) == -1
    assert lib.unipool_destroy(None) == 0


def test_debug_mode_adds_a_guard_band_per_workspace_region(lib):
    """UNIPOOL_DEBUG=1 (read once per process, hence the child): 256 bytes behind each of the 13
    regions of a bf16 workspace, 12 of an fp32 one (no split router weights there)."""
    import subprocess
    import sys
    code = (
        "from paper_2605_06665_b200 import binding as B\n"
        "for dt in (B.BF16, B.FP32):\n"
        "    print(B.workspace_bytes(B.make_config(256, 512, 16, 2, 4, 512, dt, 1e-6, 2.0)))\n"
    )
    sizes = {}
    for flag in ("0", "1"):
        env = dict(os.environ, UNIPOOL_DEBUG=flag)
        out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, check=True)
        sizes[flag] = [int(v) for v in out.stdout.split()]
    assert sizes["1"][0] - sizes["0"][0] == 13 * 256
    assert sizes["1"][1] - sizes["0"][1] == 12 * 256
