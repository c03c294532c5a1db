"""The C-ABI library: it builds, loads, and exports every function include/eexit.h declares.  Host-only calls."""
import ctypes
import os
import re
import shutil

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "eexit.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ee_\w+|dssd_\w+)\s*\(", text)) - {"ee_status", "ee_path"})


@pytest.fixture(scope="module")
def lib():
    from paper_2407_21082_b200 import _lib, build
    if not os.path.exists(build.LIB):
        if shutil.which("nvcc") is None and not os.path.exists("/usr/local/cuda/bin/nvcc"):
            pytest.skip("library not built and nvcc not available")
        build.build()
    return _lib.load()


def test_header_declares_the_three_calls():
    names = _declared_functions()
    for required in ("ee_exit_head", "ee_compact", "dssd_accept", "ee_exit_head_workspace_bytes", "ee_status_string"):
        assert required in names


def test_library_exports_every_declared_symbol(lib):
    from paper_2407_21082_b200 import _lib
    for name in _declared_functions():
        assert hasattr(lib, name), name
        assert name in _lib.PROTOTYPES, f"{name} has no ctypes prototype"
    assert sorted(_lib.PROTOTYPES) == _declared_functions()


def test_status_strings(lib):
    seen = {lib.ee_status_string(i).decode() for i in range(8)}
    assert len(seen) == 8 and lib.ee_status_string(0) == b"ok"
    assert lib.ee_status_string(99) == b"unknown status"


def test_workspace_bytes_is_pure_and_validates(lib):
    f = lib.ee_exit_head_workspace_bytes
    assert f(8, 512, 50304) >= 256 and f(8, 512, 50304) == f(8, 512, 50304)
    assert f(16384, 2560, 50304) >= 16384 * 2560 * 2          # holds the bf16 LayerNorm output
    assert f(16384, 2560, 50304) < 1 << 30
    for bad in [(-1, 512, 10), (8, 513, 10), (8, 4, 10), (8, 512, 0), (8, 8200, 10)]:
        assert f(*bad) == 0
    assert f(0, 512, 10) >= 256


def test_argument_errors_come_back_before_any_launch(lib):
    # these return from validation; nothing touches a device
    assert lib.ee_exit_head(None, 512, None, None, 1e-5, None, 8, 512, 100, None, 1.0, None, None, None, None,
                            None, 0, None) == 1                                   # EE_ERR_NULL
    assert lib.ee_exit_head(None, 512, None, None, 1e-5, None, 8, 500, 100, None, 1.0, None, None, None, None,
                            None, 0, None) == 2                                   # EE_ERR_SHAPE (d % 8)
    assert lib.ee_exit_head(None, 512, None, None, 1e-5, None, 0, 512, 100, None, 1.0, None, None, None, None,
                            None, 0, None) == 0                                   # M = 0 is a no-op
    assert lib.dssd_accept(None, None, None, 4, 0, 0, None, None, None, None) == 2
    assert lib.dssd_accept(None, None, None, 4, 8, 7, None, None, None, None) == 2
    assert lib.dssd_accept(None, None, None, 0, 8, 8, None, None, None, None) == 0
    assert lib.dssd_accept(None, None, None, 4, 8, 8, None, None, None, None) == 1
    assert lib.ee_compact(None, None, 0, 5, 8, None, None, None, None) == 1
    assert lib.ee_workspace_init(None, 0, None) == 1
    buf = ctypes.create_string_buffer(1024)
    addr = (ctypes.addressof(buf) + 255) // 256 * 256
    assert lib.ee_workspace_init(ctypes.c_void_p(addr + 8), 512, None) == 3      # EE_ERR_ALIGN
    assert lib.ee_workspace_init(ctypes.c_void_p(addr), 16, None) == 4           # EE_ERR_WORKSPACE


def test_argument_errors_of_the_later_entry_points(lib):
    """ee_compact_accept, ee_exit_head_multi_host, ee_calibrate, ee_cascade: validation returns before any launch."""
    from paper_2407_21082_b200 import _lib
    N = None
    # compaction + accept in one launch: the shape rules of both parts
    assert lib.ee_compact_accept(N, N, 0, 4, 8, N, N, N, N, N, N, 2, 0, 0, N, N, N, N) == 2          # k < 1
    assert lib.ee_compact_accept(N, N, 0, 4, 8, N, N, N, N, N, N, 2, 4, 3, N, N, N, N) == 2          # kv < k
    assert lib.ee_compact_accept(N, N, 0, 4, 8, N, N, N, N, N, N, 2, 4, 4, N, N, N, N) == 1          # kept_count NULL
    # packed results
    assert lib.ee_exit_head_results_bytes(3, 64) == 3 * 832 and lib.ee_exit_head_results_bytes(1, 1) == 16
    assert lib.ee_exit_head_results_bytes(0, 64) == 0 and lib.ee_exit_head_results_bytes(2, -1) == 0
    heads = (_lib.EEHead * 2)()
    assert lib.ee_exit_head_multi_host(heads, 2, 1e-5, 8, 500, 100, N, N, N, N, N, 0, N) == 2        # d % 8
    assert lib.ee_exit_head_multi_host(heads, 2, 1e-5, 8, 512, 100, N, N, N, N, N, 0, N) == 1        # NULL buffers
    assert lib.ee_exit_head_multi_host(heads, 0, 1e-5, 8, 512, 100, N, N, N, N, N, 0, N) == 0        # no heads: no-op
    # calibration
    assert lib.ee_calibrate_workspace_bytes(-1) == 0
    w0, w1 = lib.ee_calibrate_workspace_bytes(0), lib.ee_calibrate_workspace_bytes(1 << 20)
    assert w0 >= 2048 and w1 >= 2 * 8 * (1 << 20) and w1 < 3 * 8 * (1 << 20)
    assert lib.ee_calibrate(N, N, N, -1, 0.5, N, N, N, 0, N) == 2
    assert lib.ee_calibrate(N, N, N, 4, 1.5, N, N, N, 0, N) == 2                                     # epsilon outside [0, 1]
    assert lib.ee_calibrate(N, N, N, 4, float("nan"), N, N, N, 0, N) == 2
    assert lib.ee_calibrate(N, N, N, 4, 0.5, N, N, N, 0, N) == 1
    # cascade
    assert lib.ee_cascade_workspace_bytes(8, 500, 100) == 0
    assert lib.ee_cascade_workspace_bytes(64, 1024, 50304) > lib.ee_exit_head_workspace_bytes(64, 1024, 50304)
    assert lib.ee_cascade(heads, 0, 1e-5, 8, 512, 100, N, N, N, N, N, 0, N) == 2                     # no heads
    assert lib.ee_cascade(heads, 2, 1e-5, 8, 512, 100, N, N, N, N, N, 0, N) == 1                     # NULL outputs
