"""The C-ABI library builds, loads, and exports every function that include/heinsen_scan.h declares;
the argument checks that run before any CUDA call behave as documented.  No GPU needed."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2311_06281_b200 import build_ext, heinsen_scan
    build_ext.build()
    return heinsen_scan.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "heinsen_scan.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(heinsen_scan_\w+|scan_linear|scan_log)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2311_06281_b200 import heinsen_scan
    names = declared_functions()
    assert len(names) >= 12
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in the header but not exported"
    assert sorted(heinsen_scan.EXPORTS + heinsen_scan.SHORT_EXPORTS) == names, "binding export list and header disagree"


def test_host_side_validation_needs_no_gpu(lib):
    buf = np.zeros(64, dtype=np.float32)
    p = buf.ctypes.data
    OK, INVALID, TOO_SMALL = 0, 1, 3
    # empty problems succeed without touching CUDA
    assert lib.heinsen_scan_log(p, p, p, p, None, None, None, None, 0, 8, 0, 0, None, 0, None) == OK
    assert lib.heinsen_scan_linear(p, p, p, p, 4, 0, 0, None, 0, None) == OK
    # null pointers, negative and oversized shapes, unsupported types, missing sign output
    assert lib.heinsen_scan_log(None, p, p, p, None, None, None, None, 2, 8, 0, 0, p, 4096, None) == INVALID
    assert lib.heinsen_scan_log(p, p, p, p, None, None, None, None, -2, 8, 0, 0, p, 4096, None) == INVALID
    assert lib.heinsen_scan_log(p, p, p, p, None, None, None, None, 2, 1 << 31, 0, 0, p, 4096, None) == INVALID
    assert lib.heinsen_scan_log(p, p, p, p, None, None, None, None, 1 << 31, 8, 0, 0, p, 4096, None) == INVALID
    assert lib.heinsen_scan_log(p, p, p, p, None, None, None, None, 2, 8, 7, 0, p, 4096, None) == INVALID
    assert lib.heinsen_scan_log(p, p, p, p, None, None, None, None, 2, 8, 1, 0, p, 4096, None) == INVALID   # bf16 -> f32
    assert lib.heinsen_scan_log(p, p, p, p, p, None, None, None, 2, 8, 0, 0, p, 4096, None) == INVALID      # no sign_x
    assert lib.heinsen_scan_linear(p, p, p, p, 2, 8, 1, p, 4096, None) == INVALID                           # bf16 linear
    # workspace: null, misaligned, too small
    assert lib.heinsen_scan_log(p, p, p, p, None, None, None, None, 2, 8, 0, 0, None, 4096, None) == INVALID
    assert lib.heinsen_scan_log(p, p, p, p, None, None, None, None, 2, 8, 0, 0, p + 4, 4096, None) == INVALID
    aligned = (p + 255) & ~255
    assert lib.heinsen_scan_log(p, p, p, p, None, None, None, None, 2, 8, 0, 0, aligned, 16, None) == TOO_SMALL
    assert lib.heinsen_scan_log_static(p, p, p, p, 1 << 20, 4096, None) == TOO_SMALL
    assert lib.heinsen_scan_log_complex(None, p, p, p, 2, 8, aligned, 1 << 20, None) == INVALID
    assert lib.heinsen_scan_log_complex(p, p, p, p, 2, 8, aligned, 64, None) == TOO_SMALL
    # the complex entry point needs the header and the look-back descriptors only (the elements are read as they are)
    assert 256 <= lib.heinsen_scan_complex_workspace_bytes(2, 8) <= 1024
    assert lib.heinsen_scan_complex_workspace_bytes(1, 1 << 24) >= lib.heinsen_scan_workspace_bytes(1, 1 << 24)
    assert lib.scan_linear(None, p, p, p, 2, 8) == INVALID and lib.scan_linear(p, p, p, p, 0, 8) == OK
    assert lib.scan_log(p, p, p, p, p, None, None, None, 2, 8) == INVALID and lib.scan_log(p, p, p, p, None, None, None, None, 2, 0) == OK
    assert lib.heinsen_scan_set_path(7) == INVALID and lib.heinsen_scan_set_path(0) == OK


def test_workspace_sizes_and_messages(lib):
    assert lib.heinsen_scan_workspace_bytes(0, 8) == 0 and lib.heinsen_scan_workspace_bytes(8, -1) == 0
    small, big = lib.heinsen_scan_workspace_bytes(1, 4096), lib.heinsen_scan_workspace_bytes(1, 1 << 26)
    assert 256 <= small <= 512 and small < big <= 1 << 20
    assert lib.heinsen_scan_workspace_bytes(16384, 2048) < 1 << 20
    assert lib.heinsen_scan_host_scratch_bytes(16, 1024, 0, 0, 0) >= 3 * 16 * 1024 * 4
    for code in range(7):
        msg = lib.heinsen_scan_strerror(code)
        assert isinstance(msg, bytes) and len(msg) > 1
    assert lib.heinsen_scan_strerror(99) == b"unknown status"
    assert lib.heinsen_scan_launch_count() >= 0 and lib.heinsen_scan_last_path() in (0, 1, 2)


def test_without_a_gpu_the_product_path_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    buf = np.zeros(4096, dtype=np.float32)
    p = (buf.ctypes.data + 255) & ~255
    status = lib.heinsen_scan_log(p, p, p, p, None, None, None, None, 2, 8, 0, 0, p, 4096, None)
    assert status in (2, 4)   # unsupported device / CUDA error: never a silent CPU result
    from paper_2311_06281_b200 import heinsen_scan
    with pytest.raises(ValueError):
        heinsen_scan.scan_log(torch.zeros(2, 8), torch.zeros(2, 8), torch.zeros(2))


def test_window_predicate_of_the_checked_build(lib):
    """The predicate the checked build (-DHEINSEN_DEBUG) applies to every shared-memory access: the access must lie
    inside [base, base + size) and be aligned to its width.  It is plain arithmetic, exported by both builds."""
    ok = lib.heinsen_scan_debug_window_ok
    base, size = 0x1000, 0x400
    assert ok(base, 16, base, size, 16) == 1 and ok(base + size - 16, 16, base, size, 16) == 1
    assert ok(base + size - 12, 16, base, size, 4) == 0            # runs over the end
    assert ok(base + size, 4, base, size, 4) == 0                  # starts at the end
    assert ok(base - 16, 16, base, size, 16) == 0                  # before the window
    assert ok(base + 4, 16, base, size, 16) == 0                   # misaligned for its width
    assert ok(base + 4, 4, base, size, 4) == 1
    assert ok(base, size + 1, base, size, 1) == 0 and ok(base, size, base, size, 1) == 1
    assert ok(base, 4, base, size, 0) == 0                         # no alignment given: refused, not divided by
    assert ok(2**64 - 8, 16, base, size, 8) == 0                   # no wrap-around
    assert lib.heinsen_scan_debug_build() == 0 and lib.heinsen_scan_debug_faults(None) == 0


def test_tuning_and_probe_arguments_are_checked_on_the_host(lib):
    """heinsen_scan_tune knows its knobs by name (no environment look-up per call) and refuses others; the roofline
    probe refuses bad arguments before it touches CUDA."""
    import ctypes
    assert lib.heinsen_scan_tune(b"WARPS", 12) == 0 and lib.heinsen_scan_tune(b"WARPS", -1) == 0
    for name in (b"ROWS_PER_WARP", b"STAGES", b"ROW_TICKETS", b"SPANS", b"NO_TMA", b"NO_FLAT", b"NO_PDL", b"LB_STAGES", b"LB_WARPS",
                 b"LB_SLEEP_IDLE", b"LB_SLEEP_READY", b"LB_CTAS_PER_SM"):
        assert lib.heinsen_scan_tune(name, -1) == 0, name
    assert lib.heinsen_scan_tune(b"NO_SUCH_KNOB", 1) == 1 and lib.heinsen_scan_tune(None, 1) == 1
    r, s = ctypes.c_double(0), ctypes.c_double(0)
    assert lib.heinsen_scan_probe_mufu(0, ctypes.byref(r), ctypes.byref(s)) == 1
    assert lib.heinsen_scan_probe_mufu(16, None, ctypes.byref(s)) == 1
