"""CPU-side checks of the boundary: the library builds, loads, and exports what include/pw.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2203_12533_b200 import build
    return build.build()


def declared_functions():
    with open(os.path.join(ROOT, "include", "pw.h")) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pw_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(libpath):
    lib = ctypes.CDLL(libpath)
    names = declared_functions()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in pw.h but not exported"


def test_binding_lists_the_same_symbols(libpath):
    from paper_2203_12533_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()


def test_version_and_status_strings(libpath):
    lib = ctypes.CDLL(libpath)
    lib.pw_status_string.restype = ctypes.c_char_p
    assert lib.pw_version() == 100
    assert lib.pw_status_string(0) == b"PW_OK"
    assert lib.pw_status_string(6) == b"PW_ERR_TIMEOUT"


def test_config_struct_matches_header():
    from paper_2203_12533_b200 import binding
    assert ctypes.sizeof(binding.LayerConfig) == 44          # 11 four-byte fields, no padding
    assert ctypes.sizeof(binding._Ptr12) == 12 * ctypes.sizeof(ctypes.c_void_p)


def test_argument_errors_need_no_gpu(libpath):
    """Validation runs before any device work, so these fail the same way without a GPU."""
    from paper_2203_12533_b200 import binding
    lib = binding.lib()
    h = ctypes.c_void_p()
    bad = binding.make_config(2048, 16, 100, 8192, 1024, 8)           # head_dim not 64/128
    assert lib.pw_layer_create(ctypes.byref(bad), ctypes.byref(h)) == 2
    assert b"head_dim" in lib.pw_last_error()
    bad = binding.make_config(2048, 16, 128, 8192, 1000, 8)           # seq_len not a multiple of 128
    assert lib.pw_layer_create(ctypes.byref(bad), ctypes.byref(h)) == 2
    bad = binding.make_config(2048, 8, 128, 8192, 1024, 8)            # heads * head_dim != d_model
    assert lib.pw_layer_create(ctypes.byref(bad), ctypes.byref(h)) == 2
    bad = binding.make_config(2048, 16, 128, 8192, 1024, 8)
    bad.struct_size = 8
    assert lib.pw_layer_create(ctypes.byref(bad), ctypes.byref(h)) == 1
    assert lib.pw_layer_create(None, ctypes.byref(h)) == 1
    import torch
    if not torch.cuda.is_available():
        ok = binding.make_config(2048, 16, 128, 8192, 1024, 8)
        assert lib.pw_layer_create(ctypes.byref(ok), ctypes.byref(h)) == 5   # no device: loud failure, no fallback


def test_tuning_knobs_validate_on_the_host(libpath):
    """pw_set_tuning / pw_get_tuning are pure host state: defaults, round trip, range checks."""
    lib = ctypes.CDLL(libpath)
    v = ctypes.c_int(-1)
    defaults = {0: 1, 1: 1, 2: 0, 3: 1, 4: 64, 5: 0, 6: 0}
    for knob, want in defaults.items():
        assert lib.pw_get_tuning(knob, ctypes.byref(v)) == 0 and v.value == want
    assert lib.pw_set_tuning(2, 128) == 0
    assert lib.pw_get_tuning(2, ctypes.byref(v)) == 0 and v.value == 128
    assert lib.pw_set_tuning(2, 100) == 1                    # not a tile width: rejected, unchanged
    assert lib.pw_get_tuning(2, ctypes.byref(v)) == 0 and v.value == 128
    assert lib.pw_set_tuning(2, 0) == 0
    assert lib.pw_set_tuning(0, 2) == 1 and lib.pw_set_tuning(99, 0) == 1 and lib.pw_set_tuning(5, -1) == 1
    assert lib.pw_get_tuning(99, ctypes.byref(v)) == 1 and lib.pw_get_tuning(0, None) == 1


def test_log_sink_receives_failures_and_nvtx_ranges_cost_nothing_without_a_tool(libpath):
    """pw_set_log: an argument error reaches the callback with the text of pw_last_error (no GPU needed);
    level 0 is silent again.  PW_TUNE_NVTX only switches ranges on: the failing call below runs through one."""
    lib = ctypes.CDLL(libpath)
    lib.pw_last_error.restype = ctypes.c_char_p
    LOGFN = ctypes.CFUNCTYPE(None, ctypes.c_int, ctypes.c_char_p, ctypes.c_void_p)
    seen = []
    cb = LOGFN(lambda level, msg, user: seen.append((level, msg.decode())))
    lib.pw_set_log.argtypes = [ctypes.c_int, LOGFN, ctypes.c_void_p]
    assert lib.pw_set_log(7, cb, None) == 1                                  # unknown level
    assert lib.pw_set_log(1, cb, None) == 0
    assert lib.pw_set_tuning(6, 1) == 0
    h = ctypes.c_void_p()
    assert lib.pw_layer_create(None, ctypes.byref(h)) == 1
    assert lib.pw_layer_fwd(None, None, None, None, None, None, None) == 1   # inside an NVTX range, no tool attached
    assert lib.pw_set_tuning(6, 0) == 0
    assert len(seen) == 2 and all(level == 1 for level, _ in seen)
    assert seen[0][1].startswith("PW_ERR_INVALID_ARG: ") and lib.pw_last_error().decode() in seen[1][1]
    assert lib.pw_set_log(0, LOGFN(0), None) == 0
    assert lib.pw_layer_create(None, ctypes.byref(h)) == 1
    assert len(seen) == 2
