"""The C-ABI library builds for sm_100a, loads without a GPU and exports every symbol eb.h declares."""
import ctypes
import os
import re

from paper_2608_07964_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "eb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(eb_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound():
    lib_path = build.build_library()
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.SYMBOLS) == names


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(binding.EbSchedResult) == 96
    assert binding.EbSchedResult.util_num.offset == 80
    assert ctypes.sizeof(binding.EbStepBuffers) == 16 * 8
    assert ctypes.sizeof(binding.EbConfig) == 48
    text = open(os.path.join(ROOT, "include", "eb.h")).read()
    for name in ("EB_MAX_MB", "EB_MAX_D", "EB_META_LEN", "EB_HOST_SLOTS"):
        assert int(re.search(name + r"\s*=\s*(\d+)", text).group(1)) == getattr(binding, name), name


def test_host_side_argument_errors_need_no_gpu():
    lib = binding.load_library()
    assert lib.eb_status_string(0) == b"ok"
    assert lib.eb_status_string(5) == b"device-side wait timed out"
    assert lib.eb_num_kernels() == 13
    assert lib.eb_kernel_name(9) == b"ffn_gateup"
    h = ctypes.c_void_p()
    e2d = (ctypes.c_int32 * 4)(0, 0, 1, 1)
    bad = binding.EbConfig(2, 4, 5, 0, 64, 64, 2, 1, 16, e2d)         # K > E
    assert lib.eb_create(ctypes.byref(bad), ctypes.byref(h)) == 2
    bad = binding.EbConfig(2, 4, 2, 0, 60, 64, 2, 1, 16, e2d)         # H not a multiple of 8
    assert lib.eb_create(ctypes.byref(bad), ctypes.byref(h)) == 2
    e2d_bad = (ctypes.c_int32 * 4)(0, 0, 1, 2)
    bad = binding.EbConfig(2, 4, 2, 0, 64, 64, 2, 1, 16, e2d_bad)     # device index out of range
    assert lib.eb_create(ctypes.byref(bad), ctypes.byref(h)) == 1
    assert lib.eb_create(None, ctypes.byref(h)) == 1
    assert lib.eb_destroy(None) == 1
