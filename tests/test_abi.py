"""The C-ABI library loads on a machine without a GPU and exports every symbol that
include/resps.h declares; host-side argument checks answer before any CUDA call."""
import ctypes
import os
import re

from paper_2601_12212_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "resps.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(resps_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    build.build()
    lib = binding.load()
    names = declared_functions()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_header_is_plain_c():
    import subprocess
    src = '#include "resps.h"\nint main(void){ return sizeof(resps_step) == 16 && sizeof(resps_shape) == 32 ? 0 : 1; }\n'
    exe = "/tmp/resps_header_check"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                    "-x", "c", "-", "-o", exe], input=src.encode(), check=True)
    assert subprocess.run([exe]).returncode == 0


def test_host_side_argument_checks_need_no_device():
    lib = binding.load()
    h = ctypes.c_void_p()
    assert lib.resps_create(None, None) == binding.RESPS_ERR_INVALID_ARG
    bad = binding.RespsShape(32, 8, 96, 1000, 1, 64, 8, 4)       # head_dim 96
    assert lib.resps_create(ctypes.byref(h), ctypes.byref(bad)) == binding.RESPS_ERR_UNSUPPORTED_SHAPE
    bad = binding.RespsShape(32, 5, 128, 1000, 1, 64, 8, 4)      # Hq % Hkv != 0
    assert lib.resps_create(ctypes.byref(h), ctypes.byref(bad)) == binding.RESPS_ERR_UNSUPPORTED_SHAPE
    bad = binding.RespsShape(32, 8, 128, 1000, 1, 129, 8, 4)     # max_tt beyond the action space
    assert lib.resps_create(ctypes.byref(h), ctypes.byref(bad)) == binding.RESPS_ERR_UNSUPPORTED_SHAPE
    bad = binding.RespsShape(32, 8, 128, 1000, 1, 64, 32, 16)    # candidate pool beyond shared memory
    assert lib.resps_create(ctypes.byref(h), ctypes.byref(bad)) == binding.RESPS_ERR_UNSUPPORTED_SHAPE
    bad = binding.RespsShape(32, 8, 128, 0, 1, 64, 8, 4)
    assert lib.resps_create(ctypes.byref(h), ctypes.byref(bad)) == binding.RESPS_ERR_INVALID_ARG
    assert lib.resps_tree_expand(None, None, 1, None, 0, 0, 0, 1, 1, None, None, None, None, None,
                                 None, None, None, None, None) == binding.RESPS_ERR_INVALID_ARG
    assert lib.resps_destroy(None) == binding.RESPS_OK
    assert binding.strerror(binding.RESPS_ERR_CAPACITY) == "capacity exceeded"
    assert binding.strerror(0) == "ok"
