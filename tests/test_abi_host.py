"""CPU-side checks of the boundary: the shared library builds, loads, exports every symbol the
header declares, and refuses to run without an sm_100 device.  No kernel is launched here."""
import ctypes as C
import os
import re

import pytest

from paper_2302_00845_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "cdgrab.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cdgrab_[a-z_0-9]+)\s*\(", text)))


def test_header_and_binding_list_the_same_calls():
    assert declared_symbols() == sorted(binding.SIGNATURES)


def test_every_declared_symbol_is_exported(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_the_five_named_calls_exist():
    for name in ("cdgrab_create", "cdgrab_begin_epoch", "cdgrab_step", "cdgrab_end_epoch",
                 "cdgrab_destroy"):
        assert name in declared_symbols()


def test_strerror_covers_all_codes(lib):
    seen = set()
    for code in range(0, -9, -1):
        msg = lib.cdgrab_strerror(code).decode()
        assert msg and msg != "unknown error"
        seen.add(msg)
    assert len(seen) == 9
    assert lib.cdgrab_strerror(-99).decode() == "unknown error"


def test_argument_validation_precedes_device_use(lib):
    h = C.c_void_p()
    assert lib.cdgrab_create(4, 63, 16, binding.F32, C.byref(h)) == binding.ERR_INVALID  # odd n
    assert lib.cdgrab_create(0, 64, 16, binding.F32, C.byref(h)) == binding.ERR_INVALID
    assert lib.cdgrab_create(4, 64, 0, binding.F32, C.byref(h)) == binding.ERR_INVALID
    assert lib.cdgrab_create(4, 64, 16, 7, C.byref(h)) == binding.ERR_INVALID
    assert lib.cdgrab_create(4, 64, 16, binding.F32, None) == binding.ERR_INVALID
    assert lib.cdgrab_destroy(None) == binding.OK
    assert lib.cdgrab_step(None, None, None) == binding.ERR_INVALID
    assert lib.cdgrab_status(None) == binding.ERR_INVALID


def test_no_cpu_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    h = C.c_void_p()
    assert lib.cdgrab_create(4, 64, 1024, binding.F32, C.byref(h)) == binding.ERR_DEVICE
    assert not h.value
    with pytest.raises(binding.CdgrabError):
        binding.CdGrab(4, 64, 1024, "f32")


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2302_00845_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b", src, flags=re.M), f
                assert "liboracle" not in src and "pairbalance_oracle" not in src, f


def test_environment_is_read_at_create_time_only():
    """Launch paths run every few microseconds: knobs are read when a handle is created (create_impl
    and the *_setup / *_supported routines it calls), never per step."""
    csrc = os.path.join(ROOT, "paper_2302_00845_b200", "csrc")
    allowed = ("create_impl", "forced_path", "cdg_fma_tma_setup", "cdg_umma_setup", "cdg_umma_supported",
               "cdg_umma_f32_setup")
    for f in sorted(os.listdir(csrc)):
        src = open(os.path.join(csrc, f)).read()
        for mt in re.finditer(r"getenv\(", src):
            head = src[:mt.start()]
            # name of the innermost function definition that starts at column 0 before the call
            defs = re.findall(r"^(?:static\s+)?(?:inline\s+)?[A-Za-z_][\w \*:<>]*?\b(\w+)\([^;{]*\)\s*\{", head, flags=re.M)
            assert defs and defs[-1] in allowed, (f, defs[-1] if defs else None)


def test_wrong_device_has_its_own_code(lib):
    assert "device" in lib.cdgrab_strerror(binding.ERR_DEVICE).decode()
