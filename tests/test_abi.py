"""CPU-side checks of the boundary: the CUDA library builds for sm_100a, loads, and exports every
symbol that include/sgemm_cube.h declares.  No compute call is made here."""
import ctypes
import os
import re

import pytest

from paper_2507_23387_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return ctypes.CDLL(build.LIB)


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sgemm_cube.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(sgemm_cube\w*)\s*\(", text)
    return sorted(set(names))


def test_header_declares_the_documented_entry_points():
    names = _declared_functions()
    for must in ("sgemm_cube_create", "sgemm_cube_destroy", "sgemm_cube_split", "sgemm_cube",
                 "sgemm_cube_unfused"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in _declared_functions():
        assert hasattr(lib, name), "missing export: %s" % name


def test_binding_lists_every_declared_symbol():
    assert sorted(binding.EXPORTS) == _declared_functions()


def test_status_strings_and_version(lib):
    lib.sgemm_cube_status_string.restype = ctypes.c_char_p
    seen = set()
    for code in range(7):
        s = lib.sgemm_cube_status_string(code)
        assert s and s not in seen
        seen.add(s)
    assert lib.sgemm_cube_status_string(99) == b"unknown status"
    assert lib.sgemm_cube_version() >= 100


def test_null_arguments_are_rejected_without_a_device(lib):
    lib.sgemm_cube_create.argtypes = [ctypes.c_void_p, ctypes.c_int]
    assert lib.sgemm_cube_create(None, 0) == binding.INVALID_ARG
    lib.sgemm_cube_destroy.argtypes = [ctypes.c_void_p]
    assert lib.sgemm_cube_destroy(None) == binding.INVALID_ARG
    lib.sgemm_cube_check.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    assert lib.sgemm_cube_check(None, None, None) == binding.INVALID_ARG


def test_binding_fails_loudly_when_library_is_missing(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(OSError):
        binding.load()


def test_input_scaling_choice_is_host_arithmetic(lib):
    import oracle
    for ra, rb in [([-14, 15, 0], [-14, 15, 0]), ([-40, -20, 0], [3, 20, 0]), ([0, 0, 1], [0, 0, 0]),
                   ([127, -127, 0], [5, 9, 0])]:
        assert binding.sgemm_cube_choose_input_scaling(ra, rb) == oracle.input_scale_exps(ra, rb)


def test_binding_constants_match_the_header():
    text = open(os.path.join(ROOT, "include", "sgemm_cube.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    values = {m.group(1): int(m.group(2)) for m in re.finditer(r"\b(SGEMM_CUBE_\w+)\s*=\s*(\d+)", text)}
    pairs = {"SGEMM_CUBE_OK": binding.OK, "SGEMM_CUBE_INVALID_ARG": binding.INVALID_ARG,
             "SGEMM_CUBE_MISALIGNED": binding.MISALIGNED, "SGEMM_CUBE_CUDA_ERROR": binding.CUDA_ERROR,
             "SGEMM_CUBE_DEVICE_TIMEOUT": binding.DEVICE_TIMEOUT,
             "SGEMM_CUBE_UNSUPPORTED_ARCH": binding.UNSUPPORTED_ARCH,
             "SGEMM_CUBE_ALLOC_FAILED": binding.ALLOC_FAILED, "SGEMM_CUBE_TOO_LARGE": binding.TOO_LARGE,
             "SGEMM_CUBE_TERMWISE": binding.TERMWISE, "SGEMM_CUBE_ELEMENTWISE": binding.ELEMENTWISE,
             "SGEMM_CUBE_ELEMENTWISE_REORDERED": binding.ELEMENTWISE_REORDERED,
             "SGEMM_CUBE_OPT_TERMWISE_K_BLOCK": binding.OPT_TERMWISE_K_BLOCK,
             "SGEMM_CUBE_OPT_ELEMENTWISE_K_BLOCK": binding.OPT_ELEMENTWISE_K_BLOCK,
             "SGEMM_CUBE_OPT_CTA_PAIR": binding.OPT_CTA_PAIR, "SGEMM_CUBE_OPT_STRATEGY": binding.OPT_STRATEGY,
             "SGEMM_CUBE_OPT_TIME_KERNEL": binding.OPT_TIME_KERNEL, "SGEMM_CUBE_OPT_SPLIT_K": binding.OPT_SPLIT_K,
             "SGEMM_CUBE_STRATEGY_AUTO": binding.STRATEGY_AUTO, "SGEMM_CUBE_STRATEGY_FUSED": binding.STRATEGY_FUSED,
             "SGEMM_CUBE_STRATEGY_TWO_PHASE": binding.STRATEGY_TWO_PHASE}
    for name, val in pairs.items():
        assert values.get(name) == val, name
    m = re.search(r"SGEMM_CUBE_STATIC_SCRATCH_BYTES\s*\((\d+)u\s*<<\s*(\d+)\)", text)
    assert m and int(m.group(1)) << int(m.group(2)) == binding.STATIC_SCRATCH_BYTES
