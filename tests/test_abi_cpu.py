"""Host-side checks that need no GPU: the library builds, loads, exports every symbol the
header declares, and rejects bad arguments before touching CUDA."""
import ctypes as C
import os
import re

import pytest

from paper_2411_17686_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "ficoco.h")).read()
    declared = set(re.findall(r"\b(ficoco_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layouts_match_header():
    # pointers first, then ints: no padding surprises between C and ctypes
    assert C.sizeof(binding.ficoco_params) == 5 * 8 + 4 * 4
    assert C.sizeof(binding.ficoco_v_args) == 11 * 8 + 8 * 4 + 8     # out_cu_seqlens last
    assert C.sizeof(binding.ficoco_l_args) == 6 * 8 + 8 * 4


def test_defaults_are_the_papers(lib):
    p = binding.ficoco_default_params()
    assert (p.lambda_, p.beta, p.gamma, p.eps, p.penalty_coef, p.window) == (0.35, 0.6, 0.6, 0.998, 2.0, 2)
    assert p.max_targets == -1 and p.flags == 3


def test_argument_validation_without_a_device(lib):
    h = C.c_void_p()
    assert lib.ficoco_create(None, 0, 10, 8, 1, 0) == -1
    assert lib.ficoco_create(C.byref(h), 0, 0, 8, 1, 0) == -1
    assert lib.ficoco_create(C.byref(h), 0, 10, 8, 1, -1) == -1
    assert lib.ficoco_create(C.byref(h), 0, 1 << 40, 8, 1, 0) == -2
    assert lib.ficoco_v_reduce(None, None, None, None) == -1
    assert lib.ficoco_l_reduce(None, None, None, None) == -1
    assert lib.ficoco_v_reduce_host(None, None, None) == -1
    assert lib.ficoco_destroy(None) == -1
    assert lib.ficoco_inspect(None, 0, None, 0, None) == -1
    for code in range(0, -9, -1):
        assert lib.ficoco_strerror(code) not in (None, b"unknown error")
    assert lib.ficoco_strerror(-99) == b"unknown error"


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libficoco.so"))
    with pytest.raises(FileNotFoundError):
        binding.load_library()
