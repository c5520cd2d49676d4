"""CPU-side checks: the shared library builds, loads and exports every symbol the header declares;
host-side validation answers without a GPU; the N>1 'replicas only' layout of bench.py."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2502_18394_b200 import build, binding
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    from paper_2502_18394_b200 import binding
    header = open(os.path.join(ROOT, "include", "spectre.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(spectre_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(binding.EXPORTS)


def test_status_strings(lib):
    assert lib.spectre_status_string(0) == b"ok"
    for s in range(1, 6):
        assert lib.spectre_status_string(s) not in (b"ok", b"unknown status")
    assert lib.spectre_status_string(99) == b"unknown status"


def test_struct_layouts_match_the_header():
    from paper_2502_18394_b200 import binding as b
    assert C.sizeof(b.Act) == 8 + 4 * 5 + 4 + 8 * 3        # ptr, dtype+BLHD, pad, strides
    assert C.sizeof(b.Cache) == 4 * 6 + 8 * 4
    assert b.GateParams.ln_eps.offset == 32 and b.GateParams.W1.offset == 40
    assert C.sizeof(b.Wavelet) == 16 + 8 * 7 and b.Wavelet.skip.offset == 16 + 8 * 6


def test_null_arguments_fail_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("covers the no-device behaviour")
    h = C.c_void_p()
    assert lib.spectre_create(C.byref(h), 0) == 4            # no CUDA device -> SPECTRE_ERR_CUDA, no fallback
    assert b"no CPU fallback" in lib.spectre_last_error()
    assert lib.spectre_mixer_forward(None, None, None, None, None, 8, None, None, 0) == 1
    assert lib.spectre_prefix_cache_append(None, None, None, None, None, 0) == 1
