"""Host-side checks that need no GPU: the library builds, loads and exports the
C ABI declared in include/luq.h; argument errors are reported, not crashed on."""
import ctypes
import os
import re

import pytest

from paper_2112_10769_b200 import binding
from paper_2112_10769_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    libbuild.build()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "luq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(luq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert set(names) == set(binding.SYMBOLS)
    for n in names:
        assert getattr(lib, n) is not None


def declared_arities():
    """Parameter count of every prototype in the header."""
    text = open(os.path.join(ROOT, "include", "luq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    out = {}
    for name, params in re.findall(r"\b(luq_[a-z0-9_]+)\s*\(([^;{]*?)\)\s*;", text, flags=re.S):
        params = params.strip()
        out[name] = 0 if params in ("", "void") else params.count(",") + 1
    return out


def test_binding_marshals_as_many_arguments_as_the_header_declares(lib):
    """The Python binding sets ctypes argtypes for every entry point; a prototype that gains or loses
    a parameter without the binding following would corrupt the call silently."""
    arities = declared_arities()
    assert set(arities) == set(binding.SYMBOLS)
    for name, count in arities.items():
        argtypes = getattr(lib, name).argtypes
        assert argtypes is not None, name
        assert len(argtypes) == count, (name, len(argtypes), count)


def test_constants_and_messages(lib):
    assert lib.luq_kmax() == 4
    assert lib.luq_strerror(0) == b"ok"
    for code in (-1, -2, -3, -4):
        assert len(lib.luq_strerror(code)) > 3


def test_null_arguments_are_rejected_without_a_gpu(lib):
    assert lib.luq_create(None, 0) == binding.ERR_ARG
    assert lib.luq_amax(None, None, 0, 0, None, None) == binding.ERR_ARG
    assert lib.luq_quant_int4(None, None, 0, 0, 0, None, None, None, None, None) == binding.ERR_ARG
    assert lib.luq_quant_grad(None, None, 0, 0, 0, None, 0, 1, None, None, None, None) == binding.ERR_ARG
    assert lib.luq_gemm_fwd(None, None, None, None, None, None, None, None, 1, 1, 32, None) == binding.ERR_ARG
    assert lib.luq_quant_int4_hindsight(None, None, 0, 0, 0, None, 0.1, None, None, None, None, None) == binding.ERR_ARG
    assert lib.luq_quant_grad_ablation(None, None, 0, 0, 0, None, 0, 1, 0, None, None, None, None) == binding.ERR_ARG
    assert lib.luq_status(None, None, None) == binding.ERR_ARG
    assert lib.luq_destroy(None) == 0
    assert lib.luq_launch_count(None) == 0


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        binding.Context(0)
    h = ctypes.c_void_p()
    assert binding.load().luq_create(ctypes.byref(h), 0) in (binding.ERR_CUDA, binding.ERR_UNSUPPORTED)
