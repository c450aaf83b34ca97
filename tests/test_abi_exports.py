"""The C-ABI library loads without a GPU and exports every function the public header declares."""
import ctypes
import os
import re

from paper_2504_08791_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "prima.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(prima_[a-z0-9_]+)\s*\(", text)))


def test_header_functions_are_exported_and_bound():
    build.build()
    names = _declared_functions()
    assert "prima_forward_window" in names and "prima_load_q4k_weights" in names
    L = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert sorted(binding.EXPORTS) == names


def test_argument_errors_need_no_gpu():
    L = binding.lib()
    assert L.prima_ctx_create(None, None, None) == binding.ERR_ARG
    assert L.prima_forward_window(None, 0, 1, None, None, 0, 1) == binding.ERR_ARG
    assert L.prima_dequant_q4k(None, 1, None, None) == binding.ERR_ARG
    assert L.prima_gemv_plan_create(None, 8, 256, 1, None) == binding.ERR_ARG
    assert b"null" in L.prima_last_error(None) or b"bad" in L.prima_last_error(None)
    cfg = binding.ModelConfig(2, 500, 4, 2, 128, 1024, 100, 16, 1, 1e-5, 1e4, 0, 0)   # hidden not a multiple of 256
    h = ctypes.c_void_p()
    assert L.prima_ctx_create(ctypes.byref(cfg), None, ctypes.byref(h)) == binding.ERR_ARG and not h.value
