"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes as C
import os
import re

from paper_1606_08495_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "w2v.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(w2v_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    names = declared_symbols()
    assert len(names) >= 15
    for name in names:
        assert getattr(lib, name) is not None
    assert set(names) == set(binding.EXPORTS)


def test_argument_checks_need_no_gpu():
    lib = binding.load()
    h = C.c_void_p()
    # vocabulary, dimension and pointer checks come before any CUDA call
    assert lib.w2v_create(1, 100, 0, None, None, None, C.byref(h)) == binding.W2V_ERR_ARG
    assert lib.w2v_create(1 << 31, 100, 0, None, None, None, C.byref(h)) == binding.W2V_ERR_ARG
    assert lib.w2v_create(100, 102, 0, None, None, None, C.byref(h)) == binding.W2V_ERR_ARG
    assert lib.w2v_create(100, 2048, 0, None, None, None, C.byref(h)) == binding.W2V_ERR_ARG
    assert lib.w2v_create(100, 100, 0, 256, None, None, C.byref(h)) == binding.W2V_ERR_ARG     # U without V
    assert lib.w2v_create(100, 100, 0, 260, 512, None, C.byref(h)) == binding.W2V_ERR_ARG      # misaligned
    assert lib.w2v_create(100, 100, 0, None, None, None, None) == binding.W2V_ERR_ARG
    assert h.value is None
    assert lib.w2v_destroy(None) == binding.W2V_OK
    assert lib.w2v_sgns_step(None, None, 0, 5, 5, 0.1, 0, None) == binding.W2V_ERR_ARG
    assert lib.w2v_partial_dots(None, None, 0, 0, 4, None) == binding.W2V_ERR_ARG
    assert lib.w2v_last_error(None) == b"invalid handle"


def test_stats_struct_layout_matches_the_header():
    assert C.sizeof(binding.StepStats) == 7 * 8 + 2 * 4
