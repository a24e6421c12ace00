"""Host-side checks that need no GPU: the C-ABI library builds, loads, and exports every entry point that
include/lethe.h declares; the binding declares a prototype for each; creating a context without a GPU fails
with a status instead of crashing."""
import ctypes
import os
import re

from paper_2511_06029_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "lethe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lethe_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert len(names) >= 10
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in lethe.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_binding_prototypes_and_no_gpu_behaviour():
    import torch
    lib = binding.load()
    for n in binding.EXPORTS:
        assert getattr(lib, n).argtypes is not None
    if not torch.cuda.is_available():
        h = ctypes.c_void_p()
        assert lib.lethe_create(ctypes.byref(h), 0, 0) == binding.ERR_CUDA and not h.value
        assert lib.lethe_last_error(None) == b"context is NULL"
        assert lib.lethe_set_tuning(None, 0, 0) == binding.ERR_INVALID_ARG


def test_struct_layout_matches_header():
    """The ctypes mirror of lethe_cache has the field order and size the header implies (9 int32, pad, 6 pointers,
    one int64, 2 pointers on LP64)."""
    assert [f[0] for f in binding.lethe_cache._fields_] == [
        "n_layers", "batch", "n_q_heads", "n_kv_heads", "head_dim", "dtype", "layout", "capacity", "page_tokens",
        "k", "v", "rel", "pos", "len", "page_table", "n_pages", "k_scale", "v_scale"]
    assert ctypes.sizeof(binding.lethe_cache) == 40 + 6 * 8 + 8 + 2 * 8
    assert (binding.F32, binding.BF16, binding.FP8_E4M3, binding.FP8_E5M2) == (0, 1, 2, 3)
