"""CPU oracle for the Lethe decode/prune hot path — TEST INFRASTRUCTURE ONLY.

This package wraps ``lethe_oracle.c`` (plain scalar C, fp64 arithmetic) with
ctypes.  Only the test-suite, the smoke check and the benchmark's CPU-baseline
leg may import it; the CUDA library never does, and shares no code with it.

State lives in CPU ``torch`` tensors (torch is used as an array container so
that bf16 storage is available); every numeric step happens in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lethe_oracle.c")
_LIB = os.path.join(_HERE, "liblethe_oracle.so")

OK, ERR_INVALID_ARG, ERR_CAPACITY, ERR_BUDGET = 0, 1, 2, 3
F32, BF16, FP8, FP8_E5M2 = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no FMA contraction, OpenMP for the timed baseline)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _CCache(ctypes.Structure):
    _fields_ = [
        ("n_layers", ctypes.c_int32), ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("paged", ctypes.c_int32), ("capacity", ctypes.c_int32), ("page_tokens", ctypes.c_int32),
        ("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("rel", ctypes.c_void_p),
        ("pos", ctypes.c_void_p), ("len", ctypes.c_void_p), ("page_table", ctypes.c_void_p),
        ("n_pages", ctypes.c_int64), ("k_scale", ctypes.c_void_p), ("v_scale", ctypes.c_void_p),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_decode_attend.restype = ctypes.c_int
        _lib.oracle_decode_attend.argtypes = [
            ctypes.POINTER(_CCache), ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p]
        _lib.oracle_estimate_sparsity.restype = ctypes.c_int
        _lib.oracle_estimate_sparsity.argtypes = [ctypes.POINTER(_CCache), ctypes.c_void_p]
        _lib.oracle_alloc_budgets.restype = ctypes.c_int
        _lib.oracle_alloc_budgets.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                              ctypes.c_int32, ctypes.c_void_p]
        _lib.oracle_rasr_prune.restype = ctypes.c_int
        _lib.oracle_rasr_prune.argtypes = [ctypes.POINTER(_CCache), ctypes.c_void_p, ctypes.c_int32,
                                           ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32]
        _lib.oracle_segment_prune.restype = ctypes.c_int
        _lib.oracle_segment_prune.argtypes = [ctypes.POINTER(_CCache), ctypes.c_int32, ctypes.c_float, ctypes.c_int32,
                                              ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32]
        _lib.oracle_collapsed_prune.restype = ctypes.c_int
        _lib.oracle_collapsed_prune.argtypes = [ctypes.POINTER(_CCache), ctypes.c_void_p, ctypes.c_int32,
                                                ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32]
        _lib.oracle_prefill_seed.restype = ctypes.c_int
        _lib.oracle_prefill_seed.argtypes = [ctypes.POINTER(_CCache), ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p,
                                             ctypes.c_float]
        _lib.oracle_e4m3_decode.restype = ctypes.c_double
        _lib.oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
        _lib.oracle_e4m3_encode.restype = ctypes.c_uint8
        _lib.oracle_e4m3_encode.argtypes = [ctypes.c_float]
        _lib.oracle_e5m2_decode.restype = ctypes.c_double
        _lib.oracle_e5m2_decode.argtypes = [ctypes.c_uint8]
        _lib.oracle_e5m2_encode.restype = ctypes.c_uint8
        _lib.oracle_e5m2_encode.argtypes = [ctypes.c_float]
        _lib.oracle_set_threads.argtypes = [ctypes.c_int]
        _lib.oracle_get_threads.restype = ctypes.c_int
        _lib.oracle_max_threads.restype = ctypes.c_int
    return _lib


def set_threads(n: int) -> None:
    lib().oracle_set_threads(int(n))


def get_threads() -> int:
    return int(lib().oracle_get_threads())


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.device.type == "cpu" and t.is_contiguous(), "oracle tensors must be contiguous CPU tensors"
    return ctypes.c_void_p(t.data_ptr())


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return F32
    if dt == torch.bfloat16:
        return BF16
    if dt == torch.float8_e4m3fn:
        return FP8
    if dt == torch.float8_e5m2:
        return FP8_E5M2
    raise ValueError(f"unsupported dtype {dt}")


@dataclass
class OracleCache:
    """Cache state of all layers (CPU tensors, layouts documented in lethe_oracle.c)."""
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    capacity: int                      # contiguous: token slots; paged: pages per item
    k: torch.Tensor
    v: torch.Tensor
    rel: torch.Tensor
    pos: torch.Tensor
    len: torch.Tensor
    page_tokens: int = 0
    page_table: Optional[torch.Tensor] = None
    k_scale: Optional[torch.Tensor] = None      # float8 caches: fp32 [L] (None = 1): stored byte x means scale * x
    v_scale: Optional[torch.Tensor] = None

    @property
    def act_dtype(self) -> torch.dtype:
        """Type of q, k_new, v_new and out: the cache's own, bf16 for a quantised cache."""
        return torch.bfloat16 if self.k.dtype in (torch.float8_e4m3fn, torch.float8_e5m2) else self.k.dtype

    @property
    def paged(self) -> bool:
        return self.page_table is not None

    @property
    def cap_tokens(self) -> int:
        return self.capacity * self.page_tokens if self.paged else self.capacity

    def _c(self) -> _CCache:
        return _CCache(self.n_layers, self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim,
                       _dtype_code(self.k.dtype), 1 if self.paged else 0, self.capacity, self.page_tokens,
                       self.k.data_ptr(), self.v.data_ptr(), self.rel.data_ptr(), self.pos.data_ptr(),
                       self.len.data_ptr(), self.page_table.data_ptr() if self.paged else None,
                       self.k.shape[0] if self.paged else 0,
                       None if self.k_scale is None else self.k_scale.data_ptr(),
                       None if self.v_scale is None else self.v_scale.data_ptr())

    def clone(self) -> "OracleCache":
        return OracleCache(self.n_layers, self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim,
                           self.capacity, self.k.clone(), self.v.clone(), self.rel.clone(), self.pos.clone(),
                           self.len.clone(), self.page_tokens,
                           None if self.page_table is None else self.page_table.clone(),
                           None if self.k_scale is None else self.k_scale.clone(),
                           None if self.v_scale is None else self.v_scale.clone())


def decode_attend(cache: OracleCache, layer_begin: int, layer_end: int, q: torch.Tensor,
                  k_new: Optional[torch.Tensor], v_new: Optional[torch.Tensor],
                  token_pos: Optional[torch.Tensor], scale: torch.Tensor, gamma: float,
                  want_lse: bool = False, want_probs: bool = False):
    """One decode step for layers [layer_begin, layer_end); returns (status, out, lse, probs)."""
    nl = layer_end - layer_begin
    out = torch.zeros((nl, cache.batch, cache.n_q_heads, cache.head_dim), dtype=cache.act_dtype)
    lse = torch.zeros((nl, cache.batch, cache.n_q_heads), dtype=torch.float32) if want_lse else None
    probs = (torch.zeros((nl, cache.batch, cache.n_q_heads, cache.cap_tokens), dtype=torch.float64)
             if want_probs else None)
    assert q.dtype == cache.act_dtype and scale.dtype == torch.float32 and scale.numel() == cache.n_layers
    for sc in (cache.k_scale, cache.v_scale):
        assert sc is None or (sc.dtype == torch.float32 and sc.numel() == cache.n_layers and sc.is_contiguous())
    if token_pos is not None:
        assert token_pos.dtype == torch.int32
    cc = cache._c()
    st = lib().oracle_decode_attend(ctypes.byref(cc), layer_begin, layer_end, _ptr(q), _ptr(k_new), _ptr(v_new),
                                    _ptr(token_pos), _ptr(scale), ctypes.c_float(gamma), _ptr(out), _ptr(lse),
                                    _ptr(probs))
    return st, out, lse, probs


def estimate_sparsity(cache: OracleCache):
    s = torch.zeros((cache.n_layers, cache.batch), dtype=torch.float32)
    cc = cache._c()
    st = lib().oracle_estimate_sparsity(ctypes.byref(cc), _ptr(s))
    return st, s


def alloc_budgets(sparsity: torch.Tensor, total_budget: torch.Tensor, k_min: int):
    assert sparsity.dtype == torch.float32 and sparsity.dim() == 2 and total_budget.dtype == torch.int64
    n_layers, batch = sparsity.shape
    budgets = torch.zeros((n_layers, batch), dtype=torch.int32)
    st = lib().oracle_alloc_budgets(n_layers, batch, _ptr(sparsity.contiguous()), _ptr(total_budget),
                                    int(k_min), _ptr(budgets))
    return st, budgets


def rasr_prune(cache: OracleCache, budgets: torch.Tensor, recent: int, sink: int, max_k: int = 0):
    """Prune in place; returns (status, keep_idx or None)."""
    assert budgets.dtype == torch.int32 and tuple(budgets.shape) == (cache.n_layers, cache.batch)
    keep = None
    if max_k > 0:
        keep = torch.zeros((cache.n_layers, cache.batch, cache.n_kv_heads, max_k), dtype=torch.int32)
    cc = cache._c()
    st = lib().oracle_rasr_prune(ctypes.byref(cc), _ptr(budgets.contiguous()), int(recent), int(sink),
                                 _ptr(keep), int(max_k))
    return st, keep


def segment_prune(cache: OracleCache, n_segments: int, tau: float, recent: int, sink: int, l_evict: torch.Tensor,
                  max_k: int = 0):
    """Algorithm 1 in place (l_evict [L][B][Hkv] int32 is updated); returns (status, keep_idx or None)."""
    assert l_evict.dtype == torch.int32 and tuple(l_evict.shape) == (cache.n_layers, cache.batch, cache.n_kv_heads)
    keep = None
    if max_k > 0:
        keep = torch.zeros((cache.n_layers, cache.batch, cache.n_kv_heads, max_k), dtype=torch.int32)
    cc = cache._c()
    st = lib().oracle_segment_prune(ctypes.byref(cc), int(n_segments), ctypes.c_float(tau), int(recent), int(sink),
                                    _ptr(l_evict), _ptr(keep), int(max_k))
    return st, keep


COLLAPSE_HEADS, COLLAPSE_HEADS_BATCH = 0, 1


def collapsed_prune(cache: OracleCache, budgets: torch.Tensor, recent: int, sink: int, scope: int, max_k: int = 0):
    """Eq. 2 as printed: one score and one retention set per (layer, sequence) [scope 0, budgets [L][B]] or per
    layer [scope 1, budgets [L]]; returns (status, keep_idx [groups][max_k] or None)."""
    groups = cache.n_layers * cache.batch if scope == COLLAPSE_HEADS else cache.n_layers
    assert budgets.dtype == torch.int32 and budgets.numel() == groups
    keep = torch.zeros((groups, max_k), dtype=torch.int32) if max_k > 0 else None
    cc = cache._c()
    st = lib().oracle_collapsed_prune(ctypes.byref(cc), _ptr(budgets.contiguous()), int(recent), int(sink), int(scope),
                                      _ptr(keep), int(max_k))
    return st, keep


def prefill_seed(cache: OracleCache, q_prompt: torch.Tensor, scale: torch.Tensor, gamma: float) -> int:
    """rel[0..P) of every item from the causal prefill attention of the P prompt queries (q_prompt [L][B][P][Hq][D])."""
    assert q_prompt.dtype == cache.k.dtype and q_prompt.dim() == 5 and scale.dtype == torch.float32
    cc = cache._c()
    return lib().oracle_prefill_seed(ctypes.byref(cc), _ptr(q_prompt), int(q_prompt.shape[2]), _ptr(scale),
                                     ctypes.c_float(gamma))
