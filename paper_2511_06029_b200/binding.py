"""Thin ctypes binding of liblethe.so: same names as the C ABI (include/lethe.h), argument marshalling only.

Every step of the path runs in the CUDA library; nothing here computes.  torch supplies device memory and
streams.  If the library has not been built (``python -m paper_2511_06029_b200.build``) loading fails loudly —
there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("LETHE_LIB", os.path.join(_HERE, "liblethe.so"))   # LETHE_LIB: an alternative build

OK, ERR_INVALID_ARG, ERR_CAPACITY, ERR_BUDGET, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED, ERR_PAGE, ERR_TOO_LARGE = range(9)
STATIC_PRUNE_MAX_ENTRIES = 4 * 1024 * 1024
F32, BF16, FP8_E4M3, FP8_E5M2 = 0, 1, 2, 3
CONTIG, PAGED = 0, 1
VARIANT_AUTO, VARIANT_SIMT, VARIANT_MMA4, VARIANT_MMA8 = 0, 1, 2, 3

EXPORTS = ["lethe_create", "lethe_destroy", "lethe_last_error", "lethe_poll_status", "lethe_set_tuning", "lethe_set_wait_limit",
           "lethe_decode_attend", "lethe_decode_attend_host", "lethe_estimate_sparsity", "lethe_alloc_budgets",
           "lethe_rasr_prune", "lethe_rasr_prune_static", "lethe_segment_prune", "lethe_prefill_seed",
           "lethe_collapsed_prune"]


class LetheError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"lethe status {status}: {msg}")
        self.status = status


class lethe_cache(ctypes.Structure):
    _fields_ = [
        ("n_layers", ctypes.c_int32), ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("layout", ctypes.c_int32), ("capacity", ctypes.c_int32), ("page_tokens", ctypes.c_int32),
        ("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("rel", ctypes.c_void_p), ("pos", ctypes.c_void_p),
        ("len", ctypes.c_void_p), ("page_table", ctypes.c_void_p), ("n_pages", ctypes.c_int64),
        ("k_scale", ctypes.c_void_p), ("v_scale", ctypes.c_void_p),
    ]


_lib = None


def load() -> ctypes.CDLL:
    """Load liblethe.so and declare the prototypes of include/lethe.h."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2511_06029_b200.build` "
                           "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, cp = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(lethe_cache)
    lib.lethe_create.restype = ctypes.c_int
    lib.lethe_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int, ctypes.c_size_t]
    lib.lethe_destroy.restype = None
    lib.lethe_destroy.argtypes = [vp]
    lib.lethe_last_error.restype = ctypes.c_char_p
    lib.lethe_last_error.argtypes = [vp]
    lib.lethe_poll_status.restype = ctypes.c_int
    lib.lethe_poll_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.lethe_set_tuning.restype = ctypes.c_int
    lib.lethe_set_tuning.argtypes = [vp, ctypes.c_int, ctypes.c_int]
    lib.lethe_set_wait_limit.restype = ctypes.c_int
    lib.lethe_set_wait_limit.argtypes = [vp, i32]
    attend_args = [vp, cp, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, ctypes.POINTER(ctypes.c_float),
                   ctypes.c_float, vp, vp, vp]
    lib.lethe_decode_attend.restype = ctypes.c_int
    lib.lethe_decode_attend.argtypes = attend_args
    lib.lethe_decode_attend_host.restype = ctypes.c_int
    lib.lethe_decode_attend_host.argtypes = attend_args
    lib.lethe_estimate_sparsity.restype = ctypes.c_int
    lib.lethe_estimate_sparsity.argtypes = [vp, cp, vp, vp]
    lib.lethe_alloc_budgets.restype = ctypes.c_int
    lib.lethe_alloc_budgets.argtypes = [vp, ctypes.c_int, ctypes.c_int, vp, vp, i32, vp, vp]
    lib.lethe_rasr_prune.restype = ctypes.c_int
    lib.lethe_rasr_prune.argtypes = [vp, cp, vp, i32, i32, vp, i32, vp]
    lib.lethe_collapsed_prune.restype = ctypes.c_int
    lib.lethe_collapsed_prune.argtypes = [vp, cp, vp, i32, i32, i32, vp, i32, vp]
    lib.lethe_segment_prune.restype = ctypes.c_int
    lib.lethe_segment_prune.argtypes = [vp, cp, i32, ctypes.c_float, i32, i32, vp, vp, i32, vp]
    lib.lethe_prefill_seed.restype = ctypes.c_int
    lib.lethe_prefill_seed.argtypes = [vp, cp, vp, i32, ctypes.POINTER(ctypes.c_float), ctypes.c_float, vp]
    lib.lethe_rasr_prune_static.restype = ctypes.c_int
    lib.lethe_rasr_prune_static.argtypes = [cp, vp, i32, i32, vp, i32, vp, vp]
    _lib = lib
    return lib


def _dp(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


class Cache:
    """Device tensors of the cache plus the C descriptor that points at them (the tensors stay owned here)."""

    def __init__(self, n_q_heads: int, k: torch.Tensor, v: torch.Tensor, rel: torch.Tensor, pos: torch.Tensor,
                 len_: torch.Tensor, page_table: Optional[torch.Tensor] = None, k_scale=None, v_scale=None):
        """k_scale, v_scale: per-layer scales of a float8_e4m3fn / float8_e5m2 cache (sequences of L floats; None = 1)."""
        self.k, self.v, self.rel, self.pos, self.len, self.page_table = k, v, rel, pos, len_, page_table
        for t in (k, v, rel, pos, len_) + ((page_table,) if page_table is not None else ()):
            assert t.is_cuda and t.is_contiguous()
        assert rel.dtype == torch.float32 and pos.dtype == torch.int32 and len_.dtype == torch.int32
        L, B, Hkv = len_.shape
        dt = {torch.float32: F32, torch.bfloat16: BF16, torch.float8_e4m3fn: FP8_E4M3, torch.float8_e5m2: FP8_E5M2}[k.dtype]
        if page_table is None:
            assert k.dim() == 5 and tuple(k.shape[:3]) == (L, B, Hkv)
            cap, D, layout, pt, npages = k.shape[3], k.shape[4], CONTIG, 0, 0
            assert tuple(rel.shape) == (L, B, Hkv, cap)
        else:
            assert k.dim() == 3 and page_table.dtype == torch.int32
            npages, pt, D = k.shape
            cap, layout = page_table.shape[3], PAGED
            assert tuple(rel.shape) == (L, B, Hkv, cap * pt)
        self.n_layers, self.batch, self.n_kv_heads, self.n_q_heads, self.head_dim = L, B, Hkv, n_q_heads, D
        self.capacity, self.page_tokens = cap, pt
        self.c = lethe_cache(L, B, n_q_heads, Hkv, D, dt, layout, cap, pt, k.data_ptr(), v.data_ptr(),
                             rel.data_ptr(), pos.data_ptr(), len_.data_ptr(),
                             page_table.data_ptr() if page_table is not None else None, npages, None, None)
        # host arrays of the per-layer scales, kept alive here
        self._k_scale = self._v_scale = None
        if dt in (FP8_E4M3, FP8_E5M2):
            for name, sc in (("k_scale", k_scale), ("v_scale", v_scale)):
                if sc is None:
                    continue
                vals = [float(x) for x in (sc.tolist() if isinstance(sc, torch.Tensor) else sc)]
                assert len(vals) == L
                arr = (ctypes.c_float * L)(*vals)
                setattr(self, "_" + name, arr)
                setattr(self.c, name, ctypes.cast(arr, ctypes.c_void_p))
        else:
            assert k_scale is None and v_scale is None, "scales belong to quantised caches"

    @property
    def act_dtype(self) -> torch.dtype:
        """Type of q, k_new, v_new and out."""
        return torch.bfloat16 if self.k.dtype in (torch.float8_e4m3fn, torch.float8_e5m2) else self.k.dtype

    @property
    def device(self):
        return self.k.device

    @property
    def cap_tokens(self) -> int:
        return self.capacity * self.page_tokens if self.page_table is not None else self.capacity


def rasr_prune_static(cache: "Cache", budgets: torch.Tensor, recent: int, sink: int,
                      keep_idx: Optional[torch.Tensor] = None, status_out: Optional[torch.Tensor] = None) -> int:
    """lethe_rasr_prune_static: the prune step for callers that may not allocate device memory (no context, fixed
    in-library scratch).  Runs on the current device and the current torch stream; returns the host-side status
    (OK, or ERR_TOO_LARGE / ERR_INVALID_ARG / ... when nothing was enqueued).  status_out: device int32[2]."""
    assert budgets.dtype == torch.int32 and budgets.is_cuda
    max_k = 0
    if keep_idx is not None:
        assert keep_idx.dtype == torch.int32 and keep_idx.is_cuda
        max_k = keep_idx.shape[-1]
    if status_out is not None:
        assert status_out.dtype == torch.int32 and status_out.is_cuda and status_out.numel() >= 2
    return int(load().lethe_rasr_prune_static(ctypes.byref(cache.c), _dp(budgets), recent, sink, _dp(keep_idx), max_k,
                                              _dp(status_out), _stream(cache.device)))


COLLAPSE_HEADS, COLLAPSE_HEADS_BATCH = 0, 1


class Context:
    """Owns one lethe_ctx.  Methods carry the C names without the prefix and raise LetheError on failure."""

    def __init__(self, device: int = 0, scratch_bytes_hint: int = 0):
        self.lib = load()
        self.device = device
        h = ctypes.c_void_p()
        st = self.lib.lethe_create(ctypes.byref(h), device, scratch_bytes_hint)
        if st != OK:
            raise LetheError(st, "lethe_create failed (needs an sm_100 GPU)")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.lib.lethe_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def last_error(self) -> str:
        return self.lib.lethe_last_error(self.h).decode()

    def _check(self, st: int):
        if st != OK:
            raise LetheError(st, self.last_error())

    def set_tuning(self, variant: int = 0, splits: int = 0):
        self._check(self.lib.lethe_set_tuning(self.h, variant, splits))

    def set_wait_limit(self, polls: int = 0):
        self._check(self.lib.lethe_set_wait_limit(self.h, polls))

    def poll_status(self):
        """Synchronise the current stream and return (status, item) of the first device-side error since last poll."""
        info = (ctypes.c_int32 * 2)()
        st = self.lib.lethe_poll_status(self.h, _stream(self.device), info)
        return st, int(info[1])

    @staticmethod
    def _scale(scale: Sequence[float]):
        arr = (ctypes.c_float * len(scale))(*[float(x) for x in scale])
        return arr

    def decode_attend(self, cache: Cache, layer_begin: int, layer_end: int, q, k_new, v_new, token_pos, scale, gamma,
                      out, lse=None, scale_c=None):
        sc = scale_c if scale_c is not None else self._scale(scale)
        self._check(self.lib.lethe_decode_attend(self.h, ctypes.byref(cache.c), layer_begin, layer_end, _dp(q),
                                                 _dp(k_new), _dp(v_new), _dp(token_pos), sc, gamma, _dp(out), _dp(lse),
                                                 _stream(self.device)))

    def decode_attend_host(self, cache: Cache, layer_begin: int, layer_end: int, q, k_new, v_new, token_pos, scale,
                           gamma, out, lse=None, scale_c=None):
        """q, k_new, v_new, token_pos, out, lse are HOST tensors (pinned for asynchronous copies)."""
        for t in (q, k_new, v_new, token_pos, out, lse):
            assert t is None or (not t.is_cuda and t.is_contiguous())
        sc = scale_c if scale_c is not None else self._scale(scale)
        self._check(self.lib.lethe_decode_attend_host(self.h, ctypes.byref(cache.c), layer_begin, layer_end, _dp(q),
                                                      _dp(k_new), _dp(v_new), _dp(token_pos), sc, gamma, _dp(out),
                                                      _dp(lse), _stream(self.device)))

    def estimate_sparsity(self, cache: Cache, sparsity: torch.Tensor):
        assert sparsity.is_cuda and sparsity.dtype == torch.float32
        self._check(self.lib.lethe_estimate_sparsity(self.h, ctypes.byref(cache.c), _dp(sparsity),
                                                     _stream(self.device)))

    def alloc_budgets(self, sparsity: torch.Tensor, total_budget: torch.Tensor, k_min: int, budgets: torch.Tensor):
        assert sparsity.dtype == torch.float32 and total_budget.dtype == torch.int64 and budgets.dtype == torch.int32
        L, B = sparsity.shape
        self._check(self.lib.lethe_alloc_budgets(self.h, L, B, _dp(sparsity), _dp(total_budget), k_min, _dp(budgets),
                                                 _stream(self.device)))

    def rasr_prune(self, cache: Cache, budgets: torch.Tensor, recent: int, sink: int,
                   keep_idx: Optional[torch.Tensor] = None):
        assert budgets.dtype == torch.int32 and budgets.is_cuda
        max_k = 0
        if keep_idx is not None:
            assert keep_idx.dtype == torch.int32 and keep_idx.is_cuda
            max_k = keep_idx.shape[-1]
        self._check(self.lib.lethe_rasr_prune(self.h, ctypes.byref(cache.c), _dp(budgets), recent, sink,
                                              _dp(keep_idx), max_k, _stream(self.device)))

    def segment_prune(self, cache: Cache, n_segments: int, tau: float, recent: int, sink: int, l_evict: torch.Tensor,
                      keep_idx: Optional[torch.Tensor] = None):
        assert l_evict.dtype == torch.int32 and l_evict.is_cuda and l_evict.is_contiguous()
        max_k = 0
        if keep_idx is not None:
            assert keep_idx.dtype == torch.int32 and keep_idx.is_cuda
            max_k = keep_idx.shape[-1]
        self._check(self.lib.lethe_segment_prune(self.h, ctypes.byref(cache.c), n_segments, tau, recent, sink,
                                                 _dp(l_evict), _dp(keep_idx), max_k, _stream(self.device)))

    def collapsed_prune(self, cache: Cache, budgets: torch.Tensor, recent: int, sink: int, scope: int,
                        keep_idx: Optional[torch.Tensor] = None):
        """scope COLLAPSE_HEADS: budgets [L][B]; COLLAPSE_HEADS_BATCH: budgets [L]; keep_idx [groups][max_k]."""
        assert budgets.dtype == torch.int32 and budgets.is_cuda and budgets.is_contiguous()
        max_k = 0
        if keep_idx is not None:
            assert keep_idx.dtype == torch.int32 and keep_idx.is_cuda
            max_k = keep_idx.shape[-1]
        self._check(self.lib.lethe_collapsed_prune(self.h, ctypes.byref(cache.c), _dp(budgets), recent, sink, scope,
                                                   _dp(keep_idx), max_k, _stream(self.device)))

    def prefill_seed(self, cache: Cache, q_prompt: torch.Tensor, scale, gamma: float):
        """q_prompt [L][B][P][Hq][D] on the device, cache dtype; overwrites rel[0..P) of every item."""
        assert q_prompt.is_cuda and q_prompt.is_contiguous() and q_prompt.dim() == 5
        self._check(self.lib.lethe_prefill_seed(self.h, ctypes.byref(cache.c), _dp(q_prompt), q_prompt.shape[2],
                                                self._scale(scale), gamma, _stream(self.device)))
