"""ctypes binding of libcake.so: argument marshalling only.

Every step of the eviction path runs inside the CUDA library; this module turns
torch tensors into device pointers, passes the current CUDA stream, and raises
`CakeError` on a non-zero status.  There is no CPU fallback: if the shared
library is missing or a tensor is not on a CUDA device the call fails.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcake.so")

CAKE_OK = 0
CAKE_ERR_ARG, CAKE_ERR_BUDGET, CAKE_ERR_CAPACITY, CAKE_ERR_NONFINITE = -1, -2, -3, -4
CAKE_ERR_TIMEOUT, CAKE_ERR_CUDA, CAKE_ERR_STATE = -5, -6, -7
CAKE_DTYPE_FP32, CAKE_DTYPE_BF16 = 0, 1
CAKE_POOL_MAX, CAKE_POOL_AVG = 0, 1

EXPORTS = [
    "cake_create", "cake_destroy", "cake_begin", "cake_score_layer", "cake_allocate",
    "cake_evict", "cake_compact", "cake_packed_rows_bound", "cake_get_indicators",
    "cake_get_preferences", "cake_get_budgets", "cake_get_positions", "cake_set_indicators",
    "cake_set_preferences", "cake_status", "cake_strerror", "cake_launch_count",
    "cake_profile_enable", "cake_profile_read", "cake_uses_tensor_cores",
    "cake_select_positions_static", "cake_plan_info", "cake_set_wait_limit", "cake_debug_skew_sync",
    "cake_decode_rows_bound", "cake_decode_begin", "cake_decode_step", "cake_decode_get_state",
    "cake_compact_int4", "cake_plan_check",
]
PROF_KINDS = ["score", "finalize", "allocate", "evict", "compact"]


class CakeConfig(ctypes.Structure):
    """Mirror of `cake_config` in include/cake.h."""
    _fields_ = [
        ("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("window", ctypes.c_int32), ("pool_kernel", ctypes.c_int32),
        ("pool_mode", ctypes.c_int32), ("var_ddof", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("gamma", ctypes.c_float),
        ("tau1", ctypes.c_float), ("tau2", ctypes.c_float),
        ("total_budget", ctypes.c_int64), ("max_requests", ctypes.c_int32),
        ("max_total_tokens", ctypes.c_int64), ("indicator_mode", ctypes.c_int32),
        ("alloc_mode", ctypes.c_int32), ("pyramid_slope", ctypes.c_float),
    ]


class CakeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib: Optional[ctypes.CDLL] = None


def load_library(path: str = LIB_PATH) -> ctypes.CDLL:
    """dlopen libcake.so and declare the signatures.  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(path):
        raise ImportError(f"{path} not found: build it with `python -m paper_2503_12491_b200.build`")
    lib = ctypes.CDLL(path)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.cake_create.argtypes = [ctypes.POINTER(CakeConfig), ctypes.POINTER(vp)]
    lib.cake_destroy.argtypes = [vp]
    lib.cake_begin.argtypes = [vp, i32, ctypes.POINTER(i64), vp]
    lib.cake_score_layer.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.cake_allocate.argtypes = [vp, i32, vp]
    lib.cake_evict.argtypes = [vp, i32, vp]
    lib.cake_compact.argtypes = [vp, i32, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), vp, vp, vp, vp, vp]
    lib.cake_compact_int4.argtypes = [vp, i32, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), i32,
                                      vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.cake_packed_rows_bound.argtypes = [vp]
    lib.cake_packed_rows_bound.restype = i64
    lib.cake_get_indicators.argtypes = [vp, i32, vp, vp]
    lib.cake_get_preferences.argtypes = [vp, vp, vp, vp, vp]
    lib.cake_get_budgets.argtypes = [vp, vp, vp]
    lib.cake_get_positions.argtypes = [vp, i32, i32, vp, i64, vp]
    lib.cake_set_indicators.argtypes = [vp, i32, vp, vp]
    lib.cake_set_preferences.argtypes = [vp, i32, vp, vp]
    lib.cake_status.argtypes = [vp, ctypes.POINTER(i32), vp]
    lib.cake_profile_enable.argtypes = [vp, i32]
    lib.cake_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64), vp]
    lib.cake_uses_tensor_cores.argtypes = [vp]
    lib.cake_select_positions_static.argtypes = [vp, i32, i32, i32, vp, vp]
    lib.cake_plan_info.argtypes = [vp, ctypes.POINTER(i32)]
    lib.cake_plan_check.argtypes = [ctypes.POINTER(CakeConfig), i32, i32, i32, ctypes.POINTER(i64),
                                    ctypes.POINTER(i32)]
    lib.cake_decode_rows_bound.argtypes = [vp]
    lib.cake_decode_rows_bound.restype = i64
    lib.cake_decode_begin.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), vp, vp, vp, i32, vp]
    lib.cake_decode_step.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
    lib.cake_decode_get_state.argtypes = [vp, i32, i32, vp, vp, vp, vp]
    lib.cake_set_wait_limit.argtypes = [vp, i64]
    lib.cake_debug_skew_sync.argtypes = [vp, i32]
    lib.cake_strerror.argtypes = [i32]
    lib.cake_strerror.restype = ctypes.c_char_p
    lib.cake_launch_count.argtypes = []
    lib.cake_launch_count.restype = i64
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("cake_packed_rows_bound", "cake_strerror", "cake_launch_count",
                        "cake_decode_rows_bound"):
            fn.restype = i32
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().cake_strerror(code).decode()


def launch_count() -> int:
    return int(load_library().cake_launch_count())


def _check(code: int, where: str) -> None:
    if code != CAKE_OK:
        raise CakeError(code, where)


def _ptr(t: Optional[torch.Tensor], dtype: Optional[torch.dtype] = None,
         pinned_ok: bool = False) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda and not (pinned_ok and t.is_pinned()):
        raise ValueError("libcake takes CUDA tensors only" +
                         (" (or pinned host tensors here)" if pinned_ok else ""))
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def select_positions_static(values: torch.Tensor, keep: int,
                            out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """cake_select_positions_static: per-head top-`keep` positions (ascending) of a CUDA fp32
    tensor [n_heads][n], for callers that may not allocate device memory.  The library call
    allocates nothing; pass `out` (int32 [n_heads][keep]) to keep torch from allocating too."""
    n_heads, n = values.shape
    if out is None:
        out = torch.empty(n_heads, max(keep, 1), dtype=torch.int32, device=values.device)[:, :keep]
        out = out.contiguous()
    _check(load_library().cake_select_positions_static(
        _ptr(values, torch.float32), n_heads, n, keep, _ptr(out, torch.int32) if keep > 0 else None,
        _stream()), "cake_select_positions_static")
    return out


class Cake:
    """One libcake context.  Method names follow the C entry points."""

    def __init__(self, *, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 window: int, pool_kernel: int, gamma: float, total_budget: int,
                 max_requests: int, max_total_tokens: int, dtype: torch.dtype = torch.bfloat16,
                 tau1: float = 1.0, tau2: float = 1.0, pool_mode: int = CAKE_POOL_MAX,
                 var_ddof: int = 0, indicator_mode: int = 0, alloc_mode: int = 0,
                 pyramid_slope: float = 0.0):
        self.lib = load_library()
        self.cfg = CakeConfig(n_layers, n_q_heads, n_kv_heads, head_dim, window, pool_kernel,
                              pool_mode, var_ddof,
                              CAKE_DTYPE_FP32 if dtype == torch.float32 else CAKE_DTYPE_BF16,
                              gamma, tau1, tau2, total_budget, max_requests, max_total_tokens,
                              indicator_mode, alloc_mode, pyramid_slope)
        self.dtype = dtype
        self._h = ctypes.c_void_p()
        _check(self.lib.cake_create(ctypes.byref(self.cfg), ctypes.byref(self._h)), "cake_create")
        self.n_req = 0
        self.total_tokens = 0
        self.seq_lens: List[int] = []

    # -- life cycle
    def destroy(self) -> None:
        if getattr(self, "_h", None) and self._h.value:
            self.lib.cake_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- the path
    def begin(self, cu_seqlens: Sequence[int]) -> None:
        n_req = len(cu_seqlens) - 1
        arr = (ctypes.c_int64 * (n_req + 1))(*[int(x) for x in cu_seqlens])
        _check(self.lib.cake_begin(self._h, n_req, arr, _stream()), "cake_begin")
        self.n_req = n_req
        self.total_tokens = int(cu_seqlens[-1]) if n_req > 0 else 0
        self.seq_lens = [int(cu_seqlens[r + 1] - cu_seqlens[r]) for r in range(n_req)]

    def score_layer(self, layer: int, q_win: torch.Tensor, k: torch.Tensor,
                    lse: Optional[torch.Tensor] = None) -> None:
        _check(self.lib.cake_score_layer(self._h, layer, _ptr(q_win, self.dtype), _ptr(k, self.dtype),
                                         _ptr(lse, torch.float32), _stream()), "cake_score_layer")

    def allocate(self, stage: int) -> None:
        _check(self.lib.cake_allocate(self._h, stage, _stream()), "cake_allocate")

    def evict(self, stage: int) -> None:
        _check(self.lib.cake_evict(self._h, stage, _stream()), "cake_evict")

    def packed_rows_bound(self) -> int:
        v = int(self.lib.cake_packed_rows_bound(self._h))
        if v < 0:
            raise CakeError(v, "cake_packed_rows_bound")
        return v

    def compact(self, k_layers: Sequence[Optional[torch.Tensor]],
                v_layers: Sequence[Optional[torch.Tensor]], *, layer_lo: int = 0,
                layer_hi: Optional[int] = None, k_out: Optional[torch.Tensor] = None,
                v_out: Optional[torch.Tensor] = None, row_offsets: Optional[torch.Tensor] = None,
                positions: Optional[torch.Tensor] = None, want_positions: bool = True
                ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor, Optional[torch.Tensor]]:
        L = self.cfg.n_layers
        hi = L if layer_hi is None else layer_hi
        dev = torch.device("cuda", torch.cuda.current_device())
        rows = self.packed_rows_bound()
        if k_out is None:
            k_out = torch.empty(max(rows, 1), self.cfg.head_dim, dtype=self.dtype, device=dev)
        if v_out is None:
            v_out = torch.empty(max(rows, 1), self.cfg.head_dim, dtype=self.dtype, device=dev)
        if row_offsets is None:
            row_offsets = torch.empty(self.n_req * L + 1, dtype=torch.int64, device=dev)
        if positions is None and want_positions:
            positions = torch.empty(max(rows, 1), dtype=torch.int32, device=dev)
        # K/V of a layer may also live in pinned host memory: the gather then fetches only the
        # retained rows over the bus
        kp = (ctypes.c_void_p * L)(*[(_ptr(t, self.dtype, True) if t is not None else None) for t in k_layers])
        vp = (ctypes.c_void_p * L)(*[(_ptr(t, self.dtype, True) if t is not None else None) for t in v_layers])
        _check(self.lib.cake_compact(self._h, layer_lo, hi, kp, vp, _ptr(k_out), _ptr(v_out),
                                     _ptr(row_offsets, torch.int64), _ptr(positions, torch.int32),
                                     _stream()), "cake_compact")
        return k_out, v_out, row_offsets, positions

    def compact_int4(self, k_layers, v_layers, group: int = 32):
        """cake_compact_int4 over all layers; returns a dict of the output tensors."""
        L, d = self.cfg.n_layers, self.cfg.head_dim
        dev = torch.device("cuda", torch.cuda.current_device())
        rows = max(self.packed_rows_bound(), 1)
        kg = rows // group + self.n_req * L * self.cfg.n_kv_heads + 1
        out = dict(k_codes=torch.zeros(rows, d // 2, dtype=torch.uint8, device=dev),
                   k_scale=torch.zeros(kg, d, dtype=torch.float32, device=dev),
                   k_zero=torch.zeros(kg, d, dtype=torch.float32, device=dev),
                   v_codes=torch.zeros(rows, d // 2, dtype=torch.uint8, device=dev),
                   v_scale=torch.zeros(rows, d // group, dtype=torch.float32, device=dev),
                   v_zero=torch.zeros(rows, d // group, dtype=torch.float32, device=dev),
                   row_offsets=torch.empty(self.n_req * L + 1, dtype=torch.int64, device=dev),
                   kgroup_offsets=torch.empty(self.n_req * L + 1, dtype=torch.int64, device=dev),
                   positions=torch.empty(rows, dtype=torch.int32, device=dev))
        kp = (ctypes.c_void_p * L)(*[_ptr(t, self.dtype) for t in k_layers])
        vp = (ctypes.c_void_p * L)(*[_ptr(t, self.dtype) for t in v_layers])
        _check(self.lib.cake_compact_int4(
            self._h, 0, L, kp, vp, group, _ptr(out["k_codes"]), _ptr(out["k_scale"]), _ptr(out["k_zero"]),
            _ptr(out["v_codes"]), _ptr(out["v_scale"]), _ptr(out["v_zero"]), _ptr(out["row_offsets"]),
            _ptr(out["kgroup_offsets"]), _ptr(out["positions"]), _stream()), "cake_compact_int4")
        return out

    # -- getters / hooks
    def get_indicators(self, layer: int) -> torch.Tensor:
        out = torch.empty(self.cfg.n_kv_heads, max(self.total_tokens, 1), dtype=torch.float32,
                          device="cuda")[:, : self.total_tokens].contiguous()
        _check(self.lib.cake_get_indicators(self._h, layer, _ptr(out), _stream()),
               "cake_get_indicators")
        return out

    def get_preferences(self) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        shape = (self.n_req, self.cfg.n_layers)
        H, V, P = (torch.zeros(shape, dtype=torch.float64, device="cuda") for _ in range(3))
        _check(self.lib.cake_get_preferences(self._h, _ptr(H), _ptr(V), _ptr(P), _stream()),
               "cake_get_preferences")
        return H, V, P

    def get_budgets(self) -> torch.Tensor:
        out = torch.zeros(self.n_req, self.cfg.n_layers, dtype=torch.int32, device="cuda")
        _check(self.lib.cake_get_budgets(self._h, _ptr(out), _stream()), "cake_get_budgets")
        return out

    def get_positions(self, req: int, layer: int, length: int) -> torch.Tensor:
        out = torch.empty(self.cfg.n_kv_heads, max(length, 1), dtype=torch.int32,
                          device="cuda")[:, :length].contiguous()
        _check(self.lib.cake_get_positions(self._h, req, layer, _ptr(out), out.numel(), _stream()),
               "cake_get_positions")
        return out

    def set_indicators(self, layer: int, values: torch.Tensor) -> None:
        _check(self.lib.cake_set_indicators(self._h, layer, _ptr(values, torch.float32), _stream()),
               "cake_set_indicators")

    def set_preferences(self, P: torch.Tensor) -> None:
        _check(self.lib.cake_set_preferences(self._h, P.shape[1], _ptr(P, torch.float64), _stream()),
               "cake_set_preferences")

    def status(self) -> int:
        s = ctypes.c_int32(0)
        _check(self.lib.cake_status(self._h, ctypes.byref(s), _stream()), "cake_status")
        return int(s.value)

    # -- decode-time eviction
    def decode_begin(self, k_layers, v_layers, update_mode: int = 0):
        """Builds the decode cache; returns (k_cache, v_cache, row_offsets)."""
        L = self.cfg.n_layers
        rows = int(self.lib.cake_decode_rows_bound(self._h))
        if rows < 0:
            raise CakeError(rows, "cake_decode_rows_bound")
        dev = torch.device("cuda", torch.cuda.current_device())
        k_cache = torch.zeros(max(rows, 1), self.cfg.head_dim, dtype=self.dtype, device=dev)
        v_cache = torch.zeros(max(rows, 1), self.cfg.head_dim, dtype=self.dtype, device=dev)
        off = torch.empty(self.n_req * L + 1, dtype=torch.int64, device=dev)
        kp = (ctypes.c_void_p * L)(*[_ptr(t, self.dtype) for t in k_layers])
        vp = (ctypes.c_void_p * L)(*[_ptr(t, self.dtype) for t in v_layers])
        _check(self.lib.cake_decode_begin(self._h, kp, vp, _ptr(k_cache), _ptr(v_cache),
                                          _ptr(off, torch.int64), update_mode, _stream()),
               "cake_decode_begin")
        return k_cache, v_cache, off

    def decode_step(self, layer: int, q_new, k_new, v_new, k_cache, v_cache) -> None:
        _check(self.lib.cake_decode_step(self._h, layer, _ptr(q_new, self.dtype), _ptr(k_new, self.dtype),
                                         _ptr(v_new, self.dtype), _ptr(k_cache), _ptr(v_cache),
                                         _stream()), "cake_decode_step")

    def decode_get_state(self, req: int, layer: int, length: int):
        """(positions, scores, slots), each [H_kv][length], entries in ascending token position."""
        H = self.cfg.n_kv_heads
        pos = torch.empty(H, length, dtype=torch.int32, device="cuda")
        sc = torch.empty(H, length, dtype=torch.float32, device="cuda")
        sl = torch.empty(H, length, dtype=torch.int32, device="cuda")
        _check(self.lib.cake_decode_get_state(self._h, req, layer, _ptr(pos), _ptr(sc), _ptr(sl),
                                              _stream()), "cake_decode_get_state")
        return pos, sc, sl

    def set_wait_limit(self, cycles: int) -> None:
        _check(self.lib.cake_set_wait_limit(self._h, cycles), "cake_set_wait_limit")

    def debug_skew_sync(self, delta: int) -> None:
        _check(self.lib.cake_debug_skew_sync(self._h, delta), "cake_debug_skew_sync")

    def plan_info(self) -> dict:
        out = (ctypes.c_int32 * 8)()
        _check(self.lib.cake_plan_info(self._h, out), "cake_plan_info")
        keys = ["tensor_cores", "ctas", "waves", "merge_ways", "a_segments", "b_segments", "ops",
                "reserved_sms"]
        return {k: int(out[i]) for i, k in enumerate(keys)}

    def uses_tensor_cores(self) -> bool:
        return int(self.lib.cake_uses_tensor_cores(self._h)) == 1

    def profile_enable(self, on: bool) -> None:
        _check(self.lib.cake_profile_enable(self._h, 1 if on else 0), "cake_profile_enable")

    def profile_read(self) -> dict:
        n = len(PROF_KINDS)
        ms = (ctypes.c_double * n)()
        cnt = (ctypes.c_int64 * n)()
        _check(self.lib.cake_profile_read(self._h, ms, cnt, _stream()), "cake_profile_read")
        return {k: {"ms": float(ms[i]), "spans": int(cnt[i])} for i, k in enumerate(PROF_KINDS)}

    # -- convenience: the whole prefill-time cascade for one batch
    def run(self, q_layers: Sequence[torch.Tensor], k_layers: Sequence[torch.Tensor],
            v_layers: Sequence[torch.Tensor], cu_seqlens: Sequence[int], **compact_kw):
        """begin; for every layer score -> allocate -> evict; compact once at the end."""
        self.begin(cu_seqlens)
        for l in range(self.cfg.n_layers):
            self.score_layer(l, q_layers[l], k_layers[l])
            self.allocate(l)
            self.evict(l)
        return self.compact(k_layers, v_layers, **compact_kw)
