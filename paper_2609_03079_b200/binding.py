"""ctypes binding of ``include/leanstream.h``: same names, argument marshalling only.

Every step of the path runs inside ``libleanstream.so``.  There is no CPU fallback: if the library is missing or
fails to load, the first call raises.  PyTorch supplies device memory (tensors) and streams only.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

from . import build as _build

LS_OK, LS_ERR_INVALID, LS_ERR_NOMEM, LS_ERR_CUDA, LS_ERR_STATE, LS_ERR_CAPACITY, LS_ERR_TIMEOUT, LS_ERR_INTERNAL = 0, -1, -2, -3, -4, -5, -6, -7
LS_ACT_RELU, LS_ACT_SILU = 0, 1
LS_WDTYPE_BF16, LS_WDTYPE_FP16 = 0, 1
LS_NORM_RMS, LS_NORM_NONE = 0, 1

EXPORTS = [
    "ls_layer_create", "ls_layer_destroy", "ls_predict", "ls_sparse_ffn_step", "ls_cache_lookup", "ls_cache_reserve",
    "ls_cache_evict", "ls_cache_snapshot", "ls_cache_wait", "ls_cache_stats", "ls_layer_status", "ls_kernel_launches",
    "ls_last_error", "ls_version", "ls_timing_enable", "ls_timing_read", "ls_set_option", "ls_topk_select_static", "ls_stack_create",
    "ls_stack_destroy", "ls_stack_decode", "ls_controller_quantize", "ls_controller_build", "ls_hash_predictor_create",
    "ls_hash_predictor_destroy", "ls_hash_predict",
]


class LeanStreamError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"leanstream error {code}: {msg}")
        self.code = code


class ls_layer_desc(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("device", C.c_int32), ("d_model", C.c_int32), ("d_ff", C.c_int32),
        ("gated", C.c_int32), ("act", C.c_int32), ("wdtype", C.c_int32), ("norm", C.c_int32), ("norm_eps", C.c_float),
        ("pred_rank", C.c_int32), ("w_gate", C.c_void_p), ("w_up", C.c_void_p), ("w_down_t", C.c_void_p),
        ("b_gate", C.c_void_p), ("b_down", C.c_void_p), ("pred_a", C.c_void_p), ("pred_b", C.c_void_p),
        ("pred_c", C.c_void_p), ("cache_rows", C.c_int64), ("max_batch", C.c_int32), ("max_sel", C.c_int32),
    ]


class ls_selection(C.Structure):
    _fields_ = [("scores", C.c_void_p), ("mask", C.c_void_p), ("idx", C.c_void_p), ("count", C.c_void_p), ("cap", C.c_int32)]


class ls_step_trace(C.Structure):
    _fields_ = [("xtilde", C.c_void_p), ("refine_masks", C.c_void_p), ("refine_counts", C.c_void_p),
                ("survive_mask", C.c_void_p), ("exec_idx", C.c_void_p)]


class ls_stack_trace(C.Structure):
    _fields_ = [("x", C.c_void_p), ("sel_idx", C.c_void_p), ("sel_count", C.c_void_p), ("sel_cap", C.c_int32),
                ("xtilde", C.c_void_p), ("refine_masks", C.c_void_p), ("mask_words", C.c_int32), ("phase_ns", C.c_void_p)]


LS_STACK_NSTAMP = 12


class ls_hash_predictor_desc(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("device", C.c_int32), ("d_model", C.c_int32), ("rank", C.c_int32), ("tau", C.c_int32),
                ("d_code", C.c_int32), ("n_layers", C.c_int32), ("d_ff", C.c_int32), ("wdtype", C.c_int32), ("pca", C.c_void_p),
                ("w1", C.c_void_p), ("w", C.c_void_p), ("tables", C.c_void_p), ("codes", C.c_void_p)]


class ls_cache_stats_t(C.Structure):
    _fields_ = [("hits", C.c_int64), ("misses", C.c_int64), ("evictions", C.c_int64), ("h2d_bytes", C.c_int64),
                ("h2d_copies", C.c_int64), ("resident", C.c_int64)]


_lib = None


def lib() -> C.CDLL:
    """The loaded shared library (built in-tree on first use when nvcc is available)."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            path = _build.build_library()
        try:
            L = C.CDLL(path)
        except OSError as e:  # no fallback: the CUDA library is the product
            raise RuntimeError(f"cannot load {path}: {e}") from e
        L.ls_layer_create.argtypes = [C.POINTER(ls_layer_desc), C.POINTER(C.c_void_p)]
        L.ls_layer_destroy.argtypes = [C.c_void_p]
        L.ls_predict.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.POINTER(ls_selection), C.c_void_p]
        L.ls_sparse_ffn_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(ls_selection),
                                         C.c_int32, C.c_int32, C.POINTER(ls_selection), C.POINTER(ls_step_trace), C.c_void_p]
        L.ls_cache_lookup.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ls_cache_reserve.argtypes = [C.c_void_p, C.POINTER(ls_selection), C.c_int32, C.c_void_p, C.POINTER(C.c_int32), C.c_void_p]
        L.ls_cache_evict.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ls_cache_snapshot.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.ls_cache_wait.argtypes = [C.c_void_p, C.c_void_p]
        L.ls_cache_stats.argtypes = [C.c_void_p, C.POINTER(ls_cache_stats_t)]
        L.ls_layer_status.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
        L.ls_set_option.argtypes = [C.c_int32, C.c_int32]
        L.ls_stack_create.argtypes = [C.POINTER(C.c_void_p), C.c_int32, C.POINTER(C.c_void_p)]
        L.ls_stack_destroy.argtypes = [C.c_void_p]
        L.ls_stack_decode.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(ls_selection), C.c_int32, C.c_int32,
                                      C.POINTER(ls_selection), C.POINTER(ls_stack_trace), C.c_void_p]
        L.ls_topk_select_static.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ls_hash_predictor_create.argtypes = [C.POINTER(ls_hash_predictor_desc), C.POINTER(C.c_void_p)]
        L.ls_hash_predictor_destroy.argtypes = [C.c_void_p]
        L.ls_hash_predict.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(ls_selection), C.c_void_p, C.c_void_p]
        L.ls_controller_quantize.argtypes = [C.c_double, C.c_double, C.c_int32]
        L.ls_controller_build.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ls_timing_enable.argtypes = [C.c_int32]
        L.ls_timing_read.argtypes = [C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_double)]
        L.ls_kernel_launches.restype = C.c_int64
        L.ls_last_error.argtypes = [C.c_char_p, C.c_size_t]
        L.ls_last_error.restype = C.c_size_t
        for name in EXPORTS:
            if name not in ("ls_kernel_launches", "ls_last_error"):
                getattr(L, name).restype = C.c_int32
        _lib = L
    return _lib


def last_error() -> str:
    buf = C.create_string_buffer(1024)
    lib().ls_last_error(buf, 1024)
    return buf.value.decode(errors="replace")


def _check(rc: int) -> None:
    if rc != LS_OK:
        raise LeanStreamError(rc, last_error())


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


class Layer:
    """Owner of one ``ls_layer*`` handle."""

    def __init__(self, handle: int, d_model: int, d_ff: int, device: int, cache_rows: int, max_batch: int, max_sel: int):
        self.handle = handle
        self.d_model, self.d_ff, self.device = d_model, d_ff, device
        self.cache_rows, self.max_batch, self.max_sel = cache_rows, max_batch, max_sel
        self.nwords = (d_ff + 31) // 32

    def close(self) -> None:
        if self.handle:
            lib().ls_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Selection:
    """Device buffers of an ``ls_selection`` (scores fp64 [d_ff], mask [ceil(d_ff/32)], idx [cap], count [1])."""

    def __init__(self, d_ff: int, cap: int, device, with_scores: bool = True, with_mask: bool = True):
        dev = torch.device("cuda", device) if isinstance(device, int) else device
        self.scores = torch.zeros(d_ff, dtype=torch.float64, device=dev) if with_scores else None
        self.mask = torch.zeros((d_ff + 31) // 32, dtype=torch.int32, device=dev) if with_mask else None
        self.idx = torch.full((max(cap, 1),), -1, dtype=torch.int32, device=dev)
        self.count = torch.zeros(1, dtype=torch.int32, device=dev)
        self.cap = cap
        self.c = ls_selection(_ptr(self.scores), _ptr(self.mask), _ptr(self.idx), _ptr(self.count), cap)

    def order(self) -> np.ndarray:
        n = int(self.count.item())
        return self.idx[:n].cpu().numpy().astype(np.int64)

    def mask_np(self) -> np.ndarray:
        return self.mask.cpu().numpy().view(np.uint32)


class StepTrace:
    """Device buffers of an ``ls_step_trace``."""

    def __init__(self, layer: Layer, nxt: Optional[Layer], n_chunks: int, batch: int, sel_cap: int):
        dev = torch.device("cuda", layer.device)
        self.xtilde = torch.zeros(n_chunks + 1, batch, layer.d_model, dtype=torch.float32, device=dev)
        self.refine_masks = self.refine_counts = None
        if nxt is not None:
            self.refine_masks = torch.zeros(n_chunks + 1, nxt.nwords, dtype=torch.int32, device=dev)
            self.refine_counts = torch.zeros(n_chunks + 1, dtype=torch.int32, device=dev)
        self.survive_mask = torch.zeros(layer.nwords, dtype=torch.int32, device=dev)
        self.exec_idx = torch.full((max(sel_cap, 1),), -1, dtype=torch.int32, device=dev)
        self.c = ls_step_trace(_ptr(self.xtilde), _ptr(self.refine_masks), _ptr(self.refine_counts), _ptr(self.survive_mask),
                               _ptr(self.exec_idx))


def _host16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("16-bit weights must be passed as raw uint16 bit patterns")
    return a


def ls_layer_create(arrays, device: int = 0, cache_rows: int = 0, max_batch: int = 1, max_sel: int = 0,
                    norm: int = LS_NORM_RMS) -> Layer:
    """Create a layer from host arrays (attributes as produced by the workload module)."""
    keep = []

    def h16(a):
        if a is None:
            return None
        a = _host16(a)
        keep.append(a)
        return a.ctypes.data

    def hf32(a):
        if a is None:
            return None
        a = np.ascontiguousarray(a, dtype=np.float32)
        keep.append(a)
        return a.ctypes.data

    d = ls_layer_desc()
    d.struct_size = C.sizeof(ls_layer_desc)
    d.device = device
    d.d_model, d.d_ff = arrays.d_model, arrays.d_ff
    d.gated = 1 if arrays.gated else 0
    d.act = LS_ACT_SILU if getattr(arrays, "act", "relu") == "silu" else LS_ACT_RELU
    d.wdtype = LS_WDTYPE_BF16 if arrays.wdtype == "bf16" else LS_WDTYPE_FP16
    d.norm = norm
    d.norm_eps = float(arrays.norm_eps)
    d.pred_rank = arrays.rank
    d.w_gate, d.w_up, d.w_down_t = h16(arrays.w_gate), h16(arrays.w_up), h16(arrays.w_down_t)
    d.b_gate, d.b_down = hf32(arrays.b_gate), hf32(arrays.b_down)
    d.pred_a, d.pred_b, d.pred_c = h16(arrays.pred_a), h16(arrays.pred_b), hf32(arrays.pred_c)
    d.cache_rows = cache_rows
    d.max_batch, d.max_sel = max_batch, max_sel
    out = C.c_void_p()
    _check(lib().ls_layer_create(C.byref(d), C.byref(out)))
    return Layer(out.value, arrays.d_model, arrays.d_ff, device, cache_rows, max(1, max_batch), max_sel or arrays.d_ff)


def ls_layer_destroy(layer: Layer) -> None:
    layer.close()


def ls_predict(layer: Layer, feature: torch.Tensor, k: int, out: Selection, stream=None) -> Selection:
    assert feature.dtype == torch.float32 and feature.is_cuda and feature.is_contiguous()
    batch = 1 if feature.dim() == 1 else feature.shape[0]
    _check(lib().ls_predict(layer.handle, feature.data_ptr(), batch, k, C.byref(out.c), _stream(stream)))
    return out


def ls_sparse_ffn_step(layer: Layer, nxt: Optional[Layer], x: torch.Tensor, x_out: torch.Tensor, sel: Selection, n_chunks: int,
                       k_next: int = 0, sel_next: Optional[Selection] = None, trace: Optional[StepTrace] = None, stream=None) -> None:
    assert x.dtype == torch.float32 and x.is_cuda and x.is_contiguous() and x_out.is_contiguous()
    batch = 1 if x.dim() == 1 else x.shape[0]
    _check(lib().ls_sparse_ffn_step(layer.handle, None if nxt is None else nxt.handle, x.data_ptr(), x_out.data_ptr(), batch,
                                    C.byref(sel.c), n_chunks, k_next, None if sel_next is None else C.byref(sel_next.c),
                                    None if trace is None else C.byref(trace.c), _stream(stream)))


def ls_cache_lookup(layer: Layer, idx: torch.Tensor, slot: torch.Tensor, nhit: Optional[torch.Tensor] = None, stream=None) -> None:
    _check(lib().ls_cache_lookup(layer.handle, idx.data_ptr(), idx.numel(), slot.data_ptr(), _ptr(nhit), _stream(stream)))


def ls_cache_reserve(layer: Layer, want: Selection, admit_ranks: int = -1, protect_mask: Optional[torch.Tensor] = None,
                     stream=None) -> int:
    n = C.c_int32(0)
    _check(lib().ls_cache_reserve(layer.handle, C.byref(want.c), admit_ranks, _ptr(protect_mask), C.byref(n), _stream(stream)))
    return n.value


def ls_cache_evict(layer: Layer, min_free: int, protect_mask: Optional[torch.Tensor] = None, evicted: Optional[torch.Tensor] = None,
                   nevicted: Optional[torch.Tensor] = None, stream=None) -> None:
    _check(lib().ls_cache_evict(layer.handle, min_free, _ptr(protect_mask), _ptr(evicted), _ptr(nevicted), _stream(stream)))


def ls_cache_snapshot(layer: Layer, resident_mask: torch.Tensor, stream=None) -> None:
    _check(lib().ls_cache_snapshot(layer.handle, resident_mask.data_ptr(), _stream(stream)))


def ls_cache_wait(layer: Layer, stream=None) -> None:
    _check(lib().ls_cache_wait(layer.handle, _stream(stream)))


def ls_cache_stats(layer: Layer) -> dict:
    s = ls_cache_stats_t()
    _check(lib().ls_cache_stats(layer.handle, C.byref(s)))
    return {k: getattr(s, k) for k, _ in ls_cache_stats_t._fields_}


def ls_layer_status(layer: Layer) -> int:
    v = C.c_int32(0)
    _check(lib().ls_layer_status(layer.handle, C.byref(v)))
    return v.value


def ls_kernel_launches() -> int:
    return int(lib().ls_kernel_launches())


def ls_version() -> int:
    return int(lib().ls_version())


LS_TIMED_GATEUP, LS_TIMED_DOWN, LS_TIMED_PREDICT, LS_TIMED_FUSED, LS_TIMED_STACK = 0, 1, 2, 3, 4


def ls_timing_enable(on: bool) -> None:
    _check(lib().ls_timing_enable(1 if on else 0))


def ls_timing_read(kind: int):
    """(launches, total_ms) of the events recorded for one kernel group since the last read."""
    n, ms = C.c_int64(0), C.c_double(0.0)
    _check(lib().ls_timing_read(kind, C.byref(n), C.byref(ms)))
    return n.value, ms.value


LS_OPT_FUSED, LS_OPT_MISS_PATH, LS_OPT_HOST_WAIT_MS = 1, 2, 3
LS_MISS_PATH_LANE, LS_MISS_PATH_GATHER = 0, 1


def ls_set_option(option: int, value: int) -> None:
    _check(lib().ls_set_option(option, value))


LS_STATIC_TOPK_MAX_N = 32768


def ls_topk_select_static(scores: torch.Tensor, k: int, idx: torch.Tensor, mask: Optional[torch.Tensor], count: torch.Tensor,
                          stream=None) -> None:
    """Top-k of a caller-provided fp64 device array without any allocation inside the library (for callers that must
    not allocate: stream capture, allocator-free serving loops).  Outputs go to the caller's tensors."""
    assert scores.dtype == torch.float64 and scores.is_cuda and scores.is_contiguous()
    _check(lib().ls_topk_select_static(scores.data_ptr(), scores.numel(), k, idx.data_ptr(), _ptr(mask), count.data_ptr(),
                                       _stream(stream)))


class Stack:
    """Owner of one ``ls_stack*`` handle (keeps its layers alive)."""

    def __init__(self, handle: int, layers):
        self.handle = handle
        self.layers = list(layers)

    def close(self) -> None:
        if self.handle:
            lib().ls_stack_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class StackTrace:
    """Device buffers of an ``ls_stack_trace``: residuals and selections at every layer boundary and, when ``n_chunks``
    is given, every partial residual feature and refined set; ``phases=True`` adds the per-CTA phase time stamps."""

    def __init__(self, stack: Stack, sel_cap: int, n_chunks: int = 0, phases: bool = False):
        L0 = stack.layers[0]
        dev = torch.device("cuda", L0.device)
        n = len(stack.layers)
        self.x = torch.zeros(n + 1, L0.d_model, dtype=torch.float32, device=dev)
        self.sel_idx = torch.full((n + 1, max(sel_cap, 1)), -1, dtype=torch.int32, device=dev)
        self.sel_count = torch.zeros(n + 1, dtype=torch.int32, device=dev)
        self.xtilde = self.refine_masks = self.phase_ns = None
        self.mask_words = max(L.nwords for L in stack.layers)
        if n_chunks > 0:
            self.xtilde = torch.zeros(n, n_chunks + 1, L0.d_model, dtype=torch.float32, device=dev)
            self.refine_masks = torch.zeros(n, n_chunks + 1, self.mask_words, dtype=torch.int32, device=dev)
        if phases:
            sms = torch.cuda.get_device_properties(dev).multi_processor_count
            self.phase_ns = torch.zeros(n, sms, LS_STACK_NSTAMP, dtype=torch.int64, device=dev)
        self.c = ls_stack_trace(_ptr(self.x), _ptr(self.sel_idx), _ptr(self.sel_count), sel_cap, _ptr(self.xtilde),
                                _ptr(self.refine_masks), self.mask_words, _ptr(self.phase_ns))


def ls_stack_create(layers) -> Stack:
    arr = (C.c_void_p * len(layers))(*[L.handle for L in layers])
    out = C.c_void_p()
    _check(lib().ls_stack_create(arr, len(layers), C.byref(out)))
    return Stack(out.value, layers)


def ls_stack_destroy(stack: Stack) -> None:
    stack.close()


def ls_stack_decode(stack: Stack, x: torch.Tensor, x_out: torch.Tensor, sel_first: Selection, n_chunks: int, k_next: int,
                    sel_out: Selection, trace: Optional[StackTrace] = None, stream=None) -> None:
    assert x.dtype == torch.float32 and x.is_cuda and x.is_contiguous() and x_out.is_contiguous()
    _check(lib().ls_stack_decode(stack.handle, x.data_ptr(), x_out.data_ptr(), C.byref(sel_first.c), n_chunks, k_next,
                                 C.byref(sel_out.c), None if trace is None else C.byref(trace.c), _stream(stream)))


def ls_controller_quantize(remaining: float, vmax: float, n_states: int) -> int:
    rc = lib().ls_controller_quantize(remaining, vmax, n_states)
    if rc < 0:
        _check(rc)
    return rc


def ls_controller_build(t_bar: np.ndarray, next_state: np.ndarray, horizon: int):
    """(lut [n_layers, n_states] int32, value [n_layers, n_states]) from host arrays t_bar [N, Q, A] and next_state [N, Q, A, S]."""
    t = np.ascontiguousarray(t_bar, dtype=np.float64)
    ns = np.ascontiguousarray(next_state, dtype=np.int32)
    N, Q, A = t.shape
    S = ns.shape[3] if ns.ndim == 4 else 0
    lut = np.full((N, Q), -2, dtype=np.int32)
    val = np.zeros((N, Q), dtype=np.float64)
    _check(lib().ls_controller_build(N, Q, A, S, horizon, t.ctypes.data, ns.ctypes.data if S else None, lut.ctypes.data, val.ctypes.data))
    return lut, val


class HashPredictor:
    """Owner of one ``ls_hash_predictor*`` handle."""

    def __init__(self, handle: int, d_ff: int, n_layers: int, device: int):
        self.handle, self.d_ff, self.n_layers, self.device = handle, d_ff, n_layers, device

    def close(self) -> None:
        if self.handle:
            lib().ls_hash_predictor_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def ls_hash_predictor_create(arrays, device: int = 0) -> HashPredictor:
    """Create from host arrays (attributes as produced by ``workload.make_hash_predictor``: packed sign bits)."""
    keep = [np.ascontiguousarray(arrays.pca), np.ascontiguousarray(arrays.w1, dtype=np.float32), np.ascontiguousarray(arrays.w_bits, dtype=np.uint32),
            np.ascontiguousarray(arrays.t_bits, dtype=np.uint32), np.ascontiguousarray(arrays.code_bits, dtype=np.uint32)]
    d = ls_hash_predictor_desc()
    d.struct_size = C.sizeof(ls_hash_predictor_desc)
    d.device = device
    d.d_model, d.rank, d.tau, d.d_code, d.n_layers, d.d_ff = arrays.d_model, arrays.rank, arrays.tau, arrays.d_code, arrays.n_layers, arrays.d_ff
    d.wdtype = LS_WDTYPE_BF16 if arrays.wdtype == "bf16" else LS_WDTYPE_FP16
    d.pca, d.w1 = keep[0].ctypes.data, keep[1].ctypes.data
    d.w = keep[2].ctypes.data if arrays.n_layers > 1 else None
    d.tables, d.codes = keep[3].ctypes.data, keep[4].ctypes.data
    out = C.c_void_p()
    _check(lib().ls_hash_predictor_create(C.byref(d), C.byref(out)))
    return HashPredictor(out.value, arrays.d_ff, arrays.n_layers, device)


def ls_hash_predict(pred: HashPredictor, feature: torch.Tensor, k: int, out: Selection, layer_idx: Optional[torch.Tensor] = None,
                    stream=None) -> Selection:
    assert feature.dtype == torch.float32 and feature.is_cuda and feature.is_contiguous()
    _check(lib().ls_hash_predict(pred.handle, feature.data_ptr(), k, C.byref(out.c), _ptr(layer_idx), _stream(stream)))
    return out
