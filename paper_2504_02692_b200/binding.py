"""ctypes binding of libgptaq.so: the same names as include/gptaq.h.

Argument marshalling only -- every arithmetic step of the solve runs in the
library's CUDA kernels.  torch is used for device memory and streams.  There
is no CPU fallback: if the shared library is missing or no CUDA device is
present, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgptaq.so")

GPTAQ_OK = 0
GPTAQ_ERR_INVALID_ARG = 1
GPTAQ_ERR_BAD_STATE = 2
GPTAQ_ERR_WORKSPACE = 3
GPTAQ_ERR_NOT_SPD = 4
GPTAQ_ERR_NONFINITE = 5
GPTAQ_ERR_TIMEOUT = 6
GPTAQ_ERR_UNSUPPORTED = 7
GPTAQ_ERR_CUDA = 8
GPTAQ_W_FP32 = 0
GPTAQ_W_BF16 = 1
GPTAQ_STATS_FP16_TENSOR = 0
GPTAQ_STATS_FP32 = 1
GPTAQ_STATS_FP16_SPLIT_TENSOR = 2
GPTAQ_STATS_FP16_SPLIT_FULL_TENSOR = 3
GPTAQ_TERM_ERR = 1
GPTAQ_TERM_ASYM = 2

_vp, _i64, _int, _sz, _f = C.c_void_p, C.c_int64, C.c_int, C.c_size_t, C.c_float

# name -> (restype, argtypes); one entry per declaration in include/gptaq.h
SIGNATURES = {
    "gptaq_state_bytes": (_sz, [_i64]),
    "gptaq_workspace_bytes": (_sz, [_i64, _i64, _i64, _int]),
    "gptaq_create": (_int, [C.POINTER(_vp), _i64, _vp, _sz, _vp, _sz, _vp]),
    "gptaq_reset": (_int, [_vp, _vp]),
    "gptaq_destroy": (_int, [_vp]),
    "gptaq_accumulate": (_int, [_vp, _vp, _vp, _i64, _i64, _vp]),
    "gptaq_flush": (_int, [_vp, _vp]),
    "gptaq_accumulate_host": (_int, [_vp, _vp, _vp, _i64, _i64, _vp, _sz, _vp]),
    "gptaq_factor": (_int, [_vp, _f, _vp]),
    "gptaq_build_P": (_int, [_vp, _f, _vp]),
    "gptaq_build_P_rowwise": (_int, [_vp, _f, _vp]),
    "gptaq_quantize": (_int, [_vp, _vp, _int, _i64, _i64, _int, _int, _int, _int, _vp, _vp, _vp, _vp, _vp]),
    "gptaq_quantize_stage_bytes": (_sz, [_i64, _i64, _int]),
    "gptaq_quantize_host": (_int, [_vp, _vp, _i64, _i64, _int, _int, _int, _int, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "gptaq_quantize_static": (_int, [_vp, _vp, _i64, _vp, _int, _i64, _i64, _int, _int, _int, _int, _vp, _vp, _vp, _vp,
                                     _vp, _vp]),
    "gptaq_sync_status": (_int, [_vp, C.POINTER(_i64), _vp]),
    "gptaq_H": (_vp, [_vp]),
    "gptaq_D": (_vp, [_vp]),
    "gptaq_U": (_vp, [_vp]),
    "gptaq_P": (_vp, [_vp]),
    "gptaq_selftest_bounded_wait": (_int, [_vp, C.c_double, _vp]),
    "gptaq_tokens": (_i64, [_vp]),
    "gptaq_set_tokens": (_int, [_vp, _i64]),
    "gptaq_set_stats_precision": (_int, [_vp, _int]),
    "gptaq_set_update_terms": (_int, [_vp, _int]),
    "gptaq_set_clip_search": (_int, [_vp, _int, _f]),
    "gptaq_set_act_order": (_int, [_vp, _int]),
    "gptaq_set_static_groups": (_int, [_vp, _int]),
    "gptaq_perm": (_vp, [_vp]),
    "gptaq_recommended_stats_precision": (_int, [_i64, _i64]),
    "gptaq_launch_count": (_i64, [_vp]),
    "gptaq_set_kernel_timing": (_int, [_vp, _int]),
    "gptaq_stats_kernel_time": (_int, [_vp, C.POINTER(C.c_double), C.POINTER(_i64)]),
    "gptaq_status_string": (C.c_char_p, [_int]),
    "gptaq_last_cuda_error": (C.c_char_p, [_vp]),
}

_lib = None


def load_library() -> C.CDLL:
    """Loads libgptaq.so (built in-tree by ``build.py``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2504_02692_b200.build` "
                "(there is no CPU fallback)")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


class GptaqError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        self.status = status
        text = load_library().gptaq_status_string(status).decode()
        super().__init__(f"{what}: {text} (status {status}){': ' + detail if detail else ''}")


def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    return int(t)


def _stream(stream) -> int | None:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream or None
    return int(stream) or None


def _check(status: int, what: str, handle=None):
    if status != GPTAQ_OK:
        detail = ""
        if handle is not None and status == GPTAQ_ERR_CUDA:
            detail = load_library().gptaq_last_cuda_error(handle).decode()
        raise GptaqError(status, what, detail)


def _need_cuda(*tensors):
    if not torch.cuda.is_available():
        raise RuntimeError("the GPTAQ kernels need a CUDA device (no CPU fallback)")
    for t in tensors:
        if t is not None and isinstance(t, torch.Tensor) and not t.is_cuda:
            raise ValueError("expected a CUDA tensor")


# ---------------------------------------------------------------- size queries
def gptaq_state_bytes(n: int) -> int:
    return load_library().gptaq_state_bytes(n)


def gptaq_workspace_bytes(n: int, m_max: int, max_batch_tokens: int, blocksize: int) -> int:
    return load_library().gptaq_workspace_bytes(n, m_max, max_batch_tokens, blocksize)


def gptaq_quantize_stage_bytes(m: int, n: int, group: int) -> int:
    return load_library().gptaq_quantize_stage_bytes(m, n, group)


# ---------------------------------------------------------------- handle
def gptaq_create(n: int, d_state: torch.Tensor, d_workspace: torch.Tensor, stream=None):
    _need_cuda(d_state, d_workspace)
    h = _vp()
    st = load_library().gptaq_create(C.byref(h), n, _ptr(d_state), d_state.numel() * d_state.element_size(),
                                     _ptr(d_workspace), d_workspace.numel() * d_workspace.element_size(),
                                     _stream(stream))
    _check(st, "gptaq_create")
    return h


def gptaq_reset(h, stream=None):
    _check(load_library().gptaq_reset(h, _stream(stream)), "gptaq_reset", h)


def gptaq_destroy(h):
    _check(load_library().gptaq_destroy(h), "gptaq_destroy")


# ---------------------------------------------------------------- the four steps
def gptaq_accumulate(h, d_X: torch.Tensor, d_Xfp: torch.Tensor, stream=None):
    """``d_X``, ``d_Xfp``: float32 CUDA tensors ``[tokens, n]`` with unit inner stride."""
    _need_cuda(d_X, d_Xfp)
    assert d_X.dtype == torch.float32 and d_Xfp.dtype == torch.float32
    assert d_X.shape == d_Xfp.shape and d_X.dim() == 2
    assert d_X.stride(1) == 1 and d_Xfp.stride(1) == 1 and d_X.stride(0) == d_Xfp.stride(0)
    tokens = d_X.shape[0]
    ld = d_X.stride(0) if tokens > 1 else max(d_X.shape[1], 1)
    st = load_library().gptaq_accumulate(h, _ptr(d_X), _ptr(d_Xfp), tokens, ld, _stream(stream))
    _check(st, "gptaq_accumulate", h)


def gptaq_flush(h, stream=None):
    """Orders ``stream`` after the statistics products that gptaq_accumulate left running."""
    _check(load_library().gptaq_flush(h, _stream(stream)), "gptaq_flush", h)


def gptaq_accumulate_host(h, h_X: torch.Tensor, h_Xfp: torch.Tensor, d_stage: torch.Tensor, stream=None):
    """Host (ideally pinned) float32 ``[tokens, n]`` inputs, staged through ``d_stage``."""
    _need_cuda(d_stage)
    assert not h_X.is_cuda and not h_Xfp.is_cuda and h_X.is_contiguous() and h_Xfp.is_contiguous()
    tokens, n = h_X.shape
    st = load_library().gptaq_accumulate_host(h, _ptr(h_X), _ptr(h_Xfp), tokens, n, _ptr(d_stage),
                                              d_stage.numel() * d_stage.element_size(), _stream(stream))
    _check(st, "gptaq_accumulate_host", h)


def gptaq_factor(h, damp: float, stream=None):
    _check(load_library().gptaq_factor(h, damp, _stream(stream)), "gptaq_factor", h)


def gptaq_build_P(h, alpha: float, stream=None):
    _check(load_library().gptaq_build_P(h, alpha, _stream(stream)), "gptaq_build_P", h)


def gptaq_build_P_rowwise(h, alpha: float, stream=None):
    """P row by row (the comparison form of the paper's latency discussion); same result as gptaq_build_P."""
    _check(load_library().gptaq_build_P_rowwise(h, alpha, _stream(stream)), "gptaq_build_P_rowwise", h)


def gptaq_quantize(h, d_W: torch.Tensor, bits: int, group: int, sym: bool, blocksize: int,
                   d_codes: torch.Tensor, d_scales: torch.Tensor, d_zeros: torch.Tensor,
                   d_Wq: torch.Tensor | None = None, stream=None):
    _need_cuda(d_W, d_codes, d_scales, d_zeros, d_Wq)
    assert d_W.dim() == 2 and d_W.stride(1) == 1
    dt = {torch.float32: GPTAQ_W_FP32, torch.bfloat16: GPTAQ_W_BF16}[d_W.dtype]
    m = d_W.shape[0]
    ldw = d_W.stride(0) if m > 1 else d_W.shape[1]
    assert d_codes.dtype == torch.uint8 and d_codes.is_contiguous()
    assert d_scales.dtype == torch.float32 and d_zeros.dtype == torch.float32
    if d_Wq is not None:
        assert d_Wq.dtype == torch.float32 and d_Wq.is_contiguous() and d_Wq.shape == d_W.shape
    st = load_library().gptaq_quantize(h, _ptr(d_W), dt, m, ldw, bits, group, int(bool(sym)), blocksize,
                                       _ptr(d_codes), _ptr(d_scales), _ptr(d_zeros), _ptr(d_Wq),
                                       _stream(stream))
    _check(st, "gptaq_quantize", h)


def gptaq_quantize_host(h, h_W: torch.Tensor, bits: int, group: int, sym: bool, blocksize: int,
                        h_codes: torch.Tensor, h_scales: torch.Tensor, h_zeros: torch.Tensor,
                        d_stage: torch.Tensor, h_Wq: torch.Tensor | None = None, stream=None):
    _need_cuda(d_stage)
    assert not h_W.is_cuda and h_W.is_contiguous() and h_W.dtype == torch.float32
    m, n = h_W.shape
    st = load_library().gptaq_quantize_host(h, _ptr(h_W), m, n, bits, group, int(bool(sym)), blocksize,
                                            _ptr(h_codes), _ptr(h_scales), _ptr(h_zeros), _ptr(h_Wq),
                                            _ptr(d_stage), d_stage.numel() * d_stage.element_size(),
                                            _stream(stream))
    _check(st, "gptaq_quantize_host", h)


GPTAQ_STATIC_MAX_N = 16384
GPTAQ_STATIC_SCRATCH_FLOATS = 1 << 20


def gptaq_quantize_static(d_U: torch.Tensor, d_P: torch.Tensor, d_W: torch.Tensor, bits: int, group: int,
                          sym: bool, blocksize: int, d_codes: torch.Tensor, d_scales: torch.Tensor,
                          d_zeros: torch.Tensor, d_Wq: torch.Tensor | None = None,
                          d_status: torch.Tensor | None = None, stream=None):
    """``gptaq_quantize`` without handle or workspace, for callers that may not allocate device
    memory: ``d_U`` / ``d_P`` are ``[n, n]`` float32 inputs and the scratch is an array built
    into the library (limits: ``n <= GPTAQ_STATIC_MAX_N``,
    ``m * 2 * blocksize <= GPTAQ_STATIC_SCRATCH_FLOATS``).  ``d_status``: optional int64[2]
    CUDA tensor that receives the device status and its index."""
    _need_cuda(d_U, d_P, d_W, d_codes, d_scales, d_zeros, d_Wq, d_status)
    n = d_U.shape[0]
    assert d_U.dtype == torch.float32 and d_P.dtype == torch.float32
    assert d_U.shape == (n, n) and d_P.shape == (n, n) and d_U.is_contiguous() and d_P.is_contiguous()
    assert d_W.dim() == 2 and d_W.stride(1) == 1 and d_W.shape[1] == n
    dt = {torch.float32: GPTAQ_W_FP32, torch.bfloat16: GPTAQ_W_BF16}[d_W.dtype]
    m = d_W.shape[0]
    ldw = d_W.stride(0) if m > 1 else d_W.shape[1]
    assert d_codes.dtype == torch.uint8 and d_codes.is_contiguous()
    assert d_scales.dtype == torch.float32 and d_zeros.dtype == torch.float32
    if d_Wq is not None:
        assert d_Wq.dtype == torch.float32 and d_Wq.is_contiguous() and d_Wq.shape == d_W.shape
    if d_status is not None:
        assert d_status.dtype == torch.int64 and d_status.numel() >= 2 and d_status.is_contiguous()
    st = load_library().gptaq_quantize_static(_ptr(d_U), _ptr(d_P), n, _ptr(d_W), dt, m, ldw, bits, group,
                                              int(bool(sym)), blocksize, _ptr(d_codes), _ptr(d_scales),
                                              _ptr(d_zeros), _ptr(d_Wq), _ptr(d_status), _stream(stream))
    if st == GPTAQ_ERR_WORKSPACE:
        raise GptaqError(st, "gptaq_quantize_static",
                         f"n = {n} (limit {GPTAQ_STATIC_MAX_N}) or m * 2 * blocksize = {m * 2 * blocksize} "
                         f"(limit {GPTAQ_STATIC_SCRATCH_FLOATS}) exceeds the built-in scratch")
    _check(st, "gptaq_quantize_static")


# ---------------------------------------------------------------- status and views
def gptaq_sync_status(h, stream=None):
    """Returns ``(status, info)`` after synchronising the stream."""
    info = _i64(0)
    st = load_library().gptaq_sync_status(h, C.byref(info), _stream(stream))
    return st, info.value


def gptaq_selftest_bounded_wait(h, seconds: float, stream=None):
    """Makes a bounded device-side wait run out on purpose; gptaq_sync_status then reports GPTAQ_ERR_TIMEOUT."""
    _check(load_library().gptaq_selftest_bounded_wait(h, seconds, _stream(stream)), "gptaq_selftest_bounded_wait", h)


def gptaq_tokens(h) -> int:
    return load_library().gptaq_tokens(h)


def gptaq_set_tokens(h, tokens: int):
    _check(load_library().gptaq_set_tokens(h, tokens), "gptaq_set_tokens", h)


def gptaq_set_stats_precision(h, precision: int):
    _check(load_library().gptaq_set_stats_precision(h, precision), "gptaq_set_stats_precision", h)


def gptaq_set_act_order(h, enable: bool):
    """Columns processed in order of decreasing diag(H); set before gptaq_factor."""
    _check(load_library().gptaq_set_act_order(h, int(bool(enable))), "gptaq_set_act_order", h)


def gptaq_set_static_groups(h, enable: bool):
    """Group grids from the original weights, per group of the caller's columns (they survive act_order)."""
    _check(load_library().gptaq_set_static_groups(h, int(bool(enable))), "gptaq_set_static_groups", h)


def gptaq_perm_ptr(h) -> int | None:
    return load_library().gptaq_perm(h)


def gptaq_set_clip_search(h, steps: int, min_ratio: float = 0.2):
    """Grids chosen by the least squared rounding error among ``steps`` shrunken min/max ranges (0: off)."""
    _check(load_library().gptaq_set_clip_search(h, steps, min_ratio), "gptaq_set_clip_search", h)


def gptaq_set_update_terms(h, terms: int):
    """Ablation switches: ``GPTAQ_TERM_ERR | GPTAQ_TERM_ASYM`` (default) = GPTAQ, ERR = GPTQ, ASYM = GPTAQ', 0 = RTN."""
    _check(load_library().gptaq_set_update_terms(h, terms), "gptaq_set_update_terms", h)


def gptaq_recommended_stats_precision(n: int, total_tokens: int) -> int:
    return load_library().gptaq_recommended_stats_precision(n, total_tokens)


def gptaq_launch_count(h) -> int:
    return load_library().gptaq_launch_count(h)


def gptaq_set_kernel_timing(h, enable: bool):
    """Brackets every launch of the statistics kernel with events on its own stream (see gptaq_stats_kernel_time)."""
    _check(load_library().gptaq_set_kernel_timing(h, int(bool(enable))), "gptaq_set_kernel_timing", h)


def gptaq_stats_kernel_time(h):
    """``(total ms, launches)`` of the statistics kernel since the last call; waits for those launches."""
    ms, n = C.c_double(0.0), _i64(0)
    _check(load_library().gptaq_stats_kernel_time(h, C.byref(ms), C.byref(n)), "gptaq_stats_kernel_time", h)
    return ms.value, n.value


def gptaq_status_string(status: int) -> str:
    return load_library().gptaq_status_string(status).decode()


def gptaq_H_ptr(h) -> int:
    return load_library().gptaq_H(h)


def gptaq_D_ptr(h) -> int:
    return load_library().gptaq_D(h)


class LayerState:
    """Owns the torch device buffers behind one handle (memory plumbing only)."""

    def __init__(self, n: int, m_max: int, max_batch_tokens: int, blocksize: int, device="cuda", stream=None,
                 total_tokens: int | None = None):
        _need_cuda()
        self.n = n
        self.device = torch.device(device)
        sb = gptaq_state_bytes(n)
        wb = gptaq_workspace_bytes(n, m_max, max_batch_tokens, blocksize)
        if sb == 0 or wb == 0:
            raise ValueError("bad sizes")
        self.state = torch.empty(sb, dtype=torch.uint8, device=self.device)
        self.workspace = torch.empty(wb, dtype=torch.uint8, device=self.device)
        self.handle = gptaq_create(n, self.state, self.workspace, stream)
        if total_tokens is not None:
            gptaq_set_stats_precision(self.handle, gptaq_recommended_stats_precision(n, total_tokens))

    def _view(self, ptr: int) -> torch.Tensor:
        off = ptr - self.state.data_ptr()
        nbytes = self.n * self.n * 4
        return self.state[off:off + nbytes].view(torch.float32).view(self.n, self.n)

    def H(self) -> torch.Tensor:
        """View of H (before factor) / U (after), ``[n, n]`` float32, current on torch's stream."""
        gptaq_flush(self.handle)
        return self._view(gptaq_H_ptr(self.handle))

    def D(self) -> torch.Tensor:
        """View of dXX^T (before build_P) / P (after), current on torch's stream."""
        gptaq_flush(self.handle)
        return self._view(gptaq_D_ptr(self.handle))

    def tokens(self) -> int:
        """Tokens accumulated so far (the divisor gptaq_factor will use)."""
        return gptaq_tokens(self.handle)

    def set_tokens(self, tokens: int):
        gptaq_set_tokens(self.handle, tokens)

    def perm(self) -> torch.Tensor | None:
        """act_order: int32 ``[n]``, sorted position -> caller column (None unless enabled and factored)."""
        ptr = gptaq_perm_ptr(self.handle)
        if not ptr:
            return None
        off = ptr - self.state.data_ptr()
        return self.state[off:off + 4 * self.n].view(torch.int32)

    def close(self):
        if self.handle is not None:
            gptaq_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
