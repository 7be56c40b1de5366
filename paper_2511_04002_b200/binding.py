"""Thin ctypes binding of the tsq C ABI (include/tsq.h): argument marshalling only.

Every step of encode and decode runs inside the CUDA library; torch is used for device
memory and streams.  Function names mirror the C entry points.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence, Tuple

import torch

F16, BF16 = 0, 1
STATUS = {0: "TSQ_OK", 1: "TSQ_ERR_INVALID_ARG", 2: "TSQ_ERR_UNSUPPORTED", 3: "TSQ_ERR_BUFFER_TOO_SMALL",
          4: "TSQ_ERR_CUDA", 5: "TSQ_ERR_CORRUPT_BLOB", 6: "TSQ_ERR_OUTLIER_OVERFLOW", 7: "TSQ_ERR_TIMEOUT"}

VARIANT_MAGNITUDES, VARIANT_SIGNED_VALUES = 0, 1

EXPORTS = ["tsq_plan", "tsq_plan_variant", "tsq_plan_sizes", "tsq_workspace_init", "tsq_workspace_set_wait_limit", "tsq_encode", "tsq_encode_noalloc", "tsq_decode",
           "tsq_blob_info",
           "tsq_workspace_status", "tsq_encode_host", "tsq_decode_host", "tsq_kernel_launch_count",
           "tsq_plan_destroy", "tsq_status_string",
           "tsq_model_kv_bits", "tsq_model_io_bits", "tsq_model_outage", "tsq_model_latency", "tsq_model_best_rate"]

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libtsq.so")
_lib: Optional[C.CDLL] = None


class TsqError(RuntimeError):
    def __init__(self, status: int, where: str):
        super().__init__("%s failed: %s (%d)" % (where, STATUS.get(status, "?"), status))
        self.status = status


class _Sizes(C.Structure):
    _fields_ = [("blob_bytes", C.c_size_t), ("workspace_bytes", C.c_size_t)]


class _Info(C.Structure):
    _fields_ = [("status", C.c_uint32), ("tokens", C.c_uint32), ("hidden", C.c_uint32), ("dtype", C.c_uint32),
                ("total_words", C.c_uint64), ("total_outliers", C.c_uint64), ("payload_bytes", C.c_uint64)]


def lib() -> C.CDLL:
    """Load libtsq.so. Raises if it has not been built: there is no fallback path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError("tsq CUDA library missing at %s; run `python -m paper_2511_04002_b200.build` "
                           "(needs nvcc). No CPU fallback exists." % _LIB_PATH)
    L = C.CDLL(_LIB_PATH)
    vp, i64, sz = C.c_void_p, C.c_int64, C.c_size_t
    L.tsq_plan.argtypes = [C.POINTER(vp), C.c_int, C.c_int, C.c_int32, i64, C.c_float, C.POINTER(C.c_int32),
                           C.c_int32, C.c_float, i64]
    L.tsq_plan_variant.argtypes = L.tsq_plan.argtypes + [C.c_int32]
    L.tsq_plan_sizes.argtypes = [vp, i64, C.POINTER(_Sizes)]
    L.tsq_workspace_init.argtypes = [vp, vp, sz, vp]
    L.tsq_workspace_set_wait_limit.argtypes = [vp, C.c_uint32, vp]
    L.tsq_encode.argtypes = [vp, vp, i64, vp, sz, vp, sz, vp]
    L.tsq_encode_noalloc.argtypes = [vp, vp, i64, vp, sz, vp]
    L.tsq_encode_noalloc.restype = C.c_int
    L.tsq_decode.argtypes = [vp, vp, sz, i64, vp, vp, sz, vp]
    L.tsq_blob_info.argtypes = [vp, C.POINTER(_Info), vp]
    L.tsq_workspace_status.argtypes = [vp, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), vp]
    L.tsq_encode_host.argtypes = [vp, vp, i64, vp, sz, C.POINTER(C.c_uint64), vp, vp, vp, sz, vp]
    L.tsq_decode_host.argtypes = [vp, vp, sz, i64, vp, vp, vp, vp, sz, vp]
    for name in ("tsq_plan", "tsq_plan_variant", "tsq_plan_sizes", "tsq_workspace_init", "tsq_workspace_set_wait_limit", "tsq_encode", "tsq_decode", "tsq_blob_info",
                 "tsq_workspace_status", "tsq_encode_host", "tsq_decode_host"):
        getattr(L, name).restype = C.c_int
    d, i32 = C.c_double, C.c_int32
    L.tsq_model_kv_bits.argtypes = [i64, i32, i32, i32, i64, d, d]
    L.tsq_model_io_bits.argtypes = [i64, i32, i32, i32, i64, d, d, i32]
    L.tsq_model_outage.argtypes = [d, d, d]
    L.tsq_model_latency.argtypes = [d, d, d, d, d]
    L.tsq_model_best_rate.argtypes = [d, d, d, d]
    for name in ("tsq_model_kv_bits", "tsq_model_io_bits", "tsq_model_outage", "tsq_model_latency", "tsq_model_best_rate"):
        getattr(L, name).restype = d
    L.tsq_kernel_launch_count.argtypes = []
    L.tsq_kernel_launch_count.restype = C.c_uint64
    L.tsq_plan_destroy.argtypes = [vp]
    L.tsq_plan_destroy.restype = None
    L.tsq_status_string.argtypes = [C.c_int]
    L.tsq_status_string.restype = C.c_char_p
    _lib = L
    return L


def _check(status: int, where: str) -> None:
    if status != 0:
        raise TsqError(status, where)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float16:
        return F16
    if dt == torch.bfloat16:
        return BF16
    raise TypeError("tsq handles float16 and bfloat16, got %s" % dt)


@dataclass
class BlobInfo:
    status: int
    tokens: int
    hidden: int
    dtype: int
    total_words: int
    total_outliers: int
    payload_bytes: int


class Plan:
    """tsq_plan_t wrapper. Methods are the C calls of the same name with pointers filled in."""

    def __init__(self, dtype: torch.dtype, hidden: int, max_tokens: int, tau: float, bits: Sequence[int],
                 delta: float = 0.2, max_outliers: int = 0, device: int = 0, variant: int = VARIANT_MAGNITUDES):
        self._h = C.c_void_p()
        arr = (C.c_int32 * len(bits))(*bits)
        if variant == VARIANT_MAGNITUDES:
            st = lib().tsq_plan(C.byref(self._h), device, dtype_code(dtype), hidden, max_tokens, tau, arr, len(bits),
                                delta, max_outliers)
        else:
            st = lib().tsq_plan_variant(C.byref(self._h), device, dtype_code(dtype), hidden, max_tokens, tau, arr,
                                        len(bits), delta, max_outliers, variant)
        _check(st, "tsq_plan")
        self.variant = variant
        self.dtype, self.hidden, self.max_tokens, self.device = dtype, hidden, max_tokens, device
        self.tau, self.bits, self.delta, self.max_outliers = tau, tuple(bits), delta, max_outliers

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h and _lib is not None:
            _lib.tsq_plan_destroy(h)

    def sizes(self, tokens: int) -> Tuple[int, int]:
        s = _Sizes()
        _check(lib().tsq_plan_sizes(self._h, tokens, C.byref(s)), "tsq_plan_sizes")
        return int(s.blob_bytes), int(s.workspace_bytes)

    def alloc(self, tokens: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor]:
        """Allocate (blob, workspace) with torch on the plan's device and initialise the workspace."""
        tokens = self.max_tokens if tokens is None else tokens
        blob_bytes, ws_bytes = self.sizes(tokens)
        dev = torch.device("cuda", self.device)
        blob = torch.empty(blob_bytes, dtype=torch.uint8, device=dev)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        self.workspace_init(ws)
        return blob, ws

    def workspace_init(self, ws: torch.Tensor, stream=None) -> None:
        _check(lib().tsq_workspace_init(self._h, ws.data_ptr(), ws.numel(), _stream(stream)), "tsq_workspace_init")

    def workspace_set_wait_limit(self, ws: torch.Tensor, polls: int, stream=None) -> None:
        _check(lib().tsq_workspace_set_wait_limit(ws.data_ptr(), polls, _stream(stream)), "tsq_workspace_set_wait_limit")

    def encode(self, x: torch.Tensor, blob: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
        assert x.is_cuda and x.is_contiguous() and x.dtype == self.dtype and x.dim() == 2 and x.shape[1] == self.hidden
        _check(lib().tsq_encode(self._h, x.data_ptr(), x.shape[0], blob.data_ptr(), blob.numel(), ws.data_ptr(),
                                ws.numel(), _stream(stream)), "tsq_encode")

    def encode_noalloc(self, x: torch.Tensor, blob: torch.Tensor, stream=None) -> None:
        """tsq_encode_noalloc: encode with the library's built-in scratch array instead of a workspace."""
        assert x.is_cuda and x.is_contiguous() and x.dtype == self.dtype and x.dim() == 2 and x.shape[1] == self.hidden
        _check(lib().tsq_encode_noalloc(self._h, x.data_ptr(), x.shape[0], blob.data_ptr(), blob.numel(),
                                        _stream(stream)), "tsq_encode_noalloc")

    def decode(self, blob: torch.Tensor, tokens: int, y: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
        assert y.is_cuda and y.is_contiguous() and y.dtype == self.dtype and tuple(y.shape) == (tokens, self.hidden)
        _check(lib().tsq_decode(self._h, blob.data_ptr(), blob.numel(), tokens, y.data_ptr(), ws.data_ptr(),
                                ws.numel(), _stream(stream)), "tsq_decode")

    def blob_info(self, blob: torch.Tensor, stream=None) -> BlobInfo:
        i = _Info()
        _check(lib().tsq_blob_info(blob.data_ptr(), C.byref(i), _stream(stream)), "tsq_blob_info")
        return BlobInfo(i.status, i.tokens, i.hidden, i.dtype, i.total_words, i.total_outliers, i.payload_bytes)

    def workspace_status(self, ws: torch.Tensor, stream=None) -> Tuple[int, int]:
        e, d = C.c_uint32(0), C.c_uint32(0)
        _check(lib().tsq_workspace_status(ws.data_ptr(), C.byref(e), C.byref(d), _stream(stream)),
               "tsq_workspace_status")
        return int(e.value), int(d.value)

    def encode_host(self, x_host: torch.Tensor, blob_host: torch.Tensor, x_dev: torch.Tensor, blob_dev: torch.Tensor,
                    ws: torch.Tensor, stream=None) -> int:
        """Host tensor in, host blob out (copies inside). Returns the payload size in bytes."""
        assert not x_host.is_cuda and x_host.is_contiguous() and x_host.dtype == self.dtype
        payload = C.c_uint64(0)
        st = lib().tsq_encode_host(self._h, x_host.data_ptr(), x_host.shape[0], blob_host.data_ptr(),
                                   blob_host.numel(), C.byref(payload), x_dev.data_ptr(), blob_dev.data_ptr(),
                                   ws.data_ptr(), ws.numel(), _stream(stream))
        _check(st, "tsq_encode_host")
        return int(payload.value)

    def decode_host(self, blob_host: torch.Tensor, tokens: int, y_host: torch.Tensor, blob_dev: torch.Tensor,
                    y_dev: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
        assert not y_host.is_cuda and y_host.is_contiguous() and y_host.dtype == self.dtype
        st = lib().tsq_decode_host(self._h, blob_host.data_ptr(), blob_host.numel(), tokens, y_host.data_ptr(),
                                   blob_dev.data_ptr(), y_dev.data_ptr(), ws.data_ptr(), ws.numel(),
                                   _stream(stream))
        _check(st, "tsq_decode_host")


def model_kv_bits(w, layer, n_layers, split_layer, hd, qa_front, qa_back) -> float:
    return float(lib().tsq_model_kv_bits(w, layer, n_layers, split_layer, hd, qa_front, qa_back))


def model_io_bits(w, layer, n_layers, split_layer, hd, qa_front, qa_back, send_kv) -> float:
    return float(lib().tsq_model_io_bits(w, layer, n_layers, split_layer, hd, qa_front, qa_back, 1 if send_kv else 0))


def model_outage(rate, bandwidth, snr) -> float:
    return float(lib().tsq_model_outage(rate, bandwidth, snr))


def model_latency(bits, rate, bandwidth, snr, epsilon) -> float:
    return float(lib().tsq_model_latency(bits, rate, bandwidth, snr, epsilon))


def model_best_rate(rate_lo, rate_hi, bandwidth, snr) -> float:
    return float(lib().tsq_model_best_rate(rate_lo, rate_hi, bandwidth, snr))


def kernel_launch_count() -> int:
    return int(lib().tsq_kernel_launch_count())


def status_string(status: int) -> str:
    return lib().tsq_status_string(status).decode()
