"""ctypes front-end of the CPU oracle (oracle/tsq_ref.cpp).

Test infrastructure only.  All buffers are host numpy arrays; 16-bit tensors
travel as raw uint16 patterns so that no library conversion sits between the
test inputs and the oracle's own arithmetic.
"""
from __future__ import annotations

import ctypes as C
from typing import Dict, Sequence

import numpy as np

from . import build as _build

F16 = 0
BF16 = 1

STATUS_NAMES = {
    0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "BUFFER_TOO_SMALL", 4: "CUDA",
    5: "CORRUPT_BLOB", 6: "OUTLIER_OVERFLOW", 7: "TIMEOUT",
}

_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        u16p, u8p, f32p, i32p = (C.POINTER(C.c_uint16), C.POINTER(C.c_uint8), C.POINTER(C.c_float),
                                 C.POINTER(C.c_int32))
        L.tsq_ref_layout.argtypes = [C.c_int, C.c_longlong, C.c_int, C.c_longlong, C.POINTER(C.c_ulonglong)]
        L.tsq_ref_layout.restype = C.c_int
        L.tsq_ref_encode.argtypes = [C.c_int, C.c_int, C.c_longlong, C.c_float, i32p, C.c_int, C.c_float,
                                     C.c_longlong, u16p, u8p, C.c_ulonglong]
        L.tsq_ref_encode.restype = C.c_int
        L.tsq_ref_encode_ex.argtypes = [C.c_int, C.c_int, C.c_longlong, C.c_float, i32p, C.c_int, C.c_float,
                                        C.c_longlong, C.c_int, u16p, u8p, C.c_ulonglong]
        L.tsq_ref_encode_ex.restype = C.c_int
        L.tsq_ref_aiq_signed.argtypes = [f32p, C.c_int, C.c_int, f32p, i32p, i32p]
        L.tsq_ref_aiq_signed.restype = C.c_int
        L.tsq_ref_decode.argtypes = [u8p, C.c_ulonglong, u16p]
        L.tsq_ref_decode.restype = C.c_int
        L.tsq_ref_ts_row.argtypes = [C.c_int, u16p, C.c_int, C.c_float, f32p, u8p, u8p, C.POINTER(C.c_longlong)]
        L.tsq_ref_ts_row.restype = C.c_int
        L.tsq_ref_aiq.argtypes = [f32p, C.c_int, C.c_int, f32p, i32p, i32p]
        L.tsq_ref_aiq.restype = C.c_int
        L.tsq_ref_select.argtypes = [f32p, C.c_int, i32p, C.c_int, C.c_float, C.POINTER(C.c_longlong),
                                     C.POINTER(C.c_int)]
        L.tsq_ref_select.restype = C.c_int
        L.tsq_ref_raw16_to_float.argtypes = [C.c_int, C.c_uint16]
        L.tsq_ref_raw16_to_float.restype = C.c_float
        L.tsq_ref_float_to_raw16.argtypes = [C.c_int, C.c_float]
        L.tsq_ref_float_to_raw16.restype = C.c_uint16
        _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, status: int):
        super().__init__("oracle status %d (%s)" % (status, STATUS_NAMES.get(status, "?")))
        self.status = status


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def _bits_arr(bits: Sequence[int]) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(list(bits), dtype=np.int32))


def layout(hidden: int, tokens: int, bmax: int, max_outliers: int = 0) -> Dict[str, int]:
    offs = (C.c_ulonglong * 9)()
    st = lib().tsq_ref_layout(hidden, tokens, bmax, max_outliers, offs)
    if st:
        raise OracleError(st)
    names = ["bits", "scale", "zp", "word_off", "out_ptr", "words", "outl", "total", "outlier_capacity"]
    return {n: int(offs[i]) for i, n in enumerate(names)}


def encode(x_raw: np.ndarray, dtype: int, tau: float, bits: Sequence[int], delta: float = 0.2,
           max_outliers: int = 0, signed_values: bool = False) -> np.ndarray:
    """x_raw: uint16 [tokens, hidden]. Returns the blob as a uint8 array. signed_values: the variant that
    quantises the signed inliers (no sign plane, Q_max = 2^b - 1)."""
    x_raw = np.ascontiguousarray(x_raw, dtype=np.uint16)
    assert x_raw.ndim == 2
    tokens, hidden = x_raw.shape
    b = _bits_arr(bits)
    bmax = int(b[-1]) if b.size and 2 <= int(b[-1]) <= 8 else 8   # invalid lists are rejected by the C side
    lay = layout(hidden, tokens, bmax, max_outliers)
    blob = np.empty(lay["total"], dtype=np.uint8)
    st = lib().tsq_ref_encode_ex(dtype, hidden, tokens, tau, _ptr(b, C.c_int32), len(b), delta, max_outliers,
                                 1 if signed_values else 0, _ptr(x_raw, C.c_uint16), _ptr(blob, C.c_uint8), blob.size)
    if st:
        raise OracleError(st)
    return blob


def decode(blob: np.ndarray) -> np.ndarray:
    """Returns uint16 [tokens, hidden]."""
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    hdr = header(blob)
    y = np.empty((hdr["tokens"], hdr["hidden"]), dtype=np.uint16)
    st = lib().tsq_ref_decode(_ptr(blob, C.c_uint8), blob.size, _ptr(y, C.c_uint16))
    if st:
        raise OracleError(st)
    return y


def header(blob: np.ndarray) -> Dict[str, object]:
    h = np.ascontiguousarray(blob[:64])
    u32 = h.view(np.uint32)
    return {
        "magic": int(u32[0]), "version": int(u32[1]), "dtype": int(u32[2]), "hidden": int(u32[3]),
        "tokens": int(u32[4]), "n_bits": int(u32[5]), "bits": [int(v) for v in h[24:31]] + [0], "variant": int(h[31]),
        "tau": float(h[32:36].view(np.float32)[0]), "delta": float(h[36:40].view(np.float32)[0]),
        "total_words": int(h[40:48].view(np.uint64)[0]), "total_outliers": int(h[48:56].view(np.uint64)[0]),
        "status": int(u32[14]), "outlier_capacity": int(u32[15]),
    }


def sections(blob: np.ndarray) -> Dict[str, np.ndarray]:
    """Views of the blob's sections, each cut to its meaningful length (the totals)."""
    hdr = header(blob)
    T, H = hdr["tokens"], hdr["hidden"]
    bmax = hdr["bits"][hdr["n_bits"] - 1]
    lay = layout(H, T, bmax, hdr["outlier_capacity"])
    n_out = min(hdr["total_outliers"], hdr["outlier_capacity"])

    def cut(name, dt, count):
        o = lay[name]
        return blob[o:o + count * np.dtype(dt).itemsize].view(dt)

    return {
        "bits": cut("bits", np.uint8, T), "scale": cut("scale", np.float32, T), "zp": cut("zp", np.int32, T),
        "word_off": cut("word_off", np.uint32, T + 1), "out_ptr": cut("out_ptr", np.uint32, T + 1),
        "words": cut("words", np.uint32, hdr["total_words"]), "outl": cut("outl", np.uint32, n_out),
    }


def ts_row(row_raw: np.ndarray, dtype: int, tau: float):
    row_raw = np.ascontiguousarray(row_raw, dtype=np.uint16)
    H = row_raw.size
    m = np.empty(H, np.float32)
    sg = np.empty(H, np.uint8)
    is_out = np.empty(H, np.uint8)
    n = C.c_longlong(0)
    st = lib().tsq_ref_ts_row(dtype, _ptr(row_raw, C.c_uint16), H, tau, _ptr(m, C.c_float), _ptr(sg, C.c_uint8),
                              _ptr(is_out, C.c_uint8), C.byref(n))
    if st:
        raise OracleError(st)
    return m, sg, is_out, int(n.value)


def aiq(m: np.ndarray, b: int):
    m = np.ascontiguousarray(m, dtype=np.float32)
    q = np.empty(m.size, np.int32)
    s = C.c_float(0)
    zp = C.c_int32(0)
    st = lib().tsq_ref_aiq(_ptr(m, C.c_float), m.size, b, C.byref(s), C.byref(zp), _ptr(q, C.c_int32))
    if st:
        raise OracleError(st)
    return float(s.value), int(zp.value), q


def aiq_signed(v: np.ndarray, b: int):
    v = np.ascontiguousarray(v, dtype=np.float32)
    q = np.empty(v.size, np.int32)
    s = C.c_float(0)
    zp = C.c_int32(0)
    st = lib().tsq_ref_aiq_signed(_ptr(v, C.c_float), v.size, b, C.byref(s), C.byref(zp), _ptr(q, C.c_int32))
    if st:
        raise OracleError(st)
    return float(s.value), int(zp.value), q


def select(m: np.ndarray, bits: Sequence[int], delta: float):
    m = np.ascontiguousarray(m, dtype=np.float32)
    b = _bits_arr(bits)
    S = (C.c_longlong * len(b))()
    bstar = C.c_int(0)
    st = lib().tsq_ref_select(_ptr(m, C.c_float), m.size, _ptr(b, C.c_int32), len(b), delta, S, C.byref(bstar))
    if st:
        raise OracleError(st)
    return [int(v) for v in S], int(bstar.value)


def raw16_to_float(dtype: int, r: int) -> float:
    return float(lib().tsq_ref_raw16_to_float(dtype, r))


def float_to_raw16(dtype: int, f: float) -> int:
    return int(lib().tsq_ref_float_to_raw16(dtype, f))
