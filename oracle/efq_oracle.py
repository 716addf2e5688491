"""ctypes wrapper over the C oracle (oracle/efq_oracle.c).  Test infrastructure only.

All arrays are numpy, host memory.  bf16 inputs are passed as float32 (exact widenings).
Paths: "exact" (double softmax attention on the unquantised inputs), "efq" (Algorithm 2
with Algorithm 1 as producer), "etq" (exp-then-quantize producer, block maximum scaled
into [4, 8)), "etq6" (same with the block maximum scaled into (3, 6]), "efq_lut" (Algorithm 1 with
the 16-level index and the folding table of the LUT variant; tau and h are not used), "etq_fp32den"
(attention_rows only: "etq" with the denominator summed from the FP32 exponentials; context, not the paper's rule).
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build

_lib = None

PATHS = {"exact": 0, "efq": 1, "etq": 2, "etq6": 3, "efq_lut": 4, "etq_fp32den": 5}
PRODUCERS = {"efq": 0, "etq": 1, "etq6": 2, "efq_lut": 3}

# (tau, h) operating points printed in the paper's "Parameter selection" paragraph.
EFQ_MEAN = (-3.06, 2.30)
EFQ_MMLU = (-2.90, 2.00)
EFQ_BALANCE = (-2.10, 2.70)


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        fp = C.POINTER(C.c_float)
        u8 = C.POINTER(C.c_uint8)
        i64 = C.c_int64
        L.efq_oracle_threads.restype = C.c_int
        L.efq_oracle_c8.restype = C.c_double
        L.efq_oracle_c8.argtypes = [C.c_int]
        L.efq_oracle_mxfp4_rows.argtypes = [fp, i64, C.c_int, fp, u8, u8]
        L.efq_oracle_mxfp4_cols.argtypes = [fp, i64, C.c_int, fp, u8, u8]
        L.efq_oracle_probgen.argtypes = [fp, i64, fp, i64, i64, C.c_float, C.c_float, C.c_float,
                                         C.c_int, u8, u8]
        L.efq_oracle_online_codes.argtypes = [fp, i64, i64, i64, i64, C.c_float, C.c_float, C.c_float,
                                              C.c_int, C.c_float, u8, u8, fp]
        L.efq_oracle_attention_rows.argtypes = [fp, fp, fp, C.c_int, C.c_int, C.c_int, i64, i64, C.c_int,
                                                C.c_int, C.c_float, C.c_float, C.c_float, i64, C.c_int, C.c_float,
                                                C.POINTER(i64), i64, fp, fp, u8, u8, fp]
        _lib = L
    return _lib


def _fp(a):
    return a.ctypes.data_as(C.POINTER(C.c_float)) if a is not None else None


def _u8(a):
    return a.ctypes.data_as(C.POINTER(C.c_uint8)) if a is not None else None


def threads() -> int:
    return int(lib().efq_oracle_threads())


def c8(c: int) -> float:
    return float(lib().efq_oracle_c8(int(c)))


def mxfp4_rows(x: np.ndarray):
    """Blocks of 32 along the last axis of a 2-D float32 array.  Returns (xhat, codes, scales)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    n, d = x.shape
    xhat = np.empty_like(x)
    codes = np.empty((n, d), dtype=np.uint8)
    scales = np.empty((n, (d + 31) // 32), dtype=np.uint8)
    lib().efq_oracle_mxfp4_rows(_fp(x), n, d, _fp(xhat), _u8(codes), _u8(scales))
    return xhat, codes, scales


def mxfp4_cols(x: np.ndarray):
    """Blocks of 32 along the first axis (keys) of a [S, d] float32 array, per channel."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    S, d = x.shape
    xhat = np.empty_like(x)
    codes = np.empty((S, d), dtype=np.uint8)
    scales = np.empty(((S + 31) // 32, d), dtype=np.uint8)
    lib().efq_oracle_mxfp4_cols(_fp(x), S, d, _fp(xhat), _u8(codes), _u8(scales))
    return xhat, codes, scales


def probgen(scores: np.ndarray, row_max: np.ndarray, sigma: float = 1.0, tau: float = EFQ_MEAN[0],
            h: float = EFQ_MEAN[1], producer: str = "efq"):
    """Standalone stage on a [rows, cols] float32 score matrix.  Returns (codes, scales):
    codes uint8 [rows, ceil(cols/32)*16] (element 2u in the low nibble of byte u),
    scales uint8 [rows, ceil(cols/32)] (E8M0: exponent + 127)."""
    assert scores.dtype == np.float32 and scores.ndim == 2 and scores.strides[1] == 4
    rows, cols = scores.shape
    ld = scores.strides[0] // 4
    row_max = np.ascontiguousarray(row_max, dtype=np.float32)
    nblk = (cols + 31) // 32
    codes = np.empty((rows, nblk * 16), dtype=np.uint8)
    scales = np.empty((rows, nblk), dtype=np.uint8)
    lib().efq_oracle_probgen(_fp(scores), ld, _fp(row_max), rows, cols, sigma, tau, h,
                             PRODUCERS[producer], _u8(codes), _u8(scales))
    return codes, scales


def online_codes(scores: np.ndarray, Bc: int, sigma: float, tau: float = EFQ_MEAN[0],
                 h: float = EFQ_MEAN[1], producer: str = "efq", rescale_threshold: float = 0.0):
    """Online (running-maximum) code generation on given raw scores [rows, n_keys].
    Returns (codes, scales, m_s [rows, ntile]).  rescale_threshold > 0 keeps the shifting maximum while the
    true maximum exceeds it by at most that much (scaled units); 0 is Algorithm 2."""
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    rows, n_keys = scores.shape
    nblk = (n_keys + 31) // 32
    ntile = (n_keys + Bc - 1) // Bc
    codes = np.empty((rows, nblk * 16), dtype=np.uint8)
    scales = np.empty((rows, nblk), dtype=np.uint8)
    ms = np.empty((rows, ntile), dtype=np.float32)
    lib().efq_oracle_online_codes(_fp(scores), n_keys, rows, n_keys, Bc, sigma, tau, h,
                                  PRODUCERS[producer], rescale_threshold, _u8(codes), _u8(scales), _fp(ms))
    return codes, scales, ms


def attention_rows(q: np.ndarray, k: np.ndarray, v: np.ndarray, rows: np.ndarray, causal: bool,
                   sigma: float, path: str = "efq", tau: float = EFQ_MEAN[0], h: float = EFQ_MEAN[1],
                   Bc: int = 128, dumps: bool = False, rescale_threshold: float = 0.0):
    """Attention forward on sampled rows.  q [B,Hq,Sq,d], k/v [B,Hkv,Sk,d] float32;
    rows int64 [n, 3] of (b, head, query index).  Returns out [n, d] float32, and with
    ``dumps`` a dict of raw scores, packed codes, scale bytes and per-tile m_s."""
    q = np.ascontiguousarray(q, dtype=np.float32)
    k = np.ascontiguousarray(k, dtype=np.float32)
    v = np.ascontiguousarray(v, dtype=np.float32)
    rows = np.ascontiguousarray(rows, dtype=np.int64).reshape(-1, 3)
    B, Hq, Sq, d = q.shape
    _, Hkv, Sk, _ = k.shape
    n = rows.shape[0]
    out = np.empty((n, d), dtype=np.float32)
    raw = codes = scales = ms = None
    if dumps and path != "exact":
        nblk = (Sk + 31) // 32
        raw = np.empty((n, Sk), dtype=np.float32)
        codes = np.empty((n, nblk * 16), dtype=np.uint8)
        scales = np.empty((n, nblk), dtype=np.uint8)
        ms = np.empty((n, (Sk + Bc - 1) // Bc), dtype=np.float32)
    lib().efq_oracle_attention_rows(_fp(q), _fp(k), _fp(v), B, Hq, Hkv, Sq, Sk, d, int(causal),
                                    sigma, tau, h, Bc, PATHS[path], rescale_threshold,
                                    rows.ctypes.data_as(C.POINTER(C.c_int64)), n, _fp(out),
                                    _fp(raw), _u8(codes), _u8(scales), _fp(ms))
    if dumps:
        return out, {"raw": raw, "codes": codes, "scales": scales, "ms": ms}
    return out


def unpack_codes(codes: np.ndarray) -> np.ndarray:
    """[rows, n/2] packed bytes -> [rows, n] one code per byte (low nibble first)."""
    lo = codes & 0xF
    hi = codes >> 4
    return np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)
