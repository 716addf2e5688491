"""ctypes binding of libefq_b200.so: same names as the C ABI in include/efq.h.

Argument marshalling only.  Tensors are torch CUDA tensors (torch is used for device
memory and streams); nothing here computes.  There is no CPU fallback: if the library
has not been built, or a call returns a non-zero status, a RuntimeError is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libefq_b200.so")

EFQ_OK = 0
STATUS_NAMES = ["EFQ_OK", "EFQ_ERR_INVALID_ARG", "EFQ_ERR_UNSUPPORTED", "EFQ_ERR_ALIGNMENT", "EFQ_ERR_WORKSPACE",
                "EFQ_ERR_ARCH", "EFQ_ERR_CUDA", "EFQ_ERR_DEVICE_TIMEOUT", "EFQ_ERR_STATIC_LIMIT"]
STATIC_SCRATCH_BYTES = 4 << 20

# every symbol include/efq.h declares
EXPORTS = ["efq_probgen", "exp_then_quantize_probgen", "efq_attention_workspace_bytes", "efq_attention_fwd",
           "exp_then_quantize_attention_fwd", "efq_quantize_qkv", "efq_attention_fwd_quantized",
           "efq_attention_fwd_host", "efq_attention_fwd_host_pipelined", "efq_attention_fwd_static", "efq_poll_status",
           "efq_attention_varlen_workspace_bytes", "efq_attention_fwd_varlen",
           "efq_exact_attention_fwd", "efq_relative_error", "efq_calibrate",
           "efq_fp4_mma_peak_probe", "efq_stage_microbench", "efq_attention_fwd_inject_timeout", "efq_status_string",
           "efq_version"]


class EfqParams(C.Structure):
    _fields_ = [("tau", C.c_float), ("h", C.c_float), ("variant", C.c_int32), ("kv_tile", C.c_int32),
                ("rescale_threshold", C.c_float)]


class EfqDebug(C.Structure):
    _fields_ = [("raw_scores", C.c_void_p), ("row_max", C.c_void_p), ("codes", C.c_void_p), ("scales", C.c_void_p),
                ("batch", C.c_int32), ("head", C.c_int32), ("q_begin", C.c_int64), ("q_end", C.c_int64)]


class EfqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{what}: {name} ({status_string(status)})")


_lib = None


def lib() -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built (no fallback path exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_09721_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i64, i32, f32 = C.c_void_p, C.c_int64, C.c_int, C.c_float
        L.efq_probgen.restype = i32
        L.efq_probgen.argtypes = [vp, i64, vp, i64, i64, f32, C.POINTER(EfqParams), vp, vp, vp]
        L.exp_then_quantize_probgen.restype = i32
        L.exp_then_quantize_probgen.argtypes = [vp, i64, vp, i64, i64, f32, i32, vp, vp, vp]
        L.efq_attention_workspace_bytes.restype = C.c_size_t
        L.efq_attention_workspace_bytes.argtypes = [i32, i32, i32, i64, i64, i32]
        L.efq_attention_fwd.restype = i32
        L.efq_attention_fwd.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i64, i32, i32, f32,
                                        C.POINTER(EfqParams), vp, C.c_size_t, C.POINTER(EfqDebug), vp]
        L.exp_then_quantize_attention_fwd.restype = i32
        L.exp_then_quantize_attention_fwd.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i64, i32, i32, f32, i32,
                                                      vp, C.c_size_t, C.POINTER(EfqDebug), vp]
        L.efq_quantize_qkv.restype = i32
        L.efq_quantize_qkv.argtypes = [vp, vp, vp, i32, i32, i32, i64, i64, i32, vp, C.c_size_t, vp]
        L.efq_attention_fwd_quantized.restype = i32
        L.efq_attention_fwd_quantized.argtypes = [vp, i32, i32, i32, i64, i64, i32, i32, f32, i32,
                                                  C.POINTER(EfqParams), vp, C.c_size_t, C.POINTER(EfqDebug), vp]
        L.efq_attention_fwd_host.restype = i32
        L.efq_attention_fwd_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i64, i64, i32, i32, f32,
                                             i32, C.POINTER(EfqParams), vp, C.c_size_t, vp]
        L.efq_attention_fwd_host_pipelined.restype = i32
        L.efq_attention_fwd_host_pipelined.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i64, i64, i32, i32,
                                                       f32, i32, C.POINTER(EfqParams), vp, C.c_size_t, i32, vp, vp, vp]
        L.efq_attention_varlen_workspace_bytes.restype = C.c_size_t
        L.efq_attention_varlen_workspace_bytes.argtypes = [C.POINTER(i64), C.POINTER(i64), i32, i32, i32, i32]
        L.efq_attention_fwd_varlen.restype = i32
        L.efq_attention_fwd_varlen.argtypes = [vp, vp, vp, vp, C.POINTER(i64), C.POINTER(i64), i32, i32, i32, i32, i32, f32,
                                               i32, C.POINTER(EfqParams), vp, C.c_size_t, vp]
        L.efq_attention_fwd_static.restype = i32
        L.efq_attention_fwd_static.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i64, i32, i32, f32,
                                               C.POINTER(EfqParams), vp]
        L.efq_attention_fwd_inject_timeout.restype = i32
        L.efq_attention_fwd_inject_timeout.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i64, i32, vp, C.c_size_t, vp]
        L.efq_exact_attention_fwd.restype = i32
        L.efq_exact_attention_fwd.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i64, i32, i32, f32, vp]
        L.efq_relative_error.restype = i32
        L.efq_relative_error.argtypes = [vp, vp, i64, vp, vp]
        L.efq_calibrate.restype = i32
        L.efq_calibrate.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i64, i64, i32, i32, f32,
                                    C.POINTER(C.c_float), i32, C.POINTER(C.c_float), i32, vp, C.POINTER(C.c_double),
                                    C.POINTER(C.c_float), C.POINTER(C.c_float), vp, C.c_size_t, vp]
        L.efq_poll_status.restype = i32
        L.efq_poll_status.argtypes = [vp, vp]
        L.efq_fp4_mma_peak_probe.restype = i32
        L.efq_fp4_mma_peak_probe.argtypes = [vp, i32, i32, C.POINTER(C.c_double), vp]
        L.efq_stage_microbench.restype = i32
        L.efq_stage_microbench.argtypes = [i32, C.POINTER(EfqParams), i32, i32, vp, vp, vp]
        L.efq_status_string.restype = C.c_char_p
        L.efq_status_string.argtypes = [i32]
        L.efq_version.restype = C.c_char_p
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().efq_status_string(int(status)).decode()


def version() -> str:
    return lib().efq_version().decode()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _params(params) -> Optional[EfqParams]:
    if params is None:
        return None
    if isinstance(params, EfqParams):
        return params
    tau, h = params[0], params[1]
    variant = params[2] if len(params) > 2 else 0
    kv_tile = params[3] if len(params) > 3 else 0
    threshold = params[4] if len(params) > 4 else 0.0
    return EfqParams(float(tau), float(h), int(variant), int(kv_tile), float(threshold))


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _check(status: int, what: str):
    if status != EFQ_OK:
        raise EfqError(status, what)


def _probgen_outputs(scores, codes, scales):
    rows, cols = scores.shape
    nblk = (cols + 31) // 32
    if codes is None:
        codes = torch.empty((rows, nblk * 16), dtype=torch.uint8, device=scores.device)
    if scales is None:
        scales = torch.empty((rows, nblk), dtype=torch.uint8, device=scores.device)
    return codes, scales


def efq_probgen(scores: torch.Tensor, row_max: torch.Tensor, score_scale: float = 1.0, params=None,
                codes: torch.Tensor = None, scales: torch.Tensor = None, stream=None):
    """EFQ probability generation on an fp32 CUDA score matrix [rows, cols] (row stride = ld).
    Returns (codes u8 [rows, ceil(cols/32)*16], scales u8 [rows, ceil(cols/32)])."""
    assert scores.is_cuda and scores.dtype == torch.float32 and scores.dim() == 2 and scores.stride(1) == 1
    assert row_max.is_cuda and row_max.dtype == torch.float32 and row_max.is_contiguous()
    codes, scales = _probgen_outputs(scores, codes, scales)
    p = _params(params)
    st = lib().efq_probgen(scores.data_ptr(), scores.stride(0), row_max.data_ptr(), scores.shape[0],
                           scores.shape[1], float(score_scale), C.byref(p) if p is not None else None,
                           codes.data_ptr(), scales.data_ptr(), _stream(stream))
    _check(st, "efq_probgen")
    return codes, scales


def exp_then_quantize_probgen(scores: torch.Tensor, row_max: torch.Tensor, score_scale: float = 1.0,
                              scale_mode: int = 0, codes: torch.Tensor = None, scales: torch.Tensor = None,
                              stream=None):
    """The exp-then-quantize producer on the same interface."""
    assert scores.is_cuda and scores.dtype == torch.float32 and scores.dim() == 2 and scores.stride(1) == 1
    assert row_max.is_cuda and row_max.dtype == torch.float32 and row_max.is_contiguous()
    codes, scales = _probgen_outputs(scores, codes, scales)
    st = lib().exp_then_quantize_probgen(scores.data_ptr(), scores.stride(0), row_max.data_ptr(), scores.shape[0],
                                         scores.shape[1], float(score_scale), int(scale_mode), codes.data_ptr(),
                                         scales.data_ptr(), _stream(stream))
    _check(st, "exp_then_quantize_probgen")
    return codes, scales


def efq_attention_workspace_bytes(B: int, Hq: int, Hkv: int, Sq: int, Sk: int, d: int) -> int:
    return int(lib().efq_attention_workspace_bytes(B, Hq, Hkv, Sq, Sk, d))


class DebugDump:
    """Device buffers for the optional debug dump of one head / query-row range."""

    def __init__(self, batch: int, head: int, q_begin: int, q_end: int, Sk: int, kv_tile: int = 128,
                 device="cuda"):
        n = q_end - q_begin
        nblk = (Sk + 31) // 32
        self.raw_scores = torch.full((n, Sk), float("nan"), dtype=torch.float32, device=device)
        self.row_max = torch.full((n, (Sk + kv_tile - 1) // kv_tile), float("nan"), dtype=torch.float32, device=device)
        self.codes = torch.zeros((n, nblk * 16), dtype=torch.uint8, device=device)
        self.scales = torch.zeros((n, nblk), dtype=torch.uint8, device=device)
        self.c = EfqDebug(self.raw_scores.data_ptr(), self.row_max.data_ptr(), self.codes.data_ptr(),
                          self.scales.data_ptr(), batch, head, q_begin, q_end)


def _attn_args(q, k, v, o, workspace):
    assert q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous() and q.dim() == 4
    assert k.is_cuda and k.dtype == torch.bfloat16 and k.is_contiguous() and k.shape == v.shape
    assert v.is_cuda and v.dtype == torch.bfloat16 and v.is_contiguous()
    B, Hq, Sq, d = q.shape
    _, Hkv, Sk, _ = k.shape
    if o is None:
        o = torch.empty((B, Hq, Sq, d), dtype=torch.float32, device=q.device)
    if workspace is None:
        nbytes = efq_attention_workspace_bytes(B, Hq, Hkv, Sq, Sk, d)
        workspace = torch.empty(max(nbytes, 1024), dtype=torch.uint8, device=q.device)
    return B, Hq, Hkv, Sq, Sk, d, o, workspace


def efq_attention_fwd(q, k, v, causal: bool = False, softmax_scale: float = 0.0, params=None, o=None,
                      workspace=None, debug: DebugDump = None, stream=None):
    """Fused FP4 attention forward with EFQ probability generation.  q bf16 [B,Hq,Sq,d],
    k/v bf16 [B,Hkv,Sk,d]; returns o fp32 [B,Hq,Sq,d]."""
    B, Hq, Hkv, Sq, Sk, d, o, workspace = _attn_args(q, k, v, o, workspace)
    p = _params(params)
    st = lib().efq_attention_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, Hq, Hkv, Sq, Sk, d,
                                 int(bool(causal)), float(softmax_scale), C.byref(p) if p is not None else None,
                                 workspace.data_ptr(), workspace.numel(),
                                 C.byref(debug.c) if debug is not None else None, _stream(stream))
    _check(st, "efq_attention_fwd")
    return o


def exp_then_quantize_attention_fwd(q, k, v, causal: bool = False, softmax_scale: float = 0.0, scale_mode: int = 0,
                                    o=None, workspace=None, debug: DebugDump = None, stream=None):
    """The MXFP4 comparison path: same pipeline, exp-then-quantize producer."""
    B, Hq, Hkv, Sq, Sk, d, o, workspace = _attn_args(q, k, v, o, workspace)
    st = lib().exp_then_quantize_attention_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, Hq, Hkv,
                                               Sq, Sk, d, int(bool(causal)), float(softmax_scale), int(scale_mode),
                                               workspace.data_ptr(), workspace.numel(),
                                               C.byref(debug.c) if debug is not None else None, _stream(stream))
    _check(st, "exp_then_quantize_attention_fwd")
    return o


def efq_quantize_qkv(q, k, v, workspace, stream=None):
    """Operand preparation only: bf16 Q/K/V -> MXFP4 copies in the workspace."""
    B, Hq, Hkv, Sq, Sk, d, _, workspace = _attn_args(q, k, v, q, workspace)
    st = lib().efq_quantize_qkv(q.data_ptr(), k.data_ptr(), v.data_ptr(), B, Hq, Hkv, Sq, Sk, d,
                                workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(st, "efq_quantize_qkv")
    return workspace


def efq_attention_fwd_quantized(o, shape, workspace, causal: bool = False, softmax_scale: float = 0.0,
                                producer: int = 0, params=None, debug: DebugDump = None, stream=None):
    """The fused forward on a workspace prepared by efq_quantize_qkv; shape = (B, Hq, Hkv, Sq, Sk, d)."""
    B, Hq, Hkv, Sq, Sk, d = shape
    p = _params(params)
    st = lib().efq_attention_fwd_quantized(o.data_ptr(), B, Hq, Hkv, Sq, Sk, d, int(bool(causal)), float(softmax_scale),
                                           int(producer), C.byref(p) if p is not None else None,
                                           workspace.data_ptr(), workspace.numel(),
                                           C.byref(debug.c) if debug is not None else None, _stream(stream))
    _check(st, "efq_attention_fwd_quantized")
    return o


def efq_attention_fwd_varlen(q, k, v, cu_seqlens_q, cu_seqlens_k, causal: bool = False, softmax_scale: float = 0.0,
                             producer: int = 0, params=None, workspace=None, stream=None):
    """Packed variable-length batch: q [total_q, Hq, d], k, v [total_k, Hkv, d] bf16 CUDA tensors (token-major);
    cu_seqlens_*: sequences of n_seqs + 1 host integers.  Returns o [total_q, Hq, d] fp32."""
    total_q, Hq, d = q.shape
    total_k, Hkv, _ = k.shape
    assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and v.shape == k.shape
    n = len(cu_seqlens_q) - 1
    assert len(cu_seqlens_k) == n + 1 and int(cu_seqlens_q[-1]) == total_q and int(cu_seqlens_k[-1]) == total_k
    cq = (C.c_int64 * (n + 1))(*[int(x) for x in cu_seqlens_q])
    ck = (C.c_int64 * (n + 1))(*[int(x) for x in cu_seqlens_k])
    if workspace is None:
        nbytes = lib().efq_attention_varlen_workspace_bytes(cq, ck, n, Hq, Hkv, d)
        if nbytes == 0:
            raise EfqError(1, "efq_attention_varlen_workspace_bytes")
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
    o = torch.empty((total_q, Hq, d), dtype=torch.float32, device=q.device)
    p = _params(params)
    st = lib().efq_attention_fwd_varlen(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), cq, ck, n, Hq, Hkv, d,
                                        int(bool(causal)), float(softmax_scale), int(producer),
                                        C.byref(p) if p is not None else None, workspace.data_ptr(), workspace.numel(),
                                        _stream(stream))
    _check(st, "efq_attention_fwd_varlen")
    return o


def efq_attention_fwd_host(q_host, k_host, v_host, o_host, q_dev, k_dev, v_dev, o_dev, causal: bool = False,
                           softmax_scale: float = 0.0, producer: int = 0, params=None, workspace=None, stream=None):
    """End-to-end form: host (pinned) inputs and output, caller-owned device staging buffers."""
    B, Hq, Sq, d = q_host.shape
    _, Hkv, Sk, _ = k_host.shape
    assert not q_host.is_cuda and not o_host.is_cuda and q_dev.is_cuda and o_dev.is_cuda
    p = _params(params)
    st = lib().efq_attention_fwd_host(q_host.data_ptr(), k_host.data_ptr(), v_host.data_ptr(), o_host.data_ptr(),
                                      q_dev.data_ptr(), k_dev.data_ptr(), v_dev.data_ptr(), o_dev.data_ptr(),
                                      B, Hq, Hkv, Sq, Sk, d, int(bool(causal)), float(softmax_scale), int(producer),
                                      C.byref(p) if p is not None else None, workspace.data_ptr(),
                                      workspace.numel(), _stream(stream))
    _check(st, "efq_attention_fwd_host")
    return o_host


def efq_attention_fwd_host_pipelined(q_host, k_host, v_host, o_host, q_dev, k_dev, v_dev, o_dev, streams,
                                     causal: bool = False, softmax_scale: float = 0.0, producer: int = 0, params=None,
                                     workspace=None, n_chunks: int = 8):
    """End-to-end form with the copies overlapped: ``streams`` = (copy-in, compute, copy-out) torch streams.
    Synchronising the compute stream completes the call."""
    B, Hq, Sq, d = q_host.shape
    _, Hkv, Sk, _ = k_host.shape
    assert not q_host.is_cuda and not o_host.is_cuda and q_dev.is_cuda and o_dev.is_cuda and len(streams) == 3
    p = _params(params)
    st = lib().efq_attention_fwd_host_pipelined(
        q_host.data_ptr(), k_host.data_ptr(), v_host.data_ptr(), o_host.data_ptr(), q_dev.data_ptr(), k_dev.data_ptr(),
        v_dev.data_ptr(), o_dev.data_ptr(), B, Hq, Hkv, Sq, Sk, d, int(bool(causal)), float(softmax_scale),
        int(producer), C.byref(p) if p is not None else None, workspace.data_ptr(), workspace.numel(), int(n_chunks),
        _stream(streams[0]), _stream(streams[1]), _stream(streams[2]))
    _check(st, "efq_attention_fwd_host_pipelined")
    return o_host


def efq_attention_fwd_static(q, k, v, causal: bool = False, softmax_scale: float = 0.0, params=None, o=None,
                             stream=None):
    """efq_attention_fwd for callers that cannot hand over a workspace: the scratch is a fixed array inside
    the library (STATIC_SCRATCH_BYTES); larger problems raise EfqError with EFQ_ERR_STATIC_LIMIT.  The output
    tensor is still the caller's: pass ``o`` to keep this call free of allocations."""
    assert q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous() and q.dim() == 4
    assert k.is_cuda and k.dtype == torch.bfloat16 and k.is_contiguous() and k.shape == v.shape
    assert v.is_cuda and v.dtype == torch.bfloat16 and v.is_contiguous()
    B, Hq, Sq, d = q.shape
    _, Hkv, Sk, _ = k.shape
    if o is None:
        o = torch.empty((B, Hq, Sq, d), dtype=torch.float32, device=q.device)
    p = _params(params)
    st = lib().efq_attention_fwd_static(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, Hq, Hkv, Sq, Sk, d,
                                        int(bool(causal)), float(softmax_scale),
                                        C.byref(p) if p is not None else None, _stream(stream))
    _check(st, "efq_attention_fwd_static")
    return o


def efq_exact_attention_fwd(q, k, v, causal: bool = False, softmax_scale: float = 0.0, o=None, stream=None):
    """FP32 softmax attention on the unquantised bf16 inputs (reference output); returns o fp32 [B,Hq,Sq,d]."""
    B, Hq, Sq, d = q.shape
    _, Hkv, Sk, _ = k.shape
    if o is None:
        o = torch.empty((B, Hq, Sq, d), dtype=torch.float32, device=q.device)
    st = lib().efq_exact_attention_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, Hq, Hkv, Sq, Sk, d,
                                       int(bool(causal)), float(softmax_scale), _stream(stream))
    _check(st, "efq_exact_attention_fwd")
    return o


def efq_relative_error(a: torch.Tensor, ref: torch.Tensor, sums: torch.Tensor = None, stream=None) -> float:
    """rho = ||a - ref||_F / ||ref||_F of two fp32 CUDA tensors (synchronises to read the two sums)."""
    assert a.is_cuda and ref.is_cuda and a.dtype == torch.float32 and ref.dtype == torch.float32
    assert a.is_contiguous() and ref.is_contiguous() and a.numel() == ref.numel()
    if sums is None:
        sums = torch.empty(2, dtype=torch.float64, device=a.device)
    st = lib().efq_relative_error(a.data_ptr(), ref.data_ptr(), a.numel(), sums.data_ptr(), _stream(stream))
    _check(st, "efq_relative_error")
    d2, r2 = (float(x) for x in sums.cpu())
    if r2 > 0.0:
        return (d2 / r2) ** 0.5
    return float("inf") if d2 > 0.0 else 0.0


def efq_calibrate(q, k, v, o_ref, taus, hs, causal: bool = False, softmax_scale: float = 0.0, workspace=None,
                  stream=None):
    """Grid search of (tau, h) (Algorithm 3).  Returns (rho [n_tau, n_h] as nested lists, (best_tau, best_h))."""
    B, Hq, Hkv, Sq, Sk, d, o_tmp, workspace = _attn_args(q, k, v, None, workspace)
    assert o_ref.is_cuda and o_ref.dtype == torch.float32 and o_ref.is_contiguous() and o_ref.shape == o_tmp.shape
    n_tau, n_h = len(taus), len(hs)
    ct = (C.c_float * n_tau)(*[float(t) for t in taus])
    ch = (C.c_float * n_h)(*[float(h) for h in hs])
    rho = (C.c_double * (n_tau * n_h))()
    bt, bh = C.c_float(0.0), C.c_float(0.0)
    sums = torch.empty(2 * n_tau * n_h, dtype=torch.float64, device=q.device)
    st = lib().efq_calibrate(q.data_ptr(), k.data_ptr(), v.data_ptr(), o_ref.data_ptr(), o_tmp.data_ptr(), B, Hq, Hkv,
                             Sq, Sk, d, int(bool(causal)), float(softmax_scale), ct, n_tau, ch, n_h, sums.data_ptr(),
                             rho, C.byref(bt), C.byref(bh), workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(st, "efq_calibrate")
    table = [[rho[i * n_h + j] for j in range(n_h)] for i in range(n_tau)]
    return table, (float(bt.value), float(bh.value))


def efq_poll_status(workspace, stream=None) -> int:
    return int(lib().efq_poll_status(workspace.data_ptr(), _stream(stream)))


def efq_fp4_mma_peak_probe(sink: torch.Tensor, num_ctas: int, iters: int, stream=None) -> float:
    """Launches the MMA-only FP4 microbenchmark; returns the FLOPs of the launch."""
    flops = C.c_double(0.0)
    st = lib().efq_fp4_mma_peak_probe(sink.data_ptr(), int(num_ctas), int(iters), C.byref(flops), _stream(stream))
    _check(st, "efq_fp4_mma_peak_probe")
    return float(flops.value)


def efq_stage_microbench(producer: int, num_ctas: int, iters: int, params=None, stream=None):
    """In-SM producer microbenchmark; returns the per-CTA cycle counts (int64 CUDA tensor [num_ctas])."""
    sink = torch.empty(num_ctas * 256, dtype=torch.int32, device="cuda")
    cycles = torch.zeros(num_ctas, dtype=torch.int64, device="cuda")
    p = _params(params)
    st = lib().efq_stage_microbench(int(producer), C.byref(p) if p is not None else None, int(num_ctas), int(iters),
                                    sink.data_ptr(), cycles.data_ptr(), _stream(stream))
    _check(st, "efq_stage_microbench")
    return cycles


def efq_attention_fwd_inject_timeout(q, k, v, o, workspace, stream=None) -> None:
    """Test hook: the forward with K/V loads left out, so a bounded device-side wait expires (see efq.h)."""
    B, Hq, Sq, d = q.shape
    _, Hkv, Sk, _ = k.shape
    st = lib().efq_attention_fwd_inject_timeout(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, Hq, Hkv, Sq,
                                                Sk, d, workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(st, "efq_attention_fwd_inject_timeout")
