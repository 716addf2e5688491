"""Double-precision numpy evaluation of the paper's equations (test infrastructure only).

These functions state the mathematics with no concern for FP32 operation order; the C
oracle's FP32 decisions must agree with them except where a value sits within rounding
distance of a threshold.
"""
from __future__ import annotations

import math

import numpy as np

C8 = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])  # code set of Sec. 3.2
LN2 = math.log(2.0)
LN6 = math.log(6.0)


def scale_exponent(M):
    """Eq. k-rule: k_b = floor((M_b + log(2/9)) / log 2), M_b the block's largest shifted score."""
    return np.floor((np.asarray(M, dtype=np.float64) + math.log(2.0 / 9.0)) / LN2)


def residual(x, k):
    """Eq. z-def: z_t = x_t - k_b log 2 - log 6."""
    return np.asarray(x, dtype=np.float64) - np.asarray(k, dtype=np.float64) * LN2 - LN6


def affine_code(z, tau, h):
    """Eq. d8-index: c_t = clip_[0,7](floor((z_t - tau) h) + 1)."""
    return np.clip(np.floor((np.asarray(z, dtype=np.float64) - tau) * h) + 1.0, 0.0, 7.0).astype(np.int64)


def efq_blocks(x, tau, h, block=32):
    """Algorithm 1 on shifted scores x [rows, n] (n a multiple of ``block``; -inf = masked).
    Returns (codes int64 [rows, n], k int64 [rows, n/block])."""
    x = np.asarray(x, dtype=np.float64)
    rows, n = x.shape
    xb = x.reshape(rows, n // block, block)
    M = xb.max(axis=2)
    with np.errstate(invalid="ignore"):
        k = scale_exponent(M)
        z = residual(xb, k[..., None])
        c = affine_code(np.where(np.isneginf(xb), -1e300, z), tau, h)
    c = np.where(np.isneginf(M)[..., None], 0, c)
    k = np.where(np.isneginf(M), -127, k)
    return c.reshape(rows, n), k.astype(np.int64)


def lut16_code(z):
    """EFQ-Softmax-LUT (Sec. 3.4): 16-level affine index folded onto the 8 codes."""
    tau16 = math.log(1.0 / 24.0)
    h16 = 14.0 / math.log(24.0)
    fold = np.array([0, 1, 1, 1, 1, 1, 2, 2, 3, 3, 4, 5, 5, 6, 7, 7])
    j = np.clip(np.floor((np.asarray(z, dtype=np.float64) - tau16) * h16) + 1.0, 0.0, 15.0).astype(np.int64)
    return fold[j]


def dequant_probabilities(codes, k, block=32):
    """p~_t = 2^{k_b} C8[c_t]  ([rows, n] codes, [rows, n/block] exponents)."""
    return C8[codes] * np.repeat(np.exp2(k.astype(np.float64)), block, axis=1)


def attention_from_operand(p, v):
    """O = (P~ V) / (P~ 1): the same operand in numerator and denominator."""
    p = np.asarray(p, dtype=np.float64)
    return (p @ np.asarray(v, dtype=np.float64)) / p.sum(axis=1, keepdims=True)


def softmax_attention(q, k, v, sigma, causal=False):
    """Textbook one-shot softmax attention in double; q [Sq,d], k,v [Sk,d]."""
    s = (np.asarray(q, np.float64) @ np.asarray(k, np.float64).T) * sigma
    Sq, Sk = s.shape
    if causal:
        i = np.arange(Sq)[:, None]
        t = np.arange(Sk)[None, :]
        s = np.where(t <= i + (Sk - Sq), s, -np.inf)
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    return (p @ np.asarray(v, np.float64)) / p.sum(axis=1, keepdims=True)
