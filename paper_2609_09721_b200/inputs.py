"""Seeded synthetic inputs for the EFQ-Softmax hot path.

This module is the only code shared by the CPU oracle's tests and the CUDA path's
tests/benchmarks.  It holds no arithmetic of the method itself: only a counter-based
random generator, bf16 rounding, and the recipes that shape the five workloads
(attention shapes of a Qwen3-8B-like GQA prefill and a WAN2.2-like video DiT, plus a
standalone score matrix for the probability-generation stage).

Everything is numpy on the host.  bf16 tensors are carried as ``uint16`` bit patterns
(numpy has no bf16); ``bf16_bits_to_f32`` widens them exactly.

Generator: element ``i`` of tensor ``tid`` under ``seed`` gets two 64-bit hashes
(splitmix64 finaliser over a counter built from ``(seed, tid, i, lane)``) turned into
two uniforms and one Box-Muller normal, so any slice of any tensor can be produced
independently and in any chunking.
"""
from __future__ import annotations

import math
import os
from dataclasses import dataclass

import numpy as np

_U64 = np.uint64
_CHUNK = 1 << 22


def _splitmix64(x: np.ndarray) -> np.ndarray:
    x = (x + _U64(0x9E3779B97F4A7C15)).astype(_U64)
    x = (x ^ (x >> _U64(30))) * _U64(0xBF58476D1CE4E5B9)
    x = (x ^ (x >> _U64(27))) * _U64(0x94D049BB133111EB)
    return x ^ (x >> _U64(31))


def _key(seed: int, tid: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _splitmix64(np.array([seed & 0xFFFFFFFFFFFFFFFF], dtype=_U64))
        k = _splitmix64(k ^ _U64(tid * 0xD1342543DE82EF95 & 0xFFFFFFFFFFFFFFFF))
    return k[0]


def hash_u64(seed: int, tid: int, start: int, count: int, lane: int = 0) -> np.ndarray:
    """64-bit hashes for flat indices ``start .. start+count-1`` of tensor ``tid``."""
    with np.errstate(over="ignore"):
        idx = np.arange(start, start + count, dtype=_U64)
        ctr = idx * _U64(2) + _U64(lane)
        return _splitmix64(_splitmix64(ctr ^ _key(seed, tid)) + _key(seed, tid))


def uniform(seed: int, tid: int, start: int, count: int, lane: int = 0) -> np.ndarray:
    """float64 uniforms in (0, 1)."""
    h = hash_u64(seed, tid, start, count, lane)
    return ((h >> _U64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _normal_chunk(args):
    seed, tid, start, n, out = args
    u1 = uniform(seed, tid, start, n, 0)
    u2 = uniform(seed, tid, start, n, 1)
    np.multiply(np.sqrt(-2.0 * np.log(u1)), np.cos((2.0 * math.pi) * u2), out=out)


def normal(seed: int, tid: int, count: int, start: int = 0) -> np.ndarray:
    """float64 N(0,1) samples for flat indices ``start .. start+count-1`` (chunks run on a thread pool;
    the values do not depend on the chunking)."""
    out = np.empty(count, dtype=np.float64)
    jobs = [(seed, tid, start + lo, min(_CHUNK, count - lo), out[lo:lo + min(_CHUNK, count - lo)])
            for lo in range(0, count, _CHUNK)]
    if len(jobs) <= 1:
        for j in jobs:
            _normal_chunk(j)
    else:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1, 32)) as ex:
            list(ex.map(_normal_chunk, jobs))
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------------------
# Workload descriptions
# --------------------------------------------------------------------------------------

@dataclass(frozen=True)
class AttentionCase:
    name: str
    B: int
    Hq: int
    Hkv: int
    Sq: int
    Sk: int
    d: int
    causal: bool
    seed: int
    recipe: str  # "iid" | "k_outliers" | "lowrank"

    @property
    def softmax_scale(self) -> float:
        return float(np.float32(1.0 / math.sqrt(self.d)))

    @property
    def flops(self) -> float:
        """4*B*Hq*Sq*Sk*d, halved for causal (FlashAttention convention)."""
        f = 4.0 * self.B * self.Hq * self.Sq * self.Sk * self.d
        return f * 0.5 if self.causal else f


def case_single_head(S: int = 1024, seed: int = 1) -> AttentionCase:
    return AttentionCase("single_head", 1, 1, 1, S, S, 128, False, seed, "iid")


def case_qwen3_8b(S: int = 16384, seed: int = 3, Hq: int = 32, Hkv: int = 8) -> AttentionCase:
    return AttentionCase(f"qwen3_8b_prefill_S{S}", 1, Hq, Hkv, S, S, 128, True, seed, "k_outliers")


def case_wan22(S: int = 32760, seed: int = 5, H: int = 24) -> AttentionCase:
    return AttentionCase(f"wan22_ti2v_5b_S{S}", 1, H, H, S, S, 128, False, seed, "lowrank")


_TID_Q, _TID_K, _TID_V = 1, 2, 3
_TID_OUTLIER = 10
_TID_PHASE = 20
_TID_W = 30


def _lowrank_part(case: AttentionCase, tid: int, H: int, S: int) -> np.ndarray:
    """2 * F @ W: rank-16 smooth component, RMS about 2, shape [H, S, d] float64."""
    r = 16
    out = np.empty((H, S, case.d), dtype=np.float64)
    s = np.arange(S, dtype=np.float64)[:, None]
    for h in range(H):
        phase = uniform(case.seed, _TID_PHASE + tid, h * r, r) * (2.0 * math.pi)
        freq = (np.arange(r, dtype=np.float64) + 1.0)[None, :]
        F = np.cos((2.0 * math.pi) * freq * s / S + phase[None, :]) * math.sqrt(2.0)
        W = normal(case.seed, _TID_W + tid, r * case.d, h * r * case.d).reshape(r, case.d) / 4.0
        out[h] = 2.0 * (F @ W)
    return out


def _gen_tensor(case: AttentionCase, tid: int, H: int, S: int) -> np.ndarray:
    """bf16 bit patterns, shape [B, H, S, d]."""
    n_per_b = H * S * case.d
    out = np.empty((case.B, H, S, case.d), dtype=np.uint16)
    for b in range(case.B):
        g = normal(case.seed, tid, n_per_b, b * n_per_b).reshape(H, S, case.d)
        if case.recipe == "k_outliers" and tid == _TID_K:
            for h in range(H):
                rank = hash_u64(case.seed, _TID_OUTLIER, (b * H + h) * case.d, case.d)
                ch = np.argsort(rank, kind="stable")[:8]
                g[h][:, ch] *= 10.0
        elif case.recipe == "lowrank":
            g += _lowrank_part(case, tid + 100 * b, H, S)
        out[b] = f32_to_bf16_bits(g.astype(np.float32))
    return out


def make_qkv(case: AttentionCase):
    """Returns (q, k, v) as uint16 bf16 bit patterns, [B,Hq,Sq,d], [B,Hkv,Sk,d], [B,Hkv,Sk,d]."""
    q = _gen_tensor(case, _TID_Q, case.Hq, case.Sq)
    k = _gen_tensor(case, _TID_K, case.Hkv, case.Sk)
    v = _gen_tensor(case, _TID_V, case.Hkv, case.Sk)
    return q, k, v


def make_score_matrix(rows: int = 4096, cols: int = 16384, seed: int = 2,
                      sigma: float = 3.0, spike: float = 12.0, spike_frac: float = 0.01):
    """Standalone-stage workload: fp32 scores N(0, sigma^2) with a seeded 1 % of the entries
    of every row set to ``spike``; returns (scores [rows, cols] float32, row_max [rows] float32)."""
    scores = np.empty((rows, cols), dtype=np.float32)
    n_spike = int(round(cols * spike_frac))
    for r0 in range(0, rows, 256):
        r1 = min(rows, r0 + 256)
        blk = (normal(seed, 1, (r1 - r0) * cols, r0 * cols) * sigma).astype(np.float32).reshape(r1 - r0, cols)
        if n_spike > 0:
            rank = hash_u64(seed, 2, r0 * cols, (r1 - r0) * cols).reshape(r1 - r0, cols)
            idx = np.argpartition(rank, n_spike - 1, axis=1)[:, :n_spike]
            np.put_along_axis(blk, idx, np.float32(spike), axis=1)
        scores[r0:r1] = blk
    return scores, scores.max(axis=1).astype(np.float32)


def sample_rows(case: AttentionCase, n_random: int = 256, tile: int = 128, seed: int = 99) -> np.ndarray:
    """Seeded sample of (b, head, query row) triples: first/last rows, rows at tile edges,
    the last rows (ragged tail) and ``n_random`` uniformly drawn ones.  int64 [n, 3]."""
    rows = []
    edge = [0, 1, tile - 1, tile, tile + 1, case.Sq // 2, case.Sq - tile - 1, case.Sq - 2, case.Sq - 1]
    for h in sorted({0, case.Hq // 2, case.Hq - 1}):
        for i in edge:
            if 0 <= i < case.Sq:
                rows.append((0, h, i))
    u = hash_u64(seed, 7, 0, 3 * n_random)
    for j in range(n_random):
        b = int(u[3 * j] % np.uint64(case.B))
        h = int(u[3 * j + 1] % np.uint64(case.Hq))
        i = int(u[3 * j + 2] % np.uint64(case.Sq))
        rows.append((b, h, i))
    rows = sorted(set(rows))
    return np.asarray(rows, dtype=np.int64).reshape(-1, 3)
