"""Pins the CPU oracle to what the paper and the mathematics fix (no GPU needed).

Each test checks the C oracle (oracle/efq_oracle.c) against something that is not the
oracle: the paper's printed constants, the threshold form of the affine rule, interval
inequalities evaluated in double, closed-form special cases, a library softmax
attention, or brute force over the code set.
"""
import math
import os

import numpy as np
import pytest

from oracle import efq_math
from paper_2609_09721_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
LN2, LN6 = math.log(2.0), math.log(6.0)


def _read(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


def _points():
    return [(n, float(t), float(h)) for n, t, h in (ln.split() for ln in _read("operating_points.txt"))]


POINTS = _points()
MEAN = next((t, h) for n, t, h in POINTS if n == "EFQ-Mean")


def _probgen_blocks(oracle, x, tau, h, producer="efq"):
    """x [rows, n] shifted scores (row max := 0, sigma := 1) -> (codes [rows, n], k [rows, n/32])."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    codes, scales = oracle.probgen(x, np.zeros(x.shape[0], np.float32), 1.0, tau, h, producer)
    return oracle.unpack_codes(codes)[:, : x.shape[1]].astype(np.int64), scales.astype(np.int64) - 127


# ---------------------------------------------------------------------------------------
# code set, packing
# ---------------------------------------------------------------------------------------

def test_code_set_matches_paper(oracle):
    paper = [float(t) for t in _read("c8_code_set.txt")[0].split()]
    assert [oracle.c8(c) for c in range(8)] == paper
    assert list(efq_math.C8) == paper
    # the index IS the E2M1 bit pattern: exponent field c>>1, mantissa bit c&1, bias 1
    for c in range(8):
        e, m = c >> 1, c & 1
        val = 0.5 * m if e == 0 else (1.0 + 0.5 * m) * 2.0 ** (e - 1)
        assert oracle.c8(c) == val


def test_codes_nonnegative_and_low_nibble_first(oracle):
    rng = np.random.default_rng(0)
    x = -np.abs(rng.normal(0, 3, (7, 96))).astype(np.float32)
    x[:, 5] = 0.0
    packed, scales = oracle.probgen(x, np.zeros(7, np.float32), 1.0, *MEAN)
    assert packed.shape == (7, 48) and scales.shape == (7, 3)
    assert np.all((packed & 0x88) == 0)  # bit 3 of every nibble (the E2M1 sign) is clear
    c, _ = _probgen_blocks(oracle, x, *MEAN)
    assert np.array_equal(packed & 0xF, c[:, 0::2]) and np.array_equal(packed >> 4, c[:, 1::2])
    # element order: a single 0 among -inf in position p shows up in nibble p
    for p in (0, 1, 2, 31, 32, 63):
        y = np.full((1, 64), -np.inf, np.float32)
        y[0, p] = 0.0
        pk, _ = oracle.probgen(y, np.zeros(1, np.float32), 1.0, *MEAN)
        nz = np.flatnonzero(oracle.unpack_codes(pk)[0])
        assert list(nz) == [p]


# ---------------------------------------------------------------------------------------
# scale rule
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("name,tau,h", POINTS)
def test_scale_interval_and_residual_range(oracle, name, tau, h):
    rng = np.random.default_rng(1)
    M = -rng.uniform(0, 80, 4000)
    M[:8] = [0.0, -1e-6, -LN2, -2 * LN2, -0.5, -10.0, -40.0, -80.0]
    x = np.full((M.size, 32), -np.inf, np.float32)
    x[:, 3] = M.astype(np.float32)
    x[:, 9] = (M - 1.0).astype(np.float32)
    _, k = _probgen_blocks(oracle, x, tau, h)
    k = k[:, 0].astype(np.float64)
    Mf = x[:, 3].astype(np.float64)
    target = 2.0 * np.exp(Mf) / 9.0           # Eq. k-interval: 2^k <= 2 e^M / 9 < 2^(k+1)
    lo, hi = np.exp2(k), np.exp2(k + 1)
    slack = 1e-5                              # FP32 decision vs double evaluation
    assert np.all(lo <= target * (1 + slack)) and np.all(target * (1 - slack) < hi)
    edge = np.minimum(np.abs(np.log2(target) - k), np.abs(np.log2(target) - k - 1)) < 1e-4
    assert np.array_equal(k[~edge], efq_math.scale_exponent(Mf)[~edge])
    assert np.all(k <= -3)                    # x <= 0  =>  2^k <= 2/9
    zmax = Mf - k * LN2 - LN6                 # bounded residual of the block maximum
    assert np.all(zmax >= math.log(0.75) - 1e-5) and np.all(zmax < math.log(1.5) + 1e-5)


def test_scale_is_exponent_only_and_clamped(oracle):
    x = np.full((3, 32), -np.inf, np.float32)
    x[0, 0] = -200.0      # below the E8M0 range: clamps to exponent -127 (byte 0)
    x[1, 0] = 0.0
    _, scales = oracle.probgen(x, np.zeros(3, np.float32), 1.0, *MEAN)
    assert scales[0, 0] == 0 and scales[1, 0] == 124 and scales[2, 0] == 0
    c, _ = _probgen_blocks(oracle, x, *MEAN)
    assert np.all(c[2] == 0)                  # fully masked block: all-zero operand


# ---------------------------------------------------------------------------------------
# affine code rule
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("name,tau,h", POINTS)
def test_affine_rule_threshold_form(oracle, name, tau, h):
    """Brute force over a fine grid of residuals z: the code is the number of thresholds
    tau + (c-1)/h, c = 1..7, that z has reached (threshold form of Eq. d8-index)."""
    thr = np.array([tau + (c - 1) / h for c in range(1, 8)])
    for M in (0.0, -0.3, -5.1234, -33.0):
        k = math.floor((M + math.log(2.0 / 9.0)) / LN2)
        zmax = M - k * LN2 - LN6
        z = np.linspace(tau - 1.0, zmax, 31 * 4000)
        x = (z + k * LN2 + LN6).astype(np.float32).reshape(-1, 31)
        x = np.concatenate([np.full((x.shape[0], 1), M, np.float32), x], axis=1)
        c, kk = _probgen_blocks(oracle, x, tau, h)
        assert np.all(kk == k)
        zz = x.astype(np.float64) - k * LN2 - LN6
        expect = (zz[..., None] >= thr).sum(-1)
        near = np.abs(zz[..., None] - thr).min(-1) < 2e-5 * max(1.0, abs(M))
        assert np.array_equal(c[~near], expect[~near])
        assert np.all(np.abs(c - expect)[near] <= 1)
        assert near.mean() < 1e-2
        # monotone non-decreasing in x
        order = np.argsort(x.ravel(), kind="stable")
        assert np.all(np.diff(c.ravel()[order]) >= 0)


@pytest.mark.parametrize("name,tau,h", POINTS)
def test_c_oracle_agrees_with_double_math(oracle, name, tau, h):
    rng = np.random.default_rng(2)
    x = -np.abs(rng.normal(0, 4, (512, 128)))
    x[rng.random(x.shape) < 0.02] = -np.inf
    x = x.astype(np.float32)
    c, k = _probgen_blocks(oracle, x, tau, h)
    cm, km = efq_math.efq_blocks(x, tau, h)
    assert np.array_equal(k, km)
    diff = c != cm
    assert diff.mean() < 1e-4 and np.all(np.abs(c - cm) <= 1)


def test_top_code_of_block_maximum(oracle):
    """The block maximum maps to code 7 whenever tau + 6/h <= ln(3/4); otherwise it can fall lower."""
    rng = np.random.default_rng(3)
    x = -np.abs(rng.normal(0, 5, (2000, 32))).astype(np.float32)
    for name, tau, h in POINTS:
        c, _ = _probgen_blocks(oracle, x, tau, h)
        top = c[np.arange(x.shape[0]), x.argmax(1)]
        if tau + 6.0 / h <= math.log(0.75):
            assert name == "EFQ-Mean" and np.all(top == 7)
        else:
            lo = math.floor((math.log(0.75) - tau) * h) + 1
            assert np.all(top >= lo) and np.all(top <= 7) and top.min() < 7


def test_worked_example(oracle):
    for ln in _read("efq_worked_example.txt"):
        parts = ln.split()
        k = int(parts[0])
        xs = [float(p.split(":")[0]) for p in parts[1:]]
        cs = [int(p.split(":")[1]) for p in parts[1:]]
        x = np.full((1, 32), -np.inf, np.float32)
        x[0, : len(xs)] = xs
        c, kk = _probgen_blocks(oracle, x, *MEAN)
        assert kk[0, 0] == k and list(c[0, : len(xs)]) == cs


def test_probability_value_tracks_exp(oracle):
    """e^x = s_b * 6 e^z, so s_b * C8[c] / e^x = C8[c] / (6 e^z) must stay inside the band the
    thresholds imply: a dropped term or wrong sign in the residual leaves it at once."""
    tau, h = MEAN
    rng = np.random.default_rng(4)
    x = -np.abs(rng.normal(0, 3, (1000, 64))).astype(np.float32)
    c, k = _probgen_blocks(oracle, x, tau, h)
    p = efq_math.dequant_probabilities(c, k)
    ratio = p / np.exp(x.astype(np.float64))
    live = (c >= 1)
    assert live.mean() > 0.3
    assert ratio[live].min() > 0.6 and ratio[live].max() < 2.4
    # code 0 only for elements far below the block maximum: 6 e^z < first threshold
    z = efq_math.residual(x.reshape(1000, 2, 32), k[..., None]).reshape(1000, 64)
    assert np.all(z[c == 0] < tau + 1e-5)


def test_ragged_tail_block(oracle):
    rng = np.random.default_rng(5)
    x = -np.abs(rng.normal(0, 3, (9, 88))).astype(np.float32)   # 88 = 2*32 + 24
    xp = np.concatenate([x, np.full((9, 8), -np.inf, np.float32)], axis=1)
    pk, sc = oracle.probgen(x, np.zeros(9, np.float32), 1.0, *MEAN)
    pk2, sc2 = oracle.probgen(xp, np.zeros(9, np.float32), 1.0, *MEAN)
    assert pk.shape == (9, 48) and np.array_equal(pk, pk2) and np.array_equal(sc, sc2)
    assert np.all(oracle.unpack_codes(pk)[:, 88:] == 0)


def test_shift_equivariance_of_the_equations():
    rng = np.random.default_rng(6)
    x = -np.abs(rng.normal(0, 3, (64, 64)))
    c0, k0 = efq_math.efq_blocks(x, *MEAN)
    for n in (1, 5, 17):
        c1, k1 = efq_math.efq_blocks(x - n * LN2, *MEAN)
        assert np.array_equal(k1, k0 - n)
        assert (c1 != c0).mean() < 1e-3


# ---------------------------------------------------------------------------------------
# MXFP4 operand quantiser and the exp-then-quantize producer
# ---------------------------------------------------------------------------------------

def test_mxfp4_roundtrip_and_ties(oracle):
    vals = []
    for e in (-20, -3, 0, 1, 9):
        blk = [6.0 * 2.0 ** e] + [s * v * 2.0 ** e for v in efq_math.C8 for s in (1, -1)]
        vals.append(blk + [0.0] * (32 - len(blk)))
    x = np.array(vals, np.float32)
    xhat, codes, scales = oracle.mxfp4_rows(x)
    assert np.array_equal(xhat, x)
    assert list(scales[:, 0]) == [127 - 20, 127 - 3, 127, 128, 136]
    ties = [tuple(float(t) for t in ln.split()) for ln in _read("e2m1_rne_ties.txt")]
    blk = np.zeros((1, 32), np.float32)
    blk[0, 0] = 6.0
    for i, (mid, _) in enumerate(ties):
        blk[0, 1 + i] = mid
        blk[0, 10 + i] = -mid
    xhat, _, _ = oracle.mxfp4_rows(blk)
    for i, (_, want) in enumerate(ties):
        assert xhat[0, 1 + i] == want and xhat[0, 10 + i] == -want


def test_mxfp4_is_nearest_and_scale_puts_amax_in_4_8(oracle):
    rng = np.random.default_rng(7)
    x = (rng.normal(0, 1, (300, 128)) * np.exp2(rng.integers(-6, 6, (300, 1)))).astype(np.float32)
    x = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(x))
    xhat, codes, scales = oracle.mxfp4_rows(x)
    e = scales.astype(np.int64) - 127
    amax = np.abs(x).reshape(300, 4, 32).max(-1)
    assert np.all(amax / np.exp2(e) >= 4.0) and np.all(amax / np.exp2(e) < 8.0)
    y = np.abs(x.astype(np.float64)).reshape(300, 4, 32) / np.exp2(e)[..., None]
    got = np.abs(xhat.astype(np.float64)).reshape(300, 4, 32) / np.exp2(e)[..., None]
    best = np.abs(np.minimum(y, 6.0)[..., None] - efq_math.C8).min(-1)      # brute force over the code set
    assert np.allclose(np.abs(np.minimum(y, 6.0) - got), best, atol=0, rtol=0)
    assert np.all(np.sign(xhat) * np.sign(x) >= 0)
    # column-wise variant is the same quantiser on the transpose
    xt = np.ascontiguousarray(x[:64].T)                # [128, 64]: blocks of 32 along axis 0
    that, _, tsc = oracle.mxfp4_cols(xt)
    rhat, _, rsc = oracle.mxfp4_rows(np.ascontiguousarray(xt.T))
    assert np.array_equal(that.T, rhat) and np.array_equal(tsc.T, rsc)


def test_etq_producer_is_nearest_code_of_exp(oracle):
    rng = np.random.default_rng(8)
    x = -np.abs(rng.normal(0, 3, (400, 64))).astype(np.float32)
    c, k = _probgen_blocks(oracle, x, *MEAN, producer="etq")
    p = np.exp(x.astype(np.float64)).reshape(400, 2, 32)
    amax = p.max(-1)
    assert np.array_equal(k, np.floor(np.log2(amax)).astype(np.int64) - 2)
    y = p / np.exp2(k)[..., None]
    got = efq_math.C8[c].reshape(400, 2, 32)
    best = np.abs(np.minimum(y, 6.0)[..., None] - efq_math.C8).min(-1)
    err = np.abs(np.minimum(y, 6.0) - got)
    assert np.all(err <= best + 1e-6)
    top = c.reshape(400, 2, 32)[np.arange(400)[:, None], np.arange(2)[None, :], p.argmax(-1)]
    assert np.all(top >= 6)
    # scale6 variant: maximum lands in (3, 6], never saturates
    c6, k6 = _probgen_blocks(oracle, x, *MEAN, producer="etq6")
    y6 = amax / np.exp2(k6)
    assert np.all(y6 > 3.0 - 1e-9) and np.all(y6 <= 6.0 + 1e-9)


# ---------------------------------------------------------------------------------------
# attention level
# ---------------------------------------------------------------------------------------

def _small_case(S=320, Hq=4, Hkv=2, causal=False, seed=11):
    case = inputs.AttentionCase("t", 1, Hq, Hkv, S, S, 128, causal, seed, "iid")
    q, k, v = (inputs.bf16_bits_to_f32(t) for t in inputs.make_qkv(case))
    rows = np.array([(0, h, i) for h in range(Hq) for i in range(0, S, 7)], np.int64)
    return case, q, k, v, rows


@pytest.mark.parametrize("causal", [False, True])
def test_exact_path_matches_library_attention(oracle, causal):
    import torch
    case, q, k, v, rows = _small_case(causal=causal)
    out = oracle.attention_rows(q, k, v, rows, causal, case.softmax_scale, "exact")
    tq, tk, tv = (torch.from_numpy(t).double() for t in (q, k, v))
    g = case.Hq // case.Hkv
    ref = torch.nn.functional.scaled_dot_product_attention(
        tq, tk.repeat_interleave(g, 1), tv.repeat_interleave(g, 1), is_causal=causal,
        scale=case.softmax_scale).numpy()
    want = ref[rows[:, 0], rows[:, 1], rows[:, 2]]
    assert np.abs(out - want).max() < 1e-6


@pytest.mark.parametrize("path", ["efq", "etq", "efq_lut"])
@pytest.mark.parametrize("causal", [False, True])
def test_online_recurrence_closed_form(oracle, path, causal):
    """Unrolled recurrence: O = sum_j w_j dA_j / sum_j w_j dl_j with w_j = exp(m_j - m_last),
    rebuilt in numpy from the dumped operand (codes, scales, per-tile maxima) and an
    independently dequantised V; also pins GQA head mapping and causal masking."""
    case, q, k, v, rows = _small_case(causal=causal)
    Bc = 128
    out, d = oracle.attention_rows(q, k, v, rows, causal, case.softmax_scale, path, Bc=Bc, dumps=True)
    codes = oracle.unpack_codes(d["codes"])[:, : case.Sk].astype(np.int64)
    kexp = d["scales"].astype(np.int64) - 127
    p = efq_math.dequant_probabilities(codes, kexp)
    ms = d["ms"].astype(np.float64)
    g = case.Hq // case.Hkv
    for n, (b, h, i) in enumerate(rows):
        vhat, _, _ = oracle.mxfp4_cols(v[b, h // g])
        nvis = i + 1 if causal else case.Sk
        assert np.all(np.isneginf(d["raw"][n, nvis:])) and np.all(np.isfinite(d["raw"][n, :nvis]))
        last = (nvis - 1) // Bc
        w = np.exp(ms[n, : last + 1] - ms[n, last])
        pw = p[n].copy()
        for j in range(last + 1):
            pw[j * Bc:(j + 1) * Bc] *= w[j]
        pw[(last + 1) * Bc:] = 0.0
        want = (pw @ vhat.astype(np.float64)) / pw.sum()
        assert np.abs(out[n] - want).max() < 1e-6
        # running maximum per tile is the scaled prefix maximum of the raw scores
        pref = np.maximum.accumulate(d["raw"][n, :nvis])
        for j in range(last + 1):
            t_end = min((j + 1) * Bc, nvis) - 1
            assert ms[n, j] == np.float32(np.float32(case.softmax_scale) * pref[t_end])


def test_raw_scores_are_exact_dot_products_of_dequantised_operands(oracle):
    case, q, k, v, rows = _small_case()
    _, d = oracle.attention_rows(q, k, v, rows[:20], False, case.softmax_scale, "efq", dumps=True)
    for n, (b, h, i) in enumerate(rows[:20]):
        qh, _, _ = oracle.mxfp4_rows(q[b, h, i:i + 1])
        kh, _, _ = oracle.mxfp4_rows(k[b, h // 2])
        want = (kh.astype(np.float64) @ qh[0].astype(np.float64)).astype(np.float32)
        assert np.array_equal(d["raw"][n], want)


def test_one_shot_matches_equations_and_single_operand(oracle):
    """With one KV tile the path is closed form: codes from the double-precision equations on
    x = sigma r - max, and O = (P~ V^) / (P~ 1)."""
    case, q, k, v, rows = _small_case(S=256)
    out, d = oracle.attention_rows(q, k, v, rows, False, case.softmax_scale, "efq", Bc=256, dumps=True)
    codes = oracle.unpack_codes(d["codes"]).astype(np.int64)
    kexp = d["scales"].astype(np.int64) - 127
    x = d["raw"].astype(np.float64) * np.float32(case.softmax_scale)
    x = x - x.max(1, keepdims=True)
    cm, km = efq_math.efq_blocks(x, *MEAN)
    assert (cm != codes).mean() < 2e-4 and np.abs(cm - codes).max() <= 1
    assert (km != kexp).mean() < 2e-3
    p = efq_math.dequant_probabilities(codes, kexp)
    for n, (b, h, i) in enumerate(rows):
        vhat, _, _ = oracle.mxfp4_cols(v[b, h // 2])
        assert np.abs(out[n] - efq_math.attention_from_operand(p[n:n + 1], vhat)[0]).max() < 1e-6
    # the standalone stage on the same scores with the final row maximum gives the same operand
    rm = (np.float32(case.softmax_scale) * d["raw"].max(1)).astype(np.float32)
    pk, sc = oracle.probgen(d["raw"], rm, case.softmax_scale, *MEAN)
    assert np.array_equal(pk, d["codes"]) and np.array_equal(sc, d["scales"])


def test_tiled_equals_one_shot_when_maximum_is_in_first_tile(oracle):
    rng = np.random.default_rng(12)
    r = rng.normal(0, 8, (50, 512)).astype(np.float32)
    r[:, 3] = 60.0
    c1, s1, _ = oracle.online_codes(r, 128, 0.25)
    c2, s2, _ = oracle.online_codes(r, 512, 0.25)
    assert np.array_equal(c1, c2) and np.array_equal(s1, s2)
    r[:, 400] = 68.0                      # maximum arrives in tile 3: tiles 0-2 were coded against the smaller one
    c3, s3, _ = oracle.online_codes(r, 128, 0.25)
    c4, s4, _ = oracle.online_codes(r, 512, 0.25)
    assert np.array_equal(s3[:, :12], s1[:, :12]) and np.array_equal(c3[:, :192], c1[:, :192])
    assert np.array_equal(s3[:, 12:], s4[:, 12:]) and np.array_equal(c3[:, 192:], c4[:, 192:])
    drop = s3[:, :12].astype(int) - s4[:, :12].astype(int)   # 2 units of x = 2/ln 2 = 2.885 octaves
    assert np.all((drop == 2) | (drop == 3)) and (drop == 3).mean() > 0.7
    

def test_uniform_row_gives_mean_of_values(oracle):
    case, q, k, v, rows = _small_case(S=192)
    q[:] = 0.0
    for path in ("efq", "etq"):
        out = oracle.attention_rows(q, k, v, rows, False, case.softmax_scale, path)
        for n, (b, h, i) in enumerate(rows):
            vhat, _, _ = oracle.mxfp4_cols(v[b, h // 2])
            assert np.abs(out[n] - vhat.astype(np.float64).mean(0)).max() < 1e-6


def test_single_visible_key_returns_its_value(oracle):
    case, q, k, v, rows = _small_case(S=160, causal=True)
    r0 = np.array([(0, h, 0) for h in range(case.Hq)], np.int64)
    for path in ("efq", "etq", "exact"):
        out = oracle.attention_rows(q, k, v, r0, True, case.softmax_scale, path)
        for n, (b, h, i) in enumerate(r0):
            want = v[b, h // 2][0] if path == "exact" else oracle.mxfp4_cols(v[b, h // 2])[0][0]
            assert np.abs(out[n] - want).max() < 1e-6


@pytest.mark.parametrize("path", ["efq", "etq", "efq_lut"])
def test_output_is_convex_combination_and_near_exact(oracle, path):
    case, q, k, v, rows = _small_case(S=384)
    out = oracle.attention_rows(q, k, v, rows, False, case.softmax_scale, path)
    ex = oracle.attention_rows(q, k, v, rows, False, case.softmax_scale, "exact")
    for n, (b, h, i) in enumerate(rows):
        vhat, _, _ = oracle.mxfp4_cols(v[b, h // 2])
        assert np.all(out[n] <= vhat.max(0) + 1e-6) and np.all(out[n] >= vhat.min(0) - 1e-6)
    rel = np.linalg.norm(out - ex) / np.linalg.norm(ex)
    assert rel < 0.35       # loose sanity bound; the paper prints no error figure (parity unpinned)


def test_lut_variant_fold_table():
    z = np.linspace(-6, 0.5, 20001)
    c = efq_math.lut16_code(z)
    assert c.min() == 0 and c.max() == 7 and np.all(np.diff(c) >= 0)
    assert efq_math.lut16_code(np.array([math.log(1 / 24) - 1e-9]))[0] == 0


# ---------------------------------------------------------------------------------------
# LUT variant (Sec. "EFQ-Softmax-LUT Variant"): 16-level index, folding table
# ---------------------------------------------------------------------------------------

# The folding table steps at j = 1, 6, 8, 10, 11, 13, 14, and j >= n  <=>  z >= tau16 + (n-1)/h16, so with
# tau16 = ln(1/24), h16 = 14/ln 24 the code is the number of thresholds 0.25 * 24^((n-1)/14) that the
# block-normalised probability 6 e^z has reached: a closed form with no floor, no table and no (tau, h).
LUT_STEPS = (1, 6, 8, 10, 11, 13, 14)
LUT_THRESHOLDS = np.array([0.25 * 24.0 ** ((n - 1) / 14.0) for n in LUT_STEPS])


def test_lut_thresholds_sit_next_to_the_e2m1_rounding_boundaries():
    rne = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])     # midpoints between neighbouring E2M1 values
    assert LUT_THRESHOLDS[0] == 0.25
    assert np.all(np.abs(LUT_THRESHOLDS / rne - 1.0) < 0.11)
    assert abs(0.25 * 24.0 ** (14 / 14.0) - 6.0) < 1e-12        # z = 0 (p~ = 6 * 2^k) is the j = 14 | 15 boundary


def test_lut_codes_count_thresholds(oracle):
    rng = np.random.default_rng(11)
    x = -rng.uniform(0, 9, (600, 32)).astype(np.float32)
    x[:, 0] = -rng.uniform(0, 3, 600).astype(np.float32)           # block maximum
    x[:, 0] = np.maximum(x[:, 0], x.max(axis=1))
    c, k = _probgen_blocks(oracle, x, 0.0, 1.0, producer="efq_lut")  # (tau, h) must not matter
    c2, k2 = _probgen_blocks(oracle, x, *MEAN, producer="efq_lut")
    assert np.array_equal(c, c2) and np.array_equal(k, k2)
    _, k_affine = _probgen_blocks(oracle, x, *MEAN)
    assert np.array_equal(k, k_affine)                              # the same block scale as the main method
    xd = x.astype(np.float64)
    p6 = 6.0 * np.exp(xd - k.astype(np.float64) * LN2 - LN6)        # 6 e^z = e^x / 2^k
    want = (p6[..., None] >= LUT_THRESHOLDS).sum(-1)
    edge = (np.abs(p6[..., None] / LUT_THRESHOLDS - 1.0) < 1e-4).any(-1)
    assert edge.mean() < 0.01
    assert np.array_equal(c[~edge], want[~edge])
    assert np.all(np.abs(c - want) <= 1)
    # fp64 evaluation of the printed equations (floor + table) agrees off the knife edges too
    z = xd - k.astype(np.float64) * LN2 - LN6
    assert np.array_equal(efq_math.lut16_code(z)[~edge], c[~edge])
    assert c.min() >= 0 and c.max() <= 7


def test_lut_block_maximum_code(oracle):
    # 6 e^{z_max} lies in [4.5, 9): the block maximum gets code 7 from 0.25 * 24^(13/14) = 4.78 on, else 6
    M = -np.linspace(0.0, 30.0, 3001)
    x = np.full((M.size, 32), -np.inf, np.float32)
    x[:, 7] = M.astype(np.float32)
    c, k = _probgen_blocks(oracle, x, *MEAN, producer="efq_lut")
    p6 = np.exp(x[:, 7].astype(np.float64)) / np.exp2(k[:, 0].astype(np.float64))
    assert np.all(p6 >= 4.5 * (1 - 1e-5)) and np.all(p6 < 9.0 * (1 + 1e-5))
    edge = np.abs(p6 / LUT_THRESHOLDS[-1] - 1.0) < 1e-4
    assert np.array_equal(c[~edge, 7], np.where(p6[~edge] >= LUT_THRESHOLDS[-1], 7, 6))
    assert set(np.unique(c[:, 7])) == {6, 7}


def test_lut_is_monotone_and_masked_keys_are_zero(oracle):
    x = np.linspace(-12.0, 0.0, 64, dtype=np.float32)[None, :].repeat(2, 0)
    x[1, ::5] = -np.inf
    c, _ = _probgen_blocks(oracle, x, *MEAN, producer="efq_lut")
    assert np.all(np.diff(c[0, :32]) >= 0) and np.all(np.diff(c[0, 32:]) >= 0)
    assert np.all(c[1, ::5] == 0)


def test_lut_attention_is_closer_to_exact_than_the_affine_rule(oracle):
    # the finer intermediate index places the thresholds next to the nearest-rounding boundaries of E2M1
    # (Sec. "EFQ-Softmax-LUT Variant": the accuracy-oriented comparison point)
    case, q, k, v, rows = _small_case(S=384)
    ex = oracle.attention_rows(q, k, v, rows, False, case.softmax_scale, "exact")
    err = {}
    for path in ("efq", "efq_lut", "etq"):
        out = oracle.attention_rows(q, k, v, rows, False, case.softmax_scale, path)
        err[path] = np.linalg.norm(out - ex) / np.linalg.norm(ex)
    assert err["efq_lut"] < err["efq"]
    assert err["efq_lut"] < 1.5 * err["etq"]


# ---------------------------------------------------------------------------------------
# thresholded rescaling (not in the paper; threshold 0 is Algorithm 2)
# ---------------------------------------------------------------------------------------

def _policy_reference(tile_max_raw, sigma, T):
    """The shifting maximum per tile, recomputed from the tile maxima alone in float32."""
    f = np.float32
    used = f(-np.inf)
    out = []
    for t in tile_max_raw:
        cand = max(used, f(t))
        if used == -np.inf or not T > 0:
            used = cand
        elif f(f(f(sigma) * cand) - f(f(sigma) * used)) > f(T):
            used = cand
        out.append(f(f(sigma) * used))
    return np.array(out, np.float32)


@pytest.mark.parametrize("T", [0.0, 0.75, 3.0, 1e9])
def test_threshold_policy_of_the_shifting_maximum(oracle, T):
    rng = np.random.default_rng(21)
    sigma = float(np.float32(0.125))
    raw = (rng.normal(0, 12, (16, 1024)) + np.linspace(0, 40, 1024)[None, :]).astype(np.float32)  # maxima keep growing
    raw[3, :200] = -np.inf
    codes, scales, ms = oracle.online_codes(raw, 128, sigma, *MEAN, rescale_threshold=T)
    c0, s0, ms0 = oracle.online_codes(raw, 128, sigma, *MEAN)
    tile_max = raw.reshape(16, 8, 128).max(-1)
    for i in range(16):
        assert np.array_equal(ms[i], _policy_reference(tile_max[i], sigma, T))
    if T == 0.0:
        assert np.array_equal(codes, c0) and np.array_equal(scales, s0) and np.array_equal(ms, ms0)
    else:
        with np.errstate(invalid="ignore"):
            assert np.all((ms <= ms0) | np.isnan(ms0 - ms))          # never above the true running maximum
            gap = ms0 - ms
        assert np.nanmax(gap) <= T * (1 + 1e-6) + 1e-6               # and at most T below it
        assert (np.diff(ms, axis=1) != 0).sum() < (np.diff(ms0, axis=1) != 0).sum() or T < 1.0
    if T >= 1e9:
        assert np.all(ms[:, 1:] == ms[:, :1]) or np.isinf(ms[3, 0])   # the first finite maximum is kept for good


def test_threshold_policy_codes_are_the_stage_codes_for_the_kept_maximum(oracle):
    """Per tile, the operand equals the standalone stage run with row_max = the kept maximum: the policy changes
    which maximum shifts the scores and nothing else; shifted scores above zero only raise the block exponents."""
    rng = np.random.default_rng(22)
    sigma = float(np.float32(0.2))
    raw = (rng.normal(0, 8, (8, 512)) + np.linspace(0, 25, 512)[None, :]).astype(np.float32)
    codes, scales, ms = oracle.online_codes(raw, 128, sigma, *MEAN, rescale_threshold=2.5)
    assert scales.max() > 124                                          # some block maximum sits above the kept maximum
    for j in range(4):
        tile = np.ascontiguousarray(raw[:, 128 * j:128 * (j + 1)])
        c, s = oracle.probgen(tile, ms[:, j].copy(), sigma, *MEAN)
        assert np.array_equal(c, codes[:, 64 * j:64 * (j + 1)]) and np.array_equal(s, scales[:, 4 * j:4 * (j + 1)])
    # shift-equivariance: against threshold 0 the codes agree wherever the two maxima differ by a multiple of
    # ln 2 ... in general they differ, but the represented probabilities relative to the same reference agree
    c0, s0, ms0 = oracle.online_codes(raw, 128, sigma, *MEAN)
    p = efq_math.C8[oracle.unpack_codes(codes)] * np.repeat(np.exp2(scales.astype(float) - 127), 32, 1) * \
        np.repeat(np.exp(ms.astype(float)), 128, 1)
    p0 = efq_math.C8[oracle.unpack_codes(c0)] * np.repeat(np.exp2(s0.astype(float) - 127), 32, 1) * \
        np.repeat(np.exp(ms0.astype(float)), 128, 1)
    big = p0 > 1e-3 * p0.max(axis=1, keepdims=True)
    both = big & (p > 0)
    assert both.sum() > 0.9 * big.sum()                                 # the smallest code may fall to zero, rarely
    assert np.all(np.abs(np.log(p[both] / p0[both])) < 0.75)            # same value up to one code step


@pytest.mark.parametrize("path", ["efq", "etq", "efq_lut"])
def test_threshold_policy_leaves_the_attention_output_in_the_same_error_band(oracle, path):
    case, q, k, v, rows = _small_case(S=384)
    ex = oracle.attention_rows(q, k, v, rows, True, case.softmax_scale, "exact")
    o0 = oracle.attention_rows(q, k, v, rows, True, case.softmax_scale, path)
    oT = oracle.attention_rows(q, k, v, rows, True, case.softmax_scale, path, rescale_threshold=4.0)
    e0 = np.linalg.norm(o0 - ex) / np.linalg.norm(ex)
    eT = np.linalg.norm(oT - ex) / np.linalg.norm(ex)
    assert abs(eT - e0) < 0.25 * e0
    assert np.linalg.norm(oT - o0) / np.linalg.norm(o0) < e0


def test_fp32_denominator_variant_of_the_baseline(oracle):
    """Context variant: the quantised operand in the numerator, FP32 exponentials in the denominator.  With one KV
    tile it is the closed form sum(p~ v^) / sum(exp(x)); against the shared-operand rule it differs by the ratio of
    the two denominators, row by row."""
    case, q, k, v, rows = _small_case(S=96)
    sigma = case.softmax_scale
    o_sh, d = oracle.attention_rows(q, k, v, rows, False, sigma, "etq", Bc=128, dumps=True)
    o_fp = oracle.attention_rows(q, k, v, rows, False, sigma, "etq_fp32den", Bc=128)
    codes = oracle.unpack_codes(d["codes"])[:, :96]
    p_q = efq_math.C8[codes] * np.repeat(np.exp2(d["scales"].astype(float) - 127), 32, 1)[:, :96]
    x = (np.float32(sigma) * d["raw"]).astype(np.float32) - d["ms"][:, :1]
    p_f = np.exp(x.astype(np.float64)).astype(np.float32).astype(np.float64)
    ratio = p_q.sum(1) / p_f.sum(1)
    assert np.abs(o_fp - o_sh * ratio[:, None]).max() < 1e-5
    assert np.abs(ratio - 1.0).max() < 0.2 and np.abs(ratio - 1.0).max() > 1e-4


# ---------------------------------------------------------------------------------------
# causal alignment with Sq != Sk, and the ragged last block of the V quantiser
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("Sq,Sk", [(100, 700), (260, 200)])
def test_causal_mask_is_bottom_right_aligned_when_sq_differs_from_sk(oracle, Sq, Sk):
    """Query i sees keys t <= i + Sk - Sq (the last query sees every key).  The exact path is compared with a
    library softmax attention under that explicit boolean mask, so a top-left alignment (t <= i) fails; rows
    that see no key (Sq > Sk, i < Sq - Sk) are zero; the dumped raw scores of the EFQ path are -inf exactly on
    the masked keys."""
    import torch
    case = inputs.AttentionCase("t", 1, 4, 2, Sq, Sk, 128, True, 21, "iid")
    q, k, v = (inputs.bf16_bits_to_f32(t) for t in inputs.make_qkv(case))
    rows = np.array([(0, h, i) for h in range(4) for i in sorted({0, 1, Sq // 3, max(Sq - Sk, 0), Sq - 2, Sq - 1}
                                                                 | set(range(5, Sq, 37)))], np.int64)
    i_idx = torch.arange(Sq)[:, None]
    t_idx = torch.arange(Sk)[None, :]
    mask = t_idx <= i_idx + (Sk - Sq)
    tq, tk, tv = (torch.from_numpy(t).double() for t in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(
        tq, tk.repeat_interleave(2, 1), tv.repeat_interleave(2, 1), attn_mask=mask, scale=case.softmax_scale).numpy()
    out = oracle.attention_rows(q, k, v, rows, True, case.softmax_scale, "exact")
    nvis = np.clip(rows[:, 2] + Sk - Sq + 1, 0, Sk)
    seen = nvis > 0
    assert seen.any() and (Sq <= Sk or (~seen).any())
    want = ref[rows[:, 0], rows[:, 1], rows[:, 2]]
    assert np.abs(out[seen] - want[seen]).max() < 1e-6
    assert np.all(out[~seen] == 0.0)
    for path in ("efq", "etq"):
        o, d = oracle.attention_rows(q, k, v, rows, True, case.softmax_scale, path, dumps=True)
        for n in range(rows.shape[0]):
            assert np.all(np.isfinite(d["raw"][n, :nvis[n]])) and np.all(np.isneginf(d["raw"][n, nvis[n]:]))
        assert np.all(o[~seen] == 0.0) and np.all(np.isfinite(o))
        # a quantised path stays in the neighbourhood of the exact one only under the same alignment
        rel = np.linalg.norm(o[seen] - out[seen]) / np.linalg.norm(out[seen])
        assert rel < 0.5


def test_v_quantiser_ragged_last_block_equals_zero_padded_block(oracle):
    """88 keys = 2 full blocks + 24: the last block takes its maximum over the 24 valid keys only, which is what
    quantising the matrix padded with zero rows to 96 keys gives (zeros change neither the maximum nor any code).
    Checked against the padded column quantiser and against the row quantiser on the padded transpose."""
    rng = np.random.default_rng(31)
    v = (rng.normal(0, 1, (88, 128)) * np.exp2(rng.integers(-3, 4, (1, 128)))).astype(np.float32)
    v = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(v))
    v[64:, 5] = 0.0                                  # a channel whose ragged block is all zero: byte 0
    v[87, 9] = 37.0                                  # the last valid key carries its block's maximum
    vp = np.zeros((96, 128), np.float32)
    vp[:88] = v
    hat, codes, sc = oracle.mxfp4_cols(v)
    hat_p, codes_p, sc_p = oracle.mxfp4_cols(vp)
    assert np.array_equal(hat, hat_p[:88]) and np.array_equal(codes, codes_p[:88]) and np.array_equal(sc, sc_p)
    rhat, rcodes, rsc = oracle.mxfp4_rows(np.ascontiguousarray(vp.T))       # blocks of 32 along the padded keys
    assert np.array_equal(hat, rhat.T[:88]) and np.array_equal(codes, rcodes.T[:88]) and np.array_equal(sc, rsc.T)
    assert sc[2, 5] == 0 and np.all(hat[64:, 5] == 0.0)
    assert sc[2, 9] == 127 + 3 and hat[87, 9] == 32.0     # 37 = 4.625 * 2^3 -> nearest code 4: the last key is really quantised


@pytest.mark.parametrize("path", ["efq", "etq", "efq_lut"])
def test_attention_with_ragged_key_count_matches_closed_form(oracle, path):
    """Sk = 88 (one KV tile, last block of 24 keys): O rebuilt from the dumped operand and a V dequantised through
    the zero-padded matrix - (P~ V^) / (P~ 1) - so a key dropped from the ragged block, in the value quantiser or
    in the producer, shows."""
    case = inputs.AttentionCase("t", 1, 4, 2, 88, 88, 128, False, 33, "iid")
    q, k, v = (inputs.bf16_bits_to_f32(t) for t in inputs.make_qkv(case))
    rows = np.array([(0, h, i) for h in range(4) for i in range(0, 88, 5)], np.int64)
    out, d = oracle.attention_rows(q, k, v, rows, False, case.softmax_scale, path, Bc=128, dumps=True)
    codes = oracle.unpack_codes(d["codes"])[:, :88].astype(np.int64)
    kexp = d["scales"].astype(np.int64) - 127
    assert kexp.shape[1] == 3
    p = efq_math.dequant_probabilities(np.pad(codes, ((0, 0), (0, 8))), kexp)[:, :88]
    assert np.all(p[:, 87] >= 0) and (p[:, 64:] > 0).any()
    for n, (b, h, i) in enumerate(rows):
        vp = np.zeros((96, 128), np.float32)
        vp[:88] = v[b, h // 2]
        vhat = oracle.mxfp4_rows(np.ascontiguousarray(vp.T))[0].T[:88]
        want = efq_math.attention_from_operand(p[n:n + 1], vhat)[0]
        assert np.abs(out[n] - want).max() < 1e-6
    # the block maximum of the ragged block is over its 24 valid keys: top code region, never a masked key
    if path == "efq":
        x = d["raw"][:, 64:88].astype(np.float64)
        top = codes[:, 64:88][np.arange(rows.shape[0]), x.argmax(1)]
        assert np.all(top == 7)
