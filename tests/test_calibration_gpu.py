"""GPU parity of the calibration helpers (Algorithm 3): the FP32 reference attention, the relative
Frobenius error and the (tau, h) grid search, each against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2609_09721_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _to_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _tensors(case):
    qb, kb, vb = inputs.make_qkv(case)
    host = tuple(inputs.bf16_bits_to_f32(t) for t in (qb, kb, vb))
    dev = tuple(_to_dev(t) for t in (qb, kb, vb))
    return host, dev


@pytest.mark.parametrize("Sq,Sk,Hq,Hkv,causal,recipe", [
    (256, 256, 2, 1, False, "iid"), (300, 300, 4, 2, True, "k_outliers"), (100, 700, 1, 1, True, "iid"),
    (260, 200, 2, 2, True, "iid"), (33, 1000, 1, 1, False, "lowrank"), (1, 1, 1, 1, True, "iid")])
def test_exact_attention_matches_the_oracle(oracle, Sq, Sk, Hq, Hkv, causal, recipe):
    case = inputs.AttentionCase("x", 1, Hq, Hkv, Sq, Sk, 128, causal, 7 + Sq + Sk, recipe)
    (q, k, v), (dq, dk, dv) = _tensors(case)
    o = binding.efq_exact_attention_fwd(dq, dk, dv, causal)
    torch.cuda.synchronize()
    rows = np.array([(0, h, i) for h in range(Hq) for i in range(Sq)], np.int64)
    want = oracle.attention_rows(q, k, v, rows, causal, case.softmax_scale, "exact")
    got = o.cpu().numpy().reshape(-1, 128)
    assert np.abs(got - want).max() <= 2e-5
    # rows with no visible key (causal, Sq > Sk) are zero
    if causal and Sq > Sk:
        assert np.all(got.reshape(Hq, Sq, 128)[:, : Sq - Sk] == 0.0)


def test_exact_attention_batch_and_explicit_scale(oracle):
    case = inputs.AttentionCase("xb", 2, 2, 1, 130, 130, 128, True, 3, "iid")
    (q, k, v), (dq, dk, dv) = _tensors(case)
    o = binding.efq_exact_attention_fwd(dq, dk, dv, True, 0.2)
    torch.cuda.synchronize()
    rows = np.array([(b, h, i) for b in range(2) for h in range(2) for i in (0, 1, 63, 64, 129)], np.int64)
    want = oracle.attention_rows(q, k, v, rows, True, 0.2, "exact")
    got = o.cpu().numpy()
    for n, (b, h, i) in enumerate(rows):
        assert np.abs(got[b, h, i] - want[n]).max() <= 2e-5


def test_relative_error_is_the_frobenius_ratio():
    rng = np.random.default_rng(0)
    ref = rng.normal(0, 1, 100003).astype(np.float32)
    a = (ref + rng.normal(0, 0.01, ref.size)).astype(np.float32)
    want = np.linalg.norm(a.astype(np.float64) - ref) / np.linalg.norm(ref.astype(np.float64))
    got = binding.efq_relative_error(torch.from_numpy(a).cuda(), torch.from_numpy(ref).cuda())
    assert abs(got - want) <= 1e-12 + 1e-9 * want
    z = torch.zeros(10, dtype=torch.float32, device="cuda")
    assert binding.efq_relative_error(z, z) == 0.0
    assert binding.efq_relative_error(z + 1.0, z) == float("inf")


def test_grid_search_matches_the_oracle_objective(oracle):
    """rho(tau, h) of every candidate equals the objective evaluated with the CPU oracle (EFQ path against the
    exact path on the same inputs), and the selected pair is the oracle's."""
    case = inputs.AttentionCase("cal", 1, 2, 1, 384, 384, 128, True, 11, "iid")
    (q, k, v), (dq, dk, dv) = _tensors(case)
    taus = [-3.4, -3.06, -2.9, -2.1]
    hs = [1.7, 2.0, 2.3, 2.7]
    o_ref = binding.efq_exact_attention_fwd(dq, dk, dv, True)
    table, best = binding.efq_calibrate(dq, dk, dv, o_ref, taus, hs, True)
    rows = np.array([(0, h, i) for h in range(2) for i in range(384)], np.int64)
    ex = oracle.attention_rows(q, k, v, rows, True, case.softmax_scale, "exact").astype(np.float64)
    want = np.zeros((4, 4))
    for i, tau in enumerate(taus):
        for j, h in enumerate(hs):
            out = oracle.attention_rows(q, k, v, rows, True, case.softmax_scale, "efq", tau, h).astype(np.float64)
            want[i, j] = np.linalg.norm(out - ex) / np.linalg.norm(ex)
    got = np.array(table)
    assert np.abs(got - want).max() <= 2e-4, (got, want)
    i, j = np.unravel_index(np.argmin(want), want.shape)
    gap = np.partition(want.ravel(), 1)[1] - want.min()
    if gap > 5e-4:                       # a clear winner: the same pair must be selected
        assert best == (pytest.approx(taus[i]), pytest.approx(hs[j]))
    assert min(min(r) for r in table) == pytest.approx(got.min())
    print("rho table (rows tau, cols h):\n", np.round(got, 4), "\nselected", best)


def test_calibrate_argument_errors():
    q = torch.zeros((1, 1, 128, 128), dtype=torch.bfloat16, device="cuda")
    o = torch.zeros((1, 1, 128, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.EfqError) as e:
        binding.efq_calibrate(q, q, q, o, [], [2.3])
    assert e.value.status == 1
    with pytest.raises(binding.EfqError) as e:
        binding.efq_calibrate(q, q, q, o, [-3.0], [-1.0])     # h must be positive
    assert e.value.status == 1
