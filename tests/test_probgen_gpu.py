"""GPU parity of the standalone probability-generation stage against the CPU oracle,
called through the C ABI.  EFQ: codes and scale bytes bit-exact.  exp-then-quantize:
statistical parity (the device exponential is an approximation)."""
import numpy as np
import pytest
import torch

from paper_2609_09721_b200 import binding, inputs

pytestmark = pytest.mark.gpu

POINTS = [(-3.06, 2.30), (-2.90, 2.00), (-2.10, 2.70)]


def _run_gpu(fn, scores, row_max, *args, ld=None, **kw):
    rows, cols = scores.shape
    if ld is None:
        d_scores = torch.from_numpy(scores).cuda()
    else:
        buf = torch.full((rows, ld), float("nan"), dtype=torch.float32, device="cuda")
        buf[:, :cols] = torch.from_numpy(scores).cuda()
        d_scores = buf[:, :cols]
    codes, scales = fn(d_scores, torch.from_numpy(row_max).cuda(), *args, **kw)
    torch.cuda.synchronize()
    return codes.cpu().numpy(), scales.cpu().numpy()


@pytest.mark.parametrize("tau,h", POINTS)
@pytest.mark.parametrize("rows,cols,ld", [(64, 4096, None), (37, 1024 * 3 + 32 * 5, None), (5, 32760, 32768),
                                          (9, 88, 96), (3, 31, 32), (1, 1, 4), (130, 2048 + 1000, 4096)])
def test_efq_probgen_bit_exact(oracle, tau, h, rows, cols, ld):
    scores, row_max = inputs.make_score_matrix(rows, cols, seed=20 + rows)
    if cols > 64:
        scores[0, 40:104] = -np.inf                      # fully masked blocks
        scores[min(1, rows - 1), : cols // 2] = -np.inf  # half-masked row
    want_c, want_s = oracle.probgen(scores, row_max, 1.0, tau, h)
    got_c, got_s = _run_gpu(binding.efq_probgen, scores, row_max, 1.0, (tau, h), ld=ld)
    assert np.array_equal(got_s, want_s)
    assert np.array_equal(got_c, want_c)


def test_efq_probgen_score_scale_and_foreign_row_max(oracle):
    """sigma != 1 and a row maximum that is not the maximum of this matrix (a running
    maximum from earlier tiles): still bit-exact."""
    scores, row_max = inputs.make_score_matrix(48, 2048, seed=5)
    sigma = float(np.float32(1.0 / np.sqrt(128.0)))
    rm = (np.float32(sigma) * row_max + np.float32(1.75)).astype(np.float32)
    want_c, want_s = oracle.probgen(scores, rm, sigma, -3.06, 2.30)
    got_c, got_s = _run_gpu(binding.efq_probgen, scores, rm, sigma, None)
    assert np.array_equal(got_s, want_s) and np.array_equal(got_c, want_c)


def test_efq_probgen_full_config(oracle):
    """The benchmarked workload: 4096 x 16384, N(0, 3^2) with 1 % of entries set to +12."""
    scores, row_max = inputs.make_score_matrix(4096, 16384, seed=2)
    want_c, want_s = oracle.probgen(scores, row_max, 1.0, -3.06, 2.30)
    got_c, got_s = _run_gpu(binding.efq_probgen, scores, row_max, 1.0, None)
    assert np.array_equal(got_s, want_s)
    assert np.array_equal(got_c, want_c)
    hist = np.bincount(oracle.unpack_codes(want_c[:64]).ravel(), minlength=8) / (64 * 16384)
    assert hist[0] > 0.3 and hist[7] > 0.01


@pytest.mark.parametrize("rows,cols,ld", [(64, 4096, None), (37, 1024 * 3 + 32 * 5, None), (5, 32760, 32768),
                                          (9, 88, 96), (3, 31, 32), (1, 1, 4)])
def test_efq_lut_probgen_bit_exact(oracle, rows, cols, ld):
    """variant 1: 16-level index + folding table; (tau, h) in the params are not read."""
    scores, row_max = inputs.make_score_matrix(rows, cols, seed=60 + rows)
    if cols > 64:
        scores[0, 40:104] = -np.inf
    want_c, want_s = oracle.probgen(scores, row_max, 1.0, producer="efq_lut")
    got_c, got_s = _run_gpu(binding.efq_probgen, scores, row_max, 1.0, (123.0, 0.5, 1), ld=ld)
    assert np.array_equal(got_s, want_s)
    assert np.array_equal(got_c, want_c)
    # same block scale as the affine rule, other codes
    aff_c, aff_s = oracle.probgen(scores, row_max, 1.0, -3.06, 2.30)
    assert np.array_equal(aff_s, want_s)
    if cols >= 1024:
        assert not np.array_equal(aff_c, want_c)


def test_efq_lut_probgen_full_config(oracle):
    scores, row_max = inputs.make_score_matrix(4096, 16384, seed=2)
    want_c, want_s = oracle.probgen(scores, row_max, 1.0, producer="efq_lut")
    got_c, got_s = _run_gpu(binding.efq_probgen, scores, row_max, 1.0, (0.0, 1.0, 1))
    assert np.array_equal(got_s, want_s)
    assert np.array_equal(got_c, want_c)


def test_probgen_unknown_variant_is_refused():
    scores = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    rm = torch.zeros(4, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.EfqError) as e:
        binding.efq_probgen(scores, rm, 1.0, (-3.06, 2.30, 2))
    assert e.value.status == 2


@pytest.mark.parametrize("mode,name", [(0, "etq"), (1, "etq6"), (2, "etq"), (3, "etq")])   # modes 2, 3: mode 0 with the scale folded into ex2 (3: part by polynomial)
def test_etq_probgen_statistical_parity(oracle, mode, name):
    scores, row_max = inputs.make_score_matrix(256, 4096 + 96, seed=7)
    scores[3, 100:300] = -np.inf
    want_c, want_s = oracle.probgen(scores, row_max, 1.0, producer=name)
    got_c, got_s = _run_gpu(binding.exp_then_quantize_probgen, scores, row_max, 1.0, mode)
    sdiff = got_s != want_s
    assert sdiff.mean() < 1e-3           # block maximum within rounding of a power of two
    ok_blocks = np.repeat(~sdiff, 16, axis=1)
    a = oracle.unpack_codes(got_c).astype(int)
    b = oracle.unpack_codes(want_c).astype(int)
    okm = np.repeat(ok_blocks, 2, axis=1)
    d = np.abs(a - b)[okm]
    assert d.max() <= 1 and (d != 0).mean() < 2e-3
    assert np.all((got_c & 0x88) == 0)


def test_probgen_reports_bad_arguments():
    s = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    rm = torch.zeros(4, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.EfqError) as e:
        binding.efq_probgen(s, rm, 1.0, (-3.06, float("nan")))
    assert e.value.status == 1
    with pytest.raises(binding.EfqError) as e:
        binding.efq_probgen(s[:, 1:33], rm, 1.0, None)      # base pointer off by 4 bytes
    assert e.value.status == 3
    with pytest.raises(binding.EfqError) as e:
        binding.efq_probgen(s, rm, 1.0, (-3.06, 2.3, 7))    # no such variant
    assert e.value.status == 2


def test_microbenchmarks_run_and_report_sane_rates():
    """The MMA-only FP4 loop and the in-SM producer loop finish (no expired wait) and land in a sane range."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    sink = torch.zeros(sms, dtype=torch.int32, device="cuda")
    flops = binding.efq_fp4_mma_peak_probe(sink, sms, 256)
    torch.cuda.synchronize()
    assert flops == 2.0 * 128 * 256 * 64 * 256 * sms
    assert (sink.cpu().numpy().view(np.uint32) != 0xDEADBEEF).all()
    rates = {}
    for prod in (0, 1):
        cyc = binding.efq_stage_microbench(prod, 2 * sms, 500)
        torch.cuda.synchronize()
        rates[prod] = 2 * 256 * 32 * 500 / float(cyc.double().mean())
    assert 5.0 < rates[1] < rates[0] < 64.0     # elements per clock per SM; exp-then-quantize is MUFU-bound
