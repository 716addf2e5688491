"""Host-side logic of bench.py without a GPU: workload table, FLOP accounting, the max-over-ranks reduction under
gloo with two processes, and the reference arm's rank handling."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2609_09721_b200 import inputs  # noqa: E402


def test_workloads_and_flop_accounting():
    c = bench.workload_case("qwen3_8b_16k")
    assert (c.B, c.Hq, c.Hkv, c.Sq, c.d, c.causal) == (1, 32, 8, 16384, 128, True)
    assert c.flops == 4 * 32 * 16384 * 16384 * 128 / 2
    w = bench.workload_case("wan22_32760")
    assert (w.Hq, w.Hkv, w.Sq, w.causal) == (24, 24, 32760, False) and w.Sq % 32 == 24
    rows = np.array([(0, 0, 0), (0, 1, 99), (0, 2, c.Sq - 1)], np.int64)
    assert bench.rows_flops(c, rows) == 4 * 128 * (1 + 100 + c.Sq)
    assert bench.rows_flops(w, rows) == 4 * 128 * 3 * w.Sk
    assert bench.whole_job_tflops(2e12, 1.0, 4) == 8000.0
    r = bench.oracle_sample_rows(c, 16, 3)
    assert r.shape == (16, 3) and r[:, 1].max() < c.Hq and r[:, 2].max() < c.Sq
    assert np.array_equal(r, bench.oracle_sample_rows(c, 16, 3))


_WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["EFQ_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
r = dist.get_rank()
out = bench.max_over_ranks([1.0 + r, 10.0 - r, 5.0])
assert out == [2.0, 10.0, 5.0], out
dist.barrier()
dist.destroy_process_group()
print("rank", r, "ok")
"""


def test_max_over_ranks_gloo_world_size_2(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29571",
                   EFQ_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                          "single_head_1024", "--steps", "2", "--warmup", "1", "--oracle-rows", "64"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "TFLOP/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["config"]["workload"] == "single_head"


def test_clock_summary_keeps_only_samples_inside_the_timed_region():
    import bench
    samples = [(9.0, 500.0, 1965.0, 100.0, {"hw_slowdown"}),        # before the region: ignored
               (10.1, 1965.0, 1965.0, 700.0, set()),
               (10.2, 1950.0, 1965.0, 900.0, {"sw_power_cap"}),
               (10.3, 1965.0, 1965.0, float("nan"), set()),
               (11.5, 300.0, 1965.0, 90.0, {"sw_thermal_slowdown"})]  # after the region: ignored
    out = bench.summarize_clock_samples(samples, 10.0, 11.0, "nvml")
    assert out["sm_mhz"] == 1965.0 and out["sm_max_mhz"] == 1965.0
    assert out["reasons"] == ["sw_power_cap"]
    assert out["samples"] == 3 and out["power_w_max"] == 900.0
    empty = bench.summarize_clock_samples(samples, 20.0, 21.0, "nvml")
    assert empty["sm_mhz"] is None and "no samples" in empty["reasons"][0]


def test_calibration_cli_grid_parsing():
    from paper_2609_09721_b200 import calibrate
    assert calibrate._grid("-3.6:-1.8:0.3") == [-3.6, -3.3, -3.0, -2.7, -2.4, -2.1, -1.8]
    assert calibrate._grid("2:2:1") == [2.0]
    assert set(calibrate.WORKLOADS) >= {"single_head_1024", "qwen3_8b_2k", "wan22_4096"}
