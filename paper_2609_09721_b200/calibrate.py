"""Offline selection of the affine rule's (tau, h) on a synthetic workload (Algorithm 3).

    python -m paper_2609_09721_b200.calibrate --workload qwen3_8b_2k --tau -3.6:-1.8:0.3 --h 1.6:3.0:0.2

Runs the fused EFQ forward for every candidate pair on the seeded inputs of the workload, measures
rho = ||O~ - O_ref||_F / ||O_ref||_F against FP32 attention on the unquantised inputs, prints the surface and
the pair with the smallest rho.  Real calibration activations are the caller's business: this tool takes the
shapes and value distributions of the synthetic workloads, nothing else.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import binding, inputs

WORKLOADS = {
    "single_head_1024": lambda: inputs.case_single_head(1024, seed=1),
    "qwen3_8b_2k": lambda: inputs.case_qwen3_8b(2048, seed=3),
    "qwen3_8b_16k": lambda: inputs.case_qwen3_8b(16384, seed=3),
    "wan22_4096": lambda: inputs.case_wan22(4096, seed=5),
}


def _grid(spec: str):
    lo, hi, step = (float(x) for x in spec.split(":"))
    n = int(round((hi - lo) / step)) + 1
    return [round(lo + i * step, 6) for i in range(n)]


def surface(case, taus, hs):
    qb, kb, vb = inputs.make_qkv(case)
    dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    q, k, v = dev(qb), dev(kb), dev(vb)
    o_ref = binding.efq_exact_attention_fwd(q, k, v, case.causal)
    table, best = binding.efq_calibrate(q, k, v, o_ref, taus, hs, case.causal)
    return np.array(table), best


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--workload", default="qwen3_8b_2k", choices=sorted(WORKLOADS))
    ap.add_argument("--tau", default="-3.6:-1.8:0.3", help="lo:hi:step")
    ap.add_argument("--h", default="1.6:3.0:0.2", help="lo:hi:step")
    args = ap.parse_args(argv)
    taus, hs = _grid(args.tau), _grid(args.h)
    case = WORKLOADS[args.workload]()
    rho, best = surface(case, taus, hs)
    print(f"workload {case.name}: rho(tau, h) = ||O~ - O_ref||_F / ||O_ref||_F, rows tau, columns h")
    print("tau\\h   " + " ".join(f"{h:7.2f}" for h in hs))
    for t, row in zip(taus, rho):
        print(f"{t:6.2f}  " + " ".join(f"{x:7.4f}" for x in row))
    print(f"selected (tau, h) = ({best[0]:.2f}, {best[1]:.2f}), rho = {rho.min():.4f}")
    for name, (t, h) in (("EFQ-Mean", (-3.06, 2.30)), ("EFQ-MMLU", (-2.90, 2.00)), ("EFQ-Balance", (-2.10, 2.70))):
        r, _ = surface(case, [t], [h])
        print(f"{name:12s} ({t:.2f}, {h:.2f}): rho = {r[0, 0]:.4f}")
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
