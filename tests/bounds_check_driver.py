"""Runs a list of small layers through the bounds-check build of the library (DAD_LIB=libdad_check.so, set by the
test that starts this script) and prints one JSON line: the checker's record and the parity of every case.  Shapes
are chosen to reach every kernel family that computes its own indices: the general products, both one-launch
forms, the fp32 dense product and the copies."""
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import dad_oracle                                   # noqa: E402
from paper_2102_09631_b200 import binding as B, workloads as wl   # noqa: E402

CASES = [  # S, N, h_in, h_out, r, iters, dtype
    (2, 16, 64, 32, 4, 2, torch.float32),        # one-launch, on chip
    (3, 70, 264, 520, 40, 2, torch.float32),     # one-launch, through L2
    (3, 2000, 96, 40, 5, 1, torch.float32),      # general pipeline, fp64 accumulation, split rows
    (2, 100, 70, 50, 7, 2, torch.bfloat16),      # bf16 in a layout the tensor-core kernels do not take
    (5, 37, 50, 70, 7, 3, torch.float32),        # odd everything
    (1, 1, 8, 8, 1, 2, torch.float32),
]


def main():
    assert B.dad_bounds_check_build(), "this driver wants the bounds-check build"
    dad_oracle.build()
    dev = torch.device("cuda:0")
    B.dad_bounds_report(reset=True)
    worst = 0.0
    for S, N, h_in, h_out, r, iters, dt in CASES:
        A, D = wl.decaying_layer(S, N, h_in, h_out, 300 + N, dt)
        Q0 = wl.start_block(S, r, h_out, 300 + N)
        Ad, Dd = A.to(dev), D.to(dev)
        plan = B.LayerPlan(Ad, Dd, r, iters)
        grad = plan.step(Ad, Dd, Q0.to(dev))
        full = torch.empty_like(grad)
        B.dad_full_grad(plan.layer, Ad, Dd, full, None, plan.ws)
        try:
            B.dad_check(plan.ws)
        except B.DadError:
            if not os.environ.get("DAD_BOUNDS_SHRINK"):   # with shortened ranges dropped accesses may leave non-finite values
                raise
        ref = dad_oracle.rank_dad_layer(A, D, Q0, iters)
        tol = 1e-5 if dt == torch.float32 else 2e-2
        e1 = np.linalg.norm(grad.double().cpu().numpy() - ref["grad"]) / max(np.linalg.norm(ref["grad"]), 1e-300)
        rf = dad_oracle.full_grad(A, D)
        e2 = np.linalg.norm(full.double().cpu().numpy() - rf) / max(np.linalg.norm(rf), 1e-300)
        worst = max(worst, e1 / tol, e2 / tol)
    count, addr, nbytes, line = B.dad_bounds_report()
    print(json.dumps({"violations": count, "first_address": addr, "first_bytes": nbytes, "first_line": line,
                      "worst_error_over_bar": worst}))


if __name__ == "__main__":
    main()
