"""Writes tests/golden/tiny_oracle.txt: a few oracle outputs for the BASELINE `tiny` workload
(seed 0, CPU generator).  Calls only `oracle/` and the input generator; never the CUDA path.

    python tests/golden/make_golden.py

The paper prints no numeric attention example, so these values pin the oracle against its own
committed state (any later change to its arithmetic must be deliberate); what pins it against the
paper and the mathematics is tests/test_oracle_pins.py."""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import bdlm_oracle as orc  # noqa: E402
from paper_2609_19242_b200 import synth  # noqa: E402

NAMES6 = ["q_clean", "k_clean", "v_clean", "q_noisy", "k_noisy", "v_noisy"]
PROBES = [(0, 0, 0, 0), (0, 1, 1, 3), (0, 15, 0, 7), (0, 16, 1, 63), (0, 127, 0, 31), (0, 255, 1, 0)]


def compute():
    w = synth.WORKLOADS["tiny"]
    x = {k: synth.to_f64(v) for k, v in synth.make_inputs(w, "cpu").items()}
    fwd = orc.attn_forward(*[x[n] for n in NAMES6], w.block_size)
    bwd = orc.attn_backward(*[x[n] for n in NAMES6], x["do_clean"], x["do_noisy"], w.block_size)
    lines = []
    for name, arr in zip(["o_clean", "o_noisy"], (fwd[0], fwd[2])):
        for p in PROBES:
            lines.append(f"{name} {p[0]} {p[1]} {p[2]} {p[3]} {arr[p]:.17e}")
    for name, arr in zip(["lse_clean", "lse_noisy"], (fwd[1], fwd[3])):
        for p in PROBES:
            lines.append(f"{name} {p[0]} {p[2]} {p[1]} 0 {arr[p[0], p[2], p[1]]:.17e}")
    for name, arr in zip(["dq_clean", "dk_clean", "dv_clean", "dq_noisy", "dk_noisy", "dv_noisy"], bwd):
        for p in PROBES:
            lines.append(f"{name} {p[0]} {p[1]} {p[2]} {p[3]} {arr[p]:.17e}")
        lines.append(f"{name} sum 0 0 0 {arr.sum():.17e}")
    return lines


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_oracle.txt")
    with open(out, "w") as f:
        f.write("# oracle outputs for the `tiny` workload (batch 1, H 2/2, d 64, L 256, block 16, seed 0);\n")
        f.write("# name batch row head dim value   (lse rows: name batch head row 0 value)\n")
        f.write("\n".join(compute()) + "\n")
    print(out)
