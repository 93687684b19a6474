"""Writes tests/golden/oracle_small_cases.json from the CPU oracle alone.

The paper prints no worked numeric example, so these are not paper values: they
freeze the oracle's outputs on a few tiny seeded cases so that an unintended
change of its arithmetic shows up as a diff.  Run from the repository root:
    python tests/golden/make_golden.py
Calls nothing but ``oracle`` and the seeded input generators.
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2401_06706_b200 import synth  # noqa: E402

CASES = [
    synth.Workload("g_with", 4, 96, "3x2x1", "fp32", "normal", 2.0, 1.0, 1.0, 1.0, 0, 11),
    synth.Workload("g_without", 4, 96, "3x2x1", "bf16", "normal", 2.5, 0.8, 1.5, 1.0, 1, 12),
    synth.Workload("g_greedy", 4, 96, "4x2", "fp16", "normal", 3.0, 1.0, 2.0, 0.0, 0, 13),
    synth.Workload("g_temp", 4, 64, "2x2x2", "fp16", "gumbel", 2.0, 1.0, 1.2, 0.7, 1, 14),
]


def run_case(w):
    inp = synth.make_inputs(w, "cpu")
    t, d, c, u = inp.host_f32()
    r = oracle.verify(t, d if w.temperature > 0 else None, inp.parent, c, u, w.temperature, w.mode)
    return {"accept_len": r.accept_len.tolist(), "tokens": r.tokens.tolist(),
            "node_accept": r.node_accept.tolist(), "node_bonus": r.node_bonus.tolist(),
            "residual_max": [float(x) for x in r.residual.max(axis=1)],
            "residual_argmax": r.residual.argmax(axis=1).tolist(),
            "ratio_sum": float(np.nansum(np.where(r.node_ratio > 0, r.node_ratio, 0.0)))}


if __name__ == "__main__":
    out = {w.name: run_case(w) for w in CASES}
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_small_cases.json")
    with open(path, "w") as f:
        json.dump(out, f, indent=1, sort_keys=True)
    print("wrote", path)
