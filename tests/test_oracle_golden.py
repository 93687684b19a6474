"""Drift check: the oracle still reproduces the values its own committed script froze."""
import importlib.util
import json
import os

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))


def test_oracle_reproduces_frozen_small_cases():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mg = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mg)
    frozen = json.load(open(os.path.join(HERE, "golden", "oracle_small_cases.json")))
    for w in mg.CASES:
        got, want = mg.run_case(w), frozen[w.name]
        for key in ("accept_len", "tokens", "node_accept", "node_bonus", "residual_argmax"):
            assert got[key] == want[key], (w.name, key)
        assert got["residual_max"] == pytest.approx(want["residual_max"], rel=1e-12)
        assert got["ratio_sum"] == pytest.approx(want["ratio_sum"], rel=1e-12)
