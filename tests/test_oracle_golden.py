"""The oracle against its stored small cases (tests/golden/oracle_small_cases.json, written by
tests/golden/make_golden.py from oracle/ alone): integers exactly, floats to 1e-12. These guard the oracle against
silent change; what pins it to the paper and the mathematics is in the other test_oracle_*.py files."""
import json
import os

import numpy as np
import pytest

import oracle

with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "oracle_small_cases.json")) as f:
    G = json.load(f)


@pytest.mark.parametrize("name", ["sss_n12", "sss_n9"])
def test_sss_small_case(name):
    c = G[name]
    y, kstar, _ = oracle.sss(np.array(c["x"]), c["rho"], c["alpha"], c["T"])
    assert int(kstar) == c["kstar"]
    assert np.allclose(y, c["y"], rtol=0, atol=1e-12)
    # and the direct O(n^2) transform gives the same numbers as the fast one
    y2, k2, _ = oracle.sss(np.array(c["x"]), c["rho"], c["alpha"], c["T"], direct=True)
    assert int(k2) == c["kstar"] and np.allclose(y2, c["y"], rtol=0, atol=1e-12)


def test_allocate_small_case():
    c = G["allocate"]
    b = oracle.allocate(np.array(c["S"], dtype=np.float32), c["B"], c["w"], c["r"], c["L"])
    assert b.tolist() == c["b"] and sum(c["b"]) == c["B"] and max(c["b"]) <= c["L"] and min(c["b"]) >= c["w"] + c["r"]


def test_select_small_case():
    c = G["select"]
    assert oracle.select(np.array(c["s"]), c["k"]).tolist() == c["idx"] == [0, 1, 2, 4]


def test_hit_score_small_case():
    c = G["hit_score"]
    s_hit, counts = oracle.hit_score(np.array(c["attn"]), np.array(c["row_len"], dtype=np.int32),
                                     np.array(c["span"], dtype=np.int32), K=c["K"])
    assert counts.tolist() == c["counts"] and np.allclose(s_hit, c["s_hit"], rtol=0, atol=1e-15)
    # by hand, spans 1..2 at both steps: head 0 takes tokens {1, 2} (two hits) then {2, 3} (one hit);
    # head 1 takes {0, 3} (the tie at 0.3 goes to the lower indices; no hit) then {0, 1} of its five tokens (one hit)
    assert c["counts"] == [3, 1] and c["s_hit"] == [0.75, 0.25]


def test_selection_spread_small_case():
    c = G["selection_spread"]
    hist, bal, peak = oracle.selection_spread(np.array(c["kept"], dtype=np.int32), np.array(c["cu"], dtype=np.int32),
                                              c["P"], c["n_bins"])
    assert hist.tolist() == c["hist"] == [3, 1, 1, 1]
    assert bal == pytest.approx(c["balance"], abs=1e-15) and peak == pytest.approx(c["peak"], abs=1e-15)
