"""Writes tests/golden/oracle_small_cases.json: the oracle's results on small fixed inputs.

The paper prints no worked numeric example of any step, so nothing here is the paper's; the stored values come from
oracle/ alone (this script imports nothing else of the repository) and pin the oracle against silent change: a commit
that alters them has to say which passage of the paper, or which reading of it, justifies the new values. The
independent checks of the oracle (closed forms, brute force, library routines) are in tests/test_oracle_*.py.

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), "..", ".."))
import oracle  # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_small_cases.json")


def cases():
    out = {}
    # Section 3.3, smoothing equations: a 12-point and a 9-point sequence (even and odd length), rho 0.9, alpha 0.5, T 2
    x12 = np.array([0.9, 0.1, 0.4, 0.8, 0.2, 0.7, 0.3, 0.6, 0.5, 0.05, 0.95, 0.15])
    x9 = np.array([0.2, 0.9, 0.1, 0.6, 0.4, 0.8, 0.3, 0.7, 0.5])
    for name, x in (("sss_n12", x12), ("sss_n9", x9)):
        y, kstar, _ = oracle.sss(x, 0.9, 0.5, 2)
        out[name] = {"x": x.tolist(), "rho": 0.9, "alpha": 0.5, "T": 2, "kstar": int(kstar), "y": np.asarray(y).tolist()}
    # Section 3.1 allocation: 6 heads, B = 100, window 4, base 2, L = 40 (one head hits its cap)
    S = np.array([0.05, 0.9, 0.3, 0.0, 0.6, 0.15], dtype=np.float32)
    out["allocate"] = {"S": S.tolist(), "B": 100, "w": 4, "r": 2, "L": 40,
                       "b": oracle.allocate(S, 100, 4, 2, 40).tolist()}
    # Top-K with ties (lower index first)
    s = np.array([0.5, 0.7, 0.5, 0.1, 0.7, 0.5, 0.2])
    out["select"] = {"s": s.tolist(), "k": 4, "idx": oracle.select(s, 4).tolist()}
    # Section 3.2 head score: 2 steps, 2 heads, rows of 6 tokens, K = 2
    attn = np.array([[[0.1, 0.4, 0.2, 0.1, 0.1, 0.1], [0.3, 0.1, 0.1, 0.3, 0.1, 0.1]],
                     [[0.05, 0.05, 0.5, 0.3, 0.05, 0.05], [0.2, 0.2, 0.2, 0.2, 0.1, 0.1]]])
    row_len = np.array([6, 5], dtype=np.int32)
    span = np.array([[1, 2], [1, 2]], dtype=np.int32)
    s_hit, counts = oracle.hit_score(attn, row_len, span, K=2)
    out["hit_score"] = {"attn": attn.tolist(), "row_len": row_len.tolist(), "span": span.tolist(), "K": 2,
                        "counts": counts.tolist(), "s_hit": s_hit.tolist()}
    # Selection spread: 2 heads, P = 10, 4 stretches
    kept = np.array([0, 1, 5, 10, 11, 2, 3, 9, 10, 11], dtype=np.int32)
    cu = np.array([0, 5, 10], dtype=np.int32)
    hist, bal, peak = oracle.selection_spread(kept, cu, 10, 4)
    out["selection_spread"] = {"kept": kept.tolist(), "cu": cu.tolist(), "P": 10, "n_bins": 4, "hist": hist.tolist(),
                               "balance": bal, "peak": peak}
    return out


if __name__ == "__main__":
    with open(OUT, "w") as f:
        json.dump(cases(), f, indent=1)
    print("wrote", OUT)
