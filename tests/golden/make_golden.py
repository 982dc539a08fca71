"""Writes the expected-value fixtures of this folder. Calls only the CPU oracle (never the CUDA path).

    python tests/golden/make_golden.py

Each fixture instantiates a definition of the paper on a tiny seeded input:
  fd_small.json     Frequent-Directions sketch of a 40 x 12 stream with ell = 4 (Method, first paragraph;
                    Algorithm 1, Phase I): sigma' of the frozen sketch, sum of delta, number of shrinks.
  scores_small.json agreement scores of 9 rows against a fixed 3 x 5 sketch (Method, paragraph on two-pass scoring;
                    Algorithm 1, Phase II) and the top-4 selection (Algorithm 1, last branch).
"""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402


def main() -> None:
    r = np.random.default_rng(20251002)
    A = (r.standard_normal((40, 3)) @ r.standard_normal((3, 12)) + 0.3 * r.standard_normal((40, 12))).round(3)
    fd = oracle.OracleFD(12, 4)
    fd.update(A)
    S, sigma = fd.finalize()
    st = fd.stats()
    with open(os.path.join(HERE, "fd_small.json"), "w") as f:
        json.dump({"cites": "Method, first paragraph; Algorithm 1, Phase I", "rows": A.tolist(), "ell": 4,
                   "sigma": sigma.tolist(), "sum_delta": st["sum_delta"], "shrinks": st["shrinks"],
                   "gram": (S.T @ S).tolist()}, f)
    S2 = np.array([[2.0, 0.0, 1.0, 0.0, 0.0], [0.0, 1.0, 0.0, -1.0, 0.0], [0.5, 0.5, 0.0, 0.0, 0.25]])
    G = r.integers(-3, 4, size=(9, 5)).astype(np.float64)
    G[4] = 0.0
    out = oracle.score(S2, G)
    with open(os.path.join(HERE, "scores_small.json"), "w") as f:
        json.dump({"cites": "Method, 'Two-pass scoring'; Algorithm 1, Phase II and selection", "S": S2.tolist(),
                   "rows": G.tolist(), "alpha": out["alpha"].tolist(), "u": out["u"].tolist(),
                   "top4": oracle.select(out["alpha"], 4 / 9).tolist()}, f)


if __name__ == "__main__":
    main()
