"""Writes the stored expected values under tests/golden/ by calling ONLY the CPU
oracle (oracle/) on seeded inputs. The paper prints no worked numeric example
for the compression event (Section 4.1 gives the rule, not values), so these
files are regression anchors for the oracle itself, not paper values.

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import alpha_oracle as O  # noqa: E402
from paper_2605_14292_b200 import synth  # noqa: E402


def main():
    ev = synth.make_c1(seed=0)
    K, V, pos, q = ev.K[0, 0, 0], ev.V[0, 0, 0], ev.pos[0, 0, 0], ev.qstat[0, 0]
    out = {"source": "oracle/alpha_oracle.py compress_event on synth.make_c1(seed=0); Section 4.1, Algorithm 1",
           "config": "N=192, d=128, fp32, positions 0..191, p_ref=192, base 10000, W=1, b=64"}
    for lam in (0.0, 0.5, 1.0):
        r = O.compress_event(K, V, pos, q, int(ev.p_ref[0]), ev.budget, lam)
        out[f"lambda_{lam}"] = {
            "idx_sorted": r.sel.idx_sorted.tolist(),
            "pick_order": r.sel.order.tolist(),
            "min_margin": float(np.min(r.sel.margins)),
            "scores_first8": [float(x) for x in r.scores[:8]],
            "score_sum": float(r.scores.sum()),
        }
    with open(os.path.join(HERE, "c1_event.json"), "w") as f:
        json.dump(out, f, indent=1)
    print("wrote c1_event.json")


if __name__ == "__main__":
    main()
