"""Writes tests/golden/peer_tables.json from the CPU oracle alone.

The paper names no random generator, so these tables pin nothing in the
paper; they freeze the oracle's own sampler so that an accidental change of
its constants or draw order is noticed.  Run: python tests/golden/make_peer_tables.py
"""
import json
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402

CASES = [  # (seed, round, N, S, R)
    (1, 0, 8, 4, 2),     # S*R > N-1: one refill
    (1, 3, 6, 3, 1),     # S*R <= N-1: all distinct
    (7, 2, 4, 5, 3),     # several epochs, repairs after refills
]

if __name__ == "__main__":
    out = []
    for seed, rnd, N, S, R in CASES:
        out.append({"seed": seed, "round": rnd, "N": N, "S": S, "R": R,
                    "idx": oracle.select_peers(seed, rnd, N, S, R).tolist()})
    with open(os.path.join(HERE, "peer_tables.json"), "w") as f:
        json.dump({"_note": "written by make_peer_tables.py from oracle/ only", "cases": out}, f)
