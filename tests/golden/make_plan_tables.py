"""Writes tests/golden/plan_tables_small.json from the integer-plan oracle (oracle/plan_ref.py only):
the block plan of two small batches, kept as stored expected values so that a change of the oracle's
reading of the plan (chunk bounds, ring steps, slots, row order) shows up as a diff.

    python tests/golden/make_plan_tables.py
"""
import json
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import plan_ref as P  # noqa: E402

CASES = [dict(lens=[5, 2, 1], degs=[3, 2, 4]), dict(lens=[64, 599, 609], degs=[1, 3, 2])]


def tables(lens, degs):
    ref = P.plan_blocks(lens, degs)
    return dict(lens=lens, degs=degs, chunk_bounds=[int(x) for x in ref["chunk_bounds"]],
                chunk_offset=[int(x) for x in ref["chunk_offset"]], pairs=[[int(v) for v in p] for p in ref["pairs"]],
                items=[[int(v) for v in i] for i in ref["items"]],
                chunk_slots=[[int(n), [int(v) for v in r]] for n, r in ref["chunk_slots"]],
                n_partial_rows=int(ref["n_partial_rows"]))


if __name__ == "__main__":
    out = [tables(**c) for c in CASES]
    with open(os.path.join(HERE, "plan_tables_small.json"), "w") as f:
        json.dump(out, f, indent=0, separators=(",", ":"))
        f.write("\n")
    print("wrote", len(out), "cases")
