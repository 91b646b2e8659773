"""Writes tests/golden/schedule_tables.txt from the oracle's closed form.

Run from the repository root:  python tests/golden/make_schedule_golden.py
Calls only ``oracle/``.  The stored tables guard the oracle against silent
changes; they are not an independent pin (those are in test_oracle_schedule).
"""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))

from oracle import OP_AG_GEMM, OP_GEMM_RS          # noqa: E402
from oracle.schedule import schedule               # noqa: E402

CASES = [(OP_AG_GEMM, 2, 2, 512), (OP_AG_GEMM, 4, 2, 4096), (OP_GEMM_RS, 4, 2, 4096),
         (OP_GEMM_RS, 8, 2, 8192), (OP_AG_GEMM, 8, 1, 4096), (OP_GEMM_RS, 3, 1, 12)]


def main():
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "schedule_tables.txt")
    with open(out, "w") as f:
        f.write("# op P rings M, then one line per entry: rank step ring part chunk peer row_begin row_count\n")
        for op, P, rings, M in CASES:
            t = schedule(op, P, rings, M)
            f.write(f"case {op} {P} {rings} {M} {len(t)}\n")
            for row in t.tolist():
                f.write(" ".join(str(v) for v in row) + "\n")


if __name__ == "__main__":
    main()
