"""Writes tests/golden/tiny_oracle_sha256.txt.  Calls only the CPU oracle (and the integer-hash input
generator); run from the repository root:  python tests/golden/make_golden.py"""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from test_oracle_layout import golden_digest  # noqa: E402

if __name__ == "__main__":
    digest, sinks = golden_digest()
    path = os.path.join(ROOT, "tests", "golden", "tiny_oracle_sha256.txt")
    with open(path, "w") as f:
        f.write("# sha256 over the oracle's outputs (mask, positions, counts, packed codes, parameters, side buffer,\n"
                "# tail, attention rounded to 1e-9) for the tiny workload on integer-hash inputs.  Not a value from the\n"
                "# paper: a regression lock written by tests/golden/make_golden.py, which calls only the CPU oracle.\n")
        f.write(digest + "\n")
    print(digest, sinks)
