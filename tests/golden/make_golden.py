"""Writes the stored expected values under tests/golden/.  Calls only the CPU oracle and the
seeded input generator -- never the CUDA library.  Run from the repository root:

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import blas_oracle as orc  # noqa: E402
from paper_2411_07211_b200 import synth  # noqa: E402


def main():
    n = 1 << 20
    x = synth.vector_np(0, 0, n, np.float32)
    y = synth.vector_np(0, 1, n, np.float32)
    res, absterms = orc.dot(n, x, 1, y, 1)
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "sdot_n1048576_seed0.txt")
    with open(out, "w") as f:
        f.write("# sdot, n=1,048,576 f32, x = stream (seed 0, 0), y = stream (seed 0, 1), inc 1.\n")
        f.write("# Result of the f64-accumulated CPU oracle, rounded once to f32.  The paper prints\n")
        f.write("# no numeric example (Section 6.2.1 only names the routine); this value is the\n")
        f.write("# oracle's own, pinned independently in tests/test_oracle_pins.py.\n")
        f.write(f"n={n}\nresult_hex={float(res).hex()}\nresult={float(res)!r}\nabsterms={absterms!r}\n")
    print(open(out).read())


if __name__ == "__main__":
    main()
