"""Writes tests/golden/blueprint_regression.txt from the oracle alone (no CUDA path).

Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import twist_oracle as o  # noqa: E402

CASES = [  # n_full S n_sub seed rnd layer kind mode
    (12, 4, 6, 7, 0, 0, 0, 0),
    (12, 4, 4, 3002, 3, 11, 1, 0),
    (32, 8, 8, 3004, 1, 31, 1, 0),
    (40, 3, 17, 5, 2, 1, 0, 0),
    (40, 2, 10, 5, 2, 1, 0, 1),
]


def main():
    with open(os.path.join(HERE, "blueprint_regression.txt"), "w") as f:
        f.write("# n_full S n_sub seed rnd layer kind mode : A row-major (written by make_golden.py from oracle/)\n")
        for c in CASES:
            A = o.sample_blueprint(c[0], c[1], c[2], [], c[3], c[4], c[5], c[6], c[7])
            f.write(" ".join(str(v) for v in c) + " : " + " ".join(str(int(v)) for v in A.reshape(-1)) + "\n")


if __name__ == "__main__":
    main()
