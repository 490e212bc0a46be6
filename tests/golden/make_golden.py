"""Writes tests/golden/route_counts.txt from the CPU oracle (and from nothing else).

Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import bf1_oracle as O  # noqa: E402

LENGTHS = [128, 257, 512, 1000, 2048, 3001, 4096, 8192, 12345, 16384, 32768]


def main():
    c = O.cfg()
    path = os.path.join(ROOT, "tests", "golden", "route_counts.txt")
    with open(path, "w") as f:
        f.write("# n_<length> = <blocks> <selected block pairs> <selected token pairs>\n")
        f.write("# written by tests/golden/make_golden.py from oracle/ (Eq. 1 route, Prop. 1 counting)\n")
        for n in LENGTHS:
            _, cnt, _, total = O.route(c, n)
            f.write("n_%d = %d %d %d  # oracle enumeration of Eq. 1, b = 64\n"
                    % (n, len(cnt), int(cnt.sum()), total))
    print("wrote", path)


if __name__ == "__main__":
    main()
