"""Writes tests/golden/live_counts.txt from the CPU oracle alone.

Run from the repository root:  python tests/golden/make_golden.py
Columns: schedule, rho numerator, rho denominator, step k, dense entries n_k*L_k, live entries.
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import litevar_oracle as orc  # noqa: E402

S256 = (1, 2, 3, 4, 5, 6, 8, 10, 13, 16)
S512 = (1, 2, 3, 4, 6, 9, 13, 18, 24, 32)


def main():
    lines = ["# schedule rho_num rho_den step dense live   (default window rule, 3 global scales)"]
    for name, scales in (("256", S256), ("512", S512)):
        for rho in ((1, 8), (1, 4), (1, 2)):
            w = orc.window_table(scales, rho=rho)
            for k in range(1, len(scales) + 1):
                n_k, L_k = orc.map_shape(scales, k)
                lines.append(f"{name} {rho[0]} {rho[1]} {k} {n_k * L_k} {orc.live_count(scales, k, w[k - 1])}")
    with open(os.path.join(HERE, "live_counts.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
