"""Writes lsh_hyperplane_d8.json: hyperplane hash keys of a few small integer points, computed with Python integers only.

The hyperplane of repetition l, bit b is a vector of random signs; coordinate c is +1 when bit 0 of
splitmix64(seed, 2^60 + (64 l + b) 2^20 + c) is set and -1 otherwise; the key bit is [<a, x> > 0] (a projection of
zero gives 0).  This script imports neither the oracle nor the CUDA package: the fixture it writes pins both.

    python tests/golden/make_lsh_hyperplane_golden.py
"""
import json
import os

M = (1 << 64) - 1


def splitmix64(seed, idx):
    z = (seed + (idx + 1) * 0x9E3779B97F4A7C15) & M
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M
    return z ^ (z >> 31)


def sign(seed, rep, bit, c):
    return 1 if splitmix64(seed, (1 << 60) + ((rep * 64 + bit) << 20) + c) & 1 else -1


def main():
    seed, L, L_low, k, d = 2006, 2, 1, 3, 8
    points = [[1, 2, 3, 4, 5, 6, 7, 8], [-1, -2, -3, -4, -5, -6, -7, -8], [0, 0, 0, 0, 0, 0, 0, 0], [5, -5, 5, -5, 5, -5, 5, -5],
              [1, 0, 0, 0, 0, 0, 0, 0], [0, 0, 0, 0, 0, 0, 0, -1], [127, 127, 127, 127, -128, -128, -128, -128], [3, 1, -4, 1, -5, 9, -2, 6]]
    planes = [[[sign(seed, l, b, c) for c in range(d)] for b in range(k)] for l in range(L + L_low)]
    keys, projections = [], []
    for l in range(L + L_low):
        bits = k if l < L else k - 1
        row, prow = [], []
        for x in points:
            proj = [sum(a * v for a, v in zip(planes[l][b], x)) for b in range(bits)]
            prow.append(proj)
            row.append(sum((1 << b) for b in range(bits) if proj[b] > 0))
        keys.append(row)
        projections.append(prow)
    out = {"comment": "hyperplane LSH keys (sign random projections) of int8 points, Python integers only; see make_lsh_hyperplane_golden.py",
           "seed": seed, "L": L, "L_low": L_low, "k": k, "d": d, "points": points, "hyperplanes": planes,
           "projections": projections, "keys": keys}
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "lsh_hyperplane_d8.json"), "w") as f:
        json.dump(out, f, indent=1)


if __name__ == "__main__":
    main()
