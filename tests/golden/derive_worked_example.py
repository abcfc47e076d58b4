"""Derives the hand-worked fixtures of this folder in exact rational arithmetic.

Independent of both the CPU oracle and the CUDA library (imports neither): it
evaluates the paper's per-pixel definition y_i = (Phi_i D) B_i^T (Eq. 2) on a
2x2 LR image with python `fractions`, so the stored values carry no rounding.
Run `python tests/golden/derive_worked_example.py` to rewrite the two .txt files.

Setting: C = 1, LR x = [[0, 1/4], [1/2, 1]], scale r = 2, k = 3, two atoms:
dict[0] = delta at the centre tap, dict[1] = 1/9 on every tap; coefficients
Phi_0 = 1/2 everywhere, Phi_1[Y][X] = (4Y + X)/16.  Up-sampling: Keys cubic
convolution with a = -3/4, half-pixel centres, indices clamped to the image;
patch positions clamped in HR coordinates.
"""
import math
import os
from fractions import Fraction as Fr

A = Fr(-3, 4)


def inner(z):
    return ((A + 2) * z - (A + 3)) * z * z + 1


def outer(z):
    return ((A * z - 5 * A) * z + 8 * A) * z - 4 * A


def taps(r, X):
    src = Fr(2 * X + 1, 2 * r) - Fr(1, 2)
    ix = math.floor(src)
    t = src - ix
    return ix, [outer(t + 1), inner(t), inner(1 - t), outer(2 - t)]


def clamp(v, lo, hi):
    return max(lo, min(hi, v))


def main():
    here = os.path.dirname(os.path.abspath(__file__))
    with open(os.path.join(here, "bicubic_weights.txt"), "w") as f:
        f.write("# Keys cubic-convolution weights, a = -3/4, half-pixel centres: closed forms per phase.\n")
        f.write("# Stage 1 up-sampling of the paper (Section II-A) with the kernel fixed by the benchmark configs.\n")
        f.write("# columns: scale phase base_offset(first tap = floor(X/scale) + base_offset) w0 w1 w2 w3\n")
        for r in (2, 3, 4):
            for ph in range(r):
                X = ph + 4 * r
                ix, w = taps(r, X)
                f.write(f"{r} {ph} {ix - 1 - X // r} " + " ".join(str(v) for v in w) + "\n")
    x = [[Fr(0), Fr(1, 4)], [Fr(1, 2), Fr(1)]]
    h = w = 2
    r = 2
    H = W = 4
    U = [[None] * W for _ in range(H)]
    for Y in range(H):
        iy, wy = taps(r, Y)
        for X in range(W):
            ix, wx = taps(r, X)
            U[Y][X] = sum(wy[a] * wx[b] * x[clamp(iy - 1 + a, 0, h - 1)][clamp(ix - 1 + b, 0, w - 1)]
                          for a in range(4) for b in range(4))
    y = [[None] * W for _ in range(H)]
    for Y in range(H):
        for X in range(W):
            box = sum(U[clamp(Y + a - 1, 0, H - 1)][clamp(X + b - 1, 0, W - 1)] for a in range(3) for b in range(3)) / 9
            y[Y][X] = Fr(1, 2) * U[Y][X] + Fr(4 * Y + X, 16) * box
    with open(os.path.join(here, "worked_example_4x4.txt"), "w") as f:
        f.write("# Hand-worked case of Eq. 2 (y_i = (Phi_i D) B_i^T) in exact rationals; setting in derive_worked_example.py.\n")
        f.write("# rows U0..U3: the up-sampled image (= output for Phi_0 = 1, Phi_1 = 0); rows y0..y3: the regression output.\n")
        for Y in range(H):
            f.write(f"U{Y} " + " ".join(str(v) for v in U[Y]) + "\n")
        for Y in range(H):
            f.write(f"y{Y} " + " ".join(str(v) for v in y[Y]) + "\n")


if __name__ == "__main__":
    main()
