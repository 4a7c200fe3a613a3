"""Coefficients of the cubic that the score kernel uses for 2^f on [0, 1) (csrc/ta_score.cu, kC0..kC3), and a
bit-level model of the kernel's polynomial exp2 in numpy.

Run as a script to print the coefficients; tests/test_exp2_poly.py checks that the constants in the CUDA source are
the ones this derivation gives and that the model stays inside the stated error.
"""
from __future__ import annotations

import numpy as np
from numpy.polynomial import polynomial as P

POLY_RANGE = 252.0                 # width of the clamped argument range [-126, 126]
POLY_MAGIC = 12582912.0 - 126.0    # 1.5 * 2^23 - 126


def remez_exp2(deg: int = 3, iters: int = 40):
    """Minimax polynomial in relative error for 2^x on [0, 1] by the Remez exchange. Returns (coefficients, error)."""
    n = deg + 2
    k = np.arange(n)
    x = 0.5 + 0.5 * np.cos(np.pi * k / (n - 1))[::-1]
    xs = np.linspace(0.0, 1.0, 200001)
    c, err_max = None, None
    for _ in range(iters):
        A = np.zeros((n, n))
        for i in range(deg + 1):
            A[:, i] = x ** i / 2.0 ** x
        A[:, -1] = (-1.0) ** k
        c = np.linalg.solve(A, np.ones(n))[:-1]
        err = P.polyval(xs, c) / 2.0 ** xs - 1.0
        err_max = float(np.max(np.abs(err)))
        # new reference: the alternating extrema of the error
        idx = [0] + [i for i in range(1, len(xs) - 1)
                     if (err[i] - err[i - 1]) * (err[i + 1] - err[i]) <= 0 and abs(err[i]) > 1e-12] + [len(xs) - 1]
        pts = []
        for i in idx:
            if pts and np.sign(err[pts[-1]]) == np.sign(err[i]):
                if abs(err[i]) > abs(err[pts[-1]]):
                    pts[-1] = i
            else:
                pts.append(i)
        while len(pts) > n:
            pts.pop(0 if abs(err[pts[0]]) < abs(err[pts[-1]]) else -1)
        if len(pts) < n:
            break
        x = xs[pts]
    return c.astype(np.float32), err_max


def exp2_poly_model(s, c, beta, coef):
    """What exp2_poly(s, c/252, (126 - beta)/252) computes, step by step in fp32 (numpy): saturating multiply-add,
    round-down multiply-add onto the magic constant, exact difference, fraction, Horner cubic, exponent splice."""
    f32 = np.float32
    s = np.asarray(s, f32)
    c252 = f32(f32(c) * f32(1.0 / POLY_RANGE))
    bias = f32((f32(126.0) - f32(beta)) * f32(1.0 / POLY_RANGE))
    t = np.clip((s.astype(np.float64) * np.float64(c252) + np.float64(bias)).astype(f32), f32(0.0), f32(1.0))
    # fma.rm(t, 252, magic): exact in float64 (t has 24 bits, the sum stays below 2^53), then floor to the fp32 grid
    y = np.floor(t.astype(np.float64) * POLY_RANGE + POLY_MAGIC)          # an integer below 2^24: exact in fp32
    w = POLY_MAGIC - y                                                    # exact
    f = (t.astype(np.float64) * POLY_RANGE + w).astype(f32)               # one rounding, as fma does
    p = f32(coef[3])
    for ci in (coef[2], coef[1], coef[0]):
        p = (p.astype(np.float64) * f.astype(np.float64) + np.float64(ci)).astype(f32)
    j = (y - 12582912.0).astype(np.int64)                                 # floor(x), in [-126, 126]
    bits = p.view(np.int32).astype(np.int64) + (j << 23)
    return (bits & 0xFFFFFFFF).astype(np.uint32).view(f32)


if __name__ == "__main__":
    coef, err = remez_exp2()
    print("coefficients", [float(v) for v in coef], "max relative error", err)
