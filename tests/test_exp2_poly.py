"""The cubic exp2 of the score kernel (host-side model): the constants in the CUDA source are the Remez solution,
the model's relative error stays below 1e-4 over the whole clamped range, and the clamps behave as documented."""
import os
import re

import numpy as np

from paper_2604_11288_b200 import exp2_poly as ep

SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2604_11288_b200", "csrc",
                   "ta_score.cu")


def _source_coefficients():
    text = open(SRC).read()
    m = re.search(r"kC0 = ([0-9.eE+-]+)f, kC1 = ([0-9.eE+-]+)f, kC2 = ([0-9.eE+-]+)f,\s*kC3 = ([0-9.eE+-]+)f", text)
    assert m, "coefficients not found in ta_score.cu"
    return np.array([float(g) for g in m.groups()], np.float32)


def test_source_constants_are_the_remez_solution():
    coef, err = ep.remez_exp2()
    assert err < 7.6e-5
    np.testing.assert_allclose(_source_coefficients(), coef, rtol=0, atol=2e-7)
    text = open(SRC).read()
    assert "kPolyRange = 252.0f" in text and "12582912.0f - 126.0f" in text


def test_model_error_and_clamps():
    coef = _source_coefficients()
    rng = np.random.default_rng(0)
    c = np.float32(0.1275)
    for beta in (0.0, -3.7, 11.25):
        x = rng.uniform(-120.0, 60.0, size=200000)
        s = ((x + beta) / c).astype(np.float32)
        got = ep.exp2_poly_model(s, c, beta, coef).astype(np.float64)
        want = np.exp2(s.astype(np.float64) * np.float64(c) - beta)
        assert np.max(np.abs(got / want - 1.0)) < 1.0e-4
    # far below the range: a tiny positive number (never negative, never NaN); far above: 2^126, which the first pass's
    # overflow check catches
    lo = ep.exp2_poly_model(np.array([-1e6, -5000.0], np.float32), c, 0.0, coef)
    assert (lo >= 0).all() and (lo < 2e-38).all()
    hi = ep.exp2_poly_model(np.array([5000.0, 1e6], np.float32), c, 0.0, coef)
    assert np.isfinite(hi).all() and (hi > 8e37).all()
    # exact powers of two come out within the polynomial's error at f = 0
    p2 = ep.exp2_poly_model((np.arange(-100, 100) / c).astype(np.float32), c, 0.0, coef).astype(np.float64)
    assert np.max(np.abs(p2 / np.exp2((np.arange(-100, 100) / c).astype(np.float32).astype(np.float64) * c) - 1)) < 1e-4
