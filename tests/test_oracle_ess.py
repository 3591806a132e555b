"""Pins for the oracle's effective-sample-size floor (Section 3.3)."""
import numpy as np
import pytest

import oracle
from test_oracle_bookkeeping import _golden


def _kish(w):
    return w.sum() ** 2 / (w ** 2).sum()


def test_printed_floors_are_twice_the_feature_width():
    g = _golden()
    n = int(g["calibration_positions"])
    for k, key in ((20, "ess_floor_ministral3b"), (12, "ess_floor_ministral8b"), (8, "ess_floor_qwen")):
        # concentrated sensitivities: the floor binds and the effective sample size lands exactly on it
        rng = np.random.default_rng(k)
        r = np.exp(3.0 * rng.standard_normal(n))
        w, alpha, cv2 = oracle.ess_weights(r, k * 128)
        assert 0.0 < alpha < 1.0
        np.testing.assert_allclose(_kish(w), g[key], rtol=1e-9)
        assert min(n, 2 * k * 128) == g[key]


@pytest.mark.parametrize("sigma", [0.0, 0.05, 1.0, 4.0])
def test_kish_identity_mean_one_and_monotone_shrinkage(sigma):
    rng = np.random.default_rng(1)
    n, p = 6000, 128
    r = np.exp(sigma * rng.standard_normal(n)) * 7.3            # any positive scale: it is normalised away
    w, alpha, cv2 = oracle.ess_weights(r, p)
    rn = r / r.mean()
    np.testing.assert_allclose(cv2, ((rn - 1) ** 2).mean(), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(w.mean(), 1.0, rtol=1e-12)                                   # mean-one weights
    np.testing.assert_allclose(_kish(w), n / (1 + alpha ** 2 * cv2), rtol=1e-10)            # Kish identity
    assert _kish(w) >= min(n, 2 * p) * (1 - 1e-12)                                          # the floor holds
    np.testing.assert_allclose(w, 1 + alpha * (rn - 1), rtol=1e-13)
    if sigma == 0.0:
        assert alpha == 1.0 and cv2 < 1e-24 and np.allclose(w, 1.0, rtol=0, atol=1e-12)
    if sigma == 0.05:
        assert alpha == 1.0                                      # mild weights pass unchanged
    assert (w > 0).all()                                        # alpha <= 1 and r >= 0 keep the weights positive


def test_short_samples_are_forced_uniform_and_zero_rows_are_uniform():
    rng = np.random.default_rng(2)
    r = np.exp(rng.standard_normal(100))
    w, alpha, _ = oracle.ess_weights(r, 128)                    # n < 2p: tau = n, so only uniform weights reach n_eff = n
    assert alpha == 0.0 and np.array_equal(w, np.ones(100))
    w, alpha, cv2 = oracle.ess_weights(np.zeros(50), 4)
    assert alpha == 1.0 and cv2 == 0.0 and np.array_equal(w, np.ones(50))
    W, A, CV = oracle.ess_weights(np.stack([r, 2 * r, np.ones(100)]), 16)
    np.testing.assert_allclose(W[0], W[1], rtol=1e-13)          # scale invariance
    assert A[2] == 1.0 and np.array_equal(W[2], np.ones(100))
