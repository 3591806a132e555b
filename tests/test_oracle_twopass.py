"""Pins for the oracle's two-pass centred construction (Section 3.4, Eq. fusedstats and the solve below it)."""
import os

import numpy as np
import pytest

import oracle
from util import rel_fro

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = line.split("=")
                out[k.strip()] = [float(x) for x in v.split()]
    return out


def _bf16_bits(x):
    """fp64 values that are exactly representable in bf16 -> their bit patterns."""
    b = oracle.bf16_encode(np.asarray(x, dtype=np.float64))
    assert np.array_equal(oracle.bf16_decode(b), np.asarray(x, dtype=np.float64))
    return b


def _traces(rng, Ls, Lt, H, T, d, lo=-8, hi=9, shift=0):
    """Small-integer traces (exact in bf16) [L][T][H][d], weights [Lt][H][T] on a grid of quarters."""
    sk = rng.integers(lo, hi, (Ls, T, H, d)).astype(np.float64) + shift
    sv = rng.integers(lo, hi, (Ls, T, H, d)).astype(np.float64) + shift
    tk = rng.integers(lo, hi, (Lt, T, H, d)).astype(np.float64)
    tv = rng.integers(lo, hi, (Lt, T, H, d)).astype(np.float64)
    wk = (rng.integers(0, 9, (Lt, H, T)) / 4.0).astype(np.float32)
    wv = (rng.integers(0, 9, (Lt, H, T)) / 4.0).astype(np.float32)
    return sk, sv, tk, tv, wk, wv


def _rows(sk, sv, tk, tv, wk, wv, sl, sh, m, Lt, H):
    comp, l, h = m // (Lt * H), (m // H) % Lt, m % H
    X = (sv if comp else sk)[sl[l], :, sh[h], :]
    Y = (tv if comp else tk)[l, :, h, :]
    w = (wv if comp else wk)[l, h, :].astype(np.float64)
    return X, Y, w


def test_hand_worked_example():
    gold = _read_golden("twopass_hand_example.txt")
    x = _bf16_bits(np.array([1, 2, 4.0]).reshape(1, 3, 1, 1))
    y = _bf16_bits(np.array([2, 3, 7.0]).reshape(1, 3, 1, 1))
    w = np.array([1, 1, 2], np.float32).reshape(1, 1, 3)
    sl, sh = np.zeros(1, np.int32), np.zeros(1, np.int32)
    sx, sy, sw = oracle.weighted_sums_traces(x, x, y, y, w, w, sl, sh, maps=[0])
    assert sx[0, 0] == gold["sum_x"][0] and sy[0, 0] == gold["sum_y"][0] and sw[0] == gold["s_w"][0]
    mu_x, mu_y = sx / sw[:, None], sy / sw[:, None]
    A, B = oracle.centered_stats_traces(x, x, y, y, w, w, sl, sh, mu_x, mu_y, maps=[0])
    assert A[0, 0, 0] == gold["A"][0] and B[0, 0, 0] == gold["B"][0]
    Theta, info = oracle.ridge_solve_centered(A[0], B[0], mu_x[0], mu_y[0], sw[0], 3, 0.0)
    W = gold["W_num"][0] / gold["W_den"][0]
    assert info == 0
    assert abs(Theta[0, 0] - W) < 1e-15 and abs(Theta[1, 0] - (4.75 - 2.75 * W)) < 1e-14


@pytest.mark.parametrize("seed", [0, 1])
def test_against_library_weighted_covariance(seed):
    """A / s_w is the weighted covariance of x and B / s_w the cross-covariance of x and y (numpy.cov with aweights)."""
    rng = np.random.default_rng(seed)
    Ls, Lt, H, T, d = 2, 3, 2, 40, 4
    sk, sv, tk, tv, wk, wv = _traces(rng, Ls, Lt, H, T, d)
    sl, sh = np.array([0, 1, 1], np.int32), np.array([1, 0], np.int32)     # crossed heads: catches a head mix-up
    args = [_bf16_bits(a) for a in (sk, sv, tk, tv)] + [wk, wv, sl, sh]
    sx, sy, sw = oracle.weighted_sums_traces(*args)
    mu_x, mu_y = sx / sw[:, None], sy / sw[:, None]
    A, B = oracle.centered_stats_traces(*args, mu_x, mu_y)
    for m in range(2 * Lt * H):
        X, Y, w = _rows(sk, sv, tk, tv, wk, wv, sl, sh, m, Lt, H)
        assert abs(sw[m] - w.sum()) < 1e-12
        assert np.allclose(mu_x[m], np.average(X, axis=0, weights=w), atol=1e-12)
        assert np.allclose(mu_y[m], np.average(Y, axis=0, weights=w), atol=1e-12)
        cov = np.cov(np.hstack([X, Y]).T, aweights=w, bias=True) * w.sum()
        assert np.allclose(A[m], cov[:d, :d], atol=1e-10)
        assert np.allclose(B[m], cov[:d, d:], atol=1e-10)
        assert not np.allclose(B[m], B[m].T, atol=1e-6)      # the pin would not see a transposed B otherwise


def test_shift_of_the_source_leaves_the_centred_statistics_unchanged():
    Ls, Lt, H, T, d = 2, 2, 1, 30, 3
    out = []
    for shift in (0, 64):                                       # 64 + small integers stay exact in bf16
        rng = np.random.default_rng(5)
        sk, sv, tk, tv, wk, wv = _traces(rng, Ls, Lt, H, T, d, lo=-1, hi=2, shift=shift)
        sl, sh = np.array([0, 1], np.int32), np.zeros(1, np.int32)
        args = [_bf16_bits(a) for a in (sk, sv, tk, tv)] + [wk, wv, sl, sh]
        sx, sy, sw = oracle.weighted_sums_traces(*args)
        mu_x, mu_y = sx / sw[:, None], sy / sw[:, None]
        out.append((mu_x, oracle.centered_stats_traces(*args, mu_x, mu_y)))
    (mu0, (A0, B0)), (mu1, (A1, B1)) = out
    assert np.allclose(mu1 - mu0, 64.0, atol=1e-12)
    assert np.allclose(A0, A1, atol=1e-9) and np.allclose(B0, B1, atol=1e-9)


@pytest.mark.parametrize("lam,raw", [(0.0, False), (0.3, False), (0.3, True)])
def test_same_map_as_the_bias_column_solve_and_the_literal_centred_route(lam, raw):
    rng = np.random.default_rng(7)
    Ls, Lt, H, T, d = 2, 2, 2, 60, 5
    sk, sv, tk, tv, wk, wv = _traces(rng, Ls, Lt, H, T, d, shift=16)
    sl, sh = np.array([0, 1], np.int32), np.array([0, 1], np.int32)
    args = [_bf16_bits(a) for a in (sk, sv, tk, tv)] + [wk, wv, sl, sh]
    sx, sy, sw = oracle.weighted_sums_traces(*args)
    mu_x, mu_y = sx / sw[:, None], sy / sw[:, None]
    A, B = oracle.centered_stats_traces(*args, mu_x, mu_y)
    G, C = oracle.stats_traces(*args)
    # algebraic identity between the two constructions
    for m in range(len(A)):
        assert np.allclose(A[m], G[m, :d, :d] - sw[m] * np.outer(mu_x[m], mu_x[m]), atol=1e-8)
        assert np.allclose(B[m], C[m, :d, :] - sw[m] * np.outer(mu_x[m], mu_y[m]), atol=1e-8)
    Th2, info2 = oracle.ridge_solve_centered(A, B, mu_x, mu_y, sw, T, lam, raw_lambda=raw)
    Th1, info1 = oracle.ridge_solve(G, C, T, lam, raw_lambda=raw)
    assert not info1.any() and not info2.any()
    assert rel_fro(Th2, Th1) < 1e-9
    if not raw:
        for m in (0, 3, 7):
            X, Y, w = _rows(sk, sv, tk, tv, wk, wv, sl, sh, m, Lt, H)
            Th3, info3 = oracle.ridge_centered(X, Y, w, lam)
            assert info3 == 0 and rel_fro(Th2[m], Th3) < 1e-9


def test_sums_add_over_chunks():
    rng = np.random.default_rng(9)
    Ls, Lt, H, T, d = 1, 2, 1, 24, 2
    sk, sv, tk, tv, wk, wv = _traces(rng, Ls, Lt, H, T, d)
    sl, sh = np.zeros(2, np.int32), np.zeros(1, np.int32)
    full = oracle.weighted_sums_traces(*[_bf16_bits(a) for a in (sk, sv, tk, tv)], wk, wv, sl, sh)
    parts = []
    for a, b in ((0, 10), (10, 24)):
        cut = [np.ascontiguousarray(x[:, a:b]) for x in (sk, sv, tk, tv)]
        parts.append(oracle.weighted_sums_traces(*[_bf16_bits(x) for x in cut], np.ascontiguousarray(wk[..., a:b]),
                                                 np.ascontiguousarray(wv[..., a:b]), sl, sh))
    for q in range(3):
        assert np.allclose(full[q], parts[0][q] + parts[1][q], atol=1e-12)
