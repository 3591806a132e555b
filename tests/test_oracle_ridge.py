"""Pins for the oracle's ridge solve (Section 3.1, closed form) and affine apply (Section 3.2)."""
import numpy as np
import pytest

import oracle
from paper_2609_00891_b200 import synth
from util import bits, rel_fro


def _problem(n, d, seed, shift=2.0):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, d)) * np.exp(0.5 * rng.standard_normal(d)) + shift * rng.standard_normal(d)
    A = rng.standard_normal((d, d)) / np.sqrt(d)
    b = rng.standard_normal(d)
    Y = X @ A + b + 0.1 * rng.standard_normal((n, d))
    w = np.exp(rng.standard_normal(n)) / (1 + np.arange(n) / 50.0)
    return X, Y, w, A, b


@pytest.mark.parametrize("lam", [1e-3, 1e-2, 1.0, 50.0])
def test_bias_column_form_equals_centred_two_pass(lam):
    """Augmented one-pass statistics with an unpenalised bias give the paper's centred estimator."""
    X, Y, w, _, _ = _problem(400, 7, 0)
    G, C = oracle.stats_f64(X, Y, w)
    Th, info = oracle.ridge_solve(G, C, 400, lam)
    Tc, info_c = oracle.ridge_centered(X, Y, w, lam)
    assert info == 0 and info_c == 0
    assert rel_fro(Th, Tc) < 1e-10


@pytest.mark.parametrize("c", [1.0, 0.37, 12.0])
def test_constant_weight_is_textbook_ridge(c):
    """w = const reduces to unweighted centred ridge with the same lambda, whatever the constant:
    least squares on the stacked system [Xc; sqrt(lambda) I] W = [Yc; 0]."""
    X, Y, _, _, _ = _problem(150, 5, 1)
    lam = 0.7
    G, C = oracle.stats_f64(X, Y, np.full(150, c))
    Th, info = oracle.ridge_solve(G, C, 150, lam)
    xb, yb = X.mean(0), Y.mean(0)
    Xs = np.concatenate([X - xb, np.sqrt(lam) * np.eye(5)])
    Ys = np.concatenate([Y - yb, np.zeros((5, 5))])
    W = np.linalg.lstsq(Xs, Ys, rcond=None)[0]
    b = yb - xb @ W
    assert info == 0
    np.testing.assert_allclose(Th[:5], W, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(Th[5], b, rtol=1e-9, atol=1e-11)


def test_exact_recovery_of_affine_map():
    rng = np.random.default_rng(2)
    n, d = 300, 6
    X = rng.standard_normal((n, d)) + 1.5
    A = rng.standard_normal((d, d))
    b = rng.standard_normal(d)
    Y = X @ A + b                                  # no noise, no rounding
    w = np.exp(rng.standard_normal(n))
    G, C = oracle.stats_f64(X, Y, w)
    lam = 1e-12 * np.trace(G[:d, :d]) / d
    Th, info = oracle.ridge_solve(G, C, n, lam, raw_lambda=True)
    assert info == 0
    np.testing.assert_allclose(Th[:d], A, atol=1e-8)
    np.testing.assert_allclose(Th[d], b, atol=1e-8)


def test_identity_map_when_target_equals_source_and_effective_dimension():
    """X = Y: W = I - lam (A + lam I)^-1 with A the centred mean-one scatter, b = mu (I - W);
    trace(W) is the ridge effective dimension, below d, tending to d (and W to I, b to 0) as lam -> 0."""
    X, _, w, _, _ = _problem(500, 6, 3)
    n, d = X.shape
    G, C = oracle.stats_f64(X, X, w)
    wm = w * n / w.sum()
    mu = (wm[:, None] * X).sum(0) / n
    Xc = X - mu
    A = Xc.T @ (wm[:, None] * Xc)
    prev = None
    for lam in (1e-9, 1e-2, 1.0, 100.0):
        Th, info = oracle.ridge_solve(G, C, n, lam)
        W, b = Th[:d], Th[d]
        assert info == 0
        np.testing.assert_allclose(W, np.eye(d) - lam * np.linalg.inv(A + lam * np.eye(d)), atol=1e-9)
        np.testing.assert_allclose(b, mu @ (np.eye(d) - W), atol=1e-9)
        deff = np.trace(A @ np.linalg.inv(A + lam * np.eye(d)))
        np.testing.assert_allclose(np.trace(W), deff, rtol=1e-9)
        assert np.trace(W) <= d + 1e-12
        if prev is not None:
            assert np.trace(W) < prev
        prev = np.trace(W)
    Th, _ = oracle.ridge_solve(G, C, n, 1e-9)
    np.testing.assert_allclose(Th[:d], np.eye(d), atol=1e-8)
    np.testing.assert_allclose(Th[d], 0, atol=1e-7)


def test_normal_equation_residual_and_shrinkage():
    X, Y, w, _, _ = _problem(400, 8, 4)
    n, d = X.shape
    G, C = oracle.stats_f64(X, Y, w)
    J = np.diag([1.0] * d + [0.0])
    prev = np.inf
    for lam in (1e-3, 1e-2, 1e-1, 1.0, 10.0, 1e3):
        Th, info = oracle.ridge_solve(G, C, n, lam)
        lam_eff = lam * w.sum() / n
        res = (G + lam_eff * J) @ Th - C
        assert info == 0 and np.linalg.norm(res) / np.linalg.norm(C) < 1e-12
        nrm = np.linalg.norm(Th[:d])
        assert nrm <= prev
        prev = nrm
    # raw-lambda mode penalises with lambda itself
    Th, _ = oracle.ridge_solve(G, C, n, 0.5, raw_lambda=True)
    assert np.linalg.norm((G + 0.5 * J) @ Th - C) / np.linalg.norm(C) < 1e-12


def test_weight_scale_invariance_of_the_fit():
    X, Y, w, _, _ = _problem(200, 4, 5)
    G, C = oracle.stats_f64(X, Y, w)
    G8, C8 = oracle.stats_f64(X, Y, 8.0 * w)
    T1, _ = oracle.ridge_solve(G, C, 200, 0.3)
    T8, _ = oracle.ridge_solve(G8, C8, 200, 0.3)
    assert rel_fro(T8, T1) < 1e-12


def test_degenerate_system_reports_pivot_and_zero_fills():
    X, Y, _, _, _ = _problem(20, 3, 6)
    G, C = oracle.stats_f64(X, Y, np.zeros(20))       # s_w = 0: nothing observed
    Th, info = oracle.ridge_solve(G, C, 20, 1e-2)
    assert info > 0 and not Th.any()
    G2, C2 = oracle.stats_f64(X, Y, np.ones(20))
    Tb, infob = oracle.ridge_solve(np.stack([G, G2]), np.stack([C, C2]), 20, 1e-2)
    assert infob[0] > 0 and infob[1] == 0 and not Tb[0].any() and np.isfinite(Tb[1]).all() and Tb[1].any()


def test_tiny_workload_recovers_generator_map():
    """The tiny workload draws Y = X A + b + 0.05 N(0,1): the fit must land on (A, b) within noise."""
    wl = synth.workload("tiny")
    sl, sh = oracle.head_map(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    law = synth.map_law(wl)
    ch = synth.make_chunk(wl, 0, sl, sh, law=law)
    a = {k: bits(v) for k, v in ch.items() if k.startswith(("src", "tgt"))}
    G, C = oracle.stats_traces(a["src_k"], a["src_v"], a["tgt_k"], a["tgt_v"],
                               ch["w_k"].numpy(), ch["w_v"].numpy(), sl, sh)
    Th, info = oracle.ridge_solve(G, C, wl.n_tokens, 1e-2)
    assert not info.any()
    A = law.A.reshape(wl.n_maps, wl.d, wl.d).double().numpy()
    b = law.b.reshape(wl.n_maps, wl.d).double().numpy()
    for m in range(wl.n_maps):
        assert rel_fro(Th[m, :wl.d], A[m]) < 0.05
        assert np.abs(Th[m, wl.d] - b[m]).max() < 0.05


# ------------------------------------------------------------------------------------------- apply
def test_apply_identity_returns_source_bits_and_matches_numpy():
    wl = synth.workload("mini_scaled")
    sl, sh = oracle.head_map(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    src = synth.make_source_cache(wl, 37)
    sk, sv = bits(src[0]), bits(src[1])
    d, p = wl.d, wl.d + 1
    Th = np.zeros((wl.n_maps, p, d))
    Th[:, :d, :] = np.eye(d)
    f64, b16 = oracle.apply_maps(sk, sv, Th, wl.Lt, wl.Ht, sl, sh)
    for comp, s in enumerate((sk, sv)):
        for l in range(wl.Lt):
            for h in range(wl.Ht):
                assert np.array_equal(b16[comp][l, :, h], s[sl[l], :, sh[h]])
    rng = np.random.default_rng(0)
    Th = rng.standard_normal((wl.n_maps, p, d))
    f64, b16 = oracle.apply_maps(sk, sv, Th, wl.Lt, wl.Ht, sl, sh)
    for comp, s in enumerate(src):
        x = s.double().numpy()
        for l in range(wl.Lt):
            for h in range(wl.Ht):
                m = (comp * wl.Lt + l) * wl.Ht + h
                ref = x[sl[l], :, sh[h]] @ Th[m, :d] + Th[m, d]
                np.testing.assert_allclose(f64[comp][l, :, h], ref, rtol=1e-12, atol=1e-12)
    assert np.array_equal(b16[0], oracle.bf16_encode(f64[0]))
    # linearity in the map: apply(T1 + T2) = apply(T1) + apply(T2)
    T2 = rng.standard_normal((wl.n_maps, p, d))
    g64, _ = oracle.apply_maps(sk, sv, T2, wl.Lt, wl.Ht, sl, sh, want_bf16=False)
    s64, _ = oracle.apply_maps(sk, sv, Th + T2, wl.Lt, wl.Ht, sl, sh, want_bf16=False)
    np.testing.assert_allclose(s64[1], f64[1] + g64[1], rtol=1e-11, atol=1e-11)
