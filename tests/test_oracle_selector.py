"""Pins for the oracle's layer selector (Section 3.1: centred single-source-layer OLS probes, held-in R^2 averaged over
KV heads and K/V, ranked)."""
import numpy as np
import pytest

import oracle


@pytest.mark.parametrize("seed,weighted", [(0, False), (1, True)])
def test_probe_r2_against_a_library_regression(seed, weighted):
    from sklearn.linear_model import LinearRegression
    from sklearn.metrics import r2_score
    rng = np.random.default_rng(seed)
    n, d = 300, 6
    X = rng.standard_normal((n, d)) + 3.0
    Y = X @ rng.standard_normal((d, d)) * 0.5 + 1.5 * rng.standard_normal((n, d)) - 2.0
    w = rng.uniform(0.2, 3.0, n) if weighted else np.ones(n)
    r2, info = oracle.probe_r2(X, Y, w)
    reg = LinearRegression().fit(X, Y, sample_weight=w)
    want = r2_score(Y, reg.predict(X), sample_weight=w, multioutput="variance_weighted")
    assert info == 0 and abs(r2 - want) < 1e-10
    assert 0.0 < r2 < 1.0


def test_probe_r2_closed_cases():
    rng = np.random.default_rng(2)
    n, d = 200, 4
    X = rng.standard_normal((n, d))
    w = rng.uniform(0.5, 2.0, n)
    r2, _ = oracle.probe_r2(X, X @ rng.standard_normal((d, d)) + 7.0, w)      # exact affine target
    assert abs(r2 - 1.0) < 1e-12
    r2, _ = oracle.probe_r2(X, rng.standard_normal((n, d)), w)                 # unrelated target: only chance fit
    assert 0.0 <= r2 < 0.1
    r2s, _ = oracle.probe_r2(X + 100.0, X @ np.eye(d) * 2.0 - 50.0, w)         # shifts do not matter (centred probe)
    assert abs(r2s - 1.0) < 1e-9
    shr, _ = oracle.probe_r2(X, X @ rng.standard_normal((d, d)), w, lambda_rel=0.5)
    assert shr < 1.0                                                           # shrinkage costs held-in fit


def test_ranking_by_brute_force():
    rng = np.random.default_rng(3)
    scores = rng.standard_normal((5, 9))
    scores[2, 4] = scores[2, 6]                                                # a tie: the lower index wins
    for k in (1, 3, 9):
        sets = oracle.rank_layers(scores, k)
        for l in range(5):
            order = sorted(range(9), key=lambda j: (-scores[l, j], j))[:k]
            assert sets[l].tolist() == sorted(order)


def test_selector_finds_the_generating_layers():
    """Targets built from known source layers: the selector must rank those layers first."""
    rng = np.random.default_rng(4)
    Ls, Lt, H, T, d = 5, 3, 2, 400, 4
    src = rng.standard_normal((2, Ls, T, H, d))
    truth = [[3, 1], [0, 4], [2, 3]]                                           # strongest, second strongest layer
    tgt = np.zeros((2, Lt, T, H, d))
    for comp in range(2):
        for l in range(Lt):
            for h in range(H):
                tgt[comp, l, :, h, :] = (src[comp, truth[l][0], :, h, :] @ rng.standard_normal((d, d))
                                          + 0.4 * src[comp, truth[l][1], :, h, :] @ rng.standard_normal((d, d))
                                          + 0.3 * rng.standard_normal((T, d)))
    enc = lambda a: oracle.bf16_encode(a).reshape(a.shape)
    w = np.ones((Lt, H, T), np.float32)
    scores = oracle.layer_scores(enc(src[0]), enc(src[1]), enc(tgt[0]), enc(tgt[1]), w, w, np.arange(H))
    sets1 = oracle.rank_layers(scores, 1)
    sets2 = oracle.rank_layers(scores, 2)
    for l in range(Lt):
        assert sets1[l, 0] == truth[l][0]
        assert sets2[l].tolist() == sorted(truth[l])
