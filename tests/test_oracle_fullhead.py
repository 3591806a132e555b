"""Pins for the oracle's full-head contrast statistics (Section 3.1, full-head feature)."""
import numpy as np

import oracle
from paper_2609_00891_b200 import synth
from util import bits


def test_layer_sets_are_k_consecutive_layers_around_the_nearest_depth_layer():
    sets = oracle.fullhead_layer_sets(40, 64, 4)
    sl, _ = oracle.head_map(40, 8, 64, 8)
    assert sets.shape == (64, 4)
    for l in range(64):
        s = sets[l].tolist()
        assert s == list(range(s[0], s[0] + 4)) and 0 <= s[0] and s[-1] <= 39
        assert sl[l] in s                                      # the nearest-depth layer is always selected
        if 1 <= sl[l] <= 37:
            assert s[0] == sl[l] - 1                           # {c-1, c, c+1, c+2}
    assert sets[0].tolist() == [0, 1, 2, 3] and sets[63].tolist() == [36, 37, 38, 39]


def test_fullhead_statistics_against_numpy_on_gathered_features():
    wl = synth.workload("mini_ragged")                         # 4 source layers x 4 heads x 128
    sl, sh = oracle.head_map(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    ch = synth.make_chunk(wl, 0, sl, sh)
    T = 96
    src = bits(ch["src_v"][:, :T].contiguous())
    tgt = bits(ch["tgt_v"][:, :T].contiguous())
    w = ch["w_v"][2, 0, :T].contiguous().numpy()
    layer_set = [1, 2]
    l = 3
    G, C = oracle.fullhead_stats(src, tgt, w, l, layer_set)
    X = np.concatenate([ch["src_v"][j, :T, g].double().numpy() for j in layer_set for g in range(wl.Hs)], axis=1)
    Xt = np.concatenate([X, np.ones((T, 1))], axis=1)
    pf = 2 * wl.Hs * wl.d + 1
    assert G.shape == (pf, pf) and C.shape == (wl.Ht, pf, wl.d)
    np.testing.assert_allclose(G, Xt.T @ (w[:, None].astype(np.float64) * Xt), rtol=1e-12, atol=1e-9)
    for h in range(wl.Ht):
        Y = ch["tgt_v"][l, :T, h].double().numpy()
        np.testing.assert_allclose(C[h], Xt.T @ (w[:, None].astype(np.float64) * Y), rtol=1e-12, atol=1e-9)
    # with one selected layer and the matched head only, the head-local statistics are a sub-block
    Gl, Cl = oracle.stats_f64(ch["src_v"][1, :T, 0].double().numpy(), ch["tgt_v"][l, :T, 0].double().numpy(), w.astype(np.float64))
    d = wl.d
    np.testing.assert_allclose(G[:d, :d], Gl[:d, :d], rtol=1e-12, atol=1e-9)
    np.testing.assert_allclose(C[0][:d], Cl[:d], rtol=1e-12, atol=1e-9)
    np.testing.assert_allclose(G[pf - 1, pf - 1], w.astype(np.float64).sum(), rtol=1e-12)


def test_general_width_solve_and_multilayer_statistics():
    rng = np.random.default_rng(3)
    n, px, dy = 400, 37, 5
    X = rng.standard_normal((n, px)) + 0.5
    A = rng.standard_normal((px, dy))
    b = rng.standard_normal(dy)
    Y = X @ A + b
    w = np.exp(rng.standard_normal(n))
    Xt = np.concatenate([X, np.ones((n, 1))], axis=1)
    G, C = Xt.T @ (w[:, None] * Xt), Xt.T @ (w[:, None] * Y)
    Th, info = oracle.ridge_solve_general(G, C, n, 1e-12, raw_lambda=True)
    assert info == 0
    np.testing.assert_allclose(Th[:px], A, atol=1e-7)              # exact recovery for a wide regressor
    np.testing.assert_allclose(Th[px], b, atol=1e-7)
    # for p = d + 1 it is the same routine as the head-local solve
    d = 6
    Xs, Ys = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    G2, C2 = oracle.stats_f64(Xs, Ys, w)
    T1, _ = oracle.ridge_solve(G2, C2, n, 0.3)
    T2, _ = oracle.ridge_solve_general(G2, C2, n, 0.3)
    assert np.array_equal(T1, T2)
    lam = 0.7
    J = np.diag([1.0] * px + [0.0])
    Th, _ = oracle.ridge_solve_general(G, C, n, lam)
    res = (G + lam * w.sum() / n * J) @ Th - C
    assert np.linalg.norm(res) / np.linalg.norm(C) < 1e-12

    wl = synth.workload("mini_ragged")
    sl, sh = oracle.head_map(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    ch = synth.make_chunk(wl, 0, sl, sh)
    T = 80
    src, tgt = bits(ch["src_k"][:, :T].contiguous()), bits(ch["tgt_k"][:, :T].contiguous())
    wt = ch["w_k"][1, 2, :T].contiguous().numpy()
    Gm, Cm = oracle.multilayer_stats(src, tgt, wt, 1, 2, 3, [0, 2, 3])
    Xf = np.concatenate([ch["src_k"][j, :T, 3].double().numpy() for j in (0, 2, 3)], axis=1)
    Xft = np.concatenate([Xf, np.ones((T, 1))], axis=1)
    Yf = ch["tgt_k"][1, :T, 2].double().numpy()
    np.testing.assert_allclose(Gm, Xft.T @ (wt[:, None].astype(np.float64) * Xft), rtol=1e-12, atol=1e-9)
    np.testing.assert_allclose(Cm, Xft.T @ (wt[:, None].astype(np.float64) * Yf), rtol=1e-12, atol=1e-9)
