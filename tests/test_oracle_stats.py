"""Pins for the oracle's sufficient statistics (Section 3.4, statistics before centring)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2609_00891_b200 import synth
from util import bits

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


def brute_stats(X, Y, w):
    """The definition with Python integers/floats, one scalar at a time."""
    n, d = len(X), len(X[0])
    p = d + 1
    G = [[0] * p for _ in range(p)]
    C = [[0] * d for _ in range(p)]
    for t in range(n):
        xt = list(X[t]) + [1]
        for i in range(p):
            for j in range(p):
                G[i][j] += w[t] * xt[i] * xt[j]
            for j in range(d):
                C[i][j] += w[t] * xt[i] * Y[t][j]
    return G, C


def test_hand_worked_example():
    gold = _read_golden("stats_hand_example.txt")
    G, C = oracle.stats_f64(np.array([[1, 2], [3, 4.0]]), np.array([[1, 0], [0, 1.0]]), np.array([1, 2.0]))
    assert G.ravel().tolist() == gold["G"]
    assert C.ravel().tolist() == gold["C"]


@pytest.mark.parametrize("n,d,seed", [(1, 1, 0), (5, 3, 1), (8, 4, 2), (7, 2, 3)])
def test_brute_force_small_integers(n, d, seed):
    rng = np.random.default_rng(seed)
    X = rng.integers(-5, 6, (n, d))
    Y = rng.integers(-5, 6, (n, d))      # Y != X and not symmetric: catches a swapped or transposed operand
    w = rng.integers(0, 4, n)
    Gb, Cb = brute_stats(X.tolist(), Y.tolist(), w.tolist())
    G, C = oracle.stats_f64(X, Y, w)
    assert np.array_equal(G, np.array(Gb, dtype=np.float64))
    assert np.array_equal(C, np.array(Cb, dtype=np.float64))


def _random_problem(n, d, seed):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, d)) * np.exp(0.5 * rng.standard_normal(d)) + rng.standard_normal(d)
    Y = rng.standard_normal((n, d)) + 0.3 * X[:, ::-1]
    w = np.exp(rng.standard_normal(n))
    return X, Y, w


def test_closed_forms_symmetry_and_library_product():
    X, Y, w = _random_problem(200, 6, 5)
    G, C = oracle.stats_f64(X, Y, w)
    d = 6
    np.testing.assert_allclose(G, G.T, rtol=1e-14, atol=1e-12)      # (w x_i) x_j vs (w x_j) x_i: rounding only
    np.testing.assert_allclose(G[d, d], w.sum(), rtol=1e-13)
    np.testing.assert_allclose(G[d, :d], (w[:, None] * X).sum(0), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(C[d], (w[:, None] * Y).sum(0), rtol=1e-12, atol=1e-12)
    Xt = np.concatenate([X, np.ones((200, 1))], axis=1)
    np.testing.assert_allclose(G, Xt.T @ (w[:, None] * Xt), rtol=1e-12, atol=1e-11)
    np.testing.assert_allclose(C, Xt.T @ (w[:, None] * Y), rtol=1e-12, atol=1e-11)
    assert np.linalg.eigvalsh(G).min() > -1e-9 * np.linalg.eigvalsh(G).max()   # PSD


def test_additive_over_token_splits_and_weight_scaling():
    X, Y, w = _random_problem(300, 5, 6)
    G, C = oracle.stats_f64(X, Y, w)
    for cut in (1, 117, 299):
        G1, C1 = oracle.stats_f64(X[:cut], Y[:cut], w[:cut])
        G2, C2 = oracle.stats_f64(X[cut:], Y[cut:], w[cut:])
        np.testing.assert_allclose(G1 + G2, G, rtol=1e-13, atol=1e-12)
        np.testing.assert_allclose(C1 + C2, C, rtol=1e-13, atol=1e-12)
    Gs, Cs = oracle.stats_f64(X, Y, 4.0 * w)                          # power of two: exact
    assert np.array_equal(Gs, 4.0 * G) and np.array_equal(Cs, 4.0 * C)


def test_zero_weight_rows_do_not_count():
    X, Y, w = _random_problem(50, 4, 7)
    w[10:20] = 0.0
    keep = w > 0
    G, C = oracle.stats_f64(X, Y, w)
    G2, C2 = oracle.stats_f64(X[keep], Y[keep], w[keep])
    np.testing.assert_allclose(G, G2, rtol=1e-14, atol=1e-13)
    np.testing.assert_allclose(C, C2, rtol=1e-14, atol=1e-13)


def test_trace_reader_matches_per_map_rows():
    """The strided bf16 reader (layout [L][T][H][d], head match, K/V, weights) against rows gathered with numpy."""
    wl = synth.workload("mini_scaled")
    sl, sh = oracle.head_map(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    ch = synth.make_chunk(wl, 0, sl, sh)
    a = {k: bits(v) for k, v in ch.items() if k.startswith(("src", "tgt"))}
    wk, wv = ch["w_k"].numpy(), ch["w_v"].numpy()
    maps = [0, 3, 7, wl.n_maps // 2, wl.n_maps - 1]
    G, C = oracle.stats_traces(a["src_k"], a["src_v"], a["tgt_k"], a["tgt_v"], wk, wv, sl, sh, maps)
    for s, m in enumerate(maps):
        comp, l, h = m // (wl.Lt * wl.Ht), (m // wl.Ht) % wl.Lt, m % wl.Ht
        src = ch["src_v" if comp else "src_k"][sl[l], :, sh[h], :].double().numpy()
        tgt = ch["tgt_v" if comp else "tgt_k"][l, :, h, :].double().numpy()
        w = (wv if comp else wk)[l, h].astype(np.float64)
        G1, C1 = oracle.stats_f64(src, tgt, w)
        np.testing.assert_allclose(G[s], G1, rtol=1e-13, atol=1e-12)
        np.testing.assert_allclose(C[s], C1, rtol=1e-13, atol=1e-12)


def test_trace_reader_accepts_head_major_layout():
    wl = synth.workload("mini_scaled")
    sl, sh = oracle.head_map(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    ch = synth.make_chunk(wl, 1, sl, sh)
    a = {k: bits(v) for k, v in ch.items() if k.startswith(("src", "tgt"))}
    wk, wv = ch["w_k"].numpy(), ch["w_v"].numpy()
    G, C = oracle.stats_traces(a["src_k"], a["src_v"], a["tgt_k"], a["tgt_v"], wk, wv, sl, sh)
    hm = {k: np.ascontiguousarray(v.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3) for k, v in a.items()}  # [L][H][T][d] storage
    G2, C2 = oracle.stats_traces(hm["src_k"], hm["src_v"], hm["tgt_k"], hm["tgt_v"], wk, wv, sl, sh)
    assert np.array_equal(G, G2) and np.array_equal(C, C2)


def test_bf16_codec_against_torch():
    g = torch.Generator().manual_seed(3)
    x = torch.randn(4096, generator=g) * torch.exp(4 * torch.randn(4096, generator=g))
    x[:4] = torch.tensor([0.0, -0.0, 1.0, -3.0e38])
    b = x.to(torch.bfloat16)                      # library round-to-nearest-even from binary32
    enc = oracle.bf16_encode(x.double().numpy())
    assert np.array_equal(enc, bits(b))
    assert np.array_equal(oracle.bf16_decode(enc), b.double().numpy())
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert oracle.bf16_decode(oracle.bf16_encode(np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8]))).tolist() == [1.0, 1 + 2.0 ** -6]
