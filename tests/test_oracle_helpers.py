"""Pins for the oracle's composed helpers, which the GPU tests use as expected values: the k > 1 apply (Section 3.2,
Eq. "localfeature": the feature concatenates the selected layers, layer-major), the rotary boundary around the key
map (Section 2.2 / Section 3.1: source embedding removed, map applied, target embedding restored) and the layer
selector's score table (Section 3.1: mean of the probe R^2 over KV heads and K/V).  Every expected value below is
written by hand or computed by another route than the helper's own."""
import os

import numpy as np

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = line.split("=")
                out[k.strip()] = float(v)
    return out


def _enc(a):
    a = np.asarray(a, dtype=np.float64)
    return oracle.bf16_encode(a).reshape(a.shape)


# ----------------------------------------------------------------------------------------------- k > 1 apply
def test_apply_multilayer_hand_example():
    """k = 2, d = 2, three source layers, two heads; every number is a small integer (exact in bf16).
    The map scales layer 2's head by 2 (first block), swaps and negates layer 0's channels (second block) and
    adds the bias (10, 20).  layer_set = (2, 0): the FIRST block of W belongs to layer 2."""
    src = np.zeros((3, 2, 2, 2))                    # [layer][token][head][channel]
    src[0, :, 1, :] = [[1, 2], [3, 4]]              # layer 0, head 1
    src[2, :, 1, :] = [[5, 6], [7, 8]]              # layer 2, head 1
    src[1, :, 1, :] = [[100, 100], [100, 100]]      # not selected: must not show up
    src[:, :, 0, :] = 50                            # other head: must not show up
    W = np.array([[2, 0], [0, 2],                   # block of layer_set[0] = layer 2
                  [0, -1], [1, 0]], float)          # block of layer_set[1] = layer 0: (x0, x1) -> (x1, -x0)
    Theta = np.vstack([W, [10, 20]])
    y, yb = oracle.apply_multilayer(_enc(src), Theta, [2, 0], 1)
    #  token 0: 2*(5, 6) + (2, -1) + (10, 20) = (22, 31);   token 1: 2*(7, 8) + (4, -3) + (10, 20) = (28, 33)
    assert np.array_equal(y, np.array([[22.0, 31.0], [28.0, 33.0]]))
    assert np.array_equal(oracle.bf16_decode(yb).reshape(y.shape), y)
    # the other order of the same set must read the blocks the other way round
    y2, _ = oracle.apply_multilayer(_enc(src), Theta, [0, 2], 1)
    #  token 0: 2*(1, 2) + (6, -5) + (10, 20) = (18, 19);   token 1: 2*(3, 4) + (8, -7) + (10, 20) = (24, 21)
    assert np.array_equal(y2, np.array([[18.0, 19.0], [24.0, 21.0]]))


def test_apply_multilayer_block_identity_and_single_layer_case():
    rng = np.random.default_rng(0)
    L, T, H, d, k = 5, 7, 3, 4, 3
    src = _enc(rng.standard_normal((L, T, H, d)))
    dec = oracle.bf16_decode(src).reshape(src.shape)
    sets = [4, 1, 2]
    for f, g in [(0, 0), (1, 2), (2, 1)]:
        Theta = np.zeros((k * d + 1, d))
        Theta[f * d:(f + 1) * d] = np.eye(d)        # block identity: returns head g of layer sets[f] unchanged
        y, yb = oracle.apply_multilayer(src, Theta, sets, g)
        assert np.array_equal(y, dec[sets[f], :, g, :])
        assert np.array_equal(yb, src[sets[f], :, g, :])
    # k = 1 reduces to the single-layer apply (a C function with its own pins)
    Theta1 = rng.standard_normal((d + 1, d))
    y, yb = oracle.apply_multilayer(src, Theta1, [3], 2)
    sl = np.full(1, 3, np.int32)
    sh = np.array([2], np.int32)
    (ok, _), (bk, _) = oracle.apply_maps(src, src, np.stack([Theta1, Theta1]), 1, 1, sl, sh)
    assert np.abs(y - ok[0, :, 0, :]).max() < 1e-14 and np.array_equal(yb, bk[0, :, 0, :])
    # linear in W: the sum of the per-layer single applies (bias counted once)
    Theta = rng.standard_normal((k * d + 1, d))
    want = Theta[-1][None, :].repeat(T, 0)
    for f, j in enumerate(sets):
        want = want + dec[j, :, 1, :] @ Theta[f * d:(f + 1) * d]
    y, _ = oracle.apply_multilayer(src, Theta, sets, 1)
    assert np.abs(y - want).max() < 1e-13


# ----------------------------------------------------------------------------------------------- rotary boundary
def test_apply_rope_rows_hand_example():
    """d = 4 at position 1 with the printed cos/sin of 1 and 0.01 (base 10000: theta = 1, 0.01)."""
    g = _read_golden("rope_hand_example.txt")
    c1, s1, c2, s2 = g["cos1"], g["sin1"], g["cos001"], g["sin001"]
    pos = np.array([1], np.int32)
    I = np.vstack([np.eye(4), np.zeros(4)])
    # (a) identity map, equal bases: the stored key comes back
    x = np.array([[1.0, 2.0, -3.0, 0.5]])
    out = oracle.apply_rope_rows(_enc(x), I, pos, 1e4, 1e4)
    assert np.abs(out - x).max() < 1e-15
    # (b) W = 0, bias e0: the bias lives in content coordinates and is rotated FORWARD by the target's angle
    Tb = np.zeros((5, 4)); Tb[4, 0] = 1.0
    out = oracle.apply_rope_rows(_enc(x), Tb, pos, 1e4, 1e4)
    assert np.abs(out - np.array([[c1, 0, s1, 0]])).max() < 1e-15
    # (c) identity map, stored key = R(1) e0 = (cos 1, 0, sin 1, 0) rounded to bf16: removing the source embedding
    # gives ~e0, restoring it gives the stored row again; a map that sends channel 0 to channel 1 instead moves the
    # content to the second pair, which turns by 0.01 rad: the source rotation must be the INVERSE one and the
    # target rotation the FORWARD one, or the signs below flip
    xs = oracle.bf16_decode(_enc(np.array([[c1, 0, s1, 0]]))).reshape(1, 4)
    P = np.zeros((5, 4)); P[0, 1] = 1.0; P[2, 3] = 1.0          # content (a, ., b, .) -> (., a, ., b)
    out = oracle.apply_rope_rows(_enc(xs), P, pos, 1e4, 1e4)
    a = c1 * xs[0, 0] + s1 * xs[0, 2]                           # content channel 0 (~1)
    b = -s1 * xs[0, 0] + c1 * xs[0, 2]                          # content channel 2 (~0)
    want = np.array([[0, a * c2 - b * s2, 0, a * s2 + b * c2]])
    assert np.abs(out - want).max() < 1e-15
    assert abs(a - 1.0) < 4e-3 and abs(b) < 4e-3               # bf16 rounding of the stored row only


def test_apply_rope_rows_different_bases_give_the_angle_difference():
    """W = I, b = 0: the row turns by pos * (theta_tgt - theta_src) in every pair."""
    rng = np.random.default_rng(1)
    d, n = 8, 12
    x = oracle.bf16_decode(_enc(rng.standard_normal((n, d)))).reshape(n, d)
    pos = rng.integers(0, 3000, n).astype(np.int32)
    bs, bt = 1e4, 5e5
    I = np.vstack([np.eye(d), np.zeros(d)])
    out = oracle.apply_rope_rows(_enc(x), I, pos, bs, bt)
    i = np.arange(d // 2)
    dphi = pos[:, None] * (bt ** (-2.0 * i / d) - bs ** (-2.0 * i / d))[None, :]
    lo, hi = x[:, :d // 2], x[:, d // 2:]
    want = np.concatenate([lo * np.cos(dphi) - hi * np.sin(dphi), lo * np.sin(dphi) + hi * np.cos(dphi)], axis=1)
    assert np.abs(out - want).max() < 1e-9                       # angles up to 3e3 rad in fp64
    assert np.abs(out - x).max() > 0.1                           # and it is not the identity
    # swapping the bases turns the other way
    out2 = oracle.apply_rope_rows(_enc(x), I, pos, bt, bs)
    want2 = np.concatenate([lo * np.cos(dphi) + hi * np.sin(dphi), -lo * np.sin(dphi) + hi * np.cos(dphi)], axis=1)
    assert np.abs(out2 - want2).max() < 1e-9


# ----------------------------------------------------------------------------------------------- layer scores
def test_layer_scores_numeric_pin():
    """scores[l][j] = mean over (K/V, head) of the probe R^2; recomputed here from numpy least squares."""
    rng = np.random.default_rng(5)
    Ls, Lt, Hs, Ht, T, d = 3, 2, 2, 3, 90, 3
    src = [_enc(rng.standard_normal((Ls, T, Hs, d)) + 1.0) for _ in range(2)]
    tgt = [_enc(rng.standard_normal((Lt, T, Ht, d)) * 0.5 - 1.0) for _ in range(2)]
    # make some pairs predictable so that the scores differ
    src_head0 = 0                                                # target head 0 reads source head 0 (src_head below)
    s0 = oracle.bf16_decode(src[0]).reshape(src[0].shape)
    t0 = oracle.bf16_decode(tgt[0]).reshape(tgt[0].shape)
    t0[1, :, 0, :] += 2.0 * s0[2, :, src_head0, :] @ rng.standard_normal((d, d))
    tgt[0] = _enc(t0)
    w = [rng.uniform(0.3, 2.0, (Lt, Ht, T)).astype(np.float32) for _ in range(2)]
    src_head = np.array([0, 1, 1], np.int32)
    got = oracle.layer_scores(src[0], src[1], tgt[0], tgt[1], w[0], w[1], src_head)
    assert got.shape == (Lt, Ls) and np.isfinite(got).all()
    dec = lambda a: oracle.bf16_decode(a).reshape(a.shape)
    for l in range(Lt):
        for j in range(Ls):
            acc = []
            for comp in range(2):
                for h in range(Ht):
                    X = dec(src[comp])[j, :, src_head[h], :]
                    Y = dec(tgt[comp])[l, :, h, :]
                    ww = w[comp][l, h].astype(np.float64)
                    sq = np.sqrt(ww)[:, None]
                    A = np.hstack([X, np.ones((T, 1))]) * sq
                    coef = np.linalg.lstsq(A, Y * sq, rcond=None)[0]
                    res = Y - np.hstack([X, np.ones((T, 1))]) @ coef
                    ybar = (ww[:, None] * Y).sum(0) / ww.sum()
                    acc.append(1.0 - (ww[:, None] * res ** 2).sum() / (ww[:, None] * (Y - ybar) ** 2).sum())
            assert abs(got[l, j] - np.mean(acc)) < 1e-10
    assert got[1, 2] > got[1, 0] + 0.05                          # the planted dependence shows in the table
    # a restricted call leaves the other rows untouched (NaN) and agrees on the requested row
    part = oracle.layer_scores(src[0], src[1], tgt[0], tgt[1], w[0], w[1], src_head, layers=[1])
    assert np.isnan(part[0]).all() and np.allclose(part[1], got[1], atol=1e-14)
