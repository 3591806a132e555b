"""Pins for the head match, the static gather schedule and the artifact size."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_printed_values.txt")


def _golden():
    out = {}
    with open(GOLD) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = line.split("=")
                out[k.strip()] = float(v)
    return out


@pytest.mark.parametrize("Ls,Lt", [(2, 2), (36, 40), (40, 64), (3, 5), (4, 6), (40, 1), (5, 3)])
def test_nearest_depth_rule_is_rounding(Ls, Lt):
    sl, sh = oracle.head_map(Ls, 8, Lt, 8)
    for l in range(Lt):
        if Lt == 1:
            assert sl[l] == 0
            continue
        x = Fraction(l * (Ls - 1), Lt - 1)
        lo = x.numerator // x.denominator
        want = lo + (1 if x - lo >= Fraction(1, 2) else 0)      # round half up
        assert sl[l] == want
        assert 0 <= sl[l] < Ls
    assert sh.tolist() == list(range(8))                       # aligned KV groups: a(h) = h


def test_match_counts_of_the_benchmark_shapes():
    sl, _ = oracle.head_map(40, 8, 64, 8)
    counts = np.bincount(sl, minlength=40)
    assert counts.min() == 1 and counts.max() == 2 and (counts == 2).sum() == 24
    for l in range(64):                                         # no ties: the rule is unambiguous here
        assert Fraction(l * 39, 63) % 1 != Fraction(1, 2)
    sl, _ = oracle.head_map(36, 8, 40, 8)
    counts = np.bincount(sl, minlength=36)
    assert (counts == 2).sum() == 4 and counts.min() == 1
    assert sl[0] == 0 and sl[-1] == 35


def test_head_fanin_when_group_counts_differ():
    _, sh = oracle.head_map(4, 2, 4, 8)
    assert sh.tolist() == [0, 0, 0, 0, 1, 1, 1, 1]
    _, sh = oracle.head_map(4, 8, 4, 2)
    assert sh.tolist() == [0, 4]


@pytest.mark.parametrize("Ls,Hs,Lt,Ht", [(2, 2, 2, 2), (3, 2, 5, 2), (40, 8, 64, 8), (4, 2, 6, 8)])
def test_work_list_groups_every_map_once(Ls, Hs, Lt, Ht):
    sl, sh = oracle.head_map(Ls, Hs, Lt, Ht)
    ic, il, ih, ib, im = oracle.work_list(Ls, Hs, Lt, Ht, sl, sh)
    groups = {}
    for m in range(2 * Lt * Ht):
        comp, l, h = m // (Lt * Ht), (m // Ht) % Lt, m % Ht
        groups.setdefault((comp, int(sl[l]), int(sh[h])), []).append(m)
    keys = sorted(groups)
    assert len(ic) == len(keys)
    assert sorted(im.tolist()) == list(range(2 * Lt * Ht))
    for i, key in enumerate(keys):
        assert (int(ic[i]), int(il[i]), int(ih[i])) == key
        assert im[ib[i]:ib[i + 1]].tolist() == groups[key]


def test_coefficient_counts_reproduce_printed_storage():
    g = _golden()
    c_full, c_local, n_bias = oracle.coefficient_counts(Lt=64, Ht=8, Hs=8, k=8, ds=128, dt=128)
    assert c_full // c_local == g["coefficient_ratio"] and c_full % c_local == 0
    assert c_full // (2 * 64 * 8 * 128) == g["width_full_qwen"]
    assert c_local // (2 * 64 * 8 * 128) == g["width_local_qwen"]
    # fp32 coefficients plus biases, decimal GB: within 0.2 % of the printed, rounded figures
    assert abs((c_full + n_bias) * 4 / 1e9 - g["mapper_storage_full_head_gb"]) / g["mapper_storage_full_head_gb"] < 2e-3
    assert abs((c_local + n_bias) * 4 / 1e9 - g["mapper_storage_head_local_gb"]) / g["mapper_storage_head_local_gb"] < 2e-3
    for k, full, local in ((20, "width_full_ministral3b", "width_local_ministral3b"),
                           (12, "width_full_ministral8b", "width_local_ministral8b")):
        cf, cl, _ = oracle.coefficient_counts(Lt=40, Ht=8, Hs=8, k=k, ds=128, dt=128)
        assert cf // (2 * 40 * 8 * 128) == g[full] and cl // (2 * 40 * 8 * 128) == g[local]
