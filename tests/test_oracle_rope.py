"""Pins for the oracle's rotary embedding at the boundary (Section 2.2, Section 3.1: source RoPE removed before the fit,
target RoPE restored after the map)."""
import os

import numpy as np
import pytest
import torch

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


def test_hand_example_unit_vectors():
    g = _read_golden("rope_hand_example.txt")
    pos = np.array([1, 1, 1], np.int32)
    out = oracle.rope_rotate(np.eye(4)[:3], pos, 10000.0)
    want = np.array([[g["cos1"], 0, g["sin1"], 0], [0, g["cos001"], 0, g["sin001"]], [-g["sin1"], 0, g["cos1"], 0]])
    assert np.abs(out - want).max() < 1e-15
    back = oracle.rope_rotate(np.eye(4)[:3], pos, 10000.0, inverse=True)
    want_inv = np.array([[g["cos1"], 0, -g["sin1"], 0], [0, g["cos001"], 0, -g["sin001"]], [g["sin1"], 0, g["cos1"], 0]])
    assert np.abs(back - want_inv).max() < 1e-15


@pytest.mark.parametrize("d,base", [(128, 1e6), (64, 1e4)])
def test_against_a_library_implementation(d, base):
    """transformers' Llama rotary embedding (rotate_half form) on fp64 tensors."""
    from transformers.models.llama.modeling_llama import apply_rotary_pos_emb
    rng = np.random.default_rng(3)
    n = 40
    x = rng.standard_normal((n, d))
    pos = rng.integers(0, 32768, n).astype(np.int32)
    inv_freq = 1.0 / (base ** (torch.arange(0, d, 2, dtype=torch.float64) / d))
    fr = torch.from_numpy(pos).double()[:, None] * inv_freq[None]
    emb = torch.cat([fr, fr], -1)
    q = torch.from_numpy(x)[None, None]
    qe, _ = apply_rotary_pos_emb(q, q, emb.cos()[None], emb.sin()[None])
    assert np.abs(qe[0, 0].numpy() - oracle.rope_rotate(x, pos, base)).max() < 1e-10   # angles up to 3e4 rad in fp64


def test_relative_position_identity_and_inverse():
    rng = np.random.default_rng(4)
    d, base = 16, 1e4
    q, k = rng.standard_normal((1, d)), rng.standard_normal((1, d))
    for m, n in [(5, 2), (100, 99), (7, 7), (3, 50)]:
        qm = oracle.rope_rotate(q, np.array([m], np.int32), base)
        kn = oracle.rope_rotate(k, np.array([n], np.int32), base)
        if m >= n:
            rel = oracle.rope_rotate(q, np.array([m - n], np.int32), base)
        else:
            rel = oracle.rope_rotate(q, np.array([n - m], np.int32), base, inverse=True)
        assert abs(float(qm @ kn.T) - float(rel @ k.T)) < 1e-12          # scores depend on m - n only
    x = rng.standard_normal((30, d))
    pos = rng.integers(0, 5000, 30).astype(np.int32)
    y = oracle.rope_rotate(x, pos, base)
    assert np.allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), atol=1e-12)
    assert np.abs(oracle.rope_rotate(y, pos, base, inverse=True) - x).max() < 1e-12
    assert np.array_equal(oracle.rope_rotate(x, np.zeros(30, np.int32), base), x)   # position 0: identity
    assert np.abs(y - x).max() > 0.1
