"""Parity of the two-pass centred construction (Section 3.4) against the fp64 oracle, through the C ABI.

Tolerance: relative Frobenius error <= 1e-3 on the centred statistics A, B and on the maps; means to fp32 accuracy."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_00891_b200 import binding as cb
from paper_2609_00891_b200 import synth
from util import bits, rel_fro, max_rel_fro_per_map

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _chunks(wl, sl, sh):
    law = synth.map_law(wl)
    return [synth.make_chunk(wl, c, sl, sh, law=law) for c in range(wl.n_chunks)]


def _shift(chunks, dx, dy):
    """Channel means far from zero: add constants and round back to bf16 (what a real trace would hold)."""
    out = []
    for ch in chunks:
        c = dict(ch)
        for k in ("src_k", "src_v"):
            c[k] = (ch[k].float() + dx).to(torch.bfloat16)
        for k in ("tgt_k", "tgt_v"):
            c[k] = (ch[k].float() + dy).to(torch.bfloat16)
        out.append(c)
    return out


def _oracle_twopass(chunks, sl, sh, maps=None):
    args = lambda ch: (bits(ch["src_k"]), bits(ch["src_v"]), bits(ch["tgt_k"]), bits(ch["tgt_v"]),
                       ch["w_k"].numpy(), ch["w_v"].numpy(), sl, sh)
    sx = sy = sw = None
    for ch in chunks:
        a, b, c = oracle.weighted_sums_traces(*args(ch), maps=maps)
        sx, sy, sw = (a, b, c) if sx is None else (sx + a, sy + b, sw + c)
    mu_x, mu_y = sx / sw[:, None], sy / sw[:, None]
    A = B = None
    for ch in chunks:
        a, b = oracle.centered_stats_traces(*args(ch), mu_x, mu_y, maps=maps)
        A, B = (a, b) if A is None else (A + a, B + b)
    return mu_x, mu_y, sw, A, B


def _gpu_twopass(wl, chunks, sl, sh, flags=0, n_splits=0):
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh, flags=flags, n_splits=n_splits)
    ctx = cb.cb_create(prob, device=DEV)
    dev = [{k: v.to(DEV) for k, v in ch.items() if torch.is_tensor(v)} for ch in chunks]
    ws = torch.empty(cb.cb_means_workspace_bytes(prob), dtype=torch.uint8, device=DEV)
    cb.cb_means_reset(ctx, ws)
    for t in dev:
        cb.cb_means_accumulate(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"], ws)
    d = wl.d
    mu = torch.full((wl.n_maps, 2 * d + 1), float("nan"), device=DEV)
    cb.cb_means_finalize(ctx, ws, mu)
    cb.cb_stats_reset(ctx)
    for t in dev:
        cb.cb_stats_accumulate_centered(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"], mu)
    A = torch.full((wl.n_maps, d, d), float("nan"), device=DEV)
    B = torch.full((wl.n_maps, d, d), float("nan"), device=DEV)
    n = cb.cb_stats_reduce_centered(ctx, mu, A, B)
    cb.cb_device_status(ctx)
    return prob, ctx, mu, A, B, n


def _solve(A, B, mu, n, lams, flags=0):
    n_maps, d, _ = A.shape
    Wb = torch.full((len(lams), n_maps, d + 1, d), float("nan"), device=DEV)
    info = torch.full((len(lams), n_maps), -1, dtype=torch.int32, device=DEV)
    cb.cb_ridge_solve_centered(A, B, mu, n, lams, flags, Wb, info)
    cb.cb_check_info(info)
    return Wb


CASES = [("tiny", cb.CB_FLAG_COMPENSATED, 0), ("tiny", 0, 3), ("mini_scaled", 0, 0), ("mini_ragged", cb.CB_FLAG_COMPENSATED, 7),
         ("mini_ragged", 0, 0), ("mid_scaled", 0, 0), ("long_unit", 0, 1), ("long_unit", cb.CB_FLAG_COMPENSATED, 1)]


@pytest.mark.parametrize("name,flags,n_splits", CASES)
def test_two_pass_matches_oracle(name, flags, n_splits):
    wl = synth.workload(name)
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    chunks = _chunks(wl, sl, sh)
    mu_x, mu_y, sw, Ao, Bo = _oracle_twopass(chunks, sl, sh)
    prob, ctx, mu, A, B, n = _gpu_twopass(wl, chunks, sl, sh, flags, n_splits)
    assert n == wl.n_tokens
    d = wl.d
    muc, Ac, Bc = mu.cpu().numpy().astype(np.float64), A.cpu().numpy(), B.cpu().numpy()
    scale = np.abs(np.concatenate([mu_x, mu_y], axis=1)).max() + 1.0
    assert np.abs(muc[:, :d] - mu_x).max() <= 2e-6 * scale and np.abs(muc[:, d:2 * d] - mu_y).max() <= 2e-6 * scale
    assert np.allclose(muc[:, 2 * d], sw, rtol=1e-6)
    tol = 1e-3                      # calls of fewer than 4,096 rows take the hi + lo fold by themselves
    print("%s flags=%d: A %.2e (max map %.2e)  B %.2e (max map %.2e)" % (
        name, flags, rel_fro(Ac, Ao), max_rel_fro_per_map(Ac, Ao), rel_fro(Bc, Bo), max_rel_fro_per_map(Bc, Bo)))
    assert np.isfinite(Ac).all() and np.isfinite(Bc).all()
    assert np.array_equal(Ac, Ac.transpose(0, 2, 1))
    assert max_rel_fro_per_map(Ac, Ao) <= tol and max_rel_fro_per_map(Bc, Bo) <= tol
    if flags & cb.CB_FLAG_COMPENSATED:
        assert rel_fro(Ac, Ao) <= 2e-5 and rel_fro(Bc, Bo) <= 2e-5
    lams = list(wl.lambdas)
    Wb = _solve(A, B, mu, n, lams).cpu().numpy()
    for i, lam in enumerate(lams):
        Th, info = oracle.ridge_solve_centered(Ao, Bo, mu_x, mu_y, sw, wl.n_tokens, lam)
        assert not info.any()
        e = rel_fro(Wb[i], Th)
        print("  lambda %g: maps rel err %.2e" % (lam, e))
        assert e <= tol
    # GPU solve alone, fed the oracle's statistics: fp64 inside, so it agrees far below the statistics' error
    Ad = torch.from_numpy(Ao.astype(np.float32)).to(DEV)
    Bd = torch.from_numpy(Bo.astype(np.float32)).to(DEV)
    mud = torch.from_numpy(np.concatenate([mu_x, mu_y, sw[:, None]], axis=1).astype(np.float32)).to(DEV)
    Th, _ = oracle.ridge_solve_centered(Ao, Bo, mu_x, mu_y, sw, wl.n_tokens, lams[0])
    assert rel_fro(_solve(Ad, Bd, mud, wl.n_tokens, lams[:1]).cpu().numpy()[0], Th) <= 2e-5


def test_same_maps_as_the_one_pass_path():
    wl = synth.workload("mid_scaled")
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    chunks = _chunks(wl, sl, sh)
    prob, ctx, mu, A, B, n = _gpu_twopass(wl, chunks, sl, sh)
    W2 = _solve(A, B, mu, n, [1e-2])
    p, d = wl.d + 1, wl.d
    cb.cb_stats_reset(ctx)
    for ch in chunks:
        t = {k: v.to(DEV) for k, v in ch.items() if torch.is_tensor(v)}
        cb.cb_stats_accumulate(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"])
    G = torch.empty((wl.n_maps, p, p), device=DEV)
    C = torch.empty((wl.n_maps, p, d), device=DEV)
    n1 = cb.cb_stats_reduce(ctx, G, C)
    W1 = torch.empty((1, wl.n_maps, p, d), device=DEV)
    info = torch.empty((1, wl.n_maps), dtype=torch.int32, device=DEV)
    cb.cb_ridge_solve(G, C, n1, [1e-2], 0, W1, info)
    cb.cb_check_info(info)
    assert n1 == n
    assert rel_fro(W2.cpu().numpy(), W1.cpu().numpy()) <= 2e-3


def test_large_channel_means_two_pass_stays_accurate_where_one_pass_does_not():
    wl = synth.workload("mid_scaled")
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    chunks = _shift(_chunks(wl, sl, sh), 48.0, -24.0)
    maps = np.arange(0, wl.n_maps, max(1, wl.n_maps // 16), dtype=np.int32)
    mu_x, mu_y, sw, Ao, Bo = _oracle_twopass(chunks, sl, sh, maps)
    lam = 1e-2
    Th, info = oracle.ridge_solve_centered(Ao, Bo, mu_x, mu_y, sw, wl.n_tokens, lam)
    assert not info.any()
    prob, ctx, mu, A, B, n = _gpu_twopass(wl, chunks, sl, sh)
    eA = max_rel_fro_per_map(A.cpu().numpy()[maps], Ao)
    eB = max_rel_fro_per_map(B.cpu().numpy()[maps], Bo)
    W2 = _solve(A, B, mu, n, [lam]).cpu().numpy()[0][maps]
    e2 = rel_fro(W2[:, :-1], Th[:, :-1])
    b2 = np.abs(W2[:, -1] - Th[:, -1]).max() / np.abs(Th[:, -1]).max()
    # one-pass path on the same shifted traces
    p, d = wl.d + 1, wl.d
    cb.cb_stats_reset(ctx)
    for ch in chunks:
        t = {k: v.to(DEV) for k, v in ch.items() if torch.is_tensor(v)}
        cb.cb_stats_accumulate(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"])
    G = torch.empty((wl.n_maps, p, p), device=DEV)
    C = torch.empty((wl.n_maps, p, d), device=DEV)
    n1 = cb.cb_stats_reduce(ctx, G, C)
    W1 = torch.empty((1, wl.n_maps, p, d), device=DEV)
    info1 = torch.empty((1, wl.n_maps), dtype=torch.int32, device=DEV)
    cb.cb_ridge_solve(G, C, n1, [lam], 0, W1, info1)
    W1 = W1.cpu().numpy()[0][maps]
    e1 = rel_fro(W1[:, :-1], Th[:, :-1]) if np.isfinite(W1).all() else float("inf")
    print("shifted traces: two-pass A %.2e B %.2e W %.2e b %.2e | one-pass W %.2e" % (eA, eB, e2, b2, e1))
    assert eA <= 1e-3 and eB <= 1e-3 and e2 <= 1e-3 and b2 <= 1e-3
    assert e1 > 10 * e2                                   # the reason this path exists


def test_chunked_equals_single_call_and_is_reproducible():
    wl = synth.workload("mini_ragged")
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    chunks = _chunks(wl, sl, sh)
    _, _, mu1, A1, B1, n1 = _gpu_twopass(wl, chunks, sl, sh)
    _, _, mu2, A2, B2, n2 = _gpu_twopass(wl, chunks, sl, sh)
    assert torch.equal(mu1, mu2) and torch.equal(A1, A2) and torch.equal(B1, B2) and n1 == n2
    cat = {k: torch.cat([c[k] for c in chunks], dim=1 if k[:3] in ("src", "tgt") else 2) for k in
           ("src_k", "src_v", "tgt_k", "tgt_v", "w_k", "w_v")}
    _, _, mu3, A3, B3, n3 = _gpu_twopass(wl, [cat], sl, sh)
    assert n3 == n1
    assert rel_fro(mu3.cpu().numpy(), mu1.cpu().numpy()) <= 1e-6
    assert rel_fro(A3.cpu().numpy(), A1.cpu().numpy()) <= 1e-3 and rel_fro(B3.cpu().numpy(), B1.cpu().numpy()) <= 1e-3


def test_argument_errors():
    wl = synth.workload("tiny")
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh)
    ctx = cb.cb_create(prob, device=DEV)
    short = torch.empty(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(cb.CbError) as e:
        cb.cb_means_reset(ctx, short)
    assert e.value.status == cb.CB_ERR_WORKSPACE
    simt = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh, flags=cb.CB_FLAG_SIMT)
    ctx2 = cb.cb_create(simt, device=DEV)
    ch = {k: v.to(DEV) for k, v in _chunks(wl, sl, sh)[0].items() if torch.is_tensor(v)}
    mu = torch.zeros((wl.n_maps, 2 * wl.d + 1), device=DEV)
    with pytest.raises(cb.CbError) as e:
        cb.cb_stats_accumulate_centered(ctx2, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"], mu)
    assert e.value.status == cb.CB_ERR_UNSUPPORTED


@pytest.mark.parametrize("T", [1, 65, 200])
def test_two_pass_few_rows(T):
    wl = synth.workload("mini_scaled")
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    ch = _chunks(wl, sl, sh)[0]
    cut = {k: (v[:, :T].contiguous() if k[:3] in ("src", "tgt") else v[:, :, :T].contiguous()) for k, v in ch.items() if torch.is_tensor(v)}
    mu_x, mu_y, sw, Ao, Bo = _oracle_twopass([cut], sl, sh)
    import dataclasses
    small = dataclasses.replace(wl, seq_lens=(T,), seqs_per_chunk=1)
    prob, ctx, mu, A, B, n = _gpu_twopass(small, [cut], sl, sh)
    assert n == T
    d = wl.d
    muc = mu.cpu().numpy().astype(np.float64)
    assert np.allclose(muc[:, :d], mu_x, atol=1e-5) and np.allclose(muc[:, d:2 * d], mu_y, atol=1e-5)
    Ac, Bc = A.cpu().numpy(), B.cpu().numpy()
    assert np.isfinite(Ac).all() and np.isfinite(Bc).all()
    if T == 1:
        assert np.abs(Ac).max() <= 1e-3 and np.abs(Bc).max() <= 1e-3          # one row: centred statistics vanish
    else:
        assert max_rel_fro_per_map(Ac, Ao) <= 1e-3 and max_rel_fro_per_map(Bc, Bo) <= 1e-3
