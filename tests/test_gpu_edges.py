"""Degenerate calls and stream semantics of the C-ABI entry points on the GPU.

* A call with zero tokens is a no-op that succeeds: statistics stay as they were, outputs are not touched.
* Every call runs on the stream it is given and nowhere else: a build and an apply issued on a side stream while the
  default stream is kept busy give bitwise the results of the same calls on the default stream."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_00891_b200 import binding as cb
from paper_2609_00891_b200 import synth
from util import bits

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _chunk(name, c=0):
    wl = synth.workload(name)
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    ch = synth.make_chunk(wl, c, sl, sh)
    t = {k: v.to(DEV) for k, v in ch.items() if torch.is_tensor(v)}
    return wl, sl, sh, ch, t


def _empty_like_chunk(t):
    e = {}
    for k in ("src_k", "src_v", "tgt_k", "tgt_v"):
        e[k] = t[k][:, :0].contiguous()
    for k in ("w_k", "w_v"):
        e[k] = t[k][:, :, :0].contiguous()
    return e


@pytest.mark.parametrize("name", ["mini_scaled", "tiny"])
def test_zero_token_calls_are_no_ops(name):
    wl, sl, sh, ch, t = _chunk(name)
    e = _empty_like_chunk(t)
    d, p, nm = wl.d, wl.d + 1, wl.n_maps
    prob = cb.Problem(wl.Ls, wl.Hs, d, wl.Lt, wl.Ht, d, sl, sh)
    ctx = cb.cb_create(prob, device=DEV)
    pos0 = torch.zeros(0, dtype=torch.int32, device=DEV)

    def stats():
        G = torch.empty(nm, p, p, device=DEV)
        C = torch.empty(nm, p, d, device=DEV)
        n = cb.cb_stats_reduce(ctx, G, C)
        return n, G, C

    cb.cb_stats_accumulate(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"])
    n0, G0, C0 = stats()
    cb.cb_stats_accumulate(ctx, e["src_k"], e["src_v"], e["tgt_k"], e["tgt_v"], e["w_k"], e["w_v"])
    cb.cb_stats_accumulate_rope(ctx, e["src_k"], e["src_v"], e["tgt_k"], e["tgt_v"], e["w_k"], e["w_v"], pos0, 1e6, 1e6)
    n1, G1, C1 = stats()
    cb.cb_device_status(ctx)
    assert n0 == n1 == ch["n_tokens"] and torch.equal(G0, G1) and torch.equal(C0, C1)
    # means pass and apply with no tokens
    mws = torch.empty(cb.cb_means_workspace_bytes(prob), dtype=torch.uint8, device=DEV)
    cb.cb_means_reset(ctx, mws)
    cb.cb_means_accumulate(ctx, e["src_k"], e["src_v"], e["tgt_k"], e["tgt_v"], e["w_k"], e["w_v"], mws)
    mu = torch.full((nm, 2 * d + 1), float("nan"), device=DEV)
    cb.cb_means_finalize(ctx, mws, mu)
    assert torch.equal(mu, torch.zeros_like(mu))                    # no weight: zero means, s_w = 0
    Wb = torch.randn(nm, p, d, device=DEV)
    for dt in (torch.bfloat16, torch.float32):
        ok = torch.empty(wl.Lt, 0, wl.Ht, d, dtype=dt, device=DEV)
        ov = torch.empty_like(ok)
        cb.cb_apply(prob, Wb, e["src_k"], e["src_v"], ok, ov)
        cb.cb_apply_rope(prob, Wb, e["src_k"], e["src_v"], ok, ov, pos0, 1e6, 1e6)
    cb.cb_last_device_status()
    # a solve of statistics without rows reports every system as degenerate and zero-fills, nothing else
    cb.cb_stats_reset(ctx)
    n2, G2, C2 = stats()
    assert n2 == 0 and not G2.any() and not C2.any()
    W2 = torch.full((1, nm, p, d), float("nan"), device=DEV)
    info = torch.full((1, nm), -7, dtype=torch.int32, device=DEV)
    cb.cb_ridge_solve(G2, C2, 0, [1e-2], 0, W2, info)
    assert (info != 0).all() and not W2.any()
    with pytest.raises(cb.CbError) as err:
        cb.cb_check_info(info)
    assert err.value.status == cb.CB_ERR_NOT_PD


def test_calls_run_on_the_stream_they_are_given():
    wl, sl, sh, ch, t = _chunk("mid_scaled")
    d, p, nm = wl.d, wl.d + 1, wl.n_maps
    prob = cb.Problem(wl.Ls, wl.Hs, d, wl.Lt, wl.Ht, d, sl, sh)
    n = ch["n_tokens"]

    def build_and_apply(stream, before=None):
        ctx = cb.cb_create(prob, device=DEV)
        G = torch.full((nm, p, p), float("nan"), device=DEV)
        C = torch.full((nm, p, d), float("nan"), device=DEV)
        Wb = torch.full((1, nm, p, d), float("nan"), device=DEV)
        info = torch.full((1, nm), -1, dtype=torch.int32, device=DEV)
        ok = torch.zeros(wl.Lt, n, wl.Ht, d, dtype=torch.bfloat16, device=DEV)
        ov = torch.zeros_like(ok)
        torch.cuda.synchronize()
        if before is not None:
            before()
        cb.cb_stats_reset(ctx, stream=stream)
        cb.cb_stats_accumulate(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"], stream=stream)
        got = cb.cb_stats_reduce(ctx, G, C, stream=stream)
        cb.cb_ridge_solve(G, C, got, [1e-2], 0, Wb, info, stream=stream)
        cb.cb_apply(prob, Wb[0], t["src_k"], t["src_v"], ok, ov, stream=stream)
        cb.cb_device_status(ctx, stream=stream)
        cb.cb_last_device_status(stream=stream)
        stream.synchronize()
        return G.clone(), C.clone(), Wb.clone(), ok.clone(), ov.clone()

    ref = build_and_apply(torch.cuda.current_stream())
    side = torch.cuda.Stream()
    # keep the default stream busy for a while: a call that slipped onto it would be ordered behind this work
    busy = torch.empty(1 << 28, dtype=torch.float32, device=DEV)

    def keep_default_stream_busy():
        for _ in range(20):
            busy.normal_()

    out = build_and_apply(side, keep_default_stream_busy)
    torch.cuda.synchronize()
    for a_, b_ in zip(ref, out):
        assert torch.equal(a_, b_)
    Go, Co = oracle.stats_traces(bits(ch["src_k"]), bits(ch["src_v"]), bits(ch["tgt_k"]), bits(ch["tgt_v"]),
                                 ch["w_k"].numpy(), ch["w_v"].numpy(), sl, sh)
    err = np.linalg.norm(out[0].cpu().numpy() - Go) / np.linalg.norm(Go)
    assert err <= 1e-3
