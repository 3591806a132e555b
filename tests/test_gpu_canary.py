"""No entry point writes outside the buffers it is given.

Every output and workspace of a call is carved out of a larger allocation whose bytes before and after the buffer
hold a known pattern; after the call (results checked elsewhere) the pattern must be intact.  Token counts are
ragged on purpose (not a multiple of the 128-token tile), so the clipped tails of the tile stores are covered.
This stands in for a memory checker, which cannot be run on the machines these tests run on."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_00891_b200 import binding as cb
from paper_2609_00891_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"
GUARD = 4096          # bytes on either side; a multiple of every alignment the library asks for
PATTERN = 0xA5


class Guarded:
    """A tensor with guard bytes around it."""

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        self.nbytes = n
        self.pad = (-n) % 256
        self.raw = torch.full((GUARD + n + self.pad + GUARD,), PATTERN, dtype=torch.uint8, device=DEV)
        self.t = self.raw[GUARD:GUARD + n].view(dtype).reshape(shape)
        if fill is not None:
            self.t.fill_(fill)

    def intact(self):
        torch.cuda.synchronize()
        head = self.raw[:GUARD]
        tail = self.raw[GUARD + self.nbytes:]
        return bool((head == PATTERN).all().item()) and bool((tail == PATTERN).all().item())


def _chunk(name, c=0):
    wl = synth.workload(name)
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    ch = synth.make_chunk(wl, c, sl, sh)
    t = {k: v.to(DEV) for k, v in ch.items() if torch.is_tensor(v)}
    return wl, sl, sh, ch, t


def _ragged(t, n):
    """The first n tokens of a chunk (contiguous copies)."""
    out = {}
    for k in ("src_k", "src_v", "tgt_k", "tgt_v"):
        out[k] = t[k][:, :n].contiguous()
    for k in ("w_k", "w_v"):
        out[k] = t[k][:, :, :n].contiguous()
    return out


@pytest.mark.parametrize("name,n_tok", [("mini_scaled", 0), ("mini_scaled", 333), ("tiny", 77), ("mid_scaled", 1000)])
def test_build_and_apply_stay_inside_their_buffers(name, n_tok):
    wl, sl, sh, ch, t = _chunk(name)
    n = n_tok or ch["n_tokens"]
    n = min(n, ch["n_tokens"])
    t = _ragged(t, n)
    d, p, nm = wl.d, wl.d + 1, wl.n_maps
    prob = cb.Problem(wl.Ls, wl.Hs, d, wl.Lt, wl.Ht, d, sl, sh)
    ws = Guarded((cb.cb_workspace_bytes(prob),), torch.uint8)
    ctx = cb.cb_create(prob, workspace=ws.t)
    cb.cb_stats_reset(ctx)
    cb.cb_stats_accumulate(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"])
    G, C = Guarded((nm, p, p), torch.float32, float("nan")), Guarded((nm, p, d), torch.float32, float("nan"))
    got = cb.cb_stats_reduce(ctx, G.t, C.t)
    cb.cb_device_status(ctx)
    assert got == n
    lams = [1e-3, 1e-1]
    Wb = Guarded((len(lams), nm, p, d), torch.float32, float("nan"))
    info = Guarded((len(lams), nm), torch.int32, -1)
    cb.cb_ridge_solve(G.t, C.t, n, lams, 0, Wb.t, info.t)
    assert ws.intact() and G.intact() and C.intact() and Wb.intact() and info.intact()
    assert torch.isfinite(G.t).all() and torch.isfinite(Wb.t).all()
    # apply: bf16 (tile stores, clipped tail) and fp32 (direct stores), with and without the rotary boundary
    pos = torch.arange(n, dtype=torch.int32, device=DEV)
    for dt in (torch.bfloat16, torch.float32):
        ok, ov = Guarded((wl.Lt, n, wl.Ht, d), dt, 0), Guarded((wl.Lt, n, wl.Ht, d), dt, 0)
        cb.cb_apply(prob, Wb.t[0], t["src_k"], t["src_v"], ok.t, ov.t)
        cb.cb_last_device_status()
        assert ok.intact() and ov.intact()
        ok2, ov2 = Guarded((wl.Lt, n, wl.Ht, d), dt, 0), Guarded((wl.Lt, n, wl.Ht, d), dt, 0)
        cb.cb_apply_rope(prob, Wb.t[0], t["src_k"], t["src_v"], ok2.t, ov2.t, pos, 1e4, 1e6)
        cb.cb_last_device_status()
        assert ok2.intact() and ov2.intact()
        assert torch.equal(ov.t, ov2.t)                  # value maps do not see the boundary
    # the static entry point
    Gs, Cs = Guarded((nm, p, p), torch.float32, float("nan")), Guarded((nm, p, d), torch.float32, float("nan"))
    try:
        cb.cb_stats_build_static(prob, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"], Gs.t, Cs.t)
    except cb.CbError as e:                              # shapes beyond its fixed scratch are refused, not overrun
        assert e.status == cb.CB_ERR_UNSUPPORTED
    else:
        cb.cb_last_device_status()
        assert Gs.intact() and Cs.intact() and torch.isfinite(Gs.t).all()


def test_two_pass_and_rope_stay_inside_their_buffers():
    wl, sl, sh, ch, t = _chunk("mini_scaled")
    n = 351
    assert n < ch["n_tokens"]
    t = _ragged(t, n)
    d, nm = wl.d, wl.n_maps
    prob = cb.Problem(wl.Ls, wl.Hs, d, wl.Lt, wl.Ht, d, sl, sh)
    ws = Guarded((cb.cb_workspace_bytes(prob),), torch.uint8)
    mws = Guarded((cb.cb_means_workspace_bytes(prob),), torch.uint8)
    ctx = cb.cb_create(prob, workspace=ws.t)
    pos = (torch.arange(n, dtype=torch.int32, device=DEV) % 150)
    mu = Guarded((nm, 2 * d + 1), torch.float32, float("nan"))
    A, B = Guarded((nm, d, d), torch.float32, float("nan")), Guarded((nm, d, d), torch.float32, float("nan"))
    Wb = Guarded((1, nm, d + 1, d), torch.float32, float("nan"))
    info = Guarded((1, nm), torch.int32, -1)
    syy = Guarded((nm, d), torch.float32, float("nan"))
    for rope in (False, True):
        if rope and d != 128:
            continue
        cb.cb_means_reset(ctx, mws.t)
        cb.cb_stats_reset(ctx)
        if rope:
            cb.cb_means_accumulate_rope(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"], mws.t, pos, 1e6, 1e6)
        else:
            cb.cb_means_accumulate(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"], mws.t)
        cb.cb_means_finalize(ctx, mws.t, mu.t)
        cb.cb_means_energy(ctx, mws.t, syy.t)
        if rope:
            cb.cb_stats_accumulate_centered_rope(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"], mu.t, pos, 1e6, 1e6)
        else:
            cb.cb_stats_accumulate_centered(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"], mu.t)
        got = cb.cb_stats_reduce_centered(ctx, mu.t, A.t, B.t)
        cb.cb_ridge_solve_centered(A.t, B.t, mu.t, got, [1e-2], 0, Wb.t, info.t)
        cb.cb_device_status(ctx)
        assert got == n
        for g in (ws, mws, mu, A, B, Wb, info, syy):
            assert g.intact()
        assert torch.isfinite(Wb.t).all()
    # one-pass accumulate with the boundary, and the in-place rotation of a cache
    cb.cb_stats_reset(ctx)
    cb.cb_stats_accumulate_rope(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"], pos, 1e6, 1e4)
    cb.cb_device_status(ctx)
    K = Guarded(tuple(t["src_k"].shape), torch.bfloat16)
    K.t.copy_(t["src_k"])
    cb.cb_rope_rotate(K.t, pos, 1e6, True)
    assert ws.intact() and K.intact()
    # ESS shrinkage of a weight table
    r = torch.rand(wl.Lt, wl.Ht, n, device=DEV) + 0.01
    w = Guarded((wl.Lt, wl.Ht, n), torch.float32, float("nan"))
    cb.cb_ess_weights(r, d + 1, w.t)
    assert w.intact() and torch.isfinite(w.t).all()


@pytest.mark.parametrize("name,k,n_tok", [("mini_ragged", 3, 0), ("deep_small", 8, 517)])
def test_wide_paths_stay_inside_their_buffers(name, k, n_tok):
    wl, sl, sh, ch, t = _chunk(name)
    n = min(n_tok or ch["n_tokens"], ch["n_tokens"])
    t = _ragged(t, n)
    d, nm = wl.d, wl.n_maps
    sets = oracle.fullhead_layer_sets(wl.Ls, wl.Lt, k)
    prob = cb.FullHeadProblem(wl.Ls, wl.Hs, d, wl.Lt, wl.Ht, d, sets)
    P = k * d + 1
    G, C = Guarded((nm, P, P), torch.float32, 0), Guarded((nm, P, d), torch.float32, 0)
    cb.cb_multilayer_stats_accumulate(prob, sh, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"], G.t, C.t)
    ws = Guarded((cb.cb_ridge_solve_large_workspace_bytes(P, d, 3),), torch.uint8)
    Wb = Guarded((1, nm, P, d), torch.float32, float("nan"))
    info = Guarded((1, nm), torch.int32, -1)
    cb.cb_ridge_solve_large(G.t, C.t, n, [1e-1], 0, Wb.t, info.t, ws.t)
    cb.cb_last_device_status()
    assert G.intact() and C.intact() and ws.intact() and Wb.intact() and info.intact()
    assert torch.isfinite(Wb.t).all()
    for dt in (torch.bfloat16, torch.float32):
        ok, ov = Guarded((wl.Lt, n, wl.Ht, d), dt, 0), Guarded((wl.Lt, n, wl.Ht, d), dt, 0)
        cb.cb_apply_multilayer(prob, sh, Wb.t[0], t["src_k"], t["src_v"], ok.t, ov.t)
        cb.cb_last_device_status()
        assert ok.intact() and ov.intact()
    # full-head contrast statistics: weights per (layer, token)
    fprob = cb.FullHeadProblem(wl.Ls, wl.Hs, d, wl.Lt, wl.Ht, d, oracle.fullhead_layer_sets(wl.Ls, wl.Lt, min(4, wl.Ls)))
    Gf = Guarded((2, wl.Lt, fprob.pf, fprob.pf), torch.float32, 0)
    Cf = Guarded((2, wl.Lt, wl.Ht, fprob.pf, d), torch.float32, 0)
    fws = Guarded((cb.cb_fullhead_workspace_bytes(fprob),), torch.uint8)
    wk = t["w_k"][:, 0].contiguous()
    wv = t["w_v"][:, 0].contiguous()
    cb.cb_fullhead_stats_accumulate(fprob, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], wk, wv, Gf.t, Cf.t, fws.t)
    cb.cb_last_device_status()
    assert Gf.intact() and Cf.intact() and fws.intact()
    assert torch.isfinite(Gf.t).all() and torch.isfinite(Cf.t).all()
