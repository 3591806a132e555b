"""A bounded device-side wait that runs out is reported, and the context and the device stay usable.

The failure is made in the one safe form: the test hook gives the waits a short poll limit and keeps the
source-tile producer from issuing any copy, so the consumers' waits run out by themselves, every block tears down
(tensor memory freed) and the kernel returns.  Nothing faults, traps or spins without a limit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_00891_b200 import binding as cb
from paper_2609_00891_b200 import synth
from util import bits, rel_fro

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture
def hooks():
    yield
    cb.cb_test_hooks(0, False)          # whatever happens, later tests run with the defaults


def _chunk(name):
    wl = synth.workload(name)
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    ch = synth.make_chunk(wl, 0, sl, sh)
    t = {k: v.to(DEV) for k, v in ch.items() if torch.is_tensor(v)}
    return wl, sl, sh, ch, t


def test_starved_accumulate_reports_timeout_and_context_recovers(hooks):
    wl, sl, sh, ch, t = _chunk("mini_scaled")
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh)
    ctx = cb.cb_create(prob, device=DEV)
    cb.cb_device_status(ctx)                                     # clean to begin with
    cb.cb_test_hooks(1 << 12, True)
    cb.cb_stats_accumulate(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"])
    with pytest.raises(cb.CbError) as e:
        cb.cb_device_status(ctx)
    assert e.value.status == cb.CB_ERR_TIMEOUT
    cb.cb_test_hooks(0, False)
    # the same context after a reset: an ordinary call is correct
    cb.cb_stats_reset(ctx)
    cb.cb_stats_accumulate(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"])
    p, d = wl.d + 1, wl.d
    G = torch.empty(wl.n_maps, p, p, device=DEV)
    C = torch.empty(wl.n_maps, p, d, device=DEV)
    n = cb.cb_stats_reduce(ctx, G, C)
    cb.cb_device_status(ctx)
    Go, Co = oracle.stats_traces(bits(ch["src_k"]), bits(ch["src_v"]), bits(ch["tgt_k"]), bits(ch["tgt_v"]),
                                 ch["w_k"].numpy(), ch["w_v"].numpy(), sl, sh)
    assert n == wl.chunk_tokens(0)
    assert rel_fro(G.cpu().numpy(), Go) <= 1e-3 and rel_fro(C.cpu().numpy(), Co) <= 1e-3


def test_starved_apply_reports_timeout_through_the_library_status_word(hooks):
    wl, sl, sh, ch, t = _chunk("mini_scaled")
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh)
    p, d, T = wl.d + 1, wl.d, wl.chunk_tokens(0)
    rng = np.random.default_rng(0)
    Theta = rng.standard_normal((wl.n_maps, p, d)) / np.sqrt(d)
    Wb = torch.from_numpy(Theta.astype(np.float32)).to(DEV)
    out_k = torch.zeros(wl.Lt, T, wl.Ht, d, device=DEV)
    out_v = torch.zeros_like(out_k)
    cb.cb_last_device_status()                                   # clean (and cleared) to begin with
    cb.cb_test_hooks(1 << 12, True)
    cb.cb_apply(prob, Wb, t["src_k"], t["src_v"], out_k, out_v)
    with pytest.raises(cb.CbError) as e:
        cb.cb_last_device_status()
    assert e.value.status == cb.CB_ERR_TIMEOUT
    cb.cb_last_device_status()                                   # reading the word cleared it
    cb.cb_test_hooks(0, False)
    cb.cb_apply(prob, Wb, t["src_k"], t["src_v"], out_k, out_v)
    cb.cb_last_device_status()
    (ok, ov), _ = oracle.apply_maps(bits(ch["src_k"]), bits(ch["src_v"]), Wb.cpu().numpy().astype(np.float64),
                                    wl.Lt, wl.Ht, sl, sh, want_bf16=False)
    assert rel_fro(out_k.cpu().numpy(), ok) <= 1e-5 and rel_fro(out_v.cpu().numpy(), ov) <= 1e-5
