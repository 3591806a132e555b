"""The allocation-free entry point (built-in scratch buffer) against the regular context-based path.

Collected last on purpose (file name), so that a run that stops at the first failure has already run every
other test.  The entry point serves callers that cannot allocate device memory for a workspace: a server
whose pool owns all device memory, a plug-in hook that must not call cudaMalloc, a hard memory cap."""
import pytest
import torch

import oracle
from paper_2609_00891_b200 import binding as cb
from paper_2609_00891_b200 import synth
from util import bits, rel_fro

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _regular(prob, t):
    ctx = cb.cb_create(prob, device=DEV)
    cb.cb_stats_accumulate(ctx, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"])
    p, d = prob.ds + 1, prob.ds
    G = torch.empty(prob.n_maps, p, p, device=DEV)
    C = torch.empty(prob.n_maps, p, d, device=DEV)
    cb.cb_stats_reduce(ctx, G, C)
    cb.cb_device_status(ctx)
    return G, C


@pytest.mark.parametrize("name,flags", [("mini_scaled", cb.CB_FLAG_COMPENSATED), ("tiny", 0)])
def test_static_scratch_entry_matches_regular_path_twice(name, flags):
    wl = synth.workload(name)
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    law = synth.map_law(wl)
    # two different batches, one call after the other: the second must not see the first one's leftovers
    batches = [synth.make_chunk(wl, 0, sl, sh, law=law), synth.make_chunk(wl, wl.n_chunks - 1, sl, sh, law=law)]
    if wl.n_chunks == 1:
        batches[1] = {k: (v.flip(1) if k[:3] in ("src", "tgt") else (v.flip(2) * 0.5 if torch.is_tensor(v) else v))
                      for k, v in batches[0].items()}
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh, flags=flags, n_splits=2)
    p, d = wl.d + 1, wl.d
    for b in batches:
        t = {k: v.to(DEV).contiguous() for k, v in b.items() if torch.is_tensor(v)}
        G_ref, C_ref = _regular(prob, t)
        G = torch.full((wl.n_maps, p, p), float("nan"), device=DEV)
        C = torch.full((wl.n_maps, p, d), float("nan"), device=DEV)
        cb.cb_stats_build_static(prob, t["src_k"], t["src_v"], t["tgt_k"], t["tgt_v"], t["w_k"], t["w_v"], G, C)
        torch.cuda.synchronize()
        assert torch.isfinite(G).all() and torch.isfinite(C).all()
        # same kernels, same split order: agreement far inside the 1e-3 the parity tests use
        assert ((G - G_ref).norm() / G_ref.norm()).item() <= 1e-6
        assert ((C - C_ref).norm() / C_ref.norm()).item() <= 1e-6
        cb.cb_last_device_status()                     # no bounded wait ran out inside the call
    # and against the oracle itself (second batch), at the tolerance of the parity tests
    Go, Co = oracle.stats_traces(bits(b["src_k"]), bits(b["src_v"]), bits(b["tgt_k"]), bits(b["tgt_v"]),
                                 b["w_k"].contiguous().numpy(), b["w_v"].contiguous().numpy(), sl, sh)
    assert rel_fro(G.cpu().numpy(), Go) <= 1e-3 and rel_fro(C.cpu().numpy(), Co) <= 1e-3


def test_static_scratch_entry_rejects_oversized_problems():
    wl = synth.workload("qwen14b_32b_500")          # 1024 maps x 132 KB: far beyond the built-in buffer
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh)
    T = 8
    src = torch.zeros(wl.Ls, T, wl.Hs, wl.d, dtype=torch.bfloat16, device=DEV)
    tgt = torch.zeros(wl.Lt, T, wl.Ht, wl.d, dtype=torch.bfloat16, device=DEV)
    w = torch.ones(wl.Lt, wl.Ht, T, device=DEV)
    G = torch.zeros(wl.n_maps, wl.d + 1, wl.d + 1, device=DEV)
    C = torch.zeros(wl.n_maps, wl.d + 1, wl.d, device=DEV)
    before = cb.cb_launch_count()
    with pytest.raises(cb.CbError) as e:
        cb.cb_stats_build_static(prob, src, src.clone(), tgt, tgt.clone(), w, w, G, C)
    assert e.value.status == cb.CB_ERR_STATIC_LIMIT and "built-in scratch" in str(e.value)
    assert cb.cb_launch_count() == before          # nothing was enqueued
