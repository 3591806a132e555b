"""Full-size check in the launch configuration the benchmark times: one 50-sequence chunk of the
14B->32B-shaped build (40 -> 64 layers, 8 KV heads x 128, 51,200 tokens, 1024 maps, plain bf16 fold) on the
tensor-core kernel, compared with the oracle on 64 sampled maps (target layers 0, 1, 2, 63: first, last,
and a pair that shares one source layer; all heads; K and V)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_00891_b200 import binding as cb
from paper_2609_00891_b200 import synth
from util import bits, rel_fro, max_rel_fro_per_map

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_full_size_chunk_sampled_maps():
    wl = synth.workload("qwen14b_32b_500")
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    assert np.array_equal(sl, oracle.head_map(wl.Ls, wl.Hs, wl.Lt, wl.Ht)[0])
    ch = synth.make_chunk(wl, 0, sl, sh, device=DEV)
    T = ch["n_tokens"]
    assert T == 51200
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh)
    ctx = cb.cb_create(prob, device=DEV)
    cb.cb_stats_accumulate(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"])
    p, d = wl.d + 1, wl.d
    G = torch.empty(wl.n_maps, p, p, device=DEV)
    C = torch.empty(wl.n_maps, p, d, device=DEV)
    n = cb.cb_stats_reduce(ctx, G, C)
    cb.cb_device_status(ctx)
    assert n == T
    lams = list(wl.lambdas)
    Wb = torch.empty(len(lams), wl.n_maps, p, d, device=DEV)
    info = torch.empty(len(lams), wl.n_maps, dtype=torch.int32, device=DEV)
    cb.cb_ridge_solve(G, C, n, lams, 0, Wb, info)
    cb.cb_check_info(info)

    # properties that hold for every map at any size
    Gc = G.cpu().numpy()
    assert np.isfinite(Gc).all() and np.array_equal(Gc, Gc.transpose(0, 2, 1))
    sw = torch.stack([ch["w_k"].double().sum(-1), ch["w_v"].double().sum(-1)]).reshape(-1).cpu().numpy()
    np.testing.assert_allclose(Gc[:, d, d], sw, rtol=1e-5)                  # G[d][d] = sum of weights
    assert (np.einsum("mii->mi", Gc) > 0).all()

    # sampled maps against the oracle: a reduced problem holding only the sampled layers
    layers = [0, 1, 2, 63]
    assert sl[1] == sl[2]                                                   # a double-matched source layer
    src_layers = sorted(set(int(sl[l]) for l in layers))
    remap = np.array([src_layers.index(int(sl[l])) for l in layers], np.int32)
    sub = {}
    for k in ("src_k", "src_v"):
        sub[k] = bits(ch[k][src_layers].cpu())
    for k in ("tgt_k", "tgt_v"):
        sub[k] = bits(ch[k][layers].cpu())
    wk = ch["w_k"][layers].cpu().numpy()
    wv = ch["w_v"][layers].cpu().numpy()
    Go, Co = oracle.stats_traces(sub["src_k"], sub["src_v"], sub["tgt_k"], sub["tgt_v"], wk, wv, remap, sh)
    idx = [(comp * wl.Lt + l) * wl.Ht + h for comp in range(2) for l in layers for h in range(wl.Ht)]
    Gs, Cs = Gc[idx], C.cpu().numpy()[idx]
    eg, ec = max_rel_fro_per_map(Gs, Go), max_rel_fro_per_map(Cs, Co)
    print("full-size chunk, 64 sampled maps: max rel err G %.2e C %.2e" % (eg, ec))
    assert eg <= 1e-3 and ec <= 1e-3
    for li, lam in enumerate(lams):
        To, io = oracle.ridge_solve(Go, Co, T, lam)
        ew = max_rel_fro_per_map(Wb[li].cpu().numpy()[idx], To)
        print("lambda %g: max rel err of fitted maps %.2e" % (lam, ew))
        assert not io.any() and ew <= 1e-3
