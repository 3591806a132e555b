"""The benchmark's configurations at their full shapes, on the default (tensor-core, plain fold) path, checked
against the oracle on sampled maps (the oracle cannot finish the full configurations in minutes)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_00891_b200 import binding as cb
from paper_2609_00891_b200 import synth
from util import bits, rel_fro, max_rel_fro_per_map

pytestmark = pytest.mark.gpu
DEV = "cuda"
TOL = 1e-3


def _sampled_oracle(wl, sl, sh, layers, chunks_host):
    """Oracle statistics of all heads, K and V, of the sampled target layers: a reduced problem with only those layers."""
    src_layers = sorted(set(int(sl[l]) for l in layers))
    remap = np.array([src_layers.index(int(sl[l])) for l in layers], np.int32)
    G = C = None
    for ch in chunks_host:
        g, c = oracle.stats_traces(bits(ch["src_k"][src_layers]), bits(ch["src_v"][src_layers]),
                                   bits(ch["tgt_k"][layers]), bits(ch["tgt_v"][layers]),
                                   ch["w_k"][layers].numpy(), ch["w_v"][layers].numpy(), remap, sh)
        G, C = (g, c) if G is None else (G + g, C + c)
    idx = [(comp * wl.Lt + l) * wl.Ht + h for comp in range(2) for l in layers for h in range(wl.Ht)]
    return G, C, idx


def _run_config(name, layers, max_chunks=None):
    wl = synth.workload(name)
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh)
    ctx = cb.cb_create(prob, device=DEV)
    law = synth.map_law(wl, DEV)
    src_layers = sorted(set(int(sl[l]) for l in layers))
    n_chunks = wl.n_chunks if max_chunks is None else min(max_chunks, wl.n_chunks)
    host, n_tok = [], 0
    for c in range(n_chunks):
        ch = synth.make_chunk(wl, c, sl, sh, device=DEV, law=law)
        cb.cb_stats_accumulate(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"])
        # host copy of the sampled layers only
        host.append({
            "src_k": _dense_layers(ch["src_k"], src_layers, wl.Ls), "src_v": _dense_layers(ch["src_v"], src_layers, wl.Ls),
            "tgt_k": _dense_layers(ch["tgt_k"], layers, wl.Lt), "tgt_v": _dense_layers(ch["tgt_v"], layers, wl.Lt),
            "w_k": _dense_layers(ch["w_k"], layers, wl.Lt), "w_v": _dense_layers(ch["w_v"], layers, wl.Lt)})
        n_tok += ch["n_tokens"]
        del ch
    p, d = wl.d + 1, wl.d
    G = torch.empty(wl.n_maps, p, p, device=DEV)
    C = torch.empty(wl.n_maps, p, d, device=DEV)
    n = cb.cb_stats_reduce(ctx, G, C)
    cb.cb_device_status(ctx)
    assert n == n_tok
    return wl, sl, sh, prob, G, C, n, host


def _dense_layers(t, keep, L):
    """Host copy of the kept layers only, still addressable by the original layer index."""
    return _Compact(t, keep)


class _Compact:
    """Only the kept layers, addressable by their original layer index (for tensors too large to hold densely)."""

    def __init__(self, t, keep):
        self.keep = list(keep)
        self.data = torch.stack([t[j].cpu() for j in self.keep])

    def __getitem__(self, layers):
        return self.data[[self.keep.index(int(j)) for j in layers]]


@pytest.mark.parametrize("name,layers,max_chunks", [
    ("qwen8b_14b", [0, 4, 5, 39], None),               # config 1 in full: 36 -> 40 layers, 64 x 1024 tokens; layers 4, 5 share a source layer
    ("ragged_long", [0, 1, 2, 63], 2),                 # config 4, first two ragged chunks of 12 sequences
])
def test_config_statistics_and_fit_on_sampled_maps(name, layers, max_chunks):
    wl, sl, sh, prob, G, C, n, host = _run_config(name, layers, max_chunks)
    if name == "qwen8b_14b":
        assert sl[4] == sl[5]
    Go, Co, idx = _sampled_oracle(wl, sl, sh, layers, host)
    Gs, Cs = G.cpu().numpy()[idx], C.cpu().numpy()[idx]
    eg, ec = max_rel_fro_per_map(Gs, Go), max_rel_fro_per_map(Cs, Co)
    print("%s (%d tokens): %d sampled maps, max rel err G %.2e C %.2e" % (name, n, len(idx), eg, ec))
    assert eg <= TOL and ec <= TOL
    p, d = wl.d + 1, wl.d
    lams = list(wl.lambdas)
    Wb = torch.empty(len(lams), wl.n_maps, p, d, device=DEV)
    info = torch.empty(len(lams), wl.n_maps, dtype=torch.int32, device=DEV)
    cb.cb_ridge_solve(G, C, n, lams, 0, Wb, info)
    cb.cb_check_info(info)
    To, io = oracle.ridge_solve(Go, Co, n, lams[0])
    ew = max_rel_fro_per_map(Wb[0].cpu().numpy()[idx], To)
    print("fitted maps: max rel err %.2e" % ew)
    assert not io.any() and ew <= TOL
    if wl.apply_tokens:
        # online apply of the fitted maps to a long source cache; oracle on the sampled maps with the GPU's maps
        T = wl.apply_tokens
        src = synth.make_source_cache(wl, T, DEV, synth.map_law(wl, DEV))
        out_k = torch.empty(wl.Lt, T, wl.Ht, d, dtype=torch.bfloat16, device=DEV)
        out_v = torch.empty_like(out_k)
        cb.cb_apply(prob, Wb[0], src[0], src[1], out_k, out_v)
        torch.cuda.synchronize()
        src_layers = sorted(set(int(sl[l]) for l in layers))
        remap = np.array([src_layers.index(int(sl[l])) for l in layers], np.int32)
        Th = np.zeros((2 * len(layers) * wl.Ht, p, d))
        Th[:] = To                                                   # oracle's maps for the sampled (reduced) problem
        (ok, ov), (bk, bv) = oracle.apply_maps(bits(src[0][src_layers].cpu()), bits(src[1][src_layers].cpu()), Th,
                                               len(layers), wl.Ht, remap, sh)
        gk = out_k[layers].float().cpu().numpy()
        gv = out_v[layers].float().cpu().numpy()
        ek, ev = rel_fro(gk, oracle.bf16_decode(bk)), rel_fro(gv, oracle.bf16_decode(bv))
        print("mapped %d-token cache (bf16) vs oracle rounded the same way: K %.2e V %.2e" % (T, ek, ev))
        assert ek <= 2e-3 and ev <= 2e-3                             # bf16 grid: one-ulp flips only
        assert rel_fro(gk, ok) <= 3e-3                               # vs unrounded fp64: the bf16 floor (~1.7e-3)


def test_config3_fullhead_sampled_group():
    """Config 3 shapes (4 source layers x 8 heads -> 4097-wide regressor), first 2,048 tokens, one (comp, layer) group
    against the oracle (the full group costs the oracle 70 GFLOP of plain fp64)."""
    wl = synth.workload("qwen14b_32b_500")
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    sets = cb.cb_fullhead_layer_sets(wl.Ls, wl.Lt, 4)
    assert np.array_equal(sets, oracle.fullhead_layer_sets(wl.Ls, wl.Lt, 4))
    import dataclasses
    small = dataclasses.replace(wl, seq_lens=(1024, 1024), seqs_per_chunk=2)
    ch = synth.make_chunk(small, 0, sl, sh, device=DEV)
    prob = cb.FullHeadProblem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sets)
    pf, d = prob.pf, wl.d
    assert pf == 4097
    G = torch.zeros(2, wl.Lt, pf, pf, device=DEV)
    C = torch.zeros(2, wl.Lt, wl.Ht, pf, d, device=DEV)
    wk, wv = ch["w_k"][:, 0].contiguous(), ch["w_v"][:, 0].contiguous()
    cb.cb_fullhead_stats_accumulate(prob, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], wk, wv, G, C)
    torch.cuda.synchronize()
    comp, l = 1, 17
    Go, Co = oracle.fullhead_stats(bits(ch["src_v"].cpu()), bits(ch["tgt_v"].cpu()), wv[l].cpu().numpy(), l, sets[l])
    eg, ec = rel_fro(G[comp, l].cpu().numpy(), Go), rel_fro(C[comp, l].cpu().numpy(), Co)
    print("config 3, (V, layer 17), 2048 tokens: rel err G %.2e C %.2e" % (eg, ec))
    assert eg <= 2e-3 and ec <= 2e-3                                   # 2,048 tokens per entry: the plain bf16 fold averages out like 1/sqrt(tokens)
    assert torch.isfinite(G).all() and torch.isfinite(C).all()
    # every other group must have been filled too (property check): the weight totals
    sw = torch.stack([wk.double().sum(-1), wv.double().sum(-1)]).cpu().numpy()
    np.testing.assert_allclose(G[:, :, pf - 1, pf - 1].cpu().numpy(), sw, rtol=1e-5)
