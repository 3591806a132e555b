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


def _sampled_oracle_chunk(sl, sh, layers, ch):
    """Oracle statistics of one chunk for all heads, K and V, of the sampled target layers: a reduced problem that
    holds only those layers (and the source layers they read)."""
    src_layers = sorted(set(int(sl[l]) for l in layers))
    remap = np.array([src_layers.index(int(sl[l])) for l in layers], np.int32)
    return oracle.stats_traces(bits(ch["src_k"][src_layers].cpu()), bits(ch["src_v"][src_layers].cpu()),
                               bits(ch["tgt_k"][layers].cpu()), bits(ch["tgt_v"][layers].cpu()),
                               ch["w_k"][layers].cpu().numpy(), ch["w_v"][layers].cpu().numpy(), remap, sh)


def _run_config(name, layers, chunks=None):
    """Streams the given chunks (all by default) of a workload through one context; the oracle's statistics of the
    sampled layers are summed chunk by chunk beside it (statistics are additive), so that no chunk is kept."""
    wl = synth.workload(name)
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh)
    ctx = cb.cb_create(prob, device=DEV)
    law = synth.map_law(wl, DEV)
    chunks = list(range(wl.n_chunks)) if chunks is None else list(chunks)
    Go = Co = None
    n_tok, sizes = 0, []
    for c in chunks:
        ch = synth.make_chunk(wl, c, sl, sh, device=DEV, law=law)
        cb.cb_stats_accumulate(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"])
        g, co = _sampled_oracle_chunk(sl, sh, layers, ch)
        Go, Co = (g, co) if Go is None else (Go + g, Co + co)
        n_tok += ch["n_tokens"]
        sizes.append(ch["n_tokens"])
        del ch
    p, d = wl.d + 1, wl.d
    G = torch.empty(wl.n_maps, p, p, device=DEV)
    C = torch.empty(wl.n_maps, p, d, device=DEV)
    n = cb.cb_stats_reduce(ctx, G, C)
    cb.cb_device_status(ctx)
    assert n == n_tok
    idx = [(comp * wl.Lt + l) * wl.Ht + h for comp in range(2) for l in layers for h in range(wl.Ht)]
    return wl, sl, sh, prob, G, C, n, (Go, Co, idx), sizes


@pytest.mark.parametrize("name,layers,chunks", [
    ("qwen8b_14b", [0, 4, 5, 39], None),               # config 1 in full: 36 -> 40 layers, 64 x 1024 tokens; layers 4, 5 share a source layer
    # config 4: the first two ragged chunks of 12 sequences and the LAST one (8 sequences: the short tail); none of
    # the three ends on a multiple of the 128-token tile, so every chunk boundary falls inside a tile
    ("ragged_long", [0, 1, 2, 63], [0, 1, 41]),
])
def test_config_statistics_and_fit_on_sampled_maps(name, layers, chunks):
    wl, sl, sh, prob, G, C, n, (Go, Co, idx), sizes = _run_config(name, layers, chunks)
    if name == "qwen8b_14b":
        assert sl[4] == sl[5]
    else:
        assert wl.n_chunks == 42 and len(wl.chunk_seq_lens(41)) == 8 and all(t % 128 for t in sizes)
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


def test_config2_full_build_on_sampled_maps():
    """Config 2 as the benchmark runs it: all ten 51,200-token calls into one context, one reduce, the solve at the three
    lambdas; 64 sampled maps (target layers 0, 1, 2, 63: first, last, and a pair sharing one source layer; all heads;
    K and V) against the oracle on all 512,000 tokens."""
    layers = [0, 1, 2, 63]
    wl, sl, sh, prob, G, C, n, (Go, Co, idx), sizes = _run_config("qwen14b_32b_500", layers)
    assert n == 512000 and sizes == [51200] * 10 and sl[1] == sl[2]
    Gs, Cs = G.cpu().numpy()[idx], C.cpu().numpy()[idx]
    eg, ec = max_rel_fro_per_map(Gs, Go), max_rel_fro_per_map(Cs, Co)
    d = wl.d
    # the tensor cores' fp32 accumulation truncates: on the all-positive diagonal of G the result is systematically
    # low, in proportion to the tokens summed in tensor memory between drains (at most 16,384)
    dg = np.einsum("mii->mi", Gs)[:, :d].astype(np.float64)
    do = np.einsum("mii->mi", Go)[:, :d]
    bias = float(np.mean((dg - do) / do))
    print("config 2, 512,000 tokens, 64 sampled maps: max rel err G %.2e C %.2e; signed mean rel err of diag(G) %.2e"
          % (eg, ec, bias))
    assert eg <= TOL and ec <= TOL
    assert -2.0e-4 < bias < 0.0
    p = d + 1
    lams = list(wl.lambdas)
    Wb = torch.empty(len(lams), wl.n_maps, p, d, device=DEV)
    info = torch.empty(len(lams), wl.n_maps, dtype=torch.int32, device=DEV)
    cb.cb_ridge_solve(G, C, n, lams, 0, Wb, info)
    cb.cb_check_info(info)
    for li, lam in enumerate(lams):
        To, io = oracle.ridge_solve(Go, Co, n, lam)
        ew = max_rel_fro_per_map(Wb[li].cpu().numpy()[idx], To)
        print("lambda %g: max rel err of fitted maps %.2e" % (lam, ew))
        assert not io.any() and ew <= TOL


def test_config3_fullhead_sampled_group():
    """Config 3 shapes (4 source layers x 8 heads -> 4097-wide regressor), 32,768 tokens, one (comp, layer) group
    against the oracle (the group costs the oracle 1.4 TFLOP of plain fp64) at the stated 1e-3, pooled over the
    group, per map, and for its worst 128 x 128 block.  31 of the 32 feature heads are unrelated to a given target
    head, so C is mostly noise blocks at small sizes (measured 1.4e-3 at 8,192 tokens, falling like 1/sqrt(tokens);
    the configuration itself has 204,800)."""
    wl = synth.workload("qwen14b_32b_500")
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    sets = cb.cb_fullhead_layer_sets(wl.Ls, wl.Lt, 4)
    assert np.array_equal(sets, oracle.fullhead_layer_sets(wl.Ls, wl.Lt, 4))
    import dataclasses
    small = dataclasses.replace(wl, seq_lens=(1024,) * 32, seqs_per_chunk=32)
    ch = synth.make_chunk(small, 0, sl, sh, device=DEV)
    prob = cb.FullHeadProblem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sets)
    pf, d = prob.pf, wl.d
    assert pf == 4097
    G = torch.zeros(2, wl.Lt, pf, pf, device=DEV)
    C = torch.zeros(2, wl.Lt, wl.Ht, pf, d, device=DEV)
    wk, wv = ch["w_k"][:, 0].contiguous(), ch["w_v"][:, 0].contiguous()
    cb.cb_fullhead_stats_accumulate(prob, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], wk, wv, G, C)
    cb.cb_last_device_status()
    comp, l = 1, 17
    Go, Co = oracle.fullhead_stats(bits(ch["src_v"].cpu()), bits(ch["tgt_v"].cpu()), wv[l].cpu().numpy(), l, sets[l])
    Gg, Cg = G[comp, l].cpu().numpy(), C[comp, l].cpu().numpy()
    eg, ec = rel_fro(Gg, Go), rel_fro(Cg, Co)
    F = (pf - 1) // d
    blk_g = max(rel_fro(Gg[i * d:(i + 1) * d, j * d:(j + 1) * d], Go[i * d:(i + 1) * d, j * d:(j + 1) * d])
                for i in range(F) for j in range(F))
    blk_c = max(rel_fro(Cg[h, i * d:(i + 1) * d], Co[h, i * d:(i + 1) * d]) for h in range(wl.Ht) for i in range(F))
    print("config 3, (V, layer 17), 32768 tokens: rel err G %.2e C %.2e; worst 128 x 128 block G %.2e C %.2e"
          % (eg, ec, blk_g, blk_c))
    # A block between two unrelated heads is a sum of terms of random sign: its value and the rounding error of the
    # bf16 weighted operand (relative 2^-9 .. 2^-8 per term) both grow like sqrt(tokens), so that block's relative
    # error stays at a few 1e-3 at any size; only the blocks that carry signal (diagonal blocks of G, C of the matched
    # head) improve like 1/sqrt(tokens).  31 of the 32 blocks of a target head's C are of the first kind in these
    # traces, so C reaches 1e-3 later than G: 1.4e-3 at 8,192 tokens, 1.1e-3 here, below 1e-3 at the configuration's
    # 204,800 tokens (next test).
    assert eg <= TOL and ec <= 1.5e-3
    assert max(rel_fro(Cg[h], Co[h]) for h in range(wl.Ht)) <= 1.5e-3     # every map's own C
    assert blk_g <= 5e-3 and blk_c <= 5e-3
    assert torch.isfinite(G).all() and torch.isfinite(C).all()
    # every other group must have been filled too (property check): the weight totals
    sw = torch.stack([wk.double().sum(-1), wv.double().sum(-1)]).cpu().numpy()
    np.testing.assert_allclose(G[:, :, pf - 1, pf - 1].cpu().numpy(), sw, rtol=1e-5)


def test_config3_full_size_sampled_outputs():
    """Config 3 itself: 200 sequences x 1,024 tokens in four 51,200-token calls, all 128 (comp, layer) groups on the
    GPU.  The oracle cannot finish a 4097-wide group at this size in minutes, so sampled outputs are compared: for one
    group (V, layer 17) and one target head, the whole C (4097 x 128), and the blocks of G that couple one source head
    across the four selected layers (eight 513 x 513 pieces), each from the oracle's k = 4 head-local statistics of
    that source head, which are by definition those entries of the full-head statistics."""
    wl = synth.workload("qwen14b_32b_500")
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    sets = cb.cb_fullhead_layer_sets(wl.Ls, wl.Lt, 4)
    prob = cb.FullHeadProblem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sets)
    pf, d, k = prob.pf, wl.d, 4
    G = torch.zeros(2, wl.Lt, pf, pf, device=DEV)
    C = torch.zeros(2, wl.Lt, wl.Ht, pf, d, device=DEV)
    law = synth.map_law(wl, DEV)
    comp, l, h = 1, 17, 5
    keep = [int(j) for j in sets[l]]
    Gp = [None] * wl.Hs
    Cp = [None] * wl.Hs
    n_tok = 0
    for c in range(4):                                            # 4 x 50 sequences = the configuration's 200
        ch = synth.make_chunk(wl, c, sl, sh, device=DEV, law=law)
        wk, wv = ch["w_k"][:, 0].contiguous(), ch["w_v"][:, 0].contiguous()      # weights per (comp, layer, token)
        cb.cb_fullhead_stats_accumulate(prob, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], wk, wv, G, C)
        src = bits(ch["src_v"][keep].cpu())                       # the four selected layers, re-indexed 0..3
        tgt = bits(ch["tgt_v"][l:l + 1].cpu())
        w = wv[l].cpu().numpy()
        for g in range(wl.Hs):
            gg, cc = oracle.multilayer_stats(src, tgt, w, 0, h, g, [0, 1, 2, 3])
            Gp[g] = gg if Gp[g] is None else Gp[g] + gg
            Cp[g] = cc if Cp[g] is None else Cp[g] + cc
        n_tok += ch["n_tokens"]
        del ch
    cb.cb_last_device_status()
    assert n_tok == 204800
    Gg, Cg = G[comp, l].cpu().numpy(), C[comp, l, h].cpu().numpy()
    Co = np.zeros((pf, d))
    num = den = 0.0
    worst = 0.0
    for g in range(wl.Hs):
        rows = np.array([(f * wl.Hs + g) * d + c_ for f in range(k) for c_ in range(d)] + [pf - 1])
        Co[rows[:-1]] = Cp[g][:-1]
        Co[pf - 1] = Cp[g][-1]
        sub = Gg[np.ix_(rows, rows)]
        num += np.linalg.norm(sub - Gp[g]) ** 2
        den += np.linalg.norm(Gp[g]) ** 2
        worst = max(worst, rel_fro(sub, Gp[g]))
    eg, ec = float(np.sqrt(num / den)), rel_fro(Cg, Co)
    print("config 3 at full size (204,800 tokens), (V, layer 17, head 5): rel err C %.2e; G pieces pooled %.2e, worst %.2e"
          % (ec, eg, worst))
    assert ec <= TOL and eg <= TOL and worst <= TOL
    assert torch.isfinite(G).all() and torch.isfinite(C).all()
