"""Layer selector (Section 3.1) on the GPU: probe R^2 from the path's own statistics against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_00891_b200 import binding as cb
from util import bits

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _traces(seed, Ls, Lt, H, T, d, truth):
    """Source layers of independent noise; every target layer is a random linear image of two known source layers
    (a strong and a weak one) plus noise, with channel offsets so that the centring matters."""
    g = torch.Generator().manual_seed(seed)
    src = torch.randn(2, Ls, T, H, d, generator=g) + 0.5
    tgt = torch.zeros(2, Lt, T, H, d)
    for comp in range(2):
        for l in range(Lt):
            for h in range(H):
                a = torch.randn(d, d, generator=g) / np.sqrt(d)
                b = torch.randn(d, d, generator=g) / np.sqrt(d)
                tgt[comp, l, :, h] = (src[comp, truth[l][0], :, h] @ a + 0.5 * src[comp, truth[l][1], :, h] @ b
                                      + 0.4 * torch.randn(T, d, generator=g) - 1.0)
    w = torch.exp(0.5 * torch.randn(2, Lt, H, T, generator=g)).float()
    return src.to(torch.bfloat16), tgt.to(torch.bfloat16), w


@pytest.mark.parametrize("d,flags", [(64, 0), (128, cb.CB_FLAG_COMPENSATED)])
def test_selector_scores_and_ranking_match_oracle(d, flags):
    Ls, Lt, H, T = 5, 3, 2, 3000
    truth = [[3, 1], [0, 4], [2, 3]]
    src, tgt, w = _traces(1, Ls, Lt, H, T, d, truth)
    sh = np.arange(H, dtype=np.int32)
    want = oracle.layer_scores(bits(src[0]), bits(src[1]), bits(tgt[0]), bits(tgt[1]), w[0].numpy(), w[1].numpy(), sh)
    dev = {"src_k": src[0].to(DEV), "src_v": src[1].to(DEV), "tgt_k": tgt[0].to(DEV), "tgt_v": tgt[1].to(DEV),
           "w_k": w[0].contiguous().to(DEV), "w_v": w[1].contiguous().to(DEV)}
    n_maps, p = 2 * Lt * H, d + 1
    scores = torch.zeros(Lt, Ls, device=DEV)
    syy = None
    for r in range(Ls):                                   # Ls probe sets with rotated layer pairing cover every (l, j)
        sl = np.array([(l + r) % Ls for l in range(Lt)], np.int32)
        prob = cb.Problem(Ls, H, d, Lt, H, d, sl, sh, flags=flags)
        ctx = cb.cb_create(prob, device=DEV)
        if syy is None:                                   # the targets' sums of squares: once, from the means pass
            ws = torch.empty(cb.cb_means_workspace_bytes(prob), dtype=torch.uint8, device=DEV)
            cb.cb_means_reset(ctx, ws)
            cb.cb_means_accumulate(ctx, dev["src_k"], dev["src_v"], dev["tgt_k"], dev["tgt_v"], dev["w_k"], dev["w_v"], ws)
            syy = torch.empty(n_maps, d, device=DEV)
            cb.cb_means_energy(ctx, ws, syy)
        cb.cb_stats_accumulate(ctx, dev["src_k"], dev["src_v"], dev["tgt_k"], dev["tgt_v"], dev["w_k"], dev["w_v"])
        G = torch.empty(n_maps, p, p, device=DEV)
        C = torch.empty(n_maps, p, d, device=DEV)
        n = cb.cb_stats_reduce(ctx, G, C)
        Wb = torch.empty(1, n_maps, p, d, device=DEV)
        info = torch.empty(1, n_maps, dtype=torch.int32, device=DEV)
        cb.cb_ridge_solve(G, C, n, [0.0], 0, Wb, info)    # ordinary least squares
        cb.cb_check_info(info)
        r2 = torch.empty(n_maps, device=DEV)
        cb.cb_probe_r2(G, C, Wb[0], syy, n, 0.0, 0, r2)
        cb.cb_probe_scores(r2, Lt, H, sl, Ls, scores)
        cb.cb_device_status(ctx)
    got = scores.cpu().numpy()
    print("scores (GPU)\n", np.round(got, 4), "\nscores (oracle)\n", np.round(want, 4))
    # R^2 is a ratio of sums the statistics carry to ~1e-3 (plain bf16 fold) or ~1e-6 (compensated)
    assert np.abs(got - want).max() <= (2e-5 if flags else 3e-3)
    for k in (1, 2):
        sets = cb.cb_rank_layers(got, k)
        assert np.array_equal(sets, oracle.rank_layers(want, k))
    assert cb.cb_rank_layers(got, 2).tolist() == [sorted(t) for t in truth]
