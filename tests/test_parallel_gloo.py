"""World-size-2 CPU (gloo) test of the multi-GPU host logic: sequence sharding, the one statistics exchange and
the gather of per-rank map slices.  The per-rank statistics come from the oracle here (no GPU in this test)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2609_00891_b200 import parallel, synth
    from util import bits

    wl = synth.workload("mini_ragged")
    sl, sh = oracle.head_map(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    law = synth.map_law(wl)
    G = C = None
    n = 0
    for c in parallel.shard_chunks(wl.n_chunks, rank, world):          # this rank's sequences
        ch = synth.make_chunk(wl, c, sl, sh, law=law)
        g, cc = oracle.stats_traces(bits(ch["src_k"]), bits(ch["src_v"]), bits(ch["tgt_k"]), bits(ch["tgt_v"]),
                                    ch["w_k"].numpy(), ch["w_v"].numpy(), sl, sh)
        G, C = (g, cc) if G is None else (G + g, C + cc)
        n += ch["n_tokens"]
    Gt, Ct = torch.from_numpy(G), torch.from_numpy(C)
    n_all = parallel.exchange_statistics(Gt, Ct, n)
    m0, m1 = parallel.shard_range(wl.n_maps, rank, world)
    Th, info = oracle.ridge_solve(Gt[m0:m1].numpy(), Ct[m0:m1].numpy(), n_all, 1e-2)
    full = parallel.gather_maps(torch.from_numpy(Th)[None], wl.n_maps)
    if rank == 0:
        torch.save({"G": Gt, "C": Ct, "n": n_all, "Wb": full}, out)
    dist.barrier()
    dist.destroy_process_group()


def test_shard_ranges_partition_everything():
    sys.path.insert(0, ROOT)
    from paper_2609_00891_b200 import parallel
    for n in (0, 1, 7, 48, 1024):
        for world in (1, 2, 3, 8):
            parts = [parallel.shard_range(n, r, world) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == n
            assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            sizes = [b - a for a, b in parts]
            assert max(sizes) - min(sizes) <= 1


@pytest.mark.timeout(300)
def test_two_rank_build_equals_single_process(tmp_path):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2609_00891_b200 import synth
    from util import bits

    out = str(tmp_path / "rank0.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    got = torch.load(out)
    wl = synth.workload("mini_ragged")
    sl, sh = oracle.head_map(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    law = synth.map_law(wl)
    G = C = None
    for c in range(wl.n_chunks):
        ch = synth.make_chunk(wl, c, sl, sh, law=law)
        g, cc = oracle.stats_traces(bits(ch["src_k"]), bits(ch["src_v"]), bits(ch["tgt_k"]), bits(ch["tgt_v"]),
                                    ch["w_k"].numpy(), ch["w_v"].numpy(), sl, sh)
        G, C = (g, cc) if G is None else (G + g, C + cc)
    assert got["n"] == wl.n_tokens
    np.testing.assert_allclose(got["G"].numpy(), G, rtol=1e-12, atol=1e-9)
    np.testing.assert_allclose(got["C"].numpy(), C, rtol=1e-12, atol=1e-9)
    Th, info = oracle.ridge_solve(G, C, wl.n_tokens, 1e-2)
    assert got["Wb"].shape == (1, wl.n_maps, wl.d + 1, wl.d)
    np.testing.assert_allclose(got["Wb"][0].numpy(), Th, rtol=1e-8, atol=1e-10)
