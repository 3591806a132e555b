"""Seeded synthetic calibration traces, weights and source caches.

This module only *draws inputs*.  It contains none of the method's arithmetic
(no statistics, no ridge solve, no affine apply, no head matching): the head
match is passed in by the caller as plain integer arrays.  Both the CUDA path
and the CPU oracle are fed the bytes produced here, so neither needs the other.

The generators stand in for KV traces of real models collected on a text
corpus: only the shapes (layers x KV heads x head width, sequence lengths) and
a rough value structure (per-channel scales, a few outlier channels, target
heads that are a noisy affine image of the matched source head, heavy-tailed
per-token weights with a causal position decay) are reproduced.

Layouts produced (all contiguous):
    traces   bf16  [L][T][H][d]      (layer, token, KV head, channel)
    weights  fp32  [L_t][H_t][T]     one tensor for K maps and one for V maps
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and recipe of one synthetic calibration workload."""

    name: str
    index: int            # position in the benchmark's config list (enters the seed)
    Ls: int
    Hs: int
    Lt: int
    Ht: int
    d: int
    seq_lens: tuple       # tokens per sequence, in order
    seqs_per_chunk: int   # how many sequences one streamed chunk holds
    lambdas: tuple
    kind: str             # "tiny" (known affine answer) or "scaled" (per-channel scales + outliers)
    noise: float
    seed: int = 0
    apply_tokens: int = 0  # length of the source cache mapped online after the fit (0: reuse chunk 0)

    @property
    def n_tokens(self) -> int:
        return int(sum(self.seq_lens))

    @property
    def n_maps(self) -> int:
        return 2 * self.Lt * self.Ht

    @property
    def n_chunks(self) -> int:
        n = len(self.seq_lens)
        return (n + self.seqs_per_chunk - 1) // self.seqs_per_chunk

    def chunk_seq_lens(self, chunk: int) -> tuple:
        a = chunk * self.seqs_per_chunk
        return self.seq_lens[a:a + self.seqs_per_chunk]

    def chunk_tokens(self, chunk: int) -> int:
        return int(sum(self.chunk_seq_lens(chunk)))


def _ragged_lengths(n_seq: int, lo: int, hi: int, seed: int) -> tuple:
    g = torch.Generator(device="cpu").manual_seed(seed)
    return tuple(int(v) for v in torch.randint(lo, hi + 1, (n_seq,), generator=g))


def workload(name: str) -> Workload:
    """The benchmark's workloads by name, plus small variants used by the tests."""
    if name == "tiny":            # 4 sequences x 256 tokens, d = 64, known affine answer
        return Workload("tiny", 0, 2, 2, 2, 2, 64, (256,) * 4, 4, (1e-2,), "tiny", 0.05)
    if name == "qwen8b_14b":      # 36 -> 40 layers, 64 x 1024 tokens
        return Workload("qwen8b_14b", 1, 36, 8, 40, 8, 128, (1024,) * 64, 16, (1e-2,), "scaled", 0.1)
    if name == "qwen14b_32b_500":  # 40 -> 64 layers, 500 x 1024 tokens: 1024 maps of 129 x 128
        return Workload("qwen14b_32b_500", 2, 40, 8, 64, 8, 128, (1024,) * 500, 50,
                        (1e-3, 1e-2, 1e-1), "scaled", 0.1)
    if name == "ragged_long":     # 500 ragged sequences, then a 32768-token cache is mapped
        lens = _ragged_lengths(500, 512, 8192, seed=4004)
        return Workload("ragged_long", 4, 40, 8, 64, 8, 128, lens, 12, (1e-2,), "scaled", 0.1,
                        apply_tokens=32768)
    # ---- reduced-size variants for tests (same recipe, fewer layers / tokens) ----
    if name == "mini_scaled":     # d = 128, ragged tail (T not a multiple of any tile), double-matched layers
        return Workload("mini_scaled", 11, 3, 2, 5, 2, 128, (301, 77, 419), 2, (1e-2,), "scaled", 0.1)
    if name == "mid_scaled":      # enough tokens per map (8709) for the plain bf16 weight fold to meet 1e-3
        return Workload("mid_scaled", 12, 2, 2, 3, 2, 128, (1024,) * 8 + (517,), 5, (1e-2,), "scaled", 0.1)
    if name == "long_unit":       # one chunk whose tokens exceed what a unit sums in tensor memory between drains
        return Workload("long_unit", 16, 2, 2, 3, 2, 128, (16384, 4099), 2, (1e-2,), "scaled", 0.1)
    if name == "very_long_unit":  # one map pair, 200,003 tokens in one call: many drains inside a unit, long rings
        return Workload("very_long_unit", 17, 1, 1, 1, 1, 128, (200003,), 1, (1e-2,), "scaled", 0.1)
    if name == "deep_small":      # enough source layers for the paper's k = 8 selected layers (regressor width 1025)
        return Workload("deep_small", 15, 10, 2, 3, 2, 128, (1100, 1000), 2, (1e-2,), "scaled", 0.1)
    if name == "deep_fit":        # k = 8 with 64 rows per regressor column (65,536 rows, width 1025): a well-posed wide fit
        return Workload("deep_fit", 18, 10, 2, 3, 2, 128, (1024,) * 64, 64, (1e-2,), "scaled", 0.1)
    if name == "mini_ragged":     # several chunks of unequal size
        lens = _ragged_lengths(9, 40, 700, seed=77)
        return Workload("mini_ragged", 14, 4, 4, 6, 4, 128, lens, 3, (1e-3, 1e-2, 1e-1), "scaled", 0.1,
                        apply_tokens=1000)
    raise KeyError(name)


def _gen(seed: int, device) -> torch.Generator:
    return torch.Generator(device=device).manual_seed(int(seed))


@dataclasses.dataclass
class MapLaw:
    """Per-workload constants of the trace law (fixed across chunks)."""

    src_scale: torch.Tensor   # fp32 [2][Ls][Hs][d]   per-channel scale of every source head
    tgt_scale: torch.Tensor   # fp32 [2][Lt][Ht][d]
    A: torch.Tensor           # fp32 [2][Lt][Ht][d][d] latent linear image
    b: torch.Tensor           # fp32 [2][Lt][Ht][d]


def _channel_scales(shape_prefix: Sequence[int], d: int, kind: str, g: torch.Generator, device) -> torch.Tensor:
    if kind == "tiny":
        return torch.ones(*shape_prefix, d, device=device)
    s = torch.exp(0.5 * torch.randn(*shape_prefix, d, generator=g, device=device))
    n_out = max(1, (2 * d) // 128)      # two outlier channels per 128 channels
    # choose outlier channels without replacement: the n_out largest of a random score
    score = torch.rand(*shape_prefix, d, generator=g, device=device)
    idx = score.topk(n_out, dim=-1).indices
    boost = torch.ones_like(s)
    boost.scatter_(-1, idx, 8.0)
    return s * boost


def map_law(wl: Workload, device="cpu") -> MapLaw:
    g = _gen(wl.seed + 1000 * wl.index + 999_983, device)
    src_scale = _channel_scales((2, wl.Ls, wl.Hs), wl.d, wl.kind, g, device)
    tgt_scale = _channel_scales((2, wl.Lt, wl.Ht), wl.d, wl.kind, g, device)
    A = torch.randn(2, wl.Lt, wl.Ht, wl.d, wl.d, generator=g, device=device) / (wl.d ** 0.5)
    b = torch.randn(2, wl.Lt, wl.Ht, wl.d, generator=g, device=device) * (0.1 ** 0.5)
    return MapLaw(src_scale, tgt_scale, A, b)


def positions_in_sequence(seq_lens: Sequence[int], device="cpu") -> torch.Tensor:
    """int64 [T]: index of every token inside its own sequence for a packed batch."""
    parts = [torch.arange(n, device=device) for n in seq_lens]
    if not parts:
        return torch.zeros(0, dtype=torch.int64, device=device)
    return torch.cat(parts)


def make_weights(Lt: int, Ht: int, seq_lens: Sequence[int], g: torch.Generator, device) -> torch.Tensor:
    """Heavy-tailed token weights with a causal position decay: exp(N(0,1)) / (1 + t/128)."""
    T = int(sum(seq_lens))
    pos = positions_in_sequence(seq_lens, device).to(torch.float32)
    decay = 1.0 / (1.0 + pos / 128.0)
    w = torch.exp(torch.randn(Lt, Ht, T, generator=g, device=device)) * decay
    return w.contiguous()


def make_source(wl: Workload, law: MapLaw, T: int, g: torch.Generator, device) -> List[torch.Tensor]:
    """[K, V] bf16 [Ls][T][Hs][d] source traces."""
    out = []
    for comp in range(2):
        x = torch.empty(wl.Ls, T, wl.Hs, wl.d, dtype=torch.bfloat16, device=device)
        for j in range(wl.Ls):
            raw = torch.randn(T, wl.Hs, wl.d, generator=g, device=device)
            x[j] = (raw * law.src_scale[comp, j]).to(torch.bfloat16)
        out.append(x)
    return out


def make_target(wl: Workload, law: MapLaw, src: List[torch.Tensor], src_layer, src_head,
                g: torch.Generator, device) -> List[torch.Tensor]:
    """[K, V] bf16 [Lt][T][Ht][d]: noisy affine image of the matched source head."""
    T = src[0].shape[1]
    out = []
    for comp in range(2):
        y = torch.empty(wl.Lt, T, wl.Ht, wl.d, dtype=torch.bfloat16, device=device)
        for l in range(wl.Lt):
            j = int(src_layer[l])
            heads = torch.as_tensor([int(h) for h in src_head], device=device)
            xs = src[comp][j].to(torch.float32)[:, heads, :]              # [T][Ht][d]
            xs = xs / law.src_scale[comp, j][heads]                       # unit-variance latent
            yl = torch.einsum("thc,hce->the", xs, law.A[comp, l]) + law.b[comp, l]
            yl = yl + wl.noise * torch.randn(T, wl.Ht, wl.d, generator=g, device=device)
            y[l] = (yl * law.tgt_scale[comp, l]).to(torch.bfloat16)
        out.append(y)
    return out


def make_chunk(wl: Workload, chunk: int, src_layer, src_head, device="cpu",
               law: Optional[MapLaw] = None) -> Dict[str, torch.Tensor]:
    """One streamed chunk of the calibration set, a pure function of (workload, chunk)."""
    if law is None:
        law = map_law(wl, device)
    lens = wl.chunk_seq_lens(chunk)
    T = int(sum(lens))
    g = _gen(wl.seed + 1000 * wl.index + chunk, device)
    src = make_source(wl, law, T, g, device)
    tgt = make_target(wl, law, src, src_layer, src_head, g, device)
    w_k = make_weights(wl.Lt, wl.Ht, lens, g, device)
    w_v = make_weights(wl.Lt, wl.Ht, lens, g, device)
    return {"src_k": src[0], "src_v": src[1], "tgt_k": tgt[0], "tgt_v": tgt[1],
            "w_k": w_k, "w_v": w_v, "n_tokens": T}


def make_source_cache(wl: Workload, T: int, device="cpu", law: Optional[MapLaw] = None) -> List[torch.Tensor]:
    """A source KV cache of T tokens from the same law (input of the online apply)."""
    if law is None:
        law = map_law(wl, device)
    g = _gen(wl.seed + 1000 * wl.index + 500_000, device)
    return make_source(wl, law, T, g, device)
