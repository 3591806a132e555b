"""ctypes binding of the C ABI declared in include/cb.h.

Argument marshalling only: every step of the path runs in the CUDA library.  torch tensors are used as plain
device buffers (data_ptr, strides) and torch streams as cudaStream_t.  There is no fallback: if the shared
library has not been built, importing a function from here raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcb.so")

CB_OK = 0
CB_ERR_INVALID_ARG, CB_ERR_UNSUPPORTED, CB_ERR_STATE, CB_ERR_WORKSPACE = 1, 2, 3, 4
CB_ERR_CUDA, CB_ERR_NOT_PD, CB_ERR_TIMEOUT, CB_ERR_STATIC_LIMIT = 5, 6, 7, 8
CB_FLAG_COMPENSATED, CB_FLAG_RAW_LAMBDA, CB_FLAG_SIMT, CB_FLAG_ONE_ROW_HEAD = 1, 2, 4, 8
CB_DTYPE_BF16, CB_DTYPE_F32 = 0, 1

EXPORTS = ("cb_status_string", "cb_head_map_nearest", "cb_work_list", "cb_workspace_bytes", "cb_token_splits", "cb_create",
           "cb_destroy", "cb_stats_reset", "cb_stats_accumulate", "cb_staging_bytes", "cb_stats_accumulate_host",
           "cb_stats_reduce", "cb_ridge_solve",
           "cb_check_info", "cb_apply", "cb_device_status", "cb_stats_build_static", "cb_fullhead_layer_sets",
           "cb_fullhead_workspace_bytes", "cb_fullhead_stats_accumulate", "cb_ess_weights", "cb_ridge_solve_large_workspace_bytes", "cb_ridge_solve_large", "cb_multilayer_workspace_bytes",
           "cb_multilayer_stats_accumulate", "cb_apply_multilayer_workspace_bytes", "cb_apply_multilayer",
           "cb_means_workspace_bytes", "cb_means_reset", "cb_means_accumulate", "cb_means_finalize",
           "cb_stats_accumulate_centered", "cb_stats_reduce_centered", "cb_ridge_solve_centered",
           "cb_stats_accumulate_rope", "cb_rope_rotate", "cb_apply_rope",
           "cb_means_accumulate_rope", "cb_stats_accumulate_centered_rope",
           "cb_means_energy", "cb_probe_r2", "cb_probe_scores", "cb_rank_layers",
           "cb_last_device_status", "cb_test_hooks", "cb_stats_state_bytes", "cb_stats_export", "cb_stats_import",
           "cb_last_cuda_error", "cb_launch_count")


class CbError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = ""
        if status == CB_ERR_CUDA:
            self.cuda_error, text = cb_last_cuda_error()
            detail = ": CUDA error %d, %s" % (self.cuda_error, text)
        super().__init__("%s: %s (status %d)%s" % (where, status_string(status), status, detail))


class _KvView(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
                ("n_layers", ctypes.c_int32), ("n_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("n_tokens", ctypes.c_int64),
                ("stride_layer", ctypes.c_int64), ("stride_token", ctypes.c_int64), ("stride_head", ctypes.c_int64)]


class _Problem(ctypes.Structure):
    _fields_ = [("Ls", ctypes.c_int32), ("Hs", ctypes.c_int32), ("ds", ctypes.c_int32),
                ("Lt", ctypes.c_int32), ("Ht", ctypes.c_int32), ("dt", ctypes.c_int32),
                ("src_layer", ctypes.POINTER(ctypes.c_int32)), ("src_head", ctypes.POINTER(ctypes.c_int32)),
                ("flags", ctypes.c_uint32), ("n_splits", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("CUDA library %s is missing: run `python -m paper_2609_00891_b200.build` "
                               "(there is no CPU fallback)" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        L.cb_status_string.restype = ctypes.c_char_p
        L.cb_status_string.argtypes = [ctypes.c_int]
        L.cb_launch_count.restype = ctypes.c_int64
        for name in EXPORTS:
            if name not in ("cb_status_string", "cb_launch_count", "cb_destroy"):
                getattr(L, name).restype = ctypes.c_int
        L.cb_destroy.restype = None
        _lib = L
    return _lib


def cb_last_cuda_error() -> Tuple[int, str]:
    """(CUDA runtime error code, its description) behind the most recent CB_ERR_CUDA; (0, "no error") if none.  Clears it."""
    text = ctypes.c_char_p()
    code = lib().cb_last_cuda_error(ctypes.byref(text))
    return int(code), (text.value or b"").decode()


def status_string(status: int) -> str:
    return lib().cb_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != CB_OK:
        raise CbError(status, where)


def _stream_ptr(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


class Problem:
    """Model shapes plus the static head match (host arrays), mirroring cb_problem."""

    def __init__(self, Ls: int, Hs: int, ds: int, Lt: int, Ht: int, dt: int,
                 src_layer: Sequence[int], src_head: Sequence[int], flags: int = 0, n_splits: int = 0):
        self.src_layer = np.ascontiguousarray(src_layer, dtype=np.int32)
        self.src_head = np.ascontiguousarray(src_head, dtype=np.int32)
        assert self.src_layer.shape == (Lt,) and self.src_head.shape == (Ht,)
        self.c = _Problem(Ls, Hs, ds, Lt, Ht, dt,
                          self.src_layer.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                          self.src_head.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                          flags, n_splits)
        self.Ls, self.Hs, self.ds, self.Lt, self.Ht, self.dt = Ls, Hs, ds, Lt, Ht, dt
        self.flags, self.n_splits = flags, n_splits

    @property
    def n_maps(self) -> int:
        return 2 * self.Lt * self.Ht

    def with_flags(self, flags: int) -> "Problem":
        return Problem(self.Ls, self.Hs, self.ds, self.Lt, self.Ht, self.dt, self.src_layer, self.src_head,
                       flags, self.n_splits)


def _kv_view(k: torch.Tensor, v: torch.Tensor) -> _KvView:
    """View of K and V tensors indexed [layer][token][head][channel] (any strides, channels contiguous)."""
    assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.dim() == 4
    assert k.shape == v.shape and k.stride() == v.stride() and k.stride(3) == 1
    L, T, H, d = k.shape
    return _KvView(k.data_ptr(), v.data_ptr(), L, H, d, T, k.stride(0), k.stride(1), k.stride(2))


# ---------------------------------------------------------------------------------------------- host-only calls
def cb_head_map_nearest(Ls: int, Hs: int, Lt: int, Ht: int) -> Tuple[np.ndarray, np.ndarray]:
    sl = np.empty(Lt, np.int32)
    sh = np.empty(Ht, np.int32)
    _check(lib().cb_head_map_nearest(Ls, Hs, Lt, Ht, sl.ctypes.data_as(ctypes.c_void_p),
                                     sh.ctypes.data_as(ctypes.c_void_p)), "cb_head_map_nearest")
    return sl, sh


def cb_work_list(prob: Problem):
    cap = 2 * prob.Ls * prob.Hs
    n = ctypes.c_int32(0)
    ic, il, ih = (np.empty(cap, np.int32) for _ in range(3))
    ib = np.empty(cap + 1, np.int32)
    im = np.empty(prob.n_maps, np.int32)
    p = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    _check(lib().cb_work_list(ctypes.byref(prob.c), ctypes.byref(n), p(ic), p(il), p(ih), p(ib), p(im)), "cb_work_list")
    k = n.value
    return ic[:k].copy(), il[:k].copy(), ih[:k].copy(), ib[:k + 1].copy(), im.copy()


def cb_token_splits(prob: Problem) -> int:
    n = ctypes.c_int32(0)
    _check(lib().cb_token_splits(ctypes.byref(prob.c), ctypes.byref(n)), "cb_token_splits")
    return int(n.value)


def cb_workspace_bytes(prob: Problem) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().cb_workspace_bytes(ctypes.byref(prob.c), ctypes.byref(n)), "cb_workspace_bytes")
    return n.value


# ---------------------------------------------------------------------------------------------- device calls
class Context:
    """Owns a cb_ctx; the workspace tensor is kept alive with it."""

    def __init__(self, prob: Problem, workspace: Optional[torch.Tensor] = None, device="cuda"):
        self.prob = prob
        if workspace is None:
            workspace = torch.empty(cb_workspace_bytes(prob), dtype=torch.uint8, device=device)
        self.workspace = workspace
        h = ctypes.c_void_p()
        _check(lib().cb_create(ctypes.byref(prob.c), ctypes.c_void_p(workspace.data_ptr()),
                               ctypes.c_size_t(workspace.numel()), ctypes.byref(h)), "cb_create")
        self.handle = h

    def close(self):
        if self.handle:
            lib().cb_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def cb_create(prob: Problem, workspace: Optional[torch.Tensor] = None, device="cuda") -> Context:
    return Context(prob, workspace, device)


def cb_destroy(ctx: Context) -> None:
    ctx.close()


def cb_stats_reset(ctx: Context, stream=None) -> None:
    _check(lib().cb_stats_reset(ctx.handle, _stream_ptr(stream)), "cb_stats_reset")


def cb_stats_accumulate(ctx: Context, src_k, src_v, tgt_k, tgt_v, w_k: torch.Tensor, w_v: torch.Tensor, stream=None) -> None:
    """Traces [L][T][H][d] bf16, weights [Lt][Ht][T] fp32 (tokens contiguous)."""
    sv, tv = _kv_view(src_k, src_v), _kv_view(tgt_k, tgt_v)
    assert w_k.dtype == torch.float32 and w_v.dtype == torch.float32 and w_k.dim() == 3
    assert w_k.stride() == w_v.stride() and (w_k.stride(2) == 1 or w_k.shape[2] <= 1)
    _check(lib().cb_stats_accumulate(ctx.handle, ctypes.byref(sv), ctypes.byref(tv),
                                     ctypes.c_void_p(w_k.data_ptr()), ctypes.c_void_p(w_v.data_ptr()),
                                     ctypes.c_int64(w_k.stride(0)), ctypes.c_int64(w_k.stride(1)),
                                     _stream_ptr(stream)), "cb_stats_accumulate")


def cb_staging_bytes(prob: Problem, n_tokens: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().cb_staging_bytes(ctypes.byref(prob.c), ctypes.c_int64(n_tokens), ctypes.byref(n)), "cb_staging_bytes")
    return n.value


def cb_stats_accumulate_host(ctx: Context, src_k, src_v, tgt_k, tgt_v, w_k, w_v, staging: torch.Tensor, stream=None) -> None:
    """Host (CPU, ideally pinned) contiguous traces [L][T][H][d] bf16 and weights [Lt][Ht][T] fp32; `staging` is a
    device uint8 tensor of at least cb_staging_bytes()."""
    for t in (src_k, src_v, tgt_k, tgt_v, w_k, w_v):
        assert t.device.type == "cpu" and t.is_contiguous()
    sv, tv = _kv_view(src_k, src_v), _kv_view(tgt_k, tgt_v)
    assert staging.is_cuda and staging.dtype == torch.uint8
    _check(lib().cb_stats_accumulate_host(ctx.handle, ctypes.byref(sv), ctypes.byref(tv),
                                          ctypes.c_void_p(w_k.data_ptr()), ctypes.c_void_p(w_v.data_ptr()),
                                          ctypes.c_void_p(staging.data_ptr()), ctypes.c_size_t(staging.numel()),
                                          _stream_ptr(stream)), "cb_stats_accumulate_host")


def cb_stats_state_bytes(ctx: Context) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().cb_stats_state_bytes(ctx.handle, ctypes.byref(n)), "cb_stats_state_bytes")
    return n.value


def cb_stats_export(ctx: Context, dst: torch.Tensor, stream=None) -> int:
    """Copies the partial statistics into `dst` (uint8 tensor, device or pinned/pageable host); returns the row count."""
    assert dst.dtype == torch.uint8 and dst.is_contiguous()
    n = ctypes.c_int64(0)
    _check(lib().cb_stats_export(ctx.handle, ctypes.c_void_p(dst.data_ptr()), ctypes.c_size_t(dst.numel()), ctypes.byref(n),
                                 _stream_ptr(stream)), "cb_stats_export")
    return int(n.value)


def cb_stats_import(ctx: Context, src: torch.Tensor, n_tokens: int, stream=None) -> None:
    assert src.dtype == torch.uint8 and src.is_contiguous()
    _check(lib().cb_stats_import(ctx.handle, ctypes.c_void_p(src.data_ptr()), ctypes.c_size_t(src.numel()),
                                 ctypes.c_int64(n_tokens), _stream_ptr(stream)), "cb_stats_import")


def cb_stats_reduce(ctx: Context, G: torch.Tensor, C: torch.Tensor, stream=None) -> int:
    p, d = ctx.prob.ds + 1, ctx.prob.ds
    assert G.dtype == torch.float32 and C.dtype == torch.float32 and G.is_contiguous() and C.is_contiguous()
    assert G.numel() == ctx.prob.n_maps * p * p and C.numel() == ctx.prob.n_maps * p * d
    n = ctypes.c_int64(0)
    _check(lib().cb_stats_reduce(ctx.handle, ctypes.c_void_p(G.data_ptr()), ctypes.c_void_p(C.data_ptr()),
                                 ctypes.byref(n), _stream_ptr(stream)), "cb_stats_reduce")
    return n.value


def cb_ridge_solve(G: torch.Tensor, C: torch.Tensor, n_tokens: int, lambdas: Sequence[float], flags: int,
                   Wb: torch.Tensor, info: torch.Tensor, stream=None) -> None:
    n_maps, p, _ = G.shape
    d = p - 1
    lam = np.ascontiguousarray(lambdas, dtype=np.float32)
    assert G.dtype == torch.float32 and C.dtype == torch.float32 and Wb.dtype == torch.float32 and info.dtype == torch.int32
    assert G.is_contiguous() and C.is_contiguous() and Wb.is_contiguous() and info.is_contiguous()
    assert Wb.numel() == len(lam) * n_maps * p * d and info.numel() == len(lam) * n_maps
    _check(lib().cb_ridge_solve(ctypes.c_void_p(G.data_ptr()), ctypes.c_void_p(C.data_ptr()), n_maps, d,
                                ctypes.c_int64(n_tokens), lam.ctypes.data_as(ctypes.c_void_p), len(lam),
                                ctypes.c_uint32(flags), ctypes.c_void_p(Wb.data_ptr()),
                                ctypes.c_void_p(info.data_ptr()), _stream_ptr(stream)), "cb_ridge_solve")


# ----------------------------------------------------------------------------- layer selector
def cb_means_energy(ctx: Context, means_ws: torch.Tensor, syy: torch.Tensor, stream=None) -> None:
    """syy: fp32 device [n_maps][d] = sum w y^2 from a means workspace filled by cb_means_accumulate."""
    assert syy.dtype == torch.float32 and syy.is_contiguous() and syy.numel() == ctx.prob.n_maps * ctx.prob.ds
    _check(lib().cb_means_energy(ctx.handle, ctypes.c_void_p(means_ws.data_ptr()), ctypes.c_size_t(means_ws.numel()),
                                 ctypes.c_void_p(syy.data_ptr()), _stream_ptr(stream)), "cb_means_energy")


def cb_probe_r2(G: torch.Tensor, C: torch.Tensor, Wb: torch.Tensor, syy: torch.Tensor, n_tokens: int, lam: float,
                flags: int, r2: torch.Tensor, stream=None) -> None:
    n_maps, p, _ = G.shape
    d = p - 1
    for t in (G, C, Wb, syy, r2):
        assert t.dtype == torch.float32 and t.is_contiguous()
    assert Wb.numel() == n_maps * p * d and syy.numel() == n_maps * d and r2.numel() == n_maps
    _check(lib().cb_probe_r2(ctypes.c_void_p(G.data_ptr()), ctypes.c_void_p(C.data_ptr()), ctypes.c_void_p(Wb.data_ptr()),
                             ctypes.c_void_p(syy.data_ptr()), n_maps, d, ctypes.c_int64(n_tokens), ctypes.c_float(lam),
                             ctypes.c_uint32(flags), ctypes.c_void_p(r2.data_ptr()), _stream_ptr(stream)), "cb_probe_r2")


def cb_probe_scores(r2: torch.Tensor, Lt: int, Ht: int, src_layer, Ls: int, scores: torch.Tensor, stream=None) -> None:
    sl = np.ascontiguousarray(src_layer, dtype=np.int32)
    assert r2.dtype == torch.float32 and scores.dtype == torch.float32 and scores.is_contiguous()
    assert r2.numel() == 2 * Lt * Ht and scores.numel() == Lt * Ls and sl.shape == (Lt,)
    _check(lib().cb_probe_scores(ctypes.c_void_p(r2.data_ptr()), Lt, Ht, sl.ctypes.data_as(ctypes.c_void_p), Ls,
                                 ctypes.c_void_p(scores.data_ptr()), _stream_ptr(stream)), "cb_probe_scores")


def cb_rank_layers(scores: np.ndarray, k: int) -> np.ndarray:
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    Lt, Ls = scores.shape
    sets = np.empty((Lt, k), np.int32)
    _check(lib().cb_rank_layers(scores.ctypes.data_as(ctypes.c_void_p), Lt, Ls, k, sets.ctypes.data_as(ctypes.c_void_p)),
           "cb_rank_layers")
    return sets


# ----------------------------------------------------------------------------- rotary embedding at the boundary
def cb_stats_accumulate_rope(ctx: Context, src_k, src_v, tgt_k, tgt_v, w_k: torch.Tensor, w_v: torch.Tensor,
                             positions: torch.Tensor, rope_base_src: float, rope_base_tgt: float, stream=None) -> None:
    """As cb_stats_accumulate; `positions` is a device int32 tensor [T]."""
    sv, tv = _kv_view(src_k, src_v), _kv_view(tgt_k, tgt_v)
    assert w_k.dtype == torch.float32 and w_v.dtype == torch.float32 and w_k.dim() == 3
    assert w_k.stride() == w_v.stride() and (w_k.stride(2) == 1 or w_k.shape[2] <= 1)
    assert positions.dtype == torch.int32 and positions.is_cuda and positions.is_contiguous()
    assert positions.numel() == src_k.shape[1]
    _check(lib().cb_stats_accumulate_rope(ctx.handle, ctypes.byref(sv), ctypes.byref(tv),
                                          ctypes.c_void_p(w_k.data_ptr()), ctypes.c_void_p(w_v.data_ptr()),
                                          ctypes.c_int64(w_k.stride(0)), ctypes.c_int64(w_k.stride(1)),
                                          ctypes.c_void_p(positions.data_ptr()), ctypes.c_double(rope_base_src),
                                          ctypes.c_double(rope_base_tgt), _stream_ptr(stream)), "cb_stats_accumulate_rope")


def cb_rope_rotate(k: torch.Tensor, positions: torch.Tensor, rope_base: float, inverse: bool, stream=None) -> None:
    """In-place rotary embedding (or its removal) of a bf16 key tensor indexed [L][T][H][d]."""
    assert k.dtype == torch.bfloat16 and k.dim() == 4 and k.stride(3) == 1
    assert positions.dtype == torch.int32 and positions.is_contiguous() and positions.numel() == k.shape[1]
    L, T, H, d = k.shape
    _check(lib().cb_rope_rotate(ctypes.c_void_p(k.data_ptr()), L, H, d, ctypes.c_int64(T),
                                ctypes.c_int64(k.stride(0)), ctypes.c_int64(k.stride(1)), ctypes.c_int64(k.stride(2)),
                                ctypes.c_void_p(positions.data_ptr()), ctypes.c_double(rope_base),
                                1 if inverse else 0, _stream_ptr(stream)), "cb_rope_rotate")


# ----------------------------------------------------------------------------- two-pass centred construction
def cb_means_workspace_bytes(prob: Problem) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().cb_means_workspace_bytes(ctypes.byref(prob.c), ctypes.byref(n)), "cb_means_workspace_bytes")
    return n.value


def cb_means_reset(ctx: Context, means_ws: torch.Tensor, stream=None) -> None:
    _check(lib().cb_means_reset(ctx.handle, ctypes.c_void_p(means_ws.data_ptr()), ctypes.c_size_t(means_ws.numel()),
                                _stream_ptr(stream)), "cb_means_reset")


def cb_means_accumulate(ctx: Context, src_k, src_v, tgt_k, tgt_v, w_k: torch.Tensor, w_v: torch.Tensor,
                        means_ws: torch.Tensor, stream=None) -> None:
    """First pass over one chunk; arguments as cb_stats_accumulate plus the uint8 device tensor `means_ws`."""
    sv, tv = _kv_view(src_k, src_v), _kv_view(tgt_k, tgt_v)
    assert w_k.dtype == torch.float32 and w_v.dtype == torch.float32 and w_k.dim() == 3
    assert w_k.stride() == w_v.stride() and (w_k.stride(2) == 1 or w_k.shape[2] <= 1)
    assert means_ws.is_cuda and means_ws.dtype == torch.uint8
    _check(lib().cb_means_accumulate(ctx.handle, ctypes.byref(sv), ctypes.byref(tv),
                                     ctypes.c_void_p(w_k.data_ptr()), ctypes.c_void_p(w_v.data_ptr()),
                                     ctypes.c_int64(w_k.stride(0)), ctypes.c_int64(w_k.stride(1)),
                                     ctypes.c_void_p(means_ws.data_ptr()), ctypes.c_size_t(means_ws.numel()),
                                     _stream_ptr(stream)), "cb_means_accumulate")


def cb_means_accumulate_rope(ctx: Context, src_k, src_v, tgt_k, tgt_v, w_k: torch.Tensor, w_v: torch.Tensor,
                             means_ws: torch.Tensor, positions: torch.Tensor, rope_base_src: float, rope_base_tgt: float,
                             stream=None) -> None:
    """As cb_means_accumulate, keys taken in content coordinates; `positions` is a device int32 tensor [T]."""
    sv, tv = _kv_view(src_k, src_v), _kv_view(tgt_k, tgt_v)
    assert w_k.dtype == torch.float32 and w_v.dtype == torch.float32 and w_k.dim() == 3
    assert w_k.stride() == w_v.stride() and (w_k.stride(2) == 1 or w_k.shape[2] <= 1)
    assert means_ws.is_cuda and means_ws.dtype == torch.uint8
    assert positions.dtype == torch.int32 and positions.is_cuda and positions.is_contiguous()
    assert positions.numel() == src_k.shape[1]
    _check(lib().cb_means_accumulate_rope(ctx.handle, ctypes.byref(sv), ctypes.byref(tv),
                                          ctypes.c_void_p(w_k.data_ptr()), ctypes.c_void_p(w_v.data_ptr()),
                                          ctypes.c_int64(w_k.stride(0)), ctypes.c_int64(w_k.stride(1)),
                                          ctypes.c_void_p(means_ws.data_ptr()), ctypes.c_size_t(means_ws.numel()),
                                          ctypes.c_void_p(positions.data_ptr()), ctypes.c_double(rope_base_src),
                                          ctypes.c_double(rope_base_tgt), _stream_ptr(stream)), "cb_means_accumulate_rope")


def cb_means_finalize(ctx: Context, means_ws: torch.Tensor, mu: torch.Tensor, stream=None) -> None:
    """mu: fp32 device [n_maps][2 d + 1] = mu_x, mu_y, s_w."""
    assert mu.dtype == torch.float32 and mu.is_contiguous() and mu.numel() == ctx.prob.n_maps * (2 * ctx.prob.ds + 1)
    _check(lib().cb_means_finalize(ctx.handle, ctypes.c_void_p(means_ws.data_ptr()), ctypes.c_size_t(means_ws.numel()),
                                   ctypes.c_void_p(mu.data_ptr()), _stream_ptr(stream)), "cb_means_finalize")


def cb_stats_accumulate_centered(ctx: Context, src_k, src_v, tgt_k, tgt_v, w_k: torch.Tensor, w_v: torch.Tensor,
                                 mu: torch.Tensor, stream=None) -> None:
    sv, tv = _kv_view(src_k, src_v), _kv_view(tgt_k, tgt_v)
    assert w_k.dtype == torch.float32 and w_v.dtype == torch.float32 and w_k.dim() == 3
    assert w_k.stride() == w_v.stride() and (w_k.stride(2) == 1 or w_k.shape[2] <= 1)
    assert mu.dtype == torch.float32 and mu.is_contiguous() and mu.numel() == ctx.prob.n_maps * (2 * ctx.prob.ds + 1)
    _check(lib().cb_stats_accumulate_centered(ctx.handle, ctypes.byref(sv), ctypes.byref(tv),
                                              ctypes.c_void_p(w_k.data_ptr()), ctypes.c_void_p(w_v.data_ptr()),
                                              ctypes.c_int64(w_k.stride(0)), ctypes.c_int64(w_k.stride(1)),
                                              ctypes.c_void_p(mu.data_ptr()), _stream_ptr(stream)),
           "cb_stats_accumulate_centered")


def cb_stats_accumulate_centered_rope(ctx: Context, src_k, src_v, tgt_k, tgt_v, w_k: torch.Tensor, w_v: torch.Tensor,
                                      mu: torch.Tensor, positions: torch.Tensor, rope_base_src: float, rope_base_tgt: float,
                                      stream=None) -> None:
    sv, tv = _kv_view(src_k, src_v), _kv_view(tgt_k, tgt_v)
    assert w_k.dtype == torch.float32 and w_v.dtype == torch.float32 and w_k.dim() == 3
    assert w_k.stride() == w_v.stride() and (w_k.stride(2) == 1 or w_k.shape[2] <= 1)
    assert mu.dtype == torch.float32 and mu.is_contiguous() and mu.numel() == ctx.prob.n_maps * (2 * ctx.prob.ds + 1)
    assert positions.dtype == torch.int32 and positions.is_cuda and positions.is_contiguous()
    assert positions.numel() == src_k.shape[1]
    _check(lib().cb_stats_accumulate_centered_rope(ctx.handle, ctypes.byref(sv), ctypes.byref(tv),
                                                   ctypes.c_void_p(w_k.data_ptr()), ctypes.c_void_p(w_v.data_ptr()),
                                                   ctypes.c_int64(w_k.stride(0)), ctypes.c_int64(w_k.stride(1)),
                                                   ctypes.c_void_p(mu.data_ptr()), ctypes.c_void_p(positions.data_ptr()),
                                                   ctypes.c_double(rope_base_src), ctypes.c_double(rope_base_tgt),
                                                   _stream_ptr(stream)), "cb_stats_accumulate_centered_rope")


def cb_stats_reduce_centered(ctx: Context, mu: torch.Tensor, A: torch.Tensor, B: torch.Tensor, stream=None) -> int:
    d = ctx.prob.ds
    assert A.dtype == torch.float32 and B.dtype == torch.float32 and A.is_contiguous() and B.is_contiguous()
    assert A.numel() == ctx.prob.n_maps * d * d and B.numel() == ctx.prob.n_maps * d * d
    n = ctypes.c_int64(0)
    _check(lib().cb_stats_reduce_centered(ctx.handle, ctypes.c_void_p(mu.data_ptr()), ctypes.c_void_p(A.data_ptr()),
                                          ctypes.c_void_p(B.data_ptr()), ctypes.byref(n), _stream_ptr(stream)),
           "cb_stats_reduce_centered")
    return n.value


def cb_ridge_solve_centered(A: torch.Tensor, B: torch.Tensor, mu: torch.Tensor, n_tokens: int, lambdas: Sequence[float],
                            flags: int, Wb: torch.Tensor, info: torch.Tensor, stream=None) -> None:
    n_maps, d, _ = A.shape
    lam = np.ascontiguousarray(lambdas, dtype=np.float32)
    assert A.dtype == torch.float32 and B.dtype == torch.float32 and mu.dtype == torch.float32
    assert Wb.dtype == torch.float32 and info.dtype == torch.int32
    assert A.is_contiguous() and B.is_contiguous() and mu.is_contiguous() and Wb.is_contiguous() and info.is_contiguous()
    assert B.shape == (n_maps, d, d) and mu.numel() == n_maps * (2 * d + 1)
    assert Wb.numel() == len(lam) * n_maps * (d + 1) * d and info.numel() == len(lam) * n_maps
    _check(lib().cb_ridge_solve_centered(ctypes.c_void_p(A.data_ptr()), ctypes.c_void_p(B.data_ptr()),
                                         ctypes.c_void_p(mu.data_ptr()), n_maps, d, ctypes.c_int64(n_tokens),
                                         lam.ctypes.data_as(ctypes.c_void_p), len(lam), ctypes.c_uint32(flags),
                                         ctypes.c_void_p(Wb.data_ptr()), ctypes.c_void_p(info.data_ptr()),
                                         _stream_ptr(stream)), "cb_ridge_solve_centered")


def cb_ridge_solve_large_workspace_bytes(P: int, d: int, n_systems: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().cb_ridge_solve_large_workspace_bytes(P, d, ctypes.c_int64(n_systems), ctypes.byref(n)),
           "cb_ridge_solve_large_workspace_bytes")
    return n.value


def cb_ridge_solve_large(G: torch.Tensor, C: torch.Tensor, n_tokens: int, lambdas: Sequence[float], flags: int,
                         Wb: torch.Tensor, info: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    """G [n_maps][P][P], C [n_maps][P][d] fp32; any P >= 2 (regressors over several source layers)."""
    n_maps, P, _ = G.shape
    d = C.shape[2]
    lam = np.ascontiguousarray(lambdas, dtype=np.float32)
    assert G.is_contiguous() and C.is_contiguous() and Wb.is_contiguous() and info.is_contiguous()
    assert G.dtype == torch.float32 and C.dtype == torch.float32 and Wb.dtype == torch.float32 and info.dtype == torch.int32
    assert C.shape == (n_maps, P, d) and Wb.numel() == len(lam) * n_maps * P * d and info.numel() == len(lam) * n_maps
    _check(lib().cb_ridge_solve_large(ctypes.c_void_p(G.data_ptr()), ctypes.c_void_p(C.data_ptr()), n_maps, P, d,
                                      ctypes.c_int64(n_tokens), lam.ctypes.data_as(ctypes.c_void_p), len(lam),
                                      ctypes.c_uint32(flags), ctypes.c_void_p(Wb.data_ptr()), ctypes.c_void_p(info.data_ptr()),
                                      ctypes.c_void_p(workspace.data_ptr()), ctypes.c_size_t(workspace.numel()),
                                      _stream_ptr(stream)), "cb_ridge_solve_large")


def cb_check_info(info: torch.Tensor, stream=None) -> None:
    bad = ctypes.c_int64(-1)
    _check(lib().cb_check_info(ctypes.c_void_p(info.data_ptr()), ctypes.c_int64(info.numel()), _stream_ptr(stream),
                               ctypes.byref(bad)), "cb_check_info (first bad index %d)" % bad.value)


def cb_apply(prob: Problem, Wb: torch.Tensor, src_k: torch.Tensor, src_v: torch.Tensor,
             tgt_k: torch.Tensor, tgt_v: torch.Tensor, stream=None) -> None:
    """Wb fp32 [n_maps][p][d]; source cache [Ls][T][Hs][d] bf16; outputs [Lt][T][Ht][d] bf16 or fp32."""
    sv = _kv_view(src_k, src_v)
    assert Wb.dtype == torch.float32 and Wb.is_contiguous()
    assert tgt_k.dtype == tgt_v.dtype and tgt_k.stride() == tgt_v.stride() and tgt_k.stride(3) == 1
    dt = {torch.bfloat16: CB_DTYPE_BF16, torch.float32: CB_DTYPE_F32}[tgt_k.dtype]
    _check(lib().cb_apply(ctypes.byref(prob.c), ctypes.c_void_p(Wb.data_ptr()), ctypes.byref(sv),
                          ctypes.c_void_p(tgt_k.data_ptr()), ctypes.c_void_p(tgt_v.data_ptr()),
                          ctypes.c_int64(tgt_k.stride(0)), ctypes.c_int64(tgt_k.stride(1)),
                          ctypes.c_int64(tgt_k.stride(2)), dt, _stream_ptr(stream)), "cb_apply")


def cb_apply_rope(prob: Problem, Wb: torch.Tensor, src_k: torch.Tensor, src_v: torch.Tensor,
                  tgt_k: torch.Tensor, tgt_v: torch.Tensor, positions: torch.Tensor,
                  rope_base_src: float, rope_base_tgt: float, stream=None) -> None:
    """As cb_apply for caches whose keys carry rotary embeddings; `positions` is a device int32 tensor [T]."""
    sv = _kv_view(src_k, src_v)
    assert Wb.dtype == torch.float32 and Wb.is_contiguous()
    assert tgt_k.dtype == tgt_v.dtype and tgt_k.stride() == tgt_v.stride() and tgt_k.stride(3) == 1
    assert positions.dtype == torch.int32 and positions.is_cuda and positions.is_contiguous()
    assert positions.numel() == src_k.shape[1]
    dt = {torch.bfloat16: CB_DTYPE_BF16, torch.float32: CB_DTYPE_F32}[tgt_k.dtype]
    _check(lib().cb_apply_rope(ctypes.byref(prob.c), ctypes.c_void_p(Wb.data_ptr()), ctypes.byref(sv),
                               ctypes.c_void_p(tgt_k.data_ptr()), ctypes.c_void_p(tgt_v.data_ptr()),
                               ctypes.c_int64(tgt_k.stride(0)), ctypes.c_int64(tgt_k.stride(1)),
                               ctypes.c_int64(tgt_k.stride(2)), dt, ctypes.c_void_p(positions.data_ptr()),
                               ctypes.c_double(rope_base_src), ctypes.c_double(rope_base_tgt), _stream_ptr(stream)),
           "cb_apply_rope")


def cb_stats_build_static(prob: Problem, src_k, src_v, tgt_k, tgt_v, w_k: torch.Tensor, w_v: torch.Tensor,
                          G: torch.Tensor, C: torch.Tensor, stream=None) -> None:
    """Statistics of one batch of rows into caller-owned G, C with the library's built-in scratch buffer: for
    callers that cannot allocate device memory for a workspace (see include/cb.h).  Same argument layout as
    cb_stats_accumulate; G [n_maps][p][p], C [n_maps][p][d] fp32 device tensors."""
    sv, tv = _kv_view(src_k, src_v), _kv_view(tgt_k, tgt_v)
    p, d = prob.ds + 1, prob.ds
    assert w_k.dtype == torch.float32 and w_v.dtype == torch.float32 and w_k.stride() == w_v.stride()
    assert G.dtype == torch.float32 and C.dtype == torch.float32 and G.is_contiguous() and C.is_contiguous()
    assert G.numel() == prob.n_maps * p * p and C.numel() == prob.n_maps * p * d
    _check(lib().cb_stats_build_static(ctypes.byref(prob.c), ctypes.byref(sv), ctypes.byref(tv),
                                       ctypes.c_void_p(w_k.data_ptr()), ctypes.c_void_p(w_v.data_ptr()),
                                       ctypes.c_int64(w_k.stride(0)), ctypes.c_int64(w_k.stride(1)),
                                       ctypes.c_void_p(G.data_ptr()), ctypes.c_void_p(C.data_ptr()),
                                       _stream_ptr(stream)), "cb_stats_build_static")


def cb_ess_weights(r_raw: torch.Tensor, p_width: int, w: torch.Tensor, alpha: Optional[torch.Tensor] = None, stream=None) -> None:
    """r_raw, w: fp32 device tensors [..., n_tokens] (rows = everything but the last axis, dense); alpha: [rows] or None."""
    assert r_raw.dtype == torch.float32 and w.dtype == torch.float32 and r_raw.is_contiguous() and w.is_contiguous()
    assert r_raw.shape == w.shape
    n = r_raw.shape[-1]
    rows = r_raw.numel() // n
    if alpha is not None:
        assert alpha.dtype == torch.float32 and alpha.numel() == rows and alpha.is_contiguous()
    _check(lib().cb_ess_weights(ctypes.c_void_p(r_raw.data_ptr()), rows, ctypes.c_int64(n), ctypes.c_int64(n),
                                ctypes.c_int64(p_width), ctypes.c_void_p(w.data_ptr()), ctypes.c_int64(n),
                                ctypes.c_void_p(alpha.data_ptr() if alpha is not None else 0), _stream_ptr(stream)),
           "cb_ess_weights")


class _FullHeadProblem(ctypes.Structure):
    _fields_ = [("Ls", ctypes.c_int32), ("Hs", ctypes.c_int32), ("ds", ctypes.c_int32),
                ("Lt", ctypes.c_int32), ("Ht", ctypes.c_int32), ("dt", ctypes.c_int32), ("k", ctypes.c_int32),
                ("layer_sets", ctypes.POINTER(ctypes.c_int32)), ("flags", ctypes.c_uint32)]


class FullHeadProblem:
    """Shapes plus the selected source layers [Lt][k] of the full-head contrast, mirroring cb_fullhead_problem."""

    def __init__(self, Ls, Hs, ds, Lt, Ht, dt, layer_sets, flags: int = 0):
        self.layer_sets = np.ascontiguousarray(layer_sets, dtype=np.int32)
        assert self.layer_sets.ndim == 2 and self.layer_sets.shape[0] == Lt
        self.k = int(self.layer_sets.shape[1])
        self.c = _FullHeadProblem(Ls, Hs, ds, Lt, Ht, dt, self.k,
                                  self.layer_sets.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), flags)
        self.Ls, self.Hs, self.ds, self.Lt, self.Ht, self.dt = Ls, Hs, ds, Lt, Ht, dt

    @property
    def pf(self) -> int:
        return self.k * self.Hs * self.ds + 1


def cb_fullhead_layer_sets(Ls: int, Lt: int, k: int = 4) -> np.ndarray:
    sets = np.empty((Lt, k), np.int32)
    _check(lib().cb_fullhead_layer_sets(Ls, Lt, k, sets.ctypes.data_as(ctypes.c_void_p)), "cb_fullhead_layer_sets")
    return sets


def cb_fullhead_workspace_bytes(prob: FullHeadProblem) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().cb_fullhead_workspace_bytes(ctypes.byref(prob.c), ctypes.byref(n)), "cb_fullhead_workspace_bytes")
    return n.value


def cb_fullhead_stats_accumulate(prob: FullHeadProblem, src_k, src_v, tgt_k, tgt_v, w_k: torch.Tensor, w_v: torch.Tensor,
                                 G: torch.Tensor, C: torch.Tensor, workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    """Adds this batch's full-head statistics to G [2][Lt][pf][pf] and C [2][Lt][Ht][pf][d] (fp32, zeroed by the
    caller before the first batch).  Weights [Lt][T] fp32."""
    sv, tv = _kv_view(src_k, src_v), _kv_view(tgt_k, tgt_v)
    assert w_k.dtype == torch.float32 and w_v.dtype == torch.float32 and w_k.dim() == 2 and w_k.stride() == w_v.stride()
    assert G.dtype == torch.float32 and C.dtype == torch.float32 and G.is_contiguous() and C.is_contiguous()
    assert G.numel() == 2 * prob.Lt * prob.pf * prob.pf and C.numel() == 2 * prob.Lt * prob.Ht * prob.pf * prob.ds
    if workspace is None:
        workspace = torch.empty(cb_fullhead_workspace_bytes(prob), dtype=torch.uint8, device=G.device)
    _check(lib().cb_fullhead_stats_accumulate(ctypes.byref(prob.c), ctypes.byref(sv), ctypes.byref(tv),
                                              ctypes.c_void_p(w_k.data_ptr()), ctypes.c_void_p(w_v.data_ptr()),
                                              ctypes.c_int64(w_k.stride(0)), ctypes.c_void_p(G.data_ptr()),
                                              ctypes.c_void_p(C.data_ptr()), ctypes.c_void_p(workspace.data_ptr()),
                                              ctypes.c_size_t(workspace.numel()), _stream_ptr(stream)),
           "cb_fullhead_stats_accumulate")


def cb_multilayer_stats_accumulate(prob: FullHeadProblem, src_head, src_k, src_v, tgt_k, tgt_v, w_k: torch.Tensor,
                                   w_v: torch.Tensor, G: torch.Tensor, C: torch.Tensor, stream=None) -> None:
    """Head-local statistics over k selected layers: adds to G [n_maps][P][P], C [n_maps][P][d], P = k*d + 1.
    Weights [Lt][Ht][T] fp32."""
    sv, tv = _kv_view(src_k, src_v), _kv_view(tgt_k, tgt_v)
    sh = np.ascontiguousarray(src_head, dtype=np.int32)
    P = prob.k * prob.ds + 1
    n_maps = 2 * prob.Lt * prob.Ht
    assert w_k.dtype == torch.float32 and w_v.dtype == torch.float32 and w_k.dim() == 3 and w_k.stride() == w_v.stride()
    assert G.dtype == torch.float32 and C.dtype == torch.float32 and G.is_contiguous() and C.is_contiguous()
    assert G.numel() == n_maps * P * P and C.numel() == n_maps * P * prob.ds
    n = ctypes.c_size_t(0)
    _check(lib().cb_multilayer_workspace_bytes(ctypes.byref(prob.c), ctypes.byref(n)), "cb_multilayer_workspace_bytes")
    ws = torch.empty(n.value, dtype=torch.uint8, device=G.device)
    _check(lib().cb_multilayer_stats_accumulate(ctypes.byref(prob.c), sh.ctypes.data_as(ctypes.c_void_p), ctypes.byref(sv),
                                                ctypes.byref(tv), ctypes.c_void_p(w_k.data_ptr()), ctypes.c_void_p(w_v.data_ptr()),
                                                ctypes.c_int64(w_k.stride(0)), ctypes.c_int64(w_k.stride(1)),
                                                ctypes.c_void_p(G.data_ptr()), ctypes.c_void_p(C.data_ptr()),
                                                ctypes.c_void_p(ws.data_ptr()), ctypes.c_size_t(ws.numel()), _stream_ptr(stream)),
           "cb_multilayer_stats_accumulate")


def cb_apply_multilayer(prob: FullHeadProblem, src_head, Wb: torch.Tensor, src_k, src_v, tgt_k, tgt_v, stream=None) -> None:
    """Wb fp32 [n_maps][k*d + 1][d]; source cache [Ls][T][Hs][d] bf16; outputs [Lt][T][Ht][d] bf16 or fp32."""
    sv = _kv_view(src_k, src_v)
    sh = np.ascontiguousarray(src_head, dtype=np.int32)
    assert Wb.dtype == torch.float32 and Wb.is_contiguous()
    assert tgt_k.dtype == tgt_v.dtype and tgt_k.stride() == tgt_v.stride() and tgt_k.stride(3) == 1
    dt = {torch.bfloat16: CB_DTYPE_BF16, torch.float32: CB_DTYPE_F32}[tgt_k.dtype]
    n = ctypes.c_size_t(0)
    _check(lib().cb_apply_multilayer_workspace_bytes(ctypes.byref(prob.c), ctypes.byref(n)), "cb_apply_multilayer_workspace_bytes")
    ws = torch.empty(n.value, dtype=torch.uint8, device=Wb.device)
    _check(lib().cb_apply_multilayer(ctypes.byref(prob.c), sh.ctypes.data_as(ctypes.c_void_p), ctypes.c_void_p(Wb.data_ptr()),
                                     ctypes.byref(sv), ctypes.c_void_p(tgt_k.data_ptr()), ctypes.c_void_p(tgt_v.data_ptr()),
                                     ctypes.c_int64(tgt_k.stride(0)), ctypes.c_int64(tgt_k.stride(1)), ctypes.c_int64(tgt_k.stride(2)),
                                     dt, ctypes.c_void_p(ws.data_ptr()), ctypes.c_size_t(ws.numel()), _stream_ptr(stream)),
           "cb_apply_multilayer")


def cb_device_status(ctx: Context, stream=None) -> None:
    _check(lib().cb_device_status(ctx.handle, _stream_ptr(stream)), "cb_device_status")


def cb_last_device_status(stream=None) -> None:
    _check(lib().cb_last_device_status(_stream_ptr(stream)), "cb_last_device_status")


def cb_test_hooks(poll_limit: int = 0, starve_producer: bool = False) -> None:
    _check(lib().cb_test_hooks(ctypes.c_uint32(poll_limit), ctypes.c_int32(1 if starve_producer else 0)), "cb_test_hooks")


def cb_launch_count() -> int:
    return int(lib().cb_launch_count())
