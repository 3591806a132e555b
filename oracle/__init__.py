"""CPU oracle (fp64) for head-local weighted affine ridge mapping of KV caches.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library never imports or calls it, and
this package imports nothing from the CUDA package.

The arithmetic lives in ``cb_oracle.c`` (plain C loops in fp64, one map per
OpenMP thread); this file only marshals numpy arrays through ctypes.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cb_oracle.c")
_LIB = os.path.join(_HERE, "libcb_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no BLAS, no tuning flags beyond -O2)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.orc_work_list.restype = ctypes.c_int32
        _lib.orc_ridge_solve.restype = ctypes.c_int32
        _lib.orc_ridge_centered.restype = ctypes.c_int32
    return _lib


def n_threads() -> int:
    """Threads the OpenMP loops will use (the cores this process may run on)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    return len(os.sched_getaffinity(0))


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i64(v) -> ctypes.c_int64:
    return ctypes.c_int64(int(v))


def _i32(v) -> ctypes.c_int32:
    return ctypes.c_int32(int(v))


# ----------------------------------------------------------------------------- bf16
def bf16_decode(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().orc_bf16_decode(_p(bits), _p(out), _i64(bits.size))
    return out


def bf16_encode(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    _load().orc_bf16_encode(_p(x), _p(out), _i64(x.size))
    return out


# ----------------------------------------------------------------------------- bookkeeping
def head_map(Ls: int, Hs: int, Lt: int, Ht: int) -> Tuple[np.ndarray, np.ndarray]:
    """(src_layer[Lt], src_head[Ht]) int32: nearest-depth layer, aligned head."""
    sl = np.empty(Lt, dtype=np.int32)
    sh = np.empty(Ht, dtype=np.int32)
    _load().orc_head_map(_i32(Ls), _i32(Hs), _i32(Lt), _i32(Ht), _p(sl), _p(sh))
    return sl, sh


def work_list(Ls: int, Hs: int, Lt: int, Ht: int, src_layer: np.ndarray, src_head: np.ndarray):
    """Static gather schedule: (item_comp, item_layer, item_head, item_begin, item_maps)."""
    src_layer = np.ascontiguousarray(src_layer, dtype=np.int32)
    src_head = np.ascontiguousarray(src_head, dtype=np.int32)
    cap = 2 * Ls * Hs
    ic = np.empty(cap, np.int32)
    il = np.empty(cap, np.int32)
    ih = np.empty(cap, np.int32)
    ib = np.empty(cap + 1, np.int32)
    im = np.empty(2 * Lt * Ht, np.int32)
    n = _load().orc_work_list(_i32(Ls), _i32(Hs), _i32(Lt), _i32(Ht), _p(src_layer), _p(src_head),
                              _p(ic), _p(il), _p(ih), _p(ib), _p(im))
    return ic[:n].copy(), il[:n].copy(), ih[:n].copy(), ib[:n + 1].copy(), im[:ib[n]].copy()


# ----------------------------------------------------------------------------- statistics
def stats_f64(X: np.ndarray, Y: np.ndarray, w: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """G [p][p], C [p][d] of one map from fp64 rows X, Y [n][d] and weights w [n]."""
    X = np.ascontiguousarray(X, dtype=np.float64)
    Y = np.ascontiguousarray(Y, dtype=np.float64)
    w = np.ascontiguousarray(w, dtype=np.float64)
    n, d = X.shape
    assert Y.shape == (n, d) and w.shape == (n,)
    G = np.empty((d + 1, d + 1), np.float64)
    C = np.empty((d + 1, d), np.float64)
    _load().orc_stats_f64(_p(X), _p(Y), _p(w), _i64(n), _i32(d), _p(G), _p(C))
    return G, C


def _trace_strides(a: np.ndarray) -> Tuple[int, int, int]:
    """Element strides (layer, token, head) of a [L][T][H][d] uint16 array with contiguous channels."""
    assert a.dtype == np.uint16 and a.ndim == 4 and a.strides[3] == 2
    return a.strides[0] // 2, a.strides[1] // 2, a.strides[2] // 2


def stats_traces(src_k: np.ndarray, src_v: np.ndarray, tgt_k: np.ndarray, tgt_v: np.ndarray,
                 w_k: np.ndarray, w_v: np.ndarray, src_layer: np.ndarray, src_head: np.ndarray,
                 maps: Optional[Sequence[int]] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Statistics of the selected maps (all by default) from bf16-bit traces [L][T][H][d] (uint16)
    and fp32 weights [Lt][Ht][T].  Returns fp64 G [n_sel][p][p], C [n_sel][p][d]."""
    Lt, T, Ht, d = tgt_k.shape
    assert src_v.shape == src_k.shape and tgt_v.shape == tgt_k.shape and src_k.shape[1] == T
    assert w_k.dtype == np.float32 and w_v.dtype == np.float32
    assert w_k.shape == (Lt, Ht, T) and w_v.shape == (Lt, Ht, T)
    assert w_k.strides[2] == 4 and w_v.strides == w_k.strides
    src_layer = np.ascontiguousarray(src_layer, dtype=np.int32)
    src_head = np.ascontiguousarray(src_head, dtype=np.int32)
    if maps is None:
        maps = np.arange(2 * Lt * Ht, dtype=np.int32)
    maps = np.ascontiguousarray(maps, dtype=np.int32)
    s = _trace_strides(src_k)
    assert _trace_strides(src_v) == s
    t = _trace_strides(tgt_k)
    assert _trace_strides(tgt_v) == t
    p = d + 1
    G = np.empty((len(maps), p, p), np.float64)
    C = np.empty((len(maps), p, d), np.float64)
    _load().orc_stats_traces(_p(src_k), _p(src_v), _i64(s[0]), _i64(s[1]), _i64(s[2]),
                             _p(tgt_k), _p(tgt_v), _i64(t[0]), _i64(t[1]), _i64(t[2]),
                             _p(w_k), _p(w_v), _i64(w_k.strides[0] // 4), _i64(w_k.strides[1] // 4),
                             _i64(T), _i32(d), _i32(Lt), _i32(Ht), _p(src_layer), _p(src_head),
                             _p(maps), _i32(len(maps)), _p(G), _p(C))
    return G, C


# ----------------------------------------------------------------------------- ridge
def ridge_solve(G: np.ndarray, C: np.ndarray, n: int, lam: float, raw_lambda: bool = False):
    """Theta = [W; b] ([..][p][d]) and info for one map or a batch of maps."""
    G = np.ascontiguousarray(G, dtype=np.float64)
    C = np.ascontiguousarray(C, dtype=np.float64)
    single = G.ndim == 2
    if single:
        G, C = G[None], C[None]
    n_maps, p, _ = G.shape
    d = p - 1
    assert C.shape == (n_maps, p, d)
    Theta = np.empty((n_maps, p, d), np.float64)
    info = np.empty(n_maps, np.int32)
    _load().orc_ridge_solve_batch(_p(G), _p(C), _i32(n_maps), _i32(d), _i64(n), ctypes.c_double(lam),
                                  _i32(1 if raw_lambda else 0), _p(Theta), _p(info))
    if single:
        return Theta[0], int(info[0])
    return Theta, info


def ridge_centered(X: np.ndarray, Y: np.ndarray, w: np.ndarray, lam: float):
    """The centred two-pass estimator with mean-one weights, exactly as the paper writes it."""
    X = np.ascontiguousarray(X, dtype=np.float64)
    Y = np.ascontiguousarray(Y, dtype=np.float64)
    w = np.ascontiguousarray(w, dtype=np.float64)
    n, d = X.shape
    Theta = np.empty((d + 1, d), np.float64)
    info = _load().orc_ridge_centered(_p(X), _p(Y), _p(w), _i64(n), _i32(d), ctypes.c_double(lam), _p(Theta))
    return Theta, int(info)


# ----------------------------------------------------------------------------- two-pass centred construction
def _trace_args(src_k, src_v, tgt_k, tgt_v, w_k, w_v, src_layer, src_head, maps):
    Lt, T, Ht, d = tgt_k.shape
    assert src_v.shape == src_k.shape and tgt_v.shape == tgt_k.shape and src_k.shape[1] == T
    assert w_k.dtype == np.float32 and w_v.dtype == np.float32
    assert w_k.shape == (Lt, Ht, T) and w_v.shape == (Lt, Ht, T)
    assert w_k.strides[2] == 4 and w_v.strides == w_k.strides
    src_layer = np.ascontiguousarray(src_layer, dtype=np.int32)
    src_head = np.ascontiguousarray(src_head, dtype=np.int32)
    if maps is None:
        maps = np.arange(2 * Lt * Ht, dtype=np.int32)
    maps = np.ascontiguousarray(maps, dtype=np.int32)
    s = _trace_strides(src_k)
    assert _trace_strides(src_v) == s
    t = _trace_strides(tgt_k)
    assert _trace_strides(tgt_v) == t
    keep = (src_layer, src_head, maps)
    args = [_p(src_k), _p(src_v), _i64(s[0]), _i64(s[1]), _i64(s[2]),
            _p(tgt_k), _p(tgt_v), _i64(t[0]), _i64(t[1]), _i64(t[2]),
            _p(w_k), _p(w_v), _i64(w_k.strides[0] // 4), _i64(w_k.strides[1] // 4),
            _i64(T), _i32(d), _i32(Lt), _i32(Ht), _p(src_layer), _p(src_head), _p(maps), _i32(len(maps))]
    return args, keep, len(maps), d


def weighted_sums_traces(src_k, src_v, tgt_k, tgt_v, w_k, w_v, src_layer, src_head, maps=None):
    """First pass of the two-pass construction on one chunk: sum w x [n_sel][d], sum w y [n_sel][d], sum w [n_sel]
    (fp64).  Sums of several chunks add; the means are sum / s_w."""
    args, keep, n_sel, d = _trace_args(src_k, src_v, tgt_k, tgt_v, w_k, w_v, src_layer, src_head, maps)
    sx = np.empty((n_sel, d), np.float64)
    sy = np.empty((n_sel, d), np.float64)
    sw = np.empty(n_sel, np.float64)
    _load().orc_means_traces(*args, _p(sx), _p(sy), _p(sw))
    return sx, sy, sw


def centered_stats_traces(src_k, src_v, tgt_k, tgt_v, w_k, w_v, src_layer, src_head, mu_x, mu_y, maps=None):
    """Second pass on one chunk: A = sum w (x - mu_x)(x - mu_x)^T, B = sum w (x - mu_x)(y - mu_y)^T, [n_sel][d][d]."""
    args, keep, n_sel, d = _trace_args(src_k, src_v, tgt_k, tgt_v, w_k, w_v, src_layer, src_head, maps)
    mu_x = np.ascontiguousarray(mu_x, dtype=np.float64)
    mu_y = np.ascontiguousarray(mu_y, dtype=np.float64)
    assert mu_x.shape == (n_sel, d) and mu_y.shape == (n_sel, d)
    A = np.empty((n_sel, d, d), np.float64)
    B = np.empty((n_sel, d, d), np.float64)
    _load().orc_centered_stats_traces(*args, _p(mu_x), _p(mu_y), _p(A), _p(B))
    return A, B


def ridge_solve_centered(A, B, mu_x, mu_y, s_w, n: int, lam: float, raw_lambda: bool = False):
    """Theta = [W; b] from centred statistics: W = (A + lambda_eff I)^-1 B, b = mu_y - mu_x W (one map or a batch)."""
    A = np.ascontiguousarray(A, dtype=np.float64)
    B = np.ascontiguousarray(B, dtype=np.float64)
    mu_x = np.ascontiguousarray(mu_x, dtype=np.float64)
    mu_y = np.ascontiguousarray(mu_y, dtype=np.float64)
    single = A.ndim == 2
    if single:
        A, B, mu_x, mu_y, s_w = A[None], B[None], mu_x[None], mu_y[None], np.array([s_w], np.float64)
    s_w = np.ascontiguousarray(s_w, dtype=np.float64)
    n_maps, d, _ = A.shape
    Theta = np.empty((n_maps, d + 1, d), np.float64)
    info = np.empty(n_maps, np.int32)
    lib = _load()
    for m in range(n_maps):
        info[m] = lib.orc_ridge_solve_centered(_p(A[m]), _p(B[m]), _p(mu_x[m]), _p(mu_y[m]), ctypes.c_double(s_w[m]),
                                               _i32(d), _i64(n), ctypes.c_double(lam), _i32(1 if raw_lambda else 0),
                                               _p(Theta[m]))
    if single:
        return Theta[0], int(info[0])
    return Theta, info


# ----------------------------------------------------------------------------- rotary embedding at the boundary
def rope_rotate(x: np.ndarray, pos: np.ndarray, base: float, inverse: bool = False) -> np.ndarray:
    """Rotate-half RoPE of rows x [n][d] (fp64) at integer positions pos [n]; inverse removes the embedding."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    n, d = x.shape
    assert pos.shape == (n,) and d % 2 == 0
    out = np.empty_like(x)
    _load().orc_rope_rotate(_p(x), _p(out), _i64(n), _i32(d), _p(pos), ctypes.c_double(base), _i32(1 if inverse else 0))
    return out


def apply_rope_rows(x_bits: np.ndarray, Theta: np.ndarray, pos: np.ndarray, base_src: float, base_tgt: float) -> np.ndarray:
    """Key rows through a map in content coordinates (Section 3.1): remove the source model's rotary embedding, apply
    y = x W + b, restore the target model's.  x_bits [n][d] bf16 bit patterns, Theta [d+1][d] (W then b); fp64 out."""
    x = bf16_decode(np.ascontiguousarray(x_bits)).reshape(x_bits.shape)
    d = x.shape[1]
    Theta = np.asarray(Theta, dtype=np.float64)
    content = rope_rotate(x, pos, base_src, inverse=True)
    mapped = content @ Theta[:d] + Theta[d]
    return rope_rotate(mapped, pos, base_tgt, inverse=False)


# ----------------------------------------------------------------------------- layer selector
def probe_r2(X: np.ndarray, Y: np.ndarray, w: np.ndarray, lambda_rel: float = 0.0):
    """Held-in R^2 (pooled over channels) of the centred weighted least-squares probe y ~ x W + b."""
    X = np.ascontiguousarray(X, dtype=np.float64)
    Y = np.ascontiguousarray(Y, dtype=np.float64)
    w = np.ascontiguousarray(w, dtype=np.float64)
    n, d = X.shape
    r2 = ctypes.c_double(0.0)
    lib = _load()
    lib.orc_probe_r2.restype = ctypes.c_int32
    info = lib.orc_probe_r2(_p(X), _p(Y), _p(w), _i64(n), _i32(d), ctypes.c_double(lambda_rel), ctypes.byref(r2))
    return r2.value, int(info)


def layer_scores(src_k, src_v, tgt_k, tgt_v, w_k, w_v, src_head, lambda_rel: float = 0.0, layers=None) -> np.ndarray:
    """scores [Lt][Ls]: mean over KV heads and K/V of the probe R^2 of (source layer j, head a(h)) -> (target layer l,
    head h).  Inputs as bf16 bit patterns [L][T][H][d] and fp32 weights [Lt][Ht][T]; `layers` restricts the target
    layers (others stay NaN)."""
    Ls, T, Hs, d = src_k.shape
    Lt, _, Ht, _ = tgt_k.shape
    dec = [bf16_decode(np.ascontiguousarray(a)).reshape(a.shape) for a in (src_k, src_v, tgt_k, tgt_v)]
    scores = np.full((Lt, Ls), np.nan)
    for l in (range(Lt) if layers is None else layers):
        for j in range(Ls):
            acc = 0.0
            for comp in range(2):
                for h in range(Ht):
                    X = dec[comp][j, :, src_head[h], :]
                    Y = dec[2 + comp][l, :, h, :]
                    r2, _ = probe_r2(X, Y, (w_v if comp else w_k)[l, h].astype(np.float64), lambda_rel)
                    acc += r2
            scores[l, j] = acc / (2 * Ht)
    return scores


def rank_layers(scores: np.ndarray, k: int) -> np.ndarray:
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    Lt, Ls = scores.shape
    sets = np.empty((Lt, k), np.int32)
    _load().orc_rank_layers(_p(scores), _i32(Lt), _i32(Ls), _i32(k), _p(sets))
    return sets


# ----------------------------------------------------------------------------- apply
def apply_maps(src_k: np.ndarray, src_v: np.ndarray, Theta: np.ndarray, Lt: int, Ht: int,
               src_layer: np.ndarray, src_head: np.ndarray, maps: Optional[Sequence[int]] = None,
               want_f64: bool = True, want_bf16: bool = True):
    """Map a source cache [Ls][T][Hs][d] (bf16 bits) to a target cache [Lt][T][Ht][d].
    Returns ((K, V) fp64 or None, (K, V) bf16 bits or None); entries of unselected maps are zero."""
    Ls, T, Hs, d = src_k.shape
    p = d + 1
    Theta = np.ascontiguousarray(Theta, dtype=np.float64)
    assert Theta.shape == (2 * Lt * Ht, p, d)
    src_layer = np.ascontiguousarray(src_layer, dtype=np.int32)
    src_head = np.ascontiguousarray(src_head, dtype=np.int32)
    if maps is None:
        maps = np.arange(2 * Lt * Ht, dtype=np.int32)
    maps = np.ascontiguousarray(maps, dtype=np.int32)
    s = _trace_strides(src_k)
    assert _trace_strides(src_v) == s
    shape = (Lt, T, Ht, d)
    ok = np.zeros(shape, np.float64) if want_f64 else None
    ov = np.zeros(shape, np.float64) if want_f64 else None
    bk = np.zeros(shape, np.uint16) if want_bf16 else None
    bv = np.zeros(shape, np.uint16) if want_bf16 else None
    _load().orc_apply(_p(src_k), _p(src_v), _i64(s[0]), _i64(s[1]), _i64(s[2]), _i64(T), _i32(d),
                      _i32(Lt), _i32(Ht), _p(src_layer), _p(src_head), _p(Theta), _p(maps), _i32(len(maps)),
                      _p(ok), _p(ov), _p(bk), _p(bv), _i64(T * Ht * d), _i64(Ht * d), _i64(d))
    return ((ok, ov) if want_f64 else None), ((bk, bv) if want_bf16 else None)


# ----------------------------------------------------------------------------- ESS floor on the weights
def ess_weights(r_raw: np.ndarray, p_width: int):
    """Shrink mean-normalised sensitivities toward uniform so that the Kish effective sample size stays at or above
    min(n, 2 p).  r_raw: [n] or [maps][n].  Returns (w, alpha, cv2) with matching leading shape."""
    r = np.ascontiguousarray(r_raw, dtype=np.float64)
    single = r.ndim == 1
    if single:
        r = r[None]
    w = np.empty_like(r)
    alpha = np.empty(len(r))
    cv2 = np.empty(len(r))
    lib = _load()
    lib.orc_ess_weights.restype = ctypes.c_double
    for i in range(len(r)):
        c = ctypes.c_double(0.0)
        alpha[i] = lib.orc_ess_weights(_p(r[i]), _i64(r.shape[1]), _i64(p_width), _p(w[i]), ctypes.byref(c))
        cv2[i] = c.value
    if single:
        return w[0], float(alpha[0]), float(cv2[0])
    return w, alpha, cv2


# ----------------------------------------------------------------------------- full-head contrast
def fullhead_layer_sets(Ls: int, Lt: int, k: int = 4) -> np.ndarray:
    """int32 [Lt][k]: k consecutive source layers around the nearest-depth layer, clipped into range."""
    sets = np.empty((Lt, k), np.int32)
    _load().orc_fullhead_layer_sets(_i32(Ls), _i32(Lt), _i32(k), _p(sets))
    return sets


def fullhead_stats(src: np.ndarray, tgt: np.ndarray, w: np.ndarray, l: int, layer_set: Sequence[int]):
    """Full-head statistics of one (component, target layer l): src/tgt are that component's bf16-bit traces
    [L][T][H][d], w fp32 [T].  Returns fp64 G [pf][pf] (pf = k*Hs*d + 1) and C [Ht][pf][d]."""
    Ls, T, Hs, d = src.shape
    Lt, T2, Ht, d2 = tgt.shape
    assert T2 == T and d2 == d and w.dtype == np.float32 and w.shape == (T,) and w.strides[0] == 4
    ls = np.ascontiguousarray(layer_set, dtype=np.int32)
    pf = len(ls) * Hs * d + 1
    G = np.empty((pf, pf), np.float64)
    C = np.empty((Ht, pf, d), np.float64)
    s, t = _trace_strides(src), _trace_strides(tgt)
    _load().orc_fullhead_stats(_p(src), _i64(s[0]), _i64(s[1]), _i64(s[2]), _p(tgt), _i64(t[0]), _i64(t[1]), _i64(t[2]),
                               _p(w), _i64(T), _i32(d), _i32(Hs), _i32(Ht), _i32(l), _p(ls), _i32(len(ls)), _p(G), _p(C))
    return G, C


def multilayer_stats(src: np.ndarray, tgt: np.ndarray, w: np.ndarray, l: int, h: int, g: int, layer_set: Sequence[int]):
    """Head-local statistics over several selected layers for one map (component given by src/tgt): the feature
    concatenates source head g of the layers in layer_set; target (l, h); w fp32 [T].  G [P][P], C [P][d], P = k*d + 1."""
    G, C = fullhead_stats(src[:, :, g:g + 1, :], tgt[:, :, h:h + 1, :], w, l, layer_set)
    return G, C[0]


def apply_multilayer(src: np.ndarray, Theta: np.ndarray, layer_set: Sequence[int], g: int):
    """Affine apply for one map over several source layers: rows x_t = concat_f src[layer_set[f]][t][g] (bf16 bits,
    widened exactly), y_t = x_t W + b in fp64 (a plain fp64 matrix product).  Returns (fp64 [T][d], bf16 bits)."""
    X = np.concatenate([bf16_decode(np.ascontiguousarray(src[j, :, g, :])) for j in layer_set], axis=1)
    Theta = np.asarray(Theta, dtype=np.float64)
    y = X @ Theta[:-1] + Theta[-1]
    return y, bf16_encode(y)


def ridge_solve_general(G: np.ndarray, C: np.ndarray, n: int, lam: float, raw_lambda: bool = False):
    """Theta [p][dy] and info for one system of any width (bias entry last, not penalised)."""
    G = np.ascontiguousarray(G, dtype=np.float64)
    C = np.ascontiguousarray(C, dtype=np.float64)
    p, dy = C.shape
    assert G.shape == (p, p)
    Theta = np.empty((p, dy), np.float64)
    lib = _load()
    lib.orc_ridge_solve_pd.restype = ctypes.c_int32
    info = lib.orc_ridge_solve_pd(_p(G), _p(C), _i32(p), _i32(dy), _i64(n), ctypes.c_double(lam),
                                  _i32(1 if raw_lambda else 0), _p(Theta))
    return Theta, int(info)


# ----------------------------------------------------------------------------- artifact size
def coefficient_counts(Lt: int, Ht: int, Hs: int, k: int, ds: int, dt: int):
    """Non-bias coefficient counts over K and V (Section 3.2): (C_full, C_local, number of bias entries).
    C_full = 2 L_t H_t (k H_s d_s) d_t,  C_local = 2 L_t H_t (k d_s) d_t."""
    c_full = 2 * Lt * Ht * (k * Hs * ds) * dt
    c_local = 2 * Lt * Ht * (k * ds) * dt
    n_bias = 2 * Lt * Ht * dt
    return c_full, c_local, n_bias
