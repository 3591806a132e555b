"""Error behaviour of the device entry points that can be checked without a GPU: argument errors are status codes
found on the host before anything is launched, and without a CUDA device the calls fail loudly (no CPU fallback)."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2609_00891_b200 import binding as cb
from paper_2609_00891_b200 import build as cb_build

pytestmark = pytest.mark.skipif(torch.cuda.is_available(), reason="host-only behaviour; the GPU suite covers the rest")


@pytest.fixture(scope="module", autouse=True)
def _built():
    cb_build.build()


def _view(L, H, d, T, ptr=0x1000, st=None, sh=None, sl=None):
    st = H * d if st is None else st
    sh = d if sh is None else sh
    sl = T * H * d if sl is None else sl
    return cb._KvView(ptr, ptr, L, H, d, T, sl, st, sh)


def _apply(prob, view, Wb=0x2000, out=0x3000, strides=None, dtype=cb.CB_DTYPE_BF16):
    s = strides or (view.n_tokens * prob.Ht * prob.dt, prob.Ht * prob.dt, prob.dt)
    return cb.lib().cb_apply(ctypes.byref(prob.c), ctypes.c_void_p(Wb), ctypes.byref(view), ctypes.c_void_p(out),
                             ctypes.c_void_p(out), ctypes.c_int64(s[0]), ctypes.c_int64(s[1]), ctypes.c_int64(s[2]),
                             dtype, ctypes.c_void_p(0))


def test_apply_argument_errors_are_reported_before_any_launch():
    sl, sh = cb.cb_head_map_nearest(4, 2, 6, 2)
    prob = cb.Problem(4, 2, 128, 6, 2, 128, sl, sh)
    before = cb.cb_launch_count()
    assert _apply(prob, _view(4, 2, 128, 0)) == cb.CB_OK                              # empty cache: no-op
    assert _apply(prob, _view(5, 2, 128, 64)) == cb.CB_ERR_INVALID_ARG               # wrong layer count
    assert _apply(prob, _view(4, 2, 128, 64, ptr=0x1004)) == cb.CB_ERR_INVALID_ARG   # misaligned cache pointer
    assert _apply(prob, _view(4, 2, 128, 64, st=2 * 128 + 4)) == cb.CB_ERR_INVALID_ARG   # stride not a multiple of 8
    assert _apply(prob, _view(4, 2, 128, 64), Wb=0) == cb.CB_ERR_INVALID_ARG         # null maps
    assert _apply(prob, _view(4, 2, 128, 64), out=0x3008) == cb.CB_ERR_INVALID_ARG   # misaligned output
    assert _apply(prob, _view(4, 2, 128, 64), dtype=7) == cb.CB_ERR_INVALID_ARG      # unknown output type
    assert _apply(prob, _view(4, 2, 128, 1 << 31)) == cb.CB_ERR_UNSUPPORTED          # too many rows for one call
    # a broadcast view (stride 0 over several heads or layers, e.g. an expanded one-head cache) cannot be tiled
    assert _apply(prob, _view(4, 2, 128, 64, sh=0)) == cb.CB_ERR_UNSUPPORTED
    assert _apply(prob, _view(4, 2, 128, 64, sl=0)) == cb.CB_ERR_UNSUPPORTED
    assert _apply(prob, _view(4, 2, 128, 64), strides=(64 * 2 * 128, 2 * 128, 0)) == cb.CB_ERR_UNSUPPORTED   # output too
    assert _apply(prob, _view(4, 2, 128, 64), strides=(0, 2 * 128, 128)) == cb.CB_ERR_UNSUPPORTED
    sl1, sh1 = cb.cb_head_map_nearest(1, 1, 6, 2)
    one = cb.Problem(1, 1, 128, 6, 2, 128, sl1, sh1)
    assert _apply(one, _view(1, 1, 128, 64, sh=0, sl=0)) == cb.CB_ERR_CUDA           # size-1 dimensions: any stride; passes the checks
    assert cb.cb_launch_count() == before


def test_solve_argument_errors():
    lam = np.array([1e-2], np.float32)
    call = lambda G, C, n_maps, d, n, nl, Wb, info: cb.lib().cb_ridge_solve(
        ctypes.c_void_p(G), ctypes.c_void_p(C), n_maps, d, ctypes.c_int64(n), lam.ctypes.data_as(ctypes.c_void_p), nl,
        ctypes.c_uint32(0), ctypes.c_void_p(Wb), ctypes.c_void_p(info), ctypes.c_void_p(0))
    assert call(0, 0x10, 4, 128, 100, 1, 0x20, 0x30) == cb.CB_ERR_INVALID_ARG
    assert call(0x10, 0x10, 4, 96, 100, 1, 0x20, 0x30) == cb.CB_ERR_UNSUPPORTED
    assert call(0x10, 0x10, 4, 128, 100, 0, 0x20, 0x30) == cb.CB_ERR_INVALID_ARG
    assert call(0x10, 0x10, 0, 128, 100, 1, 0x20, 0x30) == cb.CB_OK                   # no systems: nothing to do
    bad = np.array([-1.0], np.float32)
    assert cb.lib().cb_ridge_solve(ctypes.c_void_p(0x10), ctypes.c_void_p(0x10), 4, 128, ctypes.c_int64(10),
                                   bad.ctypes.data_as(ctypes.c_void_p), 1, ctypes.c_uint32(0), ctypes.c_void_p(0x20),
                                   ctypes.c_void_p(0x30), ctypes.c_void_p(0)) == cb.CB_ERR_INVALID_ARG


def test_without_a_device_the_path_fails_loudly():
    sl, sh = cb.cb_head_map_nearest(2, 2, 2, 2)
    prob = cb.Problem(2, 2, 64, 2, 2, 64, sl, sh)
    h = ctypes.c_void_p()
    ws = np.zeros(cb.cb_workspace_bytes(prob) + 256, np.uint8)
    addr = (ws.ctypes.data + 255) // 256 * 256
    st = cb.lib().cb_create(ctypes.byref(prob.c), ctypes.c_void_p(addr), ctypes.c_size_t(cb.cb_workspace_bytes(prob)), ctypes.byref(h))
    assert st == cb.CB_ERR_CUDA and not h                                            # no context, no fallback
    assert _apply(prob, _view(2, 2, 64, 64)) == cb.CB_ERR_CUDA
    assert "CUDA" in cb.status_string(cb.CB_ERR_CUDA)
    with pytest.raises(cb.CbError):
        cb.cb_create(prob, workspace=torch.zeros(16, dtype=torch.uint8))              # workspace too small


def test_static_entry_point_shares_the_argument_checks():
    sl, sh = cb.cb_head_map_nearest(4, 2, 6, 2)
    prob = cb.Problem(4, 2, 128, 6, 2, 128, sl, sh)

    def call(vs, vt, wk=0x100, wv=0x100):
        return cb.lib().cb_stats_build_static(ctypes.byref(prob.c), ctypes.byref(vs), ctypes.byref(vt), ctypes.c_void_p(wk),
                                              ctypes.c_void_p(wv), ctypes.c_int64(2 * 64), ctypes.c_int64(64),
                                              ctypes.c_void_p(0x200), ctypes.c_void_p(0x300), ctypes.c_void_p(0))
    ok_s, ok_t = _view(4, 2, 128, 64), _view(6, 2, 128, 64)
    assert call(ok_s, ok_t, wk=0x102) == cb.CB_ERR_INVALID_ARG                         # weights must be 4-byte aligned
    assert call(_view(4, 2, 128, 64, sh=-128), ok_t) == cb.CB_ERR_INVALID_ARG          # negative stride
    assert call(_view(4, 2, 128, 64, sh=0), ok_t) == cb.CB_ERR_UNSUPPORTED             # broadcast over two heads
    assert call(ok_s, _view(6, 2, 128, 32)) == cb.CB_ERR_INVALID_ARG                   # token counts differ
    assert call(ok_s, ok_t) == cb.CB_ERR_CUDA                                          # passes the checks; no device here


def test_checkpoint_calls_reject_a_missing_context():
    null = ctypes.c_void_p(0)
    n = ctypes.c_size_t(0)
    t = ctypes.c_int64(0)
    assert cb.lib().cb_stats_state_bytes(null, ctypes.byref(n)) == cb.CB_ERR_STATE
    assert cb.lib().cb_stats_export(null, ctypes.c_void_p(0x100), ctypes.c_size_t(64), ctypes.byref(t), null) == cb.CB_ERR_STATE
    assert cb.lib().cb_stats_import(null, ctypes.c_void_p(0x100), ctypes.c_size_t(64), ctypes.c_int64(0), null) == cb.CB_ERR_STATE


def test_cuda_failures_carry_the_runtime_error_code():
    cb.cb_last_cuda_error()                                                           # clear whatever earlier tests left
    assert cb.cb_last_cuda_error() == (0, "no error")
    sl, sh = cb.cb_head_map_nearest(2, 2, 2, 2)
    prob = cb.Problem(2, 2, 64, 2, 2, 64, sl, sh)
    assert _apply(prob, _view(2, 2, 64, 64)) == cb.CB_ERR_CUDA                        # no device on this machine
    code, text = cb.cb_last_cuda_error()
    assert code != 0 and text and text != "no error"
    assert cb.cb_last_cuda_error() == (0, "no error")                                 # reading cleared it
    with pytest.raises(cb.CbError) as e:
        cb._check(cb.lib().cb_last_device_status(ctypes.c_void_p(0)), "cb_last_device_status")
    assert e.value.status == cb.CB_ERR_CUDA and e.value.cuda_error != 0 and "CUDA error" in str(e.value)


def test_status_calls_without_a_device():
    assert cb.lib().cb_last_device_status(ctypes.c_void_p(0)) == cb.CB_ERR_CUDA
    assert cb.lib().cb_test_hooks(ctypes.c_uint32(1 << 12), 1) == cb.CB_OK             # host state only
    assert cb.lib().cb_test_hooks(ctypes.c_uint32(0), 0) == cb.CB_OK


def test_workspace_and_static_limits():
    sl, sh = cb.cb_head_map_nearest(40, 8, 64, 8)
    prob = cb.Problem(40, 8, 128, 64, 8, 128, sl, sh)
    v_s, v_t = _view(40, 8, 128, 64), _view(64, 8, 128, 64)
    st = cb.lib().cb_stats_build_static(ctypes.byref(prob.c), ctypes.byref(v_s), ctypes.byref(v_t), ctypes.c_void_p(0x100),
                                        ctypes.c_void_p(0x100), ctypes.c_int64(8 * 64), ctypes.c_int64(64),
                                        ctypes.c_void_p(0x200), ctypes.c_void_p(0x300), ctypes.c_void_p(0))
    assert st == cb.CB_ERR_STATIC_LIMIT
    n = ctypes.c_size_t(0)
    assert cb.lib().cb_ridge_solve_large_workspace_bytes(1025, 128, ctypes.c_int64(1), ctypes.byref(n)) == cb.CB_OK
    assert n.value >= 8 * (1088 * 1088 + 1088 * 128)
    assert cb.lib().cb_ridge_solve_large_workspace_bytes(1025, 100, ctypes.c_int64(1), ctypes.byref(n)) == cb.CB_ERR_INVALID_ARG


def test_two_pass_entry_points_reject_bad_arguments_on_the_host():
    sl, sh = cb.cb_head_map_nearest(40, 8, 64, 8)
    prob = cb.Problem(40, 8, 128, 64, 8, 128, sl, sh)
    assert cb.cb_means_workspace_bytes(prob) == 8 * 1024 * (3 * 128 + 2) * 8          # fp64, 8 splits per map
    null = ctypes.c_void_p(0)
    L = cb.lib()
    assert L.cb_means_reset(null, ctypes.c_void_p(0x1000), ctypes.c_size_t(1 << 30), null) == cb.CB_ERR_STATE
    assert L.cb_means_finalize(null, ctypes.c_void_p(0x1000), ctypes.c_size_t(1 << 30), ctypes.c_void_p(0x10), null) == cb.CB_ERR_STATE
    assert L.cb_stats_reduce_centered(null, ctypes.c_void_p(0x10), ctypes.c_void_p(0x10), ctypes.c_void_p(0x10), null, null) == cb.CB_ERR_STATE
    lam = np.array([1e-2], np.float32)
    call = lambda A, B, mu, n_maps, d, nl: L.cb_ridge_solve_centered(
        ctypes.c_void_p(A), ctypes.c_void_p(B), ctypes.c_void_p(mu), n_maps, d, ctypes.c_int64(100),
        lam.ctypes.data_as(ctypes.c_void_p), nl, ctypes.c_uint32(0), ctypes.c_void_p(0x20), ctypes.c_void_p(0x30), null)
    before = cb.cb_launch_count()
    assert call(0x10, 0x10, 0, 4, 128, 1) == cb.CB_ERR_INVALID_ARG                    # no means
    assert call(0x10, 0x10, 0x10, 4, 100, 1) == cb.CB_ERR_UNSUPPORTED
    assert call(0x10, 0x10, 0x10, 4, 128, 17) == cb.CB_ERR_INVALID_ARG
    assert call(0x10, 0x10, 0x10, 0, 128, 1) == cb.CB_OK
    assert cb.cb_launch_count() == before


def test_selector_host_logic_and_argument_errors():
    scores = np.array([[0.1, 0.9, 0.9, 0.3], [0.5, 0.2, 0.7, 0.6]], np.float32)
    assert cb.cb_rank_layers(scores, 1).tolist() == [[1], [2]]                          # tie -> lower index
    assert cb.cb_rank_layers(scores, 2).tolist() == [[1, 2], [2, 3]]
    assert cb.cb_rank_layers(scores, 4).tolist() == [[0, 1, 2, 3], [0, 1, 2, 3]]
    L = cb.lib()
    null = ctypes.c_void_p(0)
    assert L.cb_rank_layers(scores.ctypes.data_as(ctypes.c_void_p), 2, 4, 5, ctypes.c_void_p(0x10)) == cb.CB_ERR_INVALID_ARG
    assert L.cb_probe_r2(null, null, null, null, 4, 128, ctypes.c_int64(10), ctypes.c_float(0), 0, null, null) == cb.CB_ERR_INVALID_ARG
    p = ctypes.c_void_p(0x10)
    assert L.cb_probe_r2(p, p, p, p, 4, 96, ctypes.c_int64(10), ctypes.c_float(0), 0, p, null) == cb.CB_ERR_UNSUPPORTED
    assert L.cb_probe_r2(p, p, p, p, 0, 128, ctypes.c_int64(10), ctypes.c_float(0), 0, p, null) == cb.CB_OK
    bad = np.array([0, 7], np.int32)
    assert L.cb_probe_scores(p, 2, 2, bad.ctypes.data_as(ctypes.c_void_p), 4, p, null) == cb.CB_ERR_INVALID_ARG


def test_token_splits_choice():
    """Left open (0), the split count balances units over 148 SMs against one more slot set per split."""
    for (Ls, Lt, H, want) in [(40, 64, 8, 1), (36, 40, 8, 3), (2, 2, 2, 8)]:
        sl, sh = cb.cb_head_map_nearest(Ls, H, Lt, H)
        assert cb.cb_token_splits(cb.Problem(Ls, H, 128, Lt, H, 128, sl, sh)) == want
        assert cb.cb_token_splits(cb.Problem(Ls, H, 128, Lt, H, 128, sl, sh, n_splits=5)) == 5
