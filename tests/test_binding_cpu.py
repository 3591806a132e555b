"""Host-side checks that need no GPU: the library loads, exports the declared ABI, and its integer
bookkeeping (head match, static gather schedule) is bit-exact against the oracle."""
import os
import re

import numpy as np
import pytest

import oracle
from paper_2609_00891_b200 import binding as cb
from paper_2609_00891_b200 import build as cb_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    cb_build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "cb.h")).read()
    declared = set(re.findall(r"\b(cb_[a-z0-9_]+)\s*\(", header))
    assert declared == set(cb.EXPORTS)
    L = cb.lib()
    for name in declared:
        assert getattr(L, name) is not None
    assert cb.status_string(cb.CB_OK) == "ok"
    assert "positive" in cb.status_string(cb.CB_ERR_NOT_PD)


@pytest.mark.parametrize("Ls,Hs,Lt,Ht", [(2, 2, 2, 2), (36, 8, 40, 8), (40, 8, 64, 8), (3, 2, 5, 2), (40, 8, 1, 8),
                                         (4, 2, 6, 8), (4, 8, 6, 2), (5, 4, 3, 4)])
def test_head_match_and_schedule_bit_exact(Ls, Hs, Lt, Ht):
    sl, sh = cb.cb_head_map_nearest(Ls, Hs, Lt, Ht)
    sl_o, sh_o = oracle.head_map(Ls, Hs, Lt, Ht)
    assert np.array_equal(sl, sl_o) and np.array_equal(sh, sh_o)
    prob = cb.Problem(Ls, Hs, 128, Lt, Ht, 128, sl, sh)
    got = cb.cb_work_list(prob)
    want = oracle.work_list(Ls, Hs, Lt, Ht, sl_o, sh_o)
    for g, w in zip(got, want):
        assert g.dtype == np.int32 and np.array_equal(g, w)


def test_schedule_with_an_arbitrary_match():
    rng = np.random.default_rng(0)
    Ls, Hs, Lt, Ht = 5, 3, 9, 6
    sl = rng.integers(0, Ls, Lt).astype(np.int32)
    sh = rng.integers(0, Hs, Ht).astype(np.int32)
    got = cb.cb_work_list(cb.Problem(Ls, Hs, 64, Lt, Ht, 64, sl, sh))
    want = oracle.work_list(Ls, Hs, Lt, Ht, sl, sh)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)


def test_argument_errors_are_status_codes():
    sl, sh = cb.cb_head_map_nearest(4, 2, 4, 2)
    with pytest.raises(cb.CbError) as e:
        cb.cb_workspace_bytes(cb.Problem(4, 2, 96, 4, 2, 96, sl, sh))       # head width not 64/128
    assert e.value.status == cb.CB_ERR_UNSUPPORTED
    with pytest.raises(cb.CbError) as e:
        cb.cb_workspace_bytes(cb.Problem(4, 2, 128, 4, 2, 64, sl, sh))      # d_s != d_t
    assert e.value.status == cb.CB_ERR_UNSUPPORTED
    bad = sl.copy()
    bad[1] = 7
    with pytest.raises(cb.CbError) as e:
        cb.cb_workspace_bytes(cb.Problem(4, 2, 128, 4, 2, 128, bad, sh))    # source layer out of range
    assert e.value.status == cb.CB_ERR_INVALID_ARG
    with pytest.raises(cb.CbError) as e:
        cb.cb_workspace_bytes(cb.Problem(4, 2, 128, 4, 2, 128, sl, sh, n_splits=1000))
    assert e.value.status == cb.CB_ERR_INVALID_ARG
    prob = cb.Problem(4, 2, 128, 4, 2, 128, sl, sh, n_splits=3)
    slot = (128 * 256 + 256 + 4) * 4
    assert cb.cb_workspace_bytes(prob) >= 3 * prob.n_maps * slot
    assert cb.cb_launch_count() == 0
