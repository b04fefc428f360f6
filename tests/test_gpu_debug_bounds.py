"""The range-checked build of the library (libtca_dbg.so, compiled with -DTCA_DEBUG_BOUNDS).

In that build every index or offset a kernel takes from memory is compared with its range before
it is used; an access that fails is skipped and the first failure is recorded where the host can
read it.  The tests hand the gather an index that is outside its logical range (not a candidate
token) but still inside the K allocation, so that neither build can touch memory it does not own,
and read the record back.  They skip themselves unless the library they load reports the checked
build.
"""
import os

import numpy as np
import pytest
import torch

import tca_harness as H
from oracle import tca_oracle as O
from paper_2512_09238_b200 import _build, binding as B
from paper_2512_09238_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture()
def checked_library(monkeypatch):
    if not os.path.exists(_build.LIB_DEBUG):
        pytest.skip("libtca_dbg.so has not been built (python -m paper_2512_09238_b200._build --debug-bounds)")
    dbg = B.load_library(_build.LIB_DEBUG)
    if not dbg.tca_build_info() & B.TCA_BUILD_DEBUG_BOUNDS:
        pytest.skip("the library does not report the range-checked build")
    monkeypatch.setattr(B, "_lib", dbg)
    return dbg


def _workload():
    return I.WORKLOADS["config1"].scaled(name="bounds", batch=1, n_q_heads=4, n_kv_heads=2, head_dim=64, L=700,
                                         dtype="bf16", block=32, window=60, seed=51, budget=("fixed", 0.4))


def test_checked_build_agrees_with_the_oracle_on_good_inputs(checked_library):
    wl = _workload()
    data = I.generate(wl)
    p = I.budget_table(wl)
    run = H.gpu_select_compact(wl, data, p)
    assert B.tca_cache_status(run.cache)[0] == B.TCA_OK
    for h in range(wl.n_kv_heads):
        res = H.oracle_select_unit(wl, data, p, 0, h, wl.L)
        S = run.idx.cpu().numpy()[run.offsets[h]:run.offsets[h + 1]].astype(np.int64)
        assert H.compare_selection(res, S, run.t.cpu().numpy()[h, :res["m"]], wl.block) == 0
    dec = H.from_device(H.gpu_decode(run, run.dev["q"][:, :, wl.L - 1, :].contiguous()))
    T = O.retained_set(run.idx.cpu().numpy()[:run.offsets[1]].astype(np.int64), run.m, wl.block, wl.L)
    want = O.attention_over_set(I.widen(data["q"][0, 0, wl.L - 1]), I.widen(data["k"][0, 0, :wl.L])[T],
                                I.widen(data["v"][0, 0, :wl.L])[T], H.scale_of(wl))
    H.check_attention(dec[0, 0], want, "bf16", "decode in the checked build")


def test_gather_index_outside_the_candidates_is_skipped_and_recorded(checked_library):
    wl = _workload()
    data = I.generate(wl)
    p = I.budget_table(wl)
    run = H.gpu_select_compact(wl, data, p)
    m_b = run.m * wl.block
    bad = m_b + 7                               # a tail token: a valid row of K, but not a candidate
    assert bad < wl.L
    victim = int(run.offsets[1]) + 3            # the fourth selected index of unit 1
    idx = run.idx.clone()
    idx[victim] = bad
    tk = np.tile(run.tbar, wl.batch).astype(np.int64)
    cache = B.Cache(run.prm, np.tile(run.n_sel, wl.batch), wl.window + wl.block, tk)
    B.tca_compact_kv(run.prm, run.dev["k"], run.dev["v"], run.L, idx, torch.from_numpy(run.offsets).cuda(),
                     run.offsets, cache)
    st, detail = B.tca_cache_status(cache)
    assert st == B.TCA_ERR_BOUNDS
    assert list(detail) == [1, 1, bad]          # unit 1, check "selected index", the offending value
    # the row was skipped (still the zero fill of tca_cache_init); its neighbours were gathered
    row = int(cache.seg_start[1]) + 3
    assert int(cache.k[row].view(torch.int16).abs().sum()) == 0
    assert int(cache.pos[row]) == -1
    good = run.idx.cpu().numpy()
    np.testing.assert_array_equal(cache.pos.cpu().numpy()[row - 1:row + 2:2], good[[victim - 1, victim + 1]])
    # a negative index is caught the same way; tca_cache_init clears the record
    B.tca_cache_init(run.prm, cache)
    assert B.tca_cache_status(cache)[0] == B.TCA_OK
    idx[victim] = -5
    B.tca_compact_kv(run.prm, run.dev["k"], run.dev["v"], run.L, idx, torch.from_numpy(run.offsets).cuda(),
                     run.offsets, cache)
    st, detail = B.tca_cache_status(cache)
    assert st == B.TCA_ERR_BOUNDS and detail[0] == 1 and detail[1] == 1


def test_block_count_outside_its_range_is_skipped_and_recorded(checked_library):
    """block_topt_kernel takes the per-block count t from the workspace; a count larger than what
    the unit's output window holds is refused (the window is what the offsets array says)."""
    wl = _workload()
    data = I.generate(wl)
    p = I.budget_table(wl)
    run = H.gpu_select_compact(wl, data, p)
    # claim one output slot fewer for the only unit that is checked: the last block no longer fits
    prm = B.make_params(1, 2, 1, 64, wl.block, wl.window, dtype=B.TCA_BF16)
    n_sel = int(run.n_sel[0])
    offsets = torch.tensor([0, n_sel - 1], dtype=torch.int64, device="cuda")
    idx = torch.full((n_sel,), -1, dtype=torch.int32, device="cuda")
    ws = B.alloc_workspace(prm, run.L, B.TCA_OP_SELECT)
    B.tca_select(prm, run.logscore[:1].contiguous(), run.L, run.n_k[:1], idx, offsets, None, None, ws)
    assert B.tca_ws_status(ws) == B.TCA_ERR_BOUNDS
    assert int(idx[n_sel - 1]) == -1            # nothing was written beyond the window
