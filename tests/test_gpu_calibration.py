"""Offline calibration (Algorithm 1, Eq. 4) on the GPU against the oracle.

Column means: every entry against the oracle's fp64 value.  Aggregated scores a_i of every
candidate of Eq. 3 and the chosen candidate: equal to the oracle's, except that a candidate
whose a_i lies within the arithmetic tolerance of tau may fall on either side of it.
"""
import numpy as np
import pytest
import torch

from oracle import tca_oracle as O
from paper_2512_09238_b200 import binding as B
from paper_2512_09238_b200 import inputs as I
import tca_harness as H

pytestmark = pytest.mark.gpu

BASE = I.WORKLOADS["config1"]
CASES = {
    # GQA 4:1, d = 128, ragged: L is no multiple of the 128-row tile
    "gqa4_d128": BASE.scaled(name="cal_gqa4", batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, L=1500,
                             dtype="bf16", block=64, window=256, seed=21),
    # d = 64, group of 2, a single partial tile beyond the first
    "g2_d64": BASE.scaled(name="cal_g2", batch=1, n_q_heads=4, n_kv_heads=2, head_dim=64, L=777,
                          dtype="bf16", block=16, window=100, seed=22),
    # odd group (the second chain idles for the last head), L below one tile + one
    "g3_d128": BASE.scaled(name="cal_g3", batch=1, n_q_heads=3, n_kv_heads=1, head_dim=128, L=130,
                           dtype="bf16", block=8, window=20, seed=23),
    # plain multi-head attention, L an exact multiple of the tile
    "mha_d64": BASE.scaled(name="cal_mha", batch=1, n_q_heads=2, n_kv_heads=2, head_dim=64, L=512,
                           dtype="bf16", block=32, window=64, seed=24),
}
COLMEAN_RTOL = 1e-3     # fp32 tensor-core scores, ex2.approx and fp32 tile sums against fp64
A_TOL = 1e-3


def _gpu_colmean(wl, data):
    prm = H.params_for(wl)
    L = wl.L
    dev = {k: H.to_device(np.ascontiguousarray(v[:, :, :L]), wl.dtype) for k, v in data.items()}
    U = wl.batch * wl.n_kv_heads
    col = torch.full((U, L), float("nan"), dtype=torch.float64, device="cuda")
    ws = B.alloc_workspace(prm, L, B.TCA_OP_CALIB)
    B.tca_calib_colmean(prm, dev["q"], dev["k"], L, col, ws)
    torch.cuda.synchronize()
    assert B.tca_ws_status(ws) == B.TCA_OK
    return prm, dev, col


def _oracle_colmean(wl, data, u):
    s, h = divmod(u, wl.n_kv_heads)
    G = wl.group
    return O.attention_column_means(I.widen(data["q"][s, h * G:(h + 1) * G, :wl.L]), I.widen(data["k"][s, h, :wl.L]),
                                    H.scale_of(wl))


@pytest.mark.parametrize("name", list(CASES))
def test_column_means_match_the_oracle(name):
    wl = CASES[name]
    data = I.generate(wl)
    prm, dev, col = _gpu_colmean(wl, data)
    got = col.cpu().numpy()
    assert np.all(np.isfinite(got))
    for u in range(wl.batch * wl.n_kv_heads):
        want = _oracle_colmean(wl, data, u)
        np.testing.assert_allclose(got[u], want, rtol=COLMEAN_RTOL, atol=1e-12, err_msg=f"{name} unit {u}")
        # each row of A sums to 1, so the means weighted back by their counts give L
        assert float(np.sum(got[u] * (wl.L - np.arange(wl.L)))) == pytest.approx(wl.L, rel=1e-4)
    # a second call gives the same bits (fixed order of every sum)
    _, _, again = _gpu_colmean(wl, data)
    assert torch.equal(col.view(torch.int64), again.view(torch.int64))


@pytest.mark.parametrize("tau", [0.9, 0.5, 0.2])
@pytest.mark.parametrize("name", ["gqa4_d128", "g2_d64"])
def test_candidate_scores_and_choice_match_the_oracle(name, tau):
    wl = CASES[name]
    data = I.generate(wl)
    prm, dev, col = _gpu_colmean(wl, data)
    L, U, G = wl.L, wl.batch * wl.n_kv_heads, wl.group
    m = (L - wl.window) // wl.block
    cands = O.candidate_grid(wl.block, 14, 1.0)
    logscore = torch.empty(U, L, dtype=torch.float64, device="cuda")
    q_last = dev["q"][:, :, L - 1, :].contiguous()
    B.tca_score(prm, q_last, dev["k"], L, logscore, B.alloc_workspace(prm, L, B.TCA_OP_SCORE))
    a_gpu = np.zeros((U, len(cands)))
    sizes = np.zeros((U, len(cands)), dtype=np.int64)
    ws_sel = B.alloc_workspace(prm, L, B.TCA_OP_SELECT)
    a_dev = torch.empty(U, dtype=torch.float64, device="cuda")
    for i, p in enumerate(cands):
        n_k, n_sel, _ = B.tca_budget_resolve(np.tile(p, (wl.n_kv_heads, 1)), m)
        per_unit = np.tile(n_sel, wl.batch)
        offsets = np.zeros(U + 1, dtype=np.int64)
        offsets[1:] = np.cumsum(per_unit)
        idx = torch.empty(max(1, int(offsets[-1])), dtype=torch.int32, device="cuda")
        off_dev = torch.from_numpy(offsets).cuda()
        B.tca_select(prm, logscore, L, n_k, idx, off_dev, None, None, ws_sel)
        B.tca_calib_score(prm, col, L, idx, off_dev, a_dev)
        torch.cuda.synchronize()
        a_gpu[:, i] = a_dev.cpu().numpy()
        sizes[:, i] = per_unit
    for u in range(U):
        s, h = divmod(u, wl.n_kv_heads)
        choice_o, a_o, sizes_o = O.calibrate_head(I.widen(data["q"][s, h * G:(h + 1) * G, :L]),
                                                  I.widen(data["k"][s, h, :L]), cands, wl.block, wl.window,
                                                  float(np.float32(wl.alpha)), tau, H.scale_of(wl))
        np.testing.assert_array_equal(sizes[u], sizes_o)
        np.testing.assert_allclose(a_gpu[u], a_o, atol=A_TOL, rtol=0, err_msg=f"{name} unit {u}")
        choice_g = B.tca_calib_choose(a_gpu[u], sizes[u], tau)
        if np.all(np.abs(a_o - tau) > A_TOL):            # no candidate sits on the threshold
            assert choice_g == choice_o
        else:                                            # either side of tau is a correct decision there
            valid = a_gpu[u] >= tau
            assert valid[choice_g] or not valid.any()
            assert sizes[u][choice_g] == sizes[u][valid].min() if valid.any() else choice_g == len(cands) - 1


def test_choose_rules_and_argument_checks():
    a = np.array([0.5, 0.95, 0.93, 0.99])
    assert B.tca_calib_choose(a, np.array([10, 30, 30, 50]), 0.9) == 1      # tie on size: lower index
    assert B.tca_calib_choose(a, np.array([10, 30, 20, 50]), 0.9) == 2      # fewest tokens among the valid
    assert B.tca_calib_choose(a, np.array([10, 30, 20, 50]), 0.999) == 3    # nothing valid: the last one
    wl = CASES["g3_d128"].scaled(dtype="f32")
    prm = H.params_for(wl)
    x = torch.zeros(1, 3, wl.L, wl.head_dim, device="cuda")
    col = torch.zeros(1, wl.L, dtype=torch.float64, device="cuda")
    assert B.tca_workspace_bytes(prm, wl.L, B.TCA_OP_CALIB) == 0
    with pytest.raises(B.TcaError):                                         # fp32 inputs are not supported
        B.tca_calib_colmean(prm, x, x[:, :1], wl.L, col, torch.zeros(4096, dtype=torch.uint8, device="cuda"))
