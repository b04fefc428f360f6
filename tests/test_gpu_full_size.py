"""Parity at the full benchmark sizes, through the same Pipeline object bench.py times.

The oracle cannot afford every output at L = 32K..128K, so selection is checked in full
(it is O(L)) and attention on sampled rows / sampled decode steps: first and last rows, rows
around the window, block and tile edges, plus random ones.
"""
import numpy as np
import pytest
import torch

import bench
import tca_harness as H
from oracle import tca_oracle as O
from paper_2512_09238_b200 import binding as B
from paper_2512_09238_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _pipeline(wl):
    data = I.generate(wl)
    p = I.budget_table(wl)
    return data, p, bench.Pipeline(wl, data, p, torch, B, host_io=False)


def _check_selection(wl, data, p, pipe, units):
    idx = pipe.idx.cpu().numpy()
    sel = {}
    accepted = 0
    for u in units:
        s, h = divmod(u, wl.n_kv_heads)
        res = H.oracle_select_unit(wl, data, p, s, h, wl.L)
        S = idx[pipe.offsets[u]:pipe.offsets[u + 1]].astype(np.int64)
        t = np.bincount(S // wl.block, minlength=res["m"])
        accepted += H.compare_selection(res, S, t, wl.block)
        sel[u] = S
    assert accepted <= max(4, len(list(units)) // 4)      # differences inside the 1e-5 band stay rare
    return sel


def _check_prefill_rows(wl, data, pipe, sel, n_random, heads_per_unit=1):
    out = pipe.O
    scale, G = H.scale_of(wl), wl.group
    m = wl.n_blocks
    for u, S in sel.items():
        s, h = divmod(u, wl.n_kv_heads)
        T = O.retained_set(S, m, wl.block, wl.L)
        K, V = I.widen(data["k"][s, h, :wl.L]), I.widen(data["v"][s, h, :wl.L])
        rows = H.sample_rows(wl.L, wl.window, wl.block, n_random, seed=u)
        for g in range(heads_per_unit):
            hq = h * G + (g * 3 + u) % G
            Q = I.widen(data["q"][s, hq, :wl.L])
            want = O.attention_rows(Q, K, V, T, wl.window, scale, rows)
            got = H.from_device(out[s, hq][torch.tensor(rows, device="cuda")])
            H.check_attention(got, want, wl.dtype, f"{wl.name} unit {u} head {hq}")


def test_config3_prefill_32k():
    wl = I.WORKLOADS["config3"]
    data, p, pipe = _pipeline(wl)
    pipe.step()
    torch.cuda.synchronize()
    assert B.tca_ws_status(pipe.ws_prefill) == B.TCA_OK
    sel = _check_selection(wl, data, p, pipe, range(pipe.U))
    _check_prefill_rows(wl, data, pipe, sel, n_random=10, heads_per_unit=2)
    # retained-token counts equal each head's budget
    for u in range(pipe.U):
        assert len(sel[u]) == pipe.n_sel[u % wl.n_kv_heads] == pipe.cache.n_global[u]


def test_config3_prefill_32k_band_first():
    """The same configuration with the window band walked first (TCA_FLAG_PREFILL_BAND_FIRST), the
    whole chain enqueued without host synchronisation: sampled rows of every unit against the oracle."""
    wl = I.WORKLOADS["config3"]
    data = I.generate(wl)
    p = I.budget_table(wl)
    pipe = bench.Pipeline(wl, data, p, torch, B, host_io=False, flags=B.TCA_FLAG_PREFILL_BAND_FIRST)
    pipe.step()
    pipe.step()
    torch.cuda.synchronize()
    assert B.tca_ws_status(pipe.ws_prefill) == B.TCA_OK
    sel = _check_selection(wl, data, p, pipe, range(pipe.U))
    _check_prefill_rows(wl, data, pipe, sel, n_random=6)


@pytest.mark.parametrize("flags", [0, B.TCA_FLAG_PREFILL_BAND_FIRST])
def test_the_step_from_host_buffers_equals_the_resident_step(flags):
    """bench.py's end-to-end step (K first, then V and Q in ascending row ranges with the compaction
    done piece by piece as V lands, O copied back per range, decode tokens in and out) against the
    step on resident inputs: every element of O and of the decode outputs bit for bit, starting from
    device buffers that hold a marker instead of the inputs."""
    wl = I.WORKLOADS["config3"].scaled(decode_steps=6)
    data = I.generate(wl)
    p = I.budget_table(wl)
    ref = bench.Pipeline(wl, data, p, torch, B, host_io=False, flags=flags)
    ref.step()
    torch.cuda.synchronize()
    pipe = bench.Pipeline(wl, data, p, torch, B, host_io=True, flags=flags)
    for t in (pipe.Qp, pipe.Kp, pipe.Vp, pipe.qd, pipe.kd, pipe.vd, pipe.cache.k, pipe.cache.v, pipe.O, pipe.Od):
        t.fill_(5.0)                                   # finite: rows past a range are masked, not skipped
    pipe.q_last.fill_(5.0)
    pipe.h_O.fill_(float("nan"))
    assert len(pipe.row_ranges) > 4
    pipe.step(host_io=True)
    torch.cuda.synchronize()
    for ws in pipe.ws_rows:
        assert B.tca_ws_status(ws) == B.TCA_OK
    assert B.tca_ws_status(pipe.ws_decode) == B.TCA_OK
    assert torch.equal(pipe.idx, ref.idx)
    assert torch.equal(pipe.h_O.view(torch.int16), ref.O.cpu().view(torch.int16))
    assert torch.equal(pipe.h_Od.view(torch.int16), ref.Od.cpu().view(torch.int16))
    assert torch.equal(pipe.cache.pos, ref.cache.pos)


@pytest.mark.parametrize("name", ["config3", "config4"])
def test_gather_prefill_equals_the_cache_path_at_full_size(name):
    """tca_attn_prefill_gather (selected rows fetched from K, V inside the attention kernel) over the
    selection of the timed pipeline: every element of O bit for bit equal to compaction + prefill,
    whose sampled rows the tests above compare with the oracle."""
    wl = I.WORKLOADS[name]
    data, p, pipe = _pipeline(wl)
    pipe.steps_decode = 0
    pipe.step()
    torch.cuda.synchronize()
    via_cache = pipe.O.clone()
    pipe.O.fill_(float("nan"))
    t = pipe.time_gather_prefill(reps=1)
    assert t["prefill_ms"] > 0
    assert B.tca_ws_status(pipe.ws_prefill) == B.TCA_OK
    assert torch.equal(pipe.O.view(torch.uint8), via_cache.view(torch.uint8))


def test_config4_prefill_128k_then_256_decode_steps():
    wl = I.WORKLOADS["config4"]
    data, p, pipe = _pipeline(wl)
    B_, prm, L, G = B, pipe.prm, wl.L, wl.group
    # the step, with the decode loop unrolled here so that chosen steps can be checked
    pipe.steps_decode = 0
    pipe.step()
    torch.cuda.synchronize()
    assert B.tca_ws_status(pipe.ws_prefill) == B.TCA_OK
    units = range(pipe.U)
    sel = _check_selection(wl, data, p, pipe, units)
    _check_prefill_rows(wl, data, pipe, {u: sel[u] for u in (0, 3, 5)}, n_random=6)
    scale = H.scale_of(wl)
    caches = {u: O.DecodeCache.from_prefill(sel[u], wl.n_blocks, L, wl.block, wl.window, p[u % wl.n_kv_heads], scale)
              for u in units}
    Kw = {u: I.widen(data["k"][0, u]) for u in (1, 6)}
    Vw = {u: I.widen(data["v"][0, u]) for u in (1, 6)}
    check_steps = {0, 126, 127, 128, 255}
    for step in range(wl.decode_steps):
        pos = L + step
        B_.tca_cache_append(prm, pipe.cache, pipe.kd[step], pipe.vd[step], pipe.qd[step])
        B_.tca_attn_decode(prm, pipe.qd[step], pipe.cache, pipe.Od[step], pipe.ws_decode)
        for u in units:
            Ku = Kw[u] if u in Kw else I.widen(data["k"][0, u, pos - wl.window - wl.block:pos + 1])
            if u in Kw:
                caches[u].append(pos, I.widen(data["q"][0, u * G:(u + 1) * G, pos]), Ku)
            else:   # only the block that may be compressed is needed: index it relative to its start
                class _Shift:
                    def __init__(self, a, off): self.a, self.off = a, off
                    def __getitem__(self, ix): return self.a[np.asarray(ix) - self.off]
                caches[u].append(pos, I.widen(data["q"][0, u * G:(u + 1) * G, pos]),
                                 _Shift(Ku, pos - wl.window - wl.block))
        if step in check_steps:
            out = H.from_device(pipe.Od[step])
            for u in (1, 6):
                for g in (0, G - 1):
                    want = caches[u].attend(I.widen(data["q"][0, u * G + g, pos]), Kw[u], Vw[u])
                    H.check_attention(out[0, u * G + g], want, wl.dtype, f"config4 decode step {step}")
    torch.cuda.synchronize()
    assert B.tca_ws_status(pipe.ws_decode) == B.TCA_OK
    cpos = pipe.cache.pos.cpu().numpy()
    for u in units:
        np.testing.assert_array_equal(cpos[pipe.cache.unit_rows(u)], caches[u].positions())
        assert pipe.cache.n_global[u] == len(sel[u]) + 2 * pipe.tbar[u % wl.n_kv_heads]   # two blocks compressed


def test_config2_decode_32k_batch4_and_dense_decode():
    wl = I.WORKLOADS["config2"]
    data, p, pipe = _pipeline(wl)
    L, G = wl.L, wl.group
    # setup (score with the newest query, select, compact), then the timed call: one decode step
    B.tca_score(pipe.prm, pipe.q_last, pipe.Kp, L, pipe.logscore, pipe.ws_score)
    B.tca_select(pipe.prm, pipe.logscore, L, pipe.n_k, pipe.idx, pipe.offsets_dev, None, None, pipe.ws_select)
    B.tca_compact_kv(pipe.prm, pipe.Kp, pipe.Vp, L, pipe.idx, pipe.offsets_dev, pipe.offsets, pipe.cache)
    out = torch.empty_like(pipe.q_last)
    B.tca_attn_decode(pipe.prm, pipe.q_last, pipe.cache, out, pipe.ws_decode)
    torch.cuda.synchronize()
    sel = _check_selection(wl, data, p, pipe, range(pipe.U))       # the selection of every unit
    units = [0, 7, 13, 22, 31]                                      # decode outputs of five of them
    got = H.from_device(out)
    scale = H.scale_of(wl)
    for u in units:
        s, h = divmod(u, wl.n_kv_heads)
        T = O.retained_set(sel[u], wl.n_blocks, wl.block, L)
        K, V = I.widen(data["k"][s, h, :L]), I.widen(data["v"][s, h, :L])
        for g in range(G):
            want = O.attention_over_set(I.widen(data["q"][s, h * G + g, L - 1]), K[T], V[T], scale)
            H.check_attention(got[s, h * G + g], want, wl.dtype, f"config2 decode unit {u}")
    # dense decode over the full cache (100 % budget) against plain softmax attention
    dense = wl.scaled(budget=("fixed", 1.0))
    pd = I.budget_table(dense)
    pipe_d = bench.Pipeline(dense, data, pd, torch, B, host_io=False)
    B.tca_score(pipe_d.prm, pipe_d.q_last, pipe_d.Kp, L, pipe_d.logscore, pipe_d.ws_score)
    B.tca_select(pipe_d.prm, pipe_d.logscore, L, pipe_d.n_k, pipe_d.idx, pipe_d.offsets_dev, None, None,
                 pipe_d.ws_select)
    B.tca_compact_kv(pipe_d.prm, pipe_d.Kp, pipe_d.Vp, L, pipe_d.idx, pipe_d.offsets_dev, pipe_d.offsets,
                     pipe_d.cache)
    B.tca_attn_decode(pipe_d.prm, pipe_d.q_last, pipe_d.cache, out, pipe_d.ws_decode)
    torch.cuda.synchronize()
    assert int(pipe_d.cache.n_global.sum() + pipe_d.cache.n_tail.sum()) == pipe_d.U * L
    got = H.from_device(out)
    for u in (0, 31):
        s, h = divmod(u, wl.n_kv_heads)
        K, V = I.widen(data["k"][s, h, :L]), I.widen(data["v"][s, h, :L])
        for g in (0, 3):
            q = I.widen(data["q"][s, h * G + g, L - 1])
            x = (K @ q) * scale
            w = np.exp(x - x.max())
            H.check_attention(got[s, h * G + g], (w / w.sum()) @ V, wl.dtype, "config2 dense decode")


@pytest.mark.parametrize("frac", [0.05, 0.10, 0.25, 0.50, 1.0])
def test_config5_budget_sweep_64k(frac):
    wl = I.WORKLOADS["config5"].scaled(budget=("fixed", frac))
    data, p, pipe = _pipeline(wl)
    pipe.step()
    torch.cuda.synchronize()
    assert B.tca_ws_status(pipe.ws_prefill) == B.TCA_OK
    sel = _check_selection(wl, data, p, pipe, range(pipe.U))       # the selection of every unit
    units = [0, 5, 11, 15]
    m = wl.n_blocks
    for u in range(pipe.U):   # uniform budget: every head keeps the same count, and sees it in its cache
        assert len(sel[u]) == pipe.n_sel[0]
        assert abs(len(sel[u]) / (m * wl.block) - frac) < 0.01
    _check_prefill_rows(wl, data, pipe, {u: sel[u] for u in units[:2]}, n_random=4)
    if frac == 1.0:   # the library's own dense baseline really is dense causal attention
        u = 11
        s, h = divmod(u, wl.n_kv_heads)
        np.testing.assert_array_equal(sel[u], np.arange(m * wl.block))
        K, V = I.widen(data["k"][s, h, :wl.L]), I.widen(data["v"][s, h, :wl.L])
        Q = I.widen(data["q"][s, h * wl.group + 1, :wl.L])
        for i in (0, 4095, 4096, 40000, wl.L - 1):
            x = (K[:i + 1] @ Q[i]) * H.scale_of(wl)
            w = np.exp(x - x.max())
            H.check_attention(H.from_device(pipe.O[s, h * wl.group + 1, i]), (w / w.sum()) @ V[:i + 1], wl.dtype,
                              f"dense row {i}")
    # the 64 decode steps ran inside step(): compare the last one with the oracle replaying the appends
    scale, G, L = H.scale_of(wl), wl.group, wl.L
    u = units[1]
    s, h = divmod(u, wl.n_kv_heads)
    cache = O.DecodeCache.from_prefill(sel[u], m, L, wl.block, wl.window, p[h], scale)
    Kw, Vw = I.widen(data["k"][s, h]), I.widen(data["v"][s, h])
    for step in range(wl.decode_steps):
        kept = cache.append(L + step, I.widen(data["q"][s, h * G:(h + 1) * G, L + step]), Kw)
        assert kept is None          # 64 steps never complete a block of 128
    last = wl.decode_steps - 1
    want = cache.attend(I.widen(data["q"][s, h * G + 2, L + last]), Kw, Vw)
    H.check_attention(H.from_device(pipe.Od[last, s, h * G + 2]), want, wl.dtype, f"config5 decode f={frac}")


def test_calibration_column_means_at_32k():
    """Algorithm 1's dense passes at L = 32768 (config 3), checked through what holds at any size:
    every row of the attention map sums to 1, so the column means weighted back by their counts
    (L - k) sum to L for every KV head; sampled columns near the end, where only a few rows are
    visible, against the oracle's definition evaluated for just those rows; Eq. 4 of the
    all-candidates selection is exactly 1 and grows with the budget."""
    wl = I.WORKLOADS["config3"]
    data, p, pipe = _pipeline(wl)
    L, U, G = wl.L, pipe.U, wl.group
    col = torch.empty(U, L, dtype=torch.float64, device="cuda")
    ws = B.alloc_workspace(pipe.prm, L, B.TCA_OP_CALIB)
    B.tca_calib_colmean(pipe.prm, pipe.Qp, pipe.Kp, L, col, ws)
    torch.cuda.synchronize()
    assert B.tca_ws_status(ws) == B.TCA_OK
    c = col.cpu().numpy()
    assert np.all(np.isfinite(c)) and np.all(c >= 0)
    np.testing.assert_allclose((c * (L - np.arange(L))).sum(1), float(L), rtol=1e-5)
    scale = H.scale_of(wl)
    n_last = 96                                              # the last 96 rows see columns >= L - 96 fully
    for u in (0, U - 1):
        s, h = divmod(u, wl.n_kv_heads)
        K = I.widen(data["k"][s, h, :L])
        want = np.zeros(n_last)
        for g in range(G):
            Q = I.widen(data["q"][s, h * G + g, L - n_last:L])
            for r in range(n_last):
                j = L - n_last + r
                x = (K[:j + 1] @ Q[r]) * scale
                a = np.exp(x - x.max())
                a /= a.sum()
                want[:r + 1] += a[L - n_last:j + 1]
        want /= G * (n_last - np.arange(n_last))
        np.testing.assert_allclose(c[u, L - n_last:], want, rtol=2e-3, atol=1e-12)
    # columns sampled over the whole range (first, around the window, tile edges, random, last) for
    # one unit against the oracle: every visible row's softmax is normalised over all of its keys
    rng = np.random.default_rng(5)
    cols = sorted({0, 1, 2, 3, 127, 128, 129, wl.window - 1, wl.window, wl.window + 1, 16383, 16384, L - 129,
                   L - 128, L - 2, L - 1} | {int(x) for x in rng.integers(0, L, size=64)})
    u = 3
    s_, h_ = divmod(u, wl.n_kv_heads)
    want = O.attention_column_means_at(I.widen(data["q"][s_, h_ * G:(h_ + 1) * G, :L]), I.widen(data["k"][s_, h_, :L]),
                                       scale, cols, rows_per_step=1024)
    np.testing.assert_allclose(c[u, cols], want, rtol=2e-3, atol=1e-12)
    # Eq. 4 for two budgets through the library's own selection
    B.tca_score(pipe.prm, pipe.q_last, pipe.Kp, L, pipe.logscore, pipe.ws_score)
    a_prev = None
    for frac in (0.25, 1.0):
        wlf = wl.scaled(budget=("fixed", frac))
        n_k, n_sel, _ = B.tca_budget_resolve(I.budget_table(wlf), pipe.m)
        offsets = np.zeros(U + 1, dtype=np.int64)
        offsets[1:] = np.cumsum(np.tile(n_sel, wl.batch))
        idx = torch.empty(int(offsets[-1]), dtype=torch.int32, device="cuda")
        off_dev = torch.from_numpy(offsets).cuda()
        B.tca_select(pipe.prm, pipe.logscore, L, n_k, idx, off_dev, None, None, pipe.ws_select)
        a = torch.empty(U, dtype=torch.float64, device="cuda")
        B.tca_calib_score(pipe.prm, col, L, idx, off_dev, a)
        a = a.cpu().numpy()
        assert np.all(a > 0) and np.all(a <= 1.0 + 1e-12)
        if frac == 1.0:
            np.testing.assert_allclose(a, 1.0, rtol=1e-12)
            assert np.all(a >= a_prev)
        a_prev = a


def test_calibration_column_means_at_128k():
    """The same dense passes at the benchmark length, L = 131072 (config 4): row sums, and the last 96
    columns (seen fully by the last 96 rows) against the definition for both end units."""
    wl = I.WORKLOADS["config4"].scaled(decode_steps=0)
    data, p, pipe = _pipeline(wl)
    L, U, G = wl.L, pipe.U, wl.group
    col = torch.empty(U, L, dtype=torch.float64, device="cuda")
    ws = B.alloc_workspace(pipe.prm, L, B.TCA_OP_CALIB)
    B.tca_calib_colmean(pipe.prm, pipe.Qp, pipe.Kp, L, col, ws)
    torch.cuda.synchronize()
    assert B.tca_ws_status(ws) == B.TCA_OK
    c = col.cpu().numpy()
    assert np.all(np.isfinite(c)) and np.all(c >= 0)
    np.testing.assert_allclose((c * (L - np.arange(L))).sum(1), float(L), rtol=1e-5)
    scale = H.scale_of(wl)
    n_last = 96
    for u in (0, U - 1):
        s, h = divmod(u, wl.n_kv_heads)
        K = I.widen(data["k"][s, h, :L])
        want = np.zeros(n_last)
        for g in range(G):
            Q = I.widen(data["q"][s, h * G + g, L - n_last:L])
            for r in range(n_last):
                j = L - n_last + r
                x = (K[:j + 1] @ Q[r]) * scale
                a = np.exp(x - x.max())
                a /= a.sum()
                want[:r + 1] += a[L - n_last:j + 1]
        want /= G * (n_last - np.arange(n_last))
        np.testing.assert_allclose(c[u, L - n_last:], want, rtol=2e-3, atol=1e-12)
