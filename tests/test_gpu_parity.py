"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element, on
seeded inputs small enough for the oracle yet spanning several tiles and ragged tails."""
import math

import numpy as np
import pytest
import torch

from oracle import tca_oracle as O
from paper_2512_09238_b200 import binding as B
from paper_2512_09238_b200 import inputs as I
import tca_harness as H

pytestmark = pytest.mark.gpu

BASE = I.WORKLOADS["config1"]
SMALL = {
    # the first benchmark configuration itself (fp32, 8 heads, L = 2048, b = 32, w = 128)
    "config1": BASE,
    # GQA 4:1, bf16, d = 128, ragged everywhere: L not a multiple of any tile, (L - w) % b != 0
    "bf16_gqa4": BASE.scaled(name="bf16_gqa4", batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, L=1500,
                             dtype="bf16", block=64, window=256, seed=11, budget=("beta", 2.0, 5.0, 0.05, 1.0)),
    "bf16_d64_g2": BASE.scaled(name="bf16_d64_g2", batch=1, n_q_heads=4, n_kv_heads=2, head_dim=64, L=777,
                               dtype="bf16", block=16, window=100, seed=12),
    "f32_d128_g8": BASE.scaled(name="f32_d128_g8", batch=1, n_q_heads=8, n_kv_heads=1, head_dim=128, L=600,
                               dtype="f32", block=8, window=50, seed=13),
    # 28/4 heads like Qwen2.5-7B: group of 7
    "bf16_g7": BASE.scaled(name="bf16_g7", batch=1, n_q_heads=7, n_kv_heads=1, head_dim=128, L=1000,
                           dtype="bf16", block=128, window=300, seed=14, budget=("fixed", 0.3)),
    "f32_g3_b1": BASE.scaled(name="f32_g3_b1", batch=1, n_q_heads=3, n_kv_heads=1, head_dim=64, L=300,
                             dtype="f32", block=1, window=17, seed=15, budget=("fixed", 1.0)),
}


@pytest.fixture(scope="module")
def runs():
    cache = {}

    def get(name):
        if name not in cache:
            wl = SMALL[name]
            data = I.generate(wl)
            p = I.budget_table(wl)
            run = H.gpu_select_compact(wl, data, p)
            oracle = [[H.oracle_select_unit(wl, data, p, s, h, wl.L) for h in range(wl.n_kv_heads)]
                      for s in range(wl.batch)]
            cache[name] = (wl, data, p, run, oracle)
        return cache[name]

    return get


@pytest.mark.parametrize("name", list(SMALL))
def test_score_matches_oracle(runs, name):
    wl, data, p, run, oracle = runs(name)
    got = run.logscore.cpu().numpy()
    for s in range(wl.batch):
        for h in range(wl.n_kv_heads):
            want = oracle[s][h]["log_s"]
            u = s * wl.n_kv_heads + h
            assert np.max(np.abs(got[u] - want)) < H.LOGSCORE_TOL
            assert abs(np.exp(got[u]).sum() - 1) < 1e-6


@pytest.mark.parametrize("name", list(SMALL))
def test_selection_matches_oracle(runs, name):
    wl, data, p, run, oracle = runs(name)
    idx = run.idx.cpu().numpy()
    t = run.t.cpu().numpy()
    hh = run.h.cpu().numpy()
    accepted = 0
    for s in range(wl.batch):
        for h in range(wl.n_kv_heads):
            u = s * wl.n_kv_heads + h
            res = oracle[s][h]
            np.testing.assert_array_equal(run.n_k[h], res["n"])
            S = idx[run.offsets[u]:run.offsets[u + 1]].astype(np.int64)
            if res["m"]:
                np.testing.assert_allclose(hh[u, :res["m"]], res["h"], rtol=2e-6, atol=1e-12)
            accepted += H.compare_selection(res, S, t[u, :res["m"]], wl.block)
    assert accepted <= 2, "differences inside the 1e-5 band should be rare"


@pytest.mark.parametrize("name", list(SMALL))
def test_compaction_is_bit_exact(runs, name):
    wl, data, p, run, oracle = runs(name)
    idx = run.idx.cpu().numpy()
    Kc = run.cache.k.view(torch.int16 if wl.dtype == "bf16" else torch.int32).cpu().numpy()
    Vc = run.cache.v.view(torch.int16 if wl.dtype == "bf16" else torch.int32).cpu().numpy()
    pos = run.cache.pos.cpu().numpy()
    state = run.cache.state.cpu().numpy().reshape(-1, B.TCA_STATE_WORDS)
    raw = np.int16 if wl.dtype == "bf16" else np.int32
    for s in range(wl.batch):
        for h in range(wl.n_kv_heads):
            u = s * wl.n_kv_heads + h
            S = idx[run.offsets[u]:run.offsets[u + 1]].astype(np.int64)
            T = O.retained_set(S, run.m, wl.block, wl.L)
            rows = run.cache.unit_rows(u)
            assert len(rows) == len(T)
            np.testing.assert_array_equal(pos[rows], T)
            np.testing.assert_array_equal(Kc[rows], data["k"][s, h, T].view(raw))
            np.testing.assert_array_equal(Vc[rows], data["v"][s, h, T].view(raw))
            assert state[u, 2] == len(S) and state[u, 4] == wl.L - run.m * wl.block and state[u, 5] == wl.L


@pytest.mark.parametrize("name", ["config1", "bf16_gqa4", "bf16_g7", "f32_g3_b1"])
def test_compaction_by_position_ranges_is_bit_identical(runs, name):
    """tca_compact_kv_range over a partition of [0, L), in a shuffled order, into a cache filled with
    a marker: K, V, positions and state equal to one tca_compact_kv; after the call for [0, p) the
    rows with position below p are in place and rows at or above p still hold the marker."""
    wl, data, p, run, oracle = runs(name)
    L = run.L
    tk = np.tile(run.tbar, wl.batch).astype(np.int64)
    cache = B.Cache(run.prm, np.tile(run.n_sel, wl.batch), wl.window + wl.block, tk)
    marker = 3.0
    cache.k.fill_(marker)
    cache.v.fill_(marker)
    offsets_dev = torch.from_numpy(run.offsets).cuda()
    cuts = sorted({0, L // 5, L // 2, L - 1, L})
    parts = [(a, b) for a, b in zip(cuts[:-1], cuts[1:]) if b > a]
    first = parts[0]
    B.tca_compact_kv_range(run.prm, run.dev["k"], run.dev["v"], L, first[0], first[1], run.idx, offsets_dev,
                           run.offsets, cache)
    torch.cuda.synchronize()
    pos = cache.pos.cpu().numpy()
    kc = cache.k.float().cpu().numpy()
    ref_pos = run.cache.pos.cpu().numpy()
    for u in range(wl.batch * wl.n_kv_heads):
        rows = np.asarray(run.cache.unit_rows(u))
        np.testing.assert_array_equal(pos[rows], ref_pos[rows])                 # all positions after any call
        late = rows[ref_pos[rows] >= first[1]]
        assert (kc[late] == marker).all()                                       # not touched yet
    for (a, b) in parts[:0:-1]:                                                 # the rest, last range first
        B.tca_compact_kv_range(run.prm, run.dev["k"], run.dev["v"], L, a, b, run.idx, offsets_dev, run.offsets, cache)
    torch.cuda.synchronize()
    raw = torch.int16 if wl.dtype == "bf16" else torch.int32
    for u in range(wl.batch * wl.n_kv_heads):
        rows = torch.as_tensor(np.asarray(run.cache.unit_rows(u)), device="cuda")
        assert torch.equal(cache.k.view(raw)[rows], run.cache.k.view(raw)[rows])
        assert torch.equal(cache.v.view(raw)[rows], run.cache.v.view(raw)[rows])
    assert torch.equal(cache.pos, run.cache.pos)
    assert torch.equal(cache.state, run.cache.state)
    assert list(cache.n_global) == list(run.cache.n_global) and list(cache.n_tail) == list(run.cache.n_tail)
    for bad in [(-1, 5), (5, 5), (0, L + 1)]:
        with pytest.raises(B.TcaError):
            B.tca_compact_kv_range(run.prm, run.dev["k"], run.dev["v"], L, bad[0], bad[1], run.idx, offsets_dev,
                                   run.offsets, cache)


def _oracle_T(run, wl, u):
    """The retained set the oracle's attention is evaluated on: the index set the GPU selected.

    Selection has its own tests (test_selection_matches_oracle compares the GPU's index set with
    the oracle's under the 1e-5 rule: equal, or different only where the oracle's scores at the
    budget boundary are closer than 1e-5).  The attention tests then ask a separate question: given
    an index set, is the attention over it right?  Feeding both sides the GPU's set keeps an
    accepted boundary difference in the selection from showing up a second time as an attention
    error, and hides nothing, because a wrong set already fails the selection test."""
    idx = run.idx.cpu().numpy()
    S = idx[run.offsets[u]:run.offsets[u + 1]].astype(np.int64)
    return O.retained_set(S, run.m, wl.block, wl.L)


@pytest.mark.parametrize("name", list(SMALL))
def test_prefill_matches_oracle_on_every_row(runs, name):
    wl, data, p, run, oracle = runs(name)
    out = H.from_device(H.gpu_prefill(run))
    scale = H.scale_of(wl)
    G = wl.group
    for s in range(wl.batch):
        for h in range(wl.n_kv_heads):
            u = s * wl.n_kv_heads + h
            T = _oracle_T(run, wl, u)                     # the GPU's own index set (see the 1e-5 rule)
            K = I.widen(data["k"][s, h, :wl.L])
            V = I.widen(data["v"][s, h, :wl.L])
            for g in range(G):
                Q = I.widen(data["q"][s, h * G + g, :wl.L])
                want = O.attention_rows(Q, K, V, T, wl.window, scale)
                H.check_attention(out[s, h * G + g], want, wl.dtype, f"{name} seq {s} head {h * G + g}")


@pytest.mark.parametrize("name", ["config1", "bf16_gqa4", "bf16_g7"])
def test_prefill_by_row_ranges_is_bit_identical(runs, name):
    """Row ranges that partition [0, L), in any order, each with its own workspace, leave O equal
    bit for bit to the single call; rows outside a range are not written."""
    wl, data, p, run, oracle = runs(name)
    whole = H.gpu_prefill(run)
    L = run.L
    cuts = sorted({0, 128, 384, min(L, 1280), L})
    cuts = [c for c in cuts if c <= L]
    parts = list(zip(cuts[:-1], cuts[1:]))
    out = torch.full_like(run.dev["q"], float("nan"))
    first = parts[-1]                                         # the last range first: order must not matter
    for (r0, r1) in [first] + parts[:-1]:
        ws = B.alloc_workspace(run.prm, L, B.TCA_OP_PREFILL)
        B.tca_attn_prefill_rows(run.prm, run.dev["q"], run.dev["k"], run.dev["v"], L, r0, r1, run.cache, out, ws)
        assert B.tca_ws_status(ws) == B.TCA_OK
        if (r0, r1) == first and len(parts) > 1:              # nothing below r0 has been written yet
            assert torch.isnan(out[:, :, :r0].float()).all()
    a, b = whole.view(torch.uint8), out.view(torch.uint8)
    assert torch.equal(a, b)
    ws = B.alloc_workspace(run.prm, L, B.TCA_OP_PREFILL)
    for bad in [(64, 128), (0, L + 1), (128, 128), (-128, 128)]:
        with pytest.raises(B.TcaError):
            B.tca_attn_prefill_rows(run.prm, run.dev["q"], run.dev["k"], run.dev["v"], L, bad[0], bad[1], run.cache,
                                    out, ws)


@pytest.mark.parametrize("name", ["bf16_gqa4", "bf16_d64_g2", "bf16_g7"])
def test_band_first_order_matches_the_oracle_and_row_ranges(runs, name):
    """TCA_FLAG_PREFILL_BAND_FIRST walks the window band before the selected keys (the order that
    lets the prefill start before the selection has finished): every row against the oracle, and
    row-range calls under the flag bit-identical to the single call under the flag."""
    wl, data, p, run, oracle = runs(name)
    run.prm.flags = B.TCA_FLAG_PREFILL_BAND_FIRST
    try:
        whole = H.gpu_prefill(run)
        L = run.L
        out = torch.full_like(run.dev["q"], float("nan"))
        for (r0, r1) in [(384, L), (0, 128), (128, 384)]:
            ws = B.alloc_workspace(run.prm, L, B.TCA_OP_PREFILL)
            B.tca_attn_prefill_rows(run.prm, run.dev["q"], run.dev["k"], run.dev["v"], L, r0, r1, run.cache, out, ws)
            assert B.tca_ws_status(ws) == B.TCA_OK
        assert torch.equal(whole.view(torch.uint8), out.view(torch.uint8))
    finally:
        run.prm.flags = 0
    got = H.from_device(whole)
    scale, G = H.scale_of(wl), wl.group
    for s_ in range(wl.batch):
        for h in range(wl.n_kv_heads):
            T = _oracle_T(run, wl, s_ * wl.n_kv_heads + h)
            K, V = I.widen(data["k"][s_, h, :wl.L]), I.widen(data["v"][s_, h, :wl.L])
            for g in range(G):
                want = O.attention_rows(I.widen(data["q"][s_, h * G + g, :wl.L]), K, V, T, wl.window, scale)
                H.check_attention(got[s_, h * G + g], want, wl.dtype, f"{name} band first head {h * G + g}")


@pytest.mark.parametrize("order", [0, B.TCA_FLAG_PREFILL_BAND_FIRST])
def test_the_chain_without_host_synchronisation_equals_the_synchronised_one(order):
    """score+select, compact and prefill are launched with programmatic dependent launch: each may
    be scheduled while its predecessor is still running and waits for it on the device.  Enqueued
    back to back, several times over the same buffers and with a changing input, the results must be
    those of running every call to completion first."""
    wl = SMALL["bf16_gqa4"].scaled(L=1400, seed=61)
    data = I.generate(wl)
    p = I.budget_table(wl)
    ref = H.gpu_select_compact(wl, data, p, flags=order)           # synchronises between the stages
    want = H.gpu_prefill(ref)
    torch.cuda.synchronize()
    prm, L = ref.prm, wl.L
    U = wl.batch * wl.n_kv_heads
    offsets_dev = torch.from_numpy(ref.offsets).cuda()
    q_last = ref.dev["q"][:, :, L - 1, :].contiguous()
    other = (ref.dev["k"].float() * 0.5).to(torch.bfloat16)        # a different K: different selection, different cache
    logscore = torch.empty(U, L, dtype=torch.float64, device="cuda")
    idx = torch.empty_like(ref.idx)
    ws_ss = B.alloc_workspace(prm, L, B.TCA_OP_SCORE_SELECT)
    ws_pf = B.alloc_workspace(prm, L, B.TCA_OP_PREFILL)
    tk = np.tile(ref.tbar, wl.batch).astype(np.int64)
    cache = B.Cache(prm, np.tile(ref.n_sel, wl.batch), wl.window + wl.block, tk)
    out = torch.empty_like(ref.dev["q"])
    for K_dev in (other, ref.dev["k"], other, ref.dev["k"]):       # ends on the reference input
        B.tca_score_select(prm, q_last, K_dev, L, ref.n_k, logscore, idx, offsets_dev, None, None, ws_ss)
        B.tca_compact_kv(prm, K_dev, ref.dev["v"], L, idx, offsets_dev, ref.offsets, cache)
        B.tca_attn_prefill(prm, ref.dev["q"], K_dev, ref.dev["v"], L, cache, out, ws_pf)
    torch.cuda.synchronize()
    assert B.tca_ws_status(ws_pf) == B.TCA_OK
    assert torch.equal(idx, ref.idx)
    assert torch.equal(cache.pos, ref.cache.pos) and torch.equal(cache.k.view(torch.int16), ref.cache.k.view(torch.int16))
    assert torch.equal(out.view(torch.uint8), want.view(torch.uint8))


@pytest.mark.parametrize("name", ["bf16_gqa4", "bf16_d64_g2", "bf16_g7"])
def test_bf16_prefill_reference_kernel_agrees(runs, name):
    """The FP32-pipe kernel and the default bf16 kernel see the same inputs."""
    wl, data, p, run, oracle = runs(name)
    fast = H.from_device(H.gpu_prefill(run))
    run.prm.flags = B.TCA_FLAG_PREFILL_SIMT
    try:
        slow = H.from_device(H.gpu_prefill(run))
    finally:
        run.prm.flags = 0
    H.check_attention(fast, slow, "bf16", name)


@pytest.mark.parametrize("name", list(SMALL))
def test_decode_over_retained_cache(runs, name):
    wl, data, p, run, oracle = runs(name)
    L, G = wl.L, wl.group
    q = run.dev["q"][:, :, L - 1, :].contiguous()
    out = H.from_device(H.gpu_decode(run, q))
    again = H.from_device(H.gpu_decode(run, q))
    np.testing.assert_array_equal(out, again)            # fixed split and merge order
    scale = H.scale_of(wl)
    for s in range(wl.batch):
        for h in range(wl.n_kv_heads):
            T = _oracle_T(run, wl, s * wl.n_kv_heads + h)
            K = I.widen(data["k"][s, h, :L])
            V = I.widen(data["v"][s, h, :L])
            for g in range(G):
                qv = I.widen(data["q"][s, h * G + g, L - 1])
                want = O.attention_over_set(qv, K[T], V[T], scale)
                H.check_attention(out[s, h * G + g], want, wl.dtype, f"{name} decode")


def test_hand_worked_selection_on_the_gpu(golden):
    g = golden("hand_selection.txt")
    b, w, L = int(g["block"][0]), int(g["window"][0]), int(g["length"][0])
    prm = B.make_params(1, 1, 1, 64, b, w, alpha=g["alpha"][0], dtype=B.TCA_F32)
    logscore = torch.from_numpy(np.log(np.array(g["s"]))).cuda().reshape(1, L)
    n_k, n_sel, tbar = B.tca_budget_resolve(np.array([g["p"]]), int(g["m"][0]))
    offsets = torch.tensor([0, int(n_sel[0])], dtype=torch.int64, device="cuda")
    idx = torch.zeros(int(n_sel[0]), dtype=torch.int32, device="cuda")
    h = torch.zeros(1, 5, dtype=torch.float64, device="cuda")
    t = torch.zeros(1, 5, dtype=torch.int32, device="cuda")
    B.tca_select(prm, logscore, L, n_k, idx, offsets, h, t, B.alloc_workspace(prm, L, B.TCA_OP_SELECT))
    np.testing.assert_allclose(h.cpu().numpy()[0], g["h"], rtol=1e-6)
    np.testing.assert_array_equal(t.cpu().numpy()[0], np.array(g["t"], dtype=int))
    np.testing.assert_array_equal(idx.cpu().numpy(), np.array(g["S"], dtype=int))
    assert tbar[0] == int(g["t_decode"][0])


def test_full_budget_reproduces_dense_attention():
    wl = SMALL["bf16_gqa4"].scaled(budget=("fixed", 1.0), seed=21, L=1100)
    data = I.generate(wl)
    p = I.budget_table(wl)
    run = H.gpu_select_compact(wl, data, p)
    assert int(run.n_sel.sum()) == wl.n_kv_heads * run.m * wl.block
    out = H.from_device(H.gpu_prefill(run))
    # independent dense reference: torch's causal attention in fp64 on the CPU
    q = torch.from_numpy(I.widen(data["q"]))
    k = torch.from_numpy(I.widen(data["k"])).repeat_interleave(wl.group, dim=1)
    v = torch.from_numpy(I.widen(data["v"])).repeat_interleave(wl.group, dim=1)
    att = (q @ k.transpose(-1, -2)) * H.scale_of(wl)
    att = att.masked_fill(~torch.ones(wl.L, wl.L, dtype=torch.bool).tril(), float("-inf"))
    want = (att.softmax(-1) @ v).numpy()
    H.check_attention(out, want, "bf16", "dense special case")


@pytest.mark.parametrize("L,w,b", [(100, 128, 32), (1, 4, 4), (64, 64, 16), (129, 1, 128)])
def test_degenerate_lengths(L, w, b):
    wl = BASE.scaled(batch=1, n_q_heads=2, n_kv_heads=2, head_dim=64, L=L, window=w, block=b, dtype="f32",
                     seed=31, budget=("fixed", 0.5))
    data = I.generate(wl)
    p = I.budget_table(wl)
    run = H.gpu_select_compact(wl, data, p)
    out = H.from_device(H.gpu_prefill(run))
    for h in range(2):
        res = H.oracle_select_unit(wl, data, p, 0, h, L)
        S = run.idx.cpu().numpy()[run.offsets[h]:run.offsets[h + 1]].astype(np.int64)
        assert H.compare_selection(res, S, run.t.cpu().numpy()[h, :res["m"]], b) == 0
        want = O.attention_rows(I.widen(data["q"][0, h]), I.widen(data["k"][0, h]), I.widen(data["v"][0, h]),
                                res["T"], w, H.scale_of(wl))
        H.check_attention(out[0, h], want, "f32", f"L={L}")


@pytest.mark.parametrize("d,G", [(64, 2), (128, 4)])
@pytest.mark.parametrize("L,w,b", [(100, 128, 32),    # w >= L: no blocks at all, n_global = 0
                                   (1, 4, 4),         # a single token
                                   (100, 16, 32),     # L below one 128-row tile, two blocks
                                   (129, 1, 128),     # one row into the second tile, w = 1, one block of 128
                                   (300, 40, 64),     # a global region shorter than one key tile
                                   (257, 300, 16)])   # w >= L across three query tiles
def test_degenerate_lengths_on_the_tensor_core_paths(L, w, b, d, G):
    """bf16 inputs, so the prefill runs on the tcgen05 kernel and the decode on the mma.sync kernel:
    every output row against the oracle on the method's edge cases."""
    wl = BASE.scaled(batch=1, n_q_heads=2 * G, n_kv_heads=2, head_dim=d, L=L, window=w, block=b, dtype="bf16",
                     seed=32, budget=("fixed", 0.5))
    data = I.generate(wl)
    p = I.budget_table(wl)
    run = H.gpu_select_compact(wl, data, p)
    out = H.from_device(H.gpu_prefill(run))
    run.prm.flags = B.TCA_FLAG_PREFILL_BAND_FIRST
    out_band = H.from_device(H.gpu_prefill(run))
    run.prm.flags = 0
    dec = H.from_device(H.gpu_decode(run, run.dev["q"][:, :, L - 1, :].contiguous()))
    scale = H.scale_of(wl)
    for h in range(2):
        res = H.oracle_select_unit(wl, data, p, 0, h, L)
        assert res["m"] == max(0, (L - w) // b)
        S = run.idx.cpu().numpy()[run.offsets[h]:run.offsets[h + 1]].astype(np.int64)
        assert H.compare_selection(res, S, run.t.cpu().numpy()[h, :res["m"]], b) == 0
        K, V = I.widen(data["k"][0, h]), I.widen(data["v"][0, h])
        for g in range(G):
            Q = I.widen(data["q"][0, h * G + g])
            want = O.attention_rows(Q, K, V, res["T"], w, scale)
            H.check_attention(out[0, h * G + g], want, "bf16", f"prefill L={L} w={w} b={b} d={d}")
            H.check_attention(out_band[0, h * G + g], want, "bf16", f"prefill, band first, L={L} w={w} b={b} d={d}")
            want_dec = O.attention_over_set(Q[L - 1], K[res["T"]], V[res["T"]], scale)
            H.check_attention(dec[0, h * G + g], want_dec, "bf16", f"decode L={L} w={w} b={b} d={d}")


def test_a_bounded_wait_that_runs_out_reports_timeout_and_leaves_the_gpu_usable():
    """Every mbarrier wait of the tensor-core kernels has a time limit and one way out.  The
    self-test entry point runs that way out in miniature (a wait of about a millisecond on a
    barrier nothing arrives at): the call must return, the status word must read TCA_ERR_TIMEOUT,
    and a prefill and a decode afterwards must still be right."""
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    assert B.tca_ws_status(ws) == B.TCA_OK
    B.tca_selftest_wait_expiry(ws, 1_000_000, waited)
    assert B.tca_ws_status(ws) == B.TCA_ERR_TIMEOUT                  # synchronises: the kernel has returned
    assert 1_000_000 <= int(waited.item()) < 1_000_000_000           # gave up after the limit, well inside a second
    assert B.tca_ws_status(ws) == B.TCA_ERR_TIMEOUT                  # sticky until the caller clears it
    with pytest.raises(B.TcaError):
        B.tca_selftest_wait_expiry(ws, 10, waited)                   # limits outside 1 us .. 100 ms are refused
    # a prefill on a workspace whose status word is set returns at once and leaves O alone
    wl = SMALL["bf16_d64_g2"]
    data = I.generate(wl)
    p = I.budget_table(wl)
    run = H.gpu_select_compact(wl, data, p)
    ws_bad = B.alloc_workspace(run.prm, run.L, B.TCA_OP_PREFILL)
    ws_bad[:4] = torch.tensor([1, 0, 0, 0], dtype=torch.uint8, device="cuda")
    O_dev = torch.full_like(run.dev["q"], 7.0)
    B.tca_attn_prefill(run.prm, run.dev["q"], run.dev["k"], run.dev["v"], run.L, run.cache, O_dev, ws_bad)
    assert B.tca_ws_status(ws_bad) == B.TCA_ERR_TIMEOUT
    assert bool((O_dev == 7.0).all())
    # and the device is fine: the normal paths still match the oracle
    out = H.from_device(H.gpu_prefill(run))
    dec = H.from_device(H.gpu_decode(run, run.dev["q"][:, :, wl.L - 1, :].contiguous()))
    scale, G = H.scale_of(wl), wl.group
    for h in range(wl.n_kv_heads):
        T = _oracle_T(run, wl, h)
        K, V = I.widen(data["k"][0, h, :wl.L]), I.widen(data["v"][0, h, :wl.L])
        Q = I.widen(data["q"][0, h * G, :wl.L])
        H.check_attention(out[0, h * G], O.attention_rows(Q, K, V, T, wl.window, scale), "bf16", "prefill after expiry")
        H.check_attention(dec[0, h * G], O.attention_over_set(Q[wl.L - 1], K[T], V[T], scale), "bf16",
                          "decode after expiry")


@pytest.mark.parametrize("name,steps", [("bf16_gqa4", 150), ("bf16_d64_g2", 40), ("f32_g3_b1", 20),
                                        ("f32_d128_g8", 30)])
def test_append_compress_and_decode_steps(name, steps):
    wl = SMALL[name].scaled(decode_steps=steps)
    data = I.generate(wl)
    p = I.budget_table(wl)
    L, G, b, w = wl.L, wl.group, wl.block, wl.window
    n_compress = (L + steps - w) // b - (L - w) // b
    run = H.gpu_select_compact(wl, data, p, extra_blocks=n_compress + 1)
    scale = H.scale_of(wl)
    caches = {}
    for s in range(wl.batch):
        for h in range(wl.n_kv_heads):
            u = s * wl.n_kv_heads + h
            S = run.idx.cpu().numpy()[run.offsets[u]:run.offsets[u + 1]].astype(np.int64)
            caches[u] = O.DecodeCache.from_prefill(S, run.m, L, b, w, p[h], scale)
            assert caches[u].t_keep == run.tbar[h]
    Kw, Vw, Qw = I.widen(data["k"]), I.widen(data["v"]), I.widen(data["q"])
    dk, dv, dq = (H.to_device(data[x], wl.dtype) for x in ("k", "v", "q"))
    fired = 0
    for step in range(steps):
        pos = L + step
        B.tca_cache_append(run.prm, run.cache, dk[:, :, pos].contiguous(), dv[:, :, pos].contiguous(),
                           dq[:, :, pos].contiguous())
        out = H.from_device(H.gpu_decode(run, dq[:, :, pos].contiguous()))
        cpos = run.cache.pos.cpu().numpy()
        state = run.cache.state.cpu().numpy().reshape(-1, B.TCA_STATE_WORDS)
        for s in range(wl.batch):
            for h in range(wl.n_kv_heads):
                u = s * wl.n_kv_heads + h
                kept = caches[u].append(pos, Qw[s, h * G:(h + 1) * G, pos], Kw[s, h])
                fired += kept is not None
                rows = run.cache.unit_rows(u)
                np.testing.assert_array_equal(cpos[rows], caches[u].positions())
                assert state[u, 2] == run.cache.n_global[u] == len(caches[u].glob)
                assert state[u, 4] == run.cache.n_tail[u] == len(caches[u].tail)
                assert state[u, 3] == run.cache.tail_head[u] and state[u, 5] == pos + 1
                if step % 7 == 0 or kept is not None or step == steps - 1:
                    for g in range(G):
                        want = caches[u].attend(Qw[s, h * G + g, pos], Kw[s, h], Vw[s, h])
                        H.check_attention(out[s, h * G + g], want, wl.dtype, f"{name} step {step}")
    assert fired == n_compress * wl.batch * wl.n_kv_heads and n_compress >= 1
    # the compressed cache holds exactly the rows of K and V it claims to hold
    raw = torch.int16 if wl.dtype == "bf16" else torch.int32
    Kc = run.cache.k.view(raw).cpu().numpy()
    for u, c in caches.items():
        s, h = divmod(u, wl.n_kv_heads)
        np.testing.assert_array_equal(Kc[run.cache.unit_rows(u)], data["k"][s, h, c.positions()].view(Kc.dtype))


@pytest.mark.parametrize("name", ["config1", "bf16_gqa4", "bf16_g7", "f32_g3_b1"])
def test_fused_score_select_is_bit_identical_to_the_two_calls(runs, name):
    """tca_score_select (the block metric formed in the tail of the score kernel) against
    tca_score + tca_select: same log s, h, t and index set, bit for bit."""
    wl, data, p, run, oracle = runs(name)
    fused = H.gpu_select_compact(wl, data, p, fused=True)
    assert torch.equal(fused.logscore.view(torch.int64), run.logscore.view(torch.int64))
    assert torch.equal(fused.h.view(torch.int64), run.h.view(torch.int64))
    assert torch.equal(fused.t, run.t) and torch.equal(fused.idx, run.idx)
    assert torch.equal(fused.cache.pos, run.cache.pos)


@pytest.mark.parametrize("name", ["config1", "bf16_gqa4", "bf16_d64_g2", "bf16_g7"])
@pytest.mark.parametrize("variant", ["entropy", "random", "flat"])
def test_selection_variants_match_their_oracles(name, variant):
    """The ablation variants (entropy concentration index, seeded random block order) and the flat
    top-B as modes of tca_select, through score -> select -> compact -> prefill, each against the
    oracle's variant; the fused call takes the same path for the entropy index."""
    wl = SMALL[name]
    data = I.generate(wl)
    p = I.budget_table(wl)
    flags = {"entropy": B.TCA_FLAG_ENTROPY_INDEX, "random": B.TCA_FLAG_RANDOM_ORDER, "flat": B.TCA_FLAG_FLAT_TOPB}[variant]
    seed = 12345
    run = H.gpu_select_compact(wl, data, p, flags=flags, seed=seed, fused=(variant == "entropy"))
    idx, t, hh = run.idx.cpu().numpy(), run.t.cpu().numpy(), run.h.cpu().numpy()
    G, scale = wl.group, H.scale_of(wl)
    differs = 0
    for s_ in range(wl.batch):
        for h in range(wl.n_kv_heads):
            u = s_ * wl.n_kv_heads + h
            K = I.widen(data["k"][s_, h, :wl.L])
            q_last = I.widen(data["q"][s_, h * G:(h + 1) * G, wl.L - 1])
            res = O.select_head_variant(q_last, K, p[h], wl.block, wl.window, float(np.float32(wl.alpha)), scale,
                                        variant, seed=seed, unit=u)
            S = idx[run.offsets[u]:run.offsets[u + 1]].astype(np.int64)
            if variant == "flat":
                assert H.compare_flat_selection(res["log_s"], S, int(run.n_sel[h]), res["m"] * wl.block) <= 1
            else:
                if variant == "random":
                    np.testing.assert_array_equal(hh[u, :res["m"]], res["h"])          # the hash keys, exactly
                else:
                    np.testing.assert_allclose(hh[u, :res["m"]], res["h"], rtol=2e-6, atol=1e-12)
                assert H.compare_selection(res, S, t[u, :res["m"]], wl.block) <= 1
            base = O.select_head(q_last, K, p[h], wl.block, wl.window, float(np.float32(wl.alpha)), scale)
            differs += not np.array_equal(base["S"], S)
    assert differs > 0 or variant == "entropy"       # a variant that changed nothing would test nothing
    # the rest of the path does not care how the set was chosen
    out = H.from_device(H.gpu_prefill(run))
    u = wl.batch * wl.n_kv_heads - 1
    s_, h = divmod(u, wl.n_kv_heads)
    T = _oracle_T(run, wl, u)
    rows = H.sample_rows(wl.L, wl.window, wl.block, 16, seed=3)
    want = O.attention_rows(I.widen(data["q"][s_, h * G, :wl.L]), I.widen(data["k"][s_, h, :wl.L]),
                            I.widen(data["v"][s_, h, :wl.L]), T, wl.window, scale, rows)
    H.check_attention(out[s_, h * G][rows], want, wl.dtype, f"{name} {variant}")


def test_flat_top_b_at_a_size_with_many_radix_passes_and_ties():
    """The flat variant's radix select over tens of thousands of candidates, with exact ties at the
    threshold (scores injected directly): equal keys go to the lower position."""
    L, b, w = 40000, 64, 1088
    m = (L - w) // b
    prm = B.make_params(1, 1, 1, 64, b, w, dtype=B.TCA_F32, flags=B.TCA_FLAG_FLAT_TOPB)
    rng = np.random.default_rng(77)
    ls = np.round(rng.standard_normal(L) * 3.0, 2)               # two decimals: thousands of exact ties
    logscore = torch.from_numpy(ls).cuda().reshape(1, L)
    pk = np.zeros((1, 7)); pk[0, 2] = 1.0                        # 4 tokens per block
    n_k, n_sel, _ = B.tca_budget_resolve(pk, m)
    offsets = torch.tensor([0, int(n_sel[0])], dtype=torch.int64, device="cuda")
    idx = torch.full((int(n_sel[0]),), -1, dtype=torch.int32, device="cuda")
    B.tca_select(prm, logscore, L, n_k, idx, offsets, None, None, B.alloc_workspace(prm, L, B.TCA_OP_SELECT))
    np.testing.assert_array_equal(idx.cpu().numpy(), O.select_tokens_flat(ls, int(n_sel[0]), m * b))


def test_capacity_and_workspace_errors():
    wl = SMALL["bf16_d64_g2"]
    data = I.generate(wl)
    p = I.budget_table(wl)
    run = H.gpu_select_compact(wl, data, p)
    q = run.dev["q"][:, :, wl.L - 1, :].contiguous()
    out = torch.empty_like(q)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.TcaError) as e:
        B.tca_attn_decode(run.prm, q, run.cache, out, small)
    assert e.value.status == B.TCA_ERR_WORKSPACE
    # a cache without room for the next compressed block refuses the append that would overflow it
    steps_to_full = wl.window + wl.block - int(run.cache.n_tail[0])
    k1, v1 = run.dev["k"][:, :, 0].contiguous(), run.dev["v"][:, :, 0].contiguous()
    for _ in range(steps_to_full - 1):
        B.tca_cache_append(run.prm, run.cache, k1, v1, q)
    with pytest.raises(B.TcaError) as e:
        B.tca_cache_append(run.prm, run.cache, k1, v1, q)
    assert e.value.status == B.TCA_ERR_CAPACITY
    torch.cuda.synchronize()
