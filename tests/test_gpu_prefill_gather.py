"""The prefill that fetches the selected keys from K and V by index inside the attention kernel
(no cache, no compaction): against the oracle on every row, and bit for bit against
compaction + prefill over the same selection."""
import numpy as np
import pytest
import torch

from oracle import tca_oracle as O
from paper_2512_09238_b200 import binding as B
from paper_2512_09238_b200 import inputs as I
import tca_harness as H

pytestmark = pytest.mark.gpu

BASE = I.WORKLOADS["config1"]
SHAPES = {
    # GQA 4:1, d = 128, ragged everywhere, per-head budgets between 5 % and 100 %
    "bf16_gqa4": BASE.scaled(name="bf16_gqa4", batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, L=1500,
                             dtype="bf16", block=64, window=256, seed=11, budget=("beta", 2.0, 5.0, 0.05, 1.0)),
    "bf16_d64_g2": BASE.scaled(name="bf16_d64_g2", batch=1, n_q_heads=4, n_kv_heads=2, head_dim=64, L=777,
                               dtype="bf16", block=16, window=100, seed=12),
    # a group of 7: the last CTA of a unit holds one head only
    "bf16_g7": BASE.scaled(name="bf16_g7", batch=1, n_q_heads=7, n_kv_heads=1, head_dim=128, L=1000,
                           dtype="bf16", block=128, window=300, seed=14, budget=("fixed", 0.3)),
    # several key tiles of selected rows per query tile and a short window
    "bf16_long_global": BASE.scaled(name="bf16_long_global", batch=1, n_q_heads=4, n_kv_heads=2, head_dim=128,
                                    L=3000, dtype="bf16", block=32, window=64, seed=15, budget=("fixed", 0.6)),
}


def gather_prefill(run, flags=0, ranges=None):
    out = torch.full_like(run.dev["q"], float("nan"))
    offsets_dev = torch.from_numpy(run.offsets).cuda()
    run.prm.flags = flags
    try:
        for (r0, r1) in (ranges or [(0, run.L)]):
            ws = B.alloc_workspace(run.prm, run.L, B.TCA_OP_PREFILL)
            B.tca_attn_prefill_gather(run.prm, run.dev["q"], run.dev["k"], run.dev["v"], run.L, r0, r1, run.idx,
                                      offsets_dev, out, ws)
            assert B.tca_ws_status(ws) == B.TCA_OK
    finally:
        run.prm.flags = 0
    return out


@pytest.mark.parametrize("name", list(SHAPES))
def test_gather_prefill_matches_the_oracle_and_the_cache_path(name):
    wl = SHAPES[name]
    data = I.generate(wl)
    p = I.budget_table(wl)
    run = H.gpu_select_compact(wl, data, p)
    via_cache = H.gpu_prefill(run)
    got_dev = gather_prefill(run)
    assert torch.equal(got_dev.view(torch.uint8), via_cache.view(torch.uint8))
    # band first, and as row ranges in a shuffled order: still the same bits
    L = run.L
    cuts = [c for c in (0, 128, 640) if c < L] + [L]
    parts = list(zip(cuts[:-1], cuts[1:]))
    band = gather_prefill(run, flags=B.TCA_FLAG_PREFILL_BAND_FIRST, ranges=parts[::-1])
    run.prm.flags = B.TCA_FLAG_PREFILL_BAND_FIRST
    band_cache = H.gpu_prefill(run)
    run.prm.flags = 0
    assert torch.equal(band.view(torch.uint8), band_cache.view(torch.uint8))
    got = H.from_device(got_dev)
    scale, G = H.scale_of(wl), wl.group
    idx = run.idx.cpu().numpy()
    for s in range(wl.batch):
        for h in range(wl.n_kv_heads):
            u = s * wl.n_kv_heads + h
            S = idx[run.offsets[u]:run.offsets[u + 1]].astype(np.int64)
            T = O.retained_set(S, run.m, wl.block, wl.L)
            K, V = I.widen(data["k"][s, h, :L]), I.widen(data["v"][s, h, :L])
            for g in range(G):
                want = O.attention_rows(I.widen(data["q"][s, h * G + g, :L]), K, V, T, wl.window, scale)
                H.check_attention(got[s, h * G + g], want, "bf16", f"{name} gather seq {s} head {h * G + g}")


@pytest.mark.parametrize("d,G", [(64, 2), (128, 4)])
@pytest.mark.parametrize("L,w,b", [(100, 128, 32),    # no blocks at all: nothing to gather
                                   (1, 4, 4),
                                   (129, 1, 128),     # one block of 128, w = 1
                                   (300, 40, 64),     # fewer selected keys than one key tile
                                   (257, 300, 16)])
def test_gather_prefill_on_degenerate_shapes(L, w, b, d, G):
    wl = BASE.scaled(batch=1, n_q_heads=2 * G, n_kv_heads=2, head_dim=d, L=L, window=w, block=b, dtype="bf16",
                     seed=32, budget=("fixed", 0.5))
    data = I.generate(wl)
    p = I.budget_table(wl)
    run = H.gpu_select_compact(wl, data, p)
    via_cache = H.gpu_prefill(run)
    assert torch.equal(gather_prefill(run).view(torch.uint8), via_cache.view(torch.uint8))
    # the other order rounds differently from the first, so it goes against the oracle
    got = H.from_device(gather_prefill(run, flags=B.TCA_FLAG_PREFILL_BAND_FIRST))
    scale = H.scale_of(wl)
    for h in range(2):
        res = H.oracle_select_unit(wl, data, p, 0, h, L)
        K, V = I.widen(data["k"][0, h]), I.widen(data["v"][0, h])
        for g in range(G):
            want = O.attention_rows(I.widen(data["q"][0, h * G + g]), K, V, res["T"], w, scale)
            H.check_attention(got[0, h * G + g], want, "bf16", f"gather, band first, L={L} w={w} b={b} d={d}")


def test_gather_prefill_straight_after_the_selection_without_host_synchronisation():
    """score + select -> gather prefill, enqueued back to back over the same buffers with a changing
    K: the kernel waits on the device for the index set it reads."""
    wl = SHAPES["bf16_gqa4"].scaled(L=1400, seed=62)
    data = I.generate(wl)
    p = I.budget_table(wl)
    ref = H.gpu_select_compact(wl, data, p)
    want = H.gpu_prefill(ref)
    torch.cuda.synchronize()
    prm, L = ref.prm, wl.L
    U = wl.batch * wl.n_kv_heads
    offsets_dev = torch.from_numpy(ref.offsets).cuda()
    q_last = ref.dev["q"][:, :, L - 1, :].contiguous()
    other = (ref.dev["k"].float() * 0.5).to(torch.bfloat16)
    logscore = torch.empty(U, L, dtype=torch.float64, device="cuda")
    idx = torch.empty_like(ref.idx)
    ws_ss = B.alloc_workspace(prm, L, B.TCA_OP_SCORE_SELECT)
    ws_pf = B.alloc_workspace(prm, L, B.TCA_OP_PREFILL)
    for order in (0, B.TCA_FLAG_PREFILL_BAND_FIRST):
        out = torch.empty_like(ref.dev["q"])
        prm.flags = order
        try:
            for K_dev in (other, ref.dev["k"], other, ref.dev["k"]):
                B.tca_score_select(prm, q_last, K_dev, L, ref.n_k, logscore, idx, offsets_dev, None, None, ws_ss)
                B.tca_attn_prefill_gather(prm, ref.dev["q"], K_dev, ref.dev["v"], L, 0, L, idx, offsets_dev, out, ws_pf)
            torch.cuda.synchronize()
            assert B.tca_ws_status(ws_pf) == B.TCA_OK
            assert torch.equal(idx, ref.idx)
            if order == 0:
                assert torch.equal(out.view(torch.uint8), want.view(torch.uint8))
            else:
                ref.prm.flags = order
                assert torch.equal(out.view(torch.uint8), H.gpu_prefill(ref).view(torch.uint8))
        finally:
            prm.flags = 0


def test_gather_prefill_refuses_what_it_does_not_support():
    wl = BASE.scaled(batch=1, n_q_heads=2, n_kv_heads=1, head_dim=64, L=300, window=32, block=16, dtype="f32", seed=5)
    data = I.generate(wl)
    run = H.gpu_select_compact(wl, data, I.budget_table(wl))
    out = torch.empty_like(run.dev["q"])
    ws = B.alloc_workspace(run.prm, run.L, B.TCA_OP_PREFILL)
    offsets_dev = torch.from_numpy(run.offsets).cuda()
    with pytest.raises(B.TcaError):                       # fp32: no tensor-core kernel
        B.tca_attn_prefill_gather(run.prm, run.dev["q"], run.dev["k"], run.dev["v"], run.L, 0, run.L, run.idx,
                                  offsets_dev, out, ws)
