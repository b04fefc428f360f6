"""Shared helpers for the GPU parity tests: run the CUDA path through the C ABI, run the
oracle on the same seeded inputs, and compare under the stated rules."""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np
import torch

from oracle import tca_oracle as O
from paper_2512_09238_b200 import binding as B
from paper_2512_09238_b200 import inputs as I

# Tolerances.  Selection: index sets bit-exact except where the oracle's scores at the
# budget boundary differ by less than 1e-5 relative (= 1e-5 absolute in log s).
# Attention: fp32 inputs max-abs <= 1e-4; bf16 inputs max-abs <= 2e-2 and rel. L2 <= 5e-3.
SEL_TOL = 1e-5
ATT_TOL = {"f32": dict(max_abs=1e-4, rel_l2=1e-4), "bf16": dict(max_abs=2e-2, rel_l2=5e-3)}
LOGSCORE_TOL = 2e-6      # fp64 dot products; only the final exp/log of the group mean is fp32


def to_device(a: np.ndarray, dtype: str) -> torch.Tensor:
    if dtype == "bf16":
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def from_device(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def params_for(wl: I.Workload, flags: int = 0, seed: int = 0) -> B.tca_params:
    return B.make_params(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.block, wl.window,
                         alpha=wl.alpha, dtype=B.TCA_BF16 if wl.dtype == "bf16" else B.TCA_F32, flags=flags, seed=seed)


def scale_of(wl: I.Workload) -> float:
    """The float32 value the library receives, as a double (so both sides use the same number)."""
    return float(np.float32(1.0 / math.sqrt(wl.head_dim)))


@dataclass
class DeviceRun:
    prm: B.tca_params
    wl: I.Workload
    L: int
    m: int
    n_k: np.ndarray
    n_sel: np.ndarray
    tbar: np.ndarray
    offsets: np.ndarray           # host [U+1]
    logscore: torch.Tensor        # [U, L] float64
    h: Optional[torch.Tensor]
    t: Optional[torch.Tensor]
    idx: torch.Tensor
    cache: B.Cache
    dev: Dict[str, torch.Tensor]


def gpu_select_compact(wl: I.Workload, data: Dict[str, np.ndarray], p: np.ndarray, L: Optional[int] = None,
                       extra_blocks: int = 0, flags: int = 0, seed: int = 0, fused: bool = False) -> DeviceRun:
    """score -> select -> compact on the GPU for the first L tokens of `data` (fused: score and
    select through the single tca_score_select call)."""
    L = wl.L if L is None else L
    prm = params_for(wl, flags, seed)
    U = wl.batch * wl.n_kv_heads
    dev = {k: to_device(np.ascontiguousarray(v[:, :, :L]), wl.dtype) for k, v in data.items()}
    m = max(0, (L - wl.window) // wl.block)
    n_k, n_sel, tbar = B.tca_budget_resolve(p, m)
    per_unit = np.tile(n_sel, wl.batch)
    offsets = np.zeros(U + 1, dtype=np.int64)
    offsets[1:] = np.cumsum(per_unit)
    offsets_dev = torch.from_numpy(offsets).cuda()
    logscore = torch.empty(U, L, dtype=torch.float64, device="cuda")
    q_last = dev["q"][:, :, L - 1, :].contiguous()
    idx = torch.full((max(1, int(offsets[-1])),), -1, dtype=torch.int32, device="cuda")
    h = torch.zeros(U, max(1, m), dtype=torch.float64, device="cuda")
    t = torch.zeros(U, max(1, m), dtype=torch.int32, device="cuda")
    if fused:
        ws = B.alloc_workspace(prm, L, B.TCA_OP_SCORE_SELECT)
        B.tca_score_select(prm, q_last, dev["k"], L, n_k, logscore, idx, offsets_dev, h, t, ws)
        assert B.tca_ws_status(ws[B.tca_workspace_bytes(prm, L, B.TCA_OP_SCORE_SELECT)
                                  - B.tca_workspace_bytes(prm, L, B.TCA_OP_SELECT):]) == B.TCA_OK
    else:
        B.tca_score(prm, q_last, dev["k"], L, logscore, B.alloc_workspace(prm, L, B.TCA_OP_SCORE))
        ws = B.alloc_workspace(prm, L, B.TCA_OP_SELECT)
        B.tca_select(prm, logscore, L, n_k, idx, offsets_dev, h, t, ws)
        assert B.tca_ws_status(ws) == B.TCA_OK
    tk = np.tile(tbar, wl.batch).astype(np.int64)
    cache = B.Cache(prm, per_unit + extra_blocks * tk, wl.window + wl.block, tk)
    B.tca_compact_kv(prm, dev["k"], dev["v"], L, idx, offsets_dev, offsets, cache)
    torch.cuda.synchronize()
    return DeviceRun(prm, wl, L, m, n_k, n_sel, tbar, offsets, logscore, h, t, idx, cache, dev)


def gpu_prefill(run: DeviceRun) -> torch.Tensor:
    O_dev = torch.empty_like(run.dev["q"])
    ws = B.alloc_workspace(run.prm, run.L, B.TCA_OP_PREFILL)
    B.tca_attn_prefill(run.prm, run.dev["q"], run.dev["k"], run.dev["v"], run.L, run.cache, O_dev, ws)
    assert B.tca_ws_status(ws) == B.TCA_OK
    return O_dev


def gpu_decode(run: DeviceRun, q: torch.Tensor) -> torch.Tensor:
    out = torch.empty_like(q)
    ws = B.alloc_workspace(run.prm, run.cache.rows_total, B.TCA_OP_DECODE)
    B.tca_attn_decode(run.prm, q, run.cache, out, ws)
    assert B.tca_ws_status(ws) == B.TCA_OK          # synchronises; a wait that gave up would leave stale partials
    return out


# ----------------------------------------------------------------------------- oracle side
def oracle_select_unit(wl: I.Workload, data, p, seq: int, h: int, L: int):
    G = wl.group
    K = I.widen(data["k"][seq, h, :L])
    q_last = I.widen(data["q"][seq, h * G:(h + 1) * G, L - 1])
    return O.select_head(q_last, K, p[h], wl.block, wl.window, float(np.float32(wl.alpha)), scale_of(wl))


def compare_selection(res: dict, gpu_S: np.ndarray, gpu_t: np.ndarray, b: int) -> int:
    """Applies the 1e-5 rule.  Returns the number of accepted differences; raises on a
    difference the rule does not cover."""
    S_o, t_o, h, ls, n = res["S"], res["t"], res["h"], res["log_s"], res["n"]
    m = res["m"]
    assert np.all(np.diff(gpu_S) > 0), "indices must be strictly ascending"
    assert len(gpu_S) == len(S_o), "retained count must equal the budget"
    if np.array_equal(gpu_S, S_o):
        return 0
    accepted = 0
    psi = O.budget_map(n, b)
    order = np.argsort(h, kind="stable")
    hs = h[order]
    edges = [r for r in range(1, m) if psi[r] != psi[r - 1]]
    edge_vals = np.array([hs[r - 1] for r in edges] + [hs[r] for r in edges])
    np.testing.assert_array_equal(np.sort(gpu_t), psi)      # still a permutation of Psi
    for j in range(m):
        blk = ls[j * b:(j + 1) * b]
        got = gpu_S[(gpu_S // b) == j] - j * b
        assert len(got) == gpu_t[j]
        if gpu_t[j] != t_o[j]:
            near = np.min(np.abs(edge_vals - h[j])) <= SEL_TOL * abs(h[j])
            assert near, f"block {j}: t differs ({gpu_t[j]} vs {t_o[j]}) away from a run boundary"
            accepted += 1
        want = np.sort(np.argsort(-blk, kind="stable")[:gpu_t[j]])
        if not np.array_equal(got, want):
            tj = int(gpu_t[j])
            boundary = np.sort(blk)[::-1][tj - 1]
            diff = np.setxor1d(got, want)
            assert np.all(np.abs(blk[diff] - boundary) < SEL_TOL), f"block {j}: wrong tokens kept"
            accepted += len(diff) // 2
    return accepted


def check_attention(got: np.ndarray, want: np.ndarray, dtype: str, what: str = "") -> None:
    tol = ATT_TOL[dtype]
    err = np.max(np.abs(got - want))
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
    assert err <= tol["max_abs"], f"{what}: max abs error {err:.3e} > {tol['max_abs']}"
    assert rel <= tol["rel_l2"], f"{what}: relative L2 error {rel:.3e} > {tol['rel_l2']}"


def sample_rows(L: int, w: int, b: int, n_random: int, seed: int) -> List[int]:
    """Query rows worth checking: first/last rows, rows around the window and block and
    tile edges, plus random ones."""
    rows = {0, 1, 2, 3, L - 1, L - 2, L // 2}
    for c in (w - 1, w, w + 1, w + b - 1, w + b, w + b + 1, 127, 128, 129, 63, 64, 65):
        if 0 <= c < L:
            rows.add(c)
    rng = np.random.default_rng(seed)
    rows.update(int(x) for x in rng.integers(0, L, size=n_random))
    return sorted(rows)


def compare_flat_selection(log_s: np.ndarray, gpu_S: np.ndarray, n_keep: int, n_candidates: int) -> int:
    """The 1e-5 rule for the flat top-B variant: the GPU's set equals the oracle's, or differs only
    in tokens whose oracle score is within 1e-5 of the n_keep-th largest.  Returns accepted swaps."""
    want = O.select_tokens_flat(log_s, n_keep, n_candidates)
    assert np.all(np.diff(gpu_S) > 0) and len(gpu_S) == n_keep and (n_keep == 0 or gpu_S.max() < n_candidates)
    if np.array_equal(gpu_S, want):
        return 0
    boundary = np.sort(log_s[:n_candidates])[::-1][n_keep - 1]
    diff = np.setxor1d(gpu_S, want)
    assert np.all(np.abs(log_s[diff] - boundary) < SEL_TOL), "flat top-B kept the wrong tokens"
    return len(diff) // 2
