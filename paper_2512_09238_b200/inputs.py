"""Seeded synthetic inputs shaped like the paper's long-context workloads.

This module only *draws data*: clustered keys/queries, values and per-head budget
tables.  It contains none of the method's arithmetic (no scoring, no selection, no
attention) and is the one module that both the CPU oracle's tests and the CUDA path's
tests/bench import, so that both sides see exactly the same bits.

The paper evaluates on LongBench-E / RULER prompts run through LLaMA-3.1-8B and
Qwen2.5-7B (Experiments, Setup); those datasets and weights are not available, so the
generator below stands in for them: a single attention layer with the same head
geometry, keys that form runs of near-duplicates (a sticky Markov chain over cluster
centroids, which is the redundancy the block metric of Eq. 6 is meant to find) and a
few heavy "sink" tokens with a 4x larger key norm.

Recipe, per (sequence, KV head), numpy ``Generator(PCG64(SeedSequence([seed, seq, head])))``:
  centroids  C[nc, d]  ~ N(0, 1)
  chain      z_0 ~ U{0..nc-1};  z_t = z_{t-1} with probability ``stay`` else U{0..nc-1}
  keys       k_t = C[z_t] + noise * N(0, 1)
  heavy set  tokens 0..3 and Bernoulli(heavy_rate); heavy keys (and queries) are scaled 4x
  values     v_t ~ N(0, 1)
  queries    every query head of the group shares C, z and the heavy set of its KV
             head, with independent noise: q_t = C[z_t] + noise * N(0, 1)
Arrays are drawn in float32, cast once to the workload dtype (bf16 = round to nearest
even) and handed unchanged to both sides.

Budget tables: the library's input is, per KV head, a configuration p over the retain
counts {1, 2, 4, ..., b} (Section 4.1).  A workload states a scalar fraction f_h of the
candidate tokens to keep; it is turned into p with the paper's log-Gaussian family
(Eq. 3, sigma = 1) by bisecting mu until sum_k k * p_k = f_h * b.  This is input
synthesis standing in for the offline calibration (Algorithm 1), not part of the
online path.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Tuple

import numpy as np

__all__ = [
    "Workload", "WORKLOADS", "generate", "budget_fractions", "fraction_to_p",
    "budget_table", "to_bf16_bits", "bf16_bits_to_f32", "widen",
]


# --------------------------------------------------------------------------- dtype helpers
def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float32 (exact)."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def widen(a: np.ndarray) -> np.ndarray:
    """Workload array (float32, or uint16 holding bf16 bits) -> float64, exactly."""
    if a.dtype == np.uint16:
        return bf16_bits_to_f32(a).astype(np.float64)
    return a.astype(np.float64)


# --------------------------------------------------------------------------- workloads
@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    L: int                    # prefill length
    dtype: str                # "f32" | "bf16"
    block: int                # b
    window: int               # w
    alpha: float = 0.5
    n_centroids: int = 64
    stay: float = 0.9
    heavy_rate: float = 0.01
    noise: float = 0.1
    seed: int = 0
    budget: Tuple = ("uniform", 0.25, 0.75)   # ("uniform", lo, hi) | ("beta", a, b, lo, hi) | ("fixed", f)
    decode_steps: int = 0     # extra tokens generated after L for the decode phase
    sigma: float = 1.0        # width of the log-Gaussian budget family

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_blocks(self) -> int:
        return max(0, (self.L - self.window) // self.block)

    @property
    def n_counts(self) -> int:          # |{1, 2, 4, ..., b}|
        return int(self.block).bit_length()

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark configurations (hyper-parameters b=128, w=4096, alpha=0.5 are the
# paper's; the first one is too short for w=4096 and uses b=32, w=128).
WORKLOADS: Dict[str, Workload] = {
    "config1": Workload("config1", 1, 8, 8, 64, 2048, "f32", 32, 128,
                        n_centroids=64, stay=0.9, heavy_rate=0.01, seed=0,
                        budget=("uniform", 0.25, 0.75)),
    "config2": Workload("config2", 4, 32, 8, 128, 32768, "bf16", 128, 4096,
                        n_centroids=256, stay=0.95, heavy_rate=0.005, seed=1,
                        budget=("beta", 2.0, 5.0, 0.05, 1.0)),
    "config3": Workload("config3", 1, 32, 8, 128, 32768, "bf16", 128, 4096,
                        n_centroids=64, stay=0.9, heavy_rate=0.01, seed=2,
                        budget=("beta", 2.0, 5.0, 0.05, 1.0)),
    "config4": Workload("config4", 1, 32, 8, 128, 131072, "bf16", 128, 4096,
                        n_centroids=1024, stay=0.97, heavy_rate=0.002, seed=3,
                        budget=("beta", 2.0, 5.0, 0.05, 1.0), decode_steps=256),
    "config5": Workload("config5", 2, 32, 8, 128, 65536, "bf16", 128, 4096,
                        n_centroids=256, stay=0.95, heavy_rate=0.005, seed=4,
                        budget=("fixed", 0.25), decode_steps=64),
}


# --------------------------------------------------------------------------- data
def _rng(seed: int, *stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, *stream])))


def _cast(x32: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return to_bf16_bits(x32)
    if dtype == "f32":
        return np.ascontiguousarray(x32, dtype=np.float32)
    raise ValueError(f"unknown dtype {dtype!r}")


def generate(wl: Workload) -> Dict[str, np.ndarray]:
    """Draw Q, K, V for a workload.

    Returns ``{"q": [B, Hq, T, d], "k": [B, Hkv, T, d], "v": [B, Hkv, T, d]}`` with
    ``T = L + decode_steps``; float32 arrays for "f32", uint16 bf16 bit patterns for
    "bf16".  Positions ``>= L`` are the tokens appended during decoding.
    """
    B, Hq, Hkv, d, G = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.group
    T = wl.L + wl.decode_steps
    odt = np.uint16 if wl.dtype == "bf16" else np.float32
    q = np.empty((B, Hq, T, d), dtype=odt)
    k = np.empty((B, Hkv, T, d), dtype=odt)
    v = np.empty((B, Hkv, T, d), dtype=odt)
    for s in range(B):
        for h in range(Hkv):
            rng = _rng(wl.seed, s, h)
            C = rng.standard_normal((wl.n_centroids, d), dtype=np.float32)
            # sticky Markov chain: z_t = fresh draw where the chain jumps, else carried
            fresh = rng.integers(0, wl.n_centroids, size=T)
            jump = rng.random(T) >= wl.stay
            jump[0] = True
            last_jump = np.maximum.accumulate(np.where(jump, np.arange(T), 0))
            z = fresh[last_jump]
            heavy = rng.random(T) < wl.heavy_rate
            heavy[:4] = True
            gain = np.where(heavy, np.float32(4.0), np.float32(1.0))[:, None]
            base = C[z]
            kk = (base + np.float32(wl.noise) * rng.standard_normal((T, d), dtype=np.float32)) * gain
            k[s, h] = _cast(kk, wl.dtype)
            v[s, h] = _cast(rng.standard_normal((T, d), dtype=np.float32), wl.dtype)
            for g in range(G):
                qq = (base + np.float32(wl.noise) * rng.standard_normal((T, d), dtype=np.float32)) * gain
                q[s, h * G + g] = _cast(qq, wl.dtype)
    return {"q": q, "k": k, "v": v}


# --------------------------------------------------------------------------- budgets
def budget_fractions(wl: Workload) -> np.ndarray:
    """Per-KV-head fraction f_h of candidate tokens to keep (shared across the batch)."""
    rng = _rng(wl.seed, 0xB0D6E7)
    kind = wl.budget[0]
    H = wl.n_kv_heads
    if kind == "uniform":
        _, lo, hi = wl.budget
        return lo + (hi - lo) * rng.random(H)
    if kind == "beta":
        _, a, b, lo, hi = wl.budget
        return lo + (hi - lo) * rng.beta(a, b, size=H)
    if kind == "fixed":
        return np.full(H, float(wl.budget[1]))
    raise ValueError(f"unknown budget kind {kind!r}")


def _log_gaussian_row(mu: float, n_counts: int, sigma: float) -> np.ndarray:
    x = np.arange(n_counts, dtype=np.float64)           # log2 of 1, 2, 4, ..., b
    z = -((x - mu) ** 2) / (2.0 * sigma * sigma)
    z -= z.max()
    p = np.exp(z)
    return p / p.sum()


def fraction_to_p(f: float, block: int, sigma: float = 1.0) -> np.ndarray:
    """Configuration p over {1, 2, 4, ..., b} whose mean retain count is f * b.

    Member of the log-Gaussian family of Eq. 3 (fixed sigma), mu found by bisection on
    [-16, log2(b) + 16].  f >= 1 gives p_b = 1 (keep everything); f * b <= 1 gives p_1 = 1.
    """
    nK = int(block).bit_length()
    ks = 2.0 ** np.arange(nK)
    p = np.zeros(nK, dtype=np.float64)
    if f >= 1.0:
        p[-1] = 1.0
        return p
    if f * block <= 1.0:
        p[0] = 1.0
        return p
    lo, hi = -16.0, float(nK - 1) + 16.0
    target = f * block
    for _ in range(60):
        mid = 0.5 * (lo + hi)
        if float(_log_gaussian_row(mid, nK, sigma) @ ks) < target:
            lo = mid
        else:
            hi = mid
    p = _log_gaussian_row(0.5 * (lo + hi), nK, sigma)
    return p / p.sum()


def budget_table(wl: Workload) -> np.ndarray:
    """p[Hkv, nK] (float64, rows sum to 1) for a workload."""
    f = budget_fractions(wl)
    return np.stack([fraction_to_p(float(x), wl.block, wl.sigma) for x in f])
