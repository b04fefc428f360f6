"""CPU oracle for the online hot path of TCA-Attention (test infrastructure).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, fp64 NumPy restatement of what the
paper defines; it shares no code with the CUDA library, is never imported by the
product path, and exists so that the kernels have something independent to be compared
against.  Only the tests, the smoke check and the benchmark's CPU-baseline leg call it.

Inputs are the exact values the GPU sees (bf16 inputs are rounded to bf16 first and then
widened to fp64 by the caller).  Token indices are 0-based (the paper is 1-based).

Notation (Section 4 of the paper): L sequence length, d_h head dimension, b block size,
w local window, m number of blocks, K = {1, 2, 4, ..., b} per-block retain counts,
p the per-head configuration over K, s the token importance, h the block metric,
Psi the budget map, t the per-block requirement, S the selected index set.

Readings taken where the paper is silent or ambiguous (each is listed in the design
notes with its justification):
  * causal mask; the local subset is the w most recent tokens *of each query*;
  * candidates for the global subset are [0, m*b) with m = floor((L - w) / b); the rest,
    R = [m*b, L), is always kept (so global and local never overlap at the last query
    and a 100 % budget is exactly dense causal attention);
  * s is normalised over all L keys (Eq. 5 literally);
  * grouped-query attention: one selection per KV head from the mean of the group's
    per-query-head softmax distributions;
  * larger h => larger retain count: blocks ranked ascending by (h, block index) and
    Psi listed ascending (Eq. 7);
  * the run lengths of Psi are floor(m * p_k) plus a largest-remainder correction so
    that Psi has exactly m entries;
  * ties inside Top(t; B) go to the lower token index;
  * decoding: the block that leaves the window is the one compressed;
  * Algorithm 1: column means over the causally visible rows; the aggregated score is the
    share of the summed column means that the retained set (selected tokens and the always-kept
    tail, the S_total of Section 4.3) holds; no valid candidate => the last candidate.

Parity pins (tests/test_oracle_pins.py): dense causal attention by an independent
brute force at 100 % budget and at w >= L; masked attention against an independently
built boolean mask; closed forms of the concentration term; a hand-worked selection
example; the exact identity ||s - s~||_1 = 2*gamma behind Theorem 1; decode == last
prefill row; invariants of the selection.  "Parity unpinned" against the authors' own
implementation: GQA aggregation, the window/partition reading, the leftover rounding,
the decode block choice, and for Algorithm 1 the normalisation of the aggregated score and
the no-valid-candidate fall-back -- the paper fixes none of them; they are pinned only to
the readings above.  Algorithm 1's column means are pinned by the harmonic-number closed
form for uniform attention and by an independently masked dense matrix, its choice rule by a
hand-worked example.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

__all__ = [
    "retain_counts", "num_blocks", "log_importance", "block_metric", "resolve_counts",
    "budget_map", "mean_retain_floor", "rank_blocks", "block_requirement",
    "select_tokens", "retained_set", "select_head", "visible_mask_row",
    "attention_rows", "attention_over_set", "candidate_grid", "DecodeCache",
    "dropped_mass", "attention_column_means", "attention_column_means_at", "aggregated_score",
    "calibrate_head", "block_metric_entropy", "random_block_keys", "select_tokens_flat",
    "select_head_variant",
]


# ----------------------------------------------------------------------------- helpers
def _logsumexp(x: np.ndarray, axis=None) -> np.ndarray:
    mx = np.max(x, axis=axis, keepdims=True)
    out = mx + np.log(np.sum(np.exp(x - mx), axis=axis, keepdims=True))
    return np.squeeze(out, axis=axis) if axis is not None else float(out.reshape(()))


def retain_counts(b: int) -> np.ndarray:
    """The set K = {1, 2, 4, ..., b} (Section 4.1)."""
    if b < 1 or (b & (b - 1)):
        raise ValueError("block size must be a power of two")
    return 2 ** np.arange(int(b).bit_length(), dtype=np.int64)


def num_blocks(L: int, b: int, w: int) -> int:
    """m: number of candidate blocks; tokens [m*b, L) form the always-kept tail.

    Section 4.2 partitions the sequence into blocks of b and puts what does not divide
    into the local subset; with the no-overlap requirement of Section 4 the candidates
    are the tokens outside the last query's window.
    """
    return max(0, (L - w) // b)


# ----------------------------------------------------------------------------- step 1: Eq. 5
def log_importance(q_last: np.ndarray, K: np.ndarray, sm_scale: float) -> np.ndarray:
    """log s for one KV head.  q_last: [G, d] (the group's last-token queries), K: [L, d].

    Eq. 5: s = softmax(q_L K^T / sqrt(d_h)) over all L keys, for each query head of the
    group; the group's distributions are averaged (a probability vector again).  The
    logarithm is returned because s underflows for long sequences.
    """
    q_last = np.atleast_2d(np.asarray(q_last, dtype=np.float64))
    K = np.asarray(K, dtype=np.float64)
    x = (q_last @ K.T) * sm_scale                       # [G, L] logits
    logp = x - _logsumexp(x, axis=1)[:, None]           # per-query-head log-softmax
    return _logsumexp(logp, axis=0) - math.log(q_last.shape[0])


# ----------------------------------------------------------------------------- step 2-3: Eq. 6
def block_metric(log_s: np.ndarray, m: int, b: int, alpha: float) -> np.ndarray:
    """h_j of Eq. 6 for blocks j < m, from log s.

    h_j = (1 - alpha) * sum_i s_i + alpha * (1 - sum_i s_i^2 / (sum_i s_i)^2).
    The second term is invariant to a common scale of the block's scores, so it is
    evaluated on s_i / max_i s_i, which never divides zero by zero.
    """
    h = np.empty(m, dtype=np.float64)
    for j in range(m):
        l = np.asarray(log_s[j * b:(j + 1) * b], dtype=np.float64)
        top = float(np.max(l))
        e = np.exp(l - top)
        mass = math.exp(top) * float(np.sum(e))
        concentration = 1.0 - float(np.sum(e * e)) / float(np.sum(e)) ** 2
        h[j] = (1.0 - alpha) * mass + alpha * concentration
    return h


# ----------------------------------------------------------------------------- step 4: Eq. 7
def resolve_counts(p: Sequence[float], m: int) -> np.ndarray:
    """n_k: how many of the m blocks get retain count k, k in K ascending.

    Eq. 7 uses floor(m * p_k), which can leave Psi shorter than m; the shortfall D is
    given, one each, to the D entries with the largest fractional part of m * p_k
    (ties to the larger k).
    """
    p = np.asarray(p, dtype=np.float64)
    if abs(float(p.sum()) - 1.0) > 1e-9 or np.any(p < 0):
        raise ValueError("configuration must be a probability vector")
    f = m * p
    n = np.floor(f).astype(np.int64)
    short = int(m - n.sum())
    frac = f - n
    order = sorted(range(len(p)), key=lambda k: (-frac[k], -k))
    for k in order[:short]:
        n[k] += 1
    assert int(n.sum()) == m
    return n


def budget_map(n: Sequence[int], b: int) -> np.ndarray:
    """Psi of Eq. 7: n_1 ones, n_2 twos, ..., n_b copies of b, in ascending order."""
    ks = retain_counts(b)
    return np.repeat(ks, np.asarray(n, dtype=np.int64))


def mean_retain_floor(p: Sequence[float], b: int) -> int:
    """t = floor(sum_k k * p_k): tokens kept from a block completed while decoding."""
    total = 0.0
    for k, pk in zip(retain_counts(b), np.asarray(p, dtype=np.float64)):
        total += float(k) * float(pk)            # ascending k; k * p_k is exact (k = 2^i)
    return int(math.floor(total))


def rank_blocks(h: np.ndarray) -> np.ndarray:
    """rank_j = position of block j when blocks are sorted ascending by (h_j, j)."""
    order = np.lexsort((np.arange(len(h)), np.asarray(h, dtype=np.float64)))
    rank = np.empty(len(h), dtype=np.int64)
    rank[order] = np.arange(len(h))
    return rank


def block_requirement(h: np.ndarray, n: Sequence[int], b: int) -> np.ndarray:
    """t_j = Psi[rank_j] (Eq. 7): the densest blocks get the largest retain counts."""
    psi = budget_map(n, b)
    return psi[rank_blocks(h)]


# ----------------------------------------------------------------------------- step 5: Eq. 8
def select_tokens(log_s: np.ndarray, t: Sequence[int], b: int) -> np.ndarray:
    """S = union_j Top(t_j; B_j) by s (Eq. 8), ascending.  Ties: lower index wins."""
    keep: List[int] = []
    for j, tj in enumerate(t):
        blk = np.asarray(log_s[j * b:(j + 1) * b], dtype=np.float64)
        order = np.argsort(-blk, kind="stable")         # stable => lower index first on ties
        keep.extend(int(j * b + i) for i in order[:int(tj)])
    return np.array(sorted(keep), dtype=np.int64)


def retained_set(S: np.ndarray, m: int, b: int, L: int) -> np.ndarray:
    """T = S union [m*b, L): everything the cache keeps after prefilling."""
    return np.concatenate([np.asarray(S, dtype=np.int64), np.arange(m * b, L, dtype=np.int64)])


def select_head(q_last, K, p, b: int, w: int, alpha: float, sm_scale: float):
    """Steps 1-6 of Algorithm 2 for one KV head.  Returns a dict of every intermediate."""
    L = K.shape[0]
    m = num_blocks(L, b, w)
    log_s = log_importance(q_last, K, sm_scale)
    h = block_metric(log_s, m, b, alpha)
    n = resolve_counts(p, m)
    t = block_requirement(h, n, b)
    S = select_tokens(log_s, t, b)
    return {"log_s": log_s, "m": m, "h": h, "n": n, "t": t, "S": S,
            "T": retained_set(S, m, b, L)}


# ----------------------------------------------------------------------------- step 7: Eq. 2
def visible_mask_row(i: int, T: np.ndarray, w: int, L: int) -> np.ndarray:
    """Boolean [L]: keys query i attends to = {j <= i : j in T or i - j < w}."""
    vis = np.zeros(L, dtype=bool)
    vis[np.asarray(T, dtype=np.int64)] = True
    lo = max(0, i - w + 1)
    vis[lo:i + 1] = True
    vis[i + 1:] = False
    return vis


def attention_over_set(q: np.ndarray, Ksel: np.ndarray, Vsel: np.ndarray, sm_scale: float) -> np.ndarray:
    """softmax(q Ksel^T * scale) Vsel for one query vector (Eq. 2 for one row)."""
    x = (np.asarray(Ksel, dtype=np.float64) @ np.asarray(q, dtype=np.float64)) * sm_scale
    x -= x.max()
    e = np.exp(x)
    return (e / e.sum()) @ np.asarray(Vsel, dtype=np.float64)


def attention_rows(Q: np.ndarray, K: np.ndarray, V: np.ndarray, T: np.ndarray, w: int,
                   sm_scale: float, rows: Optional[Sequence[int]] = None) -> np.ndarray:
    """Sparse causal attention (Eq. 2) for one query head: rows of Q -> [len(rows), d].

    Query i attends to [K^G; K^L] = keys {j <= i : j in T} plus its own last w keys,
    taken as a set.
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    L = K.shape[0]
    rows = range(Q.shape[0]) if rows is None else rows
    out = np.empty((len(rows), V.shape[1]), dtype=np.float64)
    for r, i in enumerate(rows):
        vis = visible_mask_row(int(i), T, w, L)
        out[r] = attention_over_set(Q[int(i)], K[vis], V[vis], sm_scale)
    return out


def dropped_mass(q: np.ndarray, K: np.ndarray, i: int, T: np.ndarray, w: int, sm_scale: float) -> float:
    """gamma_i of Theorem 1: dense-softmax mass of the causally visible keys not kept."""
    L = K.shape[0]
    x = (np.asarray(K[:i + 1], dtype=np.float64) @ np.asarray(q, dtype=np.float64)) * sm_scale
    x -= x.max()
    e = np.exp(x)
    vis = visible_mask_row(i, T, w, L)[:i + 1]
    return float(e[~vis].sum() / e.sum())


# ----------------------------------------------------------------------------- Eq. 3
def candidate_grid(b: int, M: int = 14, sigma: float = 1.0) -> np.ndarray:
    """The M log-Gaussian candidate configurations of Eq. 3, [M, |K|].

    mu^i = log2(1 + (i - 1)(b - 1)/(M - 1)), i = 1..M;  p_k ~ exp(-(log2 k - mu)^2 / 2 sigma^2).
    """
    x = np.log2(retain_counts(b).astype(np.float64))
    rows = []
    for i in range(1, M + 1):
        mu = math.log2(1.0 + (i - 1) * (b - 1) / (M - 1))
        phi = np.exp(-((x - mu) ** 2) / (2.0 * sigma * sigma))
        rows.append(phi / phi.sum())
    return np.stack(rows)


# ----------------------------------------------------------------------------- Algorithm 1 (offline)
def attention_column_means(Q: np.ndarray, K: np.ndarray, sm_scale: float) -> np.ndarray:
    """Inner term of Eq. 4: c[k] = mean over the non-zero entries of column k of A.

    A = softmax(Q K^T sm_scale) with the causal mask (reading R1), so the non-zero entries of
    column k are the rows j >= k and there are L - k of them.  Q is [G, L, d] (the query heads
    that share the KV head; G = 1 for plain multi-head attention); the result is the mean of
    the G heads' columns, the same aggregation as for the importance of Eq. 5.  Returns [L].
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    if Q.ndim == 2:
        Q = Q[None]
    G, L, _ = Q.shape
    col = np.zeros(L, dtype=np.float64)
    for g in range(G):
        for j in range(L):
            x = (K[:j + 1] @ Q[g, j]) * sm_scale
            x -= x.max()
            e = np.exp(x)
            col[:j + 1] += e / e.sum()
    return col / (G * (L - np.arange(L, dtype=np.float64)))


def attention_column_means_at(Q: np.ndarray, K: np.ndarray, sm_scale: float, cols: Sequence[int],
                              rows_per_step: int = 512) -> np.ndarray:
    """attention_column_means for the chosen columns only, for sequences too long to afford all.

    The same definition: c[k] = (1 / (L - k)) * sum_{j >= k} A[j, k], averaged over the G query
    heads, with A[j, :] the softmax of row j over its visible keys 0..j.  Rows are taken
    `rows_per_step` at a time only so that the logits of a step fit in memory (one matrix product
    per step instead of one product per row); every row's softmax is still normalised over all of
    its visible keys.  Returns [len(cols)].
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    if Q.ndim == 2:
        Q = Q[None]
    G, L, _ = Q.shape
    cols = np.asarray(cols, dtype=np.int64)
    total = np.zeros(len(cols), dtype=np.float64)
    for g in range(G):
        for j0 in range(0, L, rows_per_step):
            j1 = min(L, j0 + rows_per_step)
            x = (Q[g, j0:j1] @ K[:j1].T) * sm_scale                  # rows j0..j1-1, keys 0..j1-1
            key = np.arange(j1)[None, :]
            row = np.arange(j0, j1)[:, None]
            x = np.where(key <= row, x, -np.inf)                      # causal: row j sees keys <= j
            lse = _logsumexp(x, axis=1)
            seen = cols < j1
            a = np.exp(x[:, cols[seen]] - lse[:, None])               # masked entries are exactly 0
            total[seen] += a.sum(axis=0)
    return total / (G * (L - cols.astype(np.float64)))


def aggregated_score(S: np.ndarray, c: np.ndarray, n_candidates: int) -> float:
    """a_i of Eq. 4 for the selected set S: the share of the aggregated score that is retained.

    Eq. 4 is the sum of c over the selected tokens.  Algorithm 1 compares it with a threshold
    tau in [0, 1] that the text calls a share "of the aggregated attention mass", and Section 4.3
    argues from "retained mass >= tau" to "dropped mass <= 1 - tau" with the retained set being
    the global subset AND the local subset.  So the sum runs over everything the method keeps,
    T = S union [n_candidates, L) (the always-kept tail is the local subset of the newest
    query), and is divided by the sum over all L tokens: keeping everything scores exactly 1,
    and 1 - a_i is the share of the score that is dropped.
    """
    c = np.asarray(c, dtype=np.float64)
    total = float(np.sum(c))
    kept = float(np.sum(c[np.asarray(S, dtype=np.int64)])) + float(np.sum(c[n_candidates:]))
    return kept / total if total > 0.0 else 1.0


def calibrate_head(Q: np.ndarray, K: np.ndarray, candidates: np.ndarray, b: int, w: int, alpha: float,
                   tau: float, sm_scale: float):
    """Algorithm 1 for one KV head: the sparsest candidate that keeps a share tau of the score.

    For every candidate p^i the online selection (Eq. 5-8 with the newest query, exactly as at
    inference) gives S_i; a_i follows Eq. 4; among the candidates with a_i >= tau the one with the
    fewest selected tokens wins (the lowest index on a tie).  If no candidate reaches tau the last
    one (the most accurate end of the sweep) is returned.  Returns (choice, a [M], sizes [M]).
    """
    Q = np.asarray(Q, dtype=np.float64)
    if Q.ndim == 2:
        Q = Q[None]
    L = K.shape[0]
    m = num_blocks(L, b, w)
    c = attention_column_means(Q, K, sm_scale)
    log_s = log_importance(Q[:, L - 1], K, sm_scale)
    h = block_metric(log_s, m, b, alpha)
    M = len(candidates)
    a = np.zeros(M, dtype=np.float64)
    sizes = np.zeros(M, dtype=np.int64)
    for i in range(M):
        t = block_requirement(h, resolve_counts(candidates[i], m), b)
        S = select_tokens(log_s, t, b)
        a[i] = aggregated_score(S, c, m * b)
        sizes[i] = len(S)
    valid = np.nonzero(a >= tau)[0]
    if len(valid) == 0:
        return M - 1, a, sizes
    choice = int(valid[np.argmin(sizes[valid])])      # argmin returns the first minimum: lowest index
    return choice, a, sizes


# ----------------------------------------------------------------------------- steps 8-9: decoding
@dataclass
class DecodeCache:
    """Retained cache of one KV head while decoding (Section 4.2, last paragraph).

    ``glob`` holds positions of the global subset, ``tail`` the always-kept recent
    tokens.  After a token is appended, when the tail holds w + b tokens its oldest b
    form a new block: they are scored with the current query (Eq. 5 restricted to the
    block: each query head's softmax is taken over the block's b keys and the group's
    distributions are averaged; with one query head the normaliser cannot change the
    order), the top t = floor(sum_k k p_k) are moved to the global subset and the rest
    dropped.
    """
    b: int
    w: int
    t_keep: int
    sm_scale: float
    glob: List[int] = field(default_factory=list)
    tail: List[int] = field(default_factory=list)

    @classmethod
    def from_prefill(cls, S: np.ndarray, m: int, L: int, b: int, w: int, p, sm_scale: float) -> "DecodeCache":
        return cls(b=b, w=w, t_keep=mean_retain_floor(p, b), sm_scale=sm_scale,
                   glob=[int(x) for x in S], tail=list(range(m * b, L)))

    def positions(self) -> np.ndarray:
        return np.array(self.glob + self.tail, dtype=np.int64)

    def append(self, pos: int, q_cur: np.ndarray, K_all: np.ndarray) -> Optional[np.ndarray]:
        """Append token ``pos``; compress if a block completed.  q_cur: [G, d] queries of
        the current token, K_all: keys indexable by position.  Returns the kept positions
        of the compressed block, or None."""
        self.tail.append(int(pos))
        if len(self.tail) < self.w + self.b:
            return None
        blk = self.tail[:self.b]
        self.tail = self.tail[self.b:]
        q_cur = np.atleast_2d(np.asarray(q_cur, dtype=np.float64))
        x = (q_cur @ np.asarray(K_all[blk], dtype=np.float64).T) * self.sm_scale   # [G, b]
        # group mean of softmax restricted to the block, in the log domain
        logp = x - _logsumexp(x, axis=1)[:, None]
        score = _logsumexp(logp, axis=0)
        order = np.argsort(-score, kind="stable")[:self.t_keep]
        kept = sorted(blk[i] for i in order)
        self.glob.extend(kept)
        return np.array(kept, dtype=np.int64)

    def attend(self, q: np.ndarray, K_all: np.ndarray, V_all: np.ndarray) -> np.ndarray:
        """One decode step for one query head: attention over the whole retained cache."""
        pos = self.positions()
        return attention_over_set(q, K_all[pos], V_all[pos], self.sm_scale)


# ----------------------------------------------------------------------------- ablation variants
# The appendix ("Effectiveness of Local-context Redundancy Metric", "Ablations on Concentration
# Index") compares the method with two variants it does not spell out: a block-wise entropy in
# place of the Herfindahl-Hirschman term of Eq. 6, and blocks "randomly sorted" instead of sorted
# by h.  A third variant, one flat top-B over all candidates of a head, is what "a per-head
# budgeted top-k" means when read without the block structure.  Readings (parity unpinned against
# the authors' code, which the paper does not show): entropy = Shannon entropy (natural log) of the
# block's scores normalised inside the block, unscaled; random order = blocks ranked by a seeded
# 64-bit hash of (seed, head unit, block index); flat = the B best candidates, ties to the lower
# index, with B the size of the global subset the configuration gives.
def block_metric_entropy(log_s: np.ndarray, m: int, b: int, alpha: float) -> np.ndarray:
    """Eq. 6 with the block entropy as concentration index:
    h_j = (1 - alpha) * sum_i s_i + alpha * H_j,  H_j = -sum_i p_i ln p_i,  p_i = s_i / sum_{B_j} s."""
    h = np.empty(m, dtype=np.float64)
    for j in range(m):
        l = np.asarray(log_s[j * b:(j + 1) * b], dtype=np.float64)
        top = float(np.max(l))
        e = np.exp(l - top)
        mass = math.exp(top) * float(np.sum(e))
        pr = e / np.sum(e)
        nz = pr > 0.0                                    # 0 * ln 0 = 0
        entropy = -float(np.sum(pr[nz] * np.log(pr[nz])))
        h[j] = (1.0 - alpha) * mass + alpha * entropy
    return h


def _splitmix64(x: int) -> int:
    """The SplitMix64 finaliser (Steele, Lea, Flood 2014), a published 64-bit mixing function."""
    mask = (1 << 64) - 1
    x = (x + 0x9E3779B97F4A7C15) & mask
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & mask
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & mask
    return x ^ (x >> 31)


def random_block_keys(seed: int, unit: int, m: int) -> np.ndarray:
    """Sort keys of the random-order variant: for block j of head unit `unit`,
    key = SplitMix64(SplitMix64(seed * 2^32 + unit) + j) >> 11, scaled to [0, 1).  Blocks are
    then ranked ascending by (key, j) exactly as they are by (h, j) in the method proper."""
    base = _splitmix64(((int(seed) & 0xFFFFFFFF) << 32) | (int(unit) & 0xFFFFFFFF))
    mask = (1 << 64) - 1
    return np.array([(_splitmix64((base + j) & mask) >> 11) * 2.0 ** -53 for j in range(m)], dtype=np.float64)


def select_tokens_flat(log_s: np.ndarray, n_keep: int, n_candidates: int) -> np.ndarray:
    """The n_keep highest-scoring tokens among the candidates [0, n_candidates), ties to the lower
    index, ascending: the whole candidate range treated as one block of Eq. 8."""
    cand = np.asarray(log_s[:n_candidates], dtype=np.float64)
    order = np.argsort(-cand, kind="stable")[:int(n_keep)]
    return np.sort(order).astype(np.int64)


def select_head_variant(q_last, K, p, b: int, w: int, alpha: float, sm_scale: float, variant: str,
                        seed: int = 0, unit: int = 0):
    """select_head for one of the variants: "entropy", "random" or "flat"."""
    L = K.shape[0]
    m = num_blocks(L, b, w)
    log_s = log_importance(q_last, K, sm_scale)
    n = resolve_counts(p, m)
    if variant == "flat":
        n_keep = int(np.sum(retain_counts(b) * n))
        S = select_tokens_flat(log_s, n_keep, m * b)
        return {"log_s": log_s, "m": m, "n": n, "S": S, "T": retained_set(S, m, b, L)}
    if variant == "entropy":
        h = block_metric_entropy(log_s, m, b, alpha)
    elif variant == "random":
        h = random_block_keys(seed, unit, m)
    else:
        raise ValueError(f"unknown variant {variant!r}")
    t = block_requirement(h, n, b)
    S = select_tokens(log_s, t, b)
    return {"log_s": log_s, "m": m, "h": h, "n": n, "t": t, "S": S, "T": retained_set(S, m, b, L)}
