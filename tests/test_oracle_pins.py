"""Pins for the CPU oracle: values and identities fixed by the paper and by mathematics.

None of these tests touches the CUDA path.  Each one is chosen so that a plausible
mistake in the oracle (dropped term, wrong sign, wrong index, transposed operand, wrong
sort direction, off-by-one in the window) makes it fail.
"""
import itertools
import math

import numpy as np
import pytest
from scipy.special import softmax as sp_softmax

from oracle import tca_oracle as O


def _rng(seed):
    return np.random.default_rng(seed)


# ----------------------------------------------------------------------------- brute force used as pins
def dense_causal_attention(Q, K, V, scale):
    """Textbook causal softmax attention on the full L x L matrix (library softmax)."""
    L = K.shape[0]
    A = (Q @ K.T) * scale
    A = np.where(np.tril(np.ones((L, L), dtype=bool)), A, -np.inf)
    return sp_softmax(A, axis=1) @ V


def masked_attention_by_definition(Q, K, V, T, w, scale):
    """Attention with a boolean mask written out from the set definition, entry by entry."""
    L = K.shape[0]
    Tset = set(int(x) for x in T)
    mask = np.zeros((L, L), dtype=bool)
    for i in range(L):
        for j in range(L):
            mask[i, j] = (j <= i) and ((j in Tset) or (i - j < w))
    A = np.where(mask, (Q @ K.T) * scale, -np.inf)
    return sp_softmax(A, axis=1) @ V


# ----------------------------------------------------------------------------- Eq. 5: importance
def test_importance_is_a_distribution_and_matches_closed_form():
    rng = _rng(1)
    d, L = 16, 200
    u = rng.standard_normal(d)
    c = rng.standard_normal(L) * 3
    K = c[:, None] * u[None, :]                     # k_j = c_j u, q = u  =>  logit_j = c_j |u|^2 scale
    scale = 1 / math.sqrt(d)
    ls = O.log_importance(u[None, :], K, scale)
    assert abs(np.exp(ls).sum() - 1) < 1e-12
    want = sp_softmax(c * (u @ u) * scale)
    np.testing.assert_allclose(np.exp(ls), want, rtol=1e-11, atol=0)


def test_importance_uses_the_scale_and_is_shift_invariant():
    rng = _rng(2)
    d, L = 8, 64
    q = rng.standard_normal((1, d))
    K = rng.standard_normal((L, d))
    a = O.log_importance(q, K, 0.5)
    # adding the same vector to every key adds a constant to every logit
    b = O.log_importance(q, K + rng.standard_normal(d)[None, :], 0.5)
    np.testing.assert_allclose(a, b, atol=1e-12)
    # doubling the scale equals doubling the query
    np.testing.assert_allclose(O.log_importance(q, K, 1.0), O.log_importance(2 * q, K, 0.5), atol=1e-12)
    assert np.max(np.abs(O.log_importance(q, K, 1.0) - a)) > 1e-3


def test_importance_group_mean_is_mean_of_softmaxes():
    rng = _rng(3)
    G, d, L = 4, 8, 50
    q = rng.standard_normal((G, d))
    K = rng.standard_normal((L, d))
    want = np.mean([sp_softmax((K @ q[g]) * 0.3) for g in range(G)], axis=0)
    np.testing.assert_allclose(np.exp(O.log_importance(q, K, 0.3)), want, rtol=1e-12)


def test_importance_survives_underflow():
    # logits far apart: probabilities underflow in fp64 but their logs must not
    K = np.array([[0.0], [-2000.0], [-4000.0]])
    ls = O.log_importance(np.array([[1.0]]), K, 1.0)
    np.testing.assert_allclose(ls, [0.0, -2000.0, -4000.0], atol=1e-9)


# ----------------------------------------------------------------------------- Eq. 6: block metric
@pytest.mark.parametrize("b", [4, 32, 128])
def test_block_metric_closed_forms(b):
    alpha = 0.3
    # uniform block: mass b*c, concentration 1 - 1/b
    c = 1e-3
    h = O.block_metric(np.log(np.full(b, c)), 1, b, alpha)[0]
    assert h == pytest.approx((1 - alpha) * b * c + alpha * (1 - 1 / b), rel=1e-13)
    # all mass on one token: concentration 0 (other tokens underflow to nothing)
    ls = np.full(b, -5000.0)
    ls[b // 2] = math.log(0.25)
    h = O.block_metric(ls, 1, b, alpha)[0]
    assert h == pytest.approx((1 - alpha) * 0.25, rel=1e-13)
    # two equal tokens: concentration 1/2
    ls = np.full(b, -5000.0)
    ls[0] = ls[-1] = math.log(0.1)
    h = O.block_metric(ls, 1, b, alpha)[0]
    assert h == pytest.approx((1 - alpha) * 0.2 + alpha * 0.5, rel=1e-13)


def test_block_metric_weights_and_scale_invariance():
    rng = _rng(4)
    b, m = 8, 3
    ls = np.log(rng.random(m * b) * 0.01)
    h0 = O.block_metric(ls, m, b, 0.0)              # alpha = 0: mass only
    np.testing.assert_allclose(h0, np.exp(ls).reshape(m, b).sum(1), rtol=1e-13)
    h1 = O.block_metric(ls, m, b, 1.0)              # alpha = 1: concentration only
    h1s = O.block_metric(ls - 7.0, m, b, 1.0)       # common scale leaves it unchanged
    np.testing.assert_allclose(h1, h1s, rtol=1e-12)
    assert np.all(h1 > 0) and np.all(h1 < 1 - 1 / b + 1e-12)
    # an empty-looking block (everything underflows) is still finite
    assert np.isfinite(O.block_metric(np.full(b, -1e5), 1, b, 0.5)[0])


# ----------------------------------------------------------------------------- Eq. 7: budget map
def test_resolve_counts_hand_case_and_invariants():
    np.testing.assert_array_equal(O.resolve_counts([0.5, 0.3, 0.2], 5), [2, 2, 1])
    np.testing.assert_array_equal(O.budget_map([2, 2, 1], 4), [1, 1, 2, 2, 4])
    assert O.mean_retain_floor([0.5, 0.3, 0.2], 4) == 1          # floor(1.9)
    rng = _rng(5)
    for _ in range(200):
        nK = int(rng.integers(1, 9))
        p = rng.dirichlet(np.ones(nK))
        m = int(rng.integers(0, 2000))
        n = O.resolve_counts(p, m)
        assert n.sum() == m and np.all(n >= 0)
        assert np.all(np.abs(n - m * p) < 1.0)
        assert np.all(n >= np.floor(m * p))
    # exact products need no correction
    np.testing.assert_array_equal(O.resolve_counts([0.25, 0.75], 8), [2, 6])
    with pytest.raises(ValueError):
        O.resolve_counts([0.5, 0.4], 10)


def test_budget_map_is_ascending_and_one_per_block():
    psi = O.budget_map([3, 0, 2, 1], 8)
    np.testing.assert_array_equal(psi, [1, 1, 1, 4, 4, 8])


def test_rank_is_ascending_with_index_tiebreak():
    h = np.array([0.3, 0.1, 0.3, 0.2, 0.1])
    np.testing.assert_array_equal(O.rank_blocks(h), [3, 0, 4, 2, 1])
    # densest block gets the largest count
    t = O.block_requirement(np.array([0.9, 0.1, 0.5]), [1, 1, 1], 4)
    np.testing.assert_array_equal(t, [4, 1, 2])


# ----------------------------------------------------------------------------- hand-worked example
def test_hand_worked_selection(golden):
    g = golden("hand_selection.txt")
    b, w, L, alpha = int(g["block"][0]), int(g["window"][0]), int(g["length"][0]), g["alpha"][0]
    s = np.array(g["s"])
    assert len(s) == L and abs(s.sum() - 1) < 1e-12
    m = O.num_blocks(L, b, w)
    assert m == int(g["m"][0])
    ls = np.log(s)
    np.testing.assert_allclose(O.block_metric(ls, m, b, 0.0), g["mass"], rtol=1e-12)
    np.testing.assert_allclose(O.block_metric(ls, m, b, 1.0), g["concentration"], rtol=1e-12)
    h = O.block_metric(ls, m, b, alpha)
    np.testing.assert_allclose(h, g["h"], rtol=1e-12)
    n = O.resolve_counts(g["p"], m)
    np.testing.assert_array_equal(n, np.array(g["n"], dtype=int))
    np.testing.assert_array_equal(O.budget_map(n, b), np.array(g["psi"], dtype=int))
    np.testing.assert_array_equal(O.rank_blocks(h), np.array(g["rank"], dtype=int))
    t = O.block_requirement(h, n, b)
    np.testing.assert_array_equal(t, np.array(g["t"], dtype=int))
    S = O.select_tokens(ls, t, b)
    np.testing.assert_array_equal(S, np.array(g["S"], dtype=int))
    np.testing.assert_array_equal(O.retained_set(S, m, b, L), np.array(g["T"], dtype=int))
    assert O.mean_retain_floor(g["p"], b) == int(g["t_decode"][0])


# ----------------------------------------------------------------------------- Eq. 8: top-t
def test_top_t_is_the_best_subset_by_brute_force():
    rng = _rng(6)
    b = 8
    for _ in range(30):
        ls = rng.standard_normal(b)
        for t in (1, 2, 4, 8):
            S = O.select_tokens(ls, [t], b)
            best = max(itertools.combinations(range(b), t), key=lambda c: sum(ls[list(c)]))
            assert sorted(best) == list(S)


def test_top_t_ties_go_to_lower_index_and_output_sorted():
    ls = np.log(np.array([.1, .3, .3, .1, .3, .1, .1, .1]))
    np.testing.assert_array_equal(O.select_tokens(ls, [2], 8), [1, 2])
    np.testing.assert_array_equal(O.select_tokens(ls, [4], 8), [0, 1, 2, 4])
    # second block is offset by b
    two = np.concatenate([ls, ls])
    np.testing.assert_array_equal(O.select_tokens(two, [1, 2], 8), [1, 9, 10])


def test_selection_invariants_on_random_heads():
    rng = _rng(7)
    b, w, L, d, G = 16, 40, 40 + 16 * 9 + 5, 8, 2
    for trial in range(5):
        K = rng.standard_normal((L, d))
        q = rng.standard_normal((G, d))
        p = rng.dirichlet(np.ones(5))
        r = O.select_head(q, K, p, b, w, 0.5, 0.35)
        m, S, t, h, n = r["m"], r["S"], r["t"], r["h"], r["n"]
        assert m == 9
        ks = O.retain_counts(b)
        assert len(S) == int((ks * n).sum())
        assert np.all(np.diff(S) > 0) and S.max() < m * b
        np.testing.assert_array_equal(np.bincount(S // b, minlength=m), t)
        np.testing.assert_array_equal(np.sort(t), O.budget_map(n, b))
        for a in range(m):
            for c in range(m):
                if h[a] < h[c]:
                    assert t[a] <= t[c]
        for j in range(m):
            blk = r["log_s"][j * b:(j + 1) * b]
            kept = np.zeros(b, bool)
            kept[S[(S // b) == j] - j * b] = True
            if kept.any() and (~kept).any():
                assert blk[kept].min() >= blk[~kept].max()
        # tail [m*b, L) always kept, once
        T = r["T"]
        assert len(set(T.tolist())) == len(T)
        np.testing.assert_array_equal(T[len(S):], np.arange(m * b, L))


# ----------------------------------------------------------------------------- Eq. 2: attention
def _toy(seed, L=96, d=8):
    rng = _rng(seed)
    return (rng.standard_normal((L, d)), rng.standard_normal((L, d)) * 1.5,
            rng.standard_normal((L, d)))


def test_full_budget_is_dense_causal_attention():
    Q, K, V = _toy(8)
    L, d = K.shape
    b, w, scale = 8, 24, 1 / math.sqrt(d)
    nK = int(b).bit_length()
    p = np.zeros(nK)
    p[-1] = 1.0                                       # every block keeps all b tokens
    r = O.select_head(Q[-1:], K, p, b, w, 0.5, scale)
    np.testing.assert_array_equal(r["T"], np.arange(L))
    got = O.attention_rows(Q, K, V, r["T"], w, scale)
    np.testing.assert_allclose(got, dense_causal_attention(Q, K, V, scale), rtol=1e-11, atol=1e-13)


def test_window_covering_everything_is_dense_causal_attention():
    Q, K, V = _toy(9, L=50)
    scale = 0.4
    p = np.array([1.0, 0, 0, 0])                       # would keep 1 per block, but there are no blocks
    r = O.select_head(Q[-1:], K, p, 8, 64, 0.5, scale)
    assert r["m"] == 0 and len(r["S"]) == 0
    got = O.attention_rows(Q, K, V, r["T"], 64, scale)
    np.testing.assert_allclose(got, dense_causal_attention(Q, K, V, scale), rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("w", [1, 5, 16])
def test_sparse_attention_matches_mask_written_from_the_definition(w):
    Q, K, V = _toy(10, L=70)
    scale = 0.37
    b = 4
    p = np.array([0.6, 0.3, 0.1])
    r = O.select_head(Q[-1:], K, p, b, w, 0.5, scale)
    got = O.attention_rows(Q, K, V, r["T"], w, scale)
    want = masked_attention_by_definition(Q, K, V, r["T"], w, scale)
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-13)
    # it really is sparse: differs from dense attention somewhere
    assert np.max(np.abs(got - dense_causal_attention(Q, K, V, scale))) > 1e-4


def test_error_identity_and_bound_of_theorem_1():
    Q, K, V = _toy(11, L=80)
    scale, b, w = 0.5, 8, 16
    p = np.array([0.5, 0.3, 0.2, 0.0])
    r = O.select_head(Q[-1:], K, p, b, w, 0.5, scale)
    dense = dense_causal_attention(Q, K, V, scale)
    sparse = O.attention_rows(Q, K, V, r["T"], w, scale)
    L = K.shape[0]
    saw_drop = False
    for i in range(L):
        gamma = O.dropped_mass(Q[i], K, i, r["T"], w, scale)
        vis = O.visible_mask_row(i, r["T"], w, L)
        x = (K[:i + 1] @ Q[i]) * scale
        s_full = sp_softmax(x)
        s_kept = np.zeros(i + 1)
        s_kept[vis[:i + 1]] = sp_softmax(x[vis[:i + 1]])
        # exact identity behind the theorem: total variation is twice the dropped mass
        assert abs(np.abs(s_full - s_kept).sum() - 2 * gamma) < 1e-12
        err = dense[i] - sparse[i]
        assert np.max(np.abs(err)) <= 2 * gamma * np.max(np.abs(V)) + 1e-12
        assert np.sum(np.abs(err)) <= 2 * gamma * np.max(np.abs(V).sum(1)) + 1e-12
        saw_drop |= gamma > 1e-6
    assert saw_drop


# ----------------------------------------------------------------------------- decoding
def test_decode_over_retained_cache_equals_last_prefill_row():
    Q, K, V = _toy(12, L=90)
    scale, b, w = 0.45, 8, 20
    p = np.array([0.4, 0.3, 0.2, 0.1])
    r = O.select_head(Q[-1:], K, p, b, w, 0.5, scale)
    L = K.shape[0]
    cache = O.DecodeCache.from_prefill(r["S"], r["m"], L, b, w, p, scale)
    np.testing.assert_array_equal(cache.positions(), r["T"])
    last = O.attention_rows(Q, K, V, r["T"], w, scale, rows=[L - 1])[0]
    np.testing.assert_allclose(cache.attend(Q[L - 1], K, V), last, rtol=1e-12, atol=1e-14)


def test_decode_append_keeps_partition_and_compresses_the_block_leaving_the_window():
    rng = _rng(13)
    b, w, d = 8, 16, 8
    L0, steps = 16 + 8 * 3, 30
    K = rng.standard_normal((L0 + steps, d))
    Qd = rng.standard_normal((L0 + steps, d))
    p = np.array([0.1, 0.2, 0.3, 0.4])                # mean retain = .1+.4+1.2+3.2 = 4.9 -> 4
    r = O.select_head(Qd[L0 - 1:L0], K[:L0], p, b, w, 0.5, 0.4)
    cache = O.DecodeCache.from_prefill(r["S"], r["m"], L0, b, w, p, 0.4)
    assert cache.t_keep == 4
    n_glob = len(cache.glob)
    for s in range(steps):
        pos = L0 + s
        kept = cache.append(pos, Qd[pos:pos + 1], K)
        m_now = O.num_blocks(pos + 1, b, w)
        # same partition as a prefill of length pos+1 would use
        assert cache.tail == list(range(m_now * b, pos + 1))
        assert w <= len(cache.tail) < w + b
        if kept is not None:
            blk = np.arange((m_now - 1) * b, m_now * b)
            assert len(kept) == 4 and set(kept) <= set(blk)
            logits = K[blk] @ Qd[pos]
            want = sorted(blk[np.argsort(-logits, kind="stable")[:4]])   # single head: order of raw logits
            assert list(kept) == want
            n_glob += 4
        assert len(cache.glob) == n_glob
    assert n_glob == len(r["S"]) + 4 * ((L0 + steps - w) // b - r["m"])


def test_decode_block_score_is_group_mean_of_block_softmaxes():
    rng = _rng(14)
    b, w, d, G = 4, 4, 6, 3
    K = rng.standard_normal((8, d)) * 2
    q = rng.standard_normal((G, d)) * 2
    cache = O.DecodeCache(b=b, w=w, t_keep=2, sm_scale=0.5, glob=[], tail=list(range(7)))
    kept = cache.append(7, q, K)
    score = np.mean([sp_softmax((K[:4] @ q[g]) * 0.5) for g in range(G)], axis=0)
    want = sorted(np.argsort(-score, kind="stable")[:2])
    assert list(kept) == want


# ----------------------------------------------------------------------------- Eq. 3: candidates
def test_candidate_grid_closed_forms(golden):
    g = golden("candidate_grid.txt")
    b, M = int(g["block"][0]), int(g["M"][0])
    C = O.candidate_grid(b, M, sigma=1.0)
    assert C.shape == (M, 8)
    np.testing.assert_allclose(C.sum(1), 1.0, rtol=1e-13)
    # mu^1 = 0: p_2/p_1 = exp(-1/2); mu^M = log2 b: p_{b/2}/p_b = exp(-1/2)
    assert g["mu_first"][0] == 0.0 and g["mu_last"][0] == 7.0
    assert C[0, 1] / C[0, 0] == pytest.approx(math.exp(-0.5), rel=1e-12)
    assert C[-1, -2] / C[-1, -1] == pytest.approx(math.exp(-0.5), rel=1e-12)
    # mu^2 = log2(140/13): log-ratio of neighbours is linear in mu
    mu2 = math.log2(g["mu_second_arg"][0])
    assert math.log(C[1, 4] / C[1, 3]) == pytest.approx(-((4 - mu2) ** 2 - (3 - mu2) ** 2) / 2, rel=1e-11)
    # budgets grow monotonically from efficiency- to accuracy-oriented
    mean_keep = C @ O.retain_counts(b)
    assert np.all(np.diff(mean_keep) > 0)
    # mean tokens kept per 128-token block for the 14 candidates, to the two decimals stored
    assert len(g["mean_retention"]) == M
    np.testing.assert_allclose(mean_keep, g["mean_retention"], atol=0.0051, rtol=0)   # half a unit of the last digit


# ----------------------------------------------------------------------------- Algorithm 1 / Eq. 4
def test_column_means_closed_form_for_uniform_attention():
    """q = 0 makes every causal row uniform, A[j, k] = 1/(j+1), so the mean of column k over its
    L - k non-zero rows is (H_L - H_k)/(L - k) with H the harmonic numbers."""
    L, d = 37, 5
    K = _rng(21).standard_normal((L, d))
    c = O.attention_column_means(np.zeros((2, L, d)), K, 0.3)
    H = np.concatenate([[0.0], np.cumsum(1.0 / np.arange(1, L + 1))])
    np.testing.assert_allclose(c, (H[L] - H[:L]) / (L - np.arange(L)), rtol=1e-13)


def test_column_means_against_a_masked_dense_matrix():
    """Independent formulation: the full L x L matrix with a -inf upper triangle, SciPy's softmax
    over rows, a column sum divided by the count of non-zero entries of that column."""
    rng = _rng(22)
    L, d, G = 29, 7, 3
    Q, K = rng.standard_normal((G, L, d)) * 1.5, rng.standard_normal((L, d)) * 1.5
    want = np.zeros(L)
    for g in range(G):
        X = (Q[g] @ K.T) * 0.4
        X[np.triu_indices(L, 1)] = -np.inf
        A = np.stack([sp_softmax(X[j]) for j in range(L)])
        nnz = (A > 0).sum(0)
        assert list(nnz) == list(L - np.arange(L))         # exactly the causally visible rows
        want += A.sum(0) / nnz
    np.testing.assert_allclose(O.attention_column_means(Q, K, 0.4), want / G, rtol=1e-12)
    # every row of A sums to 1: weighting the means back by their counts gives L
    c1 = O.attention_column_means(Q[:1], K, 0.4)
    assert float(np.sum(c1 * (L - np.arange(L)))) == pytest.approx(L, rel=1e-12)


def test_sampled_column_means_equal_the_full_evaluation():
    """The chunked, sampled-column form used at long sequence lengths is the same function: equal
    to the row-by-row evaluation on every column, for chunk sizes that do and do not divide L."""
    rng = _rng(24)
    L, d, G = 61, 6, 2
    Q, K = rng.standard_normal((G, L, d)) * 1.3, rng.standard_normal((L, d)) * 1.3
    full = O.attention_column_means(Q, K, 0.45)
    for step in (1, 7, 16, 61, 100):
        np.testing.assert_allclose(O.attention_column_means_at(Q, K, 0.45, np.arange(L), step), full, rtol=1e-12)
    cols = np.array([0, 5, 17, 59, 60])
    np.testing.assert_allclose(O.attention_column_means_at(Q, K, 0.45, cols, 8), full[cols], rtol=1e-12)


def test_aggregated_score_is_the_retained_share_of_all_column_means():
    """4 candidates and 2 always-kept tail tokens, values chosen so that the plain sum of Eq. 4
    (0.625), a share of the candidates only (0.625 / 1.125), a share of everything without the
    tail in the numerator (0.625 / 4.125) and the retained share (3.625 / 4.125) all differ."""
    c = np.array([0.5, 0.25, 0.125, 0.25, 2.0, 1.0])
    assert O.aggregated_score(np.array([0, 2]), c, 4) == pytest.approx(3.625 / 4.125, rel=1e-15)
    assert O.aggregated_score(np.arange(4), c, 4) == pytest.approx(1.0, rel=1e-15)
    assert O.aggregated_score(np.array([], dtype=np.int64), c, 4) == pytest.approx(3.0 / 4.125, rel=1e-15)
    # no tail at all: the share of the candidates
    assert O.aggregated_score(np.array([1]), c[:4], 4) == pytest.approx(0.25 / 1.125, rel=1e-15)


def test_aggregated_score_is_one_minus_the_dropped_share():
    """Section 4.3 reads the threshold as a bound on what is dropped: a_i = 1 - (column means of
    the tokens that are neither selected nor in the tail) / (all column means)."""
    rng = _rng(23)
    c = rng.random(40)
    S = np.array([0, 3, 4, 17, 22])
    dropped = np.setdiff1d(np.arange(32), S)
    assert O.aggregated_score(S, c, 32) == pytest.approx(1.0 - c[dropped].sum() / c.sum(), rel=1e-13)


def test_calibration_picks_the_sparsest_candidate_that_reaches_tau():
    """Two blocks of four tokens with a hand-made key layout: the newest query (and every other
    query) looks almost only at token 1 of block 0 and token 2 of block 1.  Candidates: one token
    per block, two per block, everything.  One token per block already holds more than 90 % of
    the aggregated score, so Algorithm 1 must return it; with tau = 0.9999 only 'everything'
    qualifies; sizes are 2, 4 and 8."""
    b, w, d = 4, 4, 4
    L = 2 * b + w
    K = np.zeros((L, d))
    K[1, 0] = K[6, 0] = 6.0                                 # the two keys every query likes
    K[:, 1] = np.linspace(0.0, 0.3, L)                      # breaks ties inside the blocks
    Q = np.zeros((1, L, d))
    Q[0, :, 0] = 3.0
    Q[0, :, 1] = 1.0
    cands = np.array([[1.0, 0.0, 0.0], [0.0, 1.0, 0.0], [0.0, 0.0, 1.0]])   # over K = {1, 2, 4}
    choice, a, sizes = O.calibrate_head(Q, K, cands, b, w, 0.5, 0.9, 1.0)
    assert list(sizes) == [2, 4, 8]
    assert a[2] == pytest.approx(1.0, rel=1e-12) and np.all(np.diff(a) > 0)
    assert a[0] > 0.9 and choice == 0
    # what candidate 0 selects is those two tokens; a_0 is the share of the column means that
    # they and the always-kept tail [8, 12) hold
    r = O.select_head(Q[:, L - 1], K, cands[0], b, w, 0.5, 1.0)
    assert list(r["S"]) == [1, 6]
    c = O.attention_column_means(Q, K, 1.0)
    assert a[0] == pytest.approx((c[1] + c[6] + c[8:].sum()) / c.sum(), rel=1e-12)
    choice_hi, _, _ = O.calibrate_head(Q, K, cands, b, w, 0.5, 0.9999, 1.0)
    assert choice_hi == 2
    # a threshold nothing reaches falls back to the last candidate; equal sizes go to the lower index
    assert O.calibrate_head(Q, K, cands[:2], b, w, 0.5, 0.99999, 1.0)[0] == 1
    assert O.calibrate_head(Q, K, np.stack([cands[1], cands[1]]), b, w, 0.5, 0.5, 1.0)[0] == 0


# ----------------------------------------------------------------------------- ablation variants
@pytest.mark.parametrize("b", [4, 32, 128])
def test_entropy_index_closed_forms(b):
    """Uniform block: H = ln b; one-hot block: H = 0; two equal scores: ln 2; a common factor on
    the block's scores leaves H unchanged; with alpha = 1 the metric is H alone."""
    uniform = np.full(b, math.log(1.0 / (3 * b)))
    onehot = np.full(b, -700.0)
    onehot[b // 2] = math.log(0.2)
    two = np.full(b, -700.0)
    two[0] = two[b - 1] = math.log(0.1)
    ls = np.concatenate([uniform, onehot, two, uniform + 2.5])
    h = O.block_metric_entropy(ls, 4, b, 1.0)
    assert h[0] == pytest.approx(math.log(b), rel=1e-12)
    assert h[1] == pytest.approx(0.0, abs=1e-12)
    assert h[2] == pytest.approx(math.log(2.0), rel=1e-12)
    assert h[3] == pytest.approx(h[0], rel=1e-12)                    # scale invariance
    mass = O.block_metric_entropy(ls, 4, b, 0.0)                     # alpha = 0: the mass term, as in Eq. 6
    np.testing.assert_allclose(mass, O.block_metric(ls, 4, b, 0.0), rtol=1e-14)
    assert mass[0] == pytest.approx(1.0 / 3.0, rel=1e-12)
    # against SciPy's entropy of the normalised block
    rng = _rng(31)
    x = rng.standard_normal(3 * b) * 2
    from scipy.stats import entropy as sp_entropy
    want = [sp_entropy(sp_softmax(x[j * b:(j + 1) * b])) for j in range(3)]
    np.testing.assert_allclose(O.block_metric_entropy(x, 3, b, 1.0), want, rtol=1e-12)


def test_random_order_is_a_seeded_permutation_of_psi():
    """The random-order variant hands out exactly the counts of Psi (a permutation of it), the
    same ones for the same seed, different ones for another seed or another head unit."""
    m, b = 40, 8
    n = O.resolve_counts([0.4, 0.3, 0.2, 0.1], m)
    psi = O.budget_map(n, b)
    k0 = O.random_block_keys(7, 3, m)
    assert np.all((k0 >= 0) & (k0 < 1)) and len(np.unique(k0)) == m
    t0 = O.block_requirement(k0, n, b)
    np.testing.assert_array_equal(np.sort(t0), psi)
    np.testing.assert_array_equal(O.block_requirement(O.random_block_keys(7, 3, m), n, b), t0)
    assert not np.array_equal(O.block_requirement(O.random_block_keys(8, 3, m), n, b), t0)
    assert not np.array_equal(O.block_requirement(O.random_block_keys(7, 4, m), n, b), t0)
    # the mixing function against its published test vector: SplitMix64 seeded with 0 gives
    # 0xE220A8397B1DCDAF as its first output
    assert O._splitmix64(0) == 0xE220A8397B1DCDAF
    # keys do not depend on the scores: the order is independent of h
    rng = _rng(32)
    h = rng.random(m)
    assert not np.array_equal(O.rank_blocks(h), O.rank_blocks(k0))


def test_flat_top_b_is_a_truncated_stable_argsort_and_a_best_subset():
    rng = _rng(33)
    ls = np.round(rng.standard_normal(24), 1)                 # rounded: ties exist
    S = O.select_tokens_flat(ls, 7, 20)
    assert np.all(np.diff(S) > 0) and len(S) == 7 and S.max() < 20
    np.testing.assert_array_equal(S, np.sort(np.lexsort((np.arange(20), -ls[:20]))[:7]))
    # best subset by brute force on a tiny tie-free case
    import itertools
    x = rng.standard_normal(9)
    best = max(itertools.combinations(range(8), 3), key=lambda c: sum(x[list(c)]))
    np.testing.assert_array_equal(O.select_tokens_flat(x, 3, 8), np.array(best))
    # ties go to the lower index; nothing outside the candidates is ever taken
    tie = np.array([1.0, 5.0, 5.0, 5.0, 0.0, 9.0])
    np.testing.assert_array_equal(O.select_tokens_flat(tie, 2, 5), [1, 2])
    # one block covering all candidates: the block-wise rule gives the same set
    np.testing.assert_array_equal(O.select_tokens_flat(x, 3, 8), O.select_tokens(x, [3], 8))


def test_variant_heads_keep_the_budget_and_differ_from_the_method():
    rng = _rng(34)
    L, d, G, b, w = 200, 16, 2, 8, 24
    K = rng.standard_normal((L, d)) * 1.5
    q = rng.standard_normal((G, d)) * 1.5
    p = np.array([0.4, 0.3, 0.2, 0.1])
    base = O.select_head(q, K, p, b, w, 0.5, 0.25)
    for variant in ("entropy", "random", "flat"):
        r = O.select_head_variant(q, K, p, b, w, 0.5, 0.25, variant, seed=5, unit=1)
        assert len(r["S"]) == len(base["S"]) and np.all(np.diff(r["S"]) > 0) and r["S"].max() < base["m"] * b
        assert not np.array_equal(r["S"], base["S"])
    flat = O.select_head_variant(q, K, p, b, w, 0.5, 0.25, "flat")
    dropped = np.setdiff1d(np.arange(base["m"] * b), flat["S"])
    assert base["log_s"][flat["S"]].min() >= base["log_s"][dropped].max()
