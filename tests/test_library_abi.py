"""CPU-side checks of the C-ABI library: it builds, loads, exports every symbol that
include/tca.h declares, and its host-only entry points agree with the oracle.  No kernel
is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import tca_oracle as O
from paper_2512_09238_b200 import _build, binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    _build.build()
    return B.lib()


def test_every_declared_symbol_is_exported():
    header = open(os.path.join(ROOT, "include", "tca.h")).read()
    body = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(tca_[a-z_]+)\s*\(", body))
    assert declared == set(B.EXPORTS)
    cdll = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(cdll, name), f"{name} is declared but not exported"
    assert B.tca_version() >= 200
    assert B.tca_build_info() == 0                       # the default build carries no range checks
    assert B.tca_strerror(0) == "ok" and "workspace" in B.tca_strerror(B.TCA_ERR_WORKSPACE)


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(B.tca_params) == 44
    assert ctypes.sizeof(B.tca_cache_desc) == 14 * 8


def test_budget_resolve_matches_oracle_and_hand_case():
    n_k, n_sel, tbar = B.tca_budget_resolve(np.array([[0.5, 0.3, 0.2]]), 5)
    np.testing.assert_array_equal(n_k, [[2, 2, 1]])
    assert n_sel[0] == 10 and tbar[0] == 1
    rng = np.random.default_rng(0)
    for _ in range(300):
        nK = int(rng.integers(1, 9))
        H = int(rng.integers(1, 5))
        p = rng.dirichlet(np.ones(nK) * rng.uniform(0.2, 3), size=H)
        m = int(rng.integers(0, 3000))
        n_k, n_sel, tbar = B.tca_budget_resolve(p, m)
        ks = 2 ** np.arange(nK)
        for h in range(H):
            np.testing.assert_array_equal(n_k[h], O.resolve_counts(p[h], m))
            assert n_sel[h] == int((ks * n_k[h]).sum())
            assert tbar[h] == O.mean_retain_floor(p[h], int(ks[-1]))
    # ties in the fractional parts go to the larger k
    n_k, _, _ = B.tca_budget_resolve(np.array([[0.25, 0.25, 0.25, 0.25]]), 6)
    np.testing.assert_array_equal(n_k, [[1, 1, 2, 2]])
    np.testing.assert_array_equal(O.resolve_counts([0.25] * 4, 6), [1, 1, 2, 2])


def test_budget_resolve_rejects_bad_tables():
    with pytest.raises(B.TcaError) as e:
        B.tca_budget_resolve(np.array([[0.5, 0.4]]), 10)
    assert e.value.status == B.TCA_ERR_INVALID_ARG
    with pytest.raises(B.TcaError):
        B.tca_budget_resolve(np.array([[1.5, -0.5]]), 10)


def test_parameter_validation_happens_on_the_host():
    ok = B.make_params(1, 8, 8, 64, 32, 128, dtype=B.TCA_F32)
    assert B.tca_workspace_bytes(ok, 2048, B.TCA_OP_SCORE) > 0
    assert B.tca_workspace_bytes(ok, 2048, 99) == 0
    for bad in (dict(head_dim=96), dict(block=48), dict(block=256), dict(n_q_heads=7), dict(window=-1),
                dict(dtype=5), dict(alpha=1.5), dict(n_q_heads=128)):
        kw = dict(batch=1, n_q_heads=8, n_kv_heads=8, head_dim=64, block=32, window=128, dtype=B.TCA_F32)
        kw.update(bad)
        assert B.tca_workspace_bytes(B.make_params(**kw), 2048, B.TCA_OP_SCORE) == 0
    # NULL buffers are refused before anything touches the device
    L = B.lib()
    st = L.tca_score(ctypes.byref(ok), None, None, 2048, None, None, 0, None)
    assert st == B.TCA_ERR_INVALID_ARG
    st = L.tca_attn_decode(ctypes.byref(ok), None, None, None, None, 0, None)
    assert st == B.TCA_ERR_INVALID_ARG
    bad = B.make_params(1, 8, 8, 96, 32, 128)
    assert L.tca_score(ctypes.byref(bad), None, None, 2048, None, None, 0, None) == B.TCA_ERR_UNSUPPORTED


def test_prefill_refuses_a_zero_window_before_touching_anything():
    """With w = 0 a query that is not selected itself would attend to nothing; the prefill entry
    points say so (the other calls accept w = 0).  The check precedes every pointer check."""
    w0 = B.make_params(1, 8, 8, 64, 32, 0)
    L = B.lib()
    assert L.tca_attn_prefill(ctypes.byref(w0), None, None, None, 2048, None, None, None, 0, None) == B.TCA_ERR_UNSUPPORTED
    assert L.tca_attn_prefill_rows(ctypes.byref(w0), None, None, None, 2048, 0, 128, None, None, None, 0,
                                   None) == B.TCA_ERR_UNSUPPORTED
    assert B.tca_workspace_bytes(w0, 2048, B.TCA_OP_SELECT) > 0
    w1 = B.make_params(1, 8, 8, 64, 32, 1)
    assert L.tca_attn_prefill(ctypes.byref(w1), None, None, None, 2048, None, None, None, 0, None) == B.TCA_ERR_INVALID_ARG


def test_gather_prefill_and_ranged_compaction_validate_their_arguments_on_the_host():
    """The two entry points added beside tca_attn_prefill_rows and tca_compact_kv refuse what they
    do not support, and bad ranges, before anything touches the device."""
    L = B.lib()
    f32 = B.make_params(1, 8, 8, 64, 32, 128, dtype=B.TCA_F32)
    assert L.tca_attn_prefill_gather(ctypes.byref(f32), None, None, None, 2048, 0, 2048, None, None, None, None, 0,
                                     None) == B.TCA_ERR_UNSUPPORTED          # tensor-core kernel only: bf16
    bf = B.make_params(1, 8, 8, 64, 32, 128, dtype=B.TCA_BF16)
    simt = B.make_params(1, 8, 8, 64, 32, 128, dtype=B.TCA_BF16, flags=B.TCA_FLAG_PREFILL_SIMT)
    assert L.tca_attn_prefill_gather(ctypes.byref(simt), None, None, None, 2048, 0, 2048, None, None, None, None, 0,
                                     None) == B.TCA_ERR_UNSUPPORTED
    assert L.tca_attn_prefill_gather(ctypes.byref(bf), None, None, None, 2048, 0, 2048, None, None, None, None, 0,
                                     None) == B.TCA_ERR_INVALID_ARG          # NULL buffers
    w0 = B.make_params(1, 8, 8, 64, 32, 0, dtype=B.TCA_BF16)
    assert L.tca_attn_prefill_gather(ctypes.byref(w0), None, None, None, 2048, 0, 2048, None, None, None, None, 0,
                                     None) == B.TCA_ERR_UNSUPPORTED          # window >= 1, as for the other prefills
    assert L.tca_compact_kv_range(ctypes.byref(bf), None, None, 2048, 0, 2048, None, None, None, None,
                                  None) == B.TCA_ERR_INVALID_ARG


def test_static_decode_limit_formula_is_the_workspace_size():
    """The limit documented for tca_attn_decode_static is tca_workspace_bytes for TCA_OP_DECODE."""
    def up(x):
        return (x + 255) // 256 * 256
    for (batch, hq, hkv, d, rows) in [(1, 32, 8, 128, 500000), (2, 8, 2, 64, 12345), (4, 7, 1, 128, 256)]:
        prm = B.make_params(batch, hq, hkv, d, 64, 512)
        U, G = batch * hkv, hq // hkv
        want = 256 + up((rows // 256 + 2 * U + 1) * G * (d + 2) * 4)
        assert B.tca_workspace_bytes(prm, rows, B.TCA_OP_DECODE) == want


def test_selection_variant_flags_are_validated():
    ok = dict(batch=1, n_q_heads=8, n_kv_heads=8, head_dim=64, block=32, window=128, dtype=B.TCA_F32)
    for flags in (0, B.TCA_FLAG_ENTROPY_INDEX, B.TCA_FLAG_RANDOM_ORDER, B.TCA_FLAG_FLAT_TOPB,
                  B.TCA_FLAG_ENTROPY_INDEX | B.TCA_FLAG_PREFILL_SIMT, B.TCA_FLAG_PREFILL_BAND_FIRST):
        assert B.tca_workspace_bytes(B.make_params(flags=flags, **ok), 2048, B.TCA_OP_SELECT) > 0
    for flags in (B.TCA_FLAG_ENTROPY_INDEX | B.TCA_FLAG_FLAT_TOPB, B.TCA_FLAG_RANDOM_ORDER | B.TCA_FLAG_ENTROPY_INDEX, 32, 1 << 20):
        assert B.tca_workspace_bytes(B.make_params(flags=flags, **ok), 2048, B.TCA_OP_SELECT) == 0
    prm = B.make_params(**ok)
    both = B.tca_workspace_bytes(prm, 2048, B.TCA_OP_SCORE_SELECT)
    assert both >= B.tca_workspace_bytes(prm, 2048, B.TCA_OP_SCORE) + B.tca_workspace_bytes(prm, 2048, B.TCA_OP_SELECT)


def test_workspace_sizes_scale_as_documented():
    prm = B.make_params(1, 32, 8, 128, 128, 4096)
    L = 131072
    score = B.tca_workspace_bytes(prm, L, B.TCA_OP_SCORE)
    assert score >= 8 * 4 * L * 8                      # logits [U, G, L] in fp64
    assert score < 1.01 * 8 * 4 * L * 8 + (1 << 20)
    sel = B.tca_workspace_bytes(prm, L, B.TCA_OP_SELECT)
    assert sel >= 8 * 992 * 12


def test_candidate_grid_host_helper_matches_eq3():
    """Eq. 3 on the host side of the library against the oracle's restatement and its closed forms."""
    for b in (2, 8, 32, 128):
        got = B.tca_calib_candidates(b, 14, 1.0)
        np.testing.assert_allclose(got, O.candidate_grid(b, 14, 1.0), rtol=1e-13, atol=1e-16)
        np.testing.assert_allclose(got.sum(1), 1.0, rtol=1e-14)
    g = B.tca_calib_candidates(128, 14, 1.0)
    assert g[0, 1] / g[0, 0] == pytest.approx(np.exp(-0.5), rel=1e-12)      # mu^1 = 0
    assert g[-1, -2] / g[-1, -1] == pytest.approx(np.exp(-0.5), rel=1e-12)  # mu^M = log2 b
    for bad in ((96, 14, 1.0), (128, 1, 1.0), (128, 14, 0.0)):
        with pytest.raises(B.TcaError):
            B.tca_calib_candidates(*bad)
    a = np.array([0.2, 0.91, 0.95])
    assert B.tca_calib_choose(a, np.array([5, 9, 9]), 0.9) == 1
    assert B.tca_calib_choose(a, np.array([5, 9, 7]), 0.9) == 2
    assert B.tca_calib_choose(a, np.array([5, 9, 7]), 0.99) == 2            # none valid: the last candidate
