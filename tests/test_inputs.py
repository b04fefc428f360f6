"""Host-side checks of the synthetic workload generator (no method arithmetic in it)."""
import numpy as np
import torch

from paper_2512_09238_b200 import inputs as I


def test_bf16_rounding_matches_an_independent_conversion():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-8, 8, 20000))).astype(np.float32)
    x[:4] = [0.0, -0.0, 1.0, 1.00390625]             # last one is an exact tie -> even
    bits = I.to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, want)
    back = I.bf16_bits_to_f32(bits)
    np.testing.assert_array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())
    assert I.widen(bits).dtype == np.float64


def test_generate_is_deterministic_and_shaped():
    wl = I.WORKLOADS["config1"].scaled(L=256, decode_steps=8)
    a, b = I.generate(wl), I.generate(wl)
    for key, H in (("q", wl.n_q_heads), ("k", wl.n_kv_heads), ("v", wl.n_kv_heads)):
        assert a[key].shape == (wl.batch, H, 264, wl.head_dim)
        np.testing.assert_array_equal(a[key], b[key])
    c = I.generate(wl.scaled(seed=5))
    assert not np.array_equal(a["k"], c["k"])
    # heavy tokens: the first four keys carry 4x the norm of a typical key
    norms = np.linalg.norm(a["k"][0, 0].astype(np.float64), axis=1)
    assert norms[:4].min() > 2.5 * np.median(norms)


def test_keys_form_runs_of_near_duplicates():
    wl = I.WORKLOADS["config2"].scaled(batch=1, n_q_heads=4, n_kv_heads=1, L=4096)
    k = I.widen(I.generate(wl)["k"][0, 0])
    kn = k / np.linalg.norm(k, axis=1, keepdims=True)
    cos_next = np.sum(kn[1:] * kn[:-1], axis=1)
    # stay probability 0.95 => most neighbours are in the same cluster
    assert np.mean(cos_next > 0.9) > 0.85


def test_budget_tables():
    for name, wl in I.WORKLOADS.items():
        p = I.budget_table(wl)
        assert p.shape == (wl.n_kv_heads, wl.n_counts)
        np.testing.assert_allclose(p.sum(1), 1.0, atol=1e-12)
        f = I.budget_fractions(wl)
        ks = 2.0 ** np.arange(wl.n_counts)
        np.testing.assert_allclose(p @ ks, f * wl.block, rtol=1e-9)
    full = I.fraction_to_p(1.0, 128)
    assert full[-1] == 1.0 and full.sum() == 1.0
    assert I.fraction_to_p(0.001, 128)[0] == 1.0
    for wl in I.WORKLOADS.values():
        assert (wl.L - wl.window) % wl.block == 0
