"""The allocation-free decode entry point against the workspace one.

tca_attn_decode_static exists for callers that cannot give the library a workspace (for
instance code running inside an engine that owns every byte of device memory, or a loop
that must not call an allocator).  It keeps its split-KV partials in an array inside the
library, shared by all calls, so the interesting cases are two calls in a row: the second
must not be disturbed by what the first left behind.  The file name sorts last on purpose:
a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import tca_harness as H
from paper_2512_09238_b200 import binding as B
from paper_2512_09238_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _workload():
    return I.WORKLOADS["config2"].scaled(name="no_alloc", batch=2, n_q_heads=8, n_kv_heads=2, L=3000, block=64,
                                         window=512, seed=41, budget=("beta", 2.0, 5.0, 0.05, 1.0))


def test_static_decode_matches_workspace_decode_twice_in_a_row():
    wl = _workload()
    data = I.generate(wl)
    run = H.gpu_select_compact(wl, data, I.budget_table(wl))
    # two different queries, so the second call cannot pass on leftovers of the first
    q1 = run.dev["q"][:, :, wl.L - 1, :].contiguous()
    q2 = run.dev["q"][:, :, wl.L // 3, :].contiguous()
    want1 = H.from_device(H.gpu_decode(run, q1))
    want2 = H.from_device(H.gpu_decode(run, q2))
    assert np.max(np.abs(want1 - want2)) > 1e-2

    got1, got2, again = torch.empty_like(q1), torch.empty_like(q2), torch.empty_like(q1)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    B.tca_attn_decode_static(run.prm, q1, run.cache, got1)
    B.tca_attn_decode_static(run.prm, q2, run.cache, got2)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_before           # the calls took no device memory

    H.check_attention(H.from_device(got1), want1, wl.dtype, "static decode, first call")
    H.check_attention(H.from_device(got2), want2, wl.dtype, "static decode, second call")
    # a third call repeating the first query reproduces it exactly
    B.tca_attn_decode_static(run.prm, q1, run.cache, again)
    torch.cuda.synchronize()
    assert torch.equal(again, got1)
    # no bounded wait gave up in any of the three calls (the only place this variant can say so)
    assert B.tca_decode_static_status() == B.TCA_OK
    assert torch.cuda.mem_get_info()[0] >= free_before


def test_static_decode_refuses_caches_beyond_its_scratch():
    wl = _workload()
    prm = H.params_for(wl)
    U = wl.batch * wl.n_kv_heads
    # a descriptor that only claims to be huge: the size check runs before anything is touched
    rows = 6_000_000
    need = (rows // 256 + 2 * U + 1) * wl.group * (wl.head_dim + 2) * 4
    assert need > B.TCA_DECODE_STATIC_SCRATCH_BYTES
    cache = B.Cache(prm, [16] * U, wl.window + wl.block, [1] * U)
    cache.desc.rows_total = rows
    q = torch.zeros(wl.batch, wl.n_q_heads, wl.head_dim, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.TcaError) as e:
        B.tca_attn_decode_static(prm, q, cache, torch.empty_like(q))
    assert e.value.status == B.TCA_ERR_SCRATCH_LIMIT
    assert "scratch" in str(e.value)
