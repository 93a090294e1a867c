"""The allocation-free entry point against the regular one.

``pd_decode_attn_static`` serves callers that cannot allocate device memory when
they need attention (a serving engine that already owns the whole device for its
KV pool, a plugin inside another framework's memory budget): its scratch is a
fixed array inside the library instead of the workspace ``pd_create`` allocates.
It must give what ``pd_decode_attn`` gives. Two calls in a row on different
inputs check that the scratch left behind by one call does not leak into the
next. This file sorts last so that a run stopping at the first failure has
already run every other test.
"""
import math

import numpy as np
import pytest
import torch

import workloads as wl
from pd_testlib import MAX_ABS_TOL, REL_L2_TOL, ctx_for

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def within_tolerance(a, b):
    a, b = a.float().cpu().numpy().astype(np.float64), b.float().cpu().numpy().astype(np.float64)
    max_abs = np.abs(a - b).max()
    den = np.linalg.norm(b, axis=-1)
    rel = (np.linalg.norm(a - b, axis=-1) / np.where(den > 1e-30, den, 1.0)).max()
    return max_abs <= MAX_ABS_TOL and rel <= REL_L2_TOL


def test_static_scratch_entry_point_matches_regular_entry_point_twice():
    import paper_2609_35158_b200 as pd

    Hq, Hkv, d = 32, 8, 128
    scale = 1.0 / math.sqrt(d)
    cases = [np.array([5000, 33, 1, 16, 12000, 700], dtype=np.int32),   # long rows are split into partials
             np.array([90, 20000, 17, 2500], dtype=np.int32)]
    for call, lens in enumerate(cases):
        B = len(lens)
        cache = wl.build_paged_cache(lens, Hkv, d, seed=900 + call, device=DEV, poison=True)
        q = wl.random_bf16((B, Hq, d), 910 + call, DEV)
        ref = torch.empty((B, Hq, d), dtype=torch.bfloat16, device=DEV)
        ref_lse = torch.empty((B, Hq), dtype=torch.float32, device=DEV)
        with ctx_for(cache, Hq) as ctx:
            pd.pd_decode_attn(ctx.h, q, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, ref, ref_lse,
                              sm_scale=scale)
            torch.cuda.synchronize()
            assert pd.pd_device_status(ctx.h)[0] == 0
        cfg = pd.pd_config(Hq, Hkv, d, wl.PAGE_SIZE, B, cache.page_table.shape[1], cache.num_pages, 0, 0)
        out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
        lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
        free_before = torch.cuda.mem_get_info()[0]  # device-wide free bytes, as the driver reports them
        pd.pd_decode_attn_static(cfg, q, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out, lse,
                                 sm_scale=scale)
        torch.cuda.synchronize()
        if call > 0:  # the first call on a device loads the module that carries the fixed array
            assert torch.cuda.mem_get_info()[0] >= free_before, "the call took device memory"
        assert torch.isfinite(out.float()).all()
        assert within_tolerance(out, ref), f"call {call}"
        np.testing.assert_allclose(lse.cpu().numpy(), ref_lse.cpu().numpy(), rtol=2e-5, atol=2e-5)


def test_static_scratch_entry_point_rejects_oversized_batches():
    import paper_2609_35158_b200 as pd

    Hq, Hkv, d = 32, 8, 128
    lens = np.full(8, 40, dtype=np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=920, device=DEV)
    q = wl.random_bf16((8, Hq, d), 921, DEV)
    out = torch.zeros((8, Hq, d), dtype=torch.bfloat16, device=DEV)
    cfg = pd.pd_config(Hq, Hkv, d, wl.PAGE_SIZE, 4096, cache.page_table.shape[1], cache.num_pages, 0, 0)
    with pytest.raises(pd.PdError) as e:  # 4096 sequences x 8 KV heads of partial slots do not fit 16 MiB
        pd.pd_decode_attn_static(cfg, q, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out,
                                 batch=4096, sm_scale=0.1)
    assert e.value.code == pd.PD_ERR_WORKSPACE
    assert torch.all(out == 0)
