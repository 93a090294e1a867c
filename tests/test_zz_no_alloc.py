"""The allocation-free entry point against the regular one.

``pd_decode_attn_static`` serves callers that cannot allocate device memory when
they need attention (a serving engine that already owns the whole device for its
KV pool, a plugin inside another framework's memory budget): its scratch is a
fixed array inside the library instead of the workspace ``pd_create`` allocates.
It must give what ``pd_decode_attn`` gives, within the tolerances every decode
test uses (its plan is a single level of equal ranges, so the bits differ), and
what the CPU oracle gives. Two calls in a row on different inputs check that the
scratch left behind by one call does not leak into the next; a last case fills
the fixed array to its limit. This file sorts last so that a run stopping at the first failure has
already run every other test.
"""
import math

import numpy as np
import pytest
import torch

import workloads as wl
from pd_testlib import MAX_ABS_TOL, REL_L2_TOL, assert_parity, ctx_for, oracle_on_cache

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
        # and against the CPU oracle, like every other decode path
        want, want_lse = oracle_on_cache(q, cache, lens, scale)
        assert_parity(out, want, f"call {call} against the oracle")
        np.testing.assert_allclose(lse.cpu().numpy(), want_lse, rtol=2e-5, atol=2e-5)


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


def largest_batch_that_fits(Hq, Hkv, d, num_sms):
    """The documented limit: status and plan words (256 B each), page prefix sums, then one (max, sum) pair
    and one fp32 output row per partial slot and head of the group, each block rounded up to 256 bytes."""
    r256 = lambda n: (n + 255) & ~255
    g = Hq // Hkv
    fits = lambda B: (512 + r256(4 * (B + 1)) + r256((num_sms * 8 + B * Hkv) * g * 8)
                      + r256((num_sms * 8 + B * Hkv) * g * d * 4)) <= (16 << 20)
    B = 1
    while fits(B + 1):
        B += 1
    return B


def test_static_scratch_entry_point_at_the_edge_of_its_fixed_array():
    """The largest batch the 16 MiB array holds at 32/8 heads, head_dim 128: the carving of the array is
    exercised up to its last block, the result is checked against the oracle, and one sequence more is refused."""
    import paper_2609_35158_b200 as pd

    Hq, Hkv, d = 32, 8, 128
    scale = 1.0 / math.sqrt(d)
    B = largest_batch_that_fits(Hq, Hkv, d, torch.cuda.get_device_properties(0).multi_processor_count)
    assert 64 < B <= 4096
    rng = np.random.default_rng(930)
    lens = rng.integers(0, 120, size=B + 1).astype(np.int32)
    lens[:8] = [3000, 1, 16, 17, 0, 2047, 15, 640]   # a few long rows so that ranges cut contexts into partials
    lens[B - 1] = 333                                # the last sequence's slots are the end of the array
    cache = wl.build_paged_cache(lens, Hkv, d, seed=931, device=DEV, poison=True)
    q = wl.random_bf16((B + 1, Hq, d), 932, DEV)
    out = torch.full((B + 1, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B + 1, Hq), float("nan"), dtype=torch.float32, device=DEV)
    cfg = pd.pd_config(Hq, Hkv, d, wl.PAGE_SIZE, B + 1, cache.page_table.shape[1], cache.num_pages, 0, 0)
    with pytest.raises(pd.PdError) as e:
        pd.pd_decode_attn_static(cfg, q, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out, lse,
                                 batch=B + 1, sm_scale=scale)
    assert e.value.code == pd.PD_ERR_WORKSPACE
    for _ in range(2):
        pd.pd_decode_attn_static(cfg, q, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out, lse,
                                 batch=B, sm_scale=scale)
    torch.cuda.synchronize()
    want, want_lse = oracle_on_cache(q[:B], cache, lens[:B], scale)
    assert_parity(out[:B], want, f"batch {B} at the limit", scale_abs_above=2.0)
    live = lens[:B] > 0
    got_lse = lse[:B].cpu().numpy()
    np.testing.assert_allclose(got_lse[live], want_lse[live], rtol=2e-5, atol=2e-5)
    assert np.all(np.isneginf(got_lse[~live])) and torch.all(out[:B][torch.from_numpy(~live).to(DEV)] == 0)
    assert torch.isnan(out[B].float()).all()         # the row past the batch was not touched
