"""Randomised GPU parity: many small problems with random geometry, lengths, split settings and poison,
for decode attention and for append-prefill attention, against the CPU oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from pd_testlib import assert_parity, ctx_for, oracle_on_cache

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("seed", range(24))
def test_decode_random_case(seed):
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128]))
    g = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2, 4, 8]))
    Hq = g * Hkv
    B = int(rng.integers(1, 13))
    kind = seed % 4
    if kind == 0:
        lens = rng.integers(0, 48, size=B)            # tiny, with empties
    elif kind == 1:
        lens = rng.integers(1, 700, size=B)
    elif kind == 2:
        lens = np.where(rng.random(B) < 0.3, rng.integers(2000, 6000, size=B), rng.integers(1, 64, size=B))
    else:
        lens = 16 * rng.integers(1, 40, size=B) + rng.choice([-1, 0, 1], size=B)  # around page boundaries
    lens = np.maximum(lens, 0).astype(np.int32)
    split = int(rng.choice([0, 0, 1, 2, 5, 13, 64, 100000]))
    cache = wl.build_paged_cache(lens, Hkv, d, seed=2000 + seed, device=DEV, poison=True,
                                 max_pages_per_seq=int(max(1, (lens.max() + 15) // 16 + rng.integers(0, 5))))
    q = wl.random_bf16((B, Hq, d), 3000 + seed, DEV)
    scale = float(rng.choice([1.0 / math.sqrt(d), 0.05, 0.3]))
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    with ctx_for(cache, Hq, max_batch=B + int(rng.integers(0, 4))) as ctx:
        ctx.pd.pd_decode_attn(ctx.h, q, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out, lse,
                              sm_scale=scale, split_pages=split)
        torch.cuda.synchronize()
        assert ctx.pd.pd_device_status(ctx.h)[0] == 0
    ref, ref_lse = oracle_on_cache(q, cache, lens, scale)
    what = f"seed {seed}: B={B} {Hq}/{Hkv} d={d} split={split} lens={lens.tolist()}"
    assert_parity(out, ref, what, scale_abs_above=2.0)
    got_lse = lse.cpu().numpy()
    empty = lens == 0
    assert np.all(np.isneginf(got_lse[empty])) and np.all(out[torch.from_numpy(empty).to(DEV)].float().cpu().numpy() == 0)
    np.testing.assert_allclose(got_lse[~empty], ref_lse[~empty], rtol=3e-5, atol=3e-5, err_msg=what)


@pytest.mark.parametrize("seed", range(12))
def test_prefill_random_case(seed):
    rng = np.random.default_rng(5000 + seed)
    d = int(rng.choice([64, 128]))
    g = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2, 4]))
    Hq = g * Hkv
    B = int(rng.integers(1, 7))
    q_lens = rng.integers(0, 200, size=B).astype(np.int32)
    if seed % 3 == 0:
        q_lens = np.minimum(q_lens, 3)
    prefix = np.where(rng.random(B) < 0.3, 0, rng.integers(0, 900, size=B)).astype(np.int32)
    lens = (prefix + q_lens).astype(np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=6000 + seed, device=DEV, poison=True,
                                 max_pages_per_seq=int(max(1, (lens.max() + 15) // 16 + 2)))
    ip = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int32)
    total = int(ip[-1])
    if total == 0:
        pytest.skip("no query tokens drawn")
    q = wl.random_bf16((total, Hq, d), 7000 + seed, DEV)
    scale = float(rng.choice([1.0 / math.sqrt(d), 0.2]))
    out = torch.full((total, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((total, Hq), float("nan"), dtype=torch.float32, device=DEV)
    with ctx_for(cache, Hq) as ctx:
        ctx.pd.pd_prefill_attn(ctx.h, q, torch.from_numpy(ip).to(DEV), cache.k_pages, cache.v_pages, cache.page_table,
                               cache.ctx_lens, out, lse, max_q_len=int(q_lens.max()) + int(rng.integers(0, 40)),
                               sm_scale=scale)
        torch.cuda.synchronize()
        assert ctx.pd.pd_device_status(ctx.h)[0] == 0
    ref, ref_lse = oracle.prefill_attn(oracle.bf16_bits(q), ip, oracle.bf16_bits(cache.k_pages),
                                       oracle.bf16_bits(cache.v_pages), cache.page_table_host, lens, scale)
    what = f"seed {seed}: {Hq}/{Hkv} d={d} q_lens={q_lens.tolist()} prefix={prefix.tolist()}"
    assert_parity(out, ref, what, scale_abs_by_magnitude=True)
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=3e-5, atol=3e-5, err_msg=what)
