"""GPU checks of the elastic KV pool (release and restore of the cache's physical memory with fixed
addresses) together with the attention path that reads from it."""
import numpy as np
import pytest
import torch

import workloads as wl
from pd_testlib import Ctx, assert_parity, oracle_on_cache

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MB = 1 << 20


def free_bytes():
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info(0)[0]


def test_release_and_restore_keep_addresses_and_results():
    import paper_2609_35158_b200 as pd

    Hq, Hkv, d = 32, 8, 128
    lens = wl.context_lengths(0, batch=12) * 8 + 100
    src = wl.build_paged_cache(lens, Hkv, d, seed=41, device=DEV)
    pool_bytes = src.k_pages.numel() * 2
    per_pool = (pool_bytes + 2 * MB - 1) // (2 * MB) * (2 * MB)
    q = wl.random_bf16((len(lens), Hq, d), 42, DEV)
    scale = d ** -0.5

    pool = pd.pd_pool_create(0, 2 * per_pool, 2 * MB)
    try:
        cap, chunk = pd.pd_pool_capacity(pool), pd.pd_pool_chunk_bytes(pool)
        assert cap >= 2 * per_pool and cap % chunk == 0 and chunk % (2 * MB) == 0
        base = pd.pd_pool_base(pool)
        assert base != 0 and base % 256 == 0
        assert pd.pd_pool_resident_bytes(pool) == 0
        with pytest.raises(ValueError):
            pd.pool_tensor(pool, 0, src.k_pages.shape, torch.bfloat16)

        def fill_and_attend(ctx):
            k = pd.pool_tensor(pool, 0, src.k_pages.shape, torch.bfloat16)
            v = pd.pool_tensor(pool, per_pool, src.v_pages.shape, torch.bfloat16)
            assert k.data_ptr() == base and v.data_ptr() == base + per_pool
            k.copy_(src.k_pages)
            v.copy_(src.v_pages)
            out = torch.full((len(lens), Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
            pd.pd_decode_attn(ctx.h, q, k, v, src.page_table, src.ctx_lens, out, sm_scale=scale)
            torch.cuda.synchronize()
            assert pd.pd_device_status(ctx.h)[0] == 0
            return out

        with Ctx(Hq, Hkv, d, len(lens), src.page_table.shape[1], src.k_pages.shape[0]) as ctx:
            before = free_bytes()
            pd.pd_pool_resize(pool, cap)
            assert pd.pd_pool_resident_bytes(pool) == cap
            assert before - free_bytes() >= cap - 64 * MB
            out_plain = torch.empty_like(q)
            pd.pd_decode_attn(ctx.h, q, src.k_pages, src.v_pages, src.page_table, src.ctx_lens, out_plain, sm_scale=scale)
            out1 = fill_and_attend(ctx)
            assert torch.equal(out1, out_plain)
            ref, _ = oracle_on_cache(q, src, lens, scale)
            assert_parity(out1, ref, "attention over the pool")

            # release: the memory goes back to the device, the range stays
            held = free_bytes()
            pd.pd_pool_resize(pool, 0)
            assert pd.pd_pool_resident_bytes(pool) == 0
            assert free_bytes() - held >= cap - 64 * MB
            assert pd.pd_pool_base(pool) == base
            other = torch.empty(cap, dtype=torch.uint8, device=DEV)  # someone else may now use the memory
            other.fill_(7)
            del other
            torch.cuda.empty_cache()

            # restore: same addresses, the context's cached descriptors of the pools are still right
            pd.pd_pool_resize(pool, cap)
            assert pd.pd_pool_base(pool) == base
            out2 = fill_and_attend(ctx)
            assert torch.equal(out2, out1)
    finally:
        pd.pd_pool_destroy(pool)


def test_partial_shrink_keeps_the_resident_prefix():
    import paper_2609_35158_b200 as pd

    pool = pd.pd_pool_create(0, 16 * MB, 2 * MB)
    try:
        chunk = pd.pd_pool_chunk_bytes(pool)
        cap = pd.pd_pool_capacity(pool)
        n_chunks = cap // chunk
        assert n_chunks >= 2
        pd.pd_pool_resize(pool, cap)
        whole = pd.pool_tensor(pool, 0, (cap // 4,), torch.int32)
        pattern = torch.arange(cap // 4, dtype=torch.int32, device=DEV) * 2654435 + 17
        whole.copy_(pattern)
        keep = (n_chunks // 2) * chunk
        pd.pd_pool_resize(pool, keep - 5)  # rounds up to whole chunks
        assert pd.pd_pool_resident_bytes(pool) == keep
        with pytest.raises(ValueError):
            pd.pool_tensor(pool, 0, (cap // 4,), torch.int32)
        head = pd.pool_tensor(pool, 0, (keep // 4,), torch.int32)
        assert torch.equal(head, pattern[: keep // 4])
        pd.pd_pool_resize(pool, cap)  # grow again: the kept part is untouched, the rest is writable
        whole = pd.pool_tensor(pool, 0, (cap // 4,), torch.int32)
        assert torch.equal(whole[: keep // 4], pattern[: keep // 4])
        whole[keep // 4:].fill_(3)
        assert int(whole[-1]) == 3
        with pytest.raises(pd.PdError) as e:
            pd.pd_pool_resize(pool, cap + 1)
        assert e.value.code == pd.PD_ERR_INVALID_ARG
        assert pd.pd_pool_resident_bytes(pool) == cap
    finally:
        pd.pd_pool_destroy(pool)
