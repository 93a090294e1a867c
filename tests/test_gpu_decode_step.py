"""GPU parity of the fused decode step (append inside the split kernel) against the two-call path
(pd_kv_append then pd_decode_attn) and against the fp64 CPU oracle.

Bars: the pools and the lengths after the step are bit-identical to those the separate append leaves;
the attention output and the LSE are bit-identical to the two-call path (same plan, same arithmetic)
and within max abs 1e-2 / per-row relative L2 5e-3 of the oracle.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from pd_testlib import assert_parity, ctx_for, oracle_on_cache

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
P = wl.PAGE_SIZE


def poisoned_cache_with_room(lens, Hkv, d, seed, reserve_tokens):
    """Every slot that holds no token is NaN (so a read of the pool at the new position would show),
    but the pages that the appends will reach are already in the table."""
    poisoned = wl.build_paged_cache(lens, Hkv, d, seed=seed, device=DEV, reserve_tokens=reserve_tokens, poison=True)
    plain = wl.build_paged_cache(lens, Hkv, d, seed=seed, device=DEV, reserve_tokens=reserve_tokens)
    poisoned.page_table.copy_(plain.page_table)
    return poisoned


def bits(t):
    return t.view(torch.int16)


def step_both_ways(lens, Hq, Hkv, d, seed, split_pages, steps=1, sm_scale=None, check_oracle=True):
    lens = np.asarray(lens, dtype=np.int32)
    B = len(lens)
    sm_scale = sm_scale or d ** -0.5
    a = poisoned_cache_with_room(lens, Hkv, d, seed, reserve_tokens=steps)
    b = poisoned_cache_with_room(lens, Hkv, d, seed, reserve_tokens=steps)
    with ctx_for(a, Hq) as ctx:
        for t in range(steps):
            q = wl.random_bf16((B, Hq, d), seed * 100 + 3 * t, DEV)
            kn = wl.random_bf16((B, Hkv, d), seed * 100 + 3 * t + 1, DEV)
            vn = wl.random_bf16((B, Hkv, d), seed * 100 + 3 * t + 2, DEV)
            out_a = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
            lse_a = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
            out_b, lse_b = out_a.clone(), lse_a.clone()
            ctx.pd.pd_kv_append(ctx.h, kn, vn, a.k_pages, a.v_pages, a.page_table, a.ctx_lens)
            ctx.pd.pd_decode_attn(ctx.h, q, a.k_pages, a.v_pages, a.page_table, a.ctx_lens, out_a, lse_a,
                                  sm_scale=sm_scale, split_pages=split_pages)
            ctx.pd.pd_decode_step(ctx.h, q, kn, vn, b.k_pages, b.v_pages, b.page_table, b.ctx_lens, out_b, lse_b,
                                  sm_scale=sm_scale, split_pages=split_pages)
            torch.cuda.synchronize()
            assert ctx.pd.pd_device_status(ctx.h)[0] == 0
            what = f"step {t}"
            assert b.ctx_lens.cpu().tolist() == (lens + t + 1).tolist(), what
            assert torch.equal(a.ctx_lens, b.ctx_lens), what
            assert torch.equal(bits(a.k_pages), bits(b.k_pages)), what + ": K pool"
            assert torch.equal(bits(a.v_pages), bits(b.v_pages)), what + ": V pool"
            assert torch.equal(bits(out_a), bits(out_b)), what + ": output"
            assert torch.equal(lse_a.view(torch.int32), lse_b.view(torch.int32)), what + ": lse"
            if check_oracle and (t == 0 or t == steps - 1):
                ref, ref_lse = oracle_on_cache(q, b, lens + t + 1, sm_scale)
                assert_parity(out_b, ref, what, scale_abs_above=2.0)
                np.testing.assert_allclose(lse_b.cpu().numpy(), ref_lse, rtol=2e-5, atol=2e-5, err_msg=what)
    return b


GEOMS = [(8, 2, 64), (32, 8, 128), (32, 4, 128), (8, 8, 64), (4, 2, 128)]


@pytest.mark.parametrize("Hq,Hkv,d", GEOMS)
@pytest.mark.parametrize("split_pages", [0, 1, 3, 100000])
def test_step_matches_append_plus_attention(Hq, Hkv, d, split_pages):
    # lengths around page boundaries: the new token opens a page (0, 16, 32), fills one (15, 31), sits inside
    lens = [0, 1, 14, 15, 16, 17, 31, 32, 33, 100, 255, 256, 257, 700]
    step_both_ways(lens, Hq, Hkv, d, seed=11, split_pages=split_pages)


def test_many_steps_cross_page_boundaries():
    rng = np.random.Generator(np.random.PCG64(5))
    lens = rng.integers(0, 400, size=37)
    step_both_ways(lens, 32, 8, 128, seed=12, split_pages=0, steps=20)


def test_only_empty_contexts():
    step_both_ways([0, 0, 0], 8, 2, 64, seed=13, split_pages=0, steps=3)


def test_config0_step():
    w = wl.WORKLOADS[0]
    lens = wl.context_lengths(0)
    step_both_ways(lens, w.num_q_heads, w.num_kv_heads, w.head_dim, seed=14, split_pages=0, sm_scale=w.sm_scale)


def test_full_size_config1_step_equals_two_call_path():
    """Bit-identity only: the two-call path at this size is checked against the oracle, every row, by
    test_gpu_parity.py::test_full_size_configs_all_rows, and identical bits need no second comparison."""
    w = wl.WORKLOADS[1]
    lens = wl.context_lengths(1)
    step_both_ways(lens, w.num_q_heads, w.num_kv_heads, w.head_dim, seed=15, split_pages=0, steps=2,
                   sm_scale=w.sm_scale, check_oracle=False)


def test_new_token_dominates_when_its_key_matches():
    Hq, Hkv, d = 4, 1, 64
    lens = np.array([30, 15, 16, 0], dtype=np.int32)
    cache = poisoned_cache_with_room(lens, Hkv, d, 16, reserve_tokens=1)
    q = wl.random_bf16((4, Hq, d), 17, DEV)
    q[:, 1:] = q[:, :1]
    k_new = (64.0 * q[:, :1].float()).to(torch.bfloat16).contiguous()
    v_new = wl.random_bf16((4, Hkv, d), 18, DEV)
    out = torch.zeros((4, Hq, d), dtype=torch.bfloat16, device=DEV)
    with ctx_for(cache, Hq) as ctx:
        ctx.pd.pd_decode_step(ctx.h, q, k_new, v_new, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens,
                              out, sm_scale=0.125)
        torch.cuda.synchronize()
        assert ctx.pd.pd_device_status(ctx.h)[0] == 0
    for h in range(Hq):
        assert torch.equal(out[:, h], v_new[:, 0])


def test_no_room_or_bad_page_is_reported_and_leaves_the_cache_alone():
    lens = np.array([16, 5, 40], dtype=np.int32)
    # poison=True alone: pages past the current ones are -1 in the table, so sequence 0 has no page for its token
    cache = wl.build_paged_cache(lens, 2, 64, seed=19, device=DEV, poison=True)
    twin = wl.build_paged_cache(lens, 2, 64, seed=19, device=DEV, poison=True)
    q = wl.random_bf16((3, 8, 64), 20, DEV)
    kn = wl.random_bf16((3, 2, 64), 21, DEV)
    vn = wl.random_bf16((3, 2, 64), 22, DEV)
    out = torch.zeros((3, 8, 64), dtype=torch.bfloat16, device=DEV)
    with ctx_for(cache, 8) as ctx:
        ctx.pd.pd_decode_step(ctx.h, q, kn, vn, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out,
                              sm_scale=0.125)
        code, seq, _ = ctx.pd.pd_device_status(ctx.h)
        assert code == ctx.pd.PD_ERR_DEVICE_FAULT and seq == 0
        assert cache.ctx_lens.cpu().tolist() == [16, 6, 41]
        # the other sequences were appended exactly as the separate append does it
        ctx.pd.pd_kv_append(ctx.h, kn, vn, twin.k_pages, twin.v_pages, twin.page_table, twin.ctx_lens)
        ctx.pd.pd_device_status(ctx.h)
        assert torch.equal(bits(cache.k_pages), bits(twin.k_pages))
        assert torch.equal(bits(cache.v_pages), bits(twin.v_pages))
        ref, _ = oracle_on_cache(q, cache, np.array([16, 6, 41]), 0.125, seq_ids=[1, 2])
        assert_parity(out[1:], ref, "sequences beside the faulty one", scale_abs_above=2.0)

    # a table row that is full: the length is reported, nothing is written
    lens = np.array([32, 7], dtype=np.int32)
    cache = wl.build_paged_cache(lens, 2, 64, seed=23, device=DEV, max_pages_per_seq=2)
    before = bits(cache.k_pages).clone()
    q = wl.random_bf16((2, 8, 64), 24, DEV)
    kn = wl.random_bf16((2, 2, 64), 25, DEV)
    out = torch.zeros((2, 8, 64), dtype=torch.bfloat16, device=DEV)
    with ctx_for(cache, 8) as ctx:
        ctx.pd.pd_decode_step(ctx.h, q, kn, kn, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out,
                              sm_scale=0.125)
        code, seq, detail = ctx.pd.pd_device_status(ctx.h)
        assert code == ctx.pd.PD_ERR_DEVICE_FAULT and seq == 0 and detail == 32
        assert cache.ctx_lens.cpu().tolist() == [32, 8]
        changed = (bits(cache.k_pages) != before).nonzero()
        assert len(changed) and bool((changed[:, 0] == int(cache.page_table_host[1, 0])).all()) and bool((changed[:, 2] == 7).all())


def test_argument_errors():
    cache = wl.build_paged_cache([5], 2, 64, seed=26, device=DEV, reserve_tokens=1)
    q = wl.random_bf16((1, 8, 64), 27, DEV)
    kn = wl.random_bf16((1, 2, 64), 28, DEV)
    out = torch.zeros_like(q)
    with ctx_for(cache, 8) as ctx:
        pd = ctx.pd
        with pytest.raises(pd.PdError) as e:
            pd.pd_decode_step(ctx.h, q, None, kn, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out)
        assert e.value.code == pd.PD_ERR_INVALID_ARG
        with pytest.raises(pd.PdError) as e:
            pd.pd_decode_step(ctx.h, q, kn, kn, cache.k_pages, cache.v_pages, cache.page_table, None, out)
        assert e.value.code == pd.PD_ERR_INVALID_ARG
        assert cache.ctx_lens.cpu().tolist() == [5]


def test_decode_step_captured_in_a_cuda_graph_replays_bit_identically():
    """pd_decode_step only enqueues kernels on the given stream (no allocation, no synchronisation, lengths advanced
    on the device), so a run of steps can be captured once and replayed: pools, lengths and outputs after 24
    replayed steps equal those of 24 eager steps bit for bit."""
    import paper_2609_35158_b200 as pd

    w = wl.WORKLOADS[0]
    lens = wl.context_lengths(0)
    B, steps, per_graph = w.batch, 24, 6
    q = wl.random_bf16((B, w.num_q_heads, w.head_dim), 301, DEV)
    kn = wl.random_bf16((B, w.num_kv_heads, w.head_dim), 302, DEV)
    vn = wl.random_bf16((B, w.num_kv_heads, w.head_dim), 303, DEV)
    results = []
    for use_graph in (False, True):
        cache = wl.build_paged_cache(lens, w.num_kv_heads, w.head_dim, seed=300, device=DEV, reserve_tokens=steps + 8)
        out = torch.full_like(q, float("nan"))
        with ctx_for(cache, w.num_q_heads) as ctx:
            def step():
                pd.pd_decode_step(ctx.h, q, kn, vn, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out,
                                  sm_scale=w.sm_scale)
            step()  # the first call encodes the tensor maps of these pools
            torch.cuda.synchronize()
            if use_graph:
                graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
                with torch.cuda.stream(side), torch.cuda.graph(graph, stream=side):
                    for _ in range(per_graph):
                        step()
                torch.cuda.synchronize()
                for _ in range(steps // per_graph):
                    graph.replay()
            else:
                for _ in range(steps):
                    step()
            torch.cuda.synchronize()
            assert pd.pd_device_status(ctx.h)[0] == 0
        results.append((out.clone(), cache.ctx_lens.clone(), cache.k_pages.clone(), cache.v_pages.clone()))
    (o0, l0, k0, v0), (o1, l1, k1, v1) = results
    assert torch.equal(l0, l1) and int(l0[0]) == int(lens[0]) + steps + 1
    assert torch.equal(o0.view(torch.int16), o1.view(torch.int16))
    assert torch.equal(k0.view(torch.int16), k1.view(torch.int16)) and torch.equal(v0.view(torch.int16), v1.view(torch.int16))
