"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle.

Tolerances (on the bf16 output): max abs error <= 1e-2 and per-row relative L2
<= 5e-3 for every (sequence, query head) row; KV append is bit-exact.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from pd_testlib import assert_parity, ctx_for, error_metrics, oracle_on_cache

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_attn(ctx, cache, q, lens_dev, sm_scale, split_pages=0, want_lse=True):
    B, Hq, d = q.shape
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=q.device)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=q.device) if want_lse else None
    ctx.pd.pd_decode_attn(ctx.h, q, cache.k_pages, cache.v_pages, cache.page_table, lens_dev, out, lse,
                          sm_scale=sm_scale, split_pages=split_pages)
    torch.cuda.synchronize()
    code, seq, detail = ctx.pd.pd_device_status(ctx.h)
    assert code == 0, f"device status {code} seq {seq} detail {detail}"
    return out, lse


# ---------------------------------------------------------------- append

@pytest.mark.parametrize("Hkv,d", [(2, 64), (8, 128), (4, 128)])
def test_kv_append_bit_exact(Hkv, d):
    lens0 = np.array([0, 1, 15, 16, 17, 31, 32, 100, 255], dtype=np.int32)
    B = len(lens0)
    cache = wl.build_paged_cache(lens0, Hkv, d, seed=31, device=DEV, reserve_tokens=20)
    k_host, v_host = oracle.bf16_bits(cache.k_pages).copy(), oracle.bf16_bits(cache.v_pages).copy()
    lens_host = lens0.copy()
    with ctx_for(cache, Hkv) as ctx:
        for step in range(20):
            kn = wl.random_bf16((B, Hkv, d), 1000 + step, DEV)
            vn = wl.random_bf16((B, Hkv, d), 2000 + step, DEV)
            ctx.pd.pd_kv_append(ctx.h, kn, vn, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens)
            assert oracle.kv_append(oracle.bf16_bits(kn), oracle.bf16_bits(vn), k_host, v_host,
                                    cache.page_table_host, lens_host) == 0
        torch.cuda.synchronize()
        assert ctx.pd.pd_device_status(ctx.h)[0] == 0
        assert np.array_equal(cache.ctx_lens.cpu().numpy(), lens_host)
        assert np.array_equal(oracle.bf16_bits(cache.k_pages), k_host)  # every byte of both pools
        assert np.array_equal(oracle.bf16_bits(cache.v_pages), v_host)
        # without advance: same slot rewritten, lengths unchanged
        kn = wl.random_bf16((B, Hkv, d), 5, DEV)
        ctx.pd.pd_kv_append(ctx.h, kn, kn, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens,
                            call_flags=ctx.pd.PD_APPEND_NO_ADVANCE)
        oracle.kv_append(oracle.bf16_bits(kn), oracle.bf16_bits(kn), k_host, v_host, cache.page_table_host,
                         lens_host, advance=False)
        torch.cuda.synchronize()
        assert np.array_equal(cache.ctx_lens.cpu().numpy(), lens_host)
        assert np.array_equal(oracle.bf16_bits(cache.k_pages), k_host)
        assert np.array_equal(oracle.bf16_bits(cache.v_pages), v_host)


def test_kv_append_out_of_range_is_skipped_and_reported():
    lens0 = np.array([16, 5], dtype=np.int32)
    cache = wl.build_paged_cache(lens0, 2, 64, seed=32, device=DEV, poison=True)  # next page of seq 0 is -1
    before_k = oracle.bf16_bits(cache.k_pages).copy()
    kn = wl.random_bf16((2, 2, 64), 6, DEV)
    with ctx_for(cache, 2) as ctx:
        ctx.pd.pd_kv_append(ctx.h, kn, kn, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens)
        code, seq, detail = ctx.pd.pd_device_status(ctx.h)
        assert code == ctx.pd.PD_ERR_DEVICE_FAULT and seq == 0
        assert cache.ctx_lens.cpu().tolist() == [16, 6]  # sequence 0 not advanced, sequence 1 appended
        after_k = oracle.bf16_bits(cache.k_pages)
        page1 = cache.page_table_host[1, 0]
        changed = np.argwhere((after_k != before_k) & ~((np.isnan(oracle.bf16_bits_to_f64(after_k))) &
                                                         np.isnan(oracle.bf16_bits_to_f64(before_k))))
        assert len(changed) and np.all(changed[:, 0] == page1) and np.all(changed[:, 2] == 5)
        assert ctx.pd.pd_device_status(ctx.h)[0] == 0  # cleared


# ---------------------------------------------------------------- attention, small and adversarial

GEOMS = [(8, 2, 64), (32, 8, 128), (32, 4, 128), (8, 8, 64), (4, 2, 128), (16, 8, 64)]


@pytest.mark.parametrize("Hq,Hkv,d", GEOMS)
@pytest.mark.parametrize("split_pages", [0, 1, 2, 3, 7, 100000])
def test_small_ragged_poisoned(Hq, Hkv, d, split_pages):
    lens = np.array([1, 15, 16, 17, 31, 33, 64, 300, 1, 1000, 47], dtype=np.int32)
    B = len(lens)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=40 + d + Hq, device=DEV, poison=True)
    q = wl.random_bf16((B, Hq, d), 7 + Hq, DEV)
    scale = 1.0 / math.sqrt(d)
    with ctx_for(cache, Hq) as ctx:
        out, lse = run_attn(ctx, cache, q, cache.ctx_lens, scale, split_pages)
        plan = ctx.pd.pd_last_plan(ctx.h)
    ref, ref_lse = oracle_on_cache(q, cache, lens, scale)
    assert_parity(out, ref, f"geom {Hq}/{Hkv}/{d} split {split_pages}")
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=2e-5, atol=2e-5)
    total = Hkv * int(((lens + 15) // 16).sum())
    assert plan["total_units"] == total
    # the plan the device used is the one the host-side function gives for the same inputs
    _starts, host_lens = ctx.pd.pd_plan_ranges(total, plan["num_workers"], split_pages)
    assert len(host_lens) == plan["num_ranges"] and int(host_lens[0]) == min(plan["pages_per_range"], total)
    if split_pages:
        assert plan["pages_per_range"] >= split_pages
        assert plan["num_ranges"] == -(-total // plan["pages_per_range"])


def test_closed_forms_on_gpu():
    """One-token context is bit-exact; tanh(1/2) and the three-token softmax to bf16 rounding."""
    d = 64
    # sequence 0: one token; 1: two tokens (tanh case); 2: three tokens; 3: overflow case; 4: empty
    lens = np.array([1, 2, 3, 20, 0], dtype=np.int32)
    cache = wl.build_paged_cache(lens, 1, d, seed=50, device=DEV, poison=True, max_pages_per_seq=4)
    q = torch.zeros((5, 1, d), dtype=torch.bfloat16, device=DEV)
    tbl = cache.page_table_host
    K, V = cache.k_pages, cache.v_pages
    q[0] = wl.random_bf16((1, d), 51, DEV)
    for b in (1, 2):
        q[b, 0, 0] = 8.0
        K[tbl[b, 0], 0, :lens[b]] = 0
        V[tbl[b, 0], 0, :lens[b]] = 0
    K[tbl[1, 0], 0, 0, 0] = 1.0
    V[tbl[1, 0], 0, 0] = 1.0
    V[tbl[1, 0], 0, 1] = -1.0
    K[tbl[2, 0], 0, 0, 0] = 1.0
    K[tbl[2, 0], 0, 1, 0] = 2.0
    for t in range(3):
        V[tbl[2, 0], 0, t, t] = 1.0
    q[3, 0, 0] = 256.0
    for t in range(20):
        K[tbl[3, t // 16], 0, t % 16] = 0
    K[tbl[3, 0], 0, 7, 0] = 32.0  # scaled logit 1024
    with ctx_for(cache, 1) as ctx:
        out, lse = run_attn(ctx, cache, q, cache.ctx_lens, 0.125)
    o = out.float().cpu().numpy()
    assert torch.equal(out[0, 0], V[tbl[0, 0], 0, 0])  # bit-exact copy of the only V row
    np.testing.assert_allclose(o[1, 0], math.tanh(0.5), rtol=2 ** -8)
    Z = 1 + math.e + math.e ** 2
    np.testing.assert_allclose(o[2, 0, :3], [math.e / Z, math.e ** 2 / Z, 1 / Z], rtol=2 ** -8)
    assert np.all(o[2, 0, 3:] == 0)
    assert torch.equal(out[3, 0], V[tbl[3, 0], 0, 7])  # weight exactly 1 on token 7
    assert np.all(o[4] == 0) and lse[4, 0].item() == -math.inf
    l = lse.cpu().numpy()
    np.testing.assert_allclose(l[1:4, 0], [math.log1p(math.e), math.log(Z), 1024.0], rtol=1e-6)


@pytest.mark.parametrize("shape", ["rising", "falling", "jumps"])
def test_running_max_refresh_paths(shape):
    """Logits that drift far from the first page's maximum: slowly (inside the rescale slack for several
    pages, then beyond it), downwards (never beyond it), and in jumps of tens of log2 units."""
    Hq, Hkv, d = 8, 1, 64
    L = 2000
    lens = np.array([L, L // 3], dtype=np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=80, device=DEV, poison=True)
    t = np.arange(L)
    if shape == "rising":
        a = np.floor(t * (30.0 / L) * 8) / 8          # logits 0 .. 60 (natural units), bf16-exact steps
    elif shape == "falling":
        a = np.floor((L - 1 - t) * (30.0 / L) * 8) / 8
    else:
        rng = np.random.default_rng(81)
        a = np.repeat(rng.integers(-120, 120, size=L // 50 + 1), 50)[:L] / 4.0  # plateaus of 50 tokens
    q = torch.zeros((2, Hq, d), dtype=torch.bfloat16, device=DEV)
    q[:, :, 0] = 16.0                                  # s_t = 0.125 * 16 * a_t = 2 a_t
    q[:, :, 1:] = (0.05 * wl.random_bf16((2, Hq, d - 1), 82, DEV).float()).to(torch.bfloat16)
    for b in range(2):
        n = int(lens[b])
        pages = torch.from_numpy(cache.page_table_host[b, np.arange(n) // 16].astype(np.int64)).to(DEV)
        slots = torch.from_numpy(np.arange(n) % 16).to(DEV)
        cache.k_pages[pages, 0, slots, 0] = torch.from_numpy(a[:n].astype(np.float32)).to(DEV).to(torch.bfloat16)
    with ctx_for(cache, Hq) as ctx:
        for split in (0, 5, 100000):
            out, lse = run_attn(ctx, cache, q, cache.ctx_lens, 0.125, split_pages=split)
            ref, ref_lse = oracle_on_cache(q, cache, lens, 0.125)
            assert_parity(out, ref, f"{shape} split {split}")
            np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=2e-5, atol=2e-5)


def test_gqa_mapping_and_identical_keys_on_gpu():
    Hq, Hkv, d = 8, 2, 64
    lens = np.array([77, 200], dtype=np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=52, device=DEV)
    for kvh in range(Hkv):
        cache.v_pages[:, kvh] = kvh + 1.0
    q = wl.random_bf16((2, Hq, d), 53, DEV)
    with ctx_for(cache, Hq) as ctx:
        out, _ = run_attn(ctx, cache, q, cache.ctx_lens, 0.125, split_pages=3)
        o = out.float().cpu().numpy()
        for h in range(Hq):
            np.testing.assert_allclose(o[:, h], h // 4 + 1, rtol=2 ** -7)
        # identical keys -> plain mean of V
        cache.k_pages[:] = cache.k_pages[0, 0, 0]
        cache.v_pages.copy_(wl.random_bf16(cache.v_pages.shape, 54, DEV))
        out, lse = run_attn(ctx, cache, q, cache.ctx_lens, 0.125, split_pages=2)
    ref, ref_lse = oracle_on_cache(q, cache, lens, 0.125)
    assert_parity(out, ref, "identical keys")
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=2e-5, atol=2e-5)


def test_page_permutation_and_rerun_are_bit_identical():
    Hq, Hkv, d = 32, 8, 128
    lens = np.array([500, 33, 1200], dtype=np.int32)
    q = wl.random_bf16((3, Hq, d), 55, DEV)
    outs = []
    for perm_seed in (60, 61):
        cache = wl.build_paged_cache(lens, Hkv, d, seed=perm_seed, device=DEV)
        if outs:  # same logical contents under another physical placement
            for b in range(3):
                n = (lens[b] + 15) // 16
                cache.k_pages[cache.page_table_host[b, :n].tolist()] = first.k_pages[first.page_table_host[b, :n].tolist()]
                cache.v_pages[cache.page_table_host[b, :n].tolist()] = first.v_pages[first.page_table_host[b, :n].tolist()]
        else:
            first = cache
        with ctx_for(cache, Hq) as ctx:
            o1, l1 = run_attn(ctx, cache, q, cache.ctx_lens, 0.0884, split_pages=5)
            o2, l2 = run_attn(ctx, cache, q, cache.ctx_lens, 0.0884, split_pages=5)
        assert torch.equal(o1, o2) and torch.equal(l1, l2)
        outs.append((o1, l1))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


def test_append_then_attend_sees_the_new_token():
    Hq, Hkv, d = 4, 1, 64
    lens = np.array([30, 16], dtype=np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=56, device=DEV, reserve_tokens=1)
    q = wl.random_bf16((2, Hq, d), 57, DEV)
    q[:, 1:] = q[:, :1]
    k_new = (64.0 * q[:, :1].float()).to(torch.bfloat16).contiguous()
    v_new = wl.random_bf16((2, Hkv, d), 58, DEV)
    with ctx_for(cache, Hq) as ctx:
        ctx.pd.pd_kv_append(ctx.h, k_new, v_new, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens)
        out, _ = run_attn(ctx, cache, q, cache.ctx_lens, 0.125)
    assert cache.ctx_lens.cpu().tolist() == [31, 17]
    for h in range(Hq):
        assert torch.equal(out[:, h], v_new[:, 0])


def test_host_step_equals_append_plus_attention():
    w = wl.WORKLOADS[0]
    lens = wl.context_lengths(0)
    B = w.batch
    caches = [wl.build_paged_cache(lens, w.num_kv_heads, w.head_dim, seed=0, device=DEV, reserve_tokens=4)
              for _ in range(2)]
    q = wl.random_bf16((B, w.num_q_heads, w.head_dim), 70, DEV)
    kn = wl.random_bf16((B, w.num_kv_heads, w.head_dim), 71, DEV)
    vn = wl.random_bf16((B, w.num_kv_heads, w.head_dim), 72, DEV)
    with ctx_for(caches[0], w.num_q_heads) as ctx:
        c = caches[0]
        ctx.pd.pd_kv_append(ctx.h, kn, vn, c.k_pages, c.v_pages, c.page_table, c.ctx_lens)
        out_dev, _ = run_attn(ctx, c, q, c.ctx_lens, w.sm_scale)
        c = caches[1]
        out_host = torch.empty((B, w.num_q_heads, w.head_dim), dtype=torch.bfloat16).pin_memory()
        ctx.pd.pd_decode_step_host(ctx.h, q.cpu().pin_memory(), kn.cpu().pin_memory(), vn.cpu().pin_memory(),
                                   c.k_pages, c.v_pages, c.page_table, c.ctx_lens, out_host, sm_scale=w.sm_scale)
        assert torch.equal(out_host, out_dev.cpu())
        assert torch.equal(caches[0].k_pages, caches[1].k_pages)
        assert c.ctx_lens.cpu().tolist() == (lens + 1).tolist()
        # host buffers that follow one another (q, k_new, v_new in one slab) take the single-copy path
        slab = torch.empty(q.numel() + kn.numel() + vn.numel(), dtype=torch.bfloat16).pin_memory()
        a, b2 = q.numel(), q.numel() + kn.numel()
        slab[:a].copy_(q.reshape(-1)); slab[a:b2].copy_(kn.reshape(-1)); slab[b2:].copy_(vn.reshape(-1))
        c2 = wl.build_paged_cache(lens, w.num_kv_heads, w.head_dim, seed=0, device=DEV, reserve_tokens=4)
        out_slab = torch.empty_like(out_host).pin_memory()
        ctx.pd.pd_decode_step_host(ctx.h, slab[:a].view(q.shape), slab[a:b2].view(kn.shape), slab[b2:].view(vn.shape),
                                   c2.k_pages, c2.v_pages, c2.page_table, c2.ctx_lens, out_slab, sm_scale=w.sm_scale)
        assert torch.equal(out_slab, out_host)
        assert torch.equal(c2.k_pages, caches[0].k_pages) and torch.equal(c2.v_pages, caches[0].v_pages)
        # pinned result buffers take the direct path (the merge kernel stores the rows on the host and raises a
        # flag), a pageable one is staged on the device and copied back: same bits either way
        direct0, staged0 = ctx.pd.pd_host_step_counts(ctx.h)
        assert direct0 == 2 and staged0 == 0
        c3 = wl.build_paged_cache(lens, w.num_kv_heads, w.head_dim, seed=0, device=DEV, reserve_tokens=4)
        out_pageable = torch.empty((B, w.num_q_heads, w.head_dim), dtype=torch.bfloat16)
        ctx.pd.pd_decode_step_host(ctx.h, q.cpu(), kn.cpu(), vn.cpu(), c3.k_pages, c3.v_pages, c3.page_table, c3.ctx_lens,
                                   out_pageable, sm_scale=w.sm_scale)
        assert ctx.pd.pd_host_step_counts(ctx.h) == (2, 1)
        assert torch.equal(out_pageable, out_host)


def test_bad_page_id_is_reported_not_fatal():
    lens = np.array([40, 40], dtype=np.int32)
    cache = wl.build_paged_cache(lens, 2, 64, seed=59, device=DEV)
    cache.page_table[1, 1] = cache.num_pages + 5
    q = wl.random_bf16((2, 8, 64), 60, DEV)
    out = torch.zeros((2, 8, 64), dtype=torch.bfloat16, device=DEV)
    with ctx_for(cache, 8) as ctx:
        ctx.pd.pd_decode_attn(ctx.h, q, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out,
                              sm_scale=0.125)
        code, seq, detail = ctx.pd.pd_device_status(ctx.h)
        assert code == ctx.pd.PD_ERR_DEVICE_FAULT and seq == 1 and detail == cache.num_pages + 5
        ref, _ = oracle_on_cache(q, cache, lens, 0.125, seq_ids=[0])
        assert_parity(out[:1], ref, "unaffected sequence")


def test_argument_errors_return_codes():
    import paper_2609_35158_b200 as pd

    with pytest.raises(pd.PdError) as e:
        pd.pd_create(8, 3, 64, 16, 4, 4, 16)
    assert e.value.code == pd.PD_ERR_INVALID_ARG
    for bad in ((8, 2, 96, 16), (8, 2, 64, 32), (32, 2, 64, 16)):
        with pytest.raises(pd.PdError) as e:
            pd.pd_create(bad[0], bad[1], bad[2], bad[3], 4, 4, 16)
        assert e.value.code == pd.PD_ERR_UNSUPPORTED
    lens = np.array([20], dtype=np.int32)
    cache = wl.build_paged_cache(lens, 2, 64, seed=61, device=DEV)
    q = wl.random_bf16((1, 8, 64), 62, DEV)
    out = torch.zeros_like(q)
    with ctx_for(cache, 8) as ctx:
        for kwargs in (dict(batch=2), dict(sm_scale=0.0), dict(sm_scale=float("nan")), dict(split_pages=-1)):
            with pytest.raises(pd.PdError) as e:
                pd.pd_decode_attn(ctx.h, q, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out,
                                  **{"sm_scale": 0.125, **kwargs})
            assert e.value.code == pd.PD_ERR_INVALID_ARG
        with pytest.raises(pd.PdError):
            pd.pd_decode_attn(ctx.h, None, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out,
                              batch=1, sm_scale=0.125)
        n0 = pd.pd_launch_count(ctx.h)
        pd.pd_decode_attn(ctx.h, q, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out,
                          sm_scale=0.125)
        assert pd.pd_launch_count(ctx.h) == n0 + 2 and pd.pd_workspace_bytes(ctx.h) > 0


# ---------------------------------------------------------------- the five workloads

def test_config0_append_then_attend():
    w = wl.WORKLOADS[0]
    lens = wl.context_lengths(0)
    B = w.batch
    cache = wl.build_paged_cache(lens, w.num_kv_heads, w.head_dim, seed=0, device=DEV, reserve_tokens=1)
    q = wl.random_bf16((B, w.num_q_heads, w.head_dim), 1, DEV)
    kn = wl.random_bf16((B, w.num_kv_heads, w.head_dim), 2, DEV)
    vn = wl.random_bf16((B, w.num_kv_heads, w.head_dim), 3, DEV)
    k_host, v_host = oracle.bf16_bits(cache.k_pages).copy(), oracle.bf16_bits(cache.v_pages).copy()
    lens_host = lens.copy()
    oracle.kv_append(oracle.bf16_bits(kn), oracle.bf16_bits(vn), k_host, v_host, cache.page_table_host, lens_host)
    ref, ref_lse = oracle.decode_attn(oracle.bf16_bits(q), k_host, v_host, cache.page_table_host, lens_host,
                                      w.sm_scale)
    with ctx_for(cache, w.num_q_heads) as ctx:
        ctx.pd.pd_kv_append(ctx.h, kn, vn, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens)
        out, lse = run_attn(ctx, cache, q, cache.ctx_lens, w.sm_scale)
    assert np.array_equal(oracle.bf16_bits(cache.k_pages), k_host)
    assert np.array_equal(oracle.bf16_bits(cache.v_pages), v_host)
    assert np.array_equal(cache.ctx_lens.cpu().numpy(), lens + 1)
    assert_parity(out, ref, "config 0")
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=2e-5, atol=2e-5)


@pytest.mark.parametrize("config", [1, 2, 3])
def test_full_size_configs_all_rows(config):
    """Configs 1-3 at full size in the automatic split mode the benchmark times; every row checked."""
    w = wl.WORKLOADS[config]
    lens = wl.context_lengths(config)
    cache = wl.build_paged_cache(lens, w.num_kv_heads, w.head_dim, seed=config, device=DEV)
    q = wl.random_bf16((w.batch, w.num_q_heads, w.head_dim), 100 + config, DEV)
    with ctx_for(cache, w.num_q_heads) as ctx:
        out, lse = run_attn(ctx, cache, q, cache.ctx_lens, w.sm_scale)
        plan = ctx.pd.pd_last_plan(ctx.h)
    assert plan["num_ranges"] >= plan["num_workers"]  # every worker warp has a first range of its own
    ref, ref_lse = oracle_on_cache(q, cache, lens, w.sm_scale)
    max_abs, rel = assert_parity(out, ref, f"config {config}")
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=2e-5, atol=2e-5)
    print(f"config {config}: max_abs {max_abs:.2e} rel_l2 {rel:.2e} plan {plan}")


def test_head_dim_64_with_every_worker_busy():
    """configs[1]'s batch and context lengths at head_dim 64 (16 worker warps per CTA there): the automatic plan
    gives every worker ranges of its own and claims more from the counter; every row checked, for the attention
    call and for the fused step (bit-identical to append + attention)."""
    Hq, Hkv, d = 32, 8, 64
    lens = wl.context_lengths(1)
    B = len(lens)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=61, device=DEV, reserve_tokens=2)
    q = wl.random_bf16((B, Hq, d), 161, DEV)
    scale = d ** -0.5
    with ctx_for(cache, Hq) as ctx:
        out, lse = run_attn(ctx, cache, q, cache.ctx_lens, scale)
        plan = ctx.pd.pd_last_plan(ctx.h)
        assert plan["num_workers"] == 16 * (plan["num_workers"] // 16) and plan["num_ranges"] > plan["num_workers"]
        ref, ref_lse = oracle_on_cache(q, cache, lens, scale)
        assert_parity(out, ref, "head_dim 64, configs[1] lengths")
        np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=2e-5, atol=2e-5)
        # one step both ways on copies of the cache
        kn = wl.random_bf16((B, Hkv, d), 162, DEV)
        vn = wl.random_bf16((B, Hkv, d), 163, DEV)
        k2, v2, l2 = cache.k_pages.clone(), cache.v_pages.clone(), cache.ctx_lens.clone()
        out_a, out_b = torch.empty_like(q), torch.empty_like(q)
        ctx.pd.pd_kv_append(ctx.h, kn, vn, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens)
        ctx.pd.pd_decode_attn(ctx.h, q, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out_a, sm_scale=scale)
        ctx.pd.pd_decode_step(ctx.h, q, kn, vn, k2, v2, cache.page_table, l2, out_b, sm_scale=scale)
        torch.cuda.synchronize()
        assert ctx.pd.pd_device_status(ctx.h)[0] == 0
    assert torch.equal(out_a.view(torch.int16), out_b.view(torch.int16))
    assert torch.equal(cache.k_pages.view(torch.int16), k2.view(torch.int16)) and torch.equal(cache.ctx_lens, l2)


def _compact_host_mirror(cache, lens, seq_ids, extra_pages):
    """Host copy of the pages the given sequences own, renumbered 0, 1, 2, ... with `extra_pages` fresh
    (NaN-filled) pages of room behind each sequence, and the table that goes with it."""
    P = wl.PAGE_SIZE
    n_pages = [(int(lens[b]) + P - 1) // P for b in seq_ids]
    table = np.full((len(seq_ids), max(n_pages) + extra_pages), -1, dtype=np.int32)
    src, cur = [], 0
    for i, (b, n) in enumerate(zip(seq_ids, n_pages)):
        table[i, :n + extra_pages] = np.arange(cur, cur + n + extra_pages)
        src.append((cur, cache.page_table_host[b, :n].astype(np.int64)))
        cur += n + extra_pages
    shape = (cur,) + tuple(cache.k_pages.shape[1:])
    k = np.full(shape, wl.NAN_BF16_BITS, dtype=np.uint16)
    v = np.full(shape, wl.NAN_BF16_BITS, dtype=np.uint16)
    for (start, phys) in src:
        idx = torch.from_numpy(phys).to(cache.k_pages.device)
        k[start:start + len(phys)] = oracle.bf16_bits(cache.k_pages.index_select(0, idx))
        v[start:start + len(phys)] = oracle.bf16_bits(cache.v_pages.index_select(0, idx))
    return k, v, table


def test_config4_multiturn_loop_with_page_allocation():
    """Config 4 at full batch: 128 steps of (allocate, append, attend) with the host free list in the loop,
    run in both forms side by side on two caches: pd_kv_append + pd_decode_attn on one, the fused
    pd_decode_step (what the benchmark times) on the other, every output of every step compared bit for bit.
    Against the oracle: the whole batch (all 512 sequences, every row) on steps 0, 1, 63, 126 and 127, and 16
    fixed sequences (shortest, longest, page openers, page fillers) on all 128 steps. The 16 live in a host
    mirror that the ORACLE's append grows from the same k_new / v_new, so their check covers the GPU append
    and the attention together; at the end the mirror must equal the device pages byte for byte."""
    w = wl.WORKLOADS[4]
    lens0 = wl.context_lengths(4)
    B, steps, P = w.batch, 128, wl.PAGE_SIZE
    full_steps = (0, 1, 63, 126, 127)
    caches = [wl.build_paged_cache(lens0, w.num_kv_heads, w.head_dim, seed=4, device=DEV, reserve_tokens=steps,
                                   preassign_reserve=False, poison=False) for _ in range(2)]
    allocs = [wl.PageAllocator(c) for c in caches]
    lens = lens0.copy()
    by_slot = lambda r: [int(b) for b in np.nonzero(lens0 % P == r)[0][:3]]
    sample = [int(np.argmin(lens0)), int(np.argmax(lens0))] + by_slot(0) + by_slot(15) + by_slot(1)
    sample = sorted(set(sample))
    sample += [b for b in range(B) if b not in sample][:16 - len(sample)]
    sample = sorted(sample)
    assert len(sample) == 16
    sample_dev = torch.tensor(sample, device=DEV)
    mk, mv, mtable = _compact_host_mirror(caches[0], lens0, sample, extra_pages=steps // P + 1)
    mlens = lens0[sample].astype(np.int32).copy()
    ar = torch.arange(B, device=DEV)
    allocated = 0
    worst = [0.0, 0.0]
    with ctx_for(caches[0], w.num_q_heads) as ctx_a, ctx_for(caches[1], w.num_q_heads) as ctx_b:
        pd = ctx_a.pd
        for step in range(steps):
            for cache, alloc in zip(caches, allocs):
                need, logical, phys = alloc.assign(lens)
                if len(need):
                    cache.page_table[torch.from_numpy(need).to(DEV), torch.from_numpy(logical).to(DEV)] = \
                        torch.from_numpy(phys).to(DEV)
            allocated += len(need)
            assert np.array_equal(caches[0].page_table_host, caches[1].page_table_host)
            q = wl.random_bf16((B, w.num_q_heads, w.head_dim), 4000 + step, DEV)
            kn = wl.random_bf16((B, w.num_kv_heads, w.head_dim), 5000 + step, DEV)
            vn = wl.random_bf16((B, w.num_kv_heads, w.head_dim), 6000 + step, DEV)
            out_a = torch.empty((B, w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device=DEV)
            out_b = torch.empty_like(out_a)
            a, b = caches
            pd.pd_kv_append(ctx_a.h, kn, vn, a.k_pages, a.v_pages, a.page_table, a.ctx_lens)
            pd.pd_decode_attn(ctx_a.h, q, a.k_pages, a.v_pages, a.page_table, a.ctx_lens, out_a, sm_scale=w.sm_scale)
            pd.pd_decode_step(ctx_b.h, q, kn, vn, b.k_pages, b.v_pages, b.page_table, b.ctx_lens, out_b,
                              sm_scale=w.sm_scale)
            assert torch.equal(out_a.view(torch.int16), out_b.view(torch.int16)), f"step {step}: fused != two calls"
            # append: the slot of every sequence holds exactly the new rows, in both caches
            pos = torch.from_numpy(lens.astype(np.int64)).to(DEV)
            for cache in caches:
                page = cache.page_table[ar, pos // P].long()
                assert torch.equal(cache.k_pages[page, :, pos % P], kn)
                assert torch.equal(cache.v_pages[page, :, pos % P], vn)
            lens = lens + 1
            # the 16 fixed sequences, every step: oracle append + oracle attention on the host mirror
            assert oracle.kv_append(oracle.bf16_bits(kn[sample_dev]), oracle.bf16_bits(vn[sample_dev]), mk, mv, mtable,
                                    mlens) == 0
            ref, _ = oracle.decode_attn(oracle.bf16_bits(q[sample_dev]), mk, mv, mtable, mlens, w.sm_scale)
            m_abs, m_rel = assert_parity(out_b[sample_dev], ref, f"config 4 step {step}, 16 fixed sequences")
            worst = [max(worst[0], m_abs), max(worst[1], m_rel)]
            if step in full_steps:
                assert pd.pd_device_status(ctx_a.h)[0] == 0 and pd.pd_device_status(ctx_b.h)[0] == 0
                assert np.array_equal(a.ctx_lens.cpu().numpy(), lens) and np.array_equal(b.ctx_lens.cpu().numpy(), lens)
                for c0 in range(0, B, 64):  # the whole batch, 64 sequences (about 3 GB of pages) at a time
                    ids = list(range(c0, min(B, c0 + 64)))
                    ref, _ = oracle_on_cache(q, b, lens, w.sm_scale, seq_ids=ids)
                    m_abs, m_rel = assert_parity(out_b[c0:c0 + len(ids)], ref, f"config 4 step {step}, sequences {c0}..")
                    worst = [max(worst[0], m_abs), max(worst[1], m_rel)]
        assert pd.pd_device_status(ctx_a.h)[0] == 0 and pd.pd_device_status(ctx_b.h)[0] == 0
    assert torch.equal(caches[0].k_pages.view(torch.int16), caches[1].k_pages.view(torch.int16))
    assert torch.equal(caches[0].v_pages.view(torch.int16), caches[1].v_pages.view(torch.int16))
    # the mirror the oracle grew equals the device pages of those sequences, byte for byte
    for i, bseq in enumerate(sample):
        n = (int(lens[bseq]) + P - 1) // P
        idx = torch.from_numpy(caches[1].page_table_host[bseq, :n].astype(np.int64)).to(DEV)
        dk, dv = oracle.bf16_bits(caches[1].k_pages.index_select(0, idx)), oracle.bf16_bits(caches[1].v_pages.index_select(0, idx))
        full, tail = int(lens[bseq]) // P, int(lens[bseq]) % P
        hk, hv = mk[mtable[i, :n]], mv[mtable[i, :n]]
        assert np.array_equal(dk[:full], hk[:full]) and np.array_equal(dv[:full], hv[:full])
        if tail:
            assert np.array_equal(dk[full, :, :tail], hk[full, :, :tail]) and np.array_equal(dv[full, :, :tail], hv[full, :, :tail])
    assert allocated >= B * (steps // 16)  # every sequence crossed page boundaries during the loop
    print(f"config 4: worst max_abs {worst[0]:.2e} rel_l2 {worst[1]:.2e}")


def test_maximum_batch_with_empty_and_tiny_contexts():
    """4096 sequences (the largest batch a context accepts), lengths 0..40 with many zeros."""
    Hq, Hkv, d, B = 8, 2, 64, 4096
    rng = np.random.default_rng(90)
    lens = rng.integers(0, 40, size=B, endpoint=True).astype(np.int32)
    lens[rng.integers(0, B, size=300)] = 0
    lens[-1] = 0
    cache = wl.build_paged_cache(lens, Hkv, d, seed=91, device=DEV, max_pages_per_seq=3)
    q = wl.random_bf16((B, Hq, d), 92, DEV)
    with ctx_for(cache, Hq) as ctx:
        for split in (0, 1):
            out, lse = run_attn(ctx, cache, q, cache.ctx_lens, 0.125, split_pages=split)
            ref, ref_lse = oracle_on_cache(q, cache, lens, 0.125)
            assert_parity(out, ref, f"max batch split {split}")
            np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=2e-5, atol=2e-5)
            empty = torch.from_numpy(lens == 0).to(DEV)
            assert torch.all(out[empty] == 0) and torch.all(torch.isinf(lse[empty]))


def test_one_very_long_sequence_alone():
    """Batch 1, 65 536 tokens: every worker warp reads a slice of the same (sequence, KV head) pairs."""
    Hq, Hkv, d = 32, 8, 128
    lens = np.array([65536], dtype=np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=93, device=DEV)
    q = wl.random_bf16((1, Hq, d), 94, DEV)
    with ctx_for(cache, Hq) as ctx:
        out, lse = run_attn(ctx, cache, q, cache.ctx_lens, 1.0 / math.sqrt(d))
    ref, ref_lse = oracle_on_cache(q, cache, lens, 1.0 / math.sqrt(d))
    assert_parity(out, ref, "single 64K sequence")
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=2e-5, atol=2e-5)
