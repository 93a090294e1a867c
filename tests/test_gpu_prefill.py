"""GPU parity of append-prefill attention (tcgen05 kernel) and the multi-token append against the oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from pd_testlib import assert_parity, ctx_for

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_prefill(ctx, cache, q, ip, lens_dev, scale, max_q_len):
    out = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device=DEV)
    ctx.pd.pd_prefill_attn(ctx.h, q, ip, cache.k_pages, cache.v_pages, cache.page_table, lens_dev, out, lse,
                           max_q_len=max_q_len, sm_scale=scale)
    torch.cuda.synchronize()
    code, seq, detail = ctx.pd.pd_device_status(ctx.h)
    assert code == 0, f"device status {code} seq {seq} detail {detail}"
    return out, lse


@pytest.mark.parametrize("Hq,Hkv,d", [(32, 8, 128), (32, 4, 128), (8, 8, 128), (4, 2, 128), (8, 2, 64), (16, 2, 64)])
def test_prefill_small_ragged_poisoned(Hq, Hkv, d):
    lens = np.array([70, 33, 5, 40, 300, 129, 1000, 128], dtype=np.int32)
    q_lens = np.array([20, 33, 1, 0, 37, 129, 200, 16], dtype=np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=100 + Hq, device=DEV, poison=True)
    ip = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int32)
    q = wl.random_bf16((int(ip[-1]), Hq, d), 101 + Hq, DEV)
    scale = 1.0 / math.sqrt(d)
    with ctx_for(cache, Hq) as ctx:
        out, lse = run_prefill(ctx, cache, q, torch.from_numpy(ip).to(DEV), cache.ctx_lens, scale, int(q_lens.max()))
    ref, ref_lse = oracle.prefill_attn(oracle.bf16_bits(q), ip, oracle.bf16_bits(cache.k_pages),
                                       oracle.bf16_bits(cache.v_pages), cache.page_table_host, lens, scale)
    assert_parity(out, ref, f"prefill {Hq}/{Hkv}/{d}", scale_abs_by_magnitude=True)
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=3e-5, atol=3e-5)


def test_prefill_first_token_and_rising_logits():
    """A fresh sequence's first token returns its own V bit-exactly; steadily rising logits force the
    output correction pass many times."""
    Hq, Hkv, d = 8, 1, 128
    L = 1500
    lens = np.array([L, 40], dtype=np.int32)
    q_lens = np.array([300, 40], dtype=np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=110, device=DEV, poison=True)
    ip = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int32)
    q = torch.zeros((int(ip[-1]), Hq, d), dtype=torch.bfloat16, device=DEV)
    q[:, :, 0] = 16.0
    q[:, :, 1:] = (0.05 * wl.random_bf16((int(ip[-1]), Hq, d - 1), 111, DEV).float()).to(torch.bfloat16)
    a = np.floor(np.arange(L) * (30.0 / L) * 8) / 8
    scale = 1.0 / math.sqrt(d)
    for b in range(2):
        n = int(lens[b])
        pages = torch.from_numpy(cache.page_table_host[b, np.arange(n) // 16].astype(np.int64)).to(DEV)
        slots = torch.from_numpy(np.arange(n) % 16).to(DEV)
        cache.k_pages[pages, 0, slots, 0] = torch.from_numpy(a[:n].astype(np.float32)).to(DEV).to(torch.bfloat16)
    with ctx_for(cache, Hq) as ctx:
        out, lse = run_prefill(ctx, cache, q, torch.from_numpy(ip).to(DEV), cache.ctx_lens, scale, 300)
    ref, ref_lse = oracle.prefill_attn(oracle.bf16_bits(q), ip, oracle.bf16_bits(cache.k_pages),
                                       oracle.bf16_bits(cache.v_pages), cache.page_table_host, lens, scale)
    assert_parity(out, ref, "rising logits", scale_abs_by_magnitude=True)
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=3e-5, atol=3e-5)
    first = cache.v_pages[cache.page_table_host[1, 0], 0, 0]
    for h in range(Hq):
        assert torch.equal(out[300, h], first)


@pytest.mark.parametrize("jump_at", [640, 700, 710, 767])
def test_prefill_logit_jump_far_beyond_the_slack(jump_at):
    """Logits that jump by ~200 log2 units inside a block (at its first column, inside its first part, inside its
    second part, at its last column): the running reference must be raised before any exponential of the part is
    taken, or the probabilities overflow."""
    Hq, Hkv, d = 8, 2, 128
    L = 1100
    lens = np.array([L], dtype=np.int32)
    q_lens = np.array([400], dtype=np.int32)  # queries at positions 700..1099: some see the jump, some do not
    cache = wl.build_paged_cache(lens, Hkv, d, seed=120, device=DEV, poison=True)
    ip = np.array([0, 400], dtype=np.int32)
    q = torch.zeros((400, Hq, d), dtype=torch.bfloat16, device=DEV)
    q[:, :, 0] = 16.0
    q[:, :, 1:] = (0.05 * wl.random_bf16((400, Hq, d - 1), 121, DEV).float()).to(torch.bfloat16)
    a = np.where(np.arange(L) >= jump_at, 100.0, 0.0).astype(np.float32)  # 16 * 100 / sqrt(128) = 141 nats
    pages = torch.from_numpy(cache.page_table_host[0, np.arange(L) // 16].astype(np.int64)).to(DEV)
    slots = torch.from_numpy(np.arange(L) % 16).to(DEV)
    for h in range(Hkv):
        cache.k_pages[pages, h, slots, 0] = torch.from_numpy(a).to(DEV).to(torch.bfloat16)
    scale = 1.0 / math.sqrt(d)
    with ctx_for(cache, Hq) as ctx:
        out, lse = run_prefill(ctx, cache, q, torch.from_numpy(ip).to(DEV), cache.ctx_lens, scale, 400)
    ref, ref_lse = oracle.prefill_attn(oracle.bf16_bits(q), ip, oracle.bf16_bits(cache.k_pages),
                                       oracle.bf16_bits(cache.v_pages), cache.page_table_host, lens, scale)
    assert np.isfinite(out.float().cpu().numpy()).all()
    assert_parity(out, ref, f"jump at {jump_at}", scale_abs_by_magnitude=True)
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=3e-5, atol=3e-5)


def test_multi_token_append_bit_exact_then_prefill():
    Hq, Hkv, d = 32, 8, 128
    lens0 = np.array([30, 0, 16, 500, 7], dtype=np.int32)
    q_lens = np.array([5, 18, 16, 0, 260], dtype=np.int32)
    cache = wl.build_paged_cache(lens0, Hkv, d, seed=120, device=DEV, reserve_tokens=260)
    ip = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int32)
    total = int(ip[-1])
    kn, vn = wl.random_bf16((total, Hkv, d), 121, DEV), wl.random_bf16((total, Hkv, d), 122, DEV)
    q = wl.random_bf16((total, Hq, d), 123, DEV)
    k_host, v_host = oracle.bf16_bits(cache.k_pages).copy(), oracle.bf16_bits(cache.v_pages).copy()
    lens = lens0.copy()
    assert oracle.kv_append_tokens(oracle.bf16_bits(kn), oracle.bf16_bits(vn), ip, k_host, v_host,
                                   cache.page_table_host, lens) == 0
    scale = 1.0 / math.sqrt(d)
    ref, _ = oracle.prefill_attn(oracle.bf16_bits(q), ip, k_host, v_host, cache.page_table_host, lens, scale)
    ip_dev = torch.from_numpy(ip).to(DEV)
    with ctx_for(cache, Hq) as ctx:
        ctx.pd.pd_kv_append_tokens(ctx.h, kn, vn, ip_dev, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens,
                                   int(q_lens.max()))
        torch.cuda.synchronize()
        assert ctx.pd.pd_device_status(ctx.h)[0] == 0
        assert np.array_equal(cache.ctx_lens.cpu().numpy(), lens)
        assert np.array_equal(oracle.bf16_bits(cache.k_pages), k_host)
        assert np.array_equal(oracle.bf16_bits(cache.v_pages), v_host)
        out, _ = run_prefill(ctx, cache, q, ip_dev, cache.ctx_lens, scale, int(q_lens.max()))
    assert_parity(out, ref, "append then prefill", scale_abs_by_magnitude=True)


def test_prefill_paper_shaped_turn_sampled_rows():
    """Qwen3-8B geometry, 8 sequences with 4K-12K cached tokens and a new turn of 256-2048 tokens."""
    Hq, Hkv, d = 32, 8, 128
    rng = np.random.default_rng(130)
    q_lens = rng.integers(256, 2048, size=8, endpoint=True).astype(np.int32)
    lens = (rng.integers(4096, 12288, size=8) + q_lens).astype(np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=131, device=DEV)
    ip = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int32)
    q = wl.random_bf16((int(ip[-1]), Hq, d), 132, DEV)
    scale = 1.0 / math.sqrt(d)
    with ctx_for(cache, Hq) as ctx:
        out, lse = run_prefill(ctx, cache, q, torch.from_numpy(ip).to(DEV), cache.ctx_lens, scale, int(q_lens.max()))
    assert torch.isfinite(out.float()).all()
    # the oracle on sampled query rows: first, last and a few random ones of every sequence
    kp, vp = oracle.bf16_bits(cache.k_pages), oracle.bf16_bits(cache.v_pages)
    for b in range(8):
        rows = sorted(set([0, int(q_lens[b]) - 1] + rng.integers(0, q_lens[b], size=3).tolist()))
        for i in rows:
            vis = np.array([lens[b] - q_lens[b] + i + 1], np.int32)
            r = int(ip[b]) + i
            ref, ref_lse = oracle.decode_attn(oracle.bf16_bits(q[r:r + 1]), kp, vp, cache.page_table_host[b][None], vis, scale)
            assert_parity(out[r:r + 1], ref, f"seq {b} row {i}", scale_abs_by_magnitude=True)
            np.testing.assert_allclose(lse[r].cpu().numpy(), ref_lse[0], rtol=3e-5, atol=3e-5)
