"""GPU parity of the FP8 (e4m3) KV path through the C ABI: whole-page quantiser and one-token append are
bit-exact against the oracle; attention over FP8 pages is within the decode tolerances (max abs 1e-2 scaled
by magnitude, per-row relative L2 5e-3) of the fp64 oracle evaluated on the SAME quantised cache."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from pd_testlib import Ctx, assert_parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
P = wl.PAGE_SIZE


def tokens_in_page(cache, lens):
    tip = np.zeros(cache.k_pages.shape[0], dtype=np.int32)
    for b, L in enumerate(lens):
        for i in range((int(L) + P - 1) // P):
            tip[cache.page_table_host[b, i]] = min(P, int(L) - i * P)
    return tip


def quantized_on_host(cache, lens, poison_codes=True):
    """The oracle's quantisation of a bf16 cache; unused slots and pages get NaN codes and NaN scales."""
    tip = tokens_in_page(cache, lens)
    k8, v8, sc = oracle.fp8_quantize_pages(oracle.bf16_bits(cache.k_pages), oracle.bf16_bits(cache.v_pages), tip)
    if poison_codes:
        for page, n in enumerate(tip):
            k8[page, :, n:] = 0x7F
            v8[page, :, n:] = 0xFF
            if n == 0:
                sc[page, :, :2] = np.nan
    return k8, v8, sc, tip


def to_dev(*arrays):
    return [torch.from_numpy(np.ascontiguousarray(a)).to(DEV) for a in arrays]


@pytest.mark.parametrize("Hkv,d", [(8, 128), (2, 64)])
def test_quantize_pages_bit_exact(Hkv, d):
    import paper_2609_35158_b200 as pd

    lens = np.array([0, 1, 15, 16, 17, 100, 333], dtype=np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=80, device=DEV, poison=True)  # NaN in every slot without a token
    cache.k_pages[cache.page_table_host[5, 0], 0, :, :] = 0  # an all-zero tile: scale 1
    cache.v_pages.mul_(0.03)
    tip = tokens_in_page(cache, lens)
    want_k, want_v, want_sc = oracle.fp8_quantize_pages(oracle.bf16_bits(cache.k_pages), oracle.bf16_bits(cache.v_pages), tip)
    NP = cache.k_pages.shape[0]
    k8 = torch.full((NP, Hkv, P, d), 0x55, dtype=torch.uint8, device=DEV)
    v8 = torch.full_like(k8, 0x55)
    sc = torch.full((NP, Hkv, 4), -1.0, dtype=torch.float32, device=DEV)
    with Ctx(Hkv, Hkv, d, len(lens), cache.page_table.shape[1], NP) as ctx:
        pd.pd_kv_quantize_pages(ctx.h, cache.k_pages, cache.v_pages, torch.from_numpy(tip).to(DEV), k8, v8, sc)
        torch.cuda.synchronize()
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), want_sc.view(np.uint32))
    assert np.array_equal(k8.cpu().numpy(), want_k)
    assert np.array_equal(v8.cpu().numpy(), want_v)
    assert want_sc[cache.page_table_host[5, 0], 0, 0] == 1.0


GEOMS = [(32, 8), (32, 4), (8, 8), (4, 2), (16, 2)]


@pytest.mark.parametrize("d", [128, 64])
@pytest.mark.parametrize("Hq,Hkv", GEOMS)
@pytest.mark.parametrize("split_pages", [0, 1, 3, 100000])
def test_fp8_attention_small_ragged_poisoned(Hq, Hkv, split_pages, d):
    import paper_2609_35158_b200 as pd

    lens = np.array([1, 15, 16, 17, 31, 33, 64, 300, 1000, 0, 2500], dtype=np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=81, device=DEV, poison=True)
    cache.v_pages.mul_(0.02)  # small values: a v_scale folded into fp16 probabilities would flush them
    k8, v8, sc, _ = quantized_on_host(cache, lens)
    q = wl.random_bf16((len(lens), Hq, d), 82, DEV)
    scale = d ** -0.5
    ref, ref_lse = oracle.fp8_decode_attn(oracle.bf16_bits(q), k8, v8, sc, cache.page_table_host, lens, scale)
    k8d, v8d, scd = to_dev(k8, v8, sc)
    out = torch.full((len(lens), Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((len(lens), Hq), float("nan"), dtype=torch.float32, device=DEV)
    with Ctx(Hq, Hkv, d, len(lens), cache.page_table.shape[1], cache.k_pages.shape[0]) as ctx:
        pd.pd_decode_attn_fp8(ctx.h, q, k8d, v8d, scd, cache.page_table, cache.ctx_lens, out, lse, sm_scale=scale,
                              split_pages=split_pages)
        torch.cuda.synchronize()
        assert pd.pd_device_status(ctx.h)[0] == 0
        again = torch.empty_like(out)
        pd.pd_decode_attn_fp8(ctx.h, q, k8d, v8d, scd, cache.page_table, cache.ctx_lens, again, sm_scale=scale,
                              split_pages=split_pages)
        torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), again.view(torch.int16))  # bit-reproducible
    # outputs here are ~0.02 in magnitude: compare relative to the output scale
    live = lens > 0
    assert_parity((out[torch.from_numpy(live).to(DEV)].float() * 50).to(torch.bfloat16), ref[live] * 50,
                  f"{Hq}/{Hkv} d={d} split {split_pages}", scale_abs_by_magnitude=True)
    got_lse = lse.cpu().numpy()
    assert np.all(np.isneginf(got_lse[~live])) and np.all(out[torch.from_numpy(~live).to(DEV)].float().cpu().numpy() == 0)
    np.testing.assert_allclose(got_lse[live], ref_lse[live], rtol=3e-5, atol=3e-5)


def test_fp8_attention_closed_form_and_dominant_key():
    import paper_2609_35158_b200 as pd

    Hq, Hkv, d, NP = 4, 1, 128, 3
    # two tokens: q.k = (1, 0) after scaling, V = +1 / -1 everywhere -> every output is tanh(1/2)
    k8 = np.zeros((NP, Hkv, P, d), dtype=np.uint8)
    v8 = np.zeros_like(k8)
    sc = np.zeros((NP, Hkv, 4), dtype=np.float32)
    k8[1, 0, 0, 0] = 0x38       # 1.0
    v8[1, 0, 0, :] = 0x40       # 2.0 * v_scale 0.5 = +1
    v8[1, 0, 1, :] = 0xC0       # -1
    sc[1, 0, 0], sc[1, 0, 1] = 2.0, 0.5   # K_0 = (2, 0, ...)
    q = torch.zeros((1, Hq, d), dtype=torch.bfloat16, device=DEV)
    q[:, :, 0] = 4.0            # scale 0.125: logits (1, 0)
    table = torch.tensor([[1, 2]], dtype=torch.int32, device=DEV)
    lens = torch.tensor([2], dtype=torch.int32, device=DEV)
    out = torch.empty_like(q)
    lse = torch.empty((1, Hq), dtype=torch.float32, device=DEV)
    k8d, v8d, scd = to_dev(k8, v8, sc)
    with Ctx(Hq, Hkv, d, 1, 2, NP) as ctx:
        pd.pd_decode_attn_fp8(ctx.h, q, k8d, v8d, scd, table, lens, out, lse, sm_scale=0.125)
        torch.cuda.synchronize()
        assert pd.pd_device_status(ctx.h)[0] == 0
    assert np.allclose(out.float().cpu().numpy(), np.tanh(0.5), atol=2e-3)
    assert np.allclose(lse.cpu().numpy(), np.log(1 + np.e), atol=1e-5)


def test_fp8_append_bit_exact_then_attend():
    import paper_2609_35158_b200 as pd

    Hq, Hkv, d = 32, 8, 128
    lens0 = np.array([0, 5, 15, 16, 31, 32, 100], dtype=np.int32)
    steps = 20
    cache = wl.build_paged_cache(lens0, Hkv, d, seed=83, device=DEV, reserve_tokens=steps)
    k8, v8, sc, _ = quantized_on_host(cache, lens0, poison_codes=False)
    lens = lens0.copy()
    k8d, v8d, scd = to_dev(k8, v8, sc)
    B = len(lens0)
    with Ctx(Hq, Hkv, d, B, cache.page_table.shape[1], cache.k_pages.shape[0]) as ctx:
        for t in range(steps):
            kn = wl.random_bf16((B, Hkv, d), 900 + 2 * t, DEV) * (1.0 + 0.2 * t)  # growing: later tokens meet the stored scale
            vn = wl.random_bf16((B, Hkv, d), 901 + 2 * t, DEV)
            n = oracle.fp8_kv_append(oracle.bf16_bits(kn), oracle.bf16_bits(vn), k8, v8, sc, cache.page_table_host, lens)
            assert n == B
            pd.pd_kv_append_fp8(ctx.h, kn, vn, k8d, v8d, scd, cache.page_table, cache.ctx_lens)
        torch.cuda.synchronize()
        assert pd.pd_device_status(ctx.h)[0] == 0
        assert np.array_equal(cache.ctx_lens.cpu().numpy(), lens)
        assert np.array_equal(scd.cpu().numpy().view(np.uint32), sc.view(np.uint32))
        assert np.array_equal(k8d.cpu().numpy(), k8) and np.array_equal(v8d.cpu().numpy(), v8)
        assert (np.abs(oracle.e4m3_to_f64(k8)) == 448.0).any()  # the growing keys saturated somewhere
        q = wl.random_bf16((B, Hq, d), 84, DEV)
        out = torch.empty((B, Hq, d), dtype=torch.bfloat16, device=DEV)
        pd.pd_decode_attn_fp8(ctx.h, q, k8d, v8d, scd, cache.page_table, cache.ctx_lens, out, sm_scale=d ** -0.5)
        torch.cuda.synchronize()
        assert pd.pd_device_status(ctx.h)[0] == 0
    ref, _ = oracle.fp8_decode_attn(oracle.bf16_bits(q), k8, v8, sc, cache.page_table_host, lens, d ** -0.5)
    assert_parity(out, ref, "after 20 FP8 appends", scale_abs_by_magnitude=True)


def test_fp8_append_errors_are_reported_and_skipped():
    import paper_2609_35158_b200 as pd

    lens = np.array([16, 5], dtype=np.int32)
    cache = wl.build_paged_cache(lens, 2, 128, seed=85, device=DEV, poison=True)  # next page of sequence 0 is -1
    NP = cache.k_pages.shape[0]
    k8 = torch.zeros((NP, 2, P, 128), dtype=torch.uint8, device=DEV)
    v8 = torch.zeros_like(k8)
    sc = torch.ones((NP, 2, 4), dtype=torch.float32, device=DEV)
    kn = wl.random_bf16((2, 2, 128), 86, DEV)
    with Ctx(2, 2, 128, 2, cache.page_table.shape[1], NP) as ctx:
        pd.pd_kv_append_fp8(ctx.h, kn, kn, k8, v8, sc, cache.page_table, cache.ctx_lens)
        code, seq, _ = pd.pd_device_status(ctx.h)
        assert code == pd.PD_ERR_DEVICE_FAULT and seq == 0
        assert cache.ctx_lens.cpu().tolist() == [16, 6]
        touched = (k8 != 0).nonzero()
        assert len(touched) and bool((touched[:, 0] == int(cache.page_table_host[1, 0])).all()) and bool((touched[:, 2] == 5).all())


def test_fp8_head_dim_64_on_the_small_config_geometry():
    """configs[0]'s geometry (16/2 heads, head_dim 64) through append + attention and through the one-call step:
    codes, scale records and lengths bit-exact against the oracle's append, attention against the FP8 oracle."""
    import paper_2609_35158_b200 as pd

    w = wl.WORKLOADS[0]
    assert w.head_dim == 64
    Hq, Hkv, d = w.num_q_heads, w.num_kv_heads, w.head_dim
    lens0 = wl.context_lengths(0).astype(np.int32)
    B, steps = len(lens0), 18  # crosses a page boundary for every sequence
    cache = wl.build_paged_cache(lens0, Hkv, d, seed=95, device=DEV, reserve_tokens=steps)  # codes of empty slots are poisoned below
    NP, MP = cache.k_pages.shape[0], cache.page_table.shape[1]
    k8, v8, sc, _ = quantized_on_host(cache, lens0)
    k8d, v8d, scd = to_dev(k8, v8, sc)
    lens = lens0.copy()
    scale = d ** -0.5
    with Ctx(Hq, Hkv, d, B, MP, NP) as ctx:
        for i in range(steps):
            q = wl.random_bf16((B, Hq, d), 960 + i, DEV)
            kn = wl.random_bf16((B, Hkv, d), 970 + i, DEV)
            vn = wl.random_bf16((B, Hkv, d), 980 + i, DEV)
            out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
            lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
            if i % 2:
                pd.pd_decode_step_fp8(ctx.h, q, kn, vn, k8d, v8d, scd, cache.page_table, cache.ctx_lens, out, lse, sm_scale=scale)
            else:
                pd.pd_kv_append_fp8(ctx.h, kn, vn, k8d, v8d, scd, cache.page_table, cache.ctx_lens)
                pd.pd_decode_attn_fp8(ctx.h, q, k8d, v8d, scd, cache.page_table, cache.ctx_lens, out, lse, sm_scale=scale)
            torch.cuda.synchronize()
            assert pd.pd_device_status(ctx.h)[0] == 0
            oracle.fp8_kv_append(oracle.bf16_bits(kn), oracle.bf16_bits(vn), k8, v8, sc, cache.page_table_host, lens)
            assert np.array_equal(cache.ctx_lens.cpu().numpy(), lens)
            if i in (0, 1, steps - 2, steps - 1):
                assert np.array_equal(k8d.cpu().numpy(), k8) and np.array_equal(v8d.cpu().numpy(), v8)
                assert np.array_equal(scd.cpu().numpy().view(np.uint32), sc.view(np.uint32))
                ref, ref_lse = oracle.fp8_decode_attn(oracle.bf16_bits(q), k8, v8, sc, cache.page_table_host, lens, scale)
                assert_parity(out, ref, f"head_dim 64 step {i}", scale_abs_by_magnitude=True)
                np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=3e-5, atol=3e-5)


def test_fp8_automatic_plan_is_one_equal_range_per_worker_on_small_totals():
    """With a fair share of at most 1024 pages per worker the automatic plan of the FP8 kernel is one equal range
    per worker: the same ranges, hence the same bits, as split_pages = fair share."""
    import paper_2609_35158_b200 as pd

    Hq, Hkv, d = 32, 8, 128
    rng = np.random.default_rng(77)
    lens = rng.integers(3000, 9000, size=24).astype(np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=97, device=DEV)
    k8, v8, sc, _ = quantized_on_host(cache, lens, poison_codes=False)
    k8d, v8d, scd = to_dev(k8, v8, sc)
    q = wl.random_bf16((len(lens), Hq, d), 98, DEV)
    outs, plans = [], []
    with Ctx(Hq, Hkv, d, len(lens), cache.page_table.shape[1], cache.k_pages.shape[0]) as ctx:
        pd.pd_decode_attn_fp8(ctx.h, q, k8d, v8d, scd, cache.page_table, cache.ctx_lens, torch.empty_like(q), sm_scale=0.088)
        torch.cuda.synchronize()
        auto = pd.pd_last_plan(ctx.h)
        fair = -(-auto["total_units"] // auto["num_workers"])
        assert fair <= 1024 and auto["num_ranges"] <= auto["num_workers"] and auto["pages_per_range"] == fair
        for split in (0, fair):
            out = torch.full_like(q, float("nan"))
            pd.pd_decode_attn_fp8(ctx.h, q, k8d, v8d, scd, cache.page_table, cache.ctx_lens, out, sm_scale=0.088, split_pages=split)
            torch.cuda.synchronize()
            assert pd.pd_device_status(ctx.h)[0] == 0
            outs.append(out)
            plans.append(pd.pd_last_plan(ctx.h))
    assert plans[0]["num_ranges"] == plans[1]["num_ranges"]
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))


@pytest.mark.parametrize("config", [1, 3])
def test_fp8_full_size_config_all_rows(config):
    """Configs 1 and 3 at full size in the automatic split mode: every (sequence, query head) row against the
    FP8 oracle, whose inputs are the ORACLE's own quantisation of the same bf16 cache (the GPU quantiser's codes
    and scale bits are checked against it on the way, page by page)."""
    import paper_2609_35158_b200 as pd

    w = wl.WORKLOADS[config]
    lens = wl.context_lengths(config)
    cache = wl.build_paged_cache(lens, w.num_kv_heads, w.head_dim, seed=config, device=DEV)
    NP = cache.k_pages.shape[0]
    B = len(lens)
    k8d = torch.empty((NP, w.num_kv_heads, P, w.head_dim), dtype=torch.uint8, device=DEV)
    v8d = torch.empty_like(k8d)
    scd = torch.empty((NP, w.num_kv_heads, 4), dtype=torch.float32, device=DEV)
    tip = tokens_in_page(cache, lens)
    q = wl.random_bf16((B, w.num_q_heads, w.head_dim), 87, DEV)
    out = torch.empty_like(q)
    lse = torch.empty((B, w.num_q_heads), dtype=torch.float32, device=DEV)
    with Ctx(w.num_q_heads, w.num_kv_heads, w.head_dim, B, cache.page_table.shape[1], NP) as ctx:
        pd.pd_kv_quantize_pages(ctx.h, cache.k_pages, cache.v_pages, torch.from_numpy(tip).to(DEV), k8d, v8d, scd)
        pd.pd_decode_attn_fp8(ctx.h, q, k8d, v8d, scd, cache.page_table, cache.ctx_lens, out, lse, sm_scale=w.sm_scale)
        torch.cuda.synchronize()
        assert pd.pd_device_status(ctx.h)[0] == 0
    worst = [0.0, 0.0]
    for c0 in range(0, B, 16):  # 16 sequences at a time keeps the host copies small
        ids = list(range(c0, min(B, c0 + 16)))
        pages = np.concatenate([cache.page_table_host[b, :(int(lens[b]) + P - 1) // P] for b in ids])
        idx = torch.from_numpy(pages.astype(np.int64)).to(DEV)
        kb = oracle.bf16_bits(cache.k_pages.index_select(0, idx))
        vb = oracle.bf16_bits(cache.v_pages.index_select(0, idx))
        k8, v8, sc = oracle.fp8_quantize_pages(kb, vb, tip[pages])
        assert np.array_equal(k8d.index_select(0, idx).cpu().numpy(), k8)
        assert np.array_equal(v8d.index_select(0, idx).cpu().numpy(), v8)
        assert np.array_equal(scd.index_select(0, idx).cpu().numpy().view(np.uint32), sc.view(np.uint32))
        table = np.full((len(ids), cache.page_table.shape[1]), -1, dtype=np.int32)
        cur = 0
        for i, b in enumerate(ids):
            n = (int(lens[b]) + P - 1) // P
            table[i, :n] = np.arange(cur, cur + n)
            cur += n
        ref, ref_lse = oracle.fp8_decode_attn(oracle.bf16_bits(q[c0:c0 + len(ids)]), k8, v8, sc, table, lens[ids], w.sm_scale)
        m_abs, m_rel = assert_parity(out[c0:c0 + len(ids)], ref, f"config {config} sequences {c0}..")
        np.testing.assert_allclose(lse[c0:c0 + len(ids)].cpu().numpy(), ref_lse, rtol=3e-5, atol=3e-5)
        worst = [max(worst[0], m_abs), max(worst[1], m_rel)]
    print(f"FP8 config {config}: worst max_abs {worst[0]:.2e} rel_l2 {worst[1]:.2e}")


@pytest.mark.parametrize("seed", range(12))
def test_fp8_random_case(seed):
    import math

    import paper_2609_35158_b200 as pd

    rng = np.random.default_rng(4000 + seed)
    d = 128 if seed % 3 else 64
    g = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2, 4, 8]))
    Hq = g * Hkv
    B = int(rng.integers(1, 13))
    kind = seed % 4
    if kind == 0:
        lens = rng.integers(0, 48, size=B)
    elif kind == 1:
        lens = rng.integers(1, 700, size=B)
    elif kind == 2:
        lens = np.where(rng.random(B) < 0.3, rng.integers(2000, 6000, size=B), rng.integers(1, 64, size=B))
    else:
        lens = 16 * rng.integers(1, 40, size=B) + rng.choice([-1, 0, 1], size=B)
    lens = np.maximum(lens, 0).astype(np.int32)
    split = int(rng.choice([0, 0, 1, 2, 5, 13, 64, 100000]))
    cache = wl.build_paged_cache(lens, Hkv, d, seed=4100 + seed, device=DEV, poison=True,
                                 max_pages_per_seq=int(max(1, (lens.max() + 15) // 16 + rng.integers(0, 5))))
    cache.k_pages.mul_(float(rng.choice([0.25, 1.0, 6.0])))
    cache.v_pages.mul_(float(rng.choice([0.01, 1.0, 30.0])))
    k8, v8, sc, _ = quantized_on_host(cache, lens)
    q = wl.random_bf16((B, Hq, d), 4200 + seed, DEV)
    scale = float(rng.choice([1.0 / math.sqrt(d), 0.05]))
    ref, ref_lse = oracle.fp8_decode_attn(oracle.bf16_bits(q), k8, v8, sc, cache.page_table_host, lens, scale)
    k8d, v8d, scd = to_dev(k8, v8, sc)
    out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    with Ctx(Hq, Hkv, d, B + int(rng.integers(0, 4)), cache.page_table.shape[1], cache.k_pages.shape[0]) as ctx:
        pd.pd_decode_attn_fp8(ctx.h, q, k8d, v8d, scd, cache.page_table, cache.ctx_lens, out, lse, sm_scale=scale,
                              split_pages=split)
        torch.cuda.synchronize()
        assert pd.pd_device_status(ctx.h)[0] == 0
    what = f"seed {seed}: B={B} {Hq}/{Hkv} split={split} lens={lens.tolist()}"
    live = lens > 0
    if live.any():
        # compare at unit output scale: divide by the RMS of the reference rows
        rms = float(np.sqrt(np.mean(ref[live] ** 2))) or 1.0
        assert_parity((out[torch.from_numpy(live).to(DEV)].float() / rms).to(torch.bfloat16), ref[live] / rms, what,
                      scale_abs_by_magnitude=True)
        np.testing.assert_allclose(lse.cpu().numpy()[live], ref_lse[live], rtol=3e-5, atol=3e-5, err_msg=what)
    assert np.all(np.isneginf(lse.cpu().numpy()[~live]))


def test_fp8_gather_scatter_bit_exact_and_attention_on_the_moved_cache():
    import paper_2609_35158_b200 as pd

    Hq, Hkv, d = 32, 8, 128
    lens = np.array([40, 1000, 17, 333, 2048], dtype=np.int32)
    B = len(lens)
    src = wl.build_paged_cache(lens, Hkv, d, seed=90, device=DEV)
    dst = wl.build_paged_cache(lens, Hkv, d, seed=91, device=DEV)  # other page ids, other contents
    k8, v8, sc, _ = quantized_on_host(src, lens, poison_codes=False)
    n_pages = (lens + P - 1) // P
    pb = np.zeros(B, dtype=np.int32)
    pb[1] = 3  # move only the pages from logical page 3 on for sequence 1 (as after a prefix hit)
    pe = n_pages.astype(np.int32)
    counts = pe - pb
    off = np.concatenate([[0], np.cumsum(counts)[:-1]]).astype(np.int64)
    total = int(counts.sum())
    want = oracle.fp8_kv_gather(k8, v8, sc, src.page_table_host, pb, pe, off, total)
    k8d, v8d, scd = to_dev(k8, v8, sc)
    d_pb, d_pe, d_off = to_dev(pb, pe, off)
    packed = torch.full((total, want.shape[1]), 0xAA, dtype=torch.uint8, device=DEV)
    NPd = dst.k_pages.shape[0]
    dk = torch.zeros((NPd, Hkv, P, d), dtype=torch.uint8, device=DEV)
    dv = torch.zeros_like(dk)
    ds = torch.zeros((NPd, Hkv, 4), dtype=torch.float32, device=DEV)
    q = wl.random_bf16((B, Hq, d), 92, DEV)
    with Ctx(Hq, Hkv, d, B, src.page_table.shape[1], src.k_pages.shape[0]) as cs, \
            Ctx(Hq, Hkv, d, B, dst.page_table.shape[1], NPd) as cd:
        pd.pd_kv_gather_fp8(cs.h, k8d, v8d, scd, src.page_table, d_pb, d_pe, d_off, packed)
        torch.cuda.synchronize()
        assert np.array_equal(packed.cpu().numpy(), want)
        # the receiver already holds the first three pages of sequence 1 (the shared prefix)
        want_k, want_v, want_s = dk.cpu().numpy(), dv.cpu().numpy(), ds.cpu().numpy()
        for lp in range(3):
            s_page, t_page = src.page_table_host[1, lp], dst.page_table_host[1, lp]
            want_k[t_page], want_v[t_page], want_s[t_page] = k8[s_page], v8[s_page], sc[s_page]
        dk.copy_(torch.from_numpy(want_k)); dv.copy_(torch.from_numpy(want_v)); ds.copy_(torch.from_numpy(want_s))
        oracle.fp8_kv_scatter(want, off, want_k, want_v, want_s, dst.page_table_host, pb, pe)
        pd.pd_kv_scatter_fp8(cd.h, packed, d_off, dk, dv, ds, dst.page_table, d_pb, d_pe)
        torch.cuda.synchronize()
        assert pd.pd_device_status(cs.h)[0] == 0 and pd.pd_device_status(cd.h)[0] == 0
        assert np.array_equal(dk.cpu().numpy(), want_k) and np.array_equal(dv.cpu().numpy(), want_v)
        assert np.array_equal(ds.cpu().numpy().view(np.uint32), want_s.view(np.uint32))
        out_s = torch.empty((B, Hq, d), dtype=torch.bfloat16, device=DEV)
        out_d = torch.empty_like(out_s)
        pd.pd_decode_attn_fp8(cs.h, q, k8d, v8d, scd, src.page_table, src.ctx_lens, out_s, sm_scale=d ** -0.5, split_pages=7)
        pd.pd_decode_attn_fp8(cd.h, q, dk, dv, ds, dst.page_table, dst.ctx_lens, out_d, sm_scale=d ** -0.5, split_pages=7)
        torch.cuda.synchronize()
        assert torch.equal(out_s.view(torch.int16), out_d.view(torch.int16))


@pytest.mark.parametrize("Hq,Hkv", [(32, 8), (8, 8), (16, 2)])
@pytest.mark.parametrize("split_pages", [0, 1, 100000])
def test_fp8_fused_step_is_bit_identical_to_append_plus_attention(Hq, Hkv, split_pages):
    """pd_decode_step_fp8 against pd_kv_append_fp8 + pd_decode_attn_fp8 over several steps: codes, scale
    records, lengths, output and LSE bit for bit; and against the oracle at the end."""
    import paper_2609_35158_b200 as pd

    d, steps = 128, 6
    lens0 = np.array([0, 1, 14, 15, 16, 17, 31, 32, 33, 100, 255, 256, 700], dtype=np.int32)
    B = len(lens0)
    cache = wl.build_paged_cache(lens0, Hkv, d, seed=95, device=DEV, reserve_tokens=steps)
    k8, v8, sc, _ = quantized_on_host(cache, lens0, poison_codes=True)
    sc[np.isnan(sc)] = 7.0  # pages that are not in use yet: any finite garbage
    a = to_dev(k8, v8, sc)
    b = to_dev(k8, v8, sc)
    lens_a, lens_b = cache.ctx_lens.clone(), cache.ctx_lens.clone()
    lens_h = lens0.copy()  # the oracle's own copy of the cache, appended to on the host
    scale = d ** -0.5
    with Ctx(Hq, Hkv, d, B, cache.page_table.shape[1], cache.k_pages.shape[0]) as ctx:
        for t in range(steps):
            q = wl.random_bf16((B, Hq, d), 960 + 3 * t, DEV)
            kn = wl.random_bf16((B, Hkv, d), 961 + 3 * t, DEV) * (1.0 + 0.5 * t)
            vn = wl.random_bf16((B, Hkv, d), 962 + 3 * t, DEV)
            assert oracle.fp8_kv_append(oracle.bf16_bits(kn), oracle.bf16_bits(vn), k8, v8, sc, cache.page_table_host, lens_h) == B
            out_a = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
            lse_a = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
            out_b, lse_b = out_a.clone(), lse_a.clone()
            pd.pd_kv_append_fp8(ctx.h, kn, vn, a[0], a[1], a[2], cache.page_table, lens_a)
            pd.pd_decode_attn_fp8(ctx.h, q, a[0], a[1], a[2], cache.page_table, lens_a, out_a, lse_a, sm_scale=scale,
                                  split_pages=split_pages)
            pd.pd_decode_step_fp8(ctx.h, q, kn, vn, b[0], b[1], b[2], cache.page_table, lens_b, out_b, lse_b,
                                  sm_scale=scale, split_pages=split_pages)
            torch.cuda.synchronize()
            assert pd.pd_device_status(ctx.h)[0] == 0
            what = f"step {t}"
            assert lens_b.cpu().tolist() == (lens0 + t + 1).tolist() and torch.equal(lens_a, lens_b), what
            assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]), what + ": codes"
            assert torch.equal(a[2].view(torch.int32), b[2].view(torch.int32)), what + ": scale records"
            assert torch.equal(out_a.view(torch.int16), out_b.view(torch.int16)), what + ": output"
            assert torch.equal(lse_a.view(torch.int32), lse_b.view(torch.int32)), what + ": lse"
    assert np.array_equal(b[0].cpu().numpy(), k8) and np.array_equal(b[1].cpu().numpy(), v8)
    assert np.array_equal(b[2].cpu().numpy().view(np.uint32), sc.view(np.uint32)) and np.array_equal(lens_h, lens0 + steps)
    ref, _ = oracle.fp8_decode_attn(oracle.bf16_bits(q), k8, v8, sc, cache.page_table_host, lens_h, scale)
    assert_parity(out_b, ref, "fused FP8 step", scale_abs_by_magnitude=True)
