"""The synthetic input recipe (workloads/): lengths in the stated ranges, reproducible by seed, page tables
that are valid scattered assignments over a pool of the stated size, poison where no token lives, a page
allocator that hands out each free page once, balanced sharding. CPU only."""
import math

import numpy as np
import pytest
import torch

import workloads as wl

P = wl.PAGE_SIZE


def test_context_lengths_follow_the_stated_distributions():
    for cfg, (lo, hi) in {0: (16, 256), 1: (2048, 16384), 3: (32768, 65536)}.items():
        lens = wl.context_lengths(cfg, batch=4000)
        assert lens.dtype == np.int32 and lens.min() >= lo and lens.max() <= hi
        assert lens.min() < lo + (hi - lo) * 0.01 and lens.max() > hi - (hi - lo) * 0.01  # both ends are reached
        assert abs(lens.mean() - (lo + hi) / 2) < 0.02 * (hi - lo)
    ln = wl.context_lengths(2, batch=20000)
    assert ln.min() >= 1024 and ln.max() <= 32768 and (ln == 32768).mean() < 0.05 and (ln == 1024).mean() < 0.01
    assert abs(np.median(ln) - 8192) < 0.03 * 8192  # lognormal with median 8192
    assert abs(np.std(np.log(ln[(ln > 1024) & (ln < 32768)])) - wl.LOGNORMAL_SIGMA) < 0.05
    mt = wl.context_lengths(4, batch=5000)
    assert mt.min() >= 256 and mt.max() <= 20 * 2048
    assert abs(mt.mean() - 10.5 * 1152) < 0.03 * 10.5 * 1152  # E[turns] * E[tokens per turn]
    # the configured batches, default seed = configuration index, reproducible
    for cfg, w in wl.WORKLOADS.items():
        a, b = wl.context_lengths(cfg), wl.context_lengths(cfg)
        assert len(a) == w.batch and np.array_equal(a, b)
        assert not np.array_equal(a, wl.context_lengths(cfg, seed=cfg + 1000))


def test_geometry_of_the_five_configurations():
    w = wl.WORKLOADS
    assert [(w[i].batch, w[i].num_q_heads, w[i].num_kv_heads, w[i].head_dim) for i in range(5)] == [
        (4, 8, 2, 64), (64, 32, 8, 128), (256, 32, 4, 128), (8, 32, 8, 128), (512, 32, 8, 128)]
    assert w[1].kv_bytes_per_token == 4096 and w[2].kv_bytes_per_token == 2048 and w[0].kv_bytes_per_token == 512
    assert w[1].sm_scale == float(np.float32(1 / math.sqrt(128))) and w[0].sm_scale == 0.125
    assert w[2].group == 8 and w[1].group == 4


@pytest.mark.parametrize("poison", [False, True])
def test_paged_cache_is_a_valid_scattered_assignment(poison):
    lens = np.array([0, 1, 15, 16, 17, 100, 333], dtype=np.int32)
    c = wl.build_paged_cache(lens, 2, 64, seed=5, reserve_tokens=20, poison=poison)
    pages_now = (lens + P - 1) // P
    pages_cap = (lens + 20 + P - 1) // P
    NP = c.k_pages.shape[0]
    assert NP == math.ceil(1.0625 * pages_cap.sum()) and c.k_pages.shape == (NP, 2, P, 64) == c.v_pages.shape
    assert c.k_pages.dtype == torch.bfloat16 and c.page_table.dtype == torch.int32
    assert np.array_equal(c.page_table.numpy(), c.page_table_host) and np.array_equal(c.ctx_lens.numpy(), lens)
    tbl = c.page_table_host
    used = np.concatenate([tbl[b, :(pages_now[b] if poison else pages_cap[b])] for b in range(len(lens))])
    assert used.min() >= 0 and used.max() < NP and len(np.unique(used)) == len(used)       # every page has one owner
    assert sorted(used.tolist() + c.free_pages) == list(range(NP)) if not poison else set(used) | set(c.free_pages) <= set(range(NP))
    assert not np.array_equal(np.sort(used), used)                                          # scattered, not in order
    for b in range(len(lens)):
        n = pages_now[b] if poison else pages_cap[b]
        assert np.all(tbl[b, n:] == -1)
    if poison:  # every slot that holds no token is NaN, every slot that holds one is finite
        k = c.k_pages.float().numpy()
        holds = np.zeros((NP, P), dtype=bool)
        for b, L in enumerate(lens):
            for i in range(pages_now[b]):
                holds[tbl[b, i], :min(P, L - i * P)] = True
        kk = np.moveaxis(k, 1, 2)  # [NP, P, Hkv, d]
        assert np.all(np.isnan(kk[~holds])) and np.all(np.isfinite(kk[holds]))
    # same seed, same cache; other seed, other values and other placement
    c2 = wl.build_paged_cache(lens, 2, 64, seed=5, reserve_tokens=20, poison=poison)
    assert torch.equal(c.page_table, c2.page_table) and torch.equal(c.v_pages.view(torch.int16), c2.v_pages.view(torch.int16))
    c3 = wl.build_paged_cache(lens, 2, 64, seed=6, reserve_tokens=20, poison=poison)
    assert not torch.equal(c.page_table, c3.page_table)
    flat = wl.build_paged_cache(lens, 2, 64, seed=5, permute=False)
    assert np.array_equal(flat.page_table_host[6, :21], np.arange(flat.page_table_host[6, 0], flat.page_table_host[6, 0] + 21))


def test_random_bf16_is_seeded_standard_normal():
    a, b = wl.random_bf16((64, 1000), 3), wl.random_bf16((64, 1000), 3)
    assert a.dtype == torch.bfloat16 and torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert not torch.equal(a, wl.random_bf16((64, 1000), 4))
    x = a.float()
    assert abs(float(x.mean())) < 0.02 and abs(float(x.std()) - 1.0) < 0.02


def test_page_allocator_hands_out_each_free_page_once():
    lens = np.array([16, 5, 31, 32], dtype=np.int32)
    c = wl.build_paged_cache(lens, 1, 64, seed=8, reserve_tokens=64, preassign_reserve=False)
    free0 = list(c.free_pages)
    alloc = wl.PageAllocator(c)
    cur = lens.copy()
    handed = []
    for step in range(40):
        need, logical, phys = alloc.assign(cur)
        # exactly the sequences whose next position opens a page that has no physical page yet
        assert sorted(need.tolist()) == [b for b in range(4) if cur[b] % P == 0]
        assert np.array_equal(logical, cur[need] // P)
        for b, lp, ph in zip(need, logical, phys):
            assert c.page_table_host[b, lp] == ph
        handed += phys.tolist()
        cur = cur + 1
    assert len(set(handed)) == len(handed) and set(handed) <= set(free0)
    assert set(c.free_pages) == set(free0) - set(handed)
    c.free_pages.clear()
    with pytest.raises(RuntimeError):
        alloc.assign(np.array([80, 1, 1, 1]))  # sequence 0 would open logical page 5, and nothing is left


def test_sharding_is_a_balanced_partition():
    rng = np.random.default_rng(9)
    lens = rng.integers(100, 40000, size=512)
    for world in (1, 2, 4, 8):
        parts = wl.shard_sequences(lens, world)
        assert len(parts) == world and sorted(np.concatenate(parts).tolist()) == list(range(512))
        loads = np.array([lens[p].sum() for p in parts])
        assert loads.max() - loads.min() <= lens.max()  # greedy longest-first: within one sequence of each other
