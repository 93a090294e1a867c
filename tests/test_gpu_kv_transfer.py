"""GPU parity of the KV page gather / scatter kernels (bit-exact) against the CPU oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
import workloads as wl
from pd_testlib import ctx_for

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def ranges_for(lens, new_tokens, P=16):
    """Logical page range that holds the last ``new_tokens[b]`` tokens of every sequence."""
    lens, new_tokens = np.asarray(lens), np.asarray(new_tokens)
    pb = ((lens - new_tokens) // P).astype(np.int32)
    pe = ((lens + P - 1) // P).astype(np.int32)
    cnt = np.maximum(pe - pb, 0)
    off = np.concatenate([[0], np.cumsum(cnt)[:-1]]).astype(np.int64)
    return pb, pe, off, int(cnt.sum())


@pytest.mark.parametrize("Hkv,d", [(2, 64), (8, 128), (4, 128)])
def test_gather_and_scatter_bit_exact(Hkv, d):
    lens = np.array([100, 16, 33, 0, 250, 1, 4000], dtype=np.int32)
    new = np.array([60, 16, 1, 0, 250, 1, 1500], dtype=np.int32)
    B = len(lens)
    src = wl.build_paged_cache(lens, Hkv, d, seed=70, device=DEV, poison=True)
    dst = wl.build_paged_cache(lens, Hkv, d, seed=71, device=DEV)
    pb, pe, off, total = ranges_for(lens, new)
    dev = lambda a: torch.from_numpy(a).to(DEV)
    packed = torch.full((total, 2, Hkv, 16, d), 1.0, dtype=torch.bfloat16, device=DEV)
    ref_packed, rc = oracle.kv_gather(oracle.bf16_bits(src.k_pages), oracle.bf16_bits(src.v_pages),
                                      src.page_table_host, pb, pe, off, total)
    assert rc == 0
    dk, dv = oracle.bf16_bits(dst.k_pages).copy(), oracle.bf16_bits(dst.v_pages).copy()
    assert oracle.kv_scatter(ref_packed, off, dk, dv, dst.page_table_host, pb, pe) == 0
    with ctx_for(src, Hkv) as ctx:
        ctx.pd.pd_kv_gather(ctx.h, src.k_pages, src.v_pages, src.page_table, dev(pb), dev(pe), dev(off), packed)
        torch.cuda.synchronize()
        assert np.array_equal(oracle.bf16_bits(packed), ref_packed)
    with ctx_for(dst, Hkv) as ctx:
        ctx.pd.pd_kv_scatter(ctx.h, packed, dev(off), dst.k_pages, dst.v_pages, dst.page_table, dev(pb), dev(pe))
        torch.cuda.synchronize()
        assert ctx.pd.pd_device_status(ctx.h)[0] == 0
        assert np.array_equal(oracle.bf16_bits(dst.k_pages), dk)   # every byte of both destination pools
        assert np.array_equal(oracle.bf16_bits(dst.v_pages), dv)


def test_transferred_cache_gives_bit_identical_attention():
    """Prefill side -> gather -> scatter into a differently placed decode-side cache -> same attention bits."""
    Hq, Hkv, d = 32, 8, 128
    lens = np.array([700, 90, 2049], dtype=np.int32)
    src = wl.build_paged_cache(lens, Hkv, d, seed=72, device=DEV)
    dst = wl.build_paged_cache(lens, Hkv, d, seed=73, device=DEV)
    pb, pe, off, total = ranges_for(lens, lens)  # whole sequences
    dev = lambda a: torch.from_numpy(a).to(DEV)
    packed = torch.empty((total, 2, Hkv, 16, d), dtype=torch.bfloat16, device=DEV)
    q = wl.random_bf16((3, Hq, d), 74, DEV)
    outs = []
    with ctx_for(src, Hq) as ctx:
        ctx.pd.pd_kv_gather(ctx.h, src.k_pages, src.v_pages, src.page_table, dev(pb), dev(pe), dev(off), packed)
        o = torch.empty_like(q)
        ctx.pd.pd_decode_attn(ctx.h, q, src.k_pages, src.v_pages, src.page_table, src.ctx_lens, o,
                              sm_scale=1 / math.sqrt(d))
        outs.append(o)
    with ctx_for(dst, Hq) as ctx:
        ctx.pd.pd_kv_scatter(ctx.h, packed, dev(off), dst.k_pages, dst.v_pages, dst.page_table, dev(pb), dev(pe))
        o = torch.empty_like(q)
        ctx.pd.pd_decode_attn(ctx.h, q, dst.k_pages, dst.v_pages, dst.page_table, dst.ctx_lens, o,
                              sm_scale=1 / math.sqrt(d))
        outs.append(o)
    torch.cuda.synchronize()
    assert torch.equal(outs[0], outs[1])


def test_transfer_reports_bad_page_id():
    lens = np.array([64, 64], dtype=np.int32)
    src = wl.build_paged_cache(lens, 2, 64, seed=75, device=DEV)
    src.page_table[1, 2] = -7
    pb, pe, off, total = ranges_for(lens, lens)
    dev = lambda a: torch.from_numpy(a).to(DEV)
    packed = torch.zeros((total, 2, 2, 16, 64), dtype=torch.bfloat16, device=DEV)
    with ctx_for(src, 2) as ctx:
        ctx.pd.pd_kv_gather(ctx.h, src.k_pages, src.v_pages, src.page_table, dev(pb), dev(pe), dev(off), packed)
        code, seq, detail = ctx.pd.pd_device_status(ctx.h)
        assert code == ctx.pd.PD_ERR_DEVICE_FAULT and seq == 1 and detail == -7
        assert torch.all(packed[off[1] + 2] == 0)                      # the skipped page was not written
        assert torch.equal(packed[0, 0], src.k_pages[src.page_table_host[0, 0]])
