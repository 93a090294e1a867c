"""CPU oracle (fp64, plain C) for paged GQA decode attention and KV append.

TEST INFRASTRUCTURE ONLY: importable from ``tests/``, from the smoke check and
from the benchmark's CPU-baseline leg. The CUDA library never imports it and it
never imports the CUDA library.

The arithmetic lives in ``pd_oracle.c`` (see its header for the definition and
the pins); this module compiles it with gcc, loads it through ctypes and
marshals NumPy arrays. bf16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pd_oracle.c")
_SRC_FP8 = os.path.join(_HERE, "pd_oracle_fp8.c")
_LIB = os.path.join(_HERE, "libpd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``pd_oracle.c`` and ``pd_oracle_fp8.c`` into ``libpd_oracle.so`` (gcc, no fast-math)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_FP8))
    if force or stale:
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-pthread", _SRC, _SRC_FP8, "-o", tmp, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        p = ctypes.c_void_p
        i = ctypes.c_int
        lib.pd_oracle_decode_attn.argtypes = [p, p, p, p, p, p, p, i, i, i, i, i, i, ctypes.c_float, p, p, i]
        lib.pd_oracle_decode_attn.restype = i
        lib.pd_oracle_lse_merge.argtypes = [p, p, i, i, p, p]
        lib.pd_oracle_lse_merge.restype = i
        lib.pd_oracle_kv_append.argtypes = [p, p, p, p, p, p, i, i, i, i, i, ctypes.c_int64, i]
        lib.pd_oracle_kv_append.restype = i
        lib.pd_oracle_prefill_attn.argtypes = [p, p, p, p, p, p, i, i, i, i, i, i, ctypes.c_float, p, p, i]
        lib.pd_oracle_prefill_attn.restype = i
        lib.pd_oracle_kv_append_tokens.argtypes = [p, p, p, p, p, p, p, i, i, i, i, i, ctypes.c_int64]
        lib.pd_oracle_kv_append_tokens.restype = i
        lib.pd_oracle_kv_gather.argtypes = [p, p, p, p, p, p, p, i, i, i, i, i, ctypes.c_int64]
        lib.pd_oracle_kv_gather.restype = i
        lib.pd_oracle_kv_scatter.argtypes = [p, p, p, p, p, p, p, i, i, i, i, i, ctypes.c_int64]
        lib.pd_oracle_kv_scatter.restype = i
        lib.pd_oracle_e4m3_to_f64.argtypes = [ctypes.c_uint8]
        lib.pd_oracle_e4m3_to_f64.restype = ctypes.c_double
        lib.pd_oracle_f32_to_e4m3.argtypes = [ctypes.c_float]
        lib.pd_oracle_f32_to_e4m3.restype = ctypes.c_uint8
        lib.pd_oracle_fp8_quantize_pages.argtypes = [p, p, p, ctypes.c_int64, i, i, i, p, p, p]
        lib.pd_oracle_fp8_quantize_pages.restype = i
        lib.pd_oracle_fp8_kv_append.argtypes = [p, p, p, p, p, p, p, i, i, i, i, i, ctypes.c_int64, i]
        lib.pd_oracle_fp8_kv_append.restype = i
        lib.pd_oracle_fp8_decode_attn.argtypes = [p, p, p, p, p, p, i, i, i, i, i, i, ctypes.c_float, i, p, p]
        lib.pd_oracle_fp8_decode_attn.restype = i
        _lib = lib
    return _lib


def bf16_bits(t) -> np.ndarray:
    """Bit patterns (uint16, C-contiguous) of a bf16 torch tensor on any device."""
    import torch

    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp64."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16
    return u.view(np.float32).astype(np.float64)


def _c(a: np.ndarray, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def decode_attn(q, k_pages, v_pages, page_table, ctx_lens, sm_scale, *, t_begin=None, t_end=None,
                nthreads: int | None = None):
    """softmax(sm_scale * q K^T) V per (sequence, query head) over a paged cache.

    q: uint16 [B, Hq, d]; k_pages/v_pages: uint16 [NP, Hkv, P, d];
    page_table: int32 [B, MP]; ctx_lens: int32 [B]. Optional ``t_begin`` /
    ``t_end`` (int32 [B]) restrict every sequence to a token range (used to form
    split partials). Returns (out fp64 [B, Hq, d], lse fp64 [B, Hq]).
    """
    lib = _load()
    q = _c(q, np.uint16)
    k_pages = _c(k_pages, np.uint16)
    v_pages = _c(v_pages, np.uint16)
    page_table = _c(page_table, np.int32)
    ctx_lens = _c(ctx_lens, np.int32)
    B, Hq, d = q.shape
    NP, Hkv, P, d2 = k_pages.shape
    assert d2 == d and v_pages.shape == k_pages.shape
    assert page_table.ndim == 2 and page_table.shape[0] >= B and ctx_lens.shape[0] >= B
    MP = page_table.shape[1]
    # every page the definition will touch must exist
    for b in range(B):
        lo = 0 if t_begin is None else int(t_begin[b])
        hi = int(ctx_lens[b]) if t_end is None else int(t_end[b])
        if hi > lo:
            assert hi <= MP * P
            used = page_table[b, lo // P:(hi + P - 1) // P]
            assert used.min() >= 0 and used.max() < NP, "page id out of range"
    tb = None if t_begin is None else _c(t_begin, np.int32)
    te = None if t_end is None else _c(t_end, np.int32)
    out = np.empty((B, Hq, d), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    if nthreads is None:
        nthreads = os.cpu_count() or 1
    rc = lib.pd_oracle_decode_attn(
        q.ctypes.data, k_pages.ctypes.data, v_pages.ctypes.data, page_table.ctypes.data,
        ctx_lens.ctypes.data, None if tb is None else tb.ctypes.data,
        None if te is None else te.ctypes.data, B, Hq, Hkv, d, P, MP,
        ctypes.c_float(np.float32(sm_scale)), out.ctypes.data, lse.ctypes.data, int(nthreads))
    if rc != 0:
        raise RuntimeError(f"pd_oracle_decode_attn failed ({rc})")
    return out, lse


def lse_merge(o_parts, lse_parts):
    """Merge partial results of one row. o_parts fp64 [n, d], lse_parts fp64 [n]."""
    lib = _load()
    o_parts = _c(o_parts, np.float64)
    lse_parts = _c(lse_parts, np.float64)
    n, d = o_parts.shape
    out = np.empty(d, dtype=np.float64)
    lse = np.empty(1, dtype=np.float64)
    rc = lib.pd_oracle_lse_merge(o_parts.ctypes.data, lse_parts.ctypes.data, n, d, out.ctypes.data,
                                 lse.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"pd_oracle_lse_merge failed ({rc})")
    return out, float(lse[0])


def kv_append(k_new, v_new, k_pages, v_pages, page_table, ctx_lens, *, advance: bool = True) -> int:
    """In-place one-token append on host mirrors of the pools (uint16) and ctx_lens (int32)."""
    lib = _load()
    for a, dt in ((k_pages, np.uint16), (v_pages, np.uint16), (ctx_lens, np.int32)):
        assert isinstance(a, np.ndarray) and a.dtype == dt and a.flags.c_contiguous and a.flags.writeable
    k_new = _c(k_new, np.uint16)
    v_new = _c(v_new, np.uint16)
    page_table = _c(page_table, np.int32)
    B, Hkv, d = k_new.shape
    NP, Hkv2, P, d2 = k_pages.shape
    assert (Hkv2, d2) == (Hkv, d) and v_pages.shape == k_pages.shape and v_new.shape == k_new.shape
    return lib.pd_oracle_kv_append(
        k_new.ctypes.data, v_new.ctypes.data, k_pages.ctypes.data, v_pages.ctypes.data,
        page_table.ctypes.data, ctx_lens.ctypes.data, B, Hkv, d, P, page_table.shape[1], NP,
        1 if advance else 0)


def kv_gather(k_pages, v_pages, page_table, page_begin, page_end, dst_page_offset, total_pages: int):
    """Pack logical pages [page_begin[b], page_end[b]) of every sequence into one buffer.

    Returns uint16 [total_pages, 2, Hkv, P, d]; packed page dst_page_offset[b] + i holds the K block then
    the V block of logical page page_begin[b] + i."""
    lib = _load()
    k_pages, v_pages = _c(k_pages, np.uint16), _c(v_pages, np.uint16)
    page_table = _c(page_table, np.int32)
    pb, pe = _c(page_begin, np.int32), _c(page_end, np.int32)
    off = _c(dst_page_offset, np.int64)
    NP, Hkv, P, d = k_pages.shape
    packed = np.zeros((total_pages, 2, Hkv, P, d), dtype=np.uint16)
    rc = lib.pd_oracle_kv_gather(k_pages.ctypes.data, v_pages.ctypes.data, page_table.ctypes.data, pb.ctypes.data,
                                 pe.ctypes.data, off.ctypes.data, packed.ctypes.data, len(pb), Hkv, d, P,
                                 page_table.shape[1], NP)
    return packed, rc


def kv_scatter(packed, src_page_offset, k_pages, v_pages, page_table, page_begin, page_end) -> int:
    """In-place unpack of a packed buffer into the pages the table names (host mirrors, uint16)."""
    lib = _load()
    for a in (k_pages, v_pages):
        assert isinstance(a, np.ndarray) and a.dtype == np.uint16 and a.flags.c_contiguous and a.flags.writeable
    packed = _c(packed, np.uint16)
    page_table = _c(page_table, np.int32)
    pb, pe = _c(page_begin, np.int32), _c(page_end, np.int32)
    off = _c(src_page_offset, np.int64)
    NP, Hkv, P, d = k_pages.shape
    return lib.pd_oracle_kv_scatter(packed.ctypes.data, off.ctypes.data, k_pages.ctypes.data, v_pages.ctypes.data,
                                    page_table.ctypes.data, pb.ctypes.data, pe.ctypes.data, len(pb), Hkv, d, P,
                                    page_table.shape[1], NP)


def prefill_attn(q, q_indptr, k_pages, v_pages, page_table, ctx_lens, sm_scale, *, nthreads: int | None = None):
    """Causal attention of packed new-token queries over prefix + themselves.

    q: uint16 [total_q, Hq, d]; q_indptr: int32 [B+1]; the cache already holds the new tokens and
    ctx_lens counts them. Returns (out fp64 [total_q, Hq, d], lse fp64 [total_q, Hq])."""
    lib = _load()
    q = _c(q, np.uint16)
    ip = _c(q_indptr, np.int32)
    k_pages, v_pages = _c(k_pages, np.uint16), _c(v_pages, np.uint16)
    page_table, ctx_lens = _c(page_table, np.int32), _c(ctx_lens, np.int32)
    total_q, Hq, d = q.shape
    NP, Hkv, P, _ = k_pages.shape
    B = len(ip) - 1
    assert ip[0] == 0 and ip[-1] == total_q and np.all(np.diff(ip) >= 0)
    for b in range(B):
        assert ctx_lens[b] >= ip[b + 1] - ip[b], "the cache must already hold the new tokens"
        if ctx_lens[b] > 0:
            used = page_table[b, :(int(ctx_lens[b]) + P - 1) // P]
            assert used.min() >= 0 and used.max() < NP, "page id out of range"
    out = np.empty((total_q, Hq, d), dtype=np.float64)
    lse = np.empty((total_q, Hq), dtype=np.float64)
    if nthreads is None:
        nthreads = os.cpu_count() or 1
    rc = lib.pd_oracle_prefill_attn(q.ctypes.data, ip.ctypes.data, k_pages.ctypes.data, v_pages.ctypes.data,
                                    page_table.ctypes.data, ctx_lens.ctypes.data, B, Hq, Hkv, d, P,
                                    page_table.shape[1], ctypes.c_float(np.float32(sm_scale)), out.ctypes.data,
                                    lse.ctypes.data, int(nthreads))
    if rc != 0:
        raise RuntimeError(f"pd_oracle_prefill_attn failed ({rc})")
    return out, lse


def kv_append_tokens(k_new, v_new, q_indptr, k_pages, v_pages, page_table, ctx_lens) -> int:
    """In-place multi-token append on host mirrors; ctx_lens grows by each sequence's token count."""
    lib = _load()
    for a, dt in ((k_pages, np.uint16), (v_pages, np.uint16), (ctx_lens, np.int32)):
        assert isinstance(a, np.ndarray) and a.dtype == dt and a.flags.c_contiguous and a.flags.writeable
    k_new, v_new = _c(k_new, np.uint16), _c(v_new, np.uint16)
    ip = _c(q_indptr, np.int32)
    page_table = _c(page_table, np.int32)
    NP, Hkv, P, d = k_pages.shape
    return lib.pd_oracle_kv_append_tokens(k_new.ctypes.data, v_new.ctypes.data, ip.ctypes.data, k_pages.ctypes.data,
                                          v_pages.ctypes.data, page_table.ctypes.data, ctx_lens.ctypes.data,
                                          len(ip) - 1, Hkv, d, P, page_table.shape[1], NP)


# ---------------------------------------------------------------- FP8 (e4m3) pages, see pd_oracle_fp8.c

def e4m3_to_f64(codes) -> np.ndarray:
    """Exact values of OCP FP8 E4M3 codes (uint8 array)."""
    lib = _load()
    codes = np.asarray(codes, dtype=np.uint8)
    table = np.array([lib.pd_oracle_e4m3_to_f64(c) for c in range(256)], dtype=np.float64)
    return table[codes]


def f32_to_e4m3(x) -> np.ndarray:
    """fp32 -> e4m3 codes, round to nearest even, saturating at +-448 (element by element through the C routine)."""
    lib = _load()
    x = np.asarray(x, dtype=np.float32)
    flat = np.array([lib.pd_oracle_f32_to_e4m3(ctypes.c_float(v)) for v in x.ravel()], dtype=np.uint8)
    return flat.reshape(x.shape)


def fp8_quantize_pages(k_pages, v_pages, tokens_in_page):
    """bf16 pools (uint16 bits) -> (k8, v8 uint8 pools, scales fp32 [NP, Hkv, 4]) with one amax scale per tile."""
    lib = _load()
    k_pages = _c(k_pages, np.uint16)
    v_pages = _c(v_pages, np.uint16)
    NP, Hkv, P, d = k_pages.shape
    tip = _c(tokens_in_page, np.int32)
    assert tip.shape == (NP,)
    k8 = np.empty(k_pages.shape, dtype=np.uint8)
    v8 = np.empty(k_pages.shape, dtype=np.uint8)
    scales = np.empty((NP, Hkv, 4), dtype=np.float32)
    rc = lib.pd_oracle_fp8_quantize_pages(k_pages.ctypes.data, v_pages.ctypes.data, tip.ctypes.data, NP, Hkv, P, d,
                                          k8.ctypes.data, v8.ctypes.data, scales.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"pd_oracle_fp8_quantize_pages failed ({rc})")
    return k8, v8, scales


def fp8_kv_append(k_new, v_new, k8, v8, scales, page_table, ctx_lens, *, advance: bool = True) -> int:
    """One-token append into FP8 pools, in place (k8, v8, scales, ctx_lens are modified)."""
    lib = _load()
    k_new = _c(k_new, np.uint16)
    v_new = _c(v_new, np.uint16)
    for a, dt in ((k8, np.uint8), (v8, np.uint8), (scales, np.float32), (ctx_lens, np.int32)):
        assert a.dtype == dt and a.flags.c_contiguous
    page_table = _c(page_table, np.int32)
    B, Hkv, d = k_new.shape
    NP, Hkv2, P, d2 = k8.shape
    assert (Hkv2, d2) == (Hkv, d)
    return lib.pd_oracle_fp8_kv_append(k_new.ctypes.data, v_new.ctypes.data, k8.ctypes.data, v8.ctypes.data,
                                       scales.ctypes.data, page_table.ctypes.data, ctx_lens.ctypes.data, B, Hkv, d, P,
                                       page_table.shape[1], NP, int(advance))


def fp8_decode_attn(q, k8, v8, scales, page_table, ctx_lens, sm_scale, *, nthreads: int | None = None):
    """Attention over FP8 pages with per-(page, KV head) scales. Returns (out fp64 [B, Hq, d], lse fp64 [B, Hq])."""
    lib = _load()
    q = _c(q, np.uint16)
    k8 = _c(k8, np.uint8)
    v8 = _c(v8, np.uint8)
    scales = _c(scales, np.float32)
    page_table = _c(page_table, np.int32)
    ctx_lens = _c(ctx_lens, np.int32)
    B, Hq, d = q.shape
    NP, Hkv, P, d2 = k8.shape
    assert d2 == d and v8.shape == k8.shape and scales.shape == (NP, Hkv, 4)
    MP = page_table.shape[1]
    for b in range(B):
        n = (int(ctx_lens[b]) + P - 1) // P
        if n:
            used = page_table[b, :n]
            assert used.min() >= 0 and used.max() < NP, "page id out of range"
    out = np.empty((B, Hq, d), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    rc = lib.pd_oracle_fp8_decode_attn(q.ctypes.data, k8.ctypes.data, v8.ctypes.data, scales.ctypes.data,
                                       page_table.ctypes.data, ctx_lens.ctypes.data, B, Hq, Hkv, d, P, MP,
                                       ctypes.c_float(np.float32(sm_scale)), int(nthreads or os.cpu_count() or 1),
                                       out.ctypes.data, lse.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"pd_oracle_fp8_decode_attn failed ({rc})")
    return out, lse


def fp8_kv_gather(k8, v8, scales, page_table, page_begin, page_end, dst_page_offset, total_pages: int) -> np.ndarray:
    """Packs logical pages [page_begin[b], page_end[b]) of every sequence: packed page i is the K block, the V
    block and the Hkv scale records (as bytes) of one pool page. Returns uint8 [total_pages, 2*Hkv*P*d + Hkv*16]."""
    k8 = _c(k8, np.uint8)
    v8 = _c(v8, np.uint8)
    scales = _c(scales, np.float32)
    NP, Hkv, P, d = k8.shape
    block = Hkv * P * d
    packed = np.zeros((total_pages, 2 * block + Hkv * 16), dtype=np.uint8)
    for b in range(len(page_begin)):
        for i, lp in enumerate(range(int(page_begin[b]), int(page_end[b]))):
            page = int(page_table[b, lp])
            row = packed[int(dst_page_offset[b]) + i]
            row[:block] = k8[page].reshape(-1)
            row[block:2 * block] = v8[page].reshape(-1)
            row[2 * block:] = scales[page].reshape(-1).view(np.uint8)
    return packed


def fp8_kv_scatter(packed, src_page_offset, k8, v8, scales, page_table, page_begin, page_end) -> None:
    """The inverse of ``fp8_kv_gather``, in place on k8, v8 and scales."""
    NP, Hkv, P, d = k8.shape
    block = Hkv * P * d
    for b in range(len(page_begin)):
        for i, lp in enumerate(range(int(page_begin[b]), int(page_end[b]))):
            page = int(page_table[b, lp])
            row = packed[int(src_page_offset[b]) + i]
            k8[page] = row[:block].reshape(Hkv, P, d)
            v8[page] = row[block:2 * block].reshape(Hkv, P, d)
            scales[page] = row[2 * block:].view(np.float32).reshape(Hkv, 4)
