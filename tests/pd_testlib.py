"""Helpers shared by the GPU parity tests: run the CUDA path, run the oracle, compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import workloads as wl

MAX_ABS_TOL = 1e-2   # on the bf16 output
REL_L2_TOL = 5e-3    # per (sequence, query head) row


def error_metrics(out_gpu_bf16: torch.Tensor, out_ref: np.ndarray):
    """max |gpu - ref| and the worst per-row relative L2 error (rows = last axis vectors)."""
    got = out_gpu_bf16.detach().float().cpu().numpy().astype(np.float64)
    diff = got - out_ref
    max_abs = float(np.abs(diff).max()) if diff.size else 0.0
    num = np.sqrt((diff ** 2).sum(axis=-1))
    den = np.sqrt((out_ref ** 2).sum(axis=-1))
    ok = den > 1e-30
    rel = np.where(ok, num / np.where(ok, den, 1.0), 0.0)
    return max_abs, float(rel.max()) if rel.size else 0.0


def assert_parity(out_gpu_bf16, out_ref, what="", scale_abs_by_magnitude=False):
    """``scale_abs_by_magnitude``: the absolute bound becomes 1e-2 * max(1, |ref|) per element. bf16 cannot
    hold a value of magnitude 4 to better than 1.6e-2, so outputs that are single V rows (contexts of a
    handful of tokens, as the first queries of a prefill see) need the bound to follow the magnitude."""
    assert torch.isfinite(out_gpu_bf16.float()).all(), f"{what}: non-finite output"
    max_abs, rel = error_metrics(out_gpu_bf16, out_ref)
    if scale_abs_by_magnitude:
        got = out_gpu_bf16.detach().float().cpu().numpy().astype(np.float64)
        max_abs = float((np.abs(got - out_ref) / np.maximum(1.0, np.abs(out_ref))).max())
    assert max_abs <= MAX_ABS_TOL, f"{what}: max abs error {max_abs:.3e} > {MAX_ABS_TOL}"
    assert rel <= REL_L2_TOL, f"{what}: per-row relative L2 {rel:.3e} > {REL_L2_TOL}"
    return max_abs, rel


def oracle_on_cache(q, cache, lens, sm_scale, seq_ids=None):
    """Oracle output for all (or the given) sequences of a device-resident cache.

    Only the pages those sequences own are brought to the host: they are gathered
    into a compact pool with a renumbered table (the result does not depend on
    physical page ids).
    """
    lens = np.asarray(lens, dtype=np.int32)
    ids = np.arange(len(lens)) if seq_ids is None else np.asarray(seq_ids)
    P = cache.k_pages.shape[2]
    table = cache.page_table.detach().cpu().numpy()
    rows, new_table, cur = [], np.full((len(ids), table.shape[1]), -1, dtype=np.int32), 0
    for i, b in enumerate(ids):
        n = (int(lens[b]) + P - 1) // P
        rows.append(table[b, :n])
        new_table[i, :n] = np.arange(cur, cur + n)
        cur += n
    phys = torch.from_numpy(np.concatenate(rows).astype(np.int64)).to(cache.k_pages.device) if cur else None
    if cur:
        kp = oracle.bf16_bits(cache.k_pages.index_select(0, phys))
        vp = oracle.bf16_bits(cache.v_pages.index_select(0, phys))
    else:
        kp = np.zeros((1,) + tuple(cache.k_pages.shape[1:]), np.uint16)
        vp = kp.copy()
    qb = oracle.bf16_bits(q[torch.from_numpy(ids).to(q.device)])
    return oracle.decode_attn(qb, kp, vp, new_table, lens[ids], sm_scale)


class Ctx:
    """Context manager around pd_create / pd_destroy for one geometry."""

    def __init__(self, Hq, Hkv, d, max_batch, MP, NP, device=0):
        import paper_2609_35158_b200 as pd

        self.pd = pd
        self.h = pd.pd_create(Hq, Hkv, d, wl.PAGE_SIZE, max_batch, MP, NP, device)

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.pd.pd_destroy(self.h)
        return False


def ctx_for(cache, Hq, max_batch=None):
    NP, Hkv, P, d = cache.k_pages.shape
    B, MP = cache.page_table.shape
    return Ctx(Hq, Hkv, d, max_batch or B, MP, NP, cache.k_pages.device.index or 0)
