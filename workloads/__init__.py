"""Seeded synthetic inputs for paged decode attention.

This module only draws numbers and lays out pages: context lengths, a
scattered page table over a permuted pool, bf16 N(0,1) tensors and a host-side
free list. It contains none of the attention or append arithmetic and is the
one module both the CPU oracle's tests and the CUDA path's tests / benchmark
may import.

The five workloads mirror the rollout shapes of the paper (rollout batch 64,
trajectories up to 32K tokens, multi-turn growth of the context, Sec. 6.1 and
Sec. 2.1; low decode concurrency while sequences wait on the environment,
Eq. 2). Values carry no meaning: attention cost depends on shapes and lengths
only, so the public benchmark the paper trains on is replaced by these draws.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

PAGE_SIZE = 16
NAN_BF16_BITS = 0x7FC0  # quiet NaN, used as poison in slots nobody may read


@dataclass(frozen=True)
class Workload:
    """Geometry of one configuration (lengths are drawn by ``context_lengths``)."""

    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int = PAGE_SIZE

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def sm_scale(self) -> float:
        return float(np.float32(1.0 / math.sqrt(self.head_dim)))

    @property
    def kv_bytes_per_token(self) -> int:
        # K row + V row of every KV head, bf16
        return 2 * self.num_kv_heads * self.head_dim * 2


WORKLOADS = {
    0: Workload("tiny_b4_h8kv2_d64", 4, 8, 2, 64),
    1: Workload("qwen3_8b_b64_ctx2k_16k", 64, 32, 8, 128),
    2: Workload("qwen3_30b_a3b_b256_lognormal8k", 256, 32, 4, 128),
    3: Workload("qwen3_8b_lowconc_b8_ctx32k_64k", 8, 32, 8, 128),
    4: Workload("qwen3_8b_multiturn_b512", 512, 32, 8, 128),
}

LOGNORMAL_SIGMA = 0.7  # natural-log units; the workload text gives only the median


def context_lengths(config: int, seed: int | None = None, batch: int | None = None) -> np.ndarray:
    """Context lengths (tokens already in the cache, before any append), int32 [B].

    All ranges are integer and inclusive at both ends. ``seed`` defaults to the
    configuration index.
    """
    w = WORKLOADS[config]
    B = w.batch if batch is None else batch
    rng = np.random.Generator(np.random.PCG64(config if seed is None else seed))
    if config == 0:
        lens = rng.integers(16, 256, size=B, endpoint=True)
    elif config == 1:
        lens = rng.integers(2048, 16384, size=B, endpoint=True)
    elif config == 2:
        z = rng.standard_normal(B)
        lens = np.clip(np.rint(np.exp(math.log(8192.0) + LOGNORMAL_SIGMA * z)), 1024, 32768)
    elif config == 3:
        lens = rng.integers(32768, 65536, size=B, endpoint=True)
    elif config == 4:
        turns = rng.integers(1, 20, size=B, endpoint=True)
        lens = np.array([rng.integers(256, 2048, size=int(t), endpoint=True).sum() for t in turns])
    else:
        raise KeyError(config)
    return lens.astype(np.int32)


@dataclass
class PagedCache:
    """Device (or host) tensors of one paged KV cache plus its host bookkeeping."""

    k_pages: "object"  # torch bf16 [NP, Hkv, P, d]
    v_pages: "object"
    page_table: "object"  # torch int32 [B, MP] on the same device
    ctx_lens: "object"  # torch int32 [B]
    page_table_host: np.ndarray  # int32 [B, MP]; -1 where unassigned
    ctx_lens_host: np.ndarray  # int32 [B]
    free_pages: list = field(default_factory=list)  # physical ids not yet assigned

    @property
    def num_pages(self) -> int:
        return int(self.k_pages.shape[0])


def random_bf16(shape, seed: int, device="cpu"):
    """bf16 N(0,1) tensor from a seeded torch generator on ``device``."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    if int(np.prod(shape)) > (1 << 24):
        return _big_randn_bf16(shape, g, device)
    return torch.randn(tuple(shape), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)


def _big_randn_bf16(shape, g, device):
    """Chunked generation along dim 0 so no fp32 copy of a multi-GB pool is held."""
    import torch

    out = torch.empty(tuple(shape), device=device, dtype=torch.bfloat16)
    rows = shape[0]
    per_row = int(np.prod(shape[1:]))
    step = max(1, (1 << 26) // max(1, per_row))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        out[r0:r1] = torch.randn((r1 - r0, *shape[1:]), generator=g, device=device, dtype=torch.float32)
    return out


def build_paged_cache(lens, num_kv_heads: int, head_dim: int, *, seed: int, device="cpu",
                      page_size: int = PAGE_SIZE, reserve_tokens: int = 0, preassign_reserve: bool = True,
                      slack: float = 1.0625, max_pages_per_seq: int | None = None,
                      poison: bool = False, permute: bool = True) -> PagedCache:
    """A scattered paged cache holding ``lens[b]`` random tokens per sequence.

    The pool has ``ceil(slack * sum_b ceil((lens[b] + reserve_tokens) / P))`` pages.
    Physical ids are a seeded permutation of the pool; sequence ``b`` takes the
    next entries of the permutation for its logical pages, so its pages are
    scattered. ``reserve_tokens`` is room for later appends: with
    ``preassign_reserve`` those pages are already in the table (entries past
    ``ceil(L/P)`` are ignored by readers), otherwise they stay on the free list
    for a host allocator to hand out. With ``poison`` every slot that holds no
    token (tails of last pages, reserved and free pages) is bf16 NaN and every
    unassigned table entry is -1. ``permute=False`` lays the pages out in logical order
    (a contiguous cache), for experiments on the cost of scattering.
    """
    import torch

    lens = np.asarray(lens, dtype=np.int64)
    B = len(lens)
    P = page_size
    pages_now = (lens + P - 1) // P
    pages_cap = (lens + reserve_tokens + P - 1) // P
    NP = int(math.ceil(slack * max(1, int(pages_cap.sum()))))
    MP = int(max(1, pages_cap.max())) if max_pages_per_seq is None else int(max_pages_per_seq)
    assert MP >= pages_cap.max()
    rng = np.random.Generator(np.random.PCG64([int(seed), 0x9A6E5]))
    perm = rng.permutation(NP).astype(np.int32) if permute else np.arange(NP, dtype=np.int32)
    table = np.full((B, MP), -1, dtype=np.int32)
    cur = 0
    for b in range(B):
        n = int(pages_cap[b] if preassign_reserve else pages_now[b])
        table[b, :n] = perm[cur:cur + n]
        cur += n
    free = [int(x) for x in perm[cur:]]
    k_pages = random_bf16((NP, num_kv_heads, P, head_dim), seed * 7919 + 1, device)
    v_pages = random_bf16((NP, num_kv_heads, P, head_dim), seed * 7919 + 2, device)
    table_dev = table.copy()
    if poison:
        valid = np.zeros((NP, P), dtype=bool)
        for b in range(B):
            L = int(lens[b])
            for i in range(int(pages_now[b])):
                valid[table[b, i], :min(P, L - i * P)] = True
        mask = torch.from_numpy(~valid).to(device)[:, None, :, None]
        nan = torch.tensor(float("nan"), dtype=torch.bfloat16, device=device)
        k_pages = torch.where(mask, nan, k_pages)
        v_pages = torch.where(mask, nan, v_pages)
        for b in range(B):
            table_dev[b, int(pages_now[b]):] = -1
    return PagedCache(
        k_pages=k_pages, v_pages=v_pages,
        page_table=torch.from_numpy(table_dev).to(device),
        ctx_lens=torch.from_numpy(lens.astype(np.int32)).to(device),
        page_table_host=table_dev, ctx_lens_host=lens.astype(np.int32), free_pages=free)


class PageAllocator:
    """Host free list: hands a fresh physical page to a sequence whose next token opens a page."""

    def __init__(self, cache: PagedCache, page_size: int = PAGE_SIZE):
        self.cache = cache
        self.P = page_size

    def pages_needed(self, lens: np.ndarray) -> np.ndarray:
        """Indices of sequences whose next append position starts a new logical page
        that has no physical page yet."""
        lens = np.asarray(lens)
        at_boundary = np.nonzero(lens % self.P == 0)[0]
        tbl = self.cache.page_table_host
        return np.array([b for b in at_boundary if tbl[b, lens[b] // self.P] < 0], dtype=np.int64)

    def assign(self, lens: np.ndarray):
        """Assign pages for the next append; returns (seq ids, logical page index, physical ids)."""
        need = self.pages_needed(lens)
        logical = np.asarray(lens)[need] // self.P
        phys = np.empty(len(need), dtype=np.int32)
        for i, b in enumerate(need):
            if not self.cache.free_pages:
                raise RuntimeError("page pool exhausted")
            phys[i] = self.cache.free_pages.pop()
            self.cache.page_table_host[b, logical[i]] = phys[i]
        return need, logical.astype(np.int64), phys


def shard_sequences(lens: np.ndarray, world_size: int) -> list:
    """Split sequence ids over ranks so that every rank holds about the same number
    of cached tokens (greedy longest-first); sequences are independent, so no data
    crosses ranks. Returns ``world_size`` sorted index arrays."""
    order = np.argsort(-np.asarray(lens, dtype=np.int64), kind="stable")
    loads = [0] * world_size
    parts: list = [[] for _ in range(world_size)]
    for b in order:
        r = int(np.argmin(loads))
        parts[r].append(int(b))
        loads[r] += int(lens[b])
    return [np.array(sorted(p), dtype=np.int64) for p in parts]
