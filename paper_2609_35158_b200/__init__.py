"""Python binding of ``libpd.so``: paged GQA decode attention + KV append on B200.

Argument marshalling only. Every function has the name and the argument order
of its C counterpart in ``include/pd.h``; tensors are torch tensors whose
``data_ptr()`` is handed to the library, streams default to torch's current
stream. Nothing here computes: if the CUDA library cannot be loaded the import
fails, there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

PD_OK = 0
PD_ERR_INVALID_ARG = -1
PD_ERR_UNSUPPORTED = -2
PD_ERR_CUDA = -3
PD_ERR_WORKSPACE = -4
PD_ERR_DEVICE_FAULT = -5
PD_ERR_TIMEOUT = -6
PD_APPEND_NO_ADVANCE = 1

# every symbol include/pd.h declares
EXPORTS = (
    "pd_create", "pd_destroy", "pd_kv_append", "pd_decode_attn", "pd_decode_attn_static", "pd_decode_step", "pd_decode_step_host",
    "pd_kv_gather", "pd_kv_scatter", "pd_kv_append_tokens", "pd_prefill_attn", "pd_device_status", "pd_read_worker_trace",
    "pd_makespan_coloc", "pd_makespan_disagg", "pd_feasible_disagg", "pd_decide", "pd_min_change_plan", "pd_toggle_gate",
    "pd_fit_decode_cost", "pd_plan_ranges", "pd_plan_walk",
    "pd_kv_quantize_pages", "pd_kv_append_fp8", "pd_decode_attn_fp8", "pd_decode_step_fp8", "pd_kv_gather_fp8", "pd_kv_scatter_fp8",
    "pd_pool_create", "pd_pool_resize", "pd_pool_base", "pd_pool_capacity", "pd_pool_chunk_bytes", "pd_pool_resident_bytes",
    "pd_pool_last_error", "pd_pool_destroy",
    "pd_set_profile_events", "pd_read_probe", "pd_host_step_counts", "pd_workspace_bytes", "pd_launch_count", "pd_last_plan", "pd_status_string", "pd_last_error", "pd_version",
)


class pd_config(ctypes.Structure):
    _fields_ = [
        ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("page_size", ctypes.c_int32), ("max_batch", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32),
        ("num_pages", ctypes.c_int64), ("device", ctypes.c_int32), ("flags", ctypes.c_uint32),
    ]


class pd_cost_model(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in (
        "B", "S", "r", "dL", "theta", "A", "b", "t_prefill", "T_over", "T_env", "K_bytes", "BW", "K_seq_bytes",
        "H_max_bytes", "prefill_tokens_per_worker")]


class pd_target(ctypes.Structure):
    _fields_ = [("N_P", ctypes.c_int32), ("N_D", ctypes.c_int32), ("N_C", ctypes.c_int32),
                ("makespan", ctypes.c_double)]


class PdError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        msg = f"{where}: {pd_status_string(code)} ({code})"
        super().__init__(msg + (f" - {detail}" if detail else ""))


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python paper_2609_35158_b200/build.py` "
            "(nvcc, sm_100a). This package has no fallback path.")
    lib = ctypes.CDLL(path)
    vp, i32, u32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint32, ctypes.c_int64, ctypes.c_float
    lib.pd_create.argtypes = [ctypes.POINTER(pd_config), ctypes.POINTER(vp)]
    lib.pd_destroy.argtypes = [vp]
    lib.pd_kv_append.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, u32, vp]
    lib.pd_decode_attn.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, f32, i32, vp]
    lib.pd_decode_attn_static.argtypes = [ctypes.POINTER(pd_config), vp, vp, vp, vp, vp, vp, vp, i32, f32, vp]
    lib.pd_kv_append_tokens.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, vp]
    lib.pd_prefill_attn.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, vp]
    lib.pd_kv_gather.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.pd_kv_scatter.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.pd_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, f32, i32, vp]
    lib.pd_decode_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, f32, i32, vp]
    lib.pd_device_status.argtypes = [vp, vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.pd_set_profile_events.argtypes = [vp, vp, vp]
    lib.pd_read_probe.argtypes = [vp, ctypes.c_size_t, i32, i32, vp, vp]
    lib.pd_host_step_counts.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    lib.pd_read_worker_trace.argtypes = [vp, vp, vp, i32, ctypes.POINTER(i32)]
    lib.pd_workspace_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
    lib.pd_launch_count.argtypes = [vp, ctypes.POINTER(i64)]
    lib.pd_last_plan.argtypes = [vp, vp, ctypes.POINTER(i64), ctypes.POINTER(i32), ctypes.POINTER(i32),
                                 ctypes.POINTER(i32)]
    dbl = ctypes.c_double
    pm, pt = ctypes.POINTER(pd_cost_model), ctypes.POINTER(pd_target)
    lib.pd_makespan_coloc.argtypes = [pm, i32]
    lib.pd_makespan_coloc.restype = dbl
    lib.pd_makespan_disagg.argtypes = [pm, i32, i32, ctypes.POINTER(dbl), ctypes.POINTER(dbl)]
    lib.pd_makespan_disagg.restype = dbl
    lib.pd_feasible_disagg.argtypes = [pm, i32, i32]
    lib.pd_decide.argtypes = [pm, i32, pt, dbl, dbl, pt]
    lib.pd_min_change_plan.argtypes = [vp, vp, vp, i32, vp, i32, vp, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.pd_toggle_gate.argtypes = [dbl, dbl, dbl, dbl, dbl]
    lib.pd_plan_ranges.argtypes = [i64, i32, i32, i32, i32, i32, i32, vp, vp, i32, ctypes.POINTER(i32)]
    lib.pd_plan_walk.argtypes = [vp, i32, i32, i64, i32, vp, vp, vp]
    lib.pd_fit_decode_cost.argtypes = [vp, vp, i32, ctypes.POINTER(dbl), ctypes.POINTER(dbl)]
    lib.pd_status_string.argtypes = [ctypes.c_int]
    lib.pd_status_string.restype = ctypes.c_char_p
    lib.pd_last_error.argtypes = [vp]
    lib.pd_last_error.restype = ctypes.c_char_p
    lib.pd_version.argtypes = []
    lib.pd_kv_quantize_pages.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    lib.pd_kv_append_fp8.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, ctypes.c_uint32, vp]
    lib.pd_decode_attn_fp8.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, f32, i32, vp]
    lib.pd_decode_step_fp8.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, f32, i32, vp]
    lib.pd_kv_gather_fp8.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.pd_kv_scatter_fp8.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp]
    u64 = ctypes.c_uint64
    lib.pd_pool_create.argtypes = [i32, u64, u64, ctypes.POINTER(vp)]
    lib.pd_pool_resize.argtypes = [vp, u64, vp]
    lib.pd_pool_destroy.argtypes = [vp]
    lib.pd_pool_base.argtypes = [vp]
    lib.pd_pool_base.restype = vp
    for name in ("pd_pool_capacity", "pd_pool_chunk_bytes", "pd_pool_resident_bytes"):
        getattr(lib, name).argtypes = [vp]
        getattr(lib, name).restype = u64
    lib.pd_pool_last_error.argtypes = [vp]
    lib.pd_pool_last_error.restype = ctypes.c_char_p
    own_restype = ("pd_status_string", "pd_last_error", "pd_makespan_coloc", "pd_makespan_disagg", "pd_pool_base",
                   "pd_pool_capacity", "pd_pool_chunk_bytes", "pd_pool_resident_bytes", "pd_pool_last_error")
    for name in EXPORTS:
        if name not in own_restype:
            getattr(lib, name).restype = ctypes.c_int
    return lib


_lib = _load()


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(rc: int, where: str, ctx=None):
    if rc != PD_OK:
        raise PdError(rc, where, pd_last_error(ctx) if ctx else "")


def pd_version() -> int:
    return _lib.pd_version()


def pd_status_string(code: int) -> str:
    return _lib.pd_status_string(code).decode()


def pd_last_error(ctx) -> str:
    return _lib.pd_last_error(ctx).decode()


def pd_create(num_q_heads, num_kv_heads, head_dim, page_size, max_batch, max_pages_per_seq, num_pages,
              device=0, flags=0):
    """Returns an opaque context handle (ctypes void pointer)."""
    cfg = pd_config(num_q_heads, num_kv_heads, head_dim, page_size, max_batch, max_pages_per_seq, num_pages,
                    device, flags)
    ctx = ctypes.c_void_p()
    _check(_lib.pd_create(ctypes.byref(cfg), ctypes.byref(ctx)), "pd_create")
    return ctx


def pd_destroy(ctx) -> None:
    _lib.pd_destroy(ctx)


def pd_kv_append(ctx, k_new, v_new, k_pages, v_pages, page_table, ctx_lens, batch=None, call_flags=0, stream=None):
    batch = k_new.shape[0] if batch is None else batch
    _check(_lib.pd_kv_append(ctx, _ptr(k_new), _ptr(v_new), _ptr(k_pages), _ptr(v_pages), _ptr(page_table),
                             _ptr(ctx_lens), batch, call_flags, _stream(stream)), "pd_kv_append", ctx)


def pd_decode_attn(ctx, q, k_pages, v_pages, page_table, ctx_lens, out, lse=None, batch=None, sm_scale=1.0,
                   split_pages=0, stream=None):
    batch = q.shape[0] if batch is None else batch
    _check(_lib.pd_decode_attn(ctx, _ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(page_table), _ptr(ctx_lens),
                               _ptr(out), _ptr(lse), batch, sm_scale, split_pages, _stream(stream)),
           "pd_decode_attn", ctx)


def pd_kv_append_tokens(ctx, k_new, v_new, q_indptr, k_pages, v_pages, page_table, ctx_lens, max_q_len, batch=None,
                        stream=None):
    batch = q_indptr.shape[0] - 1 if batch is None else batch
    _check(_lib.pd_kv_append_tokens(ctx, _ptr(k_new), _ptr(v_new), _ptr(q_indptr), _ptr(k_pages), _ptr(v_pages),
                                    _ptr(page_table), _ptr(ctx_lens), batch, max_q_len, _stream(stream)),
           "pd_kv_append_tokens", ctx)


def pd_prefill_attn(ctx, q, q_indptr, k_pages, v_pages, page_table, ctx_lens, out, lse=None, max_q_len=0, batch=None,
                    sm_scale=1.0, stream=None):
    batch = q_indptr.shape[0] - 1 if batch is None else batch
    _check(_lib.pd_prefill_attn(ctx, _ptr(q), _ptr(q_indptr), _ptr(k_pages), _ptr(v_pages), _ptr(page_table),
                                _ptr(ctx_lens), _ptr(out), _ptr(lse), batch, max_q_len, sm_scale, _stream(stream)),
           "pd_prefill_attn", ctx)


def pd_kv_gather(ctx, k_pages, v_pages, page_table, page_begin, page_end, packed_page_offset, packed, batch=None,
                 stream=None):
    batch = page_begin.shape[0] if batch is None else batch
    _check(_lib.pd_kv_gather(ctx, _ptr(k_pages), _ptr(v_pages), _ptr(page_table), _ptr(page_begin), _ptr(page_end),
                             _ptr(packed_page_offset), _ptr(packed), batch, _stream(stream)), "pd_kv_gather", ctx)


def pd_kv_scatter(ctx, packed, packed_page_offset, k_pages, v_pages, page_table, page_begin, page_end, batch=None,
                  stream=None):
    batch = page_begin.shape[0] if batch is None else batch
    _check(_lib.pd_kv_scatter(ctx, _ptr(packed), _ptr(packed_page_offset), _ptr(k_pages), _ptr(v_pages),
                              _ptr(page_table), _ptr(page_begin), _ptr(page_end), batch, _stream(stream)),
           "pd_kv_scatter", ctx)


def pd_decode_attn_static(cfg: pd_config, q, k_pages, v_pages, page_table, ctx_lens, out, lse=None, batch=None,
                          sm_scale=1.0, stream=None):
    """Attention for callers that may not allocate: no context, scratch lives in a fixed array
    inside the library. ``cfg`` is a ``pd_config`` describing the geometry and the device."""
    batch = q.shape[0] if batch is None else batch
    _check(_lib.pd_decode_attn_static(ctypes.byref(cfg), _ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(page_table),
                                      _ptr(ctx_lens), _ptr(out), _ptr(lse), batch, sm_scale, _stream(stream)),
           "pd_decode_attn_static")


def pd_decode_step(ctx, q, k_new, v_new, k_pages, v_pages, page_table, ctx_lens, out, lse=None, batch=None,
                   sm_scale=1.0, split_pages=0, stream=None):
    batch = q.shape[0] if batch is None else batch
    _check(_lib.pd_decode_step(ctx, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pages), _ptr(v_pages), _ptr(page_table),
                               _ptr(ctx_lens), _ptr(out), _ptr(lse), batch, sm_scale, split_pages, _stream(stream)),
           "pd_decode_step", ctx)


def pd_decode_step_host(ctx, q_host, k_new_host, v_new_host, k_pages, v_pages, page_table, ctx_lens, out_host,
                        batch=None, sm_scale=1.0, split_pages=0, stream=None):
    """q_host, k_new_host, v_new_host, out_host are CPU tensors (pinned for full copy speed)."""
    for t in (q_host, k_new_host, v_new_host, out_host):
        assert not t.is_cuda and t.is_contiguous()
    batch = q_host.shape[0] if batch is None else batch
    _check(_lib.pd_decode_step_host(ctx, _ptr(q_host), _ptr(k_new_host), _ptr(v_new_host), _ptr(k_pages),
                                    _ptr(v_pages), _ptr(page_table), _ptr(ctx_lens), _ptr(out_host), batch,
                                    sm_scale, split_pages, _stream(stream)), "pd_decode_step_host", ctx)


def pd_kv_quantize_pages(ctx, k_pages, v_pages, tokens_in_page, k8, v8, kv_scales, stream=None):
    _check(_lib.pd_kv_quantize_pages(ctx, _ptr(k_pages), _ptr(v_pages), _ptr(tokens_in_page), _ptr(k8), _ptr(v8),
                                     _ptr(kv_scales), _stream(stream)), "pd_kv_quantize_pages", ctx)


def pd_kv_append_fp8(ctx, k_new, v_new, k8, v8, kv_scales, page_table, ctx_lens, batch=None, call_flags=0, stream=None):
    batch = k_new.shape[0] if batch is None else batch
    _check(_lib.pd_kv_append_fp8(ctx, _ptr(k_new), _ptr(v_new), _ptr(k8), _ptr(v8), _ptr(kv_scales), _ptr(page_table),
                                 _ptr(ctx_lens), batch, call_flags, _stream(stream)), "pd_kv_append_fp8", ctx)


def pd_decode_attn_fp8(ctx, q, k8, v8, kv_scales, page_table, ctx_lens, out, lse=None, batch=None, sm_scale=1.0,
                       split_pages=0, stream=None):
    batch = q.shape[0] if batch is None else batch
    _check(_lib.pd_decode_attn_fp8(ctx, _ptr(q), _ptr(k8), _ptr(v8), _ptr(kv_scales), _ptr(page_table), _ptr(ctx_lens),
                                   _ptr(out), _ptr(lse), batch, sm_scale, split_pages, _stream(stream)),
           "pd_decode_attn_fp8", ctx)


def pd_decode_step_fp8(ctx, q, k_new, v_new, k8, v8, kv_scales, page_table, ctx_lens, out, lse=None, batch=None,
                       sm_scale=1.0, split_pages=0, stream=None):
    batch = q.shape[0] if batch is None else batch
    _check(_lib.pd_decode_step_fp8(ctx, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k8), _ptr(v8), _ptr(kv_scales),
                                   _ptr(page_table), _ptr(ctx_lens), _ptr(out), _ptr(lse), batch, sm_scale, split_pages,
                                   _stream(stream)), "pd_decode_step_fp8", ctx)


def pd_kv_gather_fp8(ctx, k8, v8, kv_scales, page_table, page_begin, page_end, packed_page_offset, packed, batch=None,
                     stream=None):
    batch = page_begin.shape[0] if batch is None else batch
    _check(_lib.pd_kv_gather_fp8(ctx, _ptr(k8), _ptr(v8), _ptr(kv_scales), _ptr(page_table), _ptr(page_begin),
                                 _ptr(page_end), _ptr(packed_page_offset), _ptr(packed), batch, _stream(stream)),
           "pd_kv_gather_fp8", ctx)


def pd_kv_scatter_fp8(ctx, packed, packed_page_offset, k8, v8, kv_scales, page_table, page_begin, page_end, batch=None,
                      stream=None):
    batch = page_begin.shape[0] if batch is None else batch
    _check(_lib.pd_kv_scatter_fp8(ctx, _ptr(packed), _ptr(packed_page_offset), _ptr(k8), _ptr(v8), _ptr(kv_scales),
                                  _ptr(page_table), _ptr(page_begin), _ptr(page_end), batch, _stream(stream)),
           "pd_kv_scatter_fp8", ctx)


def pd_pool_create(device: int, capacity_bytes: int, chunk_bytes: int = 0):
    """Elastic KV pool: a fixed device address range backed chunk by chunk; returns the opaque handle."""
    h = ctypes.c_void_p()
    _check(_lib.pd_pool_create(device, capacity_bytes, chunk_bytes, ctypes.byref(h)), "pd_pool_create")
    return h


def _check_pool(rc, where, pool):
    if rc != PD_OK:
        raise PdError(rc, where, (_lib.pd_pool_last_error(pool) or b"").decode())


def pd_pool_resize(pool, resident_bytes: int, stream_to_drain=None):
    s = None if stream_to_drain is None else _stream(stream_to_drain)
    _check_pool(_lib.pd_pool_resize(pool, resident_bytes, s), "pd_pool_resize", pool)


def pd_pool_base(pool) -> int:
    return _lib.pd_pool_base(pool) or 0


def pd_pool_capacity(pool) -> int:
    return _lib.pd_pool_capacity(pool)


def pd_pool_chunk_bytes(pool) -> int:
    return _lib.pd_pool_chunk_bytes(pool)


def pd_pool_resident_bytes(pool) -> int:
    return _lib.pd_pool_resident_bytes(pool)


def pd_pool_last_error(pool) -> str:
    return (_lib.pd_pool_last_error(pool) or b"").decode()


def pd_pool_destroy(pool):
    _check(_lib.pd_pool_destroy(pool), "pd_pool_destroy")


class _DeviceRange:
    """Exposes raw device bytes through the CUDA array interface so torch can alias them."""

    def __init__(self, ptr: int, nbytes: int):
        self.__cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|u1", "data": (ptr, False), "version": 2}


def pool_tensor(pool, offset_bytes: int, shape, dtype, device: int = 0):
    """A torch tensor aliasing ``shape`` elements of ``dtype`` at ``offset_bytes`` of the pool's range
    (no copy, no ownership). Only the resident prefix may be touched."""
    n = 1
    for s in shape:
        n *= int(s)
    nbytes = n * torch.empty((), dtype=dtype).element_size()
    if offset_bytes < 0 or offset_bytes + nbytes > pd_pool_resident_bytes(pool):
        raise ValueError("the requested range is not resident")
    raw = torch.as_tensor(_DeviceRange(pd_pool_base(pool) + offset_bytes, nbytes), device=f"cuda:{device}")
    return raw.view(dtype).view(*shape)


def pd_device_status(ctx, stream=None):
    """(code, seq, detail) of the first latched device fault; clears it."""
    code, seq, detail = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _lib.pd_device_status(ctx, _stream(stream), ctypes.byref(code), ctypes.byref(seq), ctypes.byref(detail))
    return code.value, seq.value, detail.value


def pd_set_profile_events(ctx, before=None, after=None) -> None:
    """``before`` / ``after``: ``torch.cuda.Event(enable_timing=True)`` objects (or None, None)."""
    def handle(ev):
        if ev is None:
            return None
        if ev.cuda_event == 0:  # torch creates the CUDA event lazily, on first record
            ev.record()
        return ev.cuda_event
    _check(_lib.pd_set_profile_events(ctx, handle(before), handle(after)), "pd_set_profile_events", ctx)


def pd_host_step_counts(ctx):
    """(calls whose result went straight to the pinned host buffer, calls that staged it on the device)."""
    d, s = ctypes.c_int64(0), ctypes.c_int64(0)
    _check(_lib.pd_host_step_counts(ctx, ctypes.byref(d), ctypes.byref(s)), "pd_host_step_counts", ctx)
    return int(d.value), int(s.value)


def pd_read_probe(src, blocks: int, threads: int, sink, stream=None) -> None:
    """Reads the whole of ``src`` once with a ``blocks`` x ``threads`` streaming kernel; ``sink`` is a 16-byte device tensor."""
    rc = _lib.pd_read_probe(_ptr(src), src.numel() * src.element_size(), blocks, threads, _ptr(sink), _stream(stream))
    _check(rc, "pd_read_probe")


def pd_read_worker_trace(ctx, max_workers=4096, stream=None):
    """uint64 array [workers, 4] of ns timestamps (needs a PD_ENABLE_TUNING build and PD_TRACE_WORKERS=1 at pd_create)."""
    import numpy as np

    buf = np.zeros((max_workers, 4), dtype=np.uint64)
    n = ctypes.c_int32()
    _check(_lib.pd_read_worker_trace(ctx, _stream(stream), buf.ctypes.data, max_workers, ctypes.byref(n)),
           "pd_read_worker_trace", ctx)
    return buf[:n.value]


def pd_workspace_bytes(ctx) -> int:
    n = ctypes.c_size_t()
    _check(_lib.pd_workspace_bytes(ctx, ctypes.byref(n)), "pd_workspace_bytes", ctx)
    return n.value


def pd_launch_count(ctx) -> int:
    n = ctypes.c_int64()
    _check(_lib.pd_launch_count(ctx, ctypes.byref(n)), "pd_launch_count", ctx)
    return n.value


def pd_last_plan(ctx, stream=None) -> dict:
    total, per, ranges, workers = ctypes.c_int64(), ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(_lib.pd_last_plan(ctx, _stream(stream), ctypes.byref(total), ctypes.byref(per), ctypes.byref(ranges),
                             ctypes.byref(workers)), "pd_last_plan", ctx)
    return {"total_units": total.value, "pages_per_range": per.value, "num_ranges": ranges.value,
            "num_workers": workers.value}


# ---- PD decision engine (host-only)

def pd_makespan_coloc(model: pd_cost_model, N: int) -> float:
    return _lib.pd_makespan_coloc(ctypes.byref(model), N)


def pd_makespan_disagg(model: pd_cost_model, N_P: int, N_D: int):
    """Returns (T_dis, T_prefill, T_decode)."""
    tp, td = ctypes.c_double(), ctypes.c_double()
    t = _lib.pd_makespan_disagg(ctypes.byref(model), N_P, N_D, ctypes.byref(tp), ctypes.byref(td))
    return t, tp.value, td.value


def pd_feasible_disagg(model: pd_cost_model, N_P: int, N_D: int) -> bool:
    return bool(_lib.pd_feasible_disagg(ctypes.byref(model), N_P, N_D))


def pd_decide(model: pd_cost_model, N_k: int, current: pd_target | None = None, ratio_threshold=0.0,
              mode_threshold=0.0) -> pd_target:
    out = pd_target()
    _check(_lib.pd_decide(ctypes.byref(model), N_k, None if current is None else ctypes.byref(current),
                          ratio_threshold, mode_threshold, ctypes.byref(out)), "pd_decide")
    return out


def pd_min_change_plan(cur_active, cur_role, dst_active, dst_role_count):
    """NumPy int32 arrays in, (new_role, d_worker, d_role) out."""
    import numpy as np

    ca, cr, da = (np.ascontiguousarray(a, dtype=np.int32) for a in (cur_active, cur_role, dst_active))
    rc = np.ascontiguousarray(dst_role_count, dtype=np.int32)
    new_role = np.full(len(ca), -1, dtype=np.int32)
    dw, dr = ctypes.c_int32(), ctypes.c_int32()
    _check(_lib.pd_min_change_plan(ca.ctypes.data, cr.ctypes.data, da.ctypes.data, len(ca), rc.ctypes.data, len(rc),
                                   new_role.ctypes.data, ctypes.byref(dw), ctypes.byref(dr)), "pd_min_change_plan")
    return new_role, dw.value, dr.value


def pd_toggle_gate(R, B, T_ded, T_full, T_toggle) -> bool:
    return bool(_lib.pd_toggle_gate(R, B, T_ded, T_full, T_toggle))


def pd_plan_ranges(total_units, n_workers, split_pages=0, max_ranges=None, min_pages=4, halving_levels=6, tail_pages=16):
    """(starts int64 [n], lens int32 [n]) of the decode kernels' plan, computed on the host."""
    import numpy as np

    max_ranges = 16 * n_workers if max_ranges is None else max_ranges
    n = ctypes.c_int32(0)
    _check(_lib.pd_plan_ranges(total_units, n_workers, split_pages, max_ranges, min_pages, halving_levels, tail_pages,
                               None, None, 0, ctypes.byref(n)), "pd_plan_ranges")
    starts = np.zeros(n.value, dtype=np.int64)
    lens = np.zeros(n.value, dtype=np.int32)
    _check(_lib.pd_plan_ranges(total_units, n_workers, split_pages, max_ranges, min_pages, halving_levels, tail_pages,
                               starts.ctypes.data, lens.ctypes.data, n.value, ctypes.byref(n)), "pd_plan_ranges")
    return starts, lens


def pd_plan_walk(cum_pages, num_kv_heads, first_unit, count):
    """(seq, kv_head, page) int32 arrays of `count` consecutive units starting at `first_unit`."""
    import numpy as np

    cum = np.ascontiguousarray(cum_pages, dtype=np.int32)
    out = [np.zeros(count, dtype=np.int32) for _ in range(3)]
    _check(_lib.pd_plan_walk(cum.ctypes.data, len(cum) - 1, num_kv_heads, first_unit, count, out[0].ctypes.data,
                             out[1].ctypes.data, out[2].ctypes.data), "pd_plan_walk")
    return tuple(out)


def pd_fit_decode_cost(concurrency, step_seconds):
    """Least-squares (A, b) of step_seconds = A + b * concurrency."""
    import numpy as np

    x = np.ascontiguousarray(concurrency, dtype=np.float64)
    y = np.ascontiguousarray(step_seconds, dtype=np.float64)
    A, b = ctypes.c_double(), ctypes.c_double()
    _check(_lib.pd_fit_decode_cost(x.ctypes.data, y.ctypes.data, len(x), ctypes.byref(A), ctypes.byref(b)),
           "pd_fit_decode_cost")
    return A.value, b.value
