"""Thin ctypes binding over libavmp.so: same names as the C ABI, argument marshalling only.

Device arguments may be torch CUDA tensors (their data_ptr is passed) or raw integer
addresses.  `stream` is a torch.cuda.Stream, a raw cudaStream_t integer, or None for
torch's current stream.  Nothing here computes anything: every step of the path runs in
the library's kernels.  If the library is missing it is built with nvcc; if that is not
possible the import fails -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional

import numpy as np
import torch

from . import build as _build

AVMP_OK, AVMP_EINVAL, AVMP_ENOSPC, AVMP_ECUDA, AVMP_ETOOBIG = 0, -1, -2, -3, -4
AVMP_STATIC_GATHER_MAX_REQS = 4096
AVMP_INVALID = 0xFFFFFFFF
AVMP_NONE64 = 0xFFFFFFFFFFFFFFFF

STAT_FIELDS = (
    "op_counter", "last_rebalance_op", "n_oom", "n_capacity_error", "n_rebalance",
    "migrated_bytes", "wasted_bytes", "relocated_blocks", "relocated_bytes", "gap_bytes",
    "cap_kv", "cap_ssm", "free_kv", "free_ssm", "fsm_state", "n_invalid",
    "unit_bytes_kv", "unit_bytes_ssm", "vid_space_kv", "vid_space_ssm", "pool_bytes_aligned",
    "error_code", "error_count", "relocation_ns_last", "relocation_ns_total",
    "step_ns_total", "step_ns_oom_retry", "step_ns_migration_plan",
)


class avmp_model_spec(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in (
        "n_attn_layers", "n_ssm_layers", "page_tokens", "kv_heads", "head_dim", "kv_elem_bytes",
        "ssm_state_elems", "ssm_conv_elems", "ssm_elem_bytes")]


class avmp_options(C.Structure):
    _fields_ = [("threshold_low_ppm", C.c_uint32), ("threshold_high_ppm", C.c_uint32),
                ("min_rebalance_interval_ops", C.c_uint64), ("migration_enabled", C.c_uint32),
                ("max_requests", C.c_uint32), ("max_pages_per_request", C.c_uint32),
                ("reclaim_gap", C.c_uint32)]


class avmp_layout(C.Structure):
    _fields_ = [("pool_bytes_aligned", C.c_uint64), ("unit_bytes", C.c_uint64 * 2),
                ("vid_space", C.c_uint64 * 2), ("cap0", C.c_uint64 * 2), ("gap0", C.c_uint64),
                ("kv_layer_bytes", C.c_uint64), ("kv_row_bytes", C.c_uint64),
                ("ssm_state_bytes", C.c_uint64), ("ssm_conv_bytes", C.c_uint64)]


class avmp_stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in STAT_FIELDS]


DRIVER_STAT_FIELDS = ("steps", "completed", "dropped", "preempted", "n_oom_admit", "n_oom_extend", "queue_next",
                      "requeued", "window", "last_batch_ops", "overflow")


class avmp_driver_stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in DRIVER_STAT_FIELDS]


SESSION_STAT_FIELDS = ("steps", "completed", "dropped", "preempted", "evicted", "n_oom_admit", "n_oom_extend",
                       "arrived", "arrival_queue", "requeued", "waiting", "window", "last_batch_ops", "forced_slot")


class avmp_session_stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in SESSION_STAT_FIELDS]


_u32p = C.POINTER(C.c_uint32)


class avmp_tables(C.Structure):
    _fields_ = [("slot_stack", _u32p * 2), ("vid_stack", _u32p * 2), ("vt", _u32p * 2), ("ow", _u32p * 2),
                ("req_state", _u32p), ("req_len", _u32p), ("req_npages", _u32p), ("req_chain", _u32p),
                ("req_ssm", _u32p), ("n_slot_stack", C.c_uint32 * 2), ("n_vid_stack", C.c_uint32 * 2),
                ("stats", avmp_stats)]


def _load():
    path = _build.build_library()          # raises if nvcc is missing and the library is absent
    L = C.CDLL(str(path))
    vp = C.c_void_p
    sig = {
        "avmp_default_options": (None, [C.POINTER(avmp_options)]),
        "avmp_derive_layout": (C.c_int, [C.POINTER(avmp_model_spec), C.c_uint64, C.c_double, C.POINTER(avmp_layout)]),
        "avmp_workspace_bytes": (C.c_size_t, [C.POINTER(avmp_model_spec), C.c_uint64, C.POINTER(avmp_options)]),
        "avmp_create": (C.c_int, [C.POINTER(vp), C.POINTER(avmp_model_spec), vp, C.c_uint64, C.c_double,
                                  C.c_uint32, C.POINTER(avmp_options), vp, C.c_size_t, vp]),
        "avmp_destroy": (C.c_int, [vp]),
        "avmp_step": (C.c_int, [vp, vp, C.c_uint32, vp, vp]),
        "avmp_step_translate": (C.c_int, [vp, vp, C.c_uint32, vp, vp, C.c_uint32, vp, vp, vp, vp]),
        "avmp_step_host": (C.c_int, [vp, vp, C.c_uint32, vp, vp]),
        "avmp_step_indirect": (C.c_int, [vp, vp, vp, C.c_uint32, vp, vp]),
        "avmp_driver_workspace_bytes": (C.c_size_t, [C.c_uint32]),
        "avmp_driver_create": (C.c_int, [C.POINTER(vp), vp, vp, vp, C.c_uint32, C.c_uint32, vp, C.c_size_t, vp]),
        "avmp_driver_destroy": (C.c_int, [vp]),
        "avmp_driver_step": (C.c_int, [vp, vp]),
        "avmp_driver_get_stats": (C.c_int, [vp, C.POINTER(avmp_driver_stats), vp]),
        "avmp_driver_export": (C.c_int, [vp, vp, vp, vp, vp, vp]),
        "avmp_session_driver_workspace_bytes": (C.c_size_t, [C.c_uint32, C.c_uint32]),
        "avmp_session_driver_create": (C.c_int, [C.POINTER(vp), vp, vp, vp, vp, vp, vp, C.c_uint32, C.c_uint32,
                                                 C.c_uint32, vp, C.c_size_t, vp]),
        "avmp_session_driver_destroy": (C.c_int, [vp]),
        "avmp_session_driver_step": (C.c_int, [vp, vp]),
        "avmp_session_driver_get_stats": (C.c_int, [vp, C.POINTER(avmp_session_stats), vp]),
        "avmp_session_driver_export": (C.c_int, [vp, vp, vp, vp, vp, vp, vp, vp, vp]),
        "avmp_translate": (C.c_int, [vp, vp, C.c_uint32, vp, vp, vp, vp]),
        "avmp_gather_kv": (C.c_int, [vp, C.c_uint32, vp, C.c_uint32, vp, vp, C.c_uint64, vp, vp]),
        "avmp_gather_kv_static": (C.c_int, [vp, C.c_uint32, vp, C.c_uint32, vp, vp, C.c_uint64, vp, vp]),
        "avmp_gather_ssm": (C.c_int, [vp, C.c_uint32, vp, C.c_uint32, vp, vp, vp]),
        "avmp_gather_kv_layers": (C.c_int, [vp, C.c_uint32, C.c_uint32, vp, C.c_uint32, vp, vp, C.c_uint64, C.c_uint64, vp, vp]),
        "avmp_gather_ssm_layers": (C.c_int, [vp, C.c_uint32, C.c_uint32, vp, C.c_uint32, vp, C.c_uint64, vp, C.c_uint64, vp]),
        "avmp_gather_step": (C.c_int, [vp, vp, C.c_uint32, C.c_uint32, C.c_uint32, vp, vp, C.c_uint64, C.c_uint64, vp,
                                       C.c_uint32, C.c_uint32, vp, C.c_uint64, vp, C.c_uint64, vp]),
        "avmp_scatter_kv": (C.c_int, [vp, C.c_uint32, vp, vp, C.c_uint32, vp, vp, vp]),
        "avmp_scatter_ssm": (C.c_int, [vp, C.c_uint32, vp, C.c_uint32, vp, vp, vp]),
        "avmp_scatter_kv_layers": (C.c_int, [vp, C.c_uint32, C.c_uint32, vp, vp, C.c_uint32, vp, vp, C.c_uint64, vp]),
        "avmp_scatter_ssm_layers": (C.c_int, [vp, C.c_uint32, C.c_uint32, vp, C.c_uint32, vp, C.c_uint64, vp, C.c_uint64, vp]),
        "avmp_get_stats": (C.c_int, [vp, C.POINTER(avmp_stats), vp]),
        "avmp_clear_error": (C.c_int, [vp, vp]),
        "avmp_export_tables": (C.c_int, [vp, C.POINTER(avmp_tables), vp]),
        "avmp_import_tables": (C.c_int, [vp, C.POINTER(avmp_tables), vp]),
        "avmp_launch_count": (C.c_uint64, [vp]),
        "avmp_error_string": (C.c_char_p, [C.c_int]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    return L


lib = _load()
LIBRARY_PATH = str(_build.LIB)


class AvmpError(RuntimeError):
    pass


def _check(rc: int, what: str):
    if rc != AVMP_OK:
        raise AvmpError(f"{what}: {lib.avmp_error_string(rc).decode()} ({rc})")


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, torch.Tensor):
        return x.data_ptr()
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return int(x)


def _stream(s) -> Optional[int]:
    if s is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(s, torch.cuda.Stream):
        return s.cuda_stream or None
    return int(s) or None


def model_spec(m) -> avmp_model_spec:
    """From any object with the nine shape fields (e.g. workloads.ModelShape)."""
    return avmp_model_spec(*(int(getattr(m, f[0])) for f in avmp_model_spec._fields_))


def avmp_default_options() -> avmp_options:
    o = avmp_options()
    lib.avmp_default_options(C.byref(o))
    return o


def avmp_derive_layout(spec: avmp_model_spec, pool_bytes: int, initial_split: float) -> avmp_layout:
    out = avmp_layout()
    _check(lib.avmp_derive_layout(C.byref(spec), pool_bytes, float(initial_split), C.byref(out)), "avmp_derive_layout")
    return out


def avmp_workspace_bytes(spec: avmp_model_spec, pool_bytes: int, opt: Optional[avmp_options]) -> int:
    return lib.avmp_workspace_bytes(C.byref(spec), pool_bytes, C.byref(opt) if opt is not None else None)


def avmp_create(spec, d_arena, pool_bytes, initial_split, migration_batch_size, opt, d_workspace,
                workspace_bytes, stream=None) -> int:
    h = C.c_void_p()
    _check(lib.avmp_create(C.byref(h), C.byref(spec), _ptr(d_arena), pool_bytes, float(initial_split),
                           migration_batch_size, C.byref(opt) if opt is not None else None,
                           _ptr(d_workspace), workspace_bytes, _stream(stream)), "avmp_create")
    return h.value


def avmp_destroy(ctx):
    _check(lib.avmp_destroy(ctx), "avmp_destroy")


def avmp_step(ctx, d_ops, n_ops, d_status, stream=None):
    _check(lib.avmp_step(ctx, _ptr(d_ops), n_ops, _ptr(d_status), _stream(stream)), "avmp_step")


def avmp_step_translate(ctx, d_ops, n_ops, d_status, d_handles, n_handles, d_pool, d_offset, d_arena_offset=None,
                        stream=None):
    _check(lib.avmp_step_translate(ctx, _ptr(d_ops), n_ops, _ptr(d_status), _ptr(d_handles), n_handles, _ptr(d_pool),
                                   _ptr(d_offset), _ptr(d_arena_offset), _stream(stream)), "avmp_step_translate")


def avmp_step_host(ctx, h_ops, n_ops, h_status, stream=None):
    _check(lib.avmp_step_host(ctx, _ptr(h_ops), n_ops, _ptr(h_status), _stream(stream)), "avmp_step_host")


def avmp_step_indirect(ctx, d_ops, d_n_ops, max_ops, d_status, stream=None):
    _check(lib.avmp_step_indirect(ctx, _ptr(d_ops), _ptr(d_n_ops), max_ops, _ptr(d_status), _stream(stream)),
           "avmp_step_indirect")


def avmp_driver_workspace_bytes(max_requests: int) -> int:
    return lib.avmp_driver_workspace_bytes(max_requests)


def avmp_driver_create(ctx, d_prompt, d_output, n_requests, concurrency, d_workspace, workspace_bytes, stream=None) -> int:
    h = C.c_void_p()
    _check(lib.avmp_driver_create(C.byref(h), ctx, _ptr(d_prompt), _ptr(d_output), n_requests, concurrency,
                                  _ptr(d_workspace), workspace_bytes, _stream(stream)), "avmp_driver_create")
    return h.value


def avmp_driver_destroy(drv):
    _check(lib.avmp_driver_destroy(drv), "avmp_driver_destroy")


def avmp_driver_step(drv, stream=None):
    _check(lib.avmp_driver_step(drv, _stream(stream)), "avmp_driver_step")


def avmp_driver_get_stats(drv, stream=None) -> dict:
    s = avmp_driver_stats()
    _check(lib.avmp_driver_get_stats(drv, C.byref(s), _stream(stream)), "avmp_driver_get_stats")
    return {k: int(getattr(s, k)) for k in DRIVER_STAT_FIELDS}


def avmp_driver_export(drv, max_requests: int, stream=None) -> dict:
    a = {k: np.zeros(max_requests, np.uint32) for k in ("state", "uid", "len", "remaining")}
    _check(lib.avmp_driver_export(drv, _ptr(a["state"]), _ptr(a["uid"]), _ptr(a["len"]), _ptr(a["remaining"]),
                                  _stream(stream)), "avmp_driver_export")
    return a


def avmp_session_driver_workspace_bytes(max_requests: int, n_sessions: int) -> int:
    return lib.avmp_session_driver_workspace_bytes(max_requests, n_sessions)


def avmp_session_driver_create(ctx, d_arrival_step, d_n_turns, d_turn_prompt, d_turn_output, d_turn_think,
                               n_sessions, max_turns, concurrency, d_workspace, workspace_bytes, stream=None) -> int:
    h = C.c_void_p()
    _check(lib.avmp_session_driver_create(C.byref(h), ctx, _ptr(d_arrival_step), _ptr(d_n_turns), _ptr(d_turn_prompt),
                                          _ptr(d_turn_output), _ptr(d_turn_think), n_sessions, max_turns, concurrency,
                                          _ptr(d_workspace), workspace_bytes, _stream(stream)),
           "avmp_session_driver_create")
    return h.value


def avmp_session_driver_destroy(drv):
    _check(lib.avmp_session_driver_destroy(drv), "avmp_session_driver_destroy")


def avmp_session_driver_step(drv, stream=None):
    _check(lib.avmp_session_driver_step(drv, _stream(stream)), "avmp_session_driver_step")


def avmp_session_driver_get_stats(drv, stream=None) -> dict:
    s = avmp_session_stats()
    _check(lib.avmp_session_driver_get_stats(drv, C.byref(s), _stream(stream)), "avmp_session_driver_get_stats")
    return {k: int(getattr(s, k)) for k in SESSION_STAT_FIELDS}


def avmp_session_driver_export(drv, max_requests: int, n_sessions: int, stream=None) -> dict:
    a = {k: np.zeros(max_requests, np.uint32) for k in ("state", "uid", "len", "remaining", "turn")}
    a["requeued"] = np.zeros(n_sessions, np.uint32)
    a["waiting"] = np.zeros(n_sessions, np.uint32)
    _check(lib.avmp_session_driver_export(drv, _ptr(a["state"]), _ptr(a["uid"]), _ptr(a["len"]), _ptr(a["remaining"]),
                                          _ptr(a["turn"]), _ptr(a["requeued"]), _ptr(a["waiting"]), _stream(stream)),
           "avmp_session_driver_export")
    return a


def avmp_translate(ctx, d_handles, n, d_pool, d_offset, d_arena_offset=None, stream=None):
    _check(lib.avmp_translate(ctx, _ptr(d_handles), n, _ptr(d_pool), _ptr(d_offset), _ptr(d_arena_offset),
                              _stream(stream)), "avmp_translate")


def avmp_gather_kv(ctx, attn_layer, d_reqs, n_reqs, d_out_k, d_out_v, out_capacity_tokens, d_cu_seqlens, stream=None):
    _check(lib.avmp_gather_kv(ctx, attn_layer, _ptr(d_reqs), n_reqs, _ptr(d_out_k), _ptr(d_out_v),
                              out_capacity_tokens, _ptr(d_cu_seqlens), _stream(stream)), "avmp_gather_kv")


def avmp_gather_kv_static(ctx, attn_layer, d_reqs, n_reqs, d_out_k, d_out_v, out_capacity_tokens, d_cu_seqlens,
                          stream=None):
    """avmp_gather_kv with the planning scratch inside the library (nothing lent, nothing allocated)."""
    _check(lib.avmp_gather_kv_static(ctx, attn_layer, _ptr(d_reqs), n_reqs, _ptr(d_out_k), _ptr(d_out_v),
                                     out_capacity_tokens, _ptr(d_cu_seqlens), _stream(stream)),
           "avmp_gather_kv_static")


def avmp_gather_ssm(ctx, ssm_layer, d_reqs, n_reqs, d_out_state, d_out_conv, stream=None):
    _check(lib.avmp_gather_ssm(ctx, ssm_layer, _ptr(d_reqs), n_reqs, _ptr(d_out_state), _ptr(d_out_conv),
                               _stream(stream)), "avmp_gather_ssm")


def avmp_gather_kv_layers(ctx, first_layer, n_layers, d_reqs, n_reqs, d_out_k, d_out_v, layer_stride_bytes,
                          out_capacity_tokens, d_cu_seqlens, stream=None):
    _check(lib.avmp_gather_kv_layers(ctx, first_layer, n_layers, _ptr(d_reqs), n_reqs, _ptr(d_out_k), _ptr(d_out_v),
                                     layer_stride_bytes, out_capacity_tokens, _ptr(d_cu_seqlens), _stream(stream)),
           "avmp_gather_kv_layers")


def avmp_gather_ssm_layers(ctx, first_layer, n_layers, d_reqs, n_reqs, d_out_state, state_layer_stride_bytes,
                           d_out_conv, conv_layer_stride_bytes, stream=None):
    _check(lib.avmp_gather_ssm_layers(ctx, first_layer, n_layers, _ptr(d_reqs), n_reqs, _ptr(d_out_state),
                                      state_layer_stride_bytes, _ptr(d_out_conv), conv_layer_stride_bytes,
                                      _stream(stream)), "avmp_gather_ssm_layers")


def avmp_gather_step(ctx, d_reqs, n_reqs, first_attn_layer, n_attn_layers, d_out_k, d_out_v, kv_layer_stride_bytes,
                     out_capacity_tokens, d_cu_seqlens, first_ssm_layer, n_ssm_layers, d_out_state,
                     state_layer_stride_bytes, d_out_conv, conv_layer_stride_bytes, stream=None):
    _check(lib.avmp_gather_step(ctx, _ptr(d_reqs), n_reqs, first_attn_layer, n_attn_layers, _ptr(d_out_k), _ptr(d_out_v),
                                kv_layer_stride_bytes, out_capacity_tokens, _ptr(d_cu_seqlens), first_ssm_layer,
                                n_ssm_layers, _ptr(d_out_state), state_layer_stride_bytes, _ptr(d_out_conv),
                                conv_layer_stride_bytes, _stream(stream)), "avmp_gather_step")


def avmp_scatter_kv(ctx, attn_layer, d_reqs, d_tok_start, n_reqs, d_in_k, d_in_v, stream=None):
    _check(lib.avmp_scatter_kv(ctx, attn_layer, _ptr(d_reqs), _ptr(d_tok_start), n_reqs, _ptr(d_in_k),
                               _ptr(d_in_v), _stream(stream)), "avmp_scatter_kv")


def avmp_scatter_ssm(ctx, ssm_layer, d_reqs, n_reqs, d_in_state, d_in_conv, stream=None):
    _check(lib.avmp_scatter_ssm(ctx, ssm_layer, _ptr(d_reqs), n_reqs, _ptr(d_in_state), _ptr(d_in_conv),
                                _stream(stream)), "avmp_scatter_ssm")


def avmp_scatter_kv_layers(ctx, first_layer, n_layers, d_reqs, d_tok_start, n_reqs, d_in_k, d_in_v, layer_stride_bytes,
                           stream=None):
    _check(lib.avmp_scatter_kv_layers(ctx, first_layer, n_layers, _ptr(d_reqs), _ptr(d_tok_start), n_reqs,
                                      _ptr(d_in_k), _ptr(d_in_v), layer_stride_bytes, _stream(stream)),
           "avmp_scatter_kv_layers")


def avmp_scatter_ssm_layers(ctx, first_layer, n_layers, d_reqs, n_reqs, d_in_state, state_layer_stride_bytes,
                            d_in_conv, conv_layer_stride_bytes, stream=None):
    _check(lib.avmp_scatter_ssm_layers(ctx, first_layer, n_layers, _ptr(d_reqs), n_reqs, _ptr(d_in_state),
                                       state_layer_stride_bytes, _ptr(d_in_conv), conv_layer_stride_bytes,
                                       _stream(stream)), "avmp_scatter_ssm_layers")


def avmp_get_stats(ctx, stream=None) -> dict:
    s = avmp_stats()
    _check(lib.avmp_get_stats(ctx, C.byref(s), _stream(stream)), "avmp_get_stats")
    return {k: int(getattr(s, k)) for k in STAT_FIELDS}


def avmp_clear_error(ctx, stream=None):
    _check(lib.avmp_clear_error(ctx, _stream(stream)), "avmp_clear_error")


def avmp_launch_count(ctx) -> int:
    return int(lib.avmp_launch_count(ctx))


def _table_arrays(layout: avmp_layout, opt: avmp_options, n_ssm_layers: int):
    R, MP = opt.max_requests, opt.max_pages_per_request
    a = {}
    for p, nm in enumerate(("kv", "ssm")):
        v = int(layout.vid_space[p])
        for t in ("slot_stack", "vid_stack", "vt", "ow"):
            a[f"{t}_{nm}"] = np.zeros(max(v, 1), np.uint32)
    a["req_state"] = np.zeros(R, np.uint32)
    a["req_len"] = np.zeros(R, np.uint32)
    a["req_npages"] = np.zeros(R, np.uint32)
    a["req_chain"] = np.zeros(R * MP, np.uint32)
    a["req_ssm"] = np.zeros(max(R * n_ssm_layers, 1), np.uint32)
    return a


def _tables_struct(a: dict) -> avmp_tables:
    t = avmp_tables()
    p32 = lambda x: x.ctypes.data_as(_u32p)
    for p, nm in enumerate(("kv", "ssm")):
        t.slot_stack[p] = p32(a[f"slot_stack_{nm}"]); t.vid_stack[p] = p32(a[f"vid_stack_{nm}"])
        t.vt[p] = p32(a[f"vt_{nm}"]); t.ow[p] = p32(a[f"ow_{nm}"])
    for k in ("req_state", "req_len", "req_npages", "req_chain", "req_ssm"):
        setattr(t, k, p32(a[k]))
    return t


def avmp_export_tables(ctx, layout: avmp_layout, opt: avmp_options, n_ssm_layers: int, stream=None):
    """-> (tables dict of numpy arrays trimmed to their valid counts, stats dict)."""
    a = _table_arrays(layout, opt, n_ssm_layers)
    t = _tables_struct(a)
    _check(lib.avmp_export_tables(ctx, C.byref(t), _stream(stream)), "avmp_export_tables")
    for p, nm in enumerate(("kv", "ssm")):
        v = int(layout.vid_space[p])
        a[f"slot_stack_{nm}"] = a[f"slot_stack_{nm}"][: t.n_slot_stack[p]]
        a[f"vid_stack_{nm}"] = a[f"vid_stack_{nm}"][: t.n_vid_stack[p]]
        a[f"vt_{nm}"] = a[f"vt_{nm}"][:v]
        a[f"ow_{nm}"] = a[f"ow_{nm}"][:v]
    a["req_ssm"] = a["req_ssm"][: opt.max_requests * n_ssm_layers]
    return a, {k: int(getattr(t.stats, k)) for k in STAT_FIELDS}


def avmp_import_tables(ctx, layout: avmp_layout, opt: avmp_options, n_ssm_layers: int, tables: dict,
                       stats: dict, stream=None):
    """Load tables (as returned by export, or built elsewhere in the same format)."""
    a = _table_arrays(layout, opt, n_ssm_layers)
    for k, v in tables.items():
        a[k][: len(v)] = v
    t = _tables_struct(a)
    for p, nm in enumerate(("kv", "ssm")):
        t.n_slot_stack[p] = len(tables[f"slot_stack_{nm}"])
        t.n_vid_stack[p] = len(tables[f"vid_stack_{nm}"])
    for k in STAT_FIELDS:
        setattr(t.stats, k, int(stats.get(k, 0)))
    _check(lib.avmp_import_tables(ctx, C.byref(t), _stream(stream)), "avmp_import_tables")


class Context:
    """Convenience owner: allocates arena and workspace as torch tensors and keeps the
    handle.  Every method forwards to the C ABI function of the same name."""

    def __init__(self, model, pool_bytes: int, initial_split: float, migration_batch_size: int, *,
                 max_requests: int, max_pages: int, threshold_low_ppm: int = 50_000,
                 threshold_high_ppm: int = 300_000, min_rebalance_interval_ops: int = 1000,
                 migration_enabled: bool = True, reclaim_gap: bool = False, device="cuda:0",
                 arena: Optional[torch.Tensor] = None):
        if not torch.cuda.is_available():
            raise AvmpError("AVMP needs a CUDA device; there is no CPU path")
        self.device = torch.device(device)
        self.model = model
        self.spec = model_spec(model)
        self.opt = avmp_options(threshold_low_ppm, threshold_high_ppm, min_rebalance_interval_ops,
                                int(migration_enabled), max_requests, max_pages, int(reclaim_gap))
        self.pool_bytes = pool_bytes
        self.layout = avmp_derive_layout(self.spec, pool_bytes, initial_split)
        ws = avmp_workspace_bytes(self.spec, pool_bytes, self.opt)
        if ws == 0:
            raise AvmpError("avmp_workspace_bytes rejected the configuration")
        with torch.cuda.device(self.device):
            self._owns_arena = arena is None
            self.arena = arena if arena is not None else torch.empty(pool_bytes, dtype=torch.uint8, device=self.device)
            self.workspace = torch.empty(ws, dtype=torch.uint8, device=self.device)
            self.handle = avmp_create(self.spec, self.arena, pool_bytes, initial_split, migration_batch_size,
                                      self.opt, self.workspace, ws)

    @classmethod
    def from_workload(cls, w, **over):
        kw = dict(max_requests=w.max_requests, max_pages=w.max_pages,
                  threshold_low_ppm=w.threshold_low_ppm, threshold_high_ppm=w.threshold_high_ppm,
                  min_rebalance_interval_ops=w.min_rebalance_interval_ops, migration_enabled=w.migration_enabled,
                  reclaim_gap=w.reclaim_gap)
        kw.update(over)
        return cls(w.model, w.pool_bytes, w.split, w.migration_batch_size, **kw)

    def close(self):
        if getattr(self, "handle", None):
            torch.cuda.synchronize(self.device)
            avmp_destroy(self.handle)
            self.handle = None
            # drop the device memory this object allocated, so that the next context fits
            self.workspace = None
            if self._owns_arena:
                self.arena = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def step(self, d_ops, n_ops, d_status, stream=None):
        avmp_step(self.handle, d_ops, n_ops, d_status, stream)

    def step_translate(self, d_ops, n_ops, d_status, d_handles, n_handles, d_pool, d_offset, d_arena_offset=None,
                       stream=None):
        avmp_step_translate(self.handle, d_ops, n_ops, d_status, d_handles, n_handles, d_pool, d_offset,
                            d_arena_offset, stream)

    def step_host(self, h_ops, n_ops, h_status, stream=None):
        avmp_step_host(self.handle, h_ops, n_ops, h_status, stream)

    def translate(self, d_handles, n, d_pool, d_offset, d_arena_offset=None, stream=None):
        avmp_translate(self.handle, d_handles, n, d_pool, d_offset, d_arena_offset, stream)

    def gather_kv(self, layer, d_reqs, n, d_out_k, d_out_v, cap_tokens, d_cu, stream=None):
        avmp_gather_kv(self.handle, layer, d_reqs, n, d_out_k, d_out_v, cap_tokens, d_cu, stream)

    def gather_kv_static(self, layer, d_reqs, n, d_out_k, d_out_v, cap_tokens, d_cu, stream=None):
        avmp_gather_kv_static(self.handle, layer, d_reqs, n, d_out_k, d_out_v, cap_tokens, d_cu, stream)

    def gather_ssm(self, layer, d_reqs, n, d_out_state, d_out_conv, stream=None):
        avmp_gather_ssm(self.handle, layer, d_reqs, n, d_out_state, d_out_conv, stream)

    def gather_kv_layers(self, first_layer, n_layers, d_reqs, n, d_out_k, d_out_v, layer_stride, cap_tokens, d_cu,
                         stream=None):
        avmp_gather_kv_layers(self.handle, first_layer, n_layers, d_reqs, n, d_out_k, d_out_v, layer_stride,
                              cap_tokens, d_cu, stream)

    def gather_ssm_layers(self, first_layer, n_layers, d_reqs, n, d_out_state, state_stride, d_out_conv,
                          conv_stride, stream=None):
        avmp_gather_ssm_layers(self.handle, first_layer, n_layers, d_reqs, n, d_out_state, state_stride,
                               d_out_conv, conv_stride, stream)

    def gather_step(self, d_reqs, n, first_attn_layer, n_attn_layers, d_out_k, d_out_v, kv_layer_stride, cap_tokens, d_cu,
                    first_ssm_layer, n_ssm_layers, d_out_state, state_stride, d_out_conv, conv_stride, stream=None):
        avmp_gather_step(self.handle, d_reqs, n, first_attn_layer, n_attn_layers, d_out_k, d_out_v, kv_layer_stride,
                         cap_tokens, d_cu, first_ssm_layer, n_ssm_layers, d_out_state, state_stride, d_out_conv,
                         conv_stride, stream)

    def scatter_kv(self, layer, d_reqs, d_tok_start, n, d_in_k, d_in_v, stream=None):
        avmp_scatter_kv(self.handle, layer, d_reqs, d_tok_start, n, d_in_k, d_in_v, stream)

    def scatter_kv_layers(self, first_layer, n_layers, d_reqs, d_tok_start, n, d_in_k, d_in_v, layer_stride, stream=None):
        avmp_scatter_kv_layers(self.handle, first_layer, n_layers, d_reqs, d_tok_start, n, d_in_k, d_in_v,
                               layer_stride, stream)

    def scatter_ssm_layers(self, first_layer, n_layers, d_reqs, n, d_in_state, state_stride, d_in_conv, conv_stride,
                           stream=None):
        avmp_scatter_ssm_layers(self.handle, first_layer, n_layers, d_reqs, n, d_in_state, state_stride,
                                d_in_conv, conv_stride, stream)

    def scatter_ssm(self, layer, d_reqs, n, d_in_state, d_in_conv, stream=None):
        avmp_scatter_ssm(self.handle, layer, d_reqs, n, d_in_state, d_in_conv, stream)

    def stats(self, stream=None) -> dict:
        return avmp_get_stats(self.handle, stream)

    def clear_error(self, stream=None):
        avmp_clear_error(self.handle, stream)

    def export_tables(self, stream=None):
        return avmp_export_tables(self.handle, self.layout, self.opt, self.spec.n_ssm_layers, stream)

    def import_tables(self, tables: dict, stats: dict, stream=None):
        avmp_import_tables(self.handle, self.layout, self.opt, self.spec.n_ssm_layers, tables, stats, stream)

    def launch_count(self) -> int:
        return avmp_launch_count(self.handle)


class DeviceDriver:
    """Owner of an on-device closed loop over a Context: uploads the request lengths, allocates the
    driver workspace, forwards to the avmp_driver_* entry points."""

    def __init__(self, ctx: Context, prompt: np.ndarray, output: np.ndarray, concurrency: int):
        self.ctx = ctx
        dev = ctx.device
        self.d_prompt = torch.from_numpy(np.ascontiguousarray(prompt, dtype=np.uint32).view(np.int32)).to(dev)
        self.d_output = torch.from_numpy(np.ascontiguousarray(output, dtype=np.uint32).view(np.int32)).to(dev)
        ws = avmp_driver_workspace_bytes(ctx.opt.max_requests)
        if ws == 0:
            raise AvmpError("avmp_driver_workspace_bytes rejected max_requests")
        with torch.cuda.device(dev):
            self.workspace = torch.empty(ws, dtype=torch.uint8, device=dev)
            self.handle = avmp_driver_create(ctx.handle, self.d_prompt, self.d_output, len(prompt), concurrency,
                                             self.workspace, ws)

    def step(self, stream=None):
        avmp_driver_step(self.handle, stream)

    def stats(self, stream=None) -> dict:
        return avmp_driver_get_stats(self.handle, stream)

    def export(self, stream=None) -> dict:
        return avmp_driver_export(self.handle, self.ctx.opt.max_requests, stream)

    def close(self):
        if getattr(self, "handle", None):
            torch.cuda.synchronize(self.ctx.device)
            avmp_driver_destroy(self.handle)
            self.handle = None
            self.workspace = self.d_prompt = self.d_output = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class SessionDriver:
    """Owner of the on-device closed loop for multi-turn sessions: uploads the session arrays
    (arrival step, turns, per-turn prompt / output / think time), allocates the workspace, forwards
    to the avmp_session_driver_* entry points."""

    def __init__(self, ctx: Context, arrival_step, n_turns, turn_prompt, turn_output, turn_think, concurrency: int):
        self.ctx = ctx
        dev = ctx.device
        self.n_sessions = len(arrival_step)
        self.max_turns = int(np.asarray(turn_prompt).shape[1])

        def up(a):
            return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint32).view(np.int32).reshape(-1)).to(dev)

        self.arrays = [up(a) for a in (arrival_step, n_turns, turn_prompt, turn_output, turn_think)]
        ws = avmp_session_driver_workspace_bytes(ctx.opt.max_requests, self.n_sessions)
        if ws == 0:
            raise AvmpError("avmp_session_driver_workspace_bytes rejected the sizes")
        with torch.cuda.device(dev):
            self.workspace = torch.empty(ws, dtype=torch.uint8, device=dev)
            self.handle = avmp_session_driver_create(ctx.handle, *self.arrays, self.n_sessions, self.max_turns,
                                                     concurrency, self.workspace, ws)

    def step(self, stream=None):
        avmp_session_driver_step(self.handle, stream)

    def stats(self, stream=None) -> dict:
        return avmp_session_driver_get_stats(self.handle, stream)

    def export(self, stream=None) -> dict:
        s = self.stats(stream)
        a = avmp_session_driver_export(self.handle, self.ctx.opt.max_requests, self.n_sessions, stream)
        a["requeued"] = a["requeued"][:s["requeued"]]
        a["waiting"] = a["waiting"][:s["waiting"]]
        return a

    def close(self):
        if getattr(self, "handle", None):
            torch.cuda.synchronize(self.ctx.device)
            avmp_session_driver_destroy(self.handle)
            self.handle = None
            self.workspace = self.arrays = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
