"""ctypes wrapper around the C oracle -- TEST INFRASTRUCTURE, not a product path.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this.
It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_DIR = Path(__file__).resolve().parent
_SO = _DIR / "libavmp_oracle.so"
_SRC = [_DIR / "avmp_oracle.c", _DIR / "avmp_oracle.h"]

INVALID = 0xFFFFFFFF
NONE64 = 0xFFFFFFFFFFFFFFFF
KV, SSM = 0, 1

STAT_FIELDS = (
    "op_counter", "last_rebalance_op", "n_oom", "n_capacity_error", "n_rebalance",
    "migrated_bytes", "wasted_bytes", "relocated_blocks", "relocated_bytes", "gap_bytes",
    "cap_kv", "cap_ssm", "free_kv", "free_ssm", "fsm_state", "n_invalid",
    "unit_bytes_kv", "unit_bytes_ssm", "vid_space_kv", "vid_space_ssm", "pool_bytes_aligned",
)
TABLES = (
    "slot_stack_kv", "slot_stack_ssm", "vid_stack_kv", "vid_stack_ssm",
    "vt_kv", "vt_ssm", "ow_kv", "ow_ssm",
    "req_state", "req_len", "req_npages", "req_chain", "req_ssm",
)


class _Model(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in (
        "n_attn_layers", "n_ssm_layers", "page_tokens", "kv_heads", "head_dim", "kv_elem_bytes",
        "ssm_state_elems", "ssm_conv_elems", "ssm_elem_bytes")]


class _Options(C.Structure):
    _fields_ = [("threshold_low_ppm", C.c_uint32), ("threshold_high_ppm", C.c_uint32),
                ("min_rebalance_interval_ops", C.c_uint64), ("migration_enabled", C.c_uint32),
                ("max_requests", C.c_uint32), ("max_pages_per_request", C.c_uint32),
                ("reclaim_gap", C.c_uint32)]


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (plain C11, -O2, no CUDA)."""
    newest = max(p.stat().st_mtime for p in _SRC)
    if force or not _SO.exists() or _SO.stat().st_mtime < newest:
        tmp = _SO.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(["gcc", "-std=c11", "-O2", "-fPIC", "-shared", "-Wall", "-Wextra",
                               "-o", str(tmp), str(_SRC[0]), "-lm"])
        os.replace(tmp, _SO)
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(str(_SO))
        vp, u32p, u64p = C.c_void_p, C.POINTER(C.c_uint32), C.POINTER(C.c_uint64)
        L.orc_create.restype = vp
        L.orc_create.argtypes = [C.POINTER(_Model), C.c_uint64, C.c_double, C.c_uint32,
                                 C.POINTER(_Options), C.c_int]
        L.orc_destroy.argtypes = [vp]
        L.orc_step.argtypes = [vp, vp, C.c_uint32, vp]
        L.orc_translate.restype = C.c_uint32
        L.orc_translate.argtypes = [vp, vp, C.c_uint32, vp, vp]
        L.orc_gather_kv.restype = C.c_uint32
        L.orc_gather_kv.argtypes = [vp, C.c_uint32, vp, C.c_uint32, vp, vp, C.c_uint64, vp]
        L.orc_gather_ssm.restype = C.c_uint32
        L.orc_gather_ssm.argtypes = [vp, C.c_uint32, vp, C.c_uint32, vp, vp]
        L.orc_scatter_kv.restype = C.c_uint32
        L.orc_scatter_kv.argtypes = [vp, C.c_uint32, vp, vp, C.c_uint32, vp, vp]
        L.orc_scatter_ssm.restype = C.c_uint32
        L.orc_scatter_ssm.argtypes = [vp, C.c_uint32, vp, C.c_uint32, vp, vp]
        L.orc_get_stats.argtypes = [vp, vp]
        L.orc_store_bytes.restype = C.POINTER(C.c_uint8)
        L.orc_store_bytes.argtypes = [vp, C.c_int, C.c_uint64, C.c_uint64]
        L.orc_table.restype = u32p
        L.orc_table.argtypes = [vp, C.c_int, u64p]
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


class Oracle:
    """One sequential AVMP allocator with optional payload stores."""

    def __init__(self, model, pool_bytes: int, split: float, migration_batch_size: int, *,
                 max_requests: int, max_pages: int, threshold_low_ppm: int = 50_000,
                 threshold_high_ppm: int = 300_000, min_rebalance_interval_ops: int = 1000,
                 migration_enabled: bool = True, reclaim_gap: bool = False, with_store: bool = False):
        self.model = model
        m = _Model(*(int(getattr(model, f[0])) for f in _Model._fields_))
        o = _Options(threshold_low_ppm, threshold_high_ppm, min_rebalance_interval_ops,
                     int(migration_enabled), max_requests, max_pages, int(reclaim_gap))
        self.max_requests, self.max_pages = max_requests, max_pages
        self._h = lib().orc_create(C.byref(m), pool_bytes, float(split), migration_batch_size,
                                   C.byref(o), int(with_store))
        if not self._h:
            raise ValueError("orc_create rejected the configuration")

    @classmethod
    def from_workload(cls, w, with_store: bool = False, **over):
        kw = dict(max_requests=w.max_requests, max_pages=w.max_pages,
                  threshold_low_ppm=w.threshold_low_ppm, threshold_high_ppm=w.threshold_high_ppm,
                  min_rebalance_interval_ops=w.min_rebalance_interval_ops,
                  migration_enabled=w.migration_enabled, reclaim_gap=w.reclaim_gap, with_store=with_store)
        kw.update(over)
        return cls(w.model, w.pool_bytes, w.split, w.migration_batch_size, **kw)

    def close(self):
        if self._h:
            lib().orc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def step(self, ops: np.ndarray) -> np.ndarray:
        ops = np.ascontiguousarray(ops)
        assert ops.dtype.itemsize == 12
        st = np.empty(len(ops), dtype=np.uint32)
        if len(ops):
            lib().orc_step(self._h, _ptr(ops), len(ops), _ptr(st))
        return st

    def translate(self, handles: np.ndarray):
        h = np.ascontiguousarray(handles, dtype=np.uint32)
        pool = np.empty(len(h), np.uint32)
        off = np.empty(len(h), np.uint64)
        bad = lib().orc_translate(self._h, _ptr(h), len(h), _ptr(pool), _ptr(off)) if len(h) else 0
        return pool, off, bad

    def gather_kv(self, layer: int, reqs: np.ndarray, capacity_tokens: int):
        r = np.ascontiguousarray(reqs, dtype=np.uint32)
        row = self.model.kv_row_bytes
        out_k = np.zeros((capacity_tokens, row), np.uint8)
        out_v = np.zeros((capacity_tokens, row), np.uint8)
        cu = np.zeros(len(r) + 1, np.uint32)
        bad = lib().orc_gather_kv(self._h, layer, _ptr(r), len(r), _ptr(out_k), _ptr(out_v),
                                  capacity_tokens, _ptr(cu))
        return out_k, out_v, cu, bad

    def gather_ssm(self, layer: int, reqs: np.ndarray):
        r = np.ascontiguousarray(reqs, dtype=np.uint32)
        st = np.zeros((len(r), self.model.state_bytes), np.uint8)
        cv = np.zeros((len(r), self.model.conv_bytes), np.uint8)
        bad = lib().orc_gather_ssm(self._h, layer, _ptr(r), len(r), _ptr(st), _ptr(cv))
        return st, cv, bad

    def scatter_kv(self, layer: int, reqs, tok_start, in_k: np.ndarray, in_v: np.ndarray) -> int:
        r = np.ascontiguousarray(reqs, dtype=np.uint32)
        t0 = np.ascontiguousarray(tok_start, dtype=np.uint32)
        in_k, in_v = np.ascontiguousarray(in_k), np.ascontiguousarray(in_v)
        return lib().orc_scatter_kv(self._h, layer, _ptr(r), _ptr(t0), len(r), _ptr(in_k), _ptr(in_v))

    def scatter_ssm(self, layer: int, reqs, in_state: np.ndarray, in_conv: np.ndarray) -> int:
        r = np.ascontiguousarray(reqs, dtype=np.uint32)
        in_state, in_conv = np.ascontiguousarray(in_state), np.ascontiguousarray(in_conv)
        return lib().orc_scatter_ssm(self._h, layer, _ptr(r), len(r), _ptr(in_state), _ptr(in_conv))

    def stats(self) -> dict:
        buf = np.zeros(len(STAT_FIELDS), np.uint64)
        lib().orc_get_stats(self._h, _ptr(buf))
        return {k: int(v) for k, v in zip(STAT_FIELDS, buf)}

    def store_bytes(self, pool: int, offset: int, n: int) -> np.ndarray:
        """Copy of n raw bytes of a store, starting at a byte offset inside that store."""
        p = lib().orc_store_bytes(self._h, pool, offset, n)
        if not p:
            raise ValueError("no payload store, or the range leaves the store")
        return np.ctypeslib.as_array(p, shape=(n,)).copy()

    def table(self, name: str) -> np.ndarray:
        cnt = C.c_uint64(0)
        p = lib().orc_table(self._h, TABLES.index(name), C.byref(cnt))
        if cnt.value == 0:
            return np.zeros(0, np.uint32)
        return np.ctypeslib.as_array(p, shape=(cnt.value,)).copy()

    def tables(self) -> dict:
        return {n: self.table(n) for n in TABLES}
