"""numpy-in / numpy-out adapter around the CUDA binding, with the same method names as the
oracle wrapper, so the same test harness can drive both.  Test code only: it moves arrays
to and from the device and calls the C ABI; it computes nothing."""
from __future__ import annotations

import numpy as np
import torch

from paper_2605_22416_b200 import binding as B


class GpuEngine:
    def __init__(self, w, device="cuda:0", **over):
        self.w = w
        self.dev = torch.device(device)
        self.ctx = B.Context.from_workload(w, device=device, **over)
        self.model = w.model
        self.max_pages = self.ctx.opt.max_pages_per_request

    def close(self):
        self.ctx.close()

    def _dev(self, a: np.ndarray, dtype=None) -> torch.Tensor:
        a = np.ascontiguousarray(a if dtype is None else np.asarray(a, dtype=dtype))
        if a.size == 0:
            return torch.zeros(16, dtype=torch.uint8, device=self.dev)
        return torch.from_numpy(a.view(np.uint8).reshape(-1)).to(self.dev)

    def step(self, ops: np.ndarray) -> np.ndarray:
        n = len(ops)
        if n == 0:
            self.ctx.step(0, 0, 0)
            return np.zeros(0, np.uint32)
        d_ops = self._dev(ops)
        d_st = torch.full((n,), 0xEE, dtype=torch.int32, device=self.dev)
        self.ctx.step(d_ops, n, d_st)
        return d_st.cpu().numpy().view(np.uint32)

    def step_translate(self, ops: np.ndarray, handles):
        """avmp_step_translate -> (statuses, pool, offset, error items, arena offset)."""
        h = np.ascontiguousarray(handles, dtype=np.uint32)
        n, nh = len(ops), len(h)
        d_st = torch.full((max(n, 1),), 0xEE, dtype=torch.int32, device=self.dev)
        pool = torch.zeros(max(nh, 1), dtype=torch.int32, device=self.dev)
        off = torch.zeros(max(nh, 1), dtype=torch.int64, device=self.dev)
        aoff = torch.zeros(max(nh, 1), dtype=torch.int64, device=self.dev)
        before = self.ctx.stats()["error_count"]
        self.ctx.step_translate(self._dev(ops), n, d_st, self._dev(h), nh, pool, off, aoff)
        bad = self.ctx.stats()["error_count"] - before
        return (d_st.cpu().numpy().view(np.uint32)[:n], pool.cpu().numpy().view(np.uint32)[:nh],
                off.cpu().numpy().view(np.uint64)[:nh], bad, aoff.cpu().numpy().view(np.uint64)[:nh])

    def step_host(self, ops: np.ndarray) -> np.ndarray:
        ops = np.ascontiguousarray(ops)
        st = np.full(len(ops), 0xEE, np.uint32)
        self.ctx.step_host(ops, len(ops), st)
        return st

    def translate(self, handles):
        h = np.ascontiguousarray(handles, dtype=np.uint32)
        n = len(h)
        d_h = self._dev(h)
        pool = torch.zeros(max(n, 1), dtype=torch.int32, device=self.dev)
        off = torch.zeros(max(n, 1), dtype=torch.int64, device=self.dev)
        aoff = torch.zeros(max(n, 1), dtype=torch.int64, device=self.dev)
        before = self.ctx.stats()["error_count"]
        self.ctx.translate(d_h, n, pool, off, aoff)
        bad = self.ctx.stats()["error_count"] - before
        return (pool.cpu().numpy().view(np.uint32)[:n], off.cpu().numpy().view(np.uint64)[:n], bad,
                aoff.cpu().numpy().view(np.uint64)[:n])

    def gather_kv(self, layer, reqs, capacity_tokens):
        r = np.ascontiguousarray(reqs, dtype=np.uint32)
        row = self.model.kv_row_bytes
        out_k = torch.zeros((max(capacity_tokens, 1), row), dtype=torch.uint8, device=self.dev)
        out_v = torch.zeros((max(capacity_tokens, 1), row), dtype=torch.uint8, device=self.dev)
        cu = torch.zeros(len(r) + 1, dtype=torch.int32, device=self.dev)
        before = self.ctx.stats()["error_count"]
        self.ctx.gather_kv(layer, self._dev(r), len(r), out_k, out_v, capacity_tokens, cu)
        bad = self.ctx.stats()["error_count"] - before
        return (out_k.cpu().numpy()[:capacity_tokens], out_v.cpu().numpy()[:capacity_tokens],
                cu.cpu().numpy().view(np.uint32), bad)

    def gather_ssm(self, layer, reqs):
        r = np.ascontiguousarray(reqs, dtype=np.uint32)
        n = len(r)
        st = torch.zeros((max(n, 1), self.model.state_bytes), dtype=torch.uint8, device=self.dev)
        cv = torch.zeros((max(n, 1), self.model.conv_bytes), dtype=torch.uint8, device=self.dev)
        before = self.ctx.stats()["error_count"]
        self.ctx.gather_ssm(layer, self._dev(r), n, st, cv)
        bad = self.ctx.stats()["error_count"] - before
        return st.cpu().numpy()[:n], cv.cpu().numpy()[:n], bad

    def gather_kv_layers(self, first, n_layers, reqs, capacity_tokens):
        r = np.ascontiguousarray(reqs, dtype=np.uint32)
        row = self.model.kv_row_bytes
        cap = max(capacity_tokens, 1)
        out_k = torch.zeros((n_layers, cap, row), dtype=torch.uint8, device=self.dev)
        out_v = torch.zeros((n_layers, cap, row), dtype=torch.uint8, device=self.dev)
        cu = torch.zeros(len(r) + 1, dtype=torch.int32, device=self.dev)
        self.ctx.gather_kv_layers(first, n_layers, self._dev(r), len(r), out_k, out_v, cap * row, capacity_tokens, cu)
        return out_k.cpu().numpy(), out_v.cpu().numpy(), cu.cpu().numpy().view(np.uint32)

    def gather_ssm_layers(self, first, n_layers, reqs):
        r = np.ascontiguousarray(reqs, dtype=np.uint32)
        n = max(len(r), 1)
        st = torch.zeros((n_layers, n, self.model.state_bytes), dtype=torch.uint8, device=self.dev)
        cv = torch.zeros((n_layers, n, self.model.conv_bytes), dtype=torch.uint8, device=self.dev)
        self.ctx.gather_ssm_layers(first, n_layers, self._dev(r), len(r), st, n * self.model.state_bytes,
                                   cv, n * self.model.conv_bytes)
        return st.cpu().numpy(), cv.cpu().numpy()

    def gather_step(self, kv_first, kv_n, ssm_first, ssm_n, reqs, capacity_tokens):
        """Both gathers in one launch -> (K [kv_n][cap][row], V, cu_seqlens, state [ssm_n][n][..], conv, error items).
        Layer strides are rounded up to the 16 bytes the entry point asks for."""
        r = np.ascontiguousarray(reqs, dtype=np.uint32)
        m = self.model
        row, n, cap = m.kv_row_bytes, max(len(r), 1), max(capacity_tokens, 1)
        up = lambda x: (x + 15) // 16 * 16
        ks, ss, cs = up(cap * row), up(n * m.state_bytes), up(n * m.conv_bytes)
        out_k = torch.zeros((kv_n, ks), dtype=torch.uint8, device=self.dev)
        out_v = torch.zeros((kv_n, ks), dtype=torch.uint8, device=self.dev)
        cu = torch.zeros(len(r) + 1, dtype=torch.int32, device=self.dev)
        st = torch.zeros((ssm_n, ss), dtype=torch.uint8, device=self.dev)
        cv = torch.zeros((ssm_n, cs), dtype=torch.uint8, device=self.dev)
        before = self.ctx.stats()["error_count"]
        self.ctx.gather_step(self._dev(r), len(r), kv_first, kv_n, out_k, out_v, ks, capacity_tokens, cu,
                             ssm_first, ssm_n, st, ss, cv, cs)
        bad = self.ctx.stats()["error_count"] - before
        return (out_k.cpu().numpy()[:, :cap * row].reshape(kv_n, cap, row), out_v.cpu().numpy()[:, :cap * row].reshape(kv_n, cap, row),
                cu.cpu().numpy().view(np.uint32), st.cpu().numpy()[:, :n * m.state_bytes].reshape(ssm_n, n, m.state_bytes),
                cv.cpu().numpy()[:, :n * m.conv_bytes].reshape(ssm_n, n, m.conv_bytes), bad)

    def scatter_kv(self, layer, reqs, tok_start, in_k, in_v) -> int:
        r = np.ascontiguousarray(reqs, dtype=np.uint32)
        before = self.ctx.stats()["error_count"]
        self.ctx.scatter_kv(layer, self._dev(r), self._dev(tok_start, np.uint32), len(r),
                            self._dev(in_k), self._dev(in_v))
        return self.ctx.stats()["error_count"] - before

    def scatter_ssm(self, layer, reqs, in_state, in_conv) -> int:
        r = np.ascontiguousarray(reqs, dtype=np.uint32)
        before = self.ctx.stats()["error_count"]
        self.ctx.scatter_ssm(layer, self._dev(r), len(r), self._dev(in_state), self._dev(in_conv))
        return self.ctx.stats()["error_count"] - before

    def stats(self) -> dict:
        return self.ctx.stats()

    def tables(self) -> dict:
        return self.ctx.export_tables()[0]


def comparable_tables(t: dict, max_requests: int, max_pages: int, n_ssm_layers: int) -> dict:
    """Tables reduced to what is defined: chains up to n_pages, SSM handles of LIVE slots."""
    out = {k: v for k, v in t.items() if not k.startswith("req_chain") and not k.startswith("req_ssm")}
    npg = t["req_npages"]
    chain = t["req_chain"].reshape(max_requests, max_pages)
    mask = np.arange(max_pages)[None, :] < npg[:, None]
    out["req_chain"] = np.where(mask, chain, 0)
    if n_ssm_layers:
        ssm = t["req_ssm"].reshape(max_requests, n_ssm_layers)
        out["req_ssm"] = np.where((t["req_state"] == 1)[:, None], ssm, 0)
    return out


def assert_same_state(gpu, oracle, w, what=""):
    gs, os_ = gpu.stats(), oracle.stats()
    for k, v in os_.items():
        assert gs[k] == v, f"{what}: stat {k}: gpu {gs[k]} != oracle {v}"
    gt = comparable_tables(gpu.tables(), gpu.ctx.opt.max_requests, gpu.max_pages, w.model.n_ssm_layers)
    ot = comparable_tables(oracle.tables(), oracle.max_requests, oracle.max_pages, w.model.n_ssm_layers)
    for k in ot:
        assert np.array_equal(gt[k], ot[k]), f"{what}: table {k} differs"
