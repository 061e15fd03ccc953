"""Test-side plumbing shared by the oracle tests and the GPU parity tests: writes the
payload a model would produce into an engine's stores and checks gathers against the
payload function.  `engine` is anything with step / scatter_kv / scatter_ssm /
gather_kv / gather_ssm taking and returning numpy arrays (the oracle wrapper, or the
numpy adapter around the CUDA binding)."""
from __future__ import annotations

from typing import Iterable, List, Sequence

import numpy as np

from paper_2605_22416_b200 import workloads as W


class PayloadHarness:
    def __init__(self, w: W.Workload, engines: Sequence, seed: int = 77,
                 kv_layers: Iterable[int] = None, ssm_layers: Iterable[int] = None):
        self.w, self.engines, self.seed = w, list(engines), seed
        m = w.model
        self.kv_layers = list(range(m.n_attn_layers)) if kv_layers is None else list(kv_layers)
        self.ssm_layers = list(range(m.n_ssm_layers)) if ssm_layers is None else list(ssm_layers)

    # -- what the model writes after a step -------------------------------------------
    def apply_writes(self, writes: List[W.TokenWrite]) -> None:
        if not writes:
            return
        m = self.w.model
        slots = np.array([x.slot for x in writes], np.uint32)
        starts = np.array([x.start for x in writes], np.uint32)
        # single-token writes (the EXTENDs) first, in one pass; the scatter order is free
        one = [i for i, x in enumerate(writes) if x.end - x.start == 1]
        many = [i for i, x in enumerate(writes) if x.end - x.start != 1]
        order = one + many
        slots, starts = slots[order], starts[order]
        u1 = [writes[i].uid for i in one]
        r1 = [writes[i].start for i in one]
        for layer in self.kv_layers:
            parts = []
            for part in (W.PAYLOAD_K, W.PAYLOAD_V):
                rows = [W.payload_single_rows(self.seed, u1, [0] * len(u1), layer, part, r1, m.kv_row_bytes)]
                rows += [W.payload_bytes(self.seed, writes[i].uid, 0, layer, part, writes[i].start,
                                         writes[i].end - writes[i].start, m.kv_row_bytes) for i in many]
                parts.append(np.concatenate(rows))
            for e in self.engines:
                assert e.scatter_kv(layer, slots, starts, parts[0], parts[1]) == 0
        adm = [x for x in writes if x.is_admit]
        if adm:
            aslots = np.array([x.slot for x in adm], np.uint32)
            for layer in self.ssm_layers:
                au, ae, z = [x.uid for x in adm], [x.epoch for x in adm], [0] * len(adm)
                st = W.payload_single_rows(self.seed, au, ae, layer, W.PAYLOAD_STATE, z, m.state_bytes)
                cv = W.payload_single_rows(self.seed, au, ae, layer, W.PAYLOAD_CONV, z, m.conv_bytes)
                for e in self.engines:
                    assert e.scatter_ssm(layer, aslots, st, cv) == 0

    # -- what a gather must return, from (uid, length) alone ----------------------------
    def expected_kv(self, layer: int, uids, lens):
        m = self.w.model
        ks = [W.payload_bytes(self.seed, int(u), 0, layer, W.PAYLOAD_K, 0, int(l), m.kv_row_bytes) for u, l in zip(uids, lens)]
        vs = [W.payload_bytes(self.seed, int(u), 0, layer, W.PAYLOAD_V, 0, int(l), m.kv_row_bytes) for u, l in zip(uids, lens)]
        cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint32)
        z = np.zeros((0, m.kv_row_bytes), np.uint8)
        return np.concatenate(ks or [z]), np.concatenate(vs or [z]), cu

    def expected_ssm(self, layer: int, uids, epochs):
        m = self.w.model
        z = [0] * len(uids)
        return (W.payload_single_rows(self.seed, uids, epochs, layer, W.PAYLOAD_STATE, z, m.state_bytes),
                W.payload_single_rows(self.seed, uids, epochs, layer, W.PAYLOAD_CONV, z, m.conv_bytes))

    def check_gathers(self, d: W.ClosedLoopDriver, kv_layer: int, ssm_layer: int, engines=None) -> int:
        """Gather the whole running batch from every engine and compare with the payload
        function.  Returns the number of tokens checked."""
        run = np.flatnonzero(d.state == 1).astype(np.uint32)
        if len(run) == 0:
            return 0
        lens = d.len[run]
        total = int(lens.sum())
        ek, ev, ecu = self.expected_kv(kv_layer, d.uid[run], lens)
        es, ec = self.expected_ssm(ssm_layer, d.uid[run], d.slot_epoch[run])
        for e in (engines or self.engines):
            k, v, cu, bad = e.gather_kv(kv_layer, run, total)
            assert bad == 0
            assert np.array_equal(cu, ecu)
            assert np.array_equal(k[:total], ek), "gathered K differs from the payload function"
            assert np.array_equal(v[:total], ev), "gathered V differs from the payload function"
            st, cv, bad = e.gather_ssm(ssm_layer, run)
            assert bad == 0
            assert np.array_equal(st, es) and np.array_equal(cv, ec)
        return total
