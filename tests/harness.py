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
        for layer in self.kv_layers:
            ks = [W.payload_bytes(self.seed, x.uid, 0, layer, W.PAYLOAD_K, x.start, x.end - x.start, m.kv_row_bytes) for x in writes]
            vs = [W.payload_bytes(self.seed, x.uid, 0, layer, W.PAYLOAD_V, x.start, x.end - x.start, m.kv_row_bytes) for x in writes]
            in_k, in_v = np.concatenate(ks), np.concatenate(vs)
            for e in self.engines:
                assert e.scatter_kv(layer, slots, starts, in_k, in_v) == 0
        adm = [x for x in writes if x.is_admit]
        if adm:
            aslots = np.array([x.slot for x in adm], np.uint32)
            for layer in self.ssm_layers:
                st = np.concatenate([W.payload_bytes(self.seed, x.uid, x.epoch, layer, W.PAYLOAD_STATE, 0, 1, m.state_bytes) for x in adm])
                cv = np.concatenate([W.payload_bytes(self.seed, x.uid, x.epoch, layer, W.PAYLOAD_CONV, 0, 1, m.conv_bytes) for x in adm])
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
        st = [W.payload_bytes(self.seed, int(u), int(e), layer, W.PAYLOAD_STATE, 0, 1, m.state_bytes) for u, e in zip(uids, epochs)]
        cv = [W.payload_bytes(self.seed, int(u), int(e), layer, W.PAYLOAD_CONV, 0, 1, m.conv_bytes) for u, e in zip(uids, epochs)]
        return (np.concatenate(st or [np.zeros((0, m.state_bytes), np.uint8)]),
                np.concatenate(cv or [np.zeros((0, m.conv_bytes), np.uint8)]))

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
