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


LAYOUT_SHAPES = [
    W.ModelShape(3, 2, 4, 2, 4, 2, 64, 16, 4),   # rows, state and window are 16-byte multiples
    W.ModelShape(2, 3, 4, 1, 3, 2, 5, 2, 4),     # 6-byte rows, 20 + 8 byte blocks padded to 32
]


def layout_workload(shape: W.ModelShape) -> W.Workload:
    """Room for 16 pages and 16 blocks, 8 request slots, a migration allowed at every operation: random
    batches followed by pure growth make both stores cede space that holds live units."""
    u_kv = shape.n_attn_layers * 2 * shape.page_tokens * shape.kv_row_bytes
    u_ssm = (shape.state_bytes + shape.conv_bytes + 15) // 16 * 16
    pool = (16 * u_kv + 16 * u_ssm + 127) // 128 * 128
    return W.Workload("layout", shape, pool, 16 * u_ssm / pool, 5, 8, 8, 12, "queue", 0, min_rebalance_interval_ops=1)


def check_unit_layout(w: W.Workload, engine, read_units, rounds: int = 12, seed: int = 5) -> dict:
    """Where inside a unit every byte lives, checked on the RAW bytes of the stores.

    The contract (include/avmp.h, model shape): a KV page is the array
    [attention layer][K, V][token in page][head][dim] of kv_elem_bytes elements; an SSM block is
    the state elements followed by the convolution window.  Known rows go in through the engine's
    scatter; a batch of pure growth then forces migrations that relocate some of the units just
    written; the bytes are then read back NOT through a gather but from the unit's address
    (`read_units(pool, handles) -> uint8[n][unit_bytes]`, which resolves the handles with
    translate and reads the store itself) and compared through a numpy reshape of the unit to the
    array shape above.  `engine` has step / scatter_kv / scatter_ssm / tables / stats."""
    m = w.model
    T, row, na = m.page_tokens, m.kv_row_bytes, m.n_attn_layers
    R, MP = w.max_requests, w.max_pages
    rng = np.random.default_rng(seed)
    seen = dict(kv_rows=0, ssm_blocks=0)
    for rnd in range(rounds):
        engine.step(W.random_op_string(seed * 1000 + rnd, 24, R, T * 3, p_invalid=0.0))
        t = engine.tables()
        held = np.flatnonzero(t["req_state"] != 0).astype(np.uint32)
        live = np.flatnonzero(t["req_state"] == 1).astype(np.uint32)
        lens = t["req_len"][held].astype(np.int64)
        tot = int(lens.sum())
        kb = rng.integers(0, 256, (na, 2, tot, row), dtype=np.uint8)
        for layer in range(na):
            assert engine.scatter_kv(layer, held, np.zeros(len(held), np.uint32), kb[layer, 0], kb[layer, 1]) == 0
        sb = rng.integers(0, 256, (m.n_ssm_layers, len(live), m.state_bytes), dtype=np.uint8)
        cb = rng.integers(0, 256, (m.n_ssm_layers, len(live), m.conv_bytes), dtype=np.uint8)
        for layer in range(m.n_ssm_layers):
            assert engine.scatter_ssm(layer, live, sb[layer], cb[layer]) == 0
        engine.step(W.make_ops(W.OP_EXTEND, live, T + 1))          # growth: migrations move written units
        t = engine.tables()
        chain = t["req_chain"].reshape(R, MP)
        src = np.concatenate([[0], np.cumsum(lens)])
        for k, r in enumerate(held):
            n_old = int(lens[k])
            pages = read_units(0, chain[r, : -(-n_old // T)])
            for j, unit in enumerate(pages):
                page = unit[: na * 2 * T * row].reshape(na, 2, T, row)   # [layer][K, V][token][head x dim]
                n_tok = min(T, n_old - j * T)
                want = kb[:, :, src[k] + j * T: src[k] + j * T + n_tok]
                assert np.array_equal(page[:, :, :n_tok], want), f"round {rnd}: page {j} of request {r}"
                seen["kv_rows"] += n_tok * na * 2
        ssm = t["req_ssm"].reshape(R, m.n_ssm_layers)
        for k, r in enumerate(live):
            if t["req_state"][r] != 1:
                continue
            blocks = read_units(1, ssm[r])
            for layer, unit in enumerate(blocks):
                assert np.array_equal(unit[: m.state_bytes], sb[layer, k]), f"round {rnd}: state of request {r}"
                assert np.array_equal(unit[m.state_bytes: m.state_bytes + m.conv_bytes], cb[layer, k])
                seen["ssm_blocks"] += 1
    seen["relocated_blocks"] = engine.stats()["relocated_blocks"]
    return seen
