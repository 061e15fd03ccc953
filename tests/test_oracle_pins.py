"""Pins for the CPU oracle: each test ties it to something other than itself --
closed forms, a hand-worked trace, separately written models, invariants, the payload
function.  No GPU needed."""
from __future__ import annotations

from pathlib import Path

import numpy as np
import pytest

import models_py as M
from harness import PayloadHarness
from invariants import check_invariants
from oracle.avmp_oracle import INVALID, NONE64, Oracle
from paper_2605_22416_b200 import workloads as W

GOLDEN = Path(__file__).resolve().parent / "golden"


def _rows(name):
    for line in (GOLDEN / name).read_text().splitlines():
        line = line.strip()
        if line and not line.startswith("#"):
            yield line


def _inv(o: Oracle, w: W.Workload):
    check_invariants(o.stats(), o.tables(), page_tokens=w.model.page_tokens,
                     n_ssm_layers=w.model.n_ssm_layers, max_pages=o.max_pages)


# ---- closed forms (Section 3.1) -----------------------------------------------------
def test_unit_sizes_and_capacities_closed_form():
    for line in _rows("config_sizes.txt"):
        name, u_kv, u_ssm, split, kv_cap, ssm_cap, v_kv, v_ssm = line.split()
        w = W.config(name, split=float(split))
        o = Oracle.from_workload(w, max_requests=4, max_pages=4)
        s = o.stats()
        assert (s["unit_bytes_kv"], s["unit_bytes_ssm"]) == (int(u_kv), int(u_ssm)), name
        assert (s["cap_kv"], s["cap_ssm"]) == (int(kv_cap), int(ssm_cap)), name
        assert (s["vid_space_kv"], s["vid_space_ssm"]) == (int(v_kv), int(v_ssm)), name
        assert s["cap_kv"] * s["unit_bytes_kv"] + s["cap_ssm"] * s["unit_bytes_ssm"] + s["gap_bytes"] == w.pool_bytes
        o.close()


def test_alignment_rules():
    # Section 3.1: 128-byte slab alignment for the pool, 16-byte alignment for units.
    m = W.ModelShape(1, 1, 16, 1, 3, 2, 5, 2, 4)     # raw page 192 B, raw block 28 B -> 32 B
    o = Oracle(m, 1000, 0.5, 1, max_requests=2, max_pages=2)
    s = o.stats()
    assert s["pool_bytes_aligned"] == 896
    assert s["unit_bytes_kv"] == 192 and s["unit_bytes_ssm"] == 32
    # SSM share: 448 aligned down to the 128-byte slab = 384; KV keeps the other 512
    assert s["cap_kv"] == 512 // 192 and s["cap_ssm"] == 384 // 32
    assert s["gap_bytes"] == 896 - 2 * 192 - 12 * 32


def test_fresh_pool_allocation_order():
    # The first k allocations of a fresh pool are slots 0..k-1 under handles (pool<<31)+i.
    w = W.config("pr1")
    o = Oracle.from_workload(w)
    assert o.step(W.make_ops(W.OP_ADMIT, [0, 1], [100, 33])).tolist() == [0, 0]
    t = o.tables()
    chain = t["req_chain"].reshape(w.max_requests, w.max_pages)
    assert chain[0, :7].tolist() == list(range(7)) and chain[1, :3].tolist() == [7, 8, 9]
    ssm = t["req_ssm"].reshape(w.max_requests, 12)
    assert ssm[0].tolist() == [(1 << 31) + i for i in range(12)]
    assert ssm[1].tolist() == [(1 << 31) + 12 + i for i in range(12)]
    pool, off, bad = o.translate(np.concatenate([chain[1, :3], ssm[1, :2]]))
    assert bad == 0 and pool.tolist() == [0, 0, 0, 1, 1]
    assert off.tolist() == [7 * 262144, 8 * 262144, 9 * 262144, 12 * 155648, 13 * 155648]
    _inv(o, w)


def test_translate_rejects_dead_handles():
    w = W.config("tiny")
    o = Oracle.from_workload(w)
    o.step(W.make_ops(W.OP_ADMIT, [0], [20]))
    pool, off, bad = o.translate(np.array([0, 1, 2, INVALID, (1 << 31) | 0, (1 << 31) | 1, 500], np.uint32))
    assert bad == 4
    assert pool.tolist() == [0, 0, INVALID, INVALID, 1, INVALID, INVALID]
    assert off.tolist() == [0, 64, NONE64, NONE64, 0, NONE64, NONE64]


# ---- the hand-worked trace ------------------------------------------------------------
@pytest.mark.parametrize("golden,reclaim", [("worked_example.txt", False), ("worked_example_reclaim.txt", True)])
def test_worked_example(golden, reclaim):
    w = W.config("tiny", reclaim_gap=reclaim)
    o = Oracle.from_workload(w)
    kinds = {"ADMIT": 1, "EXTEND": 2, "FINISH": 3}
    cols = ("cap_kv", "free_kv", "cap_ssm", "free_ssm", "gap_bytes", "migrated_bytes", "wasted_bytes",
            "n_rebalance", "relocated_blocks", "n_oom", "n_capacity_error")
    extra = {}
    for line in _rows(golden):
        if "|" in line:
            l, r = line.split("|")
            k, req, tok = l.split()
            exp = [int(x) for x in r.split()]
            st = o.step(W.make_ops(kinds[k], [int(req)], int(tok)))
            s = o.stats()
            assert int(st[0]) == exp[0], line
            assert [s[c] for c in cols] == exp[1:12], line
            last = -1 if s["last_rebalance_op"] == NONE64 else s["last_rebalance_op"]
            assert last == exp[12], line
            _inv(o, w)
        else:
            extra[line.split(":")[0].strip()] = line.split(":")[1]
    t = o.tables()
    chain = t["req_chain"].reshape(w.max_requests, w.max_pages)
    ssm = t["req_ssm"].reshape(w.max_requests, 1)
    for key, val in extra.items():
        if key.startswith("chain") or key.startswith("ssm "):
            kind, r = key.split()
            vids, slots = ([int(x) for x in part.split()] for part in val.split("->"))
            if kind == "chain":
                assert chain[int(r), :len(vids)].tolist() == vids
                assert t["vt_kv"][vids].tolist() == slots
                assert o.translate(np.array(vids, np.uint32))[1].tolist() == [64 * s for s in slots]
            else:
                assert [h & 0x7FFFFFFF for h in ssm[int(r)].tolist()] == vids
                assert t["vt_ssm"][vids].tolist() == slots
    assert t["slot_stack_kv"].tolist() == [int(x) for x in extra["kv_stack"].split()]
    assert t["slot_stack_ssm"].tolist() == [int(x) for x in extra["ssm_stack"].split()]


# ---- migration arithmetic (Section 3.2 waste formula) -----------------------------------
def test_migration_arithmetic_by_hand():
    models = {"pr1": W.PR1_MODEL, "jamba_like": W.JAMBA_LIKE}
    for line in _rows("migration_arithmetic.txt"):
        name, donor, B, gain, waste = line.split()
        B, gain, waste = int(B), int(gain), int(waste)
        m = models[name]
        u_kv, u_ssm = M.unit_sizes(m)
        # a pool with 1000 units on each side, exactly
        pool = 1000 * u_kv + 1000 * u_ssm
        split = (1000 * u_ssm) / pool
        o = Oracle(m, pool, split, B, max_requests=1100, max_pages=1024, min_rebalance_interval_ops=1)
        s0 = o.stats()
        if donor == "ssm":
            # exhaust KV with one long request; the next page raises CapacityError(KV)
            o.step(W.make_ops(W.OP_ADMIT, [0], [s0["cap_kv"] * 16]))
            st = o.step(W.make_ops(W.OP_EXTEND, [0], [1]))
            d, r = "ssm", "kv"
        else:
            n_fit = s0["cap_ssm"] // m.n_ssm_layers
            o.step(W.make_ops(W.OP_ADMIT, np.arange(n_fit), 1))
            st = o.step(W.make_ops(W.OP_ADMIT, [n_fit], [1]))
            d, r = "kv", "ssm"
        s = o.stats()
        assert s["n_rebalance"] == 1
        assert s[f"cap_{d}"] == s0[f"cap_{d}"] - B
        assert s[f"cap_{r}"] == s0[f"cap_{r}"] + gain
        assert s["wasted_bytes"] == waste and s["gap_bytes"] == s0["gap_bytes"] + waste
        assert s["migrated_bytes"] == B * s0[f"unit_bytes_{d}"]
        # the retry succeeds only if the gain covers the need
        need = 1 if d == "ssm" else m.n_ssm_layers
        have = gain + (s0["cap_ssm"] - n_fit * m.n_ssm_layers if d == "kv" else 0)
        assert int(st[0]) == (W.ST_OK if have >= need else W.ST_OOM)


def test_no_whole_unit_no_migration():
    # B x donor unit smaller than one recipient unit: the migration is not started at all.
    m = W.JAMBA_LIKE                      # KV page 256 KiB < SSM block 608 KiB
    u_kv, u_ssm = M.unit_sizes(m)
    pool = 100 * u_kv + 29 * u_ssm
    o = Oracle(m, pool, 28.5 * u_ssm / pool, 2, max_requests=4, max_pages=8, min_rebalance_interval_ops=1)
    s0 = o.stats()
    assert s0["cap_ssm"] == 28 and s0["cap_kv"] >= 100
    assert o.step(W.make_ops(W.OP_ADMIT, [0, 1], [1, 1])).tolist() == [W.ST_OK, W.ST_OOM]
    s = o.stats()
    assert s["n_rebalance"] == 0 and s["n_capacity_error"] == 1 and s["last_rebalance_op"] == NONE64
    assert s["cap_kv"] == s0["cap_kv"] and s["cap_ssm"] == 28


def test_reclaim_gap_offers_stranded_bytes_again():
    # Variant of the waste rule: one ceded KV page (256 KiB) is less than an SSM block (608 KiB),
    # but together with 400 000 B already lying between the pools it makes one block.
    m = W.JAMBA_LIKE
    u_kv, u_ssm = M.unit_sizes(m)
    pool = 10 * u_kv + 28 * u_ssm + 400_000
    split = (28 * u_ssm + 400_000 - 300) / pool       # the slack sits in the SSM share: no 11th page
    for reclaim in (False, True):
        o = Oracle(m, pool, split, 1, max_requests=4, max_pages=8, min_rebalance_interval_ops=1,
                   reclaim_gap=reclaim)
        s0 = o.stats()
        assert (s0["cap_kv"], s0["cap_ssm"], s0["gap_bytes"]) == (10, 28, 400_000)
        st = o.step(W.make_ops(W.OP_ADMIT, [0, 1], [1, 1])).tolist()
        s = o.stats()
        if not reclaim:
            assert st == [W.ST_OK, W.ST_OOM] and s["n_rebalance"] == 0 and s["gap_bytes"] == 400_000
        else:
            # 400 000 + 262 144 = 662 144 = 1 block + 39 552: still not the 28 blocks an admit needs
            assert st == [W.ST_OK, W.ST_OOM] and s["n_rebalance"] == 1
            assert (s["cap_kv"], s["cap_ssm"], s["gap_bytes"]) == (9, 29, 39_552)
            assert s["wasted_bytes"] == 0 and s["migrated_bytes"] == u_kv
            # the second page offered meets a gap of 39 552: 301 696 B is no block, nothing happens
            assert o.step(W.make_ops(W.OP_ADMIT, [1], [1])).tolist() == [W.ST_OOM]
            s2 = o.stats()
            assert s2["n_rebalance"] == 1 and s2["gap_bytes"] == 39_552 and s2["cap_kv"] == 9
        _inv(o, W.config("short_uniform"))


# ---- configuration validation (Section 4.6) ----------------------------------------------
def test_threshold_validation():
    with pytest.raises(ValueError):
        Oracle(W.TINY_MODEL, 1024, 0.5, 1, max_requests=2, max_pages=2,
               threshold_low_ppm=300_000, threshold_high_ppm=300_000)
    with pytest.raises(ValueError):
        Oracle(W.TINY_MODEL, 1024, 0.5, 1, max_requests=2, max_pages=2,
               threshold_low_ppm=400_000, threshold_high_ppm=300_000)


# ---- separately written models ------------------------------------------------------------
def _tiny_variants():
    for seed in range(6):
        for B in (1, 2, 3, 5):
            yield seed, B


def _run_ops_against(o: Oracle, model, ops):
    """Step one op at a time through both; returns the status lists."""
    a, b = [], []
    for op in ops:
        a.append(int(o.step(ops[len(a):len(a) + 1])[0]))
        b.append(model.op(int(op["kind"]), int(op["flags"]), int(op["req"]), int(op["tokens"])))
    return a, b


@pytest.mark.parametrize("seed,B", list(_tiny_variants()))
def test_naive_model_on_tiny_inputs(seed, B):
    """Brute force: every prefix of a random op string leaves identical handles, slots and
    chains in a list-based model written separately."""
    w = W.config("tiny", migration_batch_size=B)
    m = w.model
    ops = W.random_op_string(seed, 300, 6, 60)
    o = Oracle.from_workload(w, max_requests=6, max_pages=8)
    nv = M.NaiveAllocator(m, w.pool_bytes, w.split, B, 6, 8, min_interval=w.min_rebalance_interval_ops)
    for i in range(len(ops)):
        st = int(o.step(ops[i:i + 1])[0])
        ex = nv.op(int(ops["kind"][i]), int(ops["flags"][i]), int(ops["req"][i]), int(ops["tokens"][i]))
        assert st == ex, (i, ops[i])
        t = o.tables()
        chain = t["req_chain"].reshape(6, 8)
        for r in range(6):
            q = nv.reqs[r]
            assert int(t["req_state"][r]) == q.state and int(t["req_len"][r]) == q.length
            assert chain[r, :len(q.chain)].tolist() == q.chain
            assert int(t["req_npages"][r]) == len(q.chain)
            if q.state == M.LIVE:
                assert t["req_ssm"].reshape(6, 1)[r].tolist() == q.ssm
        for p, nm in enumerate(("kv", "ssm")):
            live = {int(v): int(s) for v, s in enumerate(t[f"vt_{nm}"]) if s != INVALID}
            assert live == nv.where[p]
            # an array stack's top is the list model's front
            assert t[f"slot_stack_{nm}"][::-1].tolist() == nv.next_slots[p]
            assert t[f"vid_stack_{nm}"][::-1].tolist() == nv.next_ids[p]
        s = o.stats()
        assert (s["cap_kv"], s["cap_ssm"]) == tuple(nv.cap)
        assert s["n_oom"] == nv.n_oom and s["n_rebalance"] == nv.n_rebalance
        assert s["relocated_blocks"] == nv.relocated
        _inv(o, w.with_(max_pages=8))
    assert o.stats()["n_rebalance"] > 0 or B == 1


@pytest.mark.parametrize("split", [0.0, 1.0])
def test_one_pool_starts_empty(split):
    """Degenerate split: one store has no capacity at all until the first CapacityError moves
    some over.  Same brute-force comparison as above."""
    w = W.config("tiny", pool_bytes=2048, split=split, migration_batch_size=4)
    o = Oracle.from_workload(w, max_requests=6, max_pages=8)
    nv = M.NaiveAllocator(w.model, w.pool_bytes, w.split, 4, 6, 8, min_interval=4)
    s0 = o.stats()
    assert (s0["cap_kv"] == 0) != (s0["cap_ssm"] == 0)
    ops = W.random_op_string(7, 400, 6, 50)
    for i in range(len(ops)):
        st = int(o.step(ops[i:i + 1])[0])
        assert st == nv.op(int(ops["kind"][i]), int(ops["flags"][i]), int(ops["req"][i]), int(ops["tokens"][i]))
        _inv(o, w.with_(max_pages=8))
    s = o.stats()
    assert s["n_rebalance"] >= 5 and s["relocated_blocks"] > 0 and s["cap_kv"] > 0 and s["cap_ssm"] > 0
    assert (s["cap_kv"], s["cap_ssm"]) == tuple(nv.cap) and s["relocated_blocks"] == nv.relocated


@pytest.mark.parametrize("name,steps", [("pr1", 700), ("short_uniform", 250), ("mixed_long", 400),
                                        ("agentic_burst", 500), ("scale", 60)])
def test_static_equivalence(name, steps):
    """Section 1.1: with migration disabled the handle abstraction changes no capacity
    outcome -- the status stream and OOM count equal a static dual pool's."""
    w = W.config(name, migration_enabled=False)
    if name == "pr1":
        w = w.with_(pool_bytes=96 * W.MiB)       # small enough to run out of memory
    if name == "scale":
        w = w.with_(pool_bytes=16 * W.GiB)
    o = Oracle.from_workload(w)
    sd = M.StaticDualPool(w.model, w.pool_bytes, w.split, w.max_requests, w.max_pages)
    n_ops = 0

    def step(ops):
        nonlocal n_ops
        st = o.step(ops)
        ex = [sd.op(int(k), int(f), int(r), int(t)) for k, f, r, t in
              zip(ops["kind"], ops["flags"], ops["req"], ops["tokens"])]
        assert st.tolist() == ex
        n_ops += len(ops)
        return st

    _, d = W.record_trace(w, step, max_steps=steps)
    s = o.stats()
    assert s["n_oom"] == sd.n_oom and s["n_rebalance"] == 0 and s["migrated_bytes"] == 0
    assert s["op_counter"] == n_ops
    assert s["n_oom"] > 0, "the workload never ran out of memory: the test shows nothing"
    _inv(o, w)


@pytest.mark.parametrize("name,steps,over", [
    ("pr1", 900, dict(pool_bytes=96 * W.MiB, min_rebalance_interval_ops=100)),
    ("short_uniform", 400, {}),
    ("mixed_long", 500, dict(migration_batch_size=64)),
    ("short_uniform", 300, dict(migration_batch_size=16, split=0.93, concurrency=128)),
    ("agentic_burst", 600, {}),
    ("scale", 60, dict(pool_bytes=16 * W.GiB)),
])
def test_counts_model_under_migration(name, steps, over):
    """Success, capacities, rebalance count, migrated and wasted bytes equal those of the
    counts-only statement of Section 3.2; migrations obey the throttle and the trigger."""
    w = W.config(name, **over)
    o = Oracle.from_workload(w)
    cm = M.CountsModel(w.model, w.pool_bytes, w.split, w.migration_batch_size, w.max_requests, w.max_pages,
                       th_high_ppm=w.threshold_high_ppm, min_interval=w.min_rebalance_interval_ops)

    def step(ops):
        st = o.step(ops)
        ex = [cm.op(int(k), int(f), int(r), int(t)) for k, f, r, t in
              zip(ops["kind"], ops["flags"], ops["req"], ops["tokens"])]
        assert st.tolist() == ex
        s = o.stats()
        assert [s["cap_kv"], s["cap_ssm"]] == cm.cap and [s["free_kv"], s["free_ssm"]] == cm.free
        return st

    W.record_trace(w, step, max_steps=steps)
    s = o.stats()
    assert s["n_rebalance"] == cm.n_rebalance > 0
    assert s["migrated_bytes"] == cm.migrated and s["wasted_bytes"] == cm.wasted
    assert s["n_oom"] == cm.n_oom and s["n_capacity_error"] == cm.n_capacity_error
    assert s["op_counter"] == cm.clock
    # throttle: consecutive migrations at least min_interval logical ops apart
    clocks = [e["clock"] for e in cm.events]
    assert all(b - a >= w.min_rebalance_interval_ops for a, b in zip(clocks, clocks[1:]))
    # trigger: donor free fraction strictly above threshold_high at the moment of the error
    assert all(e["donor_free"] * 10**6 > w.threshold_high_ppm * e["donor_cap"] for e in cm.events)
    _inv(o, w)


def test_no_donor_means_static_behaviour():
    # Section 4.6 failure modes: both pools saturated -> the trigger finds no donor.
    w = W.config("tiny", migration_batch_size=3)
    o = Oracle.from_workload(w)
    # 5 SSM blocks and 8 KV pages: fill both
    st = o.step(W.make_ops(W.OP_ADMIT, [0, 1, 2, 3], [32, 32, 32, 16]))
    assert st.tolist() == [0, 0, 0, 0]
    assert o.stats()["free_kv"] == 1 and o.stats()["free_ssm"] == 1
    st = o.step(W.make_ops(W.OP_EXTEND, [0, 1], [1, 1]))
    assert st.tolist() == [0, 1]
    s = o.stats()
    assert s["n_rebalance"] == 0 and s["n_oom"] == 1 and s["n_capacity_error"] == 1
    assert s["fsm_state"] == 1      # KV free fraction 0 < threshold_low: KV_PRESSURED


def test_ssm_shortage_is_handled_before_kv_shortage():
    """Group allocation checks the SSM pool first.  Worked by hand: 16 KV pages / 10 SSM blocks,
    B = 3.  Ten one-page requests fill the SSM store (KV: 6 of 16 free = 0.375).  An admit that
    needs 1 block and exactly the 6 free pages raises CapacityError(SSM); KV donates 3 pages
    (192 B -> 2 blocks); now only 3 pages are free, so the same op raises CapacityError(KV), which
    the throttle keeps from migrating: OOM after two handler runs and one migration.  (Checking KV
    first would see 6 <= 6, run one handler only, and still end OOM.)"""
    w = W.config("tiny", pool_bytes=2048, migration_batch_size=3)
    o = Oracle.from_workload(w, max_requests=12, max_pages=8)
    assert (o.step(W.make_ops(W.OP_ADMIT, np.arange(10), 1)) == 0).all()
    s = o.stats()
    assert (s["free_kv"], s["free_ssm"]) == (6, 0)
    st = o.step(W.make_ops(W.OP_ADMIT, [10], 96))
    s = o.stats()
    assert int(st[0]) == W.ST_OOM
    assert (s["n_capacity_error"], s["n_rebalance"], s["n_oom"]) == (2, 1, 1)
    assert (s["cap_kv"], s["free_kv"], s["cap_ssm"], s["free_ssm"]) == (13, 3, 12, 2)
    assert s["migrated_bytes"] == 192 and s["wasted_bytes"] == 0 and s["last_rebalance_op"] == 11


def test_threshold_comparisons_are_strict():
    """Section 3.2: the donor must have a free fraction *greater than* threshold_high.  With exactly
    0.30 free (3 of 10 blocks) nothing migrates; with 0.40 (4 of 10) it does."""
    w = W.config("tiny", pool_bytes=2048, migration_batch_size=2)          # 16 KV pages, 10 SSM blocks
    for n_req, tokens, migrates in ((7, [48, 48, 32, 32, 32, 32, 32], False), (6, [48, 48, 48, 48, 32, 32], True)):
        o = Oracle.from_workload(w, max_requests=8, max_pages=8)
        s0 = o.stats()
        assert (s0["cap_kv"], s0["cap_ssm"]) == (16, 10)
        assert (o.step(W.make_ops(W.OP_ADMIT, np.arange(n_req), tokens)) == 0).all()
        s = o.stats()
        assert s["free_kv"] == 0 and s["free_ssm"] == 10 - n_req
        st = o.step(W.make_ops(W.OP_EXTEND, [0], 1))
        s = o.stats()
        assert s["n_capacity_error"] == 1
        assert (s["n_rebalance"] == 1) == migrates and int(st[0]) == (W.ST_OK if migrates else W.ST_OOM)
    # threshold_low labels the state only when the free fraction is *below* it: 1 free of 20 is exactly 0.05
    m = W.ModelShape(1, 1, 16, 1, 1, 2, 20, 4, 4)
    o = Oracle(m, 1536, 256 / 1536, 1, max_requests=4, max_pages=32, migration_enabled=False)   # 1280 B KV + 256 B SSM
    s0 = o.stats()
    assert s0["cap_kv"] == 20, s0
    o.step(W.make_ops(W.OP_ADMIT, [0], 19 * 16))
    st = o.step(W.make_ops(W.OP_ADMIT, [1], 2 * 16))       # needs 2 pages, 1 free: CapacityError(KV)
    s = o.stats()
    assert int(st[0]) == W.ST_OOM and s["free_kv"] == 1 and s["fsm_state"] == 0      # 0.05 is not < 0.05
    o.step(W.make_ops(W.OP_EXTEND, [0], 16))                # takes the last page
    o.step(W.make_ops(W.OP_EXTEND, [0], 16))                # CapacityError at 0 free: now pressured
    assert o.stats()["fsm_state"] == 1


# ---- threshold_low null result (Section 4.5, stage 2) and determinism (Section 4.1) ------
def _digest(o: Oracle):
    import hashlib
    h = hashlib.sha256()
    for k, v in sorted(o.tables().items()):
        h.update(k.encode())
        h.update(np.ascontiguousarray(v).tobytes())
    s = o.stats()
    s.pop("fsm_state")
    h.update(repr(sorted(s.items())).encode())
    return h.hexdigest()


def test_threshold_low_changes_nothing_and_runs_are_deterministic():
    digests = []
    for th_low in (20_000, 50_000, 100_000, 50_000):
        w = W.config("pr1", pool_bytes=96 * W.MiB, min_rebalance_interval_ops=100, threshold_low_ppm=th_low)
        o = Oracle.from_workload(w)
        trace, _ = W.record_trace(w, o.step, max_steps=600)
        digests.append((_digest(o), [s.tobytes() for _, s in trace]))
        assert o.stats()["n_rebalance"] > 0 and o.stats()["n_oom"] > 0
    assert all(d == digests[0] for d in digests[1:])


# ---- payload: gathers and relocation against the payload function -------------------------
def test_gather_matches_payload_function_through_migrations():
    """Everything a gather returns must be what was written for that (request, token),
    wherever the allocator put it and however often a migration moved it."""
    w = W.config("pr1", pool_bytes=24 * W.MiB, concurrency=12, min_rebalance_interval_ops=50,
                 migration_batch_size=6, n_requests=150)
    o = Oracle.from_workload(w, with_store=True)
    h = PayloadHarness(w, [o])
    checked = 0

    def on_step(d, ops, status):
        nonlocal checked
        h.apply_writes(d.writes)
        if d.step % 7 == 0:
            checked += h.check_gathers(d, d.step % 4, d.step % 12)

    W.record_trace(w, o.step, max_steps=700, on_step=on_step)
    s = o.stats()
    assert s["relocated_blocks"] > 5 and s["n_rebalance"] > 3, s
    assert checked > 10_000
    _inv(o, w)


def test_naive_payload_shadow_copies():
    """Tiny case with real bytes in both models: after random ops with migrations, every
    live token / block reads the same bytes through the oracle's gather and through the
    list model's own bookkeeping."""
    w = W.config("tiny", migration_batch_size=2)
    m = w.model
    o = Oracle.from_workload(w, with_store=True, max_requests=6, max_pages=8)
    nv = M.NaiveAllocator(m, w.pool_bytes, w.split, 2, 6, 8, min_interval=4)
    ops = W.random_op_string(11, 400, 6, 40, p_invalid=0.02)
    rng = np.random.default_rng(5)
    for i in range(len(ops)):
        k, f, r, t = (int(ops[c][i]) for c in ("kind", "flags", "req", "tokens"))
        before = nv.reqs[r].length if r < 6 else 0
        st = int(o.step(ops[i:i + 1])[0])
        assert st == nv.op(k, f, r, t)
        if st == 0 and k in (1, 2):
            n_new = nv.reqs[r].length - before
            kb = rng.integers(0, 256, (n_new, 2), dtype=np.uint8)
            vb = rng.integers(0, 256, (n_new, 2), dtype=np.uint8)
            assert o.scatter_kv(0, [r], [before], kb, vb) == 0
            for j in range(n_new):
                for part, src in ((0, kb), (1, vb)):
                    buf, off, row = nv.kv_row(r, 0, part, before + j)
                    buf[off:off + row] = src[j].tobytes()
            if k == 1:
                sb = rng.integers(0, 256, (1, 80), dtype=np.uint8)
                cb = rng.integers(0, 256, (1, 16), dtype=np.uint8)
                assert o.scatter_ssm(0, [r], sb, cb) == 0
                nv.ssm_block(r, 0)[:96] = sb.tobytes() + cb.tobytes()
        for q in range(6):
            rq = nv.reqs[q]
            if rq.state != M.EMPTY and rq.length:
                gk, gv, cu, bad = o.gather_kv(0, [q], rq.length)
                assert bad == 0 and cu.tolist() == [0, rq.length]
                for tkn in range(rq.length):
                    for part, got in ((0, gk), (1, gv)):
                        buf, off, row = nv.kv_row(q, 0, part, tkn)
                        assert bytes(buf[off:off + row]) == got[tkn].tobytes()
            if rq.state == M.LIVE:
                gs, gc, bad = o.gather_ssm(0, [q])
                assert bad == 0 and gs.tobytes() + gc.tobytes() == bytes(nv.ssm_block(q, 0)[:96])
    assert nv.relocated > 0


def test_gather_error_items():
    w = W.config("tiny")
    o = Oracle.from_workload(w, with_store=True)
    o.step(W.make_ops(W.OP_ADMIT, [0, 1], [20, 5]))
    o.step(W.make_ops(W.OP_FINISH, [1], 0, W.FLAG_KEEP_KV))
    k, v, cu, bad = o.gather_kv(0, [0, 3, 1], 25)
    assert bad == 1 and cu.tolist() == [0, 20, 20, 25]      # slot 3 is empty
    k, v, cu, bad = o.gather_kv(0, [0, 1], 22)
    assert bad == 1 and cu.tolist() == [0, 20, 25]           # request 1 would pass the capacity
    st, cv, bad = o.gather_ssm(0, [0, 1])
    assert bad == 1                                           # request 1 kept only its KV


def test_invalid_ops_advance_the_clock_and_change_nothing():
    w = W.config("tiny")
    o = Oracle.from_workload(w)
    o.step(W.make_ops(W.OP_ADMIT, [0], [20]))
    before = _digest(o)
    ops = np.concatenate([
        W.make_ops(9, [0], 1),                      # unknown kind
        W.make_ops(W.OP_ADMIT, [0], 5),             # slot already live
        W.make_ops(W.OP_ADMIT, [1], 0),             # zero tokens
        W.make_ops(W.OP_EXTEND, [2], 1),            # nothing there
        W.make_ops(W.OP_FINISH, [99], 0),           # slot out of range
        W.make_ops(W.OP_EXTEND, [0], 16 * 8),       # chain would pass max_pages
        W.make_ops(W.OP_ADMIT, [3], 4, W.FLAG_RESUME),  # resume of an empty slot
    ])
    assert o.step(ops).tolist() == [4, 2, 4, 2, 2, 3, 2]
    s = o.stats()
    assert s["op_counter"] == 8 and s["n_invalid"] == 7 and s["n_oom"] == 0
    o2 = Oracle.from_workload(w)
    o2.step(W.make_ops(W.OP_ADMIT, [0], [20]))
    t1, t2 = o.tables(), o2.tables()
    assert all(np.array_equal(t1[k], t2[k]) for k in t1)
    assert before != ""


# ---- bytes inside a unit (Section 3.1 unit contents; layout promised by the C header) ---------
from harness import LAYOUT_SHAPES, check_unit_layout, layout_workload  # noqa: E402


@pytest.mark.parametrize("shape", LAYOUT_SHAPES)
def test_bytes_inside_a_unit_follow_the_documented_layout(shape):
    """A KV page is [layer][K, V][token][head][dim], an SSM block is state then window: read from the
    raw store bytes at the translated offsets, after migrations have relocated written units."""
    w = layout_workload(shape)
    o = Oracle.from_workload(w, with_store=True)
    s = o.stats()
    unit = (s["unit_bytes_kv"], s["unit_bytes_ssm"])

    def read_units(pool, handles):
        p, off, bad = o.translate(np.asarray(handles, np.uint32))
        assert bad == 0 and (p == pool).all()
        return [o.store_bytes(pool, int(x), unit[pool]) for x in off]

    seen = check_unit_layout(w, o, read_units)
    assert seen["kv_rows"] > 1000 and seen["ssm_blocks"] > 40 and seen["relocated_blocks"] > 4
    _inv(o, w)


@pytest.mark.parametrize("seed", range(4))
def test_naive_model_on_engine_shaped_batches(seed):
    """The same brute-force comparison on batches in an engine step's order whose kinds share slots (finished and
    admitted again, parked and resumed, extended and admitted in one batch) and repeat ops back to back: the
    sequences the GPU path's window-shape shortcut must get right are pinned on the oracle side too."""
    w = W.config("tiny", migration_batch_size=1 + seed % 3, min_rebalance_interval_ops=3 + seed)
    o = Oracle.from_workload(w, max_requests=6, max_pages=8)
    nv = M.NaiveAllocator(w.model, w.pool_bytes, w.split, w.migration_batch_size, 6, 8,
                          min_interval=w.min_rebalance_interval_ops)
    for rnd in range(60):
        ops = W.engine_shaped_batch(77 * seed + rnd, 6, 50, p_pick=0.3 + 0.05 * (rnd % 8), repeats=rnd % 3 == 2)
        st = o.step(ops)
        for i in range(len(ops)):
            ex = nv.op(int(ops["kind"][i]), int(ops["flags"][i]), int(ops["req"][i]), int(ops["tokens"][i]))
            assert int(st[i]) == ex, (rnd, i, ops[i])
        t = o.tables()
        chain = t["req_chain"].reshape(6, 8)
        for r in range(6):
            q = nv.reqs[r]
            assert int(t["req_state"][r]) == q.state and int(t["req_len"][r]) == q.length
            assert chain[r, :len(q.chain)].tolist() == q.chain
        for p, nm in enumerate(("kv", "ssm")):
            assert t[f"slot_stack_{nm}"][::-1].tolist() == nv.next_slots[p]
            assert t[f"vid_stack_{nm}"][::-1].tolist() == nv.next_ids[p]
        s = o.stats()
        assert (s["cap_kv"], s["cap_ssm"]) == tuple(nv.cap) and s["n_oom"] == nv.n_oom and s["n_rebalance"] == nv.n_rebalance
        _inv(o, w.with_(max_pages=8))
    assert o.stats()["n_rebalance"] > 0 and o.stats()["n_oom"] > 0
