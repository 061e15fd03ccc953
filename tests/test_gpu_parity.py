"""GPU parity: the CUDA path through the C ABI against the CPU oracle, bit for bit
(tolerance 0: the path performs no floating-point arithmetic)."""
from __future__ import annotations

import os
from pathlib import Path

import numpy as np
import pytest

from harness import PayloadHarness
from invariants import check_invariants
from paper_2605_22416_b200 import workloads as W

pytestmark = pytest.mark.gpu

GOLDEN = Path(__file__).resolve().parent / "golden"


@pytest.fixture(scope="module")
def env():
    import torch
    from gpu_engine import GpuEngine, assert_same_state
    from oracle.avmp_oracle import Oracle
    assert torch.cuda.is_available()
    return dict(GpuEngine=GpuEngine, Oracle=Oracle, same=assert_same_state, torch=torch)


def _pair(env, w, with_store=False, **over):
    g = env["GpuEngine"](w, **over)
    o = env["Oracle"].from_workload(w, with_store=with_store, **over)
    return g, o


def test_library_is_loaded_from_the_tree(env):
    from paper_2605_22416_b200 import binding
    assert Path(binding.LIBRARY_PATH).exists()
    maps = Path("/proc/self/maps").read_text()
    assert "libavmp.so" in maps


@pytest.mark.parametrize("golden,reclaim", [("worked_example.txt", False), ("worked_example_reclaim.txt", True)])
def test_worked_example_on_gpu(env, golden, reclaim):
    w = W.config("tiny", reclaim_gap=reclaim)
    g = env["GpuEngine"](w)
    kinds = {"ADMIT": 1, "EXTEND": 2, "FINISH": 3}
    cols = ("cap_kv", "free_kv", "cap_ssm", "free_ssm", "gap_bytes", "migrated_bytes", "wasted_bytes",
            "n_rebalance", "relocated_blocks", "n_oom", "n_capacity_error")
    for line in (GOLDEN / golden).read_text().splitlines():
        if "|" not in line or line.startswith("#"):
            continue
        l, r = line.split("|")
        k, req, tok = l.split()
        exp = [int(x) for x in r.split()]
        st = g.step(W.make_ops(kinds[k], [int(req)], int(tok)))
        s = g.stats()
        assert int(st[0]) == exp[0], line
        assert [s[c] for c in cols] == exp[1:12], line
    pool, off, bad, aoff = g.translate(np.array([9, 8, 2, (1 << 31) | 2], np.uint32))
    if reclaim:
        assert bad == 0 and pool.tolist() == [0, 0, 0, 1] and off.tolist() == [576, 512, 0, 192]
        return
    assert bad == 0 and pool.tolist() == [0, 0, 0, 1] and off.tolist() == [128, 512, 64, 192]
    # arena placement: KV grows up from 0, SSM slot j ends at pool_end - j * U
    assert aoff.tolist() == [128, 512, 64, 1024 - 3 * 96]


@pytest.mark.parametrize("seed,batch", [(0, 1), (1, 7), (2, 32), (3, 300), (4, 1500)])
def test_random_op_strings_tiny(env, seed, batch):
    """Unscheduled ops (any order, repeated slots inside a batch, invalid ops): statuses,
    counters and every table equal the oracle's after each batch."""
    w = W.config("tiny", migration_batch_size=1 + seed % 4, reclaim_gap=bool(seed % 2))
    g, o = _pair(env, w, max_requests=6, max_pages=8)
    ops = W.random_op_string(100 + seed, 3000, 6, 60)
    for i in range(0, len(ops), batch):
        b = ops[i:i + batch]
        sg, so = g.step(b), o.step(b)
        assert np.array_equal(sg, so), (i, sg[:20], so[:20])
        if (i // batch) % 5 == 0 or batch >= 300:
            env["same"](g, o, w, f"batch at {i}")
    env["same"](g, o, w, "end")
    s = g.stats()
    assert s["n_rebalance"] > 0 and s["n_oom"] > 0
    assert s["relocated_blocks"] > 0 or w.migration_batch_size == 1
    check_invariants(s, g.tables(), page_tokens=16, n_ssm_layers=1, max_pages=8)


@pytest.mark.parametrize("split", [0.0, 1.0])
def test_one_pool_starts_empty(env, split):
    """Degenerate split: one store starts with zero capacity."""
    w = W.config("tiny", pool_bytes=2048, split=split, migration_batch_size=4)
    g, o = _pair(env, w, max_requests=6, max_pages=8)
    ops = W.random_op_string(7, 1200, 6, 50)
    for i in range(0, len(ops), 40):
        b = ops[i:i + 40]
        assert np.array_equal(g.step(b), o.step(b)), i
        env["same"](g, o, w, f"batch at {i}")
    assert g.stats()["n_rebalance"] >= 5


def test_longest_chain_and_full_pools(env):
    """Maximum sizes: a chain that fills max_pages exactly, one page more (TOO_LONG), a pool
    filled to its last unit, and the largest batch the host entry point accepts."""
    w = W.config("pr1", pool_bytes=64 * W.MiB, migration_enabled=False)
    g, o = _pair(env, w)
    cap_kv = o.stats()["cap_kv"]
    assert cap_kv == 128
    ops = np.concatenate([
        W.make_ops(W.OP_ADMIT, [0], 40 * 16),            # exactly max_pages
        W.make_ops(W.OP_EXTEND, [0], 1),                 # one more page: TOO_LONG
        W.make_ops(W.OP_ADMIT, [1], 40 * 16),
        W.make_ops(W.OP_ADMIT, [2], 40 * 16),
        W.make_ops(W.OP_ADMIT, [3], 8 * 16),             # the pool's last 8 pages
        W.make_ops(W.OP_ADMIT, [4], 1),                  # nothing left: OOM
        W.make_ops(W.OP_FINISH, [1], 0),
        W.make_ops(W.OP_ADMIT, [4], 40 * 16 + 1),        # 41 pages: TOO_LONG before any capacity check
        W.make_ops(W.OP_ADMIT, [4], 40 * 16),
    ])
    sg, so = g.step(ops), o.step(ops)
    assert np.array_equal(sg, so) and so.tolist() == [0, 3, 0, 0, 0, 1, 0, 3, 0]
    env["same"](g, o, w, "full pools")
    assert g.stats()["free_kv"] == 0
    big = W.random_op_string(3, 65536, 32, 200)
    assert np.array_equal(g.step_host(big), o.step(big))
    env["same"](g, o, w, "65536-op batch")


@pytest.mark.parametrize("case", range(int(os.environ.get("AVMP_RANDOM_CASES", "10"))))   # more cases on demand
def test_random_shapes_and_policies(env, case):
    """Random cache shapes (rows that are and are not 16-byte multiples: both copy paths), pool
    sizes, splits, migration_batch_size, throttle and thresholds; random op batches; payload written
    and gathered back through both implementations after every batch."""
    rng = np.random.default_rng(1000 + case)
    shape = W.ModelShape(int(rng.integers(1, 4)), int(rng.integers(1, 5)), int(rng.choice([4, 16])),
                         int(rng.integers(1, 3)), int(rng.choice([1, 4, 8, 64])), 2,
                         int(rng.integers(3, 40)) * (4 if case % 2 else 1), int(rng.integers(1, 9)) * (4 if case % 2 else 1), 4)
    row = shape.kv_row_bytes
    u = max(shape.n_attn_layers * 2 * shape.page_tokens * row, (shape.ssm_state_elems + shape.ssm_conv_elems) * 4)
    pool = int(rng.integers(10, 60)) * u
    w = W.Workload(f"rand{case}", shape, pool, float(rng.choice([0.0, 0.3, 0.5, 0.7, 1.0])), int(rng.integers(1, 9)),
                   8, 8, 6, "queue", 0, min_rebalance_interval_ops=int(rng.integers(1, 20)),
                   threshold_high_ppm=int(rng.choice([100_000, 300_000, 500_000])), reclaim_gap=case >= 7)
    g, o = _pair(env, w, with_store=True)
    for rnd in range(25):
        ops = W.random_op_string(case * 100 + rnd, int(rng.integers(1, 40)), 8, shape.page_tokens * 3, p_invalid=0.05)
        assert np.array_equal(g.step(ops), o.step(ops)), (case, rnd)
        env["same"](g, o, w, f"case {case} round {rnd}")
        t = o.tables()
        held = np.flatnonzero(t["req_state"] != 0).astype(np.uint32)
        live = np.flatnonzero(t["req_state"] == 1).astype(np.uint32)
        lens = t["req_len"][held]
        tot = int(lens.sum())
        for layer in range(shape.n_attn_layers):
            kb = rng.integers(0, 256, (tot, row), dtype=np.uint8)
            vb = rng.integers(0, 256, (tot, row), dtype=np.uint8)
            for e in (g, o):
                assert e.scatter_kv(layer, held, np.zeros(len(held), np.uint32), kb, vb) == 0
            gk, gv, gcu, gb = g.gather_kv(layer, held, tot)
            ok, ov, ocu, ob = o.gather_kv(layer, held, tot)
            assert gb == ob == 0 and np.array_equal(gcu, ocu)
            assert np.array_equal(gk, kb) and np.array_equal(gv, vb) and np.array_equal(ok, kb) and np.array_equal(ov, vb)
        for layer in range(shape.n_ssm_layers):
            sb = rng.integers(0, 256, (len(live), shape.state_bytes), dtype=np.uint8)
            cb = rng.integers(0, 256, (len(live), shape.conv_bytes), dtype=np.uint8)
            for e in (g, o):
                assert e.scatter_ssm(layer, live, sb, cb) == 0
            gs, gc, gb = g.gather_ssm(layer, live)
            assert gb == 0 and np.array_equal(gs, sb) and np.array_equal(gc, cb)
        # both gathers of all layers in one launch, on the held list (KV_ONLY slots are SSM error items)
        fk, fv, fcu, fs, fc, fbad = g.gather_step(0, shape.n_attn_layers, 0, shape.n_ssm_layers, held, tot)
        assert fbad == (len(held) - len(live)) * shape.n_ssm_layers
        is_live = t["req_state"][held] == 1
        for layer in range(shape.n_attn_layers):
            ok, ov, ocu, _ = o.gather_kv(layer, held, tot)
            assert np.array_equal(fcu, ocu) and np.array_equal(fk[layer, :tot], ok) and np.array_equal(fv[layer, :tot], ov)
        for layer in range(shape.n_ssm_layers):
            os_, oc, _ = o.gather_ssm(layer, held)
            assert np.array_equal(fs[layer, :len(held)][is_live], os_[is_live])
            assert np.array_equal(fc[layer, :len(held)][is_live], oc[is_live])
        g.ctx.clear_error()
    assert g.stats()["error_code"] == 0


def test_many_migrations_inside_one_batch(env):
    """min_interval 1: a single batch holds many migrations in both directions, so the step
    runs as several plan/copy rounds; payload must follow every relocation."""
    w = W.config("tiny", migration_batch_size=3, min_rebalance_interval_ops=1, pool_bytes=2048)
    g, o = _pair(env, w, with_store=True, max_requests=16, max_pages=8)
    rng = np.random.default_rng(3)
    for rnd in range(30):
        ops = W.random_op_string(500 + rnd, 64, 16, 60, p_invalid=0.02)
        sg, so = g.step(ops), o.step(ops)
        assert np.array_equal(sg, so)
        env["same"](g, o, w, f"round {rnd}")
        # write fresh bytes for every token / block both sides hold, then read them back
        t = o.tables()
        held = np.flatnonzero(t["req_state"] != 0).astype(np.uint32)
        lens = t["req_len"][held]
        tot = int(lens.sum())
        kb = rng.integers(0, 256, (tot, 2), dtype=np.uint8)
        vb = rng.integers(0, 256, (tot, 2), dtype=np.uint8)
        zeros = np.zeros(len(held), np.uint32)
        for e in (g, o):
            assert e.scatter_kv(0, held, zeros, kb, vb) == 0
        live = np.flatnonzero(t["req_state"] == 1).astype(np.uint32)
        sb = rng.integers(0, 256, (len(live), 80), dtype=np.uint8)
        cb = rng.integers(0, 256, (len(live), 16), dtype=np.uint8)
        for e in (g, o):
            assert e.scatter_ssm(0, live, sb, cb) == 0
        # a batch of pure growth: forces migrations that relocate what was just written
        grow = W.make_ops(W.OP_EXTEND, live, 17)
        assert np.array_equal(g.step(grow), o.step(grow))
        env["same"](g, o, w, f"round {rnd} after growth")
        t = o.tables()
        new_lens = t["req_len"][held]
        tot = int(new_lens.sum())
        gk, gv, gcu, gb = g.gather_kv(0, held, tot)
        ok, ov, ocu, ob = o.gather_kv(0, held, tot)
        assert gb == ob == 0 and np.array_equal(gcu, ocu)
        # tokens appended by `grow` were never written: compare the written prefix of each request
        src = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        for k in range(len(held)):
            a0, n_old = int(gcu[k]), int(lens[k])
            assert np.array_equal(gk[a0:a0 + n_old], kb[src[k]:src[k] + n_old])
            assert np.array_equal(gv[a0:a0 + n_old], vb[src[k]:src[k] + n_old])
            assert np.array_equal(ok[a0:a0 + n_old], kb[src[k]:src[k] + n_old])
        gs, gc, gb = g.gather_ssm(0, live)
        os_, oc, ob = o.gather_ssm(0, live)
        assert gb == ob == 0 and np.array_equal(gs, sb) and np.array_equal(gc, cb)
        assert np.array_equal(os_, sb) and np.array_equal(oc, cb)
    assert g.stats()["n_rebalance"] > 15 and g.stats()["relocated_blocks"] > 10


def _check_fused_gathers(g, h, d, w, kl, sl):
    """The multi-layer entry points (the launch configuration the benchmark times) on a range of
    layers around the written ones: the written layer against the payload function, its
    neighbours against the single-layer entry point."""
    run = d.running_slots.astype(np.uint32)
    if len(run) == 0:
        return
    m = w.model
    lens = d.len[run]
    tot = int(lens.sum())
    k0 = max(0, min(kl - 1, m.n_attn_layers - 3))
    nk = min(3, m.n_attn_layers - k0)
    gk, gv, gcu = g.gather_kv_layers(k0, nk, run, tot)
    ek, ev_, ecu = h.expected_kv(kl, d.uid[run], lens)
    assert np.array_equal(gcu, ecu)
    assert np.array_equal(gk[kl - k0][:tot], ek) and np.array_equal(gv[kl - k0][:tot], ev_)
    for l in range(nk):
        if k0 + l != kl:
            sk, sv, scu, bad = g.gather_kv(k0 + l, run, tot)
            assert bad == 0 and np.array_equal(gk[l][:tot], sk) and np.array_equal(gv[l][:tot], sv)
    s0 = max(0, min(sl - 1, m.n_ssm_layers - 3))
    ns = min(3, m.n_ssm_layers - s0)
    gs, gc = g.gather_ssm_layers(s0, ns, run)
    es, ec = h.expected_ssm(sl, d.uid[run], d.slot_epoch[run])
    assert np.array_equal(gs[sl - s0], es) and np.array_equal(gc[sl - s0], ec)
    for l in range(ns):
        if s0 + l != sl:
            ss, sc_, bad = g.gather_ssm(s0 + l, run)
            assert bad == 0 and np.array_equal(gs[l], ss) and np.array_equal(gc[l], sc_)


def _closed_loop_parity(env, w, steps, *, with_store, kv_layers, ssm_layers, table_every, gather_every,
                        max_migration_checks=10**9):
    g, o = _pair(env, w, with_store=with_store)
    engines = [g, o] if with_store else [g]
    h = PayloadHarness(w, engines, kv_layers=kv_layers, ssm_layers=ssm_layers)
    seen = dict(reb=0, tokens=0, mig_checks=0, fused=0)

    def step(ops):
        so = o.step(ops)
        sg = g.step(ops)
        assert np.array_equal(sg, so), f"statuses differ at step {d.step}"
        return so

    d = W.ClosedLoopDriver(w)

    def on_step(d, ops, status):
        h.apply_writes(d.writes)
        s = o.stats()
        migrated = s["n_rebalance"] != seen["reb"] and seen["mig_checks"] < max_migration_checks
        if migrated:
            seen["mig_checks"] += 1
        seen["reb"] = s["n_rebalance"]
        gs = g.stats()
        assert all(gs[k] == v for k, v in s.items()), f"counters differ at step {d.step}"
        if d.step % table_every == 0 or migrated:
            env["same"](g, o, w, f"step {d.step}")
        if d.step % gather_every == 0 or migrated:
            kl = kv_layers[d.step % len(kv_layers)]
            sl = ssm_layers[d.step % len(ssm_layers)]
            seen["tokens"] += h.check_gathers(d, kl, sl)
            if seen["fused"] < 3 and len(d.running_slots) > 1:      # a few times per run: it moves GBs to the host
                seen["fused"] += 1
                _check_fused_gathers(g, h, d, w, kl, sl)
            if len(d.running_slots):
                # translate of every live handle of the running batch, both implementations
                run = d.running_slots.astype(np.uint32)
                t = o.tables()
                handles = np.concatenate([t["req_chain"].reshape(w.max_requests, w.max_pages)[r, :t["req_npages"][r]]
                                          for r in run] + [t["req_ssm"].reshape(w.max_requests, -1)[run].reshape(-1)])
                pg, og, bg, ag = g.translate(handles)
                po, oo, bo = o.translate(handles)
                assert bg == bo == 0 and np.array_equal(pg, po) and np.array_equal(og, oo)
                # placement in the arena: KV units from the base up, SSM units from the end down
                st_ = o.stats()
                expect = np.where(po == 0, oo, np.uint64(st_["pool_bytes_aligned"] - st_["unit_bytes_ssm"]) - oo)
                assert np.array_equal(ag, expect)

    W.record_trace(w, step, max_steps=steps, driver=d, on_step=on_step)
    env["same"](g, o, w, "end")
    s = g.stats()
    check_invariants(s, g.tables(), page_tokens=w.model.page_tokens, n_ssm_layers=w.model.n_ssm_layers,
                     max_pages=w.max_pages)
    assert s["error_code"] == 0
    return s, seen, d


def test_pr1_every_step(env):
    """Config 1 in full: statuses every step, all tables and counters every step, full gathers
    of the running batch (GPU == oracle == payload function) every few steps."""
    w = W.config("pr1")
    s, seen, d = _closed_loop_parity(env, w, None, with_store=True, kv_layers=[0, 3], ssm_layers=[0, 11],
                                     table_every=1, gather_every=8)
    assert d.completed == 2000 and s["n_rebalance"] > 10 and s["n_oom"] > 100
    assert seen["tokens"] > 500_000


def test_pr1_small_pool_relocations(env):
    """Config 1's model in a pool small enough that migrations must move live blocks."""
    w = W.config("pr1", pool_bytes=24 * W.MiB, concurrency=12, min_rebalance_interval_ops=50,
                 migration_batch_size=6, n_requests=300)
    s, seen, d = _closed_loop_parity(env, w, 1500, with_store=True, kv_layers=[1, 2], ssm_layers=[3, 7],
                                     table_every=1, gather_every=3)
    assert s["relocated_blocks"] > 10 and s["n_rebalance"] > 5


@pytest.mark.parametrize("name,steps,over", [
    ("pr1", 1200, dict(pool_bytes=24 * W.MiB, concurrency=12, min_rebalance_interval_ops=50,
                       migration_batch_size=6, n_requests=300)),
    ("mixed_long", 300, dict(migration_batch_size=4)),
])
def test_reclaim_gap_variant(env, name, steps, over):
    """The variant of the waste rule that offers the gap between the pools again: same closed loop,
    same comparisons; capacities must differ from the paper's rule on the same trace prefix."""
    w = W.config(name, reclaim_gap=True, **over)
    small = name == "pr1"
    s, seen, d = _closed_loop_parity(env, w, steps, with_store=small, kv_layers=[1], ssm_layers=[3],
                                     table_every=1 if small else 64, gather_every=5 if small else 97,
                                     max_migration_checks=12)
    assert s["n_rebalance"] > 3 and s["wasted_bytes"] == 0
    u = (s["unit_bytes_kv"], s["unit_bytes_ssm"])
    assert s["gap_bytes"] < max(u)          # never a whole recipient unit left lying


def test_multi_layer_gathers(env):
    """avmp_gather_kv_layers / avmp_gather_ssm_layers: one launch for a range of layers gives,
    layer by layer, the oracle's single-layer gathers (and the payload function's bytes)."""
    w = W.config("pr1", pool_bytes=48 * W.MiB, concurrency=16, min_rebalance_interval_ops=50,
                 migration_batch_size=6, n_requests=120)
    g, o = _pair(env, w, with_store=True)
    h = PayloadHarness(w, [g, o])              # payload on every layer
    d = W.ClosedLoopDriver(w)

    def step(ops):
        so = o.step(ops)
        assert np.array_equal(g.step(ops), so)
        return so

    W.record_trace(w, step, max_steps=260, driver=d, on_step=lambda d, a, b: h.apply_writes(d.writes))
    assert g.stats()["n_rebalance"] > 0
    run = d.running_slots.astype(np.uint32)
    assert len(run) > 3
    tot = int(d.len[run].sum())
    m = w.model
    for first, nl in ((0, m.n_attn_layers), (1, 2), (3, 1)):
        gk, gv, gcu = g.gather_kv_layers(first, nl, run, tot)
        for l in range(nl):
            ok, ov, ocu, bad = o.gather_kv(first + l, run, tot)
            assert bad == 0 and np.array_equal(gcu, ocu)
            assert np.array_equal(gk[l][:tot], ok) and np.array_equal(gv[l][:tot], ov)
            ek, ev_, _ = h.expected_kv(first + l, d.uid[run], d.len[run])
            assert np.array_equal(gk[l][:tot], ek) and np.array_equal(gv[l][:tot], ev_)
    for first, nl in ((0, m.n_ssm_layers), (5, 3), (11, 1)):
        gs, gc = g.gather_ssm_layers(first, nl, run)
        for l in range(nl):
            os_, oc, bad = o.gather_ssm(first + l, run)
            assert bad == 0 and np.array_equal(gs[l], os_) and np.array_equal(gc[l], oc)
    # the write side for a range of layers: fresh bytes in through one launch, out through per-layer gathers
    torch = env["torch"]
    rng = np.random.default_rng(9)
    reqs = torch.from_numpy(run.view(np.int32)).cuda()
    nl = 3
    kb = rng.integers(0, 256, (nl, tot, m.kv_row_bytes), dtype=np.uint8)
    vb = rng.integers(0, 256, (nl, tot, m.kv_row_bytes), dtype=np.uint8)
    g.ctx.scatter_kv_layers(1, nl, reqs, None, len(run), torch.from_numpy(kb).cuda(), torch.from_numpy(vb).cuda(),
                            tot * m.kv_row_bytes)
    sb = rng.integers(0, 256, (4, len(run), m.state_bytes), dtype=np.uint8)
    cb = rng.integers(0, 256, (4, len(run), m.conv_bytes), dtype=np.uint8)
    g.ctx.scatter_ssm_layers(6, 4, reqs, len(run), torch.from_numpy(sb).cuda(), len(run) * m.state_bytes,
                             torch.from_numpy(cb).cuda(), len(run) * m.conv_bytes)
    for l in range(nl):
        gk, gv, _, bad = g.gather_kv(1 + l, run, tot)
        assert bad == 0 and np.array_equal(gk, kb[l]) and np.array_equal(gv, vb[l])
    for l in range(4):
        gs, gc, bad = g.gather_ssm(6 + l, run)
        assert bad == 0 and np.array_equal(gs, sb[l]) and np.array_equal(gc, cb[l])
    gk, gv, _, bad = g.gather_kv(0, run, tot)                       # untouched layers keep their bytes
    ek, ev_, _ = h.expected_kv(0, d.uid[run], d.len[run])
    assert np.array_equal(gk, ek) and np.array_equal(gv, ev_)
    assert g.stats()["error_code"] == 0


@pytest.mark.parametrize("name,steps,over", [
    ("short_uniform", 1200, {}),
    ("short_uniform", 500, dict(seed=1)),
    ("short_uniform", 500, dict(seed=2, migration_enabled=False)),
    ("mixed_long", 700, dict(migration_batch_size=4)),
    ("mixed_long", 700, dict(migration_batch_size=16)),
    ("mixed_long", 700, dict(migration_batch_size=64)),
    ("mixed_long", 150, dict(migration_batch_size=16, split=0.1)),   # the mirrored reading of "split"
    ("agentic_burst", 900, {}),
])
def test_full_size_configs(env, name, steps, over):
    """Configs 2-4 at their full pool sizes and step batches: statuses and counters every
    step, tables every 64 steps and after every migration, gathers of the running batch on
    one attention and one SSM layer against the payload function."""
    w = W.config(name, **over)
    s, seen, d = _closed_loop_parity(env, w, steps, with_store=False, kv_layers=[1], ssm_layers=[5],
                                     table_every=64, gather_every=97, max_migration_checks=12)
    assert seen["tokens"] > 0
    if w.migration_enabled and w.split != 0.1:
        assert s["n_rebalance"] > 0
    if name == "agentic_burst":
        assert s["relocated_blocks"] > 100


@pytest.mark.parametrize("name,over,n_requests,max_steps", [
    ("short_uniform", dict(seed=0), None, None),
    ("short_uniform", dict(seed=1), None, None),
    ("short_uniform", dict(seed=2), None, None),
    ("mixed_long", dict(migration_batch_size=16), None, None),
    ("mixed_long", dict(migration_batch_size=64), None, None),
    ("agentic_burst", {}, None, 20_000),
    ("scale", {}, None, None),
    ("scale", dict(split=0.9, migration_enabled=False), 30_000, None),
])
def test_full_traces_allocator_only(env, name, over, n_requests, max_steps):
    """The whole trace of every configuration (config 5: all 1 000 000 requests, 3.8e8 operations in
    370 000 steps; its static 0.9 partition on the first 30 000), allocator only: every status of every
    step, the counters every 512 steps, every table at the end."""
    w = W.config(name, **over)
    g, o = _pair(env, w)
    d = W.ClosedLoopDriver(w, requests=W.make_requests(w, n_requests) if n_requests else None)

    def step(ops):
        so = o.step(ops)
        sg = g.step(ops)
        assert np.array_equal(sg, so), f"statuses differ at step {d.step}"
        if d.step % 512 == 0:
            gs, os_ = g.stats(), o.stats()
            assert all(gs[k] == v for k, v in os_.items()), f"counters differ at step {d.step}"
        return so

    W.record_trace(w, step, max_steps=max_steps, driver=d)
    env["same"](g, o, w, "end of trace")
    s = g.stats()
    assert s["error_code"] == 0 and s["op_counter"] > 1_000_000
    if max_steps is None:
        assert d.done and s["free_kv"] == s["cap_kv"] and s["free_ssm"] == s["cap_ssm"]   # everything was returned


@pytest.mark.parametrize("split,enabled", [(0.5, True), (0.5, False), (0.9, False)])
def test_scale_config(env, split, enabled):
    """Config 5: 72-layer model, 120 GiB pool resident in HBM, step batch 1024; payload on three
    attention and three SSM layers (first, middle, last), gathers of the whole running batch on a
    rotating pair of them against the payload function."""
    w = W.config("scale", split=split, migration_enabled=enabled)
    s, seen, d = _closed_loop_parity(env, w, 240 if enabled else 120, with_store=False, kv_layers=[0, 4, 8],
                                     ssm_layers=[0, 31, 62], table_every=40, gather_every=47, max_migration_checks=4)
    assert seen["tokens"] > (1_000_000 if enabled else 500_000) and s["op_counter"] > 90_000


def test_sensitivity_sweep_cells_match_the_oracle(env):
    """The sweep of Section 4.5 (migration_batch_size, thresholds, static partition): every cell's
    summary from the GPU run equals the oracle's on the same closed loop, B = 1 behaves like the
    static partition, and changing threshold_low changes nothing."""
    from paper_2605_22416_b200 import sweep
    base = W.config("pr1", pool_bytes=96 * W.MiB, min_rebalance_interval_ops=100)
    rows_g, rows_o = [], []
    for w in sweep.cells(base, "all"):
        rows_g.append(sweep.gpu_cell(w, 400))
        o = env["Oracle"].from_workload(w)
        r = sweep.run_cell(w, o.step, o.stats, 400)
        rows_o.append(r)
    for a, b in zip(rows_g, rows_o):
        for k in b:
            if k not in ("relocation_ms", "oom_retry_share", "migration_plan_share"):
                assert a[k] == b[k], (k, a, b)
    static, b1 = rows_o[0], rows_o[1]
    assert not static["dynamic"] and b1["B"] == 1
    # one 152 KiB SSM block cannot make a 256 KiB KV page: B = 1 never migrates here and equals the
    # static partition event for event (the paper's B = 1 row equals its static total too)
    assert all(b1[k] == static[k] for k in ("n_oom", "rebalances", "completed", "ops", "cap_kv", "cap_ssm"))
    assert any(r["rebalances"] > 0 and r["relocated_mib"] > 0 for r in rows_o)
    th = [r for r in rows_o if r["dynamic"] and r["B"] == base.migration_batch_size and not r["reclaim_gap"]]
    ref = {k: v for k, v in th[0].items() if k not in ("th_low",)}
    same_high = [r for r in th if r["th_high"] == th[0]["th_high"]]
    assert len(same_high) >= 3
    for r in same_high:
        assert {k: v for k, v in r.items() if k != "th_low"} == ref   # stage-2 null result


@pytest.mark.parametrize("name,steps,over", [
    ("pr1", 900, dict(pool_bytes=40 * W.MiB, min_rebalance_interval_ops=100)),       # OOMs, pre-emptions
    ("pr1", 400, dict(pool_bytes=8 * W.MiB, migration_enabled=False, n_requests=300)),  # unservable drops
    ("pr1", 500, dict(pool_bytes=40 * W.MiB, min_rebalance_interval_ops=100, reclaim_gap=True)),
    ("short_uniform", 500, {}),
    ("mixed_long", 400, dict(migration_batch_size=64)),
    ("scale", 60, {}),
])
def test_device_closed_loop_matches_host_loop(env, name, steps, over):
    """The on-device scheduler (batch built and statuses folded back by kernels, no host round trip)
    ends in exactly the state the host-side batch builder reaches against the oracle: allocator
    tables and counters, request slots, queue position, every scheduler counter."""
    from paper_2605_22416_b200 import binding as B
    w = W.config(name, **over)
    reqs = W.make_requests(w, min(w.n_requests, 40_000))
    g = env["GpuEngine"](w)
    dd = B.DeviceDriver(g.ctx, reqs.prompt, reqs.output, w.concurrency)
    for _ in range(steps):
        dd.step()
    o = env["Oracle"].from_workload(w)
    d = W.ClosedLoopDriver(w, requests=reqs)
    n = 0
    while n < steps:
        ops = d.next_batch()
        d.feed(o.step(ops))
        n += 1
    env["same"](g, o, w, "device loop vs host loop")
    ds, ex = dd.stats(), dd.export()
    assert ds["steps"] == steps and ds["overflow"] == 0
    assert ds["completed"] == d.completed and ds["dropped"] == d.dropped and ds["preempted"] == d.preempted
    assert ds["n_oom_admit"] == d.n_oom_admit and ds["n_oom_extend"] == d.n_oom_extend
    assert ds["window"] == d.window
    assert ds["queue_next"] - ds["requeued"] == d._next - len(d.front)
    run = d.state == 1
    assert np.array_equal(ex["state"] == 1, run)
    assert np.array_equal(ex["uid"][run], d.uid[run].astype(np.uint32))
    assert np.array_equal(ex["len"][run], d.len[run].astype(np.uint32))
    assert np.array_equal(ex["remaining"][run], d.remaining[run].astype(np.uint32))
    assert g.stats()["error_code"] == 0
    if name == "pr1":
        assert d.n_oom_admit > 0 and (d.preempted > 0 or d.dropped > 0)
    dd.close()


@pytest.mark.parametrize("name,over,n_requests", [
    ("pr1", {}, None),
    ("short_uniform", {}, None),
    ("mixed_long", dict(migration_batch_size=16), None),
    ("scale", {}, 60_000),
])
def test_device_loop_whole_traces(env, name, over, n_requests):
    """The on-device loop run until its request list is exhausted (config 5: its first 60 000 requests),
    step for step beside the host loop on the oracle: counters every 5000 steps, everything at the end."""
    from paper_2605_22416_b200 import binding as B
    w = W.config(name, **over)
    reqs = W.make_requests(w, n_requests) if n_requests else W.make_requests(w)
    g, o = _pair(env, w)
    dd = B.DeviceDriver(g.ctx, reqs.prompt, reqs.output, w.concurrency)
    d = W.ClosedLoopDriver(w, requests=reqs)
    n = 0
    while not d.done:
        dd.step()
        d.feed(o.step(d.next_batch()))
        n += 1
        if n % 5000 == 0:
            ds = dd.stats()
            assert (ds["completed"], ds["preempted"], ds["dropped"]) == (d.completed, d.preempted, d.dropped), n
            env["same"](g, o, w, f"{name} at step {n}")
    ds = dd.stats()
    assert (ds["completed"], ds["preempted"], ds["dropped"]) == (d.completed, d.preempted, d.dropped)
    assert ds["n_oom_admit"] == d.n_oom_admit and ds["n_oom_extend"] == d.n_oom_extend and ds["overflow"] == 0
    assert d.completed + d.dropped == len(reqs.prompt) and ds["steps"] == n
    env["same"](g, o, w, f"{name} end of trace")
    assert (dd.export()["state"] == 0).all() and g.stats()["error_code"] == 0
    dd.close()


@pytest.mark.parametrize("steps,over", [
    (20_000, {}),                                                         # the whole arrival horizon
    (1200, dict(pool_bytes=3 * W.GiB)),                                  # tight: evictions, failed resumes
    (900, dict(pool_bytes=2 * W.GiB, concurrency=64, split=0.3)),         # pre-emptions, no free slot
    (700, dict(pool_bytes=3 * W.GiB, max_requests=96, concurrency=96)),   # slots run out before memory
    (600, dict(pool_bytes=3 * W.GiB, reclaim_gap=True, migration_batch_size=32)),
    (800, dict(max_requests=24, concurrency=24)),                         # parked sessions hold every slot
])
def test_device_session_loop_matches_host_loop(env, steps, over):
    """The on-device scheduler for multi-turn sessions (arrivals, parking with KEEP_KV, resume after the
    think time, eviction of the longest-parked chain, pre-emption, drops) against the host-side batch
    builder running on the oracle: allocator tables and counters, every slot, both queues in order and
    every scheduler counter, compared every 100 steps (every 1000 on the long run)."""
    from paper_2605_22416_b200 import binding as B
    w = W.config("agentic_burst", **over)
    ses = W.make_sessions(w)
    g = env["GpuEngine"](w)
    sd = B.SessionDriver(g.ctx, ses.arrival_step, ses.n_turns, ses.turn_prompt, ses.turn_output, ses.turn_think,
                         w.concurrency)
    o = env["Oracle"].from_workload(w)
    d = W.ClosedLoopDriver(w, sessions=ses)
    done = 0
    while done < steps:
        n = min(100 if steps <= 2000 else 1000, steps - done)
        for _ in range(n):
            sd.step()
            d.feed(o.step(d.next_batch()))
        done += n
        what = f"session loop at step {done}"
        ds, ex = sd.stats(), sd.export()
        for k in ("completed", "dropped", "preempted", "evicted", "n_oom_admit", "n_oom_extend", "window"):
            assert ds[k] == getattr(d, k), (what, k, ds[k], getattr(d, k))
        assert ds["steps"] == done and ds["arrived"] == d._next and ds["arrival_queue"] == len(d.back), what
        assert ex["requeued"].tolist() == [e.uid for e in d.front], what
        assert ex["waiting"].tolist() == [e.uid for _, _, e in d.resume_q], what
        forced = list(d._forced)
        assert ds["forced_slot"] == (forced[0] if forced else 2**64 - 1), what
        assert np.array_equal(ex["state"], d.state.astype(np.uint32)), what
        held = d.state != 0
        for k, a in (("uid", d.uid), ("len", d.len), ("turn", d.turn)):
            assert np.array_equal(ex[k][held], a[held].astype(np.uint32)), (what, k)
        run = d.state == 1
        assert np.array_equal(ex["remaining"][run], d.remaining[run].astype(np.uint32)), what
        env["same"](g, o, w, what)
    assert g.stats()["error_code"] == 0
    assert d.completed > 0 and (d.evicted > 0 or (d.state == 2).any())
    sd.close()


@pytest.mark.parametrize("kind", ["queue", "sessions"])
def test_device_loop_replayed_from_a_cuda_graph(env, kind):
    """Fifty engine steps of the on-device loop captured once in a CUDA graph and replayed ten
    times: same final state as five hundred steps of the host loop on the oracle."""
    torch = env["torch"]
    from paper_2605_22416_b200 import binding as B
    if kind == "queue":
        w = W.config("pr1", pool_bytes=40 * W.MiB, min_rebalance_interval_ops=100)
        reqs = W.make_requests(w)
        g = env["GpuEngine"](w)
        dd = B.DeviceDriver(g.ctx, reqs.prompt, reqs.output, w.concurrency)
        host = dict(requests=reqs)
    else:
        w = W.config("agentic_burst", pool_bytes=3 * W.GiB)
        ses = W.make_sessions(w)
        g = env["GpuEngine"](w)
        dd = B.SessionDriver(g.ctx, ses.arrival_step, ses.n_turns, ses.turn_prompt, ses.turn_output,
                             ses.turn_think, w.concurrency)
        host = dict(sessions=ses)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            for _ in range(50):
                dd.step(stream)
    for _ in range(10):
        graph.replay()
    torch.cuda.synchronize()
    o = env["Oracle"].from_workload(w)
    d = W.ClosedLoopDriver(w, **host)
    for _ in range(500):
        d.feed(o.step(d.next_batch()))
    env["same"](g, o, w, "graph replay vs host loop")
    ds = dd.stats()
    assert ds["steps"] == 500 and ds["completed"] == d.completed and ds["preempted"] == d.preempted
    assert g.stats()["n_rebalance"] > 0
    dd.close()


def test_edge_cases(env):
    w = W.config("tiny")
    g, o = _pair(env, w, with_store=True)
    assert len(g.step(np.zeros(0, W.OP_DTYPE))) == 0                     # empty batch
    ops = W.make_ops(W.OP_ADMIT, [0, 1], [20, 5])
    assert np.array_equal(g.step(ops), o.step(ops))
    fin = W.make_ops(W.OP_FINISH, [1], 0, W.FLAG_KEEP_KV)
    assert np.array_equal(g.step(fin), o.step(fin))
    # gather error items: empty slot, capacity overflow, KV_ONLY request in an SSM gather
    for reqs, cap in (([0, 3, 1], 25), ([0, 1], 22), ([0, 1], 25), ([], 0)):
        gk, gv, gcu, gb = g.gather_kv(0, reqs, cap)
        ok, ov, ocu, ob = o.gather_kv(0, reqs, cap)
        assert gb == ob and np.array_equal(gcu, ocu), (reqs, cap)
    assert g.stats()["error_code"] in (2, 3) and g.stats()["error_count"] == 2
    g.ctx.clear_error()
    assert g.stats()["error_count"] == 0
    gs, gc, gb = g.gather_ssm(0, [0, 1])
    assert gb == 1 and g.stats()["error_code"] == 2
    # translate: dead and out-of-range handles
    hs = np.array([0, 1, 2, 0xFFFFFFFF, (1 << 31) | 0, (1 << 31) | 1, 500], np.uint32)
    pg, og, bg, _ = g.translate(hs)
    po, oo, bo = o.translate(hs)
    assert bg == bo == 3 and np.array_equal(pg, po) and np.array_equal(og, oo)
    # host-buffer entry point
    ops = W.random_op_string(9, 200, 8, 40)
    assert np.array_equal(g.step_host(ops), o.step(ops))
    env["same"](g, o, w, "after step_host")


@pytest.mark.parametrize("n_list", [1024, 1025, 3000])
def test_long_request_lists(env, n_list):
    """KV gathers plan inside the copy kernel up to 1024 requests and through a separate plan kernel
    beyond: a few requests repeated in a long list, on both sides of the switch, single-layer and
    multi-layer, against the oracle."""
    w = W.config("pr1", pool_bytes=64 * W.MiB, max_requests=3008)     # a list may not exceed the slot table
    g, o = _pair(env, w, with_store=True)
    h = PayloadHarness(w, [g, o], kv_layers=[0, 1, 2], ssm_layers=[1])
    d = W.ClosedLoopDriver(w)

    def step(ops):
        so = o.step(ops)
        assert np.array_equal(g.step(ops), so)
        return so

    W.record_trace(w, step, max_steps=40, driver=d, on_step=lambda d, a, b: h.apply_writes(d.writes))
    run = np.flatnonzero(d.state == 1).astype(np.uint32)
    assert len(run) >= 8
    reqs = np.resize(run[:6], n_list).astype(np.uint32)
    reqs[5::97] = 2000                                           # a few empty slots in between
    total = int(o.tables()["req_len"][reqs].sum())
    for layer in (0, 2):
        gk, gv, gcu, gb = g.gather_kv(layer, reqs, total)
        ok, ov, ocu, ob = o.gather_kv(layer, reqs, total)
        assert gb == ob and np.array_equal(gcu, ocu)
        assert np.array_equal(gk, ok) and np.array_equal(gv, ov)
    fk, fv, fcu = g.gather_kv_layers(0, 3, reqs, total)
    for l in range(3):
        ok, ov, ocu, _ = o.gather_kv(l, reqs, total)
        assert np.array_equal(fk[l, :total], ok) and np.array_equal(fv[l, :total], ov) and np.array_equal(fcu, ocu)
    g.ctx.clear_error()


def test_kv_gathers_on_two_streams(env):
    """Two KV gathers with different request lists issued on two streams (they may overlap on the GPU):
    lists of up to 1024 requests are planned inside each launch, so the results equal the ones of the
    same calls issued one after the other."""
    torch = env["torch"]
    w = W.config("short_uniform", concurrency=96)
    g = env["GpuEngine"](w)
    n = 90
    lens = (np.arange(n) * 37 % 300 + 20).astype(np.uint32)
    assert (g.step(W.make_ops(W.OP_ADMIT, np.arange(n), lens)) == 0).all()
    dev, row = g.dev, w.model.kv_row_bytes
    rng = np.random.default_rng(5)
    lists = [rng.permutation(n)[:70].astype(np.uint32), rng.permutation(n)[:55].astype(np.uint32)]
    tot = [int(lens[l].sum()) for l in lists]
    # payload: every page of the arena gets bytes of its own
    g.ctx.arena[:].copy_(torch.randint(0, 256, (g.ctx.arena.numel(),), dtype=torch.uint8, device=dev))
    d_lists = [torch.from_numpy(l.view(np.int32)).to(dev) for l in lists]

    def buffers():
        return [(torch.zeros((t, row), dtype=torch.uint8, device=dev), torch.zeros((t, row), dtype=torch.uint8, device=dev),
                 torch.zeros(len(l) + 1, dtype=torch.int32, device=dev)) for t, l in zip(tot, lists)]

    ref = buffers()
    for i in range(2):
        g.ctx.gather_kv(i, d_lists[i], len(lists[i]), ref[i][0], ref[i][1], tot[i], ref[i][2])
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for rep in range(20):
        out = buffers()
        torch.cuda.synchronize()
        for i in range(2):
            g.ctx.gather_kv(i, d_lists[i], len(lists[i]), out[i][0], out[i][1], tot[i], out[i][2],
                            stream=streams[i].cuda_stream)
        torch.cuda.synchronize()
        for i in range(2):
            assert all(torch.equal(a, b) for a, b in zip(out[i], ref[i])), (rep, i)
    assert g.stats()["error_code"] == 0


def test_both_pools_short_in_one_op(env):
    """An admit short in both pools: SSM handler first (migrates), then the KV handler (throttled)."""
    w = W.config("tiny", pool_bytes=2048, migration_batch_size=3)
    g, o = _pair(env, w, max_requests=12, max_pages=8)
    ops = np.concatenate([W.make_ops(W.OP_ADMIT, np.arange(10), 1), W.make_ops(W.OP_ADMIT, [10], 96)])
    sg, so = g.step(ops), o.step(ops)
    assert np.array_equal(sg, so) and so[-1] == W.ST_OOM
    s = g.stats()
    assert (s["n_capacity_error"], s["n_rebalance"], s["cap_kv"], s["free_kv"], s["cap_ssm"], s["free_ssm"]) == (2, 1, 13, 3, 12, 2)
    env["same"](g, o, w, "both short")


def test_create_rejects_bad_configurations(env):
    from paper_2605_22416_b200 import binding as B
    torch = env["torch"]
    spec = B.model_spec(W.TINY_MODEL)
    arena = torch.empty(4096, dtype=torch.uint8, device="cuda")
    opt = B.avmp_default_options()
    opt.max_requests, opt.max_pages_per_request = 4, 4
    ws_bytes = B.avmp_workspace_bytes(spec, 1024, opt)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    bad = B.avmp_options(300_000, 300_000, 1000, 1, 4, 4)        # threshold_low >= threshold_high
    with pytest.raises(B.AvmpError):
        B.avmp_create(spec, arena, 1024, 0.5, 1, bad, ws, ws_bytes)
    with pytest.raises(B.AvmpError):
        B.avmp_create(spec, arena, 1024, 0.5, 1, opt, ws, ws_bytes - 256)   # workspace too small
    with pytest.raises(B.AvmpError):
        B.avmp_create(spec, arena, 1024, 1.5, 1, opt, ws, ws_bytes)          # split outside [0, 1]
    with pytest.raises(B.AvmpError):
        B.avmp_create(spec, arena.data_ptr() + 8, 1024, 0.5, 1, opt, ws, ws_bytes)  # misaligned arena
    h = B.avmp_create(spec, arena, 1024, 0.5, 1, opt, ws, ws_bytes)
    B.avmp_destroy(h)


def test_export_import_roundtrip(env):
    """Snapshot / restore: tables built by the oracle drive the GPU gathers directly."""
    w = W.config("pr1", pool_bytes=24 * W.MiB, concurrency=12, min_rebalance_interval_ops=50,
                 migration_batch_size=6, n_requests=60)
    g, o = _pair(env, w, with_store=True)
    h = PayloadHarness(w, [g, o], kv_layers=[0], ssm_layers=[0])
    d = W.ClosedLoopDriver(w)

    def step(ops):
        so = o.step(ops)
        assert np.array_equal(g.step(ops), so)
        return so

    W.record_trace(w, step, max_steps=150, driver=d, on_step=lambda d, a, b: h.apply_writes(d.writes))
    tables, stats = g.ctx.export_tables()
    g2 = env["GpuEngine"](w, arena=g.ctx.arena)           # same payload bytes, fresh tables
    g2.ctx.import_tables(o.tables(), o.stats())            # tables from the ORACLE
    env["same"](g2, o, w, "imported")
    assert h.check_gathers(d, 0, 0, engines=[g2]) > 0
    # and the imported context keeps stepping identically
    def step2(ops):
        so = o.step(ops)
        assert np.array_equal(g2.step(ops), so)
        return so

    W.record_trace(w, step2, max_steps=200, driver=d)
    env["same"](g2, o, w, "after more steps")


def test_import_rejects_inconsistent_snapshots(env):
    """A snapshot that the kernels could not have produced is refused on the host and the context stays
    as it was: the kernels index the tables without bounds checks."""
    from paper_2605_22416_b200.binding import AvmpError
    w = W.config("pr1", pool_bytes=24 * W.MiB, concurrency=12, min_rebalance_interval_ops=50,
                 migration_batch_size=6, n_requests=60)
    g, o = _pair(env, w)
    d = W.ClosedLoopDriver(w)

    def step(ops):
        so = o.step(ops)
        assert np.array_equal(g.step(ops), so)
        return so

    W.record_trace(w, step, max_steps=120, driver=d)
    good_t, good_s = g.ctx.export_tables()
    assert good_s["n_rebalance"] > 0 and (good_t["req_state"] == 1).sum() >= 4
    live = int(np.flatnonzero(good_t["req_state"] == 1)[0])
    mp, ns = g.max_pages, w.model.n_ssm_layers

    def variant(f_tables=None, f_stats=None):
        t = {k: v.copy() for k, v in good_t.items()}
        s = dict(good_s)
        if f_tables: f_tables(t)
        if f_stats: f_stats(s)
        return t, s

    def set_(key, idx, val):
        def f(t): t[key][idx] = val
        return f

    bad = {
        "free slot beyond the store": variant(set_("slot_stack_kv", 0, good_s["cap_kv"])),
        "free slot twice": variant(set_("slot_stack_ssm", 0, int(good_t["slot_stack_ssm"][1]))),
        "chain handle beyond the id space": variant(set_("req_chain", live * mp, good_s["vid_space_kv"] + 5)),
        "chain handle of a free id": variant(set_("req_chain", live * mp, int(good_t["vid_stack_kv"][0]))),
        "chain handle with the SSM tag": variant(set_("req_chain", live * mp, int(good_t["req_chain"][live * mp]) | (1 << 31))),
        "SSM handle held twice": variant(set_("req_ssm", live * ns, int(good_t["req_ssm"][live * ns + 1]))),
        "page table entry beyond the store": variant(set_("vt_kv", int(good_t["req_chain"][live * mp]), good_s["cap_kv"] + 1)),
        "owner table not the inverse": variant(set_("ow_ssm", int(good_t["vt_ssm"][int(good_t["req_ssm"][live * ns]) & 0x7FFFFFFF]), 0x12345)),
        "length does not match the pages": variant(set_("req_len", live, int(good_t["req_len"][live]) + 64)),
        "unknown request state": variant(set_("req_state", live, 7)),
        "capacity does not conserve the pool": variant(None, lambda s: s.__setitem__("cap_kv", s["cap_kv"] + 1)),
        "last rebalance in the future": variant(None, lambda s: s.__setitem__("last_rebalance_op", s["op_counter"] + 9)),
    }
    for what, (t, s) in bad.items():
        with pytest.raises(AvmpError):
            g.ctx.import_tables(t, s)
        env["same"](g, o, w, f"context untouched after: {what}")
    g.ctx.import_tables(good_t, good_s)                     # the unmodified snapshot goes in
    env["same"](g, o, w, "after importing the good snapshot")
    ops = d.next_batch()
    assert np.array_equal(g.step(ops), o.step(ops))


def test_import_rejects_a_held_request_without_tokens(env):
    """ADMIT and EXTEND take at least one token, so no sequence of operations leaves a held request
    with zero tokens; a snapshot that says otherwise (its page returned to the free lists by hand, every
    other table consistent) is refused, so the gathers never meet a request without rows."""
    from paper_2605_22416_b200.binding import AvmpError
    w = W.config("tiny")
    g, o = _pair(env, w)
    ops = W.make_ops(W.OP_ADMIT, [0], 1)
    assert np.array_equal(g.step(ops), o.step(ops))
    t, s = g.ctx.export_tables()
    g.ctx.import_tables(t, s)                                   # as exported: accepted
    h = int(t["req_chain"][0])
    slot = int(t["vt_kv"][h])
    t["slot_stack_kv"] = np.append(t["slot_stack_kv"], np.uint32(slot))
    t["vid_stack_kv"] = np.append(t["vid_stack_kv"], np.uint32(h))
    t["vt_kv"][h] = 0xFFFFFFFF
    t["ow_kv"][slot] = 0xFFFFFFFF
    t["req_len"][0] = 0
    t["req_npages"][0] = 0
    s["free_kv"] += 1
    with pytest.raises(AvmpError):
        g.ctx.import_tables(t, s)
    env["same"](g, o, w, "context untouched")


@pytest.mark.parametrize("shape", range(2))
def test_bytes_inside_a_unit_follow_the_documented_layout_on_gpu(env, shape):
    """The same raw-byte check as the oracle's pin, on the device arena: handles resolved with
    avmp_translate (d_arena_offset), the unit read straight from the arena tensor and viewed as
    [layer][K, V][token][head][dim] (state then window for SSM blocks), after migrations have
    relocated some of the written units.  Shape 0 takes the bulk-copy kernels, shape 1 the generic ones."""
    from harness import LAYOUT_SHAPES, check_unit_layout, layout_workload
    w = layout_workload(LAYOUT_SHAPES[shape])
    g = env["GpuEngine"](w)
    s = g.stats()
    unit = (s["unit_bytes_kv"], s["unit_bytes_ssm"])
    arena = g.ctx.arena

    def read_units(pool, handles):
        p, off, bad, aoff = g.translate(np.asarray(handles, np.uint32))
        assert bad == 0 and (p == pool).all()
        return [arena[int(a): int(a) + unit[pool]].cpu().numpy() for a in aoff]

    seen = check_unit_layout(w, g, read_units)
    assert seen["kv_rows"] > 1000 and seen["ssm_blocks"] > 40 and seen["relocated_blocks"] > 4
    assert g.stats()["error_code"] == 0
    # and the same bytes through the oracle's stores: both sides place every byte alike
    o = env["Oracle"].from_workload(w, with_store=True)

    def read_units_o(pool, handles):
        p, off, bad = o.translate(np.asarray(handles, np.uint32))
        return [o.store_bytes(pool, int(x), unit[pool]) for x in off]

    assert check_unit_layout(w, o, read_units_o) == seen
    env["same"](g, o, w, "layout run")


@pytest.mark.parametrize("n_list", [0, 8, 1024, 1500])
def test_step_gather_in_one_launch(env, n_list):
    """avmp_gather_step: every attention layer and every SSM layer of a request list in one launch equals the
    oracle's single-layer gathers (and the multi-layer entry points); lists on both sides of the 1024-entry
    plan switch, with empty slots in between; layer sub-ranges; a buffer one row too small."""
    w = W.config("pr1", pool_bytes=64 * W.MiB, max_requests=1536, concurrency=16, min_rebalance_interval_ops=50,
                 migration_batch_size=6, n_requests=120)
    g, o = _pair(env, w, with_store=True)
    h = PayloadHarness(w, [g, o])
    d = W.ClosedLoopDriver(w)

    def step(ops):
        so = o.step(ops)
        assert np.array_equal(g.step(ops), so)
        return so

    W.record_trace(w, step, max_steps=120, driver=d, on_step=lambda d, a, b: h.apply_writes(d.writes))
    assert g.stats()["n_rebalance"] > 0
    m = w.model
    run = d.running_slots.astype(np.uint32)
    assert len(run) >= 8
    reqs = np.resize(run[:8], n_list).astype(np.uint32)
    if n_list > 8:
        reqs[4::53] = 1400                                       # empty slots
    n_empty = int((reqs == 1400).sum())
    tot = int(o.tables()["req_len"][reqs].sum())

    def check(kv_first, kv_n, ssm_first, ssm_n, cap):
        fk, fv, fcu, fs, fc, bad = g.gather_step(kv_first, kv_n, ssm_first, ssm_n, reqs, cap)
        want_bad = 0
        for l in range(kv_n):
            ok, ov, ocu, ob = o.gather_kv(kv_first + l, reqs, cap)
            want_bad += ob if l == 0 else 0                      # the KV plan reports a list's bad items once
            assert np.array_equal(fcu, ocu)
            assert np.array_equal(fk[l, :cap], ok) and np.array_equal(fv[l, :cap], ov), (l, cap)
        for l in range(ssm_n):
            os_, oc, ob = o.gather_ssm(ssm_first + l, reqs)
            want_bad += ob
            assert np.array_equal(fs[l, :len(reqs)], os_) and np.array_equal(fc[l, :len(reqs)], oc), l
        assert bad == want_bad and want_bad == n_empty * (1 + ssm_n) + (1 if cap < tot else 0)
        return fk, fv, fs, fc

    fk, fv, fs, fc = check(0, m.n_attn_layers, 0, m.n_ssm_layers, tot)
    if n_list:
        gk, gv, _ = g.gather_kv_layers(0, m.n_attn_layers, reqs, tot)
        gs, gc = g.gather_ssm_layers(0, m.n_ssm_layers, reqs)
        assert np.array_equal(fk, gk) and np.array_equal(fv, gv) and np.array_equal(fs, gs) and np.array_equal(fc, gc)
        check(1, 2, 7, 3, tot)
        check(3, 1, 11, 1, tot - 1)                               # the last request does not fit: it copies nothing
    g.ctx.clear_error()


@pytest.mark.parametrize("name,steps,over", [
    ("pr1", 500, dict(pool_bytes=24 * W.MiB, concurrency=12, min_rebalance_interval_ops=50, migration_batch_size=6,
                      n_requests=300)),                                            # relocations in most migrations
    ("tiny", 60, dict(min_rebalance_interval_ops=1, migration_batch_size=2)),      # several rounds per step
    ("short_uniform", 300, dict(migration_enabled=False)),                         # no relocation launch at all
    ("short_uniform", 400, {}),
])
def test_step_translate_equals_step_then_translate(env, name, steps, over):
    """avmp_step_translate (the translation rides on the step's relocation-copy launch): statuses, tables and the
    translation of a handle list against the tables AFTER the step -- the handles every slot held before the
    step, so some are dead by then and some were relocated by the step's migration."""
    w = W.config(name, **over)
    g, o = _pair(env, w)
    d = W.ClosedLoopDriver(w)
    seen = dict(dead=0, handles=0)
    for _ in range(steps):
        if d.done:
            break
        t = o.tables()
        held = np.flatnonzero(t["req_state"] != 0)
        chain = t["req_chain"].reshape(w.max_requests, w.max_pages)
        ssm = t["req_ssm"].reshape(w.max_requests, -1)
        handles = np.concatenate([chain[r, :t["req_npages"][r]] for r in held] +
                                 [ssm[r] for r in held if t["req_state"][r] == 1] + [np.zeros(0, np.uint32)]).astype(np.uint32)
        ops = d.next_batch()
        so = o.step(ops)
        po, oo, bo = o.translate(handles)
        sg, pg, og, bg, ag = g.step_translate(ops, handles)
        assert np.array_equal(sg, so) and bg == bo
        assert np.array_equal(pg, po) and np.array_equal(og, oo)
        st_ = o.stats()
        live = po != 0xFFFFFFFF
        expect = np.where(po == 0, oo, np.uint64(st_["pool_bytes_aligned"] - st_["unit_bytes_ssm"]) - oo)
        assert np.array_equal(ag[live], expect[live])
        seen["dead"] += bo
        seen["handles"] += len(handles)
        d.feed(so)
        if d.step % 50 == 0:
            env["same"](g, o, w, f"step {d.step}")
        g.ctx.clear_error()
    env["same"](g, o, w, "end")
    assert seen["handles"] > 500 and seen["dead"] > 0
    if w.migration_enabled:
        assert g.stats()["n_rebalance"] > 0


@pytest.mark.parametrize("case,slots,pool_kib,interval,tokens", [
    (0, 8, 1, 4, 40),            # the hand-sized pool: shortages and migrations in most batches
    (1, 40, 6, 7, 60),
    (2, 300, 40_000, 100, 200),  # two windows of 256 ops: the shape is judged per window
    (3, 300, 2_000, 50, 200),    # the same, tight
    (4, 1500, 12_000, 300, 120), # 1024-op windows; tight enough for OOM storms
    (5, 1500, 400_000, 1000, 120),
])
def test_engine_shaped_batches_with_shared_slots(env, case, slots, pool_kib, interval, tokens):
    """Batches in an engine step's order (FINISH*, EXTEND*, ADMIT*, ascending slots inside a kind -- the shape the
    step kernel recognises and handles without its same-slot table) whose kinds share slots: finished and admitted
    again in one batch, parked with KEEP_KV and resumed, extended and admitted; every third batch also repeats some
    ops back to back (equal slots inside a kind: no longer that shape).  Statuses and every table against the
    oracle after every batch."""
    model = W.TINY_MODEL if case < 2 else W.SMALL_UNIT_MODEL
    w = W.Workload(f"shaped{case}", model, pool_kib * 1024, 0.5, 1 + case % 3 if case < 2 else 16 * (1 + case % 3),
                   slots, slots, 16, "queue", 0, min_rebalance_interval_ops=interval, reclaim_gap=bool(case % 2))
    g, o = _pair(env, w)
    rounds = 120 if slots <= 300 else 40
    shortages = 0
    for rnd in range(rounds):
        ops = W.engine_shaped_batch(1000 * case + rnd, slots, tokens, p_pick=0.25 + 0.5 * ((rnd * 7) % 10) / 10,
                                    repeats=rnd % 3 == 2)
        if len(ops) == 0:
            continue
        sg, so = g.step(ops), o.step(ops)
        assert np.array_equal(sg, so), (case, rnd, np.flatnonzero(sg != so)[:10], sg[sg != so][:10], so[sg != so][:10])
        shortages += int((so == W.ST_OOM).sum())
        if rnd % 4 == 0 or slots <= 40:
            env["same"](g, o, w, f"case {case} round {rnd}")
    env["same"](g, o, w, "end")
    s = g.stats()
    check_invariants(s, g.tables(), page_tokens=16, n_ssm_layers=model.n_ssm_layers, max_pages=16)
    assert s["n_invalid"] > 0                      # shared slots make some ops BAD_REQ, as they must
    if case in (0, 1, 3, 4):
        assert shortages > 0 and s["n_rebalance"] > 0
