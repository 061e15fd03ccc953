"""Randomised differential pins for the oracle (hypothesis): random cache shapes, pool sizes,
splits, migration_batch_size, throttle intervals and thresholds, random op strings with repeats
and invalid ops -- statuses, capacities and counters must equal the separately written models
after every op, and the structural invariants must hold.  No GPU needed."""
from __future__ import annotations

import numpy as np
from hypothesis import HealthCheck, given, settings, strategies as st

import models_py as M
from invariants import check_invariants
from oracle.avmp_oracle import Oracle
from paper_2605_22416_b200 import workloads as W

shapes = st.builds(
    W.ModelShape,
    n_attn_layers=st.integers(1, 3), n_ssm_layers=st.integers(1, 4), page_tokens=st.sampled_from([4, 16]),
    kv_heads=st.integers(1, 2), head_dim=st.sampled_from([1, 4, 8]), kv_elem_bytes=st.just(2),
    ssm_state_elems=st.integers(3, 40), ssm_conv_elems=st.integers(1, 9), ssm_elem_bytes=st.just(4),
)


@settings(max_examples=60, deadline=None, suppress_health_check=[HealthCheck.too_slow])
@given(shape=shapes, pool_units=st.integers(6, 40), split=st.sampled_from([0.0, 0.2, 0.5, 0.8, 1.0]),
       B=st.integers(1, 9), interval=st.integers(1, 12), th_high=st.sampled_from([100_000, 300_000, 600_000]),
       seed=st.integers(0, 10_000), enabled=st.booleans(), reclaim=st.booleans())
def test_oracle_equals_naive_and_counts_models(shape, pool_units, split, B, interval, th_high, seed, enabled,
                                               reclaim):
    u_kv, u_ssm = M.unit_sizes(shape)
    pool = pool_units * max(u_kv, u_ssm)
    kv0, ssm0, _ = M.initial_caps(shape, pool, split)
    if kv0 == 0 and ssm0 == 0:
        return
    R, MP = 5, 6
    kw = dict(th_high_ppm=th_high, min_interval=interval, enabled=enabled, reclaim=reclaim)
    o = Oracle(shape, pool, split, B, max_requests=R, max_pages=MP, threshold_low_ppm=50_000,
               threshold_high_ppm=th_high, min_rebalance_interval_ops=interval, migration_enabled=enabled,
               reclaim_gap=reclaim)
    nv = M.NaiveAllocator(shape, pool, split, B, R, MP, **kw)
    cm = M.CountsModel(shape, pool, split, B, R, MP, **kw)
    ops = W.random_op_string(seed, 120, R, shape.page_tokens * 4, p_invalid=0.08)
    for i in range(len(ops)):
        k, f, r, t = (int(ops[c][i]) for c in ("kind", "flags", "req", "tokens"))
        got = int(o.step(ops[i:i + 1])[0])
        assert got == nv.op(k, f, r, t) == cm.op(k, f, r, t), (i, k, f, r, t)
    s = o.stats()
    assert [s["cap_kv"], s["cap_ssm"]] == nv.cap == cm.cap
    assert [s["free_kv"], s["free_ssm"]] == cm.free
    assert s["n_oom"] == nv.n_oom == cm.n_oom and s["n_rebalance"] == nv.n_rebalance == cm.n_rebalance
    assert s["migrated_bytes"] == cm.migrated and s["wasted_bytes"] == cm.wasted
    assert s["relocated_blocks"] == nv.relocated and s["op_counter"] == len(ops)
    t = o.tables()
    chain = t["req_chain"].reshape(R, MP)
    for q in range(R):
        assert chain[q, :len(nv.reqs[q].chain)].tolist() == nv.reqs[q].chain
    check_invariants(s, t, page_tokens=shape.page_tokens, n_ssm_layers=shape.n_ssm_layers, max_pages=MP)
