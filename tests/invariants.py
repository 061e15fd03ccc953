"""Structural invariants of an AVMP state (tables + counters), whoever produced it."""
from __future__ import annotations

import numpy as np

INVALID = 0xFFFFFFFF
EMPTY, LIVE, KV_ONLY = 0, 1, 2


def check_invariants(stats: dict, t: dict, *, page_tokens: int, n_ssm_layers: int, max_pages: int):
    U = (stats["unit_bytes_kv"], stats["unit_bytes_ssm"])
    cap = (stats["cap_kv"], stats["cap_ssm"])
    free = (stats["free_kv"], stats["free_ssm"])
    V = (stats["vid_space_kv"], stats["vid_space_ssm"])
    # pool bytes are conserved: both stores plus the gap make up the aligned pool
    assert cap[0] * U[0] + cap[1] * U[1] + stats["gap_bytes"] == stats["pool_bytes_aligned"]
    used_units = [0, 0]
    for p, name in enumerate(("kv", "ssm")):
        S, W = t[f"slot_stack_{name}"], t[f"vid_stack_{name}"]
        VT, OW = t[f"vt_{name}"], t[f"ow_{name}"]
        assert len(S) == free[p]
        assert len(np.unique(S)) == len(S) and (len(S) == 0 or S.max() < cap[p])
        assert len(np.unique(W)) == len(W) and (len(W) == 0 or W.max() < V[p])
        live_v = np.flatnonzero(VT != INVALID)
        live_s = np.flatnonzero(OW != INVALID)
        used = cap[p] - free[p]
        used_units[p] = used
        assert len(live_v) == used and len(live_s) == used
        assert len(W) == V[p] - used
        # VT and OW are mutually inverse on live entries; no slot is mapped twice
        assert (OW[VT[live_v]] == live_v).all()
        assert (VT[OW[live_s]] == live_s).all()
        assert len(live_s) == 0 or live_s.max() < cap[p]
        # free and live partition [0, cap)
        assert not np.intersect1d(S, live_s).size
        assert not np.intersect1d(W, live_v).size
    st, ln, npg = t["req_state"], t["req_len"], t["req_npages"]
    R = len(st)
    chain = t["req_chain"].reshape(R, max_pages)
    ssm = t["req_ssm"].reshape(R, max(n_ssm_layers, 1))[:, :n_ssm_layers] if n_ssm_layers else None
    holds = st != EMPTY
    assert (npg[~holds] == 0).all() and (ln[~holds] == 0).all()
    assert (ln[holds] >= 1).all()          # a held request has at least one token: zero-token ops are rejected
    assert (npg == -(-ln.astype(np.int64) // page_tokens)).all()
    kv_handles = np.concatenate([chain[r, :npg[r]] for r in np.flatnonzero(holds)] or [np.zeros(0, np.uint32)])
    assert len(kv_handles) == used_units[0]
    assert (kv_handles >> 31 == 0).all()
    assert len(np.unique(kv_handles)) == len(kv_handles)
    assert (t["vt_kv"][kv_handles & 0x7FFFFFFF] != INVALID).all()   # every handle resolves
    live = st == LIVE
    if n_ssm_layers:
        sh = ssm[live].reshape(-1)
        assert len(sh) == used_units[1]
        assert (sh >> 31 == 1).all()
        assert len(np.unique(sh)) == len(sh)
        assert (t["vt_ssm"][sh & 0x7FFFFFFF] != INVALID).all()
    else:
        assert used_units[1] == 0
