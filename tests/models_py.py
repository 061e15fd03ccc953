"""Independent pure-Python models used to pin the C oracle (test code only).

Three models, each written separately from the oracle and from one another:

* `StaticDualPool`   -- two fixed pools, two integers each, no handles, no migration:
                         the static dual-pool baseline the paper compares with (Section 4.1,
                         "Baseline fidelity"); its OOM sequence must equal AVMP's with migration
                         off (Section 1.1, first contribution).
* `CountsModel`      -- AVMP's rebalancer reduced to unit counts (Section 3.2): whether an
                         operation succeeds depends only on counts, so this checks the policy
                         independently of free lists and page tables.
* `NaiveAllocator`   -- handles, slots and chains kept in dicts and Python lists, with
                         erase/insert list surgery instead of array stacks; payload kept per
                         request as dense shadow copies.  Only for tiny inputs.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

ADMIT, EXTEND, FINISH = 1, 2, 3
KEEP_KV, RESUME = 1, 2
OK, OOM, BAD_REQ, TOO_LONG, BAD_ARG = 0, 1, 2, 3, 4
EMPTY, LIVE, KV_ONLY = 0, 1, 2
INVALID = 0xFFFFFFFF


def unit_sizes(model):
    """Section 3.1 unit sizes: KV page = page_tokens x per-token bytes (K and V of every
    attention layer); SSM block = one layer's state elements x element bytes."""
    kv = model.n_attn_layers * 2 * model.page_tokens * model.kv_heads * model.head_dim * model.kv_elem_bytes
    ssm = (model.ssm_state_elems + model.ssm_conv_elems) * model.ssm_elem_bytes
    up16 = lambda x: -(-x // 16) * 16
    return up16(kv), up16(ssm)


def initial_caps(model, pool_bytes, split):
    u_kv, u_ssm = unit_sizes(model)
    p_al = pool_bytes // 128 * 128
    ssm_bytes = (p_al * round(split * 1e6) // 10**6) // 128 * 128
    return (p_al - ssm_bytes) // u_kv, ssm_bytes // u_ssm, p_al


class _ReqCounts:
    """Shared request bookkeeping for the two counts-only models."""

    def __init__(self, model, max_requests, max_pages):
        self.T = model.page_tokens
        self.ns = model.n_ssm_layers
        self.max_requests, self.max_pages = max_requests, max_pages
        self.state = [EMPTY] * max_requests
        self.len = [0] * max_requests
        self.pages = [0] * max_requests

    def classify(self, kind, flags, req, tokens):
        """-> (status or None, need_kv, need_ssm, new_len)."""
        if kind not in (ADMIT, EXTEND, FINISH):
            return BAD_ARG, 0, 0, 0
        if req >= self.max_requests:
            return BAD_REQ, 0, 0, 0
        st = self.state[req]
        if kind == FINISH:
            return (None if st in (LIVE, KV_ONLY) else BAD_REQ), 0, 0, 0
        if tokens == 0:
            return BAD_ARG, 0, 0, 0
        if kind == ADMIT:
            want = KV_ONLY if flags & RESUME else EMPTY
            if st != want:
                return BAD_REQ, 0, 0, 0
        elif st != LIVE:
            return BAD_REQ, 0, 0, 0
        new_len = self.len[req] + tokens
        pages = -(-new_len // self.T)
        if pages > self.max_pages:
            return TOO_LONG, 0, 0, 0
        return None, pages - self.pages[req], (self.ns if kind == ADMIT else 0), new_len


class StaticDualPool(_ReqCounts):
    """Two static regions sized once at start-up; an operation that does not fit is an OOM."""

    def __init__(self, model, pool_bytes, split, max_requests, max_pages):
        super().__init__(model, max_requests, max_pages)
        self.kv_total, self.ssm_total, _ = initial_caps(model, pool_bytes, split)
        self.kv_used = self.ssm_used = 0
        self.n_oom = 0

    def op(self, kind, flags, req, tokens):
        st, nk, ns, new_len = self.classify(kind, flags, req, tokens)
        if st is not None:
            return st
        if kind == FINISH:
            if not flags & KEEP_KV:
                self.kv_used -= self.pages[req]
                self.pages[req] = self.len[req] = 0
            if self.state[req] == LIVE:
                self.ssm_used -= self.ns
            self.state[req] = KV_ONLY if flags & KEEP_KV else EMPTY
            return OK
        if self.ssm_used + ns > self.ssm_total or self.kv_used + nk > self.kv_total:
            self.n_oom += 1
            return OOM
        self.ssm_used += ns
        self.kv_used += nk
        self.pages[req] += nk
        self.len[req] = new_len
        self.state[req] = LIVE
        return OK


class CountsModel(_ReqCounts):
    """Section 3.2 with units only: capacities, free counts, the logical clock, the throttle,
    the threshold_high trigger and the waste formula."""

    def __init__(self, model, pool_bytes, split, B, max_requests, max_pages, *, th_high_ppm=300_000,
                 min_interval=1000, enabled=True, reclaim=False):
        super().__init__(model, max_requests, max_pages)
        kv, ssm, p_al = initial_caps(model, pool_bytes, split)
        self.U = list(unit_sizes(model))
        self.cap = [kv, ssm]
        self.free = [kv, ssm]
        self.p_al, self.reclaim = p_al, reclaim
        self.B, self.th_high, self.min_interval, self.enabled = B, th_high_ppm, min_interval, enabled
        self.clock = 0
        self.last: Optional[int] = None
        self.n_oom = self.n_rebalance = self.migrated = self.wasted = self.n_capacity_error = 0
        self.events: List[dict] = []

    def _handler(self, x):
        y = 1 - x
        self.n_capacity_error += 1
        if not self.enabled or self.cap[y] == 0:
            return
        # free fraction of the other pool strictly above threshold_high
        if not self.free[y] * 10**6 > self.th_high * self.cap[y]:
            return
        if self.last is not None and self.clock - self.last < self.min_interval:
            return
        n = min(self.B, self.free[y])
        gain, waste = divmod(n * self.U[y], self.U[x])
        if self.reclaim:
            # everything between the two pools after the donor shrank is on offer (no stored gap:
            # the middle follows from the capacities)
            middle = self.p_al - (self.cap[y] - n) * self.U[y] - self.cap[x] * self.U[x]
            gain, waste = middle // self.U[x], 0
        if gain == 0:
            return
        self.events.append(dict(clock=self.clock, donor=y, n=n, gain=gain, waste=waste,
                                donor_free=self.free[y], donor_cap=self.cap[y]))
        self.cap[y] -= n
        self.free[y] -= n
        self.cap[x] += gain
        self.free[x] += gain
        self.migrated += n * self.U[y]
        self.wasted += waste
        self.n_rebalance += 1
        self.last = self.clock

    def op(self, kind, flags, req, tokens):
        self.clock += 1
        st, nk, ns, new_len = self.classify(kind, flags, req, tokens)
        if st is not None:
            return st
        if kind == FINISH:
            if not flags & KEEP_KV:
                self.free[0] += self.pages[req]
                self.pages[req] = self.len[req] = 0
            if self.state[req] == LIVE:
                self.free[1] += self.ns
            self.state[req] = KV_ONLY if flags & KEEP_KV else EMPTY
            return OK
        if ns > self.free[1]:
            self._handler(1)
        if nk > self.free[0]:
            self._handler(0)
        if ns > self.free[1] or nk > self.free[0]:
            self.n_oom += 1
            return OOM
        self.free[1] -= ns
        self.free[0] -= nk
        self.pages[req] += nk
        self.len[req] = new_len
        self.state[req] = LIVE
        return OK


@dataclass
class _NaiveReq:
    state: int = EMPTY
    length: int = 0
    chain: List[int] = None
    ssm: List[int] = None


class NaiveAllocator:
    """Brute-force AVMP for tiny pools.  Free slots / ids are Python lists whose *front* is
    the next one handed out (so every pop is an erase at index 0 and every free an insert at
    index 0 -- the mirror image of an array stack).  Payload lives in `bytes_at[pool][slot]`."""

    def __init__(self, model, pool_bytes, split, B, max_requests, max_pages, *, th_high_ppm=300_000,
                 min_interval=1000, enabled=True, reclaim=False):
        self.model = model
        kv, ssm, p_al = initial_caps(model, pool_bytes, split)
        self.p_al, self.reclaim = p_al, reclaim
        self.U = list(unit_sizes(model))
        self.cap = [kv, ssm]
        self.next_slots = [list(range(kv)), list(range(ssm))]
        self.next_ids = [list(range(p_al // self.U[0])), list(range(p_al // self.U[1]))]
        self.where: List[Dict[int, int]] = [{}, {}]          # id -> slot, live only
        self.bytes_at: List[Dict[int, bytearray]] = [{}, {}]  # slot -> payload
        self.B, self.th_high, self.min_interval, self.enabled = B, th_high_ppm, min_interval, enabled
        self.max_requests, self.max_pages = max_requests, max_pages
        self.reqs = [_NaiveReq(chain=[], ssm=[]) for _ in range(max_requests)]
        self.clock = 0
        self.last = None
        self.n_oom = self.n_rebalance = self.relocated = 0

    def _take(self, p):
        slot = self.next_slots[p].pop(0)
        ident = self.next_ids[p].pop(0)
        self.where[p][ident] = slot
        self.bytes_at[p].setdefault(slot, bytearray(self.U[p]))
        return (p << 31) | ident

    def _give(self, h):
        p, ident = h >> 31, h & 0x7FFFFFFF
        slot = self.where[p].pop(ident)
        self.next_slots[p].insert(0, slot)
        self.next_ids[p].insert(0, ident)

    def _handler(self, x):
        y = 1 - x
        if not self.enabled or self.cap[y] == 0:
            return
        nfree = len(self.next_slots[y])
        if not nfree * 10**6 > self.th_high * self.cap[y]:
            return
        if self.last is not None and self.clock - self.last < self.min_interval:
            return
        n = min(self.B, nfree)
        gain = n * self.U[y] // self.U[x]
        if self.reclaim:
            gain = (self.p_al - (self.cap[y] - n) * self.U[y] - self.cap[x] * self.U[x]) // self.U[x]
        if gain == 0:
            return
        newcap = self.cap[y] - n
        self.next_slots[y] = [s for s in self.next_slots[y] if s < newcap]
        slot_owner = {s: i for i, s in self.where[y].items()}
        for s in sorted(s for s in slot_owner if s >= newcap):
            d = self.next_slots[y].pop(0)
            self.bytes_at[y][d] = bytearray(self.bytes_at[y][s])
            self.where[y][slot_owner[s]] = d
            self.relocated += 1
        self.cap[y] = newcap
        self.next_slots[x] = list(range(self.cap[x], self.cap[x] + gain)) + self.next_slots[x]
        self.cap[x] += gain
        self.n_rebalance += 1
        self.last = self.clock

    def op(self, kind, flags, req, tokens):
        self.clock += 1
        m = self.model
        if kind not in (ADMIT, EXTEND, FINISH):
            return BAD_ARG
        if req >= self.max_requests:
            return BAD_REQ
        r = self.reqs[req]
        if kind == FINISH:
            if r.state not in (LIVE, KV_ONLY):
                return BAD_REQ
            if not flags & KEEP_KV:
                for h in r.chain:
                    self._give(h)
                r.chain, r.length = [], 0
            if r.state == LIVE:
                for h in r.ssm:
                    self._give(h)
                r.ssm = []
            r.state = KV_ONLY if flags & KEEP_KV else EMPTY
            return OK
        if tokens == 0:
            return BAD_ARG
        if kind == ADMIT:
            if r.state != (KV_ONLY if flags & RESUME else EMPTY):
                return BAD_REQ
        elif r.state != LIVE:
            return BAD_REQ
        pages = -(-(r.length + tokens) // m.page_tokens)
        if pages > self.max_pages:
            return TOO_LONG
        nk = pages - len(r.chain)
        ns = m.n_ssm_layers if kind == ADMIT else 0
        if ns > len(self.next_slots[1]):
            self._handler(1)
        if nk > len(self.next_slots[0]):
            self._handler(0)
        if ns > len(self.next_slots[1]) or nk > len(self.next_slots[0]):
            self.n_oom += 1
            return OOM
        if ns:
            r.ssm = [self._take(1) for _ in range(ns)]
        r.chain += [self._take(0) for _ in range(nk)]
        r.length += tokens
        r.state = LIVE
        return OK

    # -- payload access by (request, layer, token) ----------------------------------
    def kv_row(self, req, layer, part, t):
        m = self.model
        row = m.kv_heads * m.head_dim * m.kv_elem_bytes
        h = self.reqs[req].chain[t // m.page_tokens]
        slot = self.where[0][h & 0x7FFFFFFF]
        off = layer * 2 * m.page_tokens * row + part * m.page_tokens * row + (t % m.page_tokens) * row
        return self.bytes_at[0][slot], off, row

    def ssm_block(self, req, layer):
        h = self.reqs[req].ssm[layer]
        return self.bytes_at[1][self.where[1][h & 0x7FFFFFFF]]
