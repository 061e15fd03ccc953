"""Seeded synthetic inputs for the AVMP hot path: model shapes, request lists, a
closed-loop batch builder and the payload byte function.

This module is shared by the CUDA path's tests/bench and by the CPU oracle's
tests.  It holds *inputs only*: shapes, random lengths, the engine-side scheduling
loop that turns per-op statuses into the next batch, and the bytes that a model
would write into its cache.  None of the allocator's arithmetic (unit sizes,
capacities, free lists, migration) lives here; both implementations consume the
arrays produced here and nothing else.

The five workload recipes follow the configurations named for this build; they
stand in for the paper's synthetic traces (Section 4.1: `uniform_short`,
`mixed_long`, `agentic_burst`), whose generator is not published.
"""
from __future__ import annotations

import math
from collections import deque
from dataclasses import dataclass, field, replace
from typing import Callable, Deque, List, Optional, Tuple

import numpy as np

# ----------------------------------------------------------------------------
# Wire format of one allocator operation (12 bytes, little endian).
# ----------------------------------------------------------------------------
OP_DTYPE = np.dtype(
    [("kind", "u1"), ("flags", "u1"), ("rsvd", "<u2"), ("req", "<u4"), ("tokens", "<u4")]
)
assert OP_DTYPE.itemsize == 12

OP_ADMIT, OP_EXTEND, OP_FINISH = 1, 2, 3
FLAG_KEEP_KV, FLAG_RESUME = 1, 2
ST_OK, ST_OOM, ST_BAD_REQ, ST_TOO_LONG, ST_BAD_ARG = 0, 1, 2, 3, 4

PAYLOAD_K, PAYLOAD_V, PAYLOAD_STATE, PAYLOAD_CONV = 0, 1, 2, 3


def make_ops(kind, req, tokens=0, flags=0) -> np.ndarray:
    """Build an op array from broadcastable columns."""
    req = np.atleast_1d(np.asarray(req, dtype=np.uint32))
    ops = np.zeros(req.shape[0], dtype=OP_DTYPE)
    ops["kind"] = kind
    ops["flags"] = flags
    ops["req"] = req
    ops["tokens"] = tokens
    return ops


# ----------------------------------------------------------------------------
# Counter-based random numbers (no hidden state: value = f(seed, stream, index)).
# ----------------------------------------------------------------------------
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)


def _mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 output function on a uint64 array (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        x = np.asarray(x, dtype=np.uint64).copy()
        x ^= x >> np.uint64(30)
        x *= np.uint64(0xBF58476D1CE4E5B9)
        x ^= x >> np.uint64(27)
        x *= np.uint64(0x94D049BB133111EB)
        x ^= x >> np.uint64(31)
    return x


_M64 = 0xFFFFFFFFFFFFFFFF


def _mix64_int(x: int) -> int:
    """The same function on one Python integer."""
    x ^= x >> 30
    x = (x * 0xBF58476D1CE4E5B9) & _M64
    x ^= x >> 27
    x = (x * 0x94D049BB133111EB) & _M64
    return x ^ (x >> 31)


def _key(seed: int, stream: int) -> np.uint64:
    a = _mix64_int(seed & _M64)
    b = _mix64_int((((stream + 0x1234567) & _M64) * 0x9E3779B97F4A7C15) & _M64)
    return np.uint64(_mix64_int(a ^ b))


def rand_u64(seed: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    idx = np.arange(start, start + n, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix64(_key(seed, stream) + (idx + np.uint64(1)) * _GOLDEN)


def rand_unit(seed: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    """Uniform doubles in [0, 1)."""
    return (rand_u64(seed, stream, n, start) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def rand_int(seed: int, stream: int, n: int, lo: int, hi: int, start: int = 0) -> np.ndarray:
    """Uniform integers in [lo, hi] inclusive."""
    u = rand_unit(seed, stream, n, start)
    return np.minimum(lo + np.floor(u * (hi - lo + 1)).astype(np.int64), hi)


def rand_normal(seed: int, stream: int, n: int) -> np.ndarray:
    """Standard normals by Box-Muller from two uniform streams."""
    u1 = 1.0 - rand_unit(seed, 2 * stream + 1000, n)  # (0, 1]
    u2 = rand_unit(seed, 2 * stream + 1001, n)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)


def rand_lognormal_int(seed, stream, n, median, sigma, lo, hi) -> np.ndarray:
    z = rand_normal(seed, stream, n)
    v = np.rint(np.exp(math.log(median) + sigma * z)).astype(np.int64)
    return np.clip(v, lo, hi)


def poisson_from_unit(u: float, mean: float) -> int:
    """Inverse-CDF Poisson draw from one uniform (small means only)."""
    p = math.exp(-mean)
    c = p
    k = 0
    while u > c and k < 10 * int(mean) + 100:
        k += 1
        p *= mean / k
        c += p
    return k


# ----------------------------------------------------------------------------
# Payload: the bytes a model would have written for (request uid, layer, part,
# token).  A pure function, so the expected content of any gather depends only on
# (uid, length), never on where an allocator placed the data.
# ----------------------------------------------------------------------------
def payload_bytes(seed: int, uid: int, epoch: int, layer: int, part: int,
                  row_start: int, n_rows: int, row_bytes: int) -> np.ndarray:
    """uint8[n_rows, row_bytes]: rows [row_start, row_start + n_rows) of the byte stream
    keyed by (seed, uid, epoch, layer, part).  A row is a token (K / V) or the whole
    state / conv block (row 0).  K / V use epoch 0; SSM state uses the admission epoch."""
    b0 = row_start * row_bytes
    b1 = (row_start + n_rows) * row_bytes
    w0, w1 = b0 // 8, -(-b1 // 8)
    w = _stream_words(_key(seed ^ 0x5EED, (uid * 64 + epoch) * 4096 + layer * 4 + part), w0, w1)
    b = w.astype("<u8", copy=False).view(np.uint8)[b0 - w0 * 8: b1 - w0 * 8]
    return b.reshape(n_rows, row_bytes)


def _stream_words(k: np.uint64, w0: int, w1: int, chunk: int = 1 << 16) -> np.ndarray:
    """Words [w0, w1) of the stream with key k: mix64(k + (i + 1) * golden).  Generated in
    cache-sized pieces with in-place arithmetic; long streams would otherwise be bound by the
    page faults of their temporaries."""
    out = np.empty(w1 - w0, np.uint64)
    with np.errstate(over="ignore"):
        for s in range(w0, w1, chunk):
            e = min(s + chunk, w1)
            x = np.arange(s + 1, e + 1, dtype=np.uint64)
            x *= _GOLDEN
            x += k
            t = x >> np.uint64(30)
            x ^= t
            x *= np.uint64(0xBF58476D1CE4E5B9)
            np.right_shift(x, np.uint64(27), out=t)
            x ^= t
            x *= np.uint64(0x94D049BB133111EB)
            np.right_shift(x, np.uint64(31), out=t)
            x ^= t
            out[s - w0:e - w0] = x
    return out


def payload_single_rows(seed: int, uids, epochs, layer: int, part: int, rows, row_bytes: int) -> np.ndarray:
    """uint8[n, row_bytes]: row rows[i] of the stream of (uids[i], epochs[i]) -- the same bytes as
    one payload_bytes call per item, computed in one pass when rows are whole 8-byte words."""
    n = len(uids)
    if n == 0:
        return np.zeros((0, row_bytes), np.uint8)
    if row_bytes % 8 or row_bytes > 8192:      # long rows: one cache-sized stream at a time
        out = np.empty((n, row_bytes), np.uint8)
        for i, (u, e, r) in enumerate(zip(uids, epochs, rows)):
            out[i] = payload_bytes(seed, int(u), int(e), layer, part, int(r), 1, row_bytes)[0]
        return out
    wpr = row_bytes // 8
    keys = np.array([_key(seed ^ 0x5EED, (int(u) * 64 + int(e)) * 4096 + layer * 4 + part)
                     for u, e in zip(uids, epochs)], dtype=np.uint64)
    with np.errstate(over="ignore"):
        idx = (np.asarray(rows, dtype=np.uint64) * np.uint64(wpr))[:, None] + np.arange(wpr, dtype=np.uint64)[None, :]
        w = _mix64(keys[:, None] + (idx + np.uint64(1)) * _GOLDEN)
    return w.astype("<u8").view(np.uint8).reshape(n, row_bytes)


# ----------------------------------------------------------------------------
# Shapes.
# ----------------------------------------------------------------------------
@dataclass(frozen=True)
class ModelShape:
    n_attn_layers: int
    n_ssm_layers: int
    page_tokens: int
    kv_heads: int
    head_dim: int
    kv_elem_bytes: int
    ssm_state_elems: int
    ssm_conv_elems: int
    ssm_elem_bytes: int

    @property
    def kv_row_bytes(self) -> int:
        """Bytes of one token's K (or V) in one attention layer: a row of the batch buffer."""
        return self.kv_heads * self.head_dim * self.kv_elem_bytes

    @property
    def state_bytes(self) -> int:
        return self.ssm_state_elems * self.ssm_elem_bytes

    @property
    def conv_bytes(self) -> int:
        return self.ssm_conv_elems * self.ssm_elem_bytes


PR1_MODEL = ModelShape(4, 12, 16, 8, 128, 2, 2048 * 16, 2048 * 3, 4)
JAMBA_LIKE = ModelShape(4, 28, 16, 8, 128, 2, 8192 * 16, 8192 * 3, 4)
SCALE_MODEL = ModelShape(9, 63, 16, 8, 128, 2, 16384 * 16, 16384 * 3, 4)
TINY_MODEL = ModelShape(1, 1, 16, 1, 1, 2, 20, 4, 4)  # 64-byte pages, 96-byte blocks
SMALL_UNIT_MODEL = ModelShape(1, 2, 16, 1, 64, 2, 256, 64, 4)  # 4 KiB pages, 1280-byte blocks: many units per GiB

MiB = 1 << 20
GiB = 1 << 30


@dataclass(frozen=True)
class Workload:
    name: str
    model: ModelShape
    pool_bytes: int
    split: float                # fraction of pool bytes given to the SSM pool at start
    migration_batch_size: int
    concurrency: int            # running requests = step batch
    max_requests: int           # request slot table
    max_pages: int              # longest chain, in pages
    kind: str                   # "queue" | "sessions"
    n_requests: int
    seed: int = 0
    migration_enabled: bool = True
    reclaim_gap: bool = False          # variant: gap bytes are offered again at the next migration
    min_rebalance_interval_ops: int = 1000
    threshold_low_ppm: int = 50_000
    threshold_high_ppm: int = 300_000
    session_steps: int = 20_000  # "sessions" only: arrival horizon in steps

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def config(name: str, **overrides) -> Workload:
    """The five named workloads (plus `tiny`), optionally overridden."""
    base = {
        "pr1": Workload("pr1", PR1_MODEL, 256 * MiB, 0.5, 8, 32, 32, 40, "queue", 2000),
        "short_uniform": Workload("short_uniform", JAMBA_LIKE, 4 * GiB, 0.5, 128, 256, 256, 24, "queue", 100_000),
        "mixed_long": Workload("mixed_long", JAMBA_LIKE, 16 * GiB, 0.9, 16, 128, 128, 4128, "queue", 20_000),
        "agentic_burst": Workload("agentic_burst", JAMBA_LIKE, 8 * GiB, 0.5, 128, 256, 4096, 1152, "sessions", 0),
        "scale": Workload("scale", SCALE_MODEL, 120 * GiB, 0.5, 128, 1024, 1024, 4096, "queue", 1_000_000),
        "tiny": Workload("tiny", TINY_MODEL, 1024, 0.5, 3, 4, 8, 8, "queue", 64,
                         min_rebalance_interval_ops=4),
    }[name]
    return replace(base, **overrides) if overrides else base


CONFIG_NAMES = ("pr1", "short_uniform", "mixed_long", "agentic_burst", "scale")


# ----------------------------------------------------------------------------
# Request lists.
# ----------------------------------------------------------------------------
@dataclass
class RequestList:
    prompt: np.ndarray   # int64[n]
    output: np.ndarray   # int64[n]


def make_requests(w: Workload, n: Optional[int] = None) -> RequestList:
    """Length pairs for the queue-type workloads; deterministic in (name, seed, index)."""
    n = w.n_requests if n is None else n
    s = w.seed
    if w.name == "pr1":
        p = rand_int(s, 1, n, 32, 512)
        o = rand_int(s, 2, n, 16, 128)
    elif w.name == "short_uniform":
        p = rand_int(s, 1, n, 16, 256)
        o = rand_int(s, 2, n, 16, 128)
    elif w.name == "mixed_long":
        short = rand_lognormal_int(s, 1, n, 512.0, 0.8, 1, 16384)
        long_ = rand_int(s, 3, n, 16384, 65536)
        is_long = rand_unit(s, 4, n) < 0.2
        p = np.where(is_long, long_, short)
        o = rand_int(s, 2, n, 64, 512)
    elif w.name == "scale":
        p = rand_lognormal_int(s, 1, n, 200.0, 1.0, 1, 32768)
        o = rand_lognormal_int(s, 2, n, 250.0, 0.9, 1, 32768)
    elif w.name == "tiny":
        p = rand_int(s, 1, n, 1, 70)
        o = rand_int(s, 2, n, 1, 20)
    elif w.name.startswith("alloc_micro"):
        p = rand_int(s, 1, n, 16, 256)
        o = rand_int(s, 2, n, 16, 128)
    else:
        raise ValueError(f"no queue recipe for {w.name}")
    return RequestList(p.astype(np.int64), o.astype(np.int64))


@dataclass
class SessionList:
    arrival_step: np.ndarray      # int64[n_sessions]
    n_turns: np.ndarray           # int64[n_sessions]
    turn_prompt: np.ndarray       # int64[n_sessions, 8]
    turn_output: np.ndarray       # int64[n_sessions, 8]
    turn_think: np.ndarray        # int64[n_sessions, 8]


def make_sessions(w: Workload) -> SessionList:
    """Bursts of multi-turn sessions: one Poisson(64) burst every 50 steps."""
    s = w.seed
    n_bursts = (w.session_steps + 49) // 50
    u = rand_unit(s, 10, n_bursts)
    sizes = np.array([poisson_from_unit(float(x), 64.0) for x in u], dtype=np.int64)
    n = int(sizes.sum())
    arrival = np.repeat(np.arange(n_bursts, dtype=np.int64) * 50, sizes)
    return SessionList(
        arrival_step=arrival,
        n_turns=rand_int(s, 11, n, 2, 8),
        turn_prompt=rand_int(s, 12, n * 8, 256, 2048).reshape(n, 8),
        turn_output=rand_int(s, 13, n * 8, 64, 256).reshape(n, 8),
        turn_think=rand_int(s, 14, n * 8, 10, 100).reshape(n, 8),
    )


# ----------------------------------------------------------------------------
# Closed-loop batch builder.
# ----------------------------------------------------------------------------
_FREE, _RUNNING, _PARKED = 0, 1, 2


@dataclass
class _Entry:
    uid: int
    prompt: int          # tokens to append on admission
    output: int          # decode tokens of this turn
    turn: int = 0
    resume_slot: int = -1  # >= 0: the parked slot whose chain is kept


@dataclass
class TokenWrite:
    """Tokens [start, end) of request `uid` became valid in slot `slot` this step."""
    slot: int
    uid: int
    epoch: int       # bumps at every admission of this uid (selects the SSM payload)
    start: int
    end: int
    is_admit: bool


class ClosedLoopDriver:
    """Turns per-op statuses into the next step's batch, the way a serving engine would.

    One step = one batch: FINISH for requests whose decode is complete (ascending
    slot), EXTEND by one token for every other running request (ascending slot),
    then ADMITs from the queue head into the lowest slots that were free when the
    step began, while running < concurrency.  Admission uses a slow-start window:
    any failed admit shrinks it to one admit per step, a step whose admits all
    succeed doubles it.  Failed admits go back to the queue head; a failed EXTEND
    stalls that request for the step.  A step in which no op succeeded pre-empts the
    most recently admitted running request (plain FINISH, re-queued at the head with
    its whole context as the prompt).  An admit that fails with nothing running is
    dropped as unservable.  Multi-turn sessions park between turns (FINISH with
    KEEP_KV) and resume after their think time; a step that ran out of memory, or in
    which an admission found no free slot, evicts the longest-parked session's chain
    (plain FINISH; it re-enters as a fresh admit with its whole context as the prompt).
    """

    def __init__(self, w: Workload, requests: Optional[RequestList] = None,
                 sessions: Optional[SessionList] = None):
        self.w = w
        R = w.max_requests
        self.state = np.zeros(R, dtype=np.int8)
        self.uid = np.full(R, -1, dtype=np.int64)
        self.len = np.zeros(R, dtype=np.int64)
        self.remaining = np.zeros(R, dtype=np.int64)
        self.turn = np.zeros(R, dtype=np.int64)
        self.admit_seq = np.zeros(R, dtype=np.int64)
        self.slot_epoch = np.zeros(R, dtype=np.int64)
        self.epoch_of_uid: dict = {}
        self._seq = 0
        self.step = 0
        self.front: Deque[_Entry] = deque()     # re-queued entries (served first)
        self.back: Deque[_Entry] = deque()      # arrived sessions waiting for a first admission
        self.resume_q: List[Tuple[int, int, _Entry]] = []   # (ready_step, seq, entry), kept sorted
        self.parked: dict = {}                  # slot -> (park_seq, entry)
        self.window = w.concurrency
        self._forced: dict = {}                 # slot -> "preempt" | "drop" | "evict"
        self._starved = False                   # the last batch left an entry without a slot
        self.completed = self.dropped = self.preempted = self.evicted = 0
        self.n_oom_admit = self.n_oom_extend = 0
        self.writes: List[TokenWrite] = []
        self._pending = None
        self._next = 0
        if w.kind == "queue":
            self.requests = requests if requests is not None else make_requests(w)
            self.sessions = None
        else:
            self.sessions = sessions if sessions is not None else make_sessions(w)
            self.requests = None

    # -- queue plumbing -------------------------------------------------------
    def _arrivals(self):
        if self.sessions is None:
            return
        s = self.sessions
        while self._next < len(s.arrival_step) and s.arrival_step[self._next] <= self.step:
            i = self._next
            self.back.append(_Entry(i, int(s.turn_prompt[i, 0]), int(s.turn_output[i, 0]), 0))
            self._next += 1

    def _pop_entry(self) -> Optional[_Entry]:
        if self.front:
            return self.front.popleft()
        if self.resume_q and self.resume_q[0][0] <= self.step:
            return self.resume_q.pop(0)[2]
        if self.sessions is not None:
            return self.back.popleft() if self.back else None
        if self._next < len(self.requests.prompt):
            i = self._next
            self._next += 1
            return _Entry(i, int(self.requests.prompt[i]), int(self.requests.output[i]))
        return None

    @property
    def done(self) -> bool:
        if (self.state != _FREE).any() or self.front or self.resume_q or self._forced:
            return False
        if self.sessions is not None:
            return not self.back and self._next >= len(self.sessions.arrival_step)
        return self._next >= len(self.requests.prompt)

    @property
    def running_slots(self) -> np.ndarray:
        return np.flatnonzero(self.state == _RUNNING)

    # -- one step ---------------------------------------------------------------
    def next_batch(self) -> np.ndarray:
        self._arrivals()
        running = self.state == _RUNNING
        fin_mask = running & (self.remaining == 0)
        forced = dict(self._forced)
        for slot, why in forced.items():
            fin_mask[slot] = True
            if why == "evict":
                # the parked chain goes away now: its resume entry becomes a fresh admission
                _, e = self.parked.pop(slot)
                e.prompt += int(self.len[slot])
                e.resume_slot = -1
        fin = np.flatnonzero(fin_mask)
        ext = np.flatnonzero(running & ~fin_mask)
        fin_flags = np.zeros(len(fin), dtype=np.uint8)
        if self.sessions is not None and len(fin):
            more = self.turn[fin] + 1 < self.sessions.n_turns[self.uid[fin]]
            more &= ~np.isin(fin, np.fromiter(forced.keys(), dtype=np.int64, count=len(forced)))
            fin_flags[more] = FLAG_KEEP_KV
        budget = min(self.w.concurrency - len(ext), self.window)
        free_slots = np.flatnonzero(self.state == _FREE)
        n_free_used = 0
        self._starved = False
        admits: List[Tuple[_Entry, int]] = []
        while budget > 0:
            e = self._pop_entry()
            if e is None:
                break
            if e.resume_slot >= 0:
                slot = e.resume_slot
            elif n_free_used < len(free_slots):
                slot = int(free_slots[n_free_used])
                n_free_used += 1
            else:
                self.front.appendleft(e)
                self._starved = True
                break
            admits.append((e, slot))
            budget -= 1
        ops = np.zeros(len(fin) + len(ext) + len(admits), dtype=OP_DTYPE)
        a, b = len(fin), len(fin) + len(ext)
        ops["kind"][:a] = OP_FINISH
        ops["flags"][:a] = fin_flags
        ops["req"][:a] = fin
        ops["kind"][a:b] = OP_EXTEND
        ops["req"][a:b] = ext
        ops["tokens"][a:b] = 1
        for j, (e, slot) in enumerate(admits):
            ops["kind"][b + j] = OP_ADMIT
            ops["flags"][b + j] = FLAG_RESUME if e.resume_slot >= 0 else 0
            ops["req"][b + j] = slot
            ops["tokens"][b + j] = e.prompt
        self._pending = (fin, fin_flags, ext, admits, forced)
        return ops

    def feed(self, status: np.ndarray) -> None:
        fin, fin_flags, ext, admits, forced = self._pending
        self._pending = None
        self._forced = {}
        status = np.asarray(status)
        a, b = len(fin), len(fin) + len(ext)
        assert len(status) == b + len(admits)
        self.writes = []
        progress = False
        oom_seen = False
        # FINISH
        if a:
            assert (status[:a] == ST_OK).all(), "FINISH of a held request cannot fail"
            progress = True
            for slot, fl in zip(fin.tolist(), fin_flags.tolist()):
                uid = int(self.uid[slot])
                why = forced.get(slot)
                if why == "preempt":
                    self.front.appendleft(_Entry(uid, int(self.len[slot]), int(self.remaining[slot]),
                                                 int(self.turn[slot])))
                    self.preempted += 1
                elif why == "drop":
                    self.parked.pop(slot, None)
                    self.dropped += 1
                elif why == "evict":
                    self.evicted += 1
                elif fl & FLAG_KEEP_KV:
                    t = int(self.turn[slot]) + 1
                    s = self.sessions
                    ready = self.step + 1 + int(s.turn_think[uid, t - 1])
                    e = _Entry(uid, int(s.turn_prompt[uid, t]), int(s.turn_output[uid, t]), t, slot)
                    self._seq += 1
                    self.state[slot] = _PARKED
                    self.parked[slot] = (self._seq, e)
                    self.resume_q.append((ready, self._seq, e))
                    self.resume_q.sort(key=lambda x: (x[0], x[1]))
                    continue
                else:
                    self.completed += 1
                self.state[slot] = _FREE
                self.len[slot] = 0
                self.uid[slot] = -1
        # EXTEND
        if b > a:
            ok = status[a:b] == ST_OK
            assert (ok | (status[a:b] == ST_OOM)).all(), "EXTEND may only succeed or run out of memory"
            oks = ext[ok]
            n_fail = int((~ok).sum())
            self.n_oom_extend += n_fail
            oom_seen |= n_fail > 0
            if len(oks):
                progress = True
                for slot in oks.tolist():
                    l = int(self.len[slot])
                    self.writes.append(TokenWrite(slot, int(self.uid[slot]), int(self.slot_epoch[slot]),
                                                  l, l + 1, False))
                self.len[oks] += 1
                self.remaining[oks] -= 1
        # ADMIT
        failed: List[_Entry] = []
        n_ok = 0
        for j, (e, slot) in enumerate(admits):
            st = int(status[b + j])
            if st == ST_OK:
                n_ok += 1
                base = int(self.len[slot]) if e.resume_slot >= 0 else 0
                if e.resume_slot >= 0:
                    self.parked.pop(slot, None)
                ep = self.epoch_of_uid.get(e.uid, -1) + 1
                self.epoch_of_uid[e.uid] = ep
                self.state[slot] = _RUNNING
                self.uid[slot] = e.uid
                self.len[slot] = base + e.prompt
                self.remaining[slot] = e.output
                self.turn[slot] = e.turn
                self.slot_epoch[slot] = ep
                self._seq += 1
                self.admit_seq[slot] = self._seq
                self.writes.append(TokenWrite(slot, e.uid, ep, base, base + e.prompt, True))
            else:
                assert st == ST_OOM, f"admit returned status {st}"
                self.n_oom_admit += 1
                failed.append(e)
        progress |= n_ok > 0
        oom_seen |= bool(failed)
        if failed:
            self.window = 1
        elif n_ok:
            self.window = min(2 * self.window, self.w.concurrency)
        n_running = int((self.state == _RUNNING).sum())
        if failed and not progress and n_running == 0 and not self.parked:
            e = failed.pop(0)            # unservable even with the pool to itself
            self.dropped += 1
        for e in reversed(failed):
            self.front.appendleft(e)
        if (oom_seen or self._starved) and self.parked:
            slot = min(self.parked, key=lambda s: self.parked[s][0])
            self._forced[slot] = "evict"
        elif not progress and n_running > 0 and len(status) > 0:
            run = np.flatnonzero(self.state == _RUNNING)
            self._forced[int(run[np.argmax(self.admit_seq[run])])] = "preempt"
        self.step += 1


def record_trace(w: Workload, step_fn: Callable[[np.ndarray], np.ndarray],
                 max_steps: Optional[int] = None, driver: Optional[ClosedLoopDriver] = None,
                 on_step: Optional[Callable[[ClosedLoopDriver, np.ndarray, np.ndarray], None]] = None):
    """Run the closed loop against `step_fn(ops) -> status`; return [(ops, status), ...]."""
    d = driver if driver is not None else ClosedLoopDriver(w)
    trace = []
    while not d.done and (max_steps is None or d.step < max_steps):
        ops = d.next_batch()
        status = np.asarray(step_fn(ops), dtype=np.uint32) if len(ops) else np.zeros(0, np.uint32)
        d.feed(status)
        trace.append((ops, status))
        if on_step is not None:
            on_step(d, ops, status)
    return trace, d


def random_op_string(seed: int, n: int, max_requests: int, max_tokens: int,
                     p_invalid: float = 0.1) -> np.ndarray:
    """Unscheduled random ops (any order, duplicates, invalid kinds and slots):
    exercises statuses and same-request dependencies inside one batch."""
    kind = rand_int(seed, 21, n, 1, 3)
    req = rand_int(seed, 22, n, 0, max_requests - 1)
    tok = rand_int(seed, 23, n, 1, max_tokens)
    fl = rand_int(seed, 24, n, 0, 3)
    u = rand_unit(seed, 25, n)
    which = rand_int(seed, 26, n, 0, 2)
    inv = u < p_invalid
    kind = np.where(inv & (which == 0), 7, kind)
    req = np.where(inv & (which == 1), max_requests + 3, req)
    tok = np.where(inv & (which == 2), 0, tok)
    ops = np.zeros(n, dtype=OP_DTYPE)
    ops["kind"] = kind
    ops["flags"] = np.where(kind == OP_FINISH, fl & FLAG_KEEP_KV, np.where(kind == OP_ADMIT, fl & FLAG_RESUME, 0))
    ops["req"] = req
    ops["tokens"] = tok
    return ops


def engine_shaped_batch(seed: int, max_requests: int, max_tokens: int, p_pick: float = 0.5,
                        repeats: bool = False) -> np.ndarray:
    """One batch in the order an engine step has -- FINISH ops, then EXTEND ops, then ADMIT ops, slots ascending
    inside each kind -- but with the slots of each kind drawn independently, so the same slot may be finished and
    admitted (or extended) in one batch, finished with KEEP_KV and resumed, or extended and admitted: the cases a
    scheduler never emits and an allocator must still get right.  repeats: some ops appear twice in a row (the
    second one sees what the first one did), which breaks the ascending order by the smallest possible margin."""
    parts = []
    for j, kind in enumerate((OP_FINISH, OP_EXTEND, OP_ADMIT)):
        u = rand_unit(seed, 31 + j, max_requests)
        slots = np.flatnonzero(u < p_pick * (0.6 if kind == OP_FINISH else 1.0))
        n = len(slots)
        tok = rand_int(seed, 41 + j, n, 1, max_tokens) if n else np.zeros(0, np.int64)
        fl = rand_int(seed, 51 + j, n, 0, 3) if n else np.zeros(0, np.int64)
        flags = (fl & FLAG_KEEP_KV) if kind == OP_FINISH else ((fl & FLAG_RESUME) if kind == OP_ADMIT else 0 * fl)
        part = make_ops(kind, slots, tok, flags)
        if repeats and n:
            part = np.repeat(part, np.where(rand_unit(seed, 61 + j, n) < 0.15, 2, 1))
        parts.append(part)
    return np.concatenate(parts)
