// On-device closed loop for multi-turn sessions (the agentic-burst workload): the scheduling that
// turns per-op statuses into the next step's batch when requests park between turns and come back.
// The paper describes that workload in one sentence (Section 4.1) and has no scheduler of its own;
// the policy below is the one of the host-side batch builder the tests run against the oracle:
//   sessions arrive in bursts (arrival step per session, ascending); each step issues FINISH for
//   running requests whose decode is complete (with KEEP_KV when the session has another turn: the
//   slot parks with its KV chain, the SSM blocks go back), EXTEND by one token for the other running
//   requests, then ADMITs, in this order of precedence: re-queued entries, parked sessions whose
//   think time is over (ordered by ready step, then by parking order; ADMIT with RESUME on their own
//   slot), newly arrived sessions -- while running < concurrency and within a slow-start window.
//   Entries that need a fresh slot stop the admission when no slot is free.  A step that saw an OOM,
//   or whose admission stopped for lack of a slot, evicts the longest-parked chain (plain FINISH;
//   that session re-enters with its whole context as the prompt); a step without any success
//   pre-empts the most recently admitted request; an admit that fails with nothing running and
//   nothing parked is dropped.
// A session has at most one pending entry at any time, so entries live in per-session arrays and
// the queues hold session indices only.
#include <cstring>
#include <new>

#include "avmp_step_body.cuh"

using namespace avmp;

namespace {

constexpr uint32_t FREE_ = 0, RUNNING_ = 1, PARKED_ = 2;
constexpr uint32_t WHY_PREEMPT = 1, WHY_EVICT = 2;
constexpr uint32_t NO_SLOT = 0xFFFFFFFFu;

struct SessState {
    uint32_t step, window, seq, n_sessions, max_turns, concurrency, R;
    uint32_t arrived;                 // sessions [0, arrived) have reached their arrival step
    uint32_t back_head;               // sessions [back_head, arrived) still wait for a first admission
    uint32_t front_count, front_buf;  // re-queued session indices, served first
    uint32_t rq_head, rq_tail, rq_buf;  // parked / evicted sessions waiting for their ready step, sorted
    uint32_t completed, dropped, preempted, evicted, n_oom_admit, n_oom_extend;
    uint32_t forced_slot, forced_why;
    uint32_t n_fin, n_ext, n_adm, n_ops;
    uint32_t took_front, took_rq, took_back, break_uid;   // what the batch builder removed from the queues
    uint32_t starved;                 // the batch left an entry without a slot
    uint32_t hi;                      // slots >= hi have never been used: the scans stop there
};

struct Sess {
    SessState *st;
    // the workload: device arrays owned by the caller
    const uint32_t *arrival_step, *n_turns, *turn_prompt, *turn_output, *turn_think;
    // pending entry of every session
    uint32_t *e_prompt, *e_output, *e_turn, *e_slot;
    // request slots
    uint32_t *slot_state, *slot_uid, *slot_len, *slot_rem, *slot_turn, *slot_seq, *slot_pseq;
    // queues
    uint32_t *front[2];
    unsigned long long *rq_key[2];    // ready step << 32 | parking number
    uint32_t *rq_uid[2];
    // per-step lists
    uint32_t *fin_slots, *fin_flags, *ext_slots, *free_slots, *adm_uid, *adm_slot, *adm_res;
    unsigned long long *new_key;
    uint32_t *new_uid;
    avmp_op *ops;
    uint32_t *status, *n_ops_word;
};

struct SessShared {
    unsigned long long tmp[32];
    uint32_t tmp32[32];
    SessState st;
    uint32_t s_completed, s_evicted, s_ext_ok, s_ext_oom, s_has_pre, s_pre_uid, s_n_parked, s_hi;
    unsigned long long s_oldest_parked, s_newest_running;
};

__device__ __forceinline__ void put_op(avmp_op *o, uint32_t kind, uint32_t flags, uint32_t req, uint32_t tokens)
{
    uint32_t *w = reinterpret_cast<uint32_t *>(o);
    w[0] = kind | (flags << 8); w[1] = req; w[2] = tokens;
}

__global__ void __launch_bounds__(kStepThreads, 1) sess_init_kernel(const Sess d, const SessState init)
{
    pdl_prologue();
    if (threadIdx.x == 0) { *d.st = init; *d.n_ops_word = 0; }
    for (uint32_t s = threadIdx.x; s < init.R; s += blockDim.x) {
        d.slot_state[s] = FREE_; d.slot_uid[s] = kInvalid; d.slot_len[s] = 0; d.slot_rem[s] = 0;
        d.slot_turn[s] = 0; d.slot_seq[s] = 0; d.slot_pseq[s] = 0;
    }
    for (uint32_t i = threadIdx.x; i < init.n_sessions; i += blockDim.x) {
        d.e_prompt[i] = 0; d.e_output[i] = 0; d.e_turn[i] = 0; d.e_slot[i] = NO_SLOT;
    }
}

// Build the next batch (whole CTA; blockDim.x >= concurrency).
__device__ void sess_build_body(const Sess &d, SessShared &sm)
{
    unsigned long long *tmp = sm.tmp;
    SessState &st = sm.st;
    const uint32_t tid = threadIdx.x, NT = blockDim.x;
    if (tid == 0) st = *d.st;
    __syncthreads();
    const uint32_t R = st.R, MT = st.max_turns, step = st.step;
    unsigned long long tot;

    // arrivals: sessions whose arrival step has come join the arrival queue with their first turn
    uint32_t arrived = st.arrived;
    for (;;) {
        const uint32_t i = arrived + tid;
        const uint32_t here = (i < st.n_sessions && d.arrival_step[i] <= step) ? 1u : 0u;
        if (here) { d.e_prompt[i] = d.turn_prompt[(size_t)i * MT]; d.e_output[i] = d.turn_output[(size_t)i * MT]; d.e_turn[i] = 0; d.e_slot[i] = NO_SLOT; }
        block_incl_scan(here, tmp, &tot);
        arrived += (uint32_t)tot;
        if (tot < NT) break;
    }
    // an evicted chain goes away now: its session will come back as a fresh admission of everything
    const uint32_t forced = st.forced_slot;
    if (tid == 0 && forced != NO_SLOT && st.forced_why == WHY_EVICT) {
        const uint32_t u = d.slot_uid[forced];
        d.e_prompt[u] += d.slot_len[forced];
        d.e_slot[u] = NO_SLOT;
    }
    __syncthreads();

    // FINISH, EXTEND and free slots, ascending (three counters packed 21 bits each)
    unsigned long long run = 0;
    const uint32_t hi = st.hi;                 // <= R; every slot at or above it is free
    for (uint32_t b = 0; b < hi; b += NT) {
        const uint32_t s = b + tid;
        uint32_t fin = 0, ext = 0, fre = 0, flags = 0;
        if (s < hi) {
            const uint32_t state = d.slot_state[s];
            if (s == forced) fin = 1;
            else if (state == RUNNING_) {
                fin = d.slot_rem[s] == 0 ? 1u : 0u; ext = 1u - fin;
                // (a turn count beyond max_turns is cut there: the per-turn arrays have max_turns columns)
                if (fin && d.slot_turn[s] + 1u < min(d.n_turns[d.slot_uid[s]], MT)) flags = AVMP_FLAG_KEEP_KV;
            } else if (state == FREE_) fre = 1;
        }
        const unsigned long long v = (unsigned long long)fin | ((unsigned long long)ext << 21) | ((unsigned long long)fre << 42);
        const unsigned long long ex = run + block_incl_scan(v, tmp, &tot) - v;
        if (fin) { const uint32_t k = (uint32_t)(ex & 0x1FFFFFu); d.fin_slots[k] = s; d.fin_flags[k] = flags; }
        if (ext) d.ext_slots[(uint32_t)((ex >> 21) & 0x1FFFFFu)] = s;
        if (fre) d.free_slots[(uint32_t)((ex >> 42) & 0x1FFFFFu)] = s;
        run += tot;
    }
    __syncthreads();
    const uint32_t n_fin = (uint32_t)(run & 0x1FFFFFu), n_ext = (uint32_t)((run >> 21) & 0x1FFFFFu);
    const uint32_t n_free_lo = (uint32_t)((run >> 42) & 0x1FFFFFu);   // free slots below hi, listed
    const uint32_t n_free = n_free_lo + (R - hi);                      // plus the untouched ones above
    uint32_t budget = st.concurrency > n_ext ? st.concurrency - n_ext : 0u;
    budget = min(budget, st.window);            // <= concurrency <= NT: one candidate per thread

    // candidates in order of precedence: re-queued, ready to resume, newly arrived
    const uint32_t fc = st.front_count, fb = st.front_buf, rb = st.rq_buf;
    const uint32_t rq_n = st.rq_tail - st.rq_head, nb = arrived - st.back_head;
    const uint32_t ready = (tid < budget && tid < rq_n && (uint32_t)(d.rq_key[rb][st.rq_head + tid] >> 32) <= step) ? 1u : 0u;
    block_incl_scan(ready, tmp, &tot);          // the queue is sorted by ready step: the ready ones lead
    const uint32_t kr = (uint32_t)tot;
    const uint32_t n_cand = min(budget, fc + kr + nb);
    uint32_t uid = kInvalid, needs_free = 0;
    if (tid < n_cand) {
        if (tid < fc) uid = d.front[fb][tid];
        else if (tid < fc + kr) uid = d.rq_uid[rb][st.rq_head + (tid - fc)];
        else uid = st.back_head + (tid - fc - kr);
        needs_free = d.e_slot[uid] == NO_SLOT ? 1u : 0u;
    }
    const uint32_t rank = (uint32_t)(block_incl_scan(needs_free, tmp, &tot) - needs_free);
    const uint32_t blocked = (needs_free && rank >= n_free) ? tid : 0xFFFFFFFFu;
    const uint32_t first_blocked = block_min(blocked, sm.tmp32);
    const uint32_t n_adm = min(n_cand, first_blocked);

    for (uint32_t j = tid; j < n_fin; j += NT) put_op(d.ops + j, AVMP_OP_FINISH, d.fin_flags[j], d.fin_slots[j], 0);
    for (uint32_t j = tid; j < n_ext; j += NT) put_op(d.ops + n_fin + j, AVMP_OP_EXTEND, 0, d.ext_slots[j], 1);
    if (tid < n_adm) {
        const uint32_t own = d.e_slot[uid];
        const uint32_t slot = needs_free ? (rank < n_free_lo ? d.free_slots[rank] : hi + (rank - n_free_lo)) : own;
        put_op(d.ops + n_fin + n_ext + tid, AVMP_OP_ADMIT, needs_free ? 0u : (uint32_t)AVMP_FLAG_RESUME, slot, d.e_prompt[uid]);
        d.adm_uid[tid] = uid; d.adm_slot[tid] = slot; d.adm_res[tid] = 1u - needs_free;
    }
    // the entry that found no free slot was taken from its queue and goes to the head of the re-queued ones
    if (tid == n_adm && n_adm < n_cand) d.st->break_uid = tid < fc ? kInvalid : uid;
    if (tid == 0) {
        SessState *o = d.st;
        if (!(n_adm < n_cand)) o->break_uid = kInvalid;
        const uint32_t popped = n_adm + ((n_adm < n_cand && n_adm >= fc) ? 1u : 0u);   // entries removed behind the re-queued ones included
        const uint32_t tf = min(n_adm, fc);
        const uint32_t tr = min(popped - min(popped, fc), kr);
        o->took_front = tf; o->took_rq = tr; o->took_back = popped - min(popped, fc) - tr;
        o->arrived = arrived;
        o->starved = n_adm < n_cand ? 1u : 0u;
        o->n_fin = n_fin; o->n_ext = n_ext; o->n_adm = n_adm; o->n_ops = n_fin + n_ext + n_adm;
        *d.n_ops_word = n_fin + n_ext + n_adm;
    }
    __syncthreads();
}

// Fold the statuses of the batch back into the slots and the queues (whole CTA).
__device__ void sess_feed_body(const Sess &d, SessShared &sm)
{
    unsigned long long *tmp = sm.tmp;
    SessState &st = sm.st;
    const uint32_t tid = threadIdx.x, NT = blockDim.x;
    if (tid == 0) {
        st = *d.st;
        sm.s_completed = sm.s_evicted = sm.s_ext_ok = sm.s_ext_oom = sm.s_has_pre = sm.s_n_parked = 0;
        sm.s_pre_uid = kInvalid;
        sm.s_hi = st.hi;
        sm.s_oldest_parked = ~0ull; sm.s_newest_running = 0ull;
    }
    __syncthreads();
    const uint32_t n_fin = st.n_fin, n_ext = st.n_ext, n_adm = st.n_adm, MT = st.max_turns, step = st.step;
    unsigned long long tot;

    // FINISH (never fails): completed, parked for the next turn, pre-empted or evicted
    uint32_t n_park = 0;
    for (uint32_t b = 0; b < n_fin; b += NT) {
        const uint32_t j = b + tid;
        uint32_t s = 0, park = 0;
        if (j < n_fin) { s = d.fin_slots[j]; park = (s != st.forced_slot && (d.fin_flags[j] & AVMP_FLAG_KEEP_KV)) ? 1u : 0u; }
        const uint32_t k = n_park + (uint32_t)(block_incl_scan(park, tmp, &tot) - park);
        if (j < n_fin) {
            const uint32_t u = d.slot_uid[s];
            if (park) {
                const uint32_t t = d.slot_turn[s] + 1u, pseq = st.seq + k + 1u;
                const uint32_t rdy = step + 1u + d.turn_think[(size_t)u * MT + t - 1u];
                d.e_prompt[u] = d.turn_prompt[(size_t)u * MT + t]; d.e_output[u] = d.turn_output[(size_t)u * MT + t];
                d.e_turn[u] = t; d.e_slot[u] = s;
                d.slot_state[s] = PARKED_; d.slot_pseq[s] = pseq;
                d.new_key[k] = ((unsigned long long)rdy << 32) | pseq; d.new_uid[k] = u;
            } else {
                if (s == st.forced_slot && st.forced_why == WHY_PREEMPT) {
                    d.e_prompt[u] = d.slot_len[s]; d.e_output[u] = d.slot_rem[s]; d.e_turn[u] = d.slot_turn[s]; d.e_slot[u] = NO_SLOT;
                    sm.s_has_pre = 1; sm.s_pre_uid = u;
                } else if (s == st.forced_slot) atomicAdd(&sm.s_evicted, 1u);
                else atomicAdd(&sm.s_completed, 1u);
                d.slot_state[s] = FREE_; d.slot_len[s] = 0; d.slot_uid[s] = kInvalid;
            }
        }
        n_park += (uint32_t)tot;
    }
    // EXTEND: one more token, or a stall
    for (uint32_t j = tid; j < n_ext; j += NT) {
        const uint32_t s = d.ext_slots[j];
        if (d.status[n_fin + j] == AVMP_ST_OK) { d.slot_len[s] += 1; d.slot_rem[s] -= 1; atomicAdd(&sm.s_ext_ok, 1u); }
        else atomicAdd(&sm.s_ext_oom, 1u);
    }
    __syncthreads();
    // ADMIT, in order (n_adm <= NT): successes take consecutive admission numbers behind the parking
    // numbers of this step, failures return to the queue head in order
    const uint32_t nf = 1u - st.front_buf;
    uint32_t ok = 0, fail = 0;
    if (tid < n_adm) { ok = d.status[n_fin + n_ext + tid] == AVMP_ST_OK ? 1u : 0u; fail = 1u - ok; }
    const unsigned long long v = (unsigned long long)ok | ((unsigned long long)fail << 32);
    const unsigned long long ex = block_incl_scan(v, tmp, &tot) - v;
    const uint32_t n_ok = (uint32_t)tot, n_fail = (uint32_t)(tot >> 32);
    if (ok) {
        const uint32_t s = d.adm_slot[tid], u = d.adm_uid[tid];
        const uint32_t base = d.adm_res[tid] ? d.slot_len[s] : 0u;
        d.slot_state[s] = RUNNING_; d.slot_uid[s] = u; d.slot_len[s] = base + d.e_prompt[u];
        d.slot_rem[s] = d.e_output[u]; d.slot_turn[s] = d.e_turn[u];
        d.slot_seq[s] = st.seq + n_park + (uint32_t)ex + 1u;
        atomicMax(&sm.s_hi, s + 1u);
    }
    __syncthreads();
    const uint32_t new_hi = sm.s_hi;
    // who is parked, who runs: the longest-parked chain and the most recently admitted request
    {
        unsigned long long oldest = ~0ull, newest = 0ull;
        uint32_t cnt = 0;
        for (uint32_t s = tid; s < new_hi; s += NT) {
            const uint32_t state = d.slot_state[s];
            if (state == PARKED_) { cnt += 1; oldest = min(oldest, ((unsigned long long)d.slot_pseq[s] << 32) | s); }
            else if (state == RUNNING_) newest = max(newest, ((unsigned long long)d.slot_seq[s] << 32) | s);
        }
        if (cnt) { atomicAdd(&sm.s_n_parked, cnt); atomicMin(&sm.s_oldest_parked, oldest); }
        if (newest) atomicMax(&sm.s_newest_running, newest);
    }
    __syncthreads();
    const bool progress = n_fin > 0 || sm.s_ext_ok > 0 || n_ok > 0;
    const bool oom_seen = sm.s_ext_oom > 0 || n_fail > 0;
    const uint32_t n_running = n_ext + n_ok, n_parked = sm.s_n_parked;
    const uint32_t drop = (n_fail > 0 && !progress && n_running == 0 && n_parked == 0) ? 1u : 0u;
    // new queue head = failed admits (minus a dropped one), the pre-empted request, the entry that
    // found no free slot, then what the batch builder left
    const uint32_t has_pre = sm.s_has_pre, has_brk = st.break_uid != kInvalid ? 1u : 0u;
    const uint32_t keep_fail = n_fail - drop, rest = st.front_count - st.took_front;
    if (fail) {
        const uint32_t pos = (uint32_t)(ex >> 32);
        if (pos >= drop) d.front[nf][pos - drop] = d.adm_uid[tid];
    }
    if (tid == 0) {
        if (has_pre) d.front[nf][keep_fail] = sm.s_pre_uid;
        if (has_brk) d.front[nf][keep_fail + has_pre] = st.break_uid;
    }
    for (uint32_t j = tid; j < rest; j += NT) d.front[nf][keep_fail + has_pre + has_brk + j] = d.front[st.front_buf][st.took_front + j];

    // the waiting queue: the builder took its first took_rq entries; this step's parked sessions are
    // merged in by (ready step, parking number)
    const uint32_t rb = st.rq_buf, head = st.rq_head + st.took_rq, n_old = st.rq_tail - head;
    uint32_t new_head = head, new_tail = st.rq_tail, new_buf = rb;
    if (n_park) {
        const uint32_t ob = 1u - rb;
        for (uint32_t i = tid; i < n_old; i += NT) {
            const unsigned long long key = d.rq_key[rb][head + i];
            uint32_t shift = 0;
            for (uint32_t k = 0; k < n_park; ++k) shift += d.new_key[k] < key ? 1u : 0u;
            d.rq_key[ob][i + shift] = key; d.rq_uid[ob][i + shift] = d.rq_uid[rb][head + i];
        }
        for (uint32_t k = tid; k < n_park; k += NT) {
            const unsigned long long key = d.new_key[k];
            uint32_t lo = 0, hi = n_old;                         // old entries below this key
            while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (d.rq_key[rb][head + mid] < key) lo = mid + 1; else hi = mid; }
            uint32_t below = lo;
            for (uint32_t q = 0; q < n_park; ++q) below += d.new_key[q] < key ? 1u : 0u;
            d.rq_key[ob][below] = key; d.rq_uid[ob][below] = d.new_uid[k];
        }
        new_head = 0; new_tail = n_old + n_park; new_buf = ob;
    }
    __syncthreads();
    if (tid == 0) {
        SessState n = st;
        n.step = step + 1;
        n.seq = st.seq + n_park + n_ok;
        n.back_head = st.back_head + st.took_back;
        n.completed = st.completed + sm.s_completed;
        n.evicted = st.evicted + sm.s_evicted;
        n.preempted = st.preempted + has_pre;
        n.dropped = st.dropped + drop;
        n.n_oom_admit = st.n_oom_admit + n_fail;
        n.n_oom_extend = st.n_oom_extend + sm.s_ext_oom;
        if (n_fail) n.window = 1;
        else if (n_ok) n.window = min(2u * st.window, st.concurrency);
        n.front_count = keep_fail + has_pre + has_brk + rest;
        n.front_buf = nf;
        n.rq_head = new_head; n.rq_tail = new_tail; n.rq_buf = new_buf;
        n.forced_slot = NO_SLOT; n.forced_why = 0;
        if ((oom_seen || st.starved) && n_parked > 0) { n.forced_slot = (uint32_t)(sm.s_oldest_parked & 0xFFFFFFFFull); n.forced_why = WHY_EVICT; }
        else if (!progress && n_running > 0 && st.n_ops > 0) { n.forced_slot = (uint32_t)(sm.s_newest_running & 0xFFFFFFFFull); n.forced_why = WHY_PREEMPT; }
        n.break_uid = kInvalid; n.starved = 0;
        n.hi = new_hi;
        *d.st = n;
    }
}

__global__ void __launch_bounds__(kStepThreads, 1) sess_build_kernel(const Sess d)
{
    __shared__ SessShared sm;
    pdl_prologue();
    sess_build_body(d, sm);
}

__global__ void __launch_bounds__(kStepThreads, 1) sess_feed_kernel(const Sess d)
{
    __shared__ SessShared sm;
    pdl_prologue();
    sess_feed_body(d, sm);
}

// One engine step in one launch: build, allocator update, fold back.  Usable when the batch can hold
// at most one migration (a second one needs the first one's relocation copy, a separate wide kernel).
template <int NT>
__global__ void __launch_bounds__(NT, 1) sess_fused_kernel(const Sess d, const Geom g)
{
    __shared__ SessShared sm;
    __shared__ stepimpl::Shared<NT> sh;
    pdl_prologue();
    sess_build_body(d, sm);
    const uint32_t n_ops = *d.n_ops_word;
    stepimpl::step_body<NT>(g, sh, d.ops, n_ops, d.status, 1);
    __syncthreads();
    sess_feed_body(d, sm);
}

constexpr size_t kAlign = 256;
inline size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
struct SessLayout { size_t st, entry[4], slot[7], front[2], rq_key[2], rq_uid[2], lists[7], new_key, new_uid, ops, status, n_ops, total; };
SessLayout sess_layout(uint32_t R, uint32_t n_sessions)
{
    SessLayout l;
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += up(b); return o; };
    l.st = take(sizeof(SessState));
    for (auto &x : l.entry) x = take((size_t)n_sessions * 4);
    for (auto &x : l.slot) x = take((size_t)R * 4);
    for (auto &x : l.front) x = take((size_t)n_sessions * 4);
    for (auto &x : l.rq_key) x = take((size_t)n_sessions * 8);
    for (auto &x : l.rq_uid) x = take((size_t)n_sessions * 4);
    for (auto &x : l.lists) x = take((size_t)(R + 8) * 4);
    l.new_key = take((size_t)(R + 8) * 8);
    l.new_uid = take((size_t)(R + 8) * 4);
    l.ops = take((size_t)(2 * R + 8) * sizeof(avmp_op));
    l.status = take((size_t)(2 * R + 8) * 4);
    l.n_ops = take(4);
    l.total = off;
    return l;
}
inline cudaStream_t S(void *s) { return reinterpret_cast<cudaStream_t>(s); }

}  // namespace

struct avmp_session_driver {
    Sess d;
    avmp_ctx *ctx;
    uint32_t R, n_sessions, max_ops, concurrency;
};

extern "C" {

AVMP_API size_t avmp_session_driver_workspace_bytes(uint32_t max_requests, uint32_t n_sessions)
{
    if (max_requests == 0 || max_requests >= (1u << 20) || n_sessions == 0 || n_sessions >= (1u << 28)) return 0;
    return sess_layout(max_requests, n_sessions).total;
}

AVMP_API int avmp_session_driver_create(avmp_session_driver **out, avmp_ctx *ctx, const uint32_t *d_arrival_step,
                                        const uint32_t *d_n_turns, const uint32_t *d_turn_prompt,
                                        const uint32_t *d_turn_output, const uint32_t *d_turn_think,
                                        uint32_t n_sessions, uint32_t max_turns, uint32_t concurrency,
                                        void *d_workspace, size_t workspace_bytes, void *stream)
{
    if (!out || !ctx || !d_arrival_step || !d_n_turns || !d_turn_prompt || !d_turn_output || !d_turn_think || !d_workspace)
        return AVMP_EINVAL;
    const uint32_t R = ctx->opt.max_requests;
    if (n_sessions == 0 || n_sessions >= (1u << 28) || max_turns == 0 || R >= (1u << 20)) return AVMP_EINVAL;
    // one admission candidate per thread of the planning block
    if (concurrency == 0 || concurrency > R || concurrency > (uint32_t)kStepThreads) return AVMP_EINVAL;
    if ((uintptr_t)d_workspace & (kAlign - 1)) return AVMP_EINVAL;
    const SessLayout l = sess_layout(R, n_sessions);
    if (workspace_bytes < l.total) return AVMP_ENOSPC;
    avmp_session_driver *dr = new (std::nothrow) avmp_session_driver();
    if (!dr) return AVMP_EINVAL;
    uint8_t *b = static_cast<uint8_t *>(d_workspace);
    auto u32 = [&](size_t o) { return reinterpret_cast<uint32_t *>(b + o); };
    auto u64 = [&](size_t o) { return reinterpret_cast<unsigned long long *>(b + o); };
    Sess &d = dr->d;
    d.st = reinterpret_cast<SessState *>(b + l.st);
    d.arrival_step = d_arrival_step; d.n_turns = d_n_turns; d.turn_prompt = d_turn_prompt;
    d.turn_output = d_turn_output; d.turn_think = d_turn_think;
    d.e_prompt = u32(l.entry[0]); d.e_output = u32(l.entry[1]); d.e_turn = u32(l.entry[2]); d.e_slot = u32(l.entry[3]);
    d.slot_state = u32(l.slot[0]); d.slot_uid = u32(l.slot[1]); d.slot_len = u32(l.slot[2]); d.slot_rem = u32(l.slot[3]);
    d.slot_turn = u32(l.slot[4]); d.slot_seq = u32(l.slot[5]); d.slot_pseq = u32(l.slot[6]);
    for (int k = 0; k < 2; ++k) { d.front[k] = u32(l.front[k]); d.rq_key[k] = u64(l.rq_key[k]); d.rq_uid[k] = u32(l.rq_uid[k]); }
    d.fin_slots = u32(l.lists[0]); d.fin_flags = u32(l.lists[1]); d.ext_slots = u32(l.lists[2]); d.free_slots = u32(l.lists[3]);
    d.adm_uid = u32(l.lists[4]); d.adm_slot = u32(l.lists[5]); d.adm_res = u32(l.lists[6]);
    d.new_key = u64(l.new_key); d.new_uid = u32(l.new_uid);
    d.ops = reinterpret_cast<avmp_op *>(b + l.ops);
    d.status = u32(l.status); d.n_ops_word = u32(l.n_ops);
    dr->ctx = ctx; dr->R = R; dr->n_sessions = n_sessions; dr->concurrency = concurrency;
    // at most `concurrency` requests run, one more slot may be evicted, at most `concurrency` are admitted
    dr->max_ops = 2 * concurrency + 1 < 2 * R ? 2 * concurrency + 1 : 2 * R;
    SessState init;
    memset(&init, 0, sizeof(init));
    init.window = concurrency; init.n_sessions = n_sessions; init.max_turns = max_turns; init.concurrency = concurrency;
    init.R = R; init.forced_slot = NO_SLOT; init.break_uid = kInvalid;
    if (launch_pdl(sess_init_kernel, dim3(1), dim3(kStepThreads), 0, S(stream), d, init) != cudaSuccess) { delete dr; return AVMP_ECUDA; }
    ctx->launches += 1;
    *out = dr;
    return AVMP_OK;
}

AVMP_API int avmp_session_driver_destroy(avmp_session_driver *dr)
{
    delete dr;
    return AVMP_OK;
}

AVMP_API int avmp_session_driver_step(avmp_session_driver *dr, void *stream)
{
    if (!dr) return AVMP_EINVAL;
    avmp_ctx *c = dr->ctx;
    const bool mig = c->opt.migration_enabled != 0;
    const uint64_t rounds = mig ? (uint64_t)(dr->max_ops - 1) / c->opt.min_rebalance_interval_ops + 1 : 1;
    if (rounds == 1) {
        // the planning block needs a thread per admission candidate and per op of a window
        const uint32_t need = dr->max_ops > dr->concurrency ? dr->max_ops : dr->concurrency;
        cudaError_t e;
        if (need <= 256) e = launch_pdl(sess_fused_kernel<256>, dim3(1), dim3(256), 0, S(stream), dr->d, c->g);
        else if (need <= 512) e = launch_pdl(sess_fused_kernel<512>, dim3(1), dim3(512), 0, S(stream), dr->d, c->g);
        else e = launch_pdl(sess_fused_kernel<1024>, dim3(1), dim3(1024), 0, S(stream), dr->d, c->g);
        if (e != cudaSuccess) return AVMP_ECUDA;
        c->launches += 1;
        if (mig) {
            if (launch_relocate(c->g, Launch{S(stream), c->n_sms, c->device}) != cudaSuccess) return AVMP_ECUDA;
            c->launches += 1;
        }
        return AVMP_OK;
    }
    if (launch_pdl(sess_build_kernel, dim3(1), dim3(kStepThreads), 0, S(stream), dr->d) != cudaSuccess) return AVMP_ECUDA;
    const int rc = avmp_step_indirect(c, dr->d.ops, dr->d.n_ops_word, dr->max_ops, dr->d.status, stream);
    if (rc != AVMP_OK) return rc;
    if (launch_pdl(sess_feed_kernel, dim3(1), dim3(kStepThreads), 0, S(stream), dr->d) != cudaSuccess) return AVMP_ECUDA;
    c->launches += 2;
    return AVMP_OK;
}

AVMP_API int avmp_session_driver_get_stats(avmp_session_driver *dr, avmp_session_stats *h, void *stream)
{
    if (!dr || !h) return AVMP_EINVAL;
    SessState s;
    if (cudaMemcpyAsync(&s, dr->d.st, sizeof(s), cudaMemcpyDeviceToHost, S(stream)) != cudaSuccess) return AVMP_ECUDA;
    if (cudaStreamSynchronize(S(stream)) != cudaSuccess) return AVMP_ECUDA;
    h->steps = s.step; h->completed = s.completed; h->dropped = s.dropped; h->preempted = s.preempted;
    h->evicted = s.evicted; h->n_oom_admit = s.n_oom_admit; h->n_oom_extend = s.n_oom_extend;
    h->arrived = s.arrived; h->arrival_queue = s.arrived - s.back_head; h->requeued = s.front_count;
    h->waiting = s.rq_tail - s.rq_head; h->window = s.window; h->last_batch_ops = s.n_ops;
    h->forced_slot = s.forced_slot == NO_SLOT ? ~0ull : s.forced_slot;
    return AVMP_OK;
}

AVMP_API int avmp_session_driver_export(avmp_session_driver *dr, uint32_t *h_state, uint32_t *h_uid, uint32_t *h_len,
                                        uint32_t *h_remaining, uint32_t *h_turn, uint32_t *h_requeued,
                                        uint32_t *h_waiting, void *stream)
{
    if (!dr || !h_state || !h_uid || !h_len || !h_remaining || !h_turn || !h_requeued || !h_waiting) return AVMP_EINVAL;
    cudaStream_t s = S(stream);
    SessState st;
    if (cudaMemcpyAsync(&st, dr->d.st, sizeof(st), cudaMemcpyDeviceToHost, s) != cudaSuccess) return AVMP_ECUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return AVMP_ECUDA;
    const size_t n = (size_t)dr->R * 4;
    bool ok = cudaMemcpyAsync(h_state, dr->d.slot_state, n, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h_uid, dr->d.slot_uid, n, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h_len, dr->d.slot_len, n, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h_remaining, dr->d.slot_rem, n, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h_turn, dr->d.slot_turn, n, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    if (ok && st.front_count)
        ok = cudaMemcpyAsync(h_requeued, dr->d.front[st.front_buf], (size_t)st.front_count * 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    if (ok && st.rq_tail > st.rq_head)
        ok = cudaMemcpyAsync(h_waiting, dr->d.rq_uid[st.rq_buf] + st.rq_head, (size_t)(st.rq_tail - st.rq_head) * 4,
                             cudaMemcpyDeviceToHost, s) == cudaSuccess;
    if (!ok || cudaStreamSynchronize(s) != cudaSuccess) return AVMP_ECUDA;
    return AVMP_OK;
}

}  // extern "C"
