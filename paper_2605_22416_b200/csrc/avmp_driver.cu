// On-device closed loop: the engine-side scheduling that turns per-op statuses into the next
// step's batch, as two single-CTA kernels around avmp_step, so that a serving loop runs step
// after step with no host round trip (the paper's harness replays its synthetic traces from the
// host, Section 4.1; its per-call retry loop is what its time decomposition of Section 4.3
// measures).  Policy, identical to the host-side batch builder used by the tests:
//   FINISH for running requests whose decode is complete (ascending slot), EXTEND by one token
//   for every other running request (ascending slot), ADMITs from the queue head into the lowest
//   slots that were free when the step began while running < concurrency and within a slow-start
//   window (any failed admit -> 1; all admits fine -> doubled); failed admits return to the queue
//   head in order; a step without any success pre-empts the most recently admitted request; an
//   admit that fails with nothing running is dropped.
#include <cstring>
#include <new>

#include "avmp_step_body.cuh"

using namespace avmp;

namespace {

constexpr uint32_t FREE_ = 0, RUNNING_ = 1;

struct DrvState {
    uint32_t step, window, seq, next, n_requests, concurrency, R, front_cap;
    uint32_t completed, dropped, preempted, n_oom_admit, n_oom_extend, overflow;
    int32_t forced_slot;
    uint32_t front_count, front_buf;
    uint32_t n_fin, n_ext, n_adm, n_ops, front_taken;
};

struct Drv {
    DrvState *st;
    uint32_t *slot_state, *slot_uid, *slot_len, *slot_rem, *slot_seq;
    uint32_t *front_uid[2], *front_prompt[2], *front_output[2];
    uint32_t *fin_slots, *ext_slots, *free_slots, *adm_slot, *adm_uid, *adm_prompt, *adm_output;
    const uint32_t *prompt, *output;
    avmp_op *ops;
    uint32_t *status, *n_ops_word;
};

__device__ __forceinline__ void put_op(avmp_op *o, uint32_t kind, uint32_t req, uint32_t tokens)
{
    uint32_t *w = reinterpret_cast<uint32_t *>(o);
    w[0] = kind; w[1] = req; w[2] = tokens;
}

__global__ void __launch_bounds__(kStepThreads, 1) drv_init_kernel(const Drv d, const DrvState init)
{
    pdl_prologue();
    if (threadIdx.x == 0) { *d.st = init; *d.n_ops_word = 0; }
    for (uint32_t s = threadIdx.x; s < init.R; s += blockDim.x) {
        d.slot_state[s] = FREE_; d.slot_uid[s] = kInvalid; d.slot_len[s] = 0; d.slot_rem[s] = 0; d.slot_seq[s] = 0;
    }
}

// Shared memory of the two scheduler passes.
struct DrvShared {
    unsigned long long tmp[32];
    DrvState st;
    uint32_t s_completed, s_ext_ok, s_ext_oom, s_pre_uid, s_pre_len, s_pre_rem, s_has_pre;
    unsigned long long s_best;
};

// Build the next batch (whole CTA; any block size).
__device__ void drv_build_body(const Drv &d, DrvShared &sm)
{
    unsigned long long *tmp = sm.tmp;
    DrvState &st = sm.st;
    const int tid = threadIdx.x;
    const uint32_t NT = blockDim.x;
    if (tid == 0) st = *d.st;
    __syncthreads();
    const uint32_t R = st.R;
    const int32_t forced = st.forced_slot;
    // compact FINISH, EXTEND and free slots, ascending (three counters packed 21 bits each)
    unsigned long long run = 0, tot;
    for (uint32_t b = 0; b < R; b += NT) {
        const uint32_t s = b + tid;
        uint32_t fin = 0, ext = 0, fre = 0;
        if (s < R) {
            const uint32_t state = d.slot_state[s];
            if (state == RUNNING_) { fin = (d.slot_rem[s] == 0 || (int32_t)s == forced) ? 1u : 0u; ext = 1u - fin; }
            else fre = 1u;
        }
        const unsigned long long v = (unsigned long long)fin | ((unsigned long long)ext << 21) | ((unsigned long long)fre << 42);
        const unsigned long long ex = run + block_incl_scan(v, tmp, &tot) - v;
        if (fin) d.fin_slots[(uint32_t)(ex & 0x1FFFFFu)] = s;
        if (ext) d.ext_slots[(uint32_t)((ex >> 21) & 0x1FFFFFu)] = s;
        if (fre) d.free_slots[(uint32_t)((ex >> 42) & 0x1FFFFFu)] = s;
        run += tot;
    }
    __syncthreads();
    const uint32_t n_fin = (uint32_t)(run & 0x1FFFFFu), n_ext = (uint32_t)((run >> 21) & 0x1FFFFFu);
    const uint32_t n_free = (uint32_t)((run >> 42) & 0x1FFFFFu);
    uint32_t budget = st.concurrency > n_ext ? st.concurrency - n_ext : 0u;
    budget = min(budget, st.window);
    const uint32_t avail = st.front_count + (st.n_requests - st.next);
    const uint32_t n_adm = min(min(budget, avail), n_free);
    const uint32_t fb = st.front_buf;
    for (uint32_t j = tid; j < n_fin; j += NT) put_op(d.ops + j, AVMP_OP_FINISH, d.fin_slots[j], 0);
    for (uint32_t j = tid; j < n_ext; j += NT) put_op(d.ops + n_fin + j, AVMP_OP_EXTEND, d.ext_slots[j], 1);
    for (uint32_t j = tid; j < n_adm; j += NT) {
        uint32_t uid, p, o;
        if (j < st.front_count) { uid = d.front_uid[fb][j]; p = d.front_prompt[fb][j]; o = d.front_output[fb][j]; }
        else { uid = st.next + (j - st.front_count); p = d.prompt[uid]; o = d.output[uid]; }
        const uint32_t slot = d.free_slots[j];
        put_op(d.ops + n_fin + n_ext + j, AVMP_OP_ADMIT, slot, p);
        d.adm_slot[j] = slot; d.adm_uid[j] = uid; d.adm_prompt[j] = p; d.adm_output[j] = o;
    }
    if (tid == 0) {
        d.st->n_fin = n_fin; d.st->n_ext = n_ext; d.st->n_adm = n_adm;
        d.st->n_ops = n_fin + n_ext + n_adm;
        d.st->front_taken = min(n_adm, st.front_count);
        *d.n_ops_word = n_fin + n_ext + n_adm;
    }
    __syncthreads();
}

// Fold the statuses of the batch back into the request slots and the queue (whole CTA).
__device__ void drv_feed_body(const Drv &d, DrvShared &sm)
{
    unsigned long long *tmp = sm.tmp;
    DrvState &st = sm.st;
    uint32_t &s_completed = sm.s_completed, &s_ext_ok = sm.s_ext_ok, &s_ext_oom = sm.s_ext_oom;
    uint32_t &s_pre_uid = sm.s_pre_uid, &s_pre_len = sm.s_pre_len, &s_pre_rem = sm.s_pre_rem, &s_has_pre = sm.s_has_pre;
    unsigned long long &s_best = sm.s_best;
    const int tid = threadIdx.x;
    const uint32_t NT = blockDim.x;
    if (tid == 0) {
        st = *d.st;
        s_completed = s_ext_ok = s_ext_oom = s_has_pre = 0;
        s_best = 0;
    }
    __syncthreads();
    const uint32_t n_fin = st.n_fin, n_ext = st.n_ext, n_adm = st.n_adm;
    // FINISH: the slot is free again; a pre-empted request goes back to the head of the queue
    for (uint32_t j = tid; j < n_fin; j += NT) {
        const uint32_t s = d.fin_slots[j];
        if ((int32_t)s == st.forced_slot) {
            s_pre_uid = d.slot_uid[s]; s_pre_len = d.slot_len[s]; s_pre_rem = d.slot_rem[s]; s_has_pre = 1;
        } else atomicAdd(&s_completed, 1u);
        d.slot_state[s] = FREE_; d.slot_len[s] = 0; d.slot_uid[s] = kInvalid;
    }
    // EXTEND: one more token, or a stall
    for (uint32_t j = tid; j < n_ext; j += NT) {
        const uint32_t s = d.ext_slots[j];
        if (d.status[n_fin + j] == AVMP_ST_OK) { d.slot_len[s] += 1; d.slot_rem[s] -= 1; atomicAdd(&s_ext_ok, 1u); }
        else atomicAdd(&s_ext_oom, 1u);
    }
    // ADMIT, in order: successes take consecutive admission numbers, failures return to the queue head
    const uint32_t nb = 1u - st.front_buf;               // the buffer the new queue head is written to
    unsigned long long run = 0, tot;
    for (uint32_t b = 0; b < n_adm; b += NT) {
        const uint32_t j = b + tid;
        uint32_t ok = 0, fail = 0;
        if (j < n_adm) { ok = d.status[n_fin + n_ext + j] == AVMP_ST_OK ? 1u : 0u; fail = 1u - ok; }
        const unsigned long long v = (unsigned long long)ok | ((unsigned long long)fail << 32);
        const unsigned long long ex = run + block_incl_scan(v, tmp, &tot) - v;
        if (ok) {
            const uint32_t s = d.adm_slot[j];
            d.slot_state[s] = RUNNING_; d.slot_uid[s] = d.adm_uid[j]; d.slot_len[s] = d.adm_prompt[j];
            d.slot_rem[s] = d.adm_output[j]; d.slot_seq[s] = st.seq + (uint32_t)ex + 1u;
        } else if (fail) {
            const uint32_t pos = (uint32_t)(ex >> 32);
            if (pos < st.front_cap) {
                d.front_uid[nb][pos] = d.adm_uid[j]; d.front_prompt[nb][pos] = d.adm_prompt[j];
                d.front_output[nb][pos] = d.adm_output[j];
            }
        }
        run += tot;
    }
    __syncthreads();
    const uint32_t n_ok = (uint32_t)run, n_fail = (uint32_t)(run >> 32);
    const bool progress = n_fin > 0 || s_ext_ok > 0 || n_ok > 0;
    const uint32_t n_running = n_ext + n_ok;
    const uint32_t drop = (n_fail > 0 && !progress && n_running == 0) ? 1u : 0u;   // unservable head entry
    // new queue head = failed admits (minus a dropped one), the pre-empted request, then what was left
    const uint32_t has_pre = s_has_pre;
    const uint32_t rest = st.front_count - st.front_taken;
    const uint32_t keep_fail = n_fail - drop;
    const uint32_t new_count = keep_fail + has_pre + rest;
    __syncthreads();
    if (drop)       // shift the failed list down by one (in place, ascending, chunk by chunk)
        for (uint32_t b = 0; b < keep_fail; b += NT) {
            const uint32_t j = b + tid;
            uint32_t u = 0, p = 0, o = 0;
            if (j < keep_fail && j + 1 < st.front_cap) { u = d.front_uid[nb][j + 1]; p = d.front_prompt[nb][j + 1]; o = d.front_output[nb][j + 1]; }
            __syncthreads();
            if (j < keep_fail) { d.front_uid[nb][j] = u; d.front_prompt[nb][j] = p; d.front_output[nb][j] = o; }
            __syncthreads();
        }
    if (tid == 0 && has_pre && keep_fail < st.front_cap) {
        d.front_uid[nb][keep_fail] = s_pre_uid; d.front_prompt[nb][keep_fail] = s_pre_len; d.front_output[nb][keep_fail] = s_pre_rem;
    }
    for (uint32_t j = tid; j < rest; j += NT) {
        const uint32_t dst = keep_fail + has_pre + j, src = st.front_taken + j;
        if (dst < st.front_cap) {
            d.front_uid[nb][dst] = d.front_uid[st.front_buf][src]; d.front_prompt[nb][dst] = d.front_prompt[st.front_buf][src];
            d.front_output[nb][dst] = d.front_output[st.front_buf][src];
        }
    }
    // pre-emption for the next step: the most recently admitted running request
    const bool need_pre = !progress && n_running > 0 && st.n_ops > 0;
    if (need_pre) {
        unsigned long long best = 0;
        for (uint32_t s = tid; s < st.R; s += NT)
            if (d.slot_state[s] == RUNNING_) best = max(best, ((unsigned long long)d.slot_seq[s] << 32) | s);
        atomicMax(&s_best, best);
    }
    __syncthreads();
    if (tid == 0) {
        DrvState n = st;
        n.step = st.step + 1;
        n.seq = st.seq + n_ok;
        n.next = st.next + (n_adm - st.front_taken);
        n.completed = st.completed + s_completed;
        n.preempted = st.preempted + has_pre;
        n.dropped = st.dropped + drop;
        n.n_oom_admit = st.n_oom_admit + n_fail;
        n.n_oom_extend = st.n_oom_extend + s_ext_oom;
        if (n_fail) n.window = 1;
        else if (n_ok) n.window = min(2u * st.window, st.concurrency);
        n.front_count = min(new_count, st.front_cap);
        if (new_count > st.front_cap) n.overflow = 1;
        n.front_buf = nb;
        n.forced_slot = need_pre ? (int32_t)(uint32_t)(s_best & 0xFFFFFFFFull) : -1;
        *d.st = n;
    }
}

__global__ void __launch_bounds__(kStepThreads, 1) drv_build_kernel(const Drv d)
{
    __shared__ DrvShared sm;
    pdl_prologue();
    drv_build_body(d, sm);
}

__global__ void __launch_bounds__(kStepThreads, 1) drv_feed_kernel(const Drv d)
{
    __shared__ DrvShared sm;
    pdl_prologue();
    drv_feed_body(d, sm);
}

// One engine step of the loop in one launch: build the batch, run the allocator over it, fold the
// statuses back.  Usable when the batch can hold at most one migration (a second one would need the
// first one's relocation copy, which is a separate wide kernel, to run in between).
template <int NT>
__global__ void __launch_bounds__(NT, 1) drv_fused_kernel(const Drv d, const Geom g)
{
    __shared__ DrvShared sm;
    __shared__ stepimpl::Shared<NT> sh;
    pdl_prologue();
    drv_build_body(d, sm);
    const uint32_t n_ops = *d.n_ops_word;
    stepimpl::step_body<NT>(g, sh, d.ops, n_ops, d.status, 1);
    __syncthreads();
    drv_feed_body(d, sm);
}

}  // namespace

struct avmp_driver {
    Drv d;
    avmp_ctx *ctx;
    uint32_t R, max_ops;
};

namespace {
constexpr size_t kAlign = 256;
inline size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
struct DrvLayout { size_t st, slot[5], front[6], lists[7], ops, status, n_ops, total; uint32_t front_cap; };
DrvLayout drv_layout(uint32_t R)
{
    DrvLayout l;
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += up(b); return o; };
    l.front_cap = 2 * R + 64;
    l.st = take(sizeof(DrvState));
    for (auto &x : l.slot) x = take((size_t)R * 4);
    for (auto &x : l.front) x = take((size_t)l.front_cap * 4);
    for (auto &x : l.lists) x = take((size_t)R * 4);
    l.ops = take((size_t)(2 * R + 8) * sizeof(avmp_op));
    l.status = take((size_t)(2 * R + 8) * 4);
    l.n_ops = take(4);
    l.total = off;
    return l;
}
inline cudaStream_t S(void *s) { return reinterpret_cast<cudaStream_t>(s); }
}  // namespace

extern "C" {

AVMP_API size_t avmp_driver_workspace_bytes(uint32_t max_requests)
{
    if (max_requests == 0 || max_requests >= (1u << 20)) return 0;
    return drv_layout(max_requests).total;
}

AVMP_API int avmp_driver_create(avmp_driver **out, avmp_ctx *ctx, const uint32_t *d_prompt, const uint32_t *d_output,
                                uint32_t n_requests, uint32_t concurrency, void *d_workspace, size_t workspace_bytes,
                                void *stream)
{
    if (!out || !ctx || !d_prompt || !d_output || !d_workspace || concurrency == 0) return AVMP_EINVAL;
    const uint32_t R = ctx->opt.max_requests;
    if (R >= (1u << 20) || concurrency > R || ((uintptr_t)d_workspace & (kAlign - 1))) return AVMP_EINVAL;
    const DrvLayout l = drv_layout(R);
    if (workspace_bytes < l.total) return AVMP_ENOSPC;
    avmp_driver *dr = new (std::nothrow) avmp_driver();
    if (!dr) return AVMP_EINVAL;
    uint8_t *b = static_cast<uint8_t *>(d_workspace);
    auto u32 = [&](size_t o) { return reinterpret_cast<uint32_t *>(b + o); };
    Drv &d = dr->d;
    d.st = reinterpret_cast<DrvState *>(b + l.st);
    d.slot_state = u32(l.slot[0]); d.slot_uid = u32(l.slot[1]); d.slot_len = u32(l.slot[2]);
    d.slot_rem = u32(l.slot[3]); d.slot_seq = u32(l.slot[4]);
    for (int k = 0; k < 2; ++k) {
        d.front_uid[k] = u32(l.front[3 * k]); d.front_prompt[k] = u32(l.front[3 * k + 1]); d.front_output[k] = u32(l.front[3 * k + 2]);
    }
    d.fin_slots = u32(l.lists[0]); d.ext_slots = u32(l.lists[1]); d.free_slots = u32(l.lists[2]);
    d.adm_slot = u32(l.lists[3]); d.adm_uid = u32(l.lists[4]); d.adm_prompt = u32(l.lists[5]); d.adm_output = u32(l.lists[6]);
    d.prompt = d_prompt; d.output = d_output;
    d.ops = reinterpret_cast<avmp_op *>(b + l.ops);
    d.status = u32(l.status); d.n_ops_word = u32(l.n_ops);
    dr->ctx = ctx; dr->R = R; dr->max_ops = 2 * R;
    DrvState init;
    memset(&init, 0, sizeof(init));
    init.window = concurrency; init.n_requests = n_requests; init.concurrency = concurrency; init.R = R;
    init.front_cap = l.front_cap; init.forced_slot = -1;
    if (launch_pdl(drv_init_kernel, dim3(1), dim3(kStepThreads), 0, S(stream), d, init) != cudaSuccess) { delete dr; return AVMP_ECUDA; }
    ctx->launches += 1;
    *out = dr;
    return AVMP_OK;
}

AVMP_API int avmp_driver_destroy(avmp_driver *dr)
{
    delete dr;
    return AVMP_OK;
}

AVMP_API int avmp_driver_step(avmp_driver *dr, void *stream)
{
    if (!dr) return AVMP_EINVAL;
    avmp_ctx *c = dr->ctx;
    const bool mig = c->opt.migration_enabled != 0;
    const uint64_t rounds = mig ? (uint64_t)(dr->max_ops - 1) / c->opt.min_rebalance_interval_ops + 1 : 1;
    if (rounds == 1) {
        // at most one migration fits in a batch: the whole step is one launch (plus the copy)
        cudaError_t e;
        if (dr->max_ops <= 256) e = launch_pdl(drv_fused_kernel<256>, dim3(1), dim3(256), 0, S(stream), dr->d, c->g);
        else if (dr->max_ops <= 512) e = launch_pdl(drv_fused_kernel<512>, dim3(1), dim3(512), 0, S(stream), dr->d, c->g);
        else e = launch_pdl(drv_fused_kernel<1024>, dim3(1), dim3(1024), 0, S(stream), dr->d, c->g);
        if (e != cudaSuccess) return AVMP_ECUDA;
        c->launches += 1;
        if (mig) {
            if (launch_relocate(c->g, Launch{S(stream), c->n_sms, c->device}) != cudaSuccess) return AVMP_ECUDA;
            c->launches += 1;
        }
        return AVMP_OK;
    }
    if (launch_pdl(drv_build_kernel, dim3(1), dim3(kStepThreads), 0, S(stream), dr->d) != cudaSuccess) return AVMP_ECUDA;
    int rc = avmp_step_indirect(c, dr->d.ops, dr->d.n_ops_word, dr->max_ops, dr->d.status, stream);
    if (rc != AVMP_OK) return rc;
    if (launch_pdl(drv_feed_kernel, dim3(1), dim3(kStepThreads), 0, S(stream), dr->d) != cudaSuccess) return AVMP_ECUDA;
    c->launches += 2;
    return AVMP_OK;
}

AVMP_API int avmp_driver_get_stats(avmp_driver *dr, avmp_driver_stats *h, void *stream)
{
    if (!dr || !h) return AVMP_EINVAL;
    DrvState s;
    if (cudaMemcpyAsync(&s, dr->d.st, sizeof(s), cudaMemcpyDeviceToHost, S(stream)) != cudaSuccess) return AVMP_ECUDA;
    if (cudaStreamSynchronize(S(stream)) != cudaSuccess) return AVMP_ECUDA;
    h->steps = s.step; h->completed = s.completed; h->dropped = s.dropped; h->preempted = s.preempted;
    h->n_oom_admit = s.n_oom_admit; h->n_oom_extend = s.n_oom_extend; h->queue_next = s.next;
    h->requeued = s.front_count; h->window = s.window; h->last_batch_ops = s.n_ops; h->overflow = s.overflow;
    return AVMP_OK;
}

AVMP_API int avmp_driver_export(avmp_driver *dr, uint32_t *h_state, uint32_t *h_uid, uint32_t *h_len,
                                uint32_t *h_remaining, void *stream)
{
    if (!dr || !h_state || !h_uid || !h_len || !h_remaining) return AVMP_EINVAL;
    const size_t n = (size_t)dr->R * 4;
    cudaStream_t s = S(stream);
    bool ok = cudaMemcpyAsync(h_state, dr->d.slot_state, n, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h_uid, dr->d.slot_uid, n, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h_len, dr->d.slot_len, n, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(h_remaining, dr->d.slot_rem, n, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    if (!ok || cudaStreamSynchronize(s) != cudaSuccess) return AVMP_ECUDA;
    return AVMP_OK;
}

}  // extern "C"
