// The allocator update of one batch as a device function over one CTA (see avmp_step.cu for the
// method): shared by the plain step kernel and by the fused on-device loop.
//
// The path is latency-bound: one CTA, a chain of dependent global round trips with block barriers
// between them.  What keeps the chain short:
//   * the free counts live in registers (every thread holds the same copy and updates it from
//     block-wide totals), so no phase ends with "thread 0 updates, everyone waits";
//   * scans and minima cost one barrier each (double-buffered partials, every thread sums the few
//     warp totals itself);
//   * a window whose ops come as FINISH*, EXTEND*, ADMIT* with ascending slots inside each kind --
//     the shape every engine step has -- is recognised with one ballot per warp: its two runs are
//     known at once, no same-slot table and no run search is needed;
//   * an alloc run whose total demand fits is committed in one pass; only a shortage takes the
//     search for the first failing op and the CapacityError handler.
#pragma once

#include "avmp_dev.cuh"

namespace avmp {
namespace stepimpl {


constexpr uint32_t INF = 0xFFFFFFFFu;
constexpr uint32_t ST_PENDING = 0xFFu;
enum : uint8_t { DIR_NONE = 0, DIR_NOP = 1, DIR_ALLOC = 2, DIR_FREE = 3 };

struct Scalars {
    unsigned long long last, n_oom, n_ce, n_reb, migrated, wasted, reloc_blocks, reloc_bytes, gap, n_invalid;
    unsigned long long counter_base;   // logical counter before the first op of this launch
    long long t_start, t_fail;         // SM clock: launch start, start of the failure being handled
    unsigned long long cyc_oom, cyc_mig;
    uint32_t cap[2], nfree[2], nvfree[2], fsm;
    uint32_t migs_done, abort, abort_idx, n_reloc, reloc_pool;
    // decision of the handler in flight
    uint32_t mig, mig_n, mig_m, newcap;
    unsigned long long mig_waste;
};

// NT = threads of the planning CTA = ops per window.  Small batches run with a small CTA: a barrier
// over 8 warps costs a fraction of one over 32.
template <int NT>
struct Shared {
    static constexpr uint32_t kHash = 2 * NT;     // open-addressing table for same-slot detection
    uint32_t excl_k[NT + 1], excl_s[NT + 1];
    uint32_t req[NT], base[NT];
    uint32_t hkey[kHash], hval[kHash];
    uint8_t dir[NT];
    unsigned long long scan_part[2][32];          // one-barrier scans: warp totals, double-buffered
    uint32_t min_part[2][32];
    unsigned long long tmp64[32];                 // the handler's and the run search's own partials
    uint32_t tmp32[32];
    uint32_t w_shape[32];                         // per warp: window-shape flag and number of FINISH ops
    uint32_t start;                               // first op of this launch (multi-round steps)
    uint32_t n_inv;                               // ops rejected in this launch
    Scalars sc;
};

// Inclusive scan over the block with ONE barrier: after it, every warp scans the (at most 32) warp totals
// for itself with shuffles.  `flip` (the same in every thread) alternates the two partial buffers, so the
// next scan may write while slow threads still read this one's partials.
template <int NT>
__device__ __forceinline__ unsigned long long scan1(unsigned long long v, unsigned long long (*part)[32], uint32_t &flip,
                                                    unsigned long long *total)
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    unsigned long long *t = part[flip & 1u];
    flip ^= 1u;
    v = warp_incl_scan(v);
    if (lane == 31) t[wid] = v;
    __syncthreads();
    const unsigned long long x = warp_incl_scan(lane < NT / 32 ? t[lane] : 0ull);
    *total = __shfl_sync(0xFFFFFFFFu, x, NT / 32 - 1);
    const unsigned long long before = __shfl_sync(0xFFFFFFFFu, x, wid ? wid - 1 : 0);
    return v + (wid ? before : 0ull);
}

template <int NT>
__device__ __forceinline__ uint32_t min1(uint32_t v, uint32_t (*part)[32], uint32_t &flip)
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint32_t *t = part[flip & 1u];
    flip ^= 1u;
    v = __reduce_min_sync(0xFFFFFFFFu, v);
    if (lane == 0) t[wid] = v;
    __syncthreads();
    return __reduce_min_sync(0xFFFFFFFFu, lane < NT / 32 ? t[lane] : INF);
}

// Section 3.2 trigger for a shortage in pool X: the donor Y must have more than threshold_high of its units free
// (strictly), the throttle must have run out, and what it can cede must make at least one whole unit of X.
__device__ __forceinline__ bool would_migrate(const Geom &g, const Scalars &sc, int X, unsigned long long counter,
                                              uint32_t donor_free)
{
    const int Y = 1 - X;
    if (!g.migration_enabled || sc.cap[Y] == 0) return false;
    if (!((unsigned long long)donor_free * 1000000ull > (unsigned long long)g.th_high * sc.cap[Y])) return false;
    if (sc.last != kNone64 && counter - sc.last < g.min_interval) return false;
    const unsigned long long n = g.B < donor_free ? g.B : donor_free;
    // reclaim_gap variant: the bytes already lying between the pools are offered again
    return (n * g.U[Y] + (g.reclaim_gap ? sc.gap : 0ull)) / g.U[X] >= 1ull;
}

// Section 3.2 handler for a shortage in pool X at logical time `counter`; whole CTA.
template <int NT>
__device__ void capacity_error(const Geom &g, Shared<NT> &sh, int X, unsigned long long counter)
{
    Scalars &sc = sh.sc;
    const int Y = 1 - X;
    const int tid = threadIdx.x;
    if (tid == 0) {
        sc.n_ce += 1;
        const uint32_t pressured = X == AVMP_POOL_KV ? AVMP_FSM_KV_PRESSURED : AVMP_FSM_SSM_PRESSURED;
        if ((unsigned long long)sc.nfree[X] * 1000000ull < (unsigned long long)g.th_low * sc.cap[X])
            sc.fsm = pressured;
        else if (sc.fsm == pressured)
            sc.fsm = AVMP_FSM_BALANCED;
        sc.mig = would_migrate(g, sc, X, counter, sc.nfree[Y]) ? 1u : 0u;
        if (sc.mig) {
            const unsigned long long n = g.B < sc.nfree[Y] ? g.B : sc.nfree[Y];
            const unsigned long long carry = g.reclaim_gap ? sc.gap : 0ull;
            const unsigned long long avail = n * g.U[Y] + carry;
            sc.mig_n = (uint32_t)n;
            sc.mig_m = (uint32_t)(avail / g.U[X]);
            sc.mig_waste = avail % g.U[X];
            sc.newcap = sc.cap[Y] - (uint32_t)n;
            sc.fsm = AVMP_FSM_REBALANCING;
        }
    }
    __syncthreads();
    if (!sc.mig) return;

    const uint32_t newcap = sc.newcap, capY = sc.cap[Y], total = sc.nfree[Y], m = sc.mig_m;
    uint32_t *SY = g.S[Y], *OWY = g.OW[Y], *VTY = g.VT[Y];
    unsigned long long tot;

    // 1. The donor shrinks at its high end: drop free slots >= newcap, keeping the order.
    //    In place, kPer consecutive entries per thread and step: a chunk is read in full (the
    //    scan's barriers) before it is written, and writes never pass the chunk's own start.
    constexpr uint32_t kPer = 8;
    uint32_t kept = 0;
    for (uint32_t b = 0; b < total; b += NT * kPer) {
        const uint32_t i0 = b + tid * kPer;
        uint32_t v[kPer];
        uint32_t cnt = 0;
#pragma unroll
        for (uint32_t k = 0; k < kPer; ++k) {
            v[k] = (i0 + k < total) ? SY[i0 + k] : INF;
            cnt += v[k] < newcap ? 1u : 0u;
        }
        const unsigned long long incl = block_incl_scan((unsigned long long)cnt, sh.tmp64, &tot);
        uint32_t o = kept + (uint32_t)incl - cnt;
#pragma unroll
        for (uint32_t k = 0; k < kPer; ++k)
            if (v[k] < newcap) SY[o++] = v[k];
        kept += (uint32_t)tot;
    }
    __syncthreads();

    // 2. Live units in the ceded range, ascending, each to the top of the compacted list.
    uint32_t nrel = 0;
    for (uint32_t b = newcap; b < capY; b += NT) {
        const uint32_t s = b + tid;
        const uint32_t v = s < capY ? OWY[s] : INF;
        const bool live = v != INF;
        const unsigned long long incl = block_incl_scan(live ? 1ull : 0ull, sh.tmp64, &tot);
        if (live) {
            const uint32_t k = nrel + (uint32_t)incl - 1u;
            const uint32_t d = SY[kept - 1u - k];
            g.reloc_src[k] = s;
            g.reloc_dst[k] = d;
            VTY[v] = d;
            OWY[d] = v;
            OWY[s] = INF;
        }
        nrel += (uint32_t)tot;
    }

    // 3. The recipient grows by whole units; the lowest new slot ends on top.
    {
        uint32_t *SX = g.S[X];
        const uint32_t top = sc.nfree[X], capX = sc.cap[X];
        for (uint32_t j = tid; j < m; j += NT) SX[top + j] = capX + m - 1u - j;
    }
    __syncthreads();
    if (tid == 0) {
        sc.nfree[Y] = kept - nrel;
        sc.cap[Y] = newcap;
        sc.nfree[X] += m;
        sc.cap[X] += m;
        if (g.reclaim_gap) {
            sc.gap = sc.mig_waste;          // the old gap went into the offer
        } else {
            sc.gap += sc.mig_waste;
            sc.wasted += sc.mig_waste;
        }
        sc.migrated += (unsigned long long)sc.mig_n * g.U[Y];
        sc.n_reb += 1;
        sc.last = counter;
        sc.reloc_blocks += nrel;
        sc.reloc_bytes += (unsigned long long)nrel * g.U[Y];
        sc.fsm = AVMP_FSM_BALANCED;
        sc.migs_done += 1;
        sc.n_reloc = nrel;
        sc.reloc_pool = (uint32_t)Y;
    }
    __syncthreads();
}

// Pop units for the ops [lo, hi) of the current alloc scan (none of them fails): unit u of the run
// takes stack entry (top - 1 - u).  fk / vk / fs / vs are the stack heights before the run.
template <int NT>
__device__ __forceinline__ void pop_units(const Geom &g, Shared<NT> &sh, uint32_t lo, uint32_t hi,
                                          uint32_t fk, uint32_t vk, uint32_t fs, uint32_t vs, uint32_t &Tk, uint32_t &Ts)
{
    const int tid = threadIdx.x;
    const uint32_t bk = sh.excl_k[lo], bs = sh.excl_s[lo];
    Tk = sh.excl_k[hi] - bk; Ts = sh.excl_s[hi] - bs;
    for (uint32_t u = tid; u < Tk; u += NT) {
        const uint32_t idx = find_owner(sh.excl_k, lo, hi, bk, u);
        const uint32_t j = u - (sh.excl_k[idx] - bk);
        const uint32_t slot = g.S[0][fk - 1u - u], vid = g.W[0][vk - 1u - u];
        g.VT[0][vid] = slot;
        g.OW[0][slot] = vid;
        g.r_chain[(unsigned long long)sh.req[idx] * g.max_pages + sh.base[idx] + j] = vid;
    }
    for (uint32_t u = tid; u < Ts; u += NT) {
        const uint32_t idx = find_owner(sh.excl_s, lo, hi, bs, u);
        const uint32_t j = u - (sh.excl_s[idx] - bs);
        const uint32_t slot = g.S[1][fs - 1u - u], vid = g.W[1][vs - 1u - u];
        g.VT[1][vid] = slot;
        g.OW[1][slot] = vid;
        g.r_ssm[(unsigned long long)sh.req[idx] * g.ns + j] = 0x80000000u | vid;
    }
}

// The whole allocator update for ops[0 .. n_ops) by the calling CTA of NT threads (callers have
// already waited for everything earlier in the stream).
template <int NT>
__device__ void step_body(const Geom &g, Shared<NT> &sh, const avmp_op *ops, const uint32_t n_ops,
                          uint32_t *status, const int first_round)
{
    constexpr uint32_t kHash = Shared<NT>::kHash;
    Scalars &sc = sh.sc;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    DevState *ds = g.st;
    uint32_t flip_s = 0, flip_m = 0;                // buffer toggles of scan1 / min1, the same in every thread

    // The first window's ops are fetched while thread 0 fetches the counters (first round: the batch
    // starts at op 0; later rounds must learn where the last one stopped).
    uint32_t pre_w0 = 0, pre_w1 = 0, pre_w2 = 0, pre_pw0 = 0, pre_pw1 = 0;
    const bool preloaded = first_round != 0;
    if (preloaded && (uint32_t)tid < n_ops) {
        const uint32_t *w = reinterpret_cast<const uint32_t *>(ops + tid);
        pre_w0 = w[0]; pre_w1 = w[1]; pre_w2 = w[2];
        if (lane == 0 && tid > 0) { pre_pw0 = w[-3]; pre_pw1 = w[-2]; }     // the op before this warp's first
    }
    if (tid == 0) {
        const unsigned long long a0 = ds->last_rebalance_op, a1 = ds->n_oom, a2 = ds->n_capacity_error, a3 = ds->n_rebalance,
                                 a4 = ds->migrated_bytes, a5 = ds->wasted_bytes, a6 = ds->relocated_blocks,
                                 a7 = ds->relocated_bytes, a8 = ds->gap_bytes, a9 = ds->n_invalid, a10 = ds->op_counter;
        const uint32_t c0 = ds->cap[0], c1 = ds->cap[1], f0 = ds->n_free[0], f1 = ds->n_free[1], v0 = ds->n_vfree[0],
                       v1 = ds->n_vfree[1], fsm = ds->fsm, pend = ds->reloc_pending, res = first_round ? 0u : ds->resume_idx;
        sc.last = a0; sc.n_oom = a1; sc.n_ce = a2; sc.n_reb = a3; sc.migrated = a4; sc.wasted = a5;
        sc.reloc_blocks = a6; sc.reloc_bytes = a7; sc.gap = a8; sc.n_invalid = a9; sc.counter_base = a10;
        sc.t_start = clock64(); sc.cyc_oom = 0; sc.cyc_mig = 0;
        sc.cap[0] = c0; sc.cap[1] = c1; sc.nfree[0] = f0; sc.nfree[1] = f1; sc.nvfree[0] = v0; sc.nvfree[1] = v1;
        sc.fsm = fsm;
        if (pend) {                         // fold the last relocation copy's duration into the total
            const unsigned long long t0 = ds->reloc_t0, t1 = ds->reloc_t1;
            if (t1 > t0) ds->reloc_ns_total += t1 - t0;
            ds->reloc_pending = 0;
        }
        sc.migs_done = 0; sc.abort = 0; sc.abort_idx = 0; sc.n_reloc = 0; sc.reloc_pool = 0;
        sc.mig = 0;
        sh.start = res;
        sh.n_inv = 0;
    }
    uint32_t start = 0;
    if (!preloaded) {
        __syncthreads();
        start = sh.start;
    }
    if (start >= n_ops) {               // an earlier round finished the batch (or the batch is empty)
        if (tid == 0) ds->n_reloc = 0;
        return;
    }
    // free counts: registers, the same in every thread (filled after the first window's barrier)
    uint32_t nf0 = 0, nv0 = 0, nf1 = 0, nv1 = 0;
    bool have_counts = false;

    uint32_t done_upto = n_ops;     // ops [start, done_upto) are applied when the launch ends
    bool aborted = false;
    for (uint32_t w0 = start; w0 < n_ops; w0 += NT) {
        const uint32_t wn = min((uint32_t)NT, n_ops - w0);
        // ---- decode (a1) ----
        uint32_t kind = 0, flags = 0, req = 0, tokens = 0, st = ST_PENDING;
        uint32_t prev_word0 = 0, prev_req = 0;
        uint8_t dir = DIR_NONE;
        if (tid < (int)wn) {
            uint32_t w0_, w1_, w2_;
            if (preloaded && w0 == 0) { w0_ = pre_w0; w1_ = pre_w1; w2_ = pre_w2; prev_word0 = pre_pw0; prev_req = pre_pw1; }
            else {
                const uint32_t *w = reinterpret_cast<const uint32_t *>(ops + (w0 + tid));
                w0_ = w[0]; w1_ = w[1]; w2_ = w[2];
                if (lane == 0 && tid > 0) { prev_word0 = w[-3]; prev_req = w[-2]; }
            }
            kind = w0_ & 0xFFu; flags = (w0_ >> 8) & 0xFFu; req = w1_; tokens = w2_;
            dir = DIR_NOP;
            if (kind != AVMP_OP_ADMIT && kind != AVMP_OP_EXTEND && kind != AVMP_OP_FINISH) st = AVMP_ST_BAD_ARG;
            else if (req >= g.R) st = AVMP_ST_BAD_REQ;
            else if (kind != AVMP_OP_FINISH && tokens == 0) st = AVMP_ST_BAD_ARG;
            else dir = kind == AVMP_OP_FINISH ? DIR_FREE : DIR_ALLOC;
        }
        sh.dir[tid] = dir;
        sh.req[tid] = req;
        // request record, fetched now so the loads overlap the bookkeeping below; ops whose slot
        // appears earlier in the window read it again when their run starts
        uint32_t pf_state = 0, pf_len = 0, pf_np = 0;
        if (dir >= DIR_ALLOC) { pf_state = g.r_state[req]; pf_len = g.r_len[req]; pf_np = g.r_npages[req]; }

        // ---- shape of the window: FINISH*, EXTEND*, ADMIT*, every op valid, slots ascending inside a kind ----
        // rank: FINISH 0 < EXTEND 1 < ADMIT 2.  An op is in place if the op before it has a lower rank, or the same
        // rank and a lower slot.  One ballot per warp; lane 0 compares with the op it fetched beside its own.
        {
            const uint32_t rank = kind == AVMP_OP_FINISH ? 0u : (kind == AVMP_OP_EXTEND ? 1u : 2u);
            uint32_t p_rank = __shfl_up_sync(0xFFFFFFFFu, rank, 1), p_req = __shfl_up_sync(0xFFFFFFFFu, req, 1);
            if (lane == 0) {
                const uint32_t pk = prev_word0 & 0xFFu;
                p_rank = pk == AVMP_OP_FINISH ? 0u : (pk == AVMP_OP_EXTEND ? 1u : 2u);
                p_req = prev_req;
            }
            bool in_place = true;
            if (tid < (int)wn) in_place = dir >= DIR_ALLOC && (tid == 0 || p_rank < rank || (p_rank == rank && p_req < req));
            const uint32_t ok = __all_sync(0xFFFFFFFFu, in_place) ? 1u : 0u;
            const uint32_t nfin = __popc(__ballot_sync(0xFFFFFFFFu, tid < (int)wn && dir == DIR_FREE));
            if (lane == 0) sh.w_shape[wid] = (ok << 31) | nfin;
        }
        __syncthreads();                                    // B1: counters, dir / req, window shape
        if (!have_counts) {
            nf0 = sc.nfree[0]; nv0 = sc.nvfree[0]; nf1 = sc.nfree[1]; nv1 = sc.nvfree[1];
            have_counts = true;
        }
        const uint32_t shape = lane < NT / 32 ? sh.w_shape[lane] : 0x80000000u;
        const bool fast = __all_sync(0xFFFFFFFFu, (shape >> 31) != 0u);
        const uint32_t nF = __reduce_add_sync(0xFFFFFFFFu, shape & 0x7FFFFFFFu);

        // ---- same-slot dependencies inside the window ----
        int prev_same = -1;        // >= 0: an earlier op of this window touches the same slot
        if (fast) {
            // Runs are [0, nF) and [nF, wn); slots are distinct inside each.  An alloc op only has to know
            // whether a FINISH of this window released its slot (its prefetched record is then stale):
            // the FINISH slots ascend, so a binary search answers that.
            if (nF > 0 && tid >= (int)nF && tid < (int)wn) {
                uint32_t lo = 0, hi = nF;
                while (lo < hi) {
                    const uint32_t mid = (lo + hi) >> 1;
                    if (sh.req[mid] < req) lo = mid + 1; else hi = mid;
                }
                if (lo < nF && sh.req[lo] == req) prev_same = (int)lo;
            }
        } else {
            // general windows: shared-memory hash, slot -> first op
            sh.hkey[tid] = INF; sh.hkey[tid + NT] = INF;
            sh.hval[tid] = INF; sh.hval[tid + NT] = INF;
            __syncthreads();
            uint32_t hs = 0;
            if (dir >= DIR_ALLOC) {
                hs = (req * 2654435761u) & (kHash - 1u);
                while (true) {
                    const uint32_t old = atomicCAS(&sh.hkey[hs], INF, req);
                    if (old == INF || old == req) break;
                    hs = (hs + 1u) & (kHash - 1u);
                }
                atomicMin(&sh.hval[hs], (uint32_t)tid);
            }
            __syncthreads();
            const bool dupflag = dir >= DIR_ALLOC && sh.hval[hs] != (uint32_t)tid;
            const int any_dup = __syncthreads_or(dupflag);
            if (any_dup && dupflag)
                for (int j = tid - 1; j >= 0; --j)
                    if (sh.dir[j] >= DIR_ALLOC && sh.req[j] == req) { prev_same = j; break; }
        }

        uint32_t cur = 0;
        while (cur < wn) {
            uint32_t end;
            uint8_t rdir;
            if (fast) {
                rdir = cur < nF ? DIR_FREE : DIR_ALLOC;
                end = cur < nF ? nF : wn;
            } else {
                const uint32_t first = block_min((tid >= (int)cur && dir >= DIR_ALLOC) ? (uint32_t)tid : INF, sh.tmp32);
                if (first == INF) break;
                rdir = sh.dir[first];
                const bool stops = tid > (int)first && tid < (int)wn &&
                                   ((dir >= DIR_ALLOC && dir != rdir) || prev_same >= (int)cur);
                end = block_min(stops ? (uint32_t)tid : wn, sh.tmp32);
            }
            const bool in_run = tid >= (int)cur && tid < (int)end && dir == rdir;
            unsigned long long tot;

            if (rdir == DIR_FREE) {
                // ---- free run (a3) ----
                uint32_t nk = 0, nsu = 0, rstate = 0;
                bool valid = false;
                const bool keep = (flags & AVMP_FLAG_KEEP_KV) != 0;
                if (in_run) {
                    const bool fresh = prev_same < 0;
                    rstate = fresh ? pf_state : g.r_state[req];
                    if (rstate == AVMP_REQ_LIVE || rstate == AVMP_REQ_KV_ONLY) {
                        valid = true;
                        nk = keep ? 0u : (fresh ? pf_np : g.r_npages[req]);
                        nsu = rstate == AVMP_REQ_LIVE ? g.ns : 0u;
                        st = AVMP_ST_OK;
                    } else st = AVMP_ST_BAD_REQ;
                }
                const unsigned long long incl = scan1<NT>(((unsigned long long)nsu << 32) | nk, sh.scan_part, flip_s, &tot);
                sh.excl_k[tid] = (uint32_t)incl - nk;
                sh.excl_s[tid] = (uint32_t)(incl >> 32) - nsu;
                if (tid == NT - 1) { sh.excl_k[NT] = (uint32_t)tot; sh.excl_s[NT] = (uint32_t)(tot >> 32); }
                __syncthreads();
                const uint32_t Tk = (uint32_t)tot, Ts = (uint32_t)(tot >> 32);
                for (uint32_t u = tid; u < Tk; u += NT) {
                    const uint32_t idx = find_owner(sh.excl_k, cur, end, 0u, u);
                    const uint32_t j = u - sh.excl_k[idx];
                    const uint32_t vid = g.r_chain[(unsigned long long)sh.req[idx] * g.max_pages + j] & 0x7FFFFFFFu;
                    const uint32_t slot = g.VT[0][vid];
                    g.VT[0][vid] = INF;
                    g.OW[0][slot] = INF;
                    g.S[0][nf0 + u] = slot;
                    g.W[0][nv0 + u] = vid;
                }
                for (uint32_t u = tid; u < Ts; u += NT) {
                    const uint32_t idx = find_owner(sh.excl_s, cur, end, 0u, u);
                    const uint32_t j = u - sh.excl_s[idx];
                    const uint32_t vid = g.r_ssm[(unsigned long long)sh.req[idx] * g.ns + j] & 0x7FFFFFFFu;
                    const uint32_t slot = g.VT[1][vid];
                    g.VT[1][vid] = INF;
                    g.OW[1][slot] = INF;
                    g.S[1][nf1 + u] = slot;
                    g.W[1][nv1 + u] = vid;
                }
                if (valid) {
                    if (!keep) { g.r_npages[req] = 0; g.r_len[req] = 0; }
                    g.r_state[req] = keep ? AVMP_REQ_KV_ONLY : AVMP_REQ_EMPTY;
                }
                nf0 += Tk; nv0 += Tk; nf1 += Ts; nv1 += Ts;
                __syncthreads();            // the lists and records are in place for what follows
            } else {
                // ---- alloc run (a4, a5-a9 on shortage) ----
                uint32_t nk = 0, nsu = 0, new_len = 0;
                bool valid = false;
                if (in_run) {
                    const bool fresh = prev_same < 0;
                    const uint32_t rstate = fresh ? pf_state : g.r_state[req];
                    bool ok_state;
                    if (kind == AVMP_OP_ADMIT)
                        ok_state = (flags & AVMP_FLAG_RESUME) ? rstate == AVMP_REQ_KV_ONLY : rstate == AVMP_REQ_EMPTY;
                    else
                        ok_state = rstate == AVMP_REQ_LIVE;
                    if (!ok_state) st = AVMP_ST_BAD_REQ;
                    else {
                        const unsigned long long nl = (unsigned long long)(fresh ? pf_len : g.r_len[req]) + tokens;
                        const unsigned long long pages = (nl + g.T - 1ull) / g.T;
                        const uint32_t have = fresh ? pf_np : g.r_npages[req];
                        if (pages > g.max_pages || nl > 0xFFFFFFFFull) st = AVMP_ST_TOO_LONG;
                        else {
                            valid = true;
                            nk = (uint32_t)pages - have;
                            nsu = kind == AVMP_OP_ADMIT ? g.ns : 0u;
                            new_len = (uint32_t)nl;
                            sh.base[tid] = have;
                        }
                    }
                }
                const unsigned long long incl = scan1<NT>(((unsigned long long)nsu << 32) | nk, sh.scan_part, flip_s, &tot);
                sh.excl_k[tid] = (uint32_t)incl - nk;
                sh.excl_s[tid] = (uint32_t)(incl >> 32) - nsu;
                if (tid == NT - 1) { sh.excl_k[NT] = (uint32_t)tot; sh.excl_s[NT] = (uint32_t)(tot >> 32); }
                __syncthreads();

                // demand of the run's ops alone (the scan covers the whole block; ops outside the run add nothing)
                if ((uint32_t)tot <= nf0 && (uint32_t)(tot >> 32) <= nf1) {
                    // everything fits: one pass
                    uint32_t Tk, Ts;
                    pop_units<NT>(g, sh, cur, end, nf0, nv0, nf1, nv1, Tk, Ts);
                    if (valid) {
                        g.r_npages[req] = sh.base[tid] + nk;
                        g.r_len[req] = new_len;
                        g.r_state[req] = AVMP_REQ_LIVE;
                        st = AVMP_ST_OK;
                    }
                    nf0 -= Tk; nv0 -= Tk; nf1 -= Ts; nv1 -= Ts;
                    __syncthreads();        // the tables are in place for what follows
                } else {
                    // Shortage somewhere in the run.  Everything before the first op that does not fit is
                    // committed; that op's CapacityError is decided by every thread alike (free counts in
                    // registers; capacities, throttle state and gap in shared memory, which only a migration
                    // changes) and thread 0 keeps the counters, so an error that cannot migrate -- the usual
                    // case under the throttle -- costs no barrier.  Only a migration takes the handler.
                    uint32_t c2 = cur;
                    while (c2 < end) {
                        // first op of [c2, end) that does not fit, given that all before it do
                        const uint32_t bk = sh.excl_k[c2], bs = sh.excl_s[c2];
                        const bool fails = valid && tid >= (int)c2 && tid < (int)end &&
                                           ((uint32_t)incl - bk > nf0 || (uint32_t)(incl >> 32) - bs > nf1);
                        const uint32_t f = min1<NT>(fails ? (uint32_t)tid : end, sh.min_part, flip_m);
                        if (f > c2) {
                            uint32_t Tk, Ts;
                            pop_units<NT>(g, sh, c2, f, nf0, nv0, nf1, nv1, Tk, Ts);
                            if (valid && tid >= (int)c2 && tid < (int)f) {
                                g.r_npages[req] = sh.base[tid] + nk;
                                g.r_len[req] = new_len;
                                g.r_state[req] = AVMP_REQ_LIVE;
                                st = AVMP_ST_OK;
                            }
                            nf0 -= Tk; nv0 -= Tk; nf1 -= Ts; nv1 -= Ts;
                        }
                        if (f >= end) break;

                        // ---- op f raises CapacityError (SSM first, then KV) ----
                        const uint32_t need_k = sh.excl_k[f + 1] - sh.excl_k[f];
                        const uint32_t need_s = sh.excl_s[f + 1] - sh.excl_s[f];
                        const unsigned long long counter = sc.counter_base + (w0 - start) + f + 1ull;
                        const bool wantA = need_s > nf1;
                        const bool trigA = wantA && would_migrate(g, sc, AVMP_POOL_SSM, counter, nf0);
                        const bool trigB = !trigA && need_k > nf0 && would_migrate(g, sc, AVMP_POOL_KV, counter, nf1);
                        if ((trigA || trigB) && sc.migs_done >= 1u) {
                            // a second migration must wait for the first one's copies: stop here
                            __syncthreads();
                            if (tid == 0) { sc.abort = 1; sc.abort_idx = f; }
                            __syncthreads();
                            break;
                        }
                        if (tid == 0) sc.t_fail = clock64();
                        auto label_only = [&](int X, uint32_t nfX) {          // thread 0: the handler without a migration
                            sc.n_ce += 1;
                            const uint32_t pressured = X == AVMP_POOL_KV ? AVMP_FSM_KV_PRESSURED : AVMP_FSM_SSM_PRESSURED;
                            if ((unsigned long long)nfX * 1000000ull < (unsigned long long)g.th_low * sc.cap[X]) sc.fsm = pressured;
                            else if (sc.fsm == pressured) sc.fsm = AVMP_FSM_BALANCED;
                        };
                        auto migrate = [&](int X) {                            // whole CTA: the handler with its migration
                            if (tid == 0) { sc.nfree[0] = nf0; sc.nvfree[0] = nv0; sc.nfree[1] = nf1; sc.nvfree[1] = nv1; }
                            __syncthreads();
                            capacity_error(g, sh, X, counter);
                            nf0 = sc.nfree[0]; nv0 = sc.nvfree[0]; nf1 = sc.nfree[1]; nv1 = sc.nvfree[1];
                        };
                        if (wantA) {
                            if (trigA) migrate(AVMP_POOL_SSM);
                            else if (tid == 0) label_only(AVMP_POOL_SSM, nf1);
                        }
                        if (need_k > nf0) {      // a migration for the SSM pool may have taken KV capacity
                            if (trigB) migrate(AVMP_POOL_KV);
                            else if (tid == 0) label_only(AVMP_POOL_KV, nf0);   // after trigA the throttle forbids a second one
                        }
                        if (need_s <= nf1 && need_k <= nf0) {
                            uint32_t Tk, Ts;
                            pop_units<NT>(g, sh, f, f + 1, nf0, nv0, nf1, nv1, Tk, Ts);
                            if (tid == (int)f) {
                                g.r_npages[req] = sh.base[tid] + nk;
                                g.r_len[req] = new_len;
                                g.r_state[req] = AVMP_REQ_LIVE;
                                st = AVMP_ST_OK;
                            }
                            nf0 -= Tk; nv0 -= Tk; nf1 -= Ts; nv1 -= Ts;
                        } else {
                            if (tid == (int)f) st = AVMP_ST_OOM;
                            if (tid == 0) sc.n_oom += 1;
                        }
                        // time decomposition (paper Section 4.3): cycles spent on this failure go to the
                        // migration bucket if it migrated, to the OOM-retry bucket otherwise
                        if (tid == 0) {
                            const unsigned long long dt = (unsigned long long)(clock64() - sc.t_fail);
                            if (trigA || trigB) sc.cyc_mig += dt; else sc.cyc_oom += dt;
                        }
                        c2 = f + 1;
                    }
                    __syncthreads();        // the tables are in place for what follows
                    aborted = sc.abort != 0;
                    if (aborted) break;
                }
            }
            cur = end;
        }
        // ---- statuses of this window ----
        const uint32_t limit = aborted ? sc.abort_idx : wn;
        const bool decided = tid < (int)limit;
        if (decided) status[w0 + tid] = st;
        const uint32_t n_inv = __popc(__ballot_sync(0xFFFFFFFFu, decided && st >= AVMP_ST_BAD_REQ && st != ST_PENDING));
        if (lane == 0 && n_inv) atomicAdd(&sh.n_inv, n_inv);
        if (aborted) { done_upto = w0 + sc.abort_idx; break; }
        if (w0 + NT < n_ops) __syncthreads();       // the next window reuses dir / req / w_shape
    }

    __syncthreads();                                // n_inv and the handler's scalars are final
    if (tid == 0) {
        ds->last_rebalance_op = sc.last; ds->n_oom = sc.n_oom; ds->n_capacity_error = sc.n_ce;
        ds->n_rebalance = sc.n_reb; ds->migrated_bytes = sc.migrated; ds->wasted_bytes = sc.wasted;
        ds->relocated_blocks = sc.reloc_blocks; ds->relocated_bytes = sc.reloc_bytes;
        ds->gap_bytes = sc.gap; ds->n_invalid = sc.n_invalid + sh.n_inv;
        ds->op_counter = sc.counter_base + (done_upto - start);
        ds->cap[0] = sc.cap[0]; ds->cap[1] = sc.cap[1];
        ds->n_free[0] = nf0; ds->n_free[1] = nf1; ds->n_vfree[0] = nv0; ds->n_vfree[1] = nv1;
        ds->fsm = sc.fsm;
        ds->resume_idx = done_upto;
        ds->cyc_total += (unsigned long long)(clock64() - sc.t_start);
        ds->cyc_oom += sc.cyc_oom;
        ds->cyc_mig += sc.cyc_mig;
        ds->n_reloc = sc.n_reloc;
        ds->reloc_pool = sc.reloc_pool;
        if (sc.n_reloc) { ds->reloc_t0 = kNone64; ds->reloc_t1 = 0; ds->reloc_pending = 1; }
    }
}


}  // namespace stepimpl
}  // namespace avmp
