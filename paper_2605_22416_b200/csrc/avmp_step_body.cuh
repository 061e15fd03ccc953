// The allocator update of one batch as a device function over one CTA (see avmp_step.cu for the
// method): shared by the plain step kernel and by the fused on-device loop.
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

// NT = threads of the planning CTA = ops per window.  Small batches run with a small CTA: the
// kernel is a chain of some forty block barriers, and a barrier over 8 warps costs a fraction of
// one over 32.
template <int NT>
struct Shared {
    static constexpr uint32_t kHash = 2 * NT;     // open-addressing table for same-slot detection
    uint32_t excl_k[NT + 1], excl_s[NT + 1];
    uint32_t req[NT], base[NT];
    uint32_t hkey[kHash], hval[kHash];
    uint8_t dir[NT];
    unsigned long long tmp64[32];
    uint32_t tmp32[32];
    Scalars sc;
};

__device__ __forceinline__ bool would_migrate(const Geom &g, const Scalars &sc, int X, unsigned long long counter)
{
    const int Y = 1 - X;
    if (!g.migration_enabled || sc.cap[Y] == 0) return false;
    if (!((unsigned long long)sc.nfree[Y] * 1000000ull > (unsigned long long)g.th_high * sc.cap[Y])) return false;
    if (sc.last != kNone64 && counter - sc.last < g.min_interval) return false;
    const unsigned long long n = g.B < sc.nfree[Y] ? g.B : sc.nfree[Y];
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
        sc.mig = would_migrate(g, sc, X, counter) ? 1u : 0u;
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

// Pop units for the ops [lo, hi) of the current alloc scan (none of them fails).
template <int NT>
__device__ __forceinline__ void commit_allocs(const Geom &g, Shared<NT> &sh, uint32_t lo, uint32_t hi)
{
    Scalars &sc = sh.sc;
    const int tid = threadIdx.x;
    const uint32_t bk = sh.excl_k[lo], bs = sh.excl_s[lo];
    const uint32_t Tk = sh.excl_k[hi] - bk, Ts = sh.excl_s[hi] - bs;
    const uint32_t fk = sc.nfree[0], vk = sc.nvfree[0], fs = sc.nfree[1], vs = sc.nvfree[1];
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
    __syncthreads();
    if (tid == 0) {
        sc.nfree[0] -= Tk; sc.nvfree[0] -= Tk;
        sc.nfree[1] -= Ts; sc.nvfree[1] -= Ts;
    }
    __syncthreads();
}

// The whole allocator update for ops[0 .. n_ops) by the calling CTA of NT threads (callers have
// already waited for everything earlier in the stream).
template <int NT>
__device__ void step_body(const Geom &g, Shared<NT> &sh, const avmp_op *__restrict__ ops, const uint32_t n_ops,
                          uint32_t *__restrict__ status, const int first_round)
{
    constexpr uint32_t kHash = Shared<NT>::kHash;
    Scalars &sc = sh.sc;
    const int tid = threadIdx.x;
    DevState *ds = g.st;

    if (tid == 0) {
        sc.last = ds->last_rebalance_op; sc.n_oom = ds->n_oom; sc.n_ce = ds->n_capacity_error;
        sc.n_reb = ds->n_rebalance; sc.migrated = ds->migrated_bytes; sc.wasted = ds->wasted_bytes;
        sc.reloc_blocks = ds->relocated_blocks; sc.reloc_bytes = ds->relocated_bytes;
        sc.gap = ds->gap_bytes; sc.n_invalid = ds->n_invalid; sc.counter_base = ds->op_counter;
        sc.t_start = clock64(); sc.cyc_oom = 0; sc.cyc_mig = 0;
        for (int p = 0; p < 2; ++p) { sc.cap[p] = ds->cap[p]; sc.nfree[p] = ds->n_free[p]; sc.nvfree[p] = ds->n_vfree[p]; }
        sc.fsm = ds->fsm;
        if (ds->reloc_pending) {            // fold the last relocation copy's duration into the total
            if (ds->reloc_t1 > ds->reloc_t0) ds->reloc_ns_total += ds->reloc_t1 - ds->reloc_t0;
            ds->reloc_pending = 0;
        }
        sc.migs_done = 0; sc.abort = 0; sc.abort_idx = 0; sc.n_reloc = 0; sc.reloc_pool = 0;
        sc.mig = 0;
        sh.excl_k[0] = first_round ? 0u : ds->resume_idx;    // borrow a slot to broadcast the start
    }
    __syncthreads();
    const uint32_t start = sh.excl_k[0];
    __syncthreads();
    if (start >= n_ops) {           // an earlier round finished the batch
        if (tid == 0) ds->n_reloc = 0;
        return;
    }

    uint32_t done_upto = n_ops;     // ops [start, done_upto) are applied when the launch ends
    for (uint32_t w0 = start; w0 < n_ops; w0 += NT) {
        const uint32_t wn = min((uint32_t)NT, n_ops - w0);
        // ---- decode (a1) ----
        uint32_t kind = 0, flags = 0, req = 0, tokens = 0, st = ST_PENDING;
        uint8_t dir = DIR_NONE;
        if (tid < wn) {
            const uint32_t *w = reinterpret_cast<const uint32_t *>(ops + (w0 + tid));
            const uint32_t w0_ = w[0];
            kind = w0_ & 0xFFu; flags = (w0_ >> 8) & 0xFFu; req = w[1]; tokens = w[2];
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
        // ---- same-slot dependencies inside the window: shared-memory hash, slot -> first op ----
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
        int prev_same = -1;
        if (any_dup && dupflag)
            for (int j = tid - 1; j >= 0; --j)
                if (sh.dir[j] >= DIR_ALLOC && sh.req[j] == req) { prev_same = j; break; }

        uint32_t cur = 0;
        while (cur < wn) {
            const uint32_t first = block_min((tid >= (int)cur && dir >= DIR_ALLOC) ? (uint32_t)tid : INF, sh.tmp32);
            if (first == INF) break;
            const uint8_t rdir = sh.dir[first];
            const bool stops = tid > (int)first && tid < (int)wn &&
                               ((dir >= DIR_ALLOC && dir != rdir) || prev_same >= (int)cur);
            const uint32_t end = block_min(stops ? (uint32_t)tid : wn, sh.tmp32);
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
                const unsigned long long incl =
                    block_incl_scan(((unsigned long long)nsu << 32) | nk, sh.tmp64, &tot);
                sh.excl_k[tid] = (uint32_t)incl - nk;
                sh.excl_s[tid] = (uint32_t)(incl >> 32) - nsu;
                if (tid == NT - 1) { sh.excl_k[NT] = (uint32_t)tot; sh.excl_s[NT] = (uint32_t)(tot >> 32); }
                __syncthreads();
                const uint32_t Tk = (uint32_t)tot, Ts = (uint32_t)(tot >> 32);
                const uint32_t fk = sc.nfree[0], vk = sc.nvfree[0], fs = sc.nfree[1], vs = sc.nvfree[1];
                for (uint32_t u = tid; u < Tk; u += NT) {
                    const uint32_t idx = find_owner(sh.excl_k, cur, end, 0u, u);
                    const uint32_t j = u - sh.excl_k[idx];
                    const uint32_t vid = g.r_chain[(unsigned long long)sh.req[idx] * g.max_pages + j] & 0x7FFFFFFFu;
                    const uint32_t slot = g.VT[0][vid];
                    g.VT[0][vid] = INF;
                    g.OW[0][slot] = INF;
                    g.S[0][fk + u] = slot;
                    g.W[0][vk + u] = vid;
                }
                for (uint32_t u = tid; u < Ts; u += NT) {
                    const uint32_t idx = find_owner(sh.excl_s, cur, end, 0u, u);
                    const uint32_t j = u - sh.excl_s[idx];
                    const uint32_t vid = g.r_ssm[(unsigned long long)sh.req[idx] * g.ns + j] & 0x7FFFFFFFu;
                    const uint32_t slot = g.VT[1][vid];
                    g.VT[1][vid] = INF;
                    g.OW[1][slot] = INF;
                    g.S[1][fs + u] = slot;
                    g.W[1][vs + u] = vid;
                }
                if (valid) {
                    if (!keep) { g.r_npages[req] = 0; g.r_len[req] = 0; }
                    g.r_state[req] = keep ? AVMP_REQ_KV_ONLY : AVMP_REQ_EMPTY;
                }
                __syncthreads();
                if (tid == 0) {
                    sc.nfree[0] += Tk; sc.nvfree[0] += Tk;
                    sc.nfree[1] += Ts; sc.nvfree[1] += Ts;
                }
                __syncthreads();
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
                const unsigned long long incl =
                    block_incl_scan(((unsigned long long)nsu << 32) | nk, sh.tmp64, &tot);
                sh.excl_k[tid] = (uint32_t)incl - nk;
                sh.excl_s[tid] = (uint32_t)(incl >> 32) - nsu;
                if (tid == NT - 1) { sh.excl_k[NT] = (uint32_t)tot; sh.excl_s[NT] = (uint32_t)(tot >> 32); }
                __syncthreads();

                uint32_t c2 = cur;
                while (c2 < end) {
                    // first op of [c2, end) that does not fit, given that all before it do
                    const uint32_t bk = sh.excl_k[c2], bs = sh.excl_s[c2];
                    const bool fails = valid && tid >= (int)c2 && tid < (int)end &&
                                       ((uint32_t)incl - bk > sc.nfree[0] || (uint32_t)(incl >> 32) - bs > sc.nfree[1]);
                    const uint32_t f = block_min(fails ? (uint32_t)tid : end, sh.tmp32);
                    if (f > c2) commit_allocs(g, sh, c2, f);
                    if (valid && tid >= (int)c2 && tid < (int)f) {
                        g.r_npages[req] = sh.base[tid] + nk;
                        g.r_len[req] = new_len;
                        g.r_state[req] = AVMP_REQ_LIVE;
                        st = AVMP_ST_OK;
                    }
                    if (f >= end) break;

                    // ---- op f raises CapacityError ----
                    const uint32_t need_k = sh.excl_k[f + 1] - sh.excl_k[f];
                    const uint32_t need_s = sh.excl_s[f + 1] - sh.excl_s[f];
                    const unsigned long long counter = sc.counter_base + (w0 - start) + f + 1ull;
                    const bool wantA = need_s > sc.nfree[1];
                    const bool trigA = wantA && would_migrate(g, sc, AVMP_POOL_SSM, counter);
                    const bool trigB = !trigA && need_k > sc.nfree[0] && would_migrate(g, sc, AVMP_POOL_KV, counter);
                    if ((trigA || trigB) && sc.migs_done >= 1u) {
                        // a second migration must wait for the first one's copies: stop here
                        __syncthreads();
                        if (tid == 0) { sc.abort = 1; sc.abort_idx = f; }
                        __syncthreads();
                        break;
                    }
                    const uint32_t migs_before = sc.migs_done;
                    if (tid == 0) sc.t_fail = clock64();
                    if (wantA) capacity_error(g, sh, AVMP_POOL_SSM, counter);
                    if (need_k > sc.nfree[0]) capacity_error(g, sh, AVMP_POOL_KV, counter);
                    const bool fits = need_s <= sc.nfree[1] && need_k <= sc.nfree[0];
                    if (fits) {
                        commit_allocs(g, sh, f, f + 1);
                        if (tid == (int)f) {
                            g.r_npages[req] = sh.base[tid] + nk;
                            g.r_len[req] = new_len;
                            g.r_state[req] = AVMP_REQ_LIVE;
                            st = AVMP_ST_OK;
                        }
                    } else {
                        if (tid == (int)f) { st = AVMP_ST_OOM; sc.n_oom += 1; }
                        __syncthreads();
                    }
                    // time decomposition (paper Section 4.3): cycles spent on this failure go to the
                    // migration bucket if it migrated, to the OOM-retry bucket otherwise
                    if (tid == 0) {
                        const unsigned long long dt = (unsigned long long)(clock64() - sc.t_fail);
                        if (sc.migs_done != migs_before) sc.cyc_mig += dt; else sc.cyc_oom += dt;
                    }
                    c2 = f + 1;
                }
                if (sc.abort) break;
            }
            cur = end;
        }
        // ---- statuses of this window ----
        const uint32_t limit = sc.abort ? sc.abort_idx : wn;
        const bool decided = tid < (int)limit;
        if (decided) status[w0 + tid] = st;
        const int n_inv = __syncthreads_count(decided && st >= AVMP_ST_BAD_REQ && st != ST_PENDING);
        if (tid == 0) sc.n_invalid += n_inv;
        __syncthreads();
        if (sc.abort) { done_upto = w0 + sc.abort_idx; break; }
    }

    if (tid == 0) {
        ds->last_rebalance_op = sc.last; ds->n_oom = sc.n_oom; ds->n_capacity_error = sc.n_ce;
        ds->n_rebalance = sc.n_reb; ds->migrated_bytes = sc.migrated; ds->wasted_bytes = sc.wasted;
        ds->relocated_blocks = sc.reloc_blocks; ds->relocated_bytes = sc.reloc_bytes;
        ds->gap_bytes = sc.gap; ds->n_invalid = sc.n_invalid;
        ds->op_counter = sc.counter_base + (done_upto - start);
        for (int p = 0; p < 2; ++p) { ds->cap[p] = sc.cap[p]; ds->n_free[p] = sc.nfree[p]; ds->n_vfree[p] = sc.nvfree[p]; }
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
