// Bandwidth kernels of the AVMP path: handle translation, the relocation copy of a
// migration (paper Section 3.2; the paper's prototype copies nothing, this build keeps one
// arena and really moves live units), and the paged KV / contiguous SSM gathers and their
// write sides (Section 2.2).  No arithmetic on payload: bytes in, bytes out.
//
// All of them are HBM-bound streaming copies built on one skeleton.  The work of a launch
// is a list of "pieces": contiguous byte runs of at most kStage bytes with a source and a
// destination, enumerated by a small functor (SSM block chunks, page slices of a KV chain,
// chunks of a relocated unit).  A persistent grid walks the piece list grid-strided at warp
// granularity: at any moment the pieces in flight form one dense window of the list that
// slides forward, which keeps the traffic spread evenly over the HBM channels (giving every
// CTA its own contiguous range instead left 148 streams marching in lockstep at a fixed
// stride and cost about 10 % of the bandwidth on this part).
//
//   * bulk path (the one real shapes take): each warp runs its own ring of kStages shared
//     memory buffers.  One lane issues 1-D bulk async copies global -> shared (completion
//     on an mbarrier) and shared -> global (bulk groups); no data passes through registers
//     and the bytes in flight per SM are fixed by the ring (warps x stages x kStage), not
//     by the compiler's scheduling.  Every wait is bounded: a warp that gives up records
//     AVMP_DEV_TIMEOUT and stops issuing.
//   * generic path: plain loads and stores, for shapes whose runs are not 16-byte multiples.
//
// Shape of the ring, measured on B200 (244 MB to 51 GB per launch): what matters most is the number of bytes
// in flight per SM.  64 KiB (2 warps x 2 stages x 16 KiB, or 1 x 2 x 32 KiB) is the optimum -- a 28-layer SSM
// gather runs at 6.5 TB/s, the measured copy peak of this part, against 6.1 TB/s with 192 KiB in flight
// (4 x 3 x 16 KiB), 6.2 with 96 or 128 KiB and 6.1 with 48 KiB; at equal bytes, fewer and larger requests
// do slightly better, stages that are not a power of two much worse.  Other things tried that did not beat it:
// register-staged 16-byte loads / stores at 2-8 CTAs per SM, a global ticket counter instead of the static
// walk, staggered warp starts, smaller pieces for small launches (those are bound by ramp and tail latency,
// not by imbalance).
// The CTA nevertheless REQUESTS 120 KiB of shared memory, so that only one copy CTA fits on an SM: every
// kernel here lets its successor in the stream start early (programmatic dependent launch), and with small
// CTAs the successors' CTAs were placed two and three to an SM while this kernel still ran, which cost the
// back-to-back steps of a serving loop 5 % (25 % with 48 KiB CTAs) through the uneven load on the SMs.
#include "avmp_dev.cuh"

namespace avmp {

namespace {

// Shape of the bulk path (fixed after sweeps on B200; see the measured alternatives above).
constexpr int kStages = 2;                      // ring depth per warp
constexpr int kBulkWarps = 2;                   // warps (rings) per CTA: 2 x 2 x 16 KiB = 64 KiB in flight per SM
constexpr int kBulkCtasPerSm = 1;                // resident CTAs per SM the kernel is compiled for
constexpr int kBulkGridPerSm = 1;                // CTAs launched per SM
constexpr int kBulkThreads = kBulkWarps * 32;
constexpr uint32_t kBulkSmemUsed = kBulkWarps * kStages * kStage;
constexpr uint32_t kBulkSmemPad = 56 * 1024;     // requested on top, unused: one copy CTA per SM (see above)
constexpr uint32_t kBulkSmem = kBulkSmemUsed + kBulkSmemPad;
constexpr int kGenThreads = 256;
constexpr int kGenCtasPerSm = 4;
constexpr uint32_t kSpinLimit = 1u << 22;

struct Piece {
    const uint8_t *src;
    uint8_t *dst;
    uint32_t bytes;      // 0: nothing to do for this piece id
};

// ------------------------------- piece enumerators ------------------------------------
// a12: SSM block <-> (state row, conv row) of the batch buffers, for n_layers consecutive
// layers (layer-major piece order; layer l's buffers start l * stride bytes further on).
template <bool SCATTER>
struct SsmPieces {
    static constexpr bool kTimed = false;
    static constexpr bool kPlans = false;
    static constexpr bool kTail = false;
    uint32_t layer0, n_layers, n, ps, per;
    const uint32_t *reqs;
    uint8_t *buf_state, *buf_conv;
    unsigned long long state_stride, conv_stride;
    __device__ unsigned long long total(const Geom &) const { return (unsigned long long)n_layers * n * per; }
    __device__ Piece get(const Geom &g, unsigned long long it) const
    {
        const unsigned long long per_layer = (unsigned long long)n * per;
        const uint32_t dl = (uint32_t)(it / per_layer);
        const uint32_t rem = (uint32_t)(it % per_layer);
        const uint32_t k = rem / per, c = rem % per;
        const unsigned long long keep = l2_policy_evict_last();
        const uint32_t r = ld_keep(reqs + k, keep);
        uint32_t slot = kInvalid;
        if (r < g.R) {
            // state and handle are read together: one round trip less on the way to the first copy
            const uint32_t state = ld_keep(g.r_state + r, keep);
            const uint32_t h = ld_keep(g.r_ssm + ((unsigned long long)r * g.ns + layer0 + dl), keep);
            if (state == AVMP_REQ_LIVE && h != kInvalid) slot = ld_keep(g.VT[1] + (h & 0x7FFFFFFFu), keep);
        }
        if (slot == kInvalid) {
            if (c == 0) record_error(g.st, AVMP_DEV_BAD_REQUEST);
            return Piece{nullptr, nullptr, 0};
        }
        uint8_t *blk = unit_ptr(g, AVMP_POOL_SSM, slot);
        uint8_t *p, *b;
        uint32_t bytes;
        if (c < ps) {
            const unsigned long long o = (unsigned long long)c * kStage;
            p = blk + o; b = buf_state + dl * state_stride + (unsigned long long)k * g.state_bytes + o;
            bytes = (uint32_t)min((unsigned long long)kStage, g.state_bytes - o);
        } else {
            const unsigned long long o = (unsigned long long)(c - ps) * kStage;
            p = blk + g.state_bytes + o; b = buf_conv + dl * conv_stride + (unsigned long long)k * g.conv_bytes + o;
            bytes = (uint32_t)min((unsigned long long)kStage, g.conv_bytes - o);
        }
        return SCATTER ? Piece{b, p, bytes} : Piece{p, b, bytes};
    }
};

// a7: chunks of the units moved by the last migration.
struct RelocPieces {
    static constexpr bool kTimed = true;     // the copy stamps the device clock: migration time is a metric
    static constexpr bool kPlans = false;
    static constexpr bool kTail = false;
    __device__ unsigned long long total(const Geom &g) const
    {
        const unsigned long long U = g.U[g.st->reloc_pool];
        return (unsigned long long)g.st->n_reloc * ((U + kStage - 1) / kStage);
    }
    __device__ Piece get(const Geom &g, unsigned long long it) const
    {
        const uint32_t pool = g.st->reloc_pool;
        const unsigned long long U = g.U[pool];
        const uint32_t per = (uint32_t)((U + kStage - 1) / kStage);
        const uint32_t k = (uint32_t)(it / per), c = (uint32_t)(it % per);
        const unsigned long long o = (unsigned long long)c * kStage;
        // dst < new capacity <= src: the two units never overlap
        return Piece{unit_ptr(g, pool, g.reloc_src[k]) + o, unit_ptr(g, pool, g.reloc_dst[k]) + o,
                     (uint32_t)min((unsigned long long)kStage, U - o)};
    }
};

// a10 for one handle: pool tag, offset inside that store, offset inside the arena.
__device__ __forceinline__ void translate_store(const Geom &g, uint32_t hv, uint32_t slot, uint32_t i, uint32_t *pool,
                                                unsigned long long *off, unsigned long long *aoff)
{
    if (slot == kInvalid) {
        pool[i] = kInvalid; off[i] = kNone64;
        if (aoff) aoff[i] = kNone64;
        record_error(g.st, AVMP_DEV_BAD_HANDLE);
    } else {
        const uint32_t p = hv >> 31;
        pool[i] = p; off[i] = (unsigned long long)slot * g.U[p];
        if (aoff) aoff[i] = (unsigned long long)(unit_ptr(g, p, slot) - g.arena);
    }
}
__device__ __forceinline__ void translate_one(const Geom &g, uint32_t hv, uint32_t i, uint32_t *pool,
                                              unsigned long long *off, unsigned long long *aoff)
{
    const uint32_t p = hv >> 31, vid = hv & 0x7FFFFFFFu;
    const uint32_t slot = (hv != kInvalid && vid < g.V[p]) ? g.VT[p][vid] : kInvalid;
    translate_store(g, hv, slot, i, pool, off, aoff);
}

// a7 + a10 in one launch: the relocation copy of a step, and the translation of a handle list against the
// tables that step left (the page table is remapped by the step kernel itself, so the look-ups do not
// depend on the copy).  Saves the third launch of an engine step's allocator part.
struct RelocTranslate : RelocPieces {
    static constexpr bool kTail = true;
    const uint32_t *h;
    uint32_t n;
    uint32_t *pool;
    unsigned long long *off, *aoff;
    __device__ void tail(const Geom &g) const
    {
        // eight handles per thread and round, their look-ups in flight together: the copy grid is small
        // (one narrow CTA per SM), so a long list would otherwise pay two dependent reads per handle in series
        constexpr int kPer = 8;
        const uint32_t stride = gridDim.x * blockDim.x;
        for (uint32_t base = blockIdx.x * blockDim.x + threadIdx.x; base < n; base += stride * kPer) {
            uint32_t hv[kPer], slot[kPer];
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const unsigned long long i = (unsigned long long)base + (unsigned long long)j * stride;
                hv[j] = i < n ? h[i] : kInvalid;
            }
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const uint32_t p = hv[j] >> 31, vid = hv[j] & 0x7FFFFFFFu;
                slot[j] = (hv[j] != kInvalid && vid < g.V[p]) ? g.VT[p][vid] : kInvalid;
            }
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const unsigned long long i = (unsigned long long)base + (unsigned long long)j * stride;
                if (i < n) translate_store(g, hv[j], slot[j], (uint32_t)i, pool, off, aoff);
            }
        }
    }
};

// a11: slices of the pages of a KV chain <-> rows of the ragged batch buffers.  A plan gives,
// per request k, the first row (cu_rows) and the first piece (cu_items); a request spanning P
// pages owns P * subs pieces, `subs` = slices per page (K slices, then V slices).  For request
// lists of up to kLocalPlanMax entries every CTA of the copy computes the plan itself into its
// shared memory (a few hundred table reads and a block scan: cheaper than a separate launch and
// its dependency, and calls on different streams share no scratch); longer lists use the plan
// kernel and the context's global scratch.
// One request's rows and pieces for a KV gather / scatter (errors recorded by the caller's choice).
__device__ __forceinline__ void kv_rows_items(const Geom &g, uint32_t st, uint32_t len, uint32_t t0, uint32_t subs,
                                              bool report, uint32_t &rows, uint32_t &items)
{
    rows = 0; items = 0;
    if (st == AVMP_REQ_EMPTY) { if (report) record_error(g.st, AVMP_DEV_BAD_REQUEST); }
    else if (t0 > len) { if (report) record_error(g.st, AVMP_DEV_BAD_REQUEST); }
    else rows = len - t0;
    if (rows) items = ((t0 + rows - 1u) / g.T - t0 / g.T + 1u) * subs;
}

__device__ __forceinline__ void kv_plan_entry(const Geom &g, const uint32_t *reqs, const uint32_t *tok_start,
                                              uint32_t k, uint32_t subs, bool report, uint32_t &rows, uint32_t &items)
{
    const uint32_t r = reqs[k];
    const bool in_range = r < g.R;
    kv_rows_items(g, in_range ? g.r_state[r] : (uint32_t)AVMP_REQ_EMPTY, in_range ? g.r_len[r] : 0u,
                  tok_start ? tok_start[k] : 0u, subs, report, rows, items);
}

constexpr uint32_t kPlanWords = 3 * (kLocalPlanMax + 1);   // shared words a local plan needs: rows, items, slots

template <bool SCATTER>
struct KvPieces {
    static constexpr bool kTimed = false;
    static constexpr bool kPlans = true;
    static constexpr bool kTail = false;
    uint32_t layer0, n_layers, n, subs;
    const uint32_t *reqs, *tok_start;
    uint8_t *buf_k, *buf_v;
    unsigned long long cap_tokens, layer_stride;
    uint32_t *cu_out;                     // cu_seqlens for the caller (local plan only; may be null)
    const uint32_t *cu_items, *cu_rows;   // set by plan(): shared memory, or the context's scratch
    const uint32_t *req_of;               // set by plan(): the list's slots (shared copy, or the caller's array)
    // Whole CTA.  `buf` holds kPlanWords words, `tmp` 32 scan words.
    __device__ void plan(const Geom &g, uint32_t *buf, unsigned long long *tmp)
    {
        if (n > kLocalPlanMax) { cu_items = g.g_cu_items; cu_rows = g.g_cu_rows; req_of = reqs; return; }
        uint32_t *rows_s = buf, *items_s = buf + kLocalPlanMax + 1, *req_s = buf + 2 * (kLocalPlanMax + 1);
        const bool lead = blockIdx.x == 0;            // one CTA reports errors and writes cu_seqlens
        // Every thread takes a run of consecutive entries: their rows and pieces (eight entries per round, so
        // that the two dependent table reads of a round are in flight together), summed on the way; ONE block
        // scan orders the runs; then each thread turns its own entries into exclusive prefix sums in place.
        constexpr int kPer = 8;
        const unsigned long long keep = l2_policy_evict_last();
        const uint32_t per = (n + blockDim.x - 1) / blockDim.x;
        const uint32_t k0 = min(n, threadIdx.x * per), k1 = min(n, k0 + per);
        unsigned long long mine = 0, tot;
        for (uint32_t kb = k0; kb < k1; kb += kPer) {
            uint32_t rr[kPer], t0[kPer], st[kPer], ln[kPer];
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                const uint32_t k = kb + i;
                rr[i] = k < k1 ? ld_keep(reqs + k, keep) : kInvalid;
                t0[i] = (k < k1 && tok_start) ? tok_start[k] : 0u;
            }
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                const bool in_range = rr[i] < g.R;
                st[i] = in_range ? ld_keep(g.r_state + rr[i], keep) : (uint32_t)AVMP_REQ_EMPTY;
                ln[i] = in_range ? ld_keep(g.r_len + rr[i], keep) : 0u;
            }
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                const uint32_t k = kb + i;
                if (k < k1) {
                    uint32_t rows, items;
                    kv_rows_items(g, st[i], ln[i], t0[i], subs, lead, rows, items);
                    rows_s[k] = rows; items_s[k] = items; req_s[k] = rr[i];
                    mine += ((unsigned long long)items << 32) | rows;
                }
            }
        }
        const unsigned long long incl = block_incl_scan(mine, tmp, &tot);
        unsigned long long run = incl - mine;
        for (uint32_t k = k0; k < k1; ++k) {
            const unsigned long long v = ((unsigned long long)items_s[k] << 32) | rows_s[k];
            rows_s[k] = (uint32_t)run;
            items_s[k] = (uint32_t)(run >> 32);
            if (lead && cu_out) cu_out[k] = (uint32_t)run;
            run += v;
        }
        if (threadIdx.x == 0) {
            rows_s[n] = (uint32_t)tot; items_s[n] = (uint32_t)(tot >> 32);
            if (lead && cu_out) cu_out[n] = (uint32_t)tot;
        }
        __syncthreads();
        cu_items = items_s; cu_rows = rows_s; req_of = req_s;
    }
    __device__ unsigned long long total(const Geom &) const { return (unsigned long long)n_layers * cu_items[n]; }
    __device__ Piece get(const Geom &g, unsigned long long it64) const
    {
        const uint32_t per_layer = cu_items[n];
        const uint32_t dl = (uint32_t)(it64 / per_layer);
        const uint32_t it = (uint32_t)(it64 % per_layer);
        const uint32_t k = find_owner(cu_items, 0u, n, 0u, it);
        const uint32_t rel = it - cu_items[k];
        const uint32_t row0 = cu_rows[k], rows = cu_rows[k + 1] - row0;
        if (!SCATTER && (unsigned long long)row0 + rows > cap_tokens) {
            if (rel == 0 && dl == 0) record_error(g.st, AVMP_DEV_OUT_OVERFLOW);
            return Piece{nullptr, nullptr, 0};
        }
        const uint32_t T = g.T, row = (uint32_t)g.row_bytes, half = subs >> 1;
        const uint32_t t0 = tok_start ? tok_start[k] : 0u;
        const uint32_t page = t0 / T + rel / subs, sub = rel % subs;
        const uint32_t part = sub / half, q = sub % half;
        // tokens of this page that belong to the copy, as a byte range of the page's K (or V) part
        const uint32_t lo_t = max(t0, page * T), hi_t = min(t0 + rows, (page + 1u) * T);
        const uint32_t b_lo = max((lo_t - page * T) * row, q * kStage);
        const uint32_t b_hi = min((hi_t - page * T) * row, (q + 1u) * kStage);
        if (b_lo >= b_hi) return Piece{nullptr, nullptr, 0};
        const uint32_t r = req_of[k];
        const unsigned long long keep = l2_policy_evict_last();
        const uint32_t h = ld_keep(g.r_chain + ((unsigned long long)r * g.max_pages + page), keep);
        const uint32_t slot = ld_keep(g.VT[0] + (h & 0x7FFFFFFFu), keep);
        uint8_t *p = g.arena + (unsigned long long)slot * g.U[0] + (unsigned long long)(layer0 + dl) * g.kv_layer_bytes +
                     (unsigned long long)part * T * row + b_lo;
        // byte b of the page part is byte (b - (t0 - page*T)*row) of the request's rows
        uint8_t *b = (part ? buf_v : buf_k) + dl * layer_stride +
                     ((unsigned long long)row0 * row + (unsigned long long)page * T * row + b_lo -
                      (unsigned long long)t0 * row);
        return SCATTER ? Piece{b, p, b_hi - b_lo} : Piece{p, b, b_hi - b_lo};
    }
};

// a11 + a12 in one launch: the KV pieces of a range of attention layers, then the SSM pieces of a
// range of SSM layers, for one request list.  A step that moves little (a few dozen requests) is
// bound by the ramp and the tail of its launches; one launch pays them once.
struct StepPieces {
    static constexpr bool kTimed = false;
    static constexpr bool kPlans = true;
    static constexpr bool kTail = false;
    KvPieces<false> kv;
    SsmPieces<false> ssm;
    __device__ void plan(const Geom &g, uint32_t *buf, unsigned long long *tmp) { kv.plan(g, buf, tmp); }
    __device__ unsigned long long total(const Geom &g) const { return kv.total(g) + ssm.total(g); }
    __device__ Piece get(const Geom &g, unsigned long long it) const
    {
        const unsigned long long nkv = kv.total(g);
        return it < nkv ? kv.get(g, it) : ssm.get(g, it - nkv);
    }
};

// ------------------------------- bulk-copy primitives ----------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Both directions carry an L2 evict-first hint: the bytes stream through once, and keeping them
// from displacing each other's lines was worth 2-5 % on this part (measured against the unhinted
// forms: without the load hint the benchmark step loses 1.7 %, without the store hint 0.5 %,
// single-layer launches 3-4 % each).
__device__ __forceinline__ unsigned long long l2_policy_evict_first()
{
    unsigned long long p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar,
                                         unsigned long long pol)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 :: "r"(dst_smem), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
__device__ __forceinline__ void bulk_s2g(void *dst, uint32_t src_smem, uint32_t bytes, unsigned long long pol)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                 :: "l"(dst), "r"(src_smem), "r"(bytes), "l"(pol) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" :: "n"(N) : "memory");
}
// wait until at most `younger` of the most recent bulk groups still read shared memory
__device__ __forceinline__ void wait_stage_free(uint32_t younger)
{
    static_assert(kStages <= 8, "extend the switch");
    switch (younger) {
    case 0: bulk_wait_read<0>(); break;
    case 1: bulk_wait_read<1>(); break;
    case 2: bulk_wait_read<2>(); break;
    case 3: bulk_wait_read<3>(); break;
    case 4: bulk_wait_read<4>(); break;
    case 5: bulk_wait_read<5>(); break;
    case 6: bulk_wait_read<6>(); break;
    default: bulk_wait_read<7>(); break;
    }
}
__device__ __forceinline__ void bulk_wait_all()
{
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// ------------------------------- the two skeletons --------------------------------------
// Lane 0 of every warp drives the warp's ring; lanes 1..31 look up the next 31 pieces in
// parallel (a lookup is a chain of three or four dependent table reads, far too slow to
// sit on the issuing lane's path) and hand them over through shared memory, one batch ahead.
struct Ring {
    uint32_t buf0, bar0;
    uint32_t n_loaded, n_stored;     // pieces issued as loads / as stores so far
    uint8_t *dst[kStages];
    uint32_t bytes[kStages];
    unsigned long long policy;       // L2 cache hint for both directions
    bool failed;

    // wait for the oldest load, then send its stage on its way to global memory
    __device__ __forceinline__ void retire_one()
    {
        const uint32_t s = n_stored % kStages, parity = (n_stored / kStages) & 1u;
        uint32_t spins = 0;
        while (!mbar_try_wait(bar0 + 8u * s, parity))
            if (++spins > kSpinLimit) { failed = true; return; }
        bulk_s2g(dst[s], buf0 + s * kStage, bytes[s], policy);
        ++n_stored;
    }
    // After a timeout: no new copies, but loads already issued still target this CTA's shared
    // memory.  Give each of them one more bounded wait (nothing is stored) before the CTA may exit.
    __device__ __forceinline__ void drain_loads()
    {
        for (uint32_t i = n_stored; i < n_loaded; ++i) {
            const uint32_t s = i % kStages, parity = (i / kStages) & 1u;
            uint32_t spins = 0;
            while (!mbar_try_wait(bar0 + 8u * s, parity))
                if (++spins > kSpinLimit) break;
        }
    }
    __device__ __forceinline__ void push(const Piece &p)
    {
        if (n_loaded - n_stored == (uint32_t)kStages) retire_one();
        if (failed) return;
        const uint32_t s = n_loaded % kStages;
        // the stage's previous occupant was piece n_loaded - kStages; its store (one bulk group per
        // piece, in order) must have finished reading the buffer.  Only younger groups may pend.
        if (n_loaded >= (uint32_t)kStages) wait_stage_free(n_stored - 1u - (n_loaded - (uint32_t)kStages));
        dst[s] = p.dst;
        bytes[s] = p.bytes;
        mbar_expect_tx(bar0 + 8u * s, p.bytes);
        bulk_g2s(buf0 + s * kStage, p.src, p.bytes, bar0 + 8u * s, policy);
        ++n_loaded;
    }
};

constexpr int kBatch = 31;   // pieces looked up per hand-over (lanes 1..31)

template <class F>
__global__ void __launch_bounds__(kBulkThreads, kBulkCtasPerSm) stream_bulk_kernel(const Geom g, const F f_in)
{
    extern __shared__ __align__(1024) uint8_t ring_mem[];
    __shared__ __align__(8) unsigned long long bars[kBulkWarps * kStages];
    __shared__ Piece handover[kBulkWarps][2][kBatch];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0)
        for (int s = 0; s < kStages; ++s) mbar_init(smem_u32(&bars[warp * kStages + s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    pdl_prologue();
    __syncthreads();
    F f = f_in;
    if constexpr (F::kTail) f.tail(g);
    if constexpr (F::kPlans) {
        __shared__ uint32_t plan_buf[kPlanWords];
        __shared__ unsigned long long plan_tmp[32];
        f.plan(g, plan_buf, plan_tmp);
    }
    const unsigned long long total = f.total(g);

    // warp w of CTA c takes pieces (w * grid + c) + j * (grid * warps), j = 0, 1, ...: at any moment
    // the pieces in flight across the grid form one dense window of the list
    const unsigned long long first = (unsigned long long)warp * gridDim.x + blockIdx.x;
    const unsigned long long stride = (unsigned long long)gridDim.x * kBulkWarps;
    if (first >= total) return;
    if (F::kTimed && lane == 0) atomicMin(&g.st->reloc_t0, global_ns());
    const unsigned long long mine = (total - first + stride - 1) / stride;       // pieces of this warp
    const uint32_t n_batches = (uint32_t)((mine + kBatch - 1) / kBatch);

    Ring ring;
    ring.buf0 = smem_u32(ring_mem) + (uint32_t)warp * kStages * kStage;
    ring.bar0 = smem_u32(&bars[warp * kStages]);
    ring.n_loaded = ring.n_stored = 0;
    ring.failed = false;
    ring.policy = l2_policy_evict_first();

    auto lookup = [&](uint32_t batch) {            // lanes 1..31
        const unsigned long long j = (unsigned long long)batch * kBatch + (lane - 1);
        Piece p{nullptr, nullptr, 0};
        if (j < mine) p = f.get(g, first + j * stride);
        handover[warp][batch & 1][lane - 1] = p;
    };
    if (lane != 0) lookup(0);
    __syncwarp();
    for (uint32_t b = 0; b < n_batches; ++b) {
        if (lane != 0) {
            if (b + 1 < n_batches) lookup(b + 1);
        } else {
            const unsigned long long left = mine - (unsigned long long)b * kBatch;
            const int cnt = left < (unsigned long long)kBatch ? (int)left : kBatch;
            for (int i = 0; i < cnt && !ring.failed; ++i) {
                const Piece p = handover[warp][b & 1][i];
                if (p.bytes) ring.push(p);
            }
        }
        __syncwarp();
    }
    if (lane == 0) {
        while (!ring.failed && ring.n_stored < ring.n_loaded) ring.retire_one();
        if (ring.failed) {
            record_error(g.st, AVMP_DEV_TIMEOUT);
            ring.drain_loads();
        }
        // Before the CTA may exit, the stores must have read their shared-memory stages; that they have
        // reached global memory is guaranteed by the end of the kernel.  The timed copy waits for that too,
        // so that its clock stamp covers the whole transfer.
        if (F::kTimed) {
            bulk_wait_all();
            atomicMax(&g.st->reloc_t1, global_ns());
        } else {
            bulk_wait_read<0>();
        }
    }
}

template <class F>
__global__ void __launch_bounds__(kGenThreads) stream_generic_kernel(const Geom g, const F f_in)
{
    const int lane = threadIdx.x & 31;
    pdl_prologue();
    F f = f_in;
    if constexpr (F::kTail) f.tail(g);
    if constexpr (F::kPlans) {
        __shared__ uint32_t plan_buf[kPlanWords];
        __shared__ unsigned long long plan_tmp[32];
        f.plan(g, plan_buf, plan_tmp);
    }
    const unsigned long long total = f.total(g);
    const unsigned long long nw = (unsigned long long)gridDim.x * (kGenThreads / 32);
    const unsigned long long it0 = (unsigned long long)(threadIdx.x >> 5) * gridDim.x + blockIdx.x;
    if (F::kTimed && lane == 0 && it0 < total) atomicMin(&g.st->reloc_t0, global_ns());
    for (unsigned long long it = it0; it < total; it += nw) {
        Piece p{nullptr, nullptr, 0};
        if (lane == 0) p = f.get(g, it);
        p.src = (const uint8_t *)__shfl_sync(0xFFFFFFFFu, (unsigned long long)p.src, 0);
        p.dst = (uint8_t *)__shfl_sync(0xFFFFFFFFu, (unsigned long long)p.dst, 0);
        p.bytes = __shfl_sync(0xFFFFFFFFu, p.bytes, 0);
        if ((((uintptr_t)p.dst | (uintptr_t)p.src | p.bytes) & 15u) == 0) {
            const uint4 *s = reinterpret_cast<const uint4 *>(p.src);
            uint4 *d = reinterpret_cast<uint4 *>(p.dst);
            for (uint32_t i = lane; i < (p.bytes >> 4); i += 32u) d[i] = s[i];
        } else {
            for (uint32_t i = lane; i < p.bytes; i += 32u) p.dst[i] = p.src[i];
        }
    }
    if (F::kTimed && lane == 0 && it0 < total) { __threadfence(); atomicMax(&g.st->reloc_t1, global_ns()); }
}

template <class F>
cudaError_t launch_stream(const Geom &g, const F &f, bool bulk_ok, const Launch &l)
{
    if (bulk_ok) {
        static bool attr_set[64] = {};   // per kernel instantiation and device
        if (!attr_set[l.device & 63]) {
            cudaError_t e = cudaFuncSetAttribute(stream_bulk_kernel<F>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBulkSmem);
            if (e != cudaSuccess) return e;
            attr_set[l.device & 63] = true;
        }
        return launch_pdl(stream_bulk_kernel<F>, dim3(l.n_sms * kBulkGridPerSm), dim3(kBulkThreads), kBulkSmem, l.stream, g, f);
    }
    return launch_pdl(stream_generic_kernel<F>, dim3(l.n_sms * kGenCtasPerSm), dim3(kGenThreads), 0, l.stream, g, f);
}

inline bool mult16(unsigned long long x) { return (x & 15ull) == 0; }

// ---- a10: translate ------------------------------------------------------------------
__global__ void translate_kernel(const Geom g, const uint32_t *h, uint32_t n,
                                 uint32_t *pool, unsigned long long *off,
                                 unsigned long long *aoff)
{
    pdl_prologue();
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x)
        translate_one(g, h[i], i, pool, off, aoff);
}

// ---- a11 plan: request list -> row prefix sums (cu_seqlens) and piece prefix sums --------
__global__ void __launch_bounds__(kStepThreads)
kv_plan_kernel(const Geom g, const uint32_t *reqs, const uint32_t *tok_start,
               uint32_t n, uint32_t subs, uint32_t *cu_out)
{
    __shared__ unsigned long long tmp[32];
    unsigned long long run_rows = 0, run_items = 0, tot;
    const int tid = threadIdx.x;
    pdl_prologue();
    for (uint32_t b = 0; b < n; b += kStepThreads) {
        const uint32_t k = b + tid;
        uint32_t rows = 0, items = 0;
        if (k < n) kv_plan_entry(g, reqs, tok_start, k, subs, true, rows, items);
        const unsigned long long incl = block_incl_scan(((unsigned long long)items << 32) | rows, tmp, &tot);
        if (k < n) {
            const uint32_t ex_rows = (uint32_t)(run_rows + (uint32_t)incl - rows);
            const uint32_t ex_items = (uint32_t)(run_items + (uint32_t)(incl >> 32) - items);
            g.g_cu_rows[k] = ex_rows;
            g.g_cu_items[k] = ex_items;
            if (cu_out) cu_out[k] = ex_rows;
        }
        run_rows += (uint32_t)tot;
        run_items += (uint32_t)(tot >> 32);
    }
    if (tid == 0) {
        g.g_cu_rows[n] = (uint32_t)run_rows;
        g.g_cu_items[n] = (uint32_t)run_items;
        if (cu_out) cu_out[n] = (uint32_t)run_rows;
        g.st->g_total_items = (uint32_t)run_items;
    }
}

}  // namespace

cudaError_t launch_relocate(const Geom &g, const Launch &l)
{
    return launch_stream(g, RelocPieces{}, mult16(g.U[0]) && mult16(g.U[1]) && mult16(g.P_al), l);
}

cudaError_t launch_relocate_translate(const Geom &g, const uint32_t *h, uint32_t n, uint32_t *pool,
                                      unsigned long long *off, unsigned long long *aoff, const Launch &l)
{
    RelocTranslate f;
    f.h = h; f.n = n; f.pool = pool; f.off = off; f.aoff = aoff;
    return launch_stream(g, f, mult16(g.U[0]) && mult16(g.U[1]) && mult16(g.P_al), l);
}

cudaError_t launch_translate(const Geom &g, const uint32_t *h, uint32_t n, uint32_t *pool,
                             unsigned long long *off, unsigned long long *aoff, const Launch &l)
{
    const int blocks = (int)min((unsigned long long)l.n_sms * 4, ((unsigned long long)n + 255) / 256);
    return launch_pdl(translate_kernel, dim3(blocks), dim3(256), 0, l.stream, g, h, n, pool, off, aoff);
}

cudaError_t launch_kv(const Geom &g, bool scatter, uint32_t layer0, uint32_t n_layers, const uint32_t *reqs,
                      const uint32_t *tok_start, uint32_t n, void *k, void *v, unsigned long long layer_stride,
                      unsigned long long cap_tokens, uint32_t *cu_out, const Launch &l)
{
    const unsigned long long part = (unsigned long long)g.T * g.row_bytes;     // K (or V) bytes of a page
    const uint32_t subs = 2u * (uint32_t)((part + kStage - 1) / kStage);
    if (n > kLocalPlanMax) {      // long request lists: plan once, into the context's scratch
        cudaError_t e = launch_pdl(kv_plan_kernel, dim3(1), dim3(kStepThreads), 0, l.stream, g, reqs, tok_start, n, subs, cu_out);
        if (e != cudaSuccess) return e;
    }
    const bool bulk_ok = mult16(g.row_bytes) && mult16(g.U[0]) && mult16(g.kv_layer_bytes) && mult16(layer_stride);
    if (scatter)
        return launch_stream(g, KvPieces<true>{layer0, n_layers, n, subs, reqs, tok_start, (uint8_t *)k, (uint8_t *)v, cap_tokens, layer_stride, cu_out, nullptr, nullptr, nullptr}, bulk_ok, l);
    return launch_stream(g, KvPieces<false>{layer0, n_layers, n, subs, reqs, tok_start, (uint8_t *)k, (uint8_t *)v, cap_tokens, layer_stride, cu_out, nullptr, nullptr, nullptr}, bulk_ok, l);
}

cudaError_t launch_step_gather(const Geom &g, const uint32_t *reqs, uint32_t n, uint32_t kv_layer0, uint32_t kv_layers,
                               void *k, void *v, unsigned long long kv_layer_stride, unsigned long long cap_tokens,
                               uint32_t *cu_out, uint32_t ssm_layer0, uint32_t ssm_layers, void *state,
                               unsigned long long state_stride, void *conv, unsigned long long conv_stride, const Launch &l)
{
    const unsigned long long part = (unsigned long long)g.T * g.row_bytes;
    const uint32_t subs = 2u * (uint32_t)((part + kStage - 1) / kStage);
    if (n > kLocalPlanMax) {
        cudaError_t e = launch_pdl(kv_plan_kernel, dim3(1), dim3(kStepThreads), 0, l.stream, g, reqs, (const uint32_t *)nullptr, n, subs, cu_out);
        if (e != cudaSuccess) return e;
    }
    const uint32_t ps = (uint32_t)((g.state_bytes + kStage - 1) / kStage), pc = (uint32_t)((g.conv_bytes + kStage - 1) / kStage);
    const bool bulk_ok = mult16(g.row_bytes) && mult16(g.U[0]) && mult16(g.kv_layer_bytes) && mult16(kv_layer_stride) &&
                         mult16(g.state_bytes) && mult16(g.conv_bytes) && mult16(g.U[1]) && mult16(g.P_al) &&
                         mult16(state_stride) && mult16(conv_stride);
    StepPieces f{KvPieces<false>{kv_layer0, kv_layers, n, subs, reqs, nullptr, (uint8_t *)k, (uint8_t *)v, cap_tokens,
                                 kv_layer_stride, cu_out, nullptr, nullptr, nullptr},
                 SsmPieces<false>{ssm_layer0, ssm_layers, n, ps, ps + pc, reqs, (uint8_t *)state, (uint8_t *)conv,
                                  state_stride, conv_stride}};
    return launch_stream(g, f, bulk_ok, l);
}

cudaError_t launch_ssm(const Geom &g, bool scatter, uint32_t layer0, uint32_t n_layers, const uint32_t *reqs, uint32_t n,
                       void *state, unsigned long long state_stride, void *conv, unsigned long long conv_stride,
                       const Launch &l)
{
    const uint32_t ps = (uint32_t)((g.state_bytes + kStage - 1) / kStage), pc = (uint32_t)((g.conv_bytes + kStage - 1) / kStage);
    const bool bulk_ok = mult16(g.state_bytes) && mult16(g.conv_bytes) && mult16(g.U[1]) && mult16(g.P_al) &&
                         mult16(state_stride) && mult16(conv_stride);
    if (scatter)
        return launch_stream(g, SsmPieces<true>{layer0, n_layers, n, ps, ps + pc, reqs, (uint8_t *)state, (uint8_t *)conv, state_stride, conv_stride}, bulk_ok, l);
    return launch_stream(g, SsmPieces<false>{layer0, n_layers, n, ps, ps + pc, reqs, (uint8_t *)state, (uint8_t *)conv, state_stride, conv_stride}, bulk_ok, l);
}

}  // namespace avmp
