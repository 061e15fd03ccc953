// Host side of the C ABI: argument checks, the Section 3.1 layout arithmetic, workspace
// carving, launch sequencing.  No device memory is allocated here; the context is a small
// host struct over the caller's arena and workspace.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "avmp_dev.cuh"

using namespace avmp;


namespace {

constexpr size_t kAlign = 256;
inline size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Carve {
    size_t off = 0;
    size_t take(size_t bytes) { size_t o = off; off += up(bytes ? bytes : 1); return o; }
};

// Offsets of every table inside the workspace, in one place so that size and carving agree.
struct WsLayout {
    size_t state, S[2], W[2], VT[2], OW[2], r_state, r_len, r_npages, r_chain, r_ssm;
    size_t reloc_src, reloc_dst, g_cu_items, g_cu_rows, stage_ops, stage_status, total;
};

WsLayout ws_layout(const avmp_layout &lay, const avmp_model_spec &spec, const avmp_options &opt)
{
    WsLayout w;
    Carve c;
    w.state = c.take(sizeof(DevState));
    for (int p = 0; p < 2; ++p) {
        const size_t v = (size_t)lay.vid_space[p] * 4;
        w.S[p] = c.take(v); w.W[p] = c.take(v); w.VT[p] = c.take(v); w.OW[p] = c.take(v);
    }
    const size_t R = opt.max_requests;
    w.r_state = c.take(R * 4); w.r_len = c.take(R * 4); w.r_npages = c.take(R * 4);
    w.r_chain = c.take(R * (size_t)opt.max_pages_per_request * 4);
    w.r_ssm = c.take(R * (size_t)spec.n_ssm_layers * 4);
    const size_t maxv = (size_t)(lay.vid_space[0] > lay.vid_space[1] ? lay.vid_space[0] : lay.vid_space[1]);
    w.reloc_src = c.take(maxv * 4); w.reloc_dst = c.take(maxv * 4);
    w.g_cu_items = c.take((R + 1) * 4); w.g_cu_rows = c.take((R + 1) * 4);
    w.stage_ops = c.take((size_t)kHostStepMaxOps * sizeof(avmp_op));
    w.stage_status = c.take((size_t)kHostStepMaxOps * 4);
    w.total = c.off;
    return w;
}

bool options_ok(const avmp_options &o)
{
    return o.threshold_low_ppm < o.threshold_high_ppm && o.threshold_high_ppm <= 1000000u &&
           o.min_rebalance_interval_ops >= 1 && o.max_requests >= 1 && o.max_pages_per_request >= 1 &&
           (uint64_t)o.max_requests * o.max_pages_per_request < (1ull << 32);
}

inline cudaStream_t S(void *s) { return reinterpret_cast<cudaStream_t>(s); }
inline Launch L(const avmp_ctx *c, void *s) { return Launch{S(s), c->n_sms, c->device}; }
inline int cu(cudaError_t e) { return e == cudaSuccess ? AVMP_OK : AVMP_ECUDA; }

void fill_stats(const avmp_ctx *c, const DevState &d, avmp_stats *o)
{
    o->op_counter = d.op_counter; o->last_rebalance_op = d.last_rebalance_op; o->n_oom = d.n_oom;
    o->n_capacity_error = d.n_capacity_error; o->n_rebalance = d.n_rebalance;
    o->migrated_bytes = d.migrated_bytes; o->wasted_bytes = d.wasted_bytes;
    o->relocated_blocks = d.relocated_blocks; o->relocated_bytes = d.relocated_bytes;
    o->gap_bytes = d.gap_bytes;
    for (int p = 0; p < 2; ++p) {
        o->cap[p] = d.cap[p]; o->free_units[p] = d.n_free[p];
        o->unit_bytes[p] = c->lay.unit_bytes[p]; o->vid_space[p] = c->lay.vid_space[p];
    }
    o->fsm_state = d.fsm; o->n_invalid = d.n_invalid;
    o->pool_bytes_aligned = c->lay.pool_bytes_aligned;
    o->error_code = d.error_code; o->error_count = d.error_count;
    const uint64_t last = (d.reloc_t1 > d.reloc_t0 && d.reloc_t0 != kNone64) ? d.reloc_t1 - d.reloc_t0 : 0;
    o->relocation_ns_last = last;
    o->relocation_ns_total = d.reloc_ns_total + (d.reloc_pending ? last : 0);
    const double ns_per_cycle = c->sm_khz > 0 ? 1e6 / (double)c->sm_khz : 0.0;
    o->step_ns_total = (uint64_t)(d.cyc_total * ns_per_cycle);
    o->step_ns_oom_retry = (uint64_t)(d.cyc_oom * ns_per_cycle);
    o->step_ns_migration_plan = (uint64_t)(d.cyc_mig * ns_per_cycle);
}

// A snapshot is accepted only if the kernels could have produced it: they index the tables
// without bounds checks, so a table that does not hang together must never reach the device.
bool tables_consistent(const avmp_ctx *c, const avmp_tables *t)
{
    const Geom &g = c->g;
    const avmp_stats &st = t->stats;
    if (st.fsm_state > AVMP_FSM_REBALANCING) return false;
    if (st.last_rebalance_op != kNone64 && st.last_rebalance_op > st.op_counter) return false;
    unsigned __int128 bytes = st.gap_bytes;
    for (int p = 0; p < 2; ++p) {
        if (st.cap[p] > g.V[p]) return false;
        bytes += (unsigned __int128)st.cap[p] * g.U[p];
    }
    if (bytes != g.P_al) return false;                         // pool bytes are conserved
    uint64_t live[2] = {0, 0};
    std::vector<uint8_t> mark;
    for (int p = 0; p < 2; ++p) {
        const uint32_t V = g.V[p], cap = (uint32_t)st.cap[p], nf = t->n_slot_stack[p], nv = t->n_vid_stack[p];
        const uint32_t *S = t->slot_stack[p], *W = t->vid_stack[p], *VT = t->vt[p], *OW = t->ow[p];
        if (nf > cap || nv > V) return false;
        mark.assign(V, 0);
        for (uint32_t i = 0; i < nf; ++i) {                    // free slots: inside the store, distinct
            if (S[i] >= cap || mark[S[i]]) return false;
            mark[S[i]] = 1;
        }
        for (uint32_t s = 0; s < V; ++s) {                     // owned slots: not free, mapped back by their id
            const uint32_t v = OW[s];
            if (v == kInvalid) continue;
            if (s >= cap || mark[s] || v >= V || VT[v] != s) return false;
            live[p] += 1;
        }
        if (live[p] != (uint64_t)cap - nf) return false;
        mark.assign(V, 0);
        for (uint32_t i = 0; i < nv; ++i) {                    // free ids: distinct, unmapped
            if (W[i] >= V || mark[W[i]] || VT[W[i]] != kInvalid) return false;
            mark[W[i]] = 1;
        }
        uint64_t mapped = 0;
        for (uint32_t v = 0; v < V; ++v) {
            if (VT[v] == kInvalid) continue;
            if (VT[v] >= cap || OW[VT[v]] != v) return false;
            mapped += 1;
        }
        if (mapped != live[p] || (uint64_t)nv != (uint64_t)V - live[p]) return false;
    }
    // every live unit belongs to exactly one request
    std::vector<uint8_t> ref[2];
    ref[0].assign(g.V[0], 0); ref[1].assign(g.V[1], 0);
    uint64_t held[2] = {0, 0};
    for (uint32_t r = 0; r < g.R; ++r) {
        const uint32_t state = t->req_state[r], np = t->req_npages[r], len = t->req_len[r];
        if (state == AVMP_REQ_EMPTY) { if (np || len) return false; continue; }
        if (state != AVMP_REQ_LIVE && state != AVMP_REQ_KV_ONLY) return false;
        // a held request has at least one token (ADMIT and EXTEND reject zero tokens)
        if (len == 0 || np > g.max_pages || ((uint64_t)len + g.T - 1) / g.T != np) return false;
        for (uint32_t j = 0; j < np; ++j) {
            const uint32_t h = t->req_chain[(size_t)r * g.max_pages + j], v = h & 0x7FFFFFFFu;
            if ((h >> 31) != AVMP_POOL_KV || v >= g.V[0] || t->vt[0][v] == kInvalid || ref[0][v]) return false;
            ref[0][v] = 1; held[0] += 1;
        }
        if (state == AVMP_REQ_LIVE)
            for (uint32_t l = 0; l < g.ns; ++l) {
                const uint32_t h = t->req_ssm[(size_t)r * g.ns + l], v = h & 0x7FFFFFFFu;
                if ((h >> 31) != AVMP_POOL_SSM || v >= g.V[1] || t->vt[1][v] == kInvalid || ref[1][v]) return false;
                ref[1][v] = 1; held[1] += 1;
            }
    }
    return held[0] == live[0] && held[1] == live[1];
}

}  // namespace

extern "C" {

void avmp_default_options(avmp_options *o)
{
    if (!o) return;
    o->threshold_low_ppm = 50000; o->threshold_high_ppm = 300000;
    o->min_rebalance_interval_ops = 1000; o->migration_enabled = 1;
    o->max_requests = 1024; o->max_pages_per_request = 4096; o->reclaim_gap = 0;
}

int avmp_derive_layout(const avmp_model_spec *m, uint64_t pool_bytes, double split, avmp_layout *out)
{
    if (!m || !out) return AVMP_EINVAL;
    if (!(split >= 0.0 && split <= 1.0) || m->page_tokens == 0) return AVMP_EINVAL;
    avmp_layout l;
    l.kv_row_bytes = (uint64_t)m->kv_heads * m->head_dim * m->kv_elem_bytes;
    l.kv_layer_bytes = 2ull * m->page_tokens * l.kv_row_bytes;
    l.ssm_state_bytes = (uint64_t)m->ssm_state_elems * m->ssm_elem_bytes;
    l.ssm_conv_bytes = (uint64_t)m->ssm_conv_elems * m->ssm_elem_bytes;
    l.unit_bytes[0] = ((uint64_t)m->n_attn_layers * l.kv_layer_bytes + 15u) & ~15ull;
    l.unit_bytes[1] = (l.ssm_state_bytes + l.ssm_conv_bytes + 15u) & ~15ull;
    if (l.unit_bytes[0] == 0 || l.unit_bytes[1] == 0) return AVMP_EINVAL;
    l.pool_bytes_aligned = pool_bytes & ~127ull;
    const uint64_t ppm = (uint64_t)llround(split * 1e6);
    const uint64_t ssm_bytes = (uint64_t)(((unsigned __int128)l.pool_bytes_aligned * ppm) / 1000000u) & ~127ull;
    l.cap0[0] = (l.pool_bytes_aligned - ssm_bytes) / l.unit_bytes[0];
    l.cap0[1] = ssm_bytes / l.unit_bytes[1];
    l.gap0 = l.pool_bytes_aligned - l.cap0[0] * l.unit_bytes[0] - l.cap0[1] * l.unit_bytes[1];
    for (int p = 0; p < 2; ++p) {
        l.vid_space[p] = l.pool_bytes_aligned / l.unit_bytes[p];
        if (l.vid_space[p] >= 0x7FFFFFFFull) return AVMP_EINVAL;
    }
    if (l.cap0[0] == 0 && l.cap0[1] == 0) return AVMP_EINVAL;
    *out = l;
    return AVMP_OK;
}

size_t avmp_workspace_bytes(const avmp_model_spec *spec, uint64_t pool_bytes, const avmp_options *opt)
{
    avmp_options o;
    if (opt) o = *opt; else avmp_default_options(&o);
    avmp_layout lay;
    if (!spec || !options_ok(o) || avmp_derive_layout(spec, pool_bytes, 0.5, &lay) != AVMP_OK) return 0;
    return ws_layout(lay, *spec, o).total;
}

int avmp_create(avmp_ctx **out, const avmp_model_spec *spec, void *d_arena, uint64_t pool_bytes,
                double initial_split, uint32_t migration_batch_size, const avmp_options *opt,
                void *d_workspace, size_t workspace_bytes, void *stream)
{
    if (!out || !spec || !d_arena || !d_workspace) return AVMP_EINVAL;
    if (((uintptr_t)d_arena | (uintptr_t)d_workspace) & (kAlign - 1)) return AVMP_EINVAL;
    avmp_options o;
    if (opt) o = *opt; else avmp_default_options(&o);
    if (!options_ok(o)) return AVMP_EINVAL;                       // Section 4.6: low >= high is invalid
    avmp_layout lay;
    if (avmp_derive_layout(spec, pool_bytes, initial_split, &lay) != AVMP_OK) return AVMP_EINVAL;
    const WsLayout w = ws_layout(lay, *spec, o);
    if (workspace_bytes < w.total) return AVMP_ENOSPC;

    avmp_ctx *c = new (std::nothrow) avmp_ctx();
    if (!c) return AVMP_EINVAL;
    c->spec = *spec; c->opt = o; c->lay = lay; c->B = migration_batch_size; c->launches = 0;
    c->d_workspace = d_workspace; c->workspace_bytes = workspace_bytes;
    int &dev = c->device;
    dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&c->sm_khz, cudaDevAttrClockRate, dev) != cudaSuccess) {
        delete c;
        return AVMP_ECUDA;
    }
    uint8_t *base = static_cast<uint8_t *>(d_workspace);
    Geom &g = c->g;
    g.P_al = lay.pool_bytes_aligned; g.U[0] = lay.unit_bytes[0]; g.U[1] = lay.unit_bytes[1];
    g.kv_layer_bytes = lay.kv_layer_bytes; g.row_bytes = lay.kv_row_bytes;
    g.state_bytes = lay.ssm_state_bytes; g.conv_bytes = lay.ssm_conv_bytes;
    g.min_interval = o.min_rebalance_interval_ops;
    g.V[0] = (uint32_t)lay.vid_space[0]; g.V[1] = (uint32_t)lay.vid_space[1];
    g.T = spec->page_tokens; g.na = spec->n_attn_layers; g.ns = spec->n_ssm_layers;
    g.R = o.max_requests; g.max_pages = o.max_pages_per_request; g.B = migration_batch_size;
    g.th_low = o.threshold_low_ppm; g.th_high = o.threshold_high_ppm; g.migration_enabled = o.migration_enabled;
    g.reclaim_gap = o.reclaim_gap ? 1u : 0u;
    g.arena = static_cast<uint8_t *>(d_arena);
    g.st = reinterpret_cast<DevState *>(base + w.state);
    for (int p = 0; p < 2; ++p) {
        g.S[p] = reinterpret_cast<uint32_t *>(base + w.S[p]); g.W[p] = reinterpret_cast<uint32_t *>(base + w.W[p]);
        g.VT[p] = reinterpret_cast<uint32_t *>(base + w.VT[p]); g.OW[p] = reinterpret_cast<uint32_t *>(base + w.OW[p]);
    }
    g.r_state = reinterpret_cast<uint32_t *>(base + w.r_state); g.r_len = reinterpret_cast<uint32_t *>(base + w.r_len);
    g.r_npages = reinterpret_cast<uint32_t *>(base + w.r_npages); g.r_chain = reinterpret_cast<uint32_t *>(base + w.r_chain);
    g.r_ssm = reinterpret_cast<uint32_t *>(base + w.r_ssm);
    g.reloc_src = reinterpret_cast<uint32_t *>(base + w.reloc_src); g.reloc_dst = reinterpret_cast<uint32_t *>(base + w.reloc_dst);
    g.g_cu_items = reinterpret_cast<uint32_t *>(base + w.g_cu_items); g.g_cu_rows = reinterpret_cast<uint32_t *>(base + w.g_cu_rows);
    c->d_stage_ops = reinterpret_cast<avmp_op *>(base + w.stage_ops);
    c->d_stage_status = reinterpret_cast<uint32_t *>(base + w.stage_status);

    DevState init;
    memset(&init, 0, sizeof(init));
    init.last_rebalance_op = kNone64;
    init.gap_bytes = lay.gap0;
    for (int p = 0; p < 2; ++p) {
        init.cap[p] = init.n_free[p] = (uint32_t)lay.cap0[p];
        init.n_vfree[p] = (uint32_t)lay.vid_space[p];
    }
    init.fsm = AVMP_FSM_BALANCED;
    // The row and piece prefix sums of a KV gather are 32-bit, like cu_seqlens: no request list of
    // up to max_requests entries (repeats allowed) may total 2^32 rows or copy pieces.
    {
        const uint64_t subs = kv_pieces_per_page(lay, spec->page_tokens);
        const uint64_t per_req = (uint64_t)o.max_pages_per_request * (spec->page_tokens > subs ? spec->page_tokens : subs);
        if ((unsigned __int128)o.max_requests * per_req >= ((unsigned __int128)1 << 32)) { delete c; return AVMP_EINVAL; }
    }
    if (launch_init(g, init, S(stream)) != cudaSuccess) { delete c; return AVMP_ECUDA; }
    // Bring avmp_gather_kv_static's in-library scratch onto this device now, while the caller still
    // has memory to spare (a failure here only shows up if that entry point is ever called).
    (void)static_gather_setup(dev);
    (void)cudaGetLastError();
    c->launches += 1;
    *out = c;
    return AVMP_OK;
}

int avmp_destroy(avmp_ctx *c)
{
    delete c;
    return AVMP_OK;
}

// A handle list to translate against the tables the step leaves (may be empty).
struct TranslateArgs {
    const uint32_t *h = nullptr;
    uint32_t n = 0;
    uint32_t *pool = nullptr;
    unsigned long long *off = nullptr, *aoff = nullptr;
};

static int step_rounds(avmp_ctx *c, const avmp_op *d_ops, uint32_t n_ops, const uint32_t *d_n_ops,
                       uint32_t *d_status, void *stream, const TranslateArgs &tr = TranslateArgs())
{
    // Section 3.2 throttle: migrations are >= min_interval logical ops apart, so a batch of n ops
    // holds at most (n - 1) / min_interval + 1 of them; one launch performs at most one.
    uint32_t rounds = 1;
    if (c->opt.migration_enabled)
        rounds = (uint32_t)((n_ops - 1) / c->opt.min_rebalance_interval_ops) + 1;
    // The copy grid is narrow (one 64-thread CTA per SM): a short handle list rides on it for free, a long one
    // (tens of thousands of handles; measured cross-over near 50 000) is faster in the wide translate kernel.
    const bool ride = c->opt.migration_enabled && tr.n && tr.n <= 32768u;
    for (uint32_t r = 0; r < rounds; ++r) {
        if (launch_step(c->g, d_ops, n_ops, d_n_ops, d_status, r == 0, S(stream)) != cudaSuccess) return AVMP_ECUDA;
        c->launches += 1;
        if (c->opt.migration_enabled) {
            // the last round's copy launch also carries the translation: two launches per step, not three
            const cudaError_t e = (ride && r + 1 == rounds)
                                      ? launch_relocate_translate(c->g, tr.h, tr.n, tr.pool, tr.off, tr.aoff, L(c, stream))
                                      : launch_relocate(c->g, L(c, stream));
            if (e != cudaSuccess) return AVMP_ECUDA;
            c->launches += 1;
        }
    }
    if (tr.n && !ride) {
        if (launch_translate(c->g, tr.h, tr.n, tr.pool, tr.off, tr.aoff, L(c, stream)) != cudaSuccess) return AVMP_ECUDA;
        c->launches += 1;
    }
    return AVMP_OK;
}

int avmp_step(avmp_ctx *c, const avmp_op *d_ops, uint32_t n_ops, uint32_t *d_status, void *stream)
{
    if (!c) return AVMP_EINVAL;
    if (n_ops == 0) return AVMP_OK;
    if (!d_ops || !d_status || ((uintptr_t)d_ops & 3) || ((uintptr_t)d_status & 3)) return AVMP_EINVAL;
    return step_rounds(c, d_ops, n_ops, nullptr, d_status, stream);
}

int avmp_step_translate(avmp_ctx *c, const avmp_op *d_ops, uint32_t n_ops, uint32_t *d_status, const uint32_t *d_handles,
                        uint32_t n_handles, uint32_t *d_pool, uint64_t *d_offset, uint64_t *d_arena_offset, void *stream)
{
    if (!c) return AVMP_EINVAL;
    if (n_handles && (!d_handles || !d_pool || !d_offset)) return AVMP_EINVAL;
    if (n_ops == 0) return avmp_translate(c, d_handles, n_handles, d_pool, d_offset, d_arena_offset, stream);
    if (!d_ops || !d_status || ((uintptr_t)d_ops & 3) || ((uintptr_t)d_status & 3)) return AVMP_EINVAL;
    TranslateArgs tr;
    tr.h = d_handles; tr.n = n_handles; tr.pool = d_pool;
    tr.off = (unsigned long long *)d_offset; tr.aoff = (unsigned long long *)d_arena_offset;
    return step_rounds(c, d_ops, n_ops, nullptr, d_status, stream, tr);
}

int avmp_step_indirect(avmp_ctx *c, const avmp_op *d_ops, const uint32_t *d_n_ops, uint32_t max_ops,
                       uint32_t *d_status, void *stream)
{
    if (!c || max_ops == 0) return AVMP_EINVAL;
    if (!d_ops || !d_n_ops || !d_status || ((uintptr_t)d_ops & 3) || ((uintptr_t)d_status & 3) || ((uintptr_t)d_n_ops & 3))
        return AVMP_EINVAL;
    return step_rounds(c, d_ops, max_ops, d_n_ops, d_status, stream);
}

int avmp_step_host(avmp_ctx *c, const avmp_op *h_ops, uint32_t n_ops, uint32_t *h_status, void *stream)
{
    if (!c) return AVMP_EINVAL;
    if (n_ops == 0) return AVMP_OK;
    if (!h_ops || !h_status || n_ops > kHostStepMaxOps) return AVMP_EINVAL;
    if (cudaMemcpyAsync(c->d_stage_ops, h_ops, (size_t)n_ops * sizeof(avmp_op), cudaMemcpyHostToDevice, S(stream)) != cudaSuccess)
        return AVMP_ECUDA;
    int rc = avmp_step(c, c->d_stage_ops, n_ops, c->d_stage_status, stream);
    if (rc != AVMP_OK) return rc;
    if (cudaMemcpyAsync(h_status, c->d_stage_status, (size_t)n_ops * 4, cudaMemcpyDeviceToHost, S(stream)) != cudaSuccess)
        return AVMP_ECUDA;
    return cu(cudaStreamSynchronize(S(stream)));
}

int avmp_translate(avmp_ctx *c, const uint32_t *d_handles, uint32_t n, uint32_t *d_pool,
                   uint64_t *d_offset, uint64_t *d_arena_offset, void *stream)
{
    if (!c) return AVMP_EINVAL;
    if (n == 0) return AVMP_OK;
    if (!d_handles || !d_pool || !d_offset) return AVMP_EINVAL;
    c->launches += 1;
    return cu(launch_translate(c->g, d_handles, n, d_pool, (unsigned long long *)d_offset,
                               (unsigned long long *)d_arena_offset, L(c, stream)));
}

int avmp_gather_kv(avmp_ctx *c, uint32_t layer, const uint32_t *d_reqs, uint32_t n, void *d_out_k,
                   void *d_out_v, uint64_t cap_tokens, uint32_t *d_cu, void *stream)
{
    if (!c || layer >= c->spec.n_attn_layers || n > c->opt.max_requests || !d_cu) return AVMP_EINVAL;
    if (n && (!d_reqs || !d_out_k || !d_out_v)) return AVMP_EINVAL;
    if (((uintptr_t)d_out_k | (uintptr_t)d_out_v) & 15) return AVMP_EINVAL;
    c->launches += n > kLocalPlanMax ? 2 : 1;      // a separate plan launch only for long lists
    return cu(launch_kv(c->g, false, layer, 1, d_reqs, nullptr, n, d_out_k, d_out_v, 0, cap_tokens, d_cu, L(c, stream)));
}

int avmp_scatter_kv(avmp_ctx *c, uint32_t layer, const uint32_t *d_reqs, const uint32_t *d_tok_start,
                    uint32_t n, const void *d_in_k, const void *d_in_v, void *stream)
{
    if (!c || layer >= c->spec.n_attn_layers || n > c->opt.max_requests) return AVMP_EINVAL;
    if (n == 0) return AVMP_OK;
    if (!d_reqs || !d_in_k || !d_in_v || (((uintptr_t)d_in_k | (uintptr_t)d_in_v) & 15)) return AVMP_EINVAL;
    c->launches += n > kLocalPlanMax ? 2 : 1;      // a separate plan launch only for long lists
    return cu(launch_kv(c->g, true, layer, 1, d_reqs, d_tok_start, n, const_cast<void *>(d_in_k),
                        const_cast<void *>(d_in_v), 0, ~0ull, nullptr, L(c, stream)));
}

int avmp_gather_ssm(avmp_ctx *c, uint32_t layer, const uint32_t *d_reqs, uint32_t n, void *d_out_state,
                    void *d_out_conv, void *stream)
{
    if (!c || layer >= c->spec.n_ssm_layers) return AVMP_EINVAL;
    if (n == 0) return AVMP_OK;
    if (!d_reqs || !d_out_state || !d_out_conv || (((uintptr_t)d_out_state | (uintptr_t)d_out_conv) & 15)) return AVMP_EINVAL;
    c->launches += 1;
    return cu(launch_ssm(c->g, false, layer, 1, d_reqs, n, d_out_state, 0, d_out_conv, 0, L(c, stream)));
}

int avmp_scatter_ssm(avmp_ctx *c, uint32_t layer, const uint32_t *d_reqs, uint32_t n, const void *d_in_state,
                     const void *d_in_conv, void *stream)
{
    if (!c || layer >= c->spec.n_ssm_layers) return AVMP_EINVAL;
    if (n == 0) return AVMP_OK;
    if (!d_reqs || !d_in_state || !d_in_conv || (((uintptr_t)d_in_state | (uintptr_t)d_in_conv) & 15)) return AVMP_EINVAL;
    c->launches += 1;
    return cu(launch_ssm(c->g, true, layer, 1, d_reqs, n, const_cast<void *>(d_in_state), 0,
                         const_cast<void *>(d_in_conv), 0, L(c, stream)));
}

int avmp_gather_kv_layers(avmp_ctx *c, uint32_t first_layer, uint32_t n_layers, const uint32_t *d_reqs, uint32_t n,
                          void *d_out_k, void *d_out_v, uint64_t layer_stride_bytes, uint64_t cap_tokens,
                          uint32_t *d_cu, void *stream)
{
    if (!c || n_layers == 0 || (uint64_t)first_layer + n_layers > c->spec.n_attn_layers) return AVMP_EINVAL;
    if (n > c->opt.max_requests || !d_cu) return AVMP_EINVAL;
    if (n && (!d_reqs || !d_out_k || !d_out_v)) return AVMP_EINVAL;
    if (((uintptr_t)d_out_k | (uintptr_t)d_out_v | layer_stride_bytes) & 15) return AVMP_EINVAL;
    if (n_layers > 1 && layer_stride_bytes < cap_tokens * c->lay.kv_row_bytes) return AVMP_EINVAL;
    c->launches += n > kLocalPlanMax ? 2 : 1;      // a separate plan launch only for long lists
    return cu(launch_kv(c->g, false, first_layer, n_layers, d_reqs, nullptr, n, d_out_k, d_out_v, layer_stride_bytes,
                        cap_tokens, d_cu, L(c, stream)));
}

int avmp_gather_ssm_layers(avmp_ctx *c, uint32_t first_layer, uint32_t n_layers, const uint32_t *d_reqs, uint32_t n,
                           void *d_out_state, uint64_t state_layer_stride_bytes, void *d_out_conv,
                           uint64_t conv_layer_stride_bytes, void *stream)
{
    if (!c || n_layers == 0 || (uint64_t)first_layer + n_layers > c->spec.n_ssm_layers) return AVMP_EINVAL;
    if (n == 0) return AVMP_OK;
    if (!d_reqs || !d_out_state || !d_out_conv) return AVMP_EINVAL;
    if (((uintptr_t)d_out_state | (uintptr_t)d_out_conv | state_layer_stride_bytes | conv_layer_stride_bytes) & 15) return AVMP_EINVAL;
    if (n_layers > 1 && (state_layer_stride_bytes < (uint64_t)n * c->lay.ssm_state_bytes ||
                         conv_layer_stride_bytes < (uint64_t)n * c->lay.ssm_conv_bytes)) return AVMP_EINVAL;
    c->launches += 1;
    return cu(launch_ssm(c->g, false, first_layer, n_layers, d_reqs, n, d_out_state, state_layer_stride_bytes,
                         d_out_conv, conv_layer_stride_bytes, L(c, stream)));
}

int avmp_gather_step(avmp_ctx *c, const uint32_t *d_reqs, uint32_t n, uint32_t first_attn_layer, uint32_t n_attn_layers,
                     void *d_out_k, void *d_out_v, uint64_t kv_layer_stride_bytes, uint64_t cap_tokens, uint32_t *d_cu,
                     uint32_t first_ssm_layer, uint32_t n_ssm_layers, void *d_out_state, uint64_t state_layer_stride_bytes,
                     void *d_out_conv, uint64_t conv_layer_stride_bytes, void *stream)
{
    if (!c || n_attn_layers == 0 || (uint64_t)first_attn_layer + n_attn_layers > c->spec.n_attn_layers) return AVMP_EINVAL;
    if (n_ssm_layers == 0 || (uint64_t)first_ssm_layer + n_ssm_layers > c->spec.n_ssm_layers) return AVMP_EINVAL;
    if (n > c->opt.max_requests || !d_cu) return AVMP_EINVAL;
    if (n && (!d_reqs || !d_out_k || !d_out_v || !d_out_state || !d_out_conv)) return AVMP_EINVAL;
    if (((uintptr_t)d_out_k | (uintptr_t)d_out_v | kv_layer_stride_bytes | (uintptr_t)d_out_state | (uintptr_t)d_out_conv |
         state_layer_stride_bytes | conv_layer_stride_bytes) & 15) return AVMP_EINVAL;
    if (n_attn_layers > 1 && kv_layer_stride_bytes < cap_tokens * c->lay.kv_row_bytes) return AVMP_EINVAL;
    if (n_ssm_layers > 1 && (state_layer_stride_bytes < (uint64_t)n * c->lay.ssm_state_bytes ||
                             conv_layer_stride_bytes < (uint64_t)n * c->lay.ssm_conv_bytes)) return AVMP_EINVAL;
    c->launches += n > kLocalPlanMax ? 2 : 1;
    return cu(launch_step_gather(c->g, d_reqs, n, first_attn_layer, n_attn_layers, d_out_k, d_out_v, kv_layer_stride_bytes,
                                 cap_tokens, d_cu, first_ssm_layer, n_ssm_layers, d_out_state, state_layer_stride_bytes,
                                 d_out_conv, conv_layer_stride_bytes, L(c, stream)));
}

int avmp_scatter_kv_layers(avmp_ctx *c, uint32_t first_layer, uint32_t n_layers, const uint32_t *d_reqs,
                           const uint32_t *d_tok_start, uint32_t n, const void *d_in_k, const void *d_in_v,
                           uint64_t layer_stride_bytes, void *stream)
{
    if (!c || n_layers == 0 || (uint64_t)first_layer + n_layers > c->spec.n_attn_layers || n > c->opt.max_requests) return AVMP_EINVAL;
    if (n == 0) return AVMP_OK;
    if (!d_reqs || !d_in_k || !d_in_v || (((uintptr_t)d_in_k | (uintptr_t)d_in_v | layer_stride_bytes) & 15)) return AVMP_EINVAL;
    c->launches += n > kLocalPlanMax ? 2 : 1;      // a separate plan launch only for long lists
    return cu(launch_kv(c->g, true, first_layer, n_layers, d_reqs, d_tok_start, n, const_cast<void *>(d_in_k),
                        const_cast<void *>(d_in_v), layer_stride_bytes, ~0ull, nullptr, L(c, stream)));
}

int avmp_scatter_ssm_layers(avmp_ctx *c, uint32_t first_layer, uint32_t n_layers, const uint32_t *d_reqs, uint32_t n,
                            const void *d_in_state, uint64_t state_layer_stride_bytes, const void *d_in_conv,
                            uint64_t conv_layer_stride_bytes, void *stream)
{
    if (!c || n_layers == 0 || (uint64_t)first_layer + n_layers > c->spec.n_ssm_layers) return AVMP_EINVAL;
    if (n == 0) return AVMP_OK;
    if (!d_reqs || !d_in_state || !d_in_conv) return AVMP_EINVAL;
    if (((uintptr_t)d_in_state | (uintptr_t)d_in_conv | state_layer_stride_bytes | conv_layer_stride_bytes) & 15) return AVMP_EINVAL;
    c->launches += 1;
    return cu(launch_ssm(c->g, true, first_layer, n_layers, d_reqs, n, const_cast<void *>(d_in_state),
                         state_layer_stride_bytes, const_cast<void *>(d_in_conv), conv_layer_stride_bytes, L(c, stream)));
}

int avmp_get_stats(avmp_ctx *c, avmp_stats *h_out, void *stream)
{
    if (!c || !h_out) return AVMP_EINVAL;
    DevState d;
    if (cudaMemcpyAsync(&d, c->g.st, sizeof(d), cudaMemcpyDeviceToHost, S(stream)) != cudaSuccess) return AVMP_ECUDA;
    if (cudaStreamSynchronize(S(stream)) != cudaSuccess) return AVMP_ECUDA;
    fill_stats(c, d, h_out);
    return AVMP_OK;
}

int avmp_clear_error(avmp_ctx *c, void *stream)
{
    if (!c) return AVMP_EINVAL;
    return cu(cudaMemsetAsync(&c->g.st->error_code, 0, 16, S(stream)));
}

int avmp_export_tables(avmp_ctx *c, avmp_tables *t, void *stream)
{
    if (!c || !t) return AVMP_EINVAL;
    const Geom &g = c->g;
    cudaStream_t s = S(stream);
    DevState d;
    bool ok = cudaMemcpyAsync(&d, g.st, sizeof(d), cudaMemcpyDeviceToHost, s) == cudaSuccess;
    auto pull = [&](uint32_t *dst, const uint32_t *src, size_t n) {
        if (dst && n) ok = ok && cudaMemcpyAsync(dst, src, n * 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    };
    for (int p = 0; p < 2; ++p) {
        pull(t->slot_stack[p], g.S[p], g.V[p]); pull(t->vid_stack[p], g.W[p], g.V[p]);
        pull(t->vt[p], g.VT[p], g.V[p]); pull(t->ow[p], g.OW[p], g.V[p]);
    }
    pull(t->req_state, g.r_state, g.R); pull(t->req_len, g.r_len, g.R); pull(t->req_npages, g.r_npages, g.R);
    pull(t->req_chain, g.r_chain, (size_t)g.R * g.max_pages); pull(t->req_ssm, g.r_ssm, (size_t)g.R * g.ns);
    if (!ok || cudaStreamSynchronize(s) != cudaSuccess) return AVMP_ECUDA;
    for (int p = 0; p < 2; ++p) { t->n_slot_stack[p] = d.n_free[p]; t->n_vid_stack[p] = d.n_vfree[p]; }
    fill_stats(c, d, &t->stats);
    return AVMP_OK;
}

int avmp_import_tables(avmp_ctx *c, const avmp_tables *t, void *stream)
{
    if (!c || !t) return AVMP_EINVAL;
    const Geom &g = c->g;
    cudaStream_t s = S(stream);
    for (int p = 0; p < 2; ++p) {
        if (!t->slot_stack[p] || !t->vid_stack[p] || !t->vt[p] || !t->ow[p]) return AVMP_EINVAL;
        if (t->n_slot_stack[p] > g.V[p] || t->n_vid_stack[p] > g.V[p] || t->stats.cap[p] > g.V[p]) return AVMP_EINVAL;
    }
    if (!t->req_state || !t->req_len || !t->req_npages || !t->req_chain || (g.ns && !t->req_ssm)) return AVMP_EINVAL;
    if (!tables_consistent(c, t)) return AVMP_EINVAL;          // nothing has been copied yet
    bool ok = true;
    auto push = [&](uint32_t *dst, const uint32_t *src, size_t n) {
        if (n) ok = ok && cudaMemcpyAsync(dst, src, n * 4, cudaMemcpyHostToDevice, s) == cudaSuccess;
    };
    for (int p = 0; p < 2; ++p) {
        push(g.S[p], t->slot_stack[p], g.V[p]); push(g.W[p], t->vid_stack[p], g.V[p]);
        push(g.VT[p], t->vt[p], g.V[p]); push(g.OW[p], t->ow[p], g.V[p]);
    }
    push(g.r_state, t->req_state, g.R); push(g.r_len, t->req_len, g.R); push(g.r_npages, t->req_npages, g.R);
    push(g.r_chain, t->req_chain, (size_t)g.R * g.max_pages); push(g.r_ssm, t->req_ssm, (size_t)g.R * g.ns);
    DevState d;
    memset(&d, 0, sizeof(d));
    const avmp_stats &st = t->stats;
    d.op_counter = st.op_counter; d.last_rebalance_op = st.last_rebalance_op; d.n_oom = st.n_oom;
    d.n_capacity_error = st.n_capacity_error; d.n_rebalance = st.n_rebalance;
    d.migrated_bytes = st.migrated_bytes; d.wasted_bytes = st.wasted_bytes;
    d.relocated_blocks = st.relocated_blocks; d.relocated_bytes = st.relocated_bytes;
    d.gap_bytes = st.gap_bytes; d.n_invalid = st.n_invalid;
    for (int p = 0; p < 2; ++p) {
        d.cap[p] = (uint32_t)st.cap[p]; d.n_free[p] = t->n_slot_stack[p]; d.n_vfree[p] = t->n_vid_stack[p];
    }
    d.fsm = (uint32_t)st.fsm_state;
    ok = ok && cudaMemcpyAsync(g.st, &d, sizeof(d), cudaMemcpyHostToDevice, s) == cudaSuccess;
    // the host arrays (and `d`) must outlive the copies
    if (!ok || cudaStreamSynchronize(s) != cudaSuccess) return AVMP_ECUDA;
    return AVMP_OK;
}

uint64_t avmp_launch_count(const avmp_ctx *c) { return c ? c->launches : 0; }

const char *avmp_error_string(int code)
{
    switch (code) {
    case AVMP_OK: return "ok";
    case AVMP_EINVAL: return "invalid argument";
    case AVMP_ENOSPC: return "workspace too small";
    case AVMP_ECUDA: return "CUDA runtime error";
    case AVMP_ETOOBIG: return "request list longer than the fixed in-library scratch allows (AVMP_STATIC_GATHER_MAX_REQS)";
    default: return "unknown error";
    }
}

}  // extern "C"
