/*
 * AVMP CPU oracle -- TEST INFRASTRUCTURE (see avmp_oracle.h for scope and pins).
 *
 * Every function below is the sequential definition written out: one operation
 * at a time, one unit at a time, no batching, no reordering.
 */
#include "avmp_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#include <sys/mman.h>

struct orc_ctx {
    orc_model m;
    orc_options o;
    uint32_t B;              /* migration_batch_size, in donor units */
    uint64_t P_al;           /* pool bytes, aligned down to 128 (Section 3.1: slab alignment) */
    uint64_t U[2];           /* native unit bytes per pool (Section 3.1) */
    uint64_t V[2];           /* virtual id space per pool */
    uint64_t kv_layer_bytes; /* bytes of one attention layer inside a page: K then V */
    uint64_t gap;
    uint32_t cap[2];
    uint32_t n_free[2];      /* entries on the slot stack */
    uint32_t n_vfree[2];     /* entries on the vid stack */
    uint32_t *S[2];          /* free physical slots, LIFO, top = last */
    uint32_t *W[2];          /* free virtual ids, LIFO, top = last */
    uint32_t *VT[2];         /* page table: vid -> slot */
    uint32_t *OW[2];         /* owner: slot -> vid */
    uint32_t *r_state, *r_len, *r_npages, *r_chain, *r_ssm;
    uint64_t op_counter, last_rebalance_op;
    uint32_t fsm;
    uint64_t n_oom, n_capacity_error, n_rebalance, migrated_bytes, wasted_bytes;
    uint64_t relocated_blocks, relocated_bytes, n_invalid;
    uint8_t *store[2];       /* payload, or NULL */
    uint64_t store_bytes[2];
};

static uint64_t align_up16(uint64_t x) { return (x + 15u) & ~(uint64_t)15u; }

orc_ctx *orc_create(const orc_model *m, uint64_t pool_bytes, double initial_split,
                    uint32_t migration_batch_size, const orc_options *opt, int with_store)
{
    if (!m || !opt) return NULL;
    if (opt->threshold_low_ppm >= opt->threshold_high_ppm) return NULL;   /* Section 4.6 */
    if (!(initial_split >= 0.0 && initial_split <= 1.0)) return NULL;
    if (m->page_tokens == 0 || opt->max_requests == 0 || opt->max_pages_per_request == 0) return NULL;

    orc_ctx *c = (orc_ctx *)calloc(1, sizeof(*c));
    if (!c) return NULL;
    c->m = *m;
    c->o = *opt;
    c->B = migration_batch_size;

    /* Section 3.1: a KV page holds page_tokens tokens of per-token bytes (K and V of every
     * attention layer); an SSM block holds one layer's state (recurrent state, then the
     * convolution window).  Units are rounded up to 16 bytes, the pool down to 128. */
    c->kv_layer_bytes = 2ull * m->page_tokens * m->kv_heads * m->head_dim * m->kv_elem_bytes;
    c->U[ORC_KV] = align_up16((uint64_t)m->n_attn_layers * c->kv_layer_bytes);
    c->U[ORC_SSM] = align_up16(((uint64_t)m->ssm_state_elems + m->ssm_conv_elems) * m->ssm_elem_bytes);
    if (c->U[ORC_KV] == 0 || c->U[ORC_SSM] == 0) { free(c); return NULL; }
    c->P_al = pool_bytes & ~(uint64_t)127u;

    uint64_t split_ppm = (uint64_t)llround(initial_split * 1e6);
    uint64_t ssm_bytes = (uint64_t)(((unsigned __int128)c->P_al * split_ppm) / 1000000u) & ~(uint64_t)127u;
    uint64_t kv_bytes = c->P_al - ssm_bytes;
    c->cap[ORC_KV] = (uint32_t)(kv_bytes / c->U[ORC_KV]);
    c->cap[ORC_SSM] = (uint32_t)(ssm_bytes / c->U[ORC_SSM]);
    c->gap = c->P_al - c->cap[ORC_KV] * c->U[ORC_KV] - c->cap[ORC_SSM] * c->U[ORC_SSM];
    for (int p = 0; p < 2; ++p) {
        c->V[p] = c->P_al / c->U[p];
        if (c->V[p] >= 0x7FFFFFFFull) { free(c); return NULL; }  /* 31-bit page id */
    }
    if (c->cap[ORC_KV] == 0 && c->cap[ORC_SSM] == 0) { free(c); return NULL; }

    for (int p = 0; p < 2; ++p) {
        uint64_t v = c->V[p] ? c->V[p] : 1;
        c->S[p] = (uint32_t *)malloc(v * 4);
        c->W[p] = (uint32_t *)malloc(v * 4);
        c->VT[p] = (uint32_t *)malloc(v * 4);
        c->OW[p] = (uint32_t *)malloc(v * 4);
        for (uint64_t i = 0; i < c->V[p]; ++i) c->VT[p][i] = c->OW[p][i] = ORC_INVALID;
        /* Fresh pools hand out slot 0, 1, 2, ... and vid 0, 1, 2, ...: the lowest index is on top. */
        c->n_free[p] = c->cap[p];
        for (uint32_t i = 0; i < c->cap[p]; ++i) c->S[p][i] = c->cap[p] - 1 - i;
        c->n_vfree[p] = (uint32_t)c->V[p];
        for (uint64_t i = 0; i < c->V[p]; ++i) c->W[p][i] = (uint32_t)(c->V[p] - 1 - i);
    }
    uint64_t R = opt->max_requests;
    c->r_state = (uint32_t *)calloc(R, 4);
    c->r_len = (uint32_t *)calloc(R, 4);
    c->r_npages = (uint32_t *)calloc(R, 4);
    c->r_chain = (uint32_t *)malloc(R * opt->max_pages_per_request * 4);
    c->r_ssm = (uint32_t *)malloc(R * (m->n_ssm_layers ? m->n_ssm_layers : 1) * 4);
    memset(c->r_chain, 0xFF, R * opt->max_pages_per_request * 4);
    memset(c->r_ssm, 0xFF, R * (m->n_ssm_layers ? m->n_ssm_layers : 1) * 4);
    c->last_rebalance_op = ORC_NONE64;
    c->fsm = ORC_BALANCED;

    if (with_store) {
        /* Section 3.2: each store spans its maximum possible capacity. */
        for (int p = 0; p < 2; ++p) {
            c->store_bytes[p] = c->V[p] * c->U[p];
            if (c->store_bytes[p] == 0) continue;
            void *mem = mmap(NULL, c->store_bytes[p], PROT_READ | PROT_WRITE,
                             MAP_PRIVATE | MAP_ANONYMOUS | MAP_NORESERVE, -1, 0);
            if (mem == MAP_FAILED) { orc_destroy(c); return NULL; }
            c->store[p] = (uint8_t *)mem;
        }
    }
    return c;
}

void orc_destroy(orc_ctx *c)
{
    if (!c) return;
    for (int p = 0; p < 2; ++p) {
        free(c->S[p]); free(c->W[p]); free(c->VT[p]); free(c->OW[p]);
        if (c->store[p]) munmap(c->store[p], c->store_bytes[p]);
    }
    free(c->r_state); free(c->r_len); free(c->r_npages); free(c->r_chain); free(c->r_ssm);
    free(c);
}

/* ---- the two primitive operations (Section 3.1: allocations return a tagged handle) ---- */
static uint32_t alloc_unit(orc_ctx *c, int p)
{
    uint32_t slot = c->S[p][--c->n_free[p]];
    uint32_t vid = c->W[p][--c->n_vfree[p]];
    c->VT[p][vid] = slot;
    c->OW[p][slot] = vid;
    return ((uint32_t)p << 31) | vid;
}

static void free_unit(orc_ctx *c, uint32_t h)
{
    int p = (int)(h >> 31);
    uint32_t vid = h & 0x7FFFFFFFu;
    uint32_t slot = c->VT[p][vid];
    c->VT[p][vid] = ORC_INVALID;
    c->OW[p][slot] = ORC_INVALID;
    c->S[p][c->n_free[p]++] = slot;
    c->W[p][c->n_vfree[p]++] = vid;
}

/* ---- Section 3.2: the CapacityError handler ---- */
static void capacity_error(orc_ctx *c, int X)
{
    int Y = 1 - X;
    c->n_capacity_error += 1;

    /* State label (Figure 2): pressured while the failing pool's free fraction is below
     * threshold_low, back to balanced once it has recovered. */
    uint32_t pressured = (X == ORC_KV) ? ORC_KV_PRESSURED : ORC_SSM_PRESSURED;
    if ((uint64_t)c->n_free[X] * 1000000u < (uint64_t)c->o.threshold_low_ppm * c->cap[X])
        c->fsm = pressured;
    else if (c->fsm == pressured)
        c->fsm = ORC_BALANCED;

    if (!c->o.migration_enabled) return;
    if (c->cap[Y] == 0) return;
    /* Trigger: the other pool's free fraction strictly above threshold_high. */
    if (!((uint64_t)c->n_free[Y] * 1000000u > (uint64_t)c->o.threshold_high_ppm * c->cap[Y])) return;
    /* Throttle: at least min_rebalance_interval_ops logical operations since the last one. */
    if (c->last_rebalance_op != ORC_NONE64 &&
        c->op_counter - c->last_rebalance_op < c->o.min_rebalance_interval_ops) return;

    uint64_t n = c->B < c->n_free[Y] ? c->B : c->n_free[Y];
    uint64_t ceded = n * c->U[Y];
    /* Section 3.2 as written: the recipient gets the whole units that fit in the ceded bytes and
     * the remainder is wasted.  With reclaim_gap (a variant, not in the paper) the bytes already
     * stranded between the pools are offered again together with the ceded ones. */
    uint64_t carry = c->o.reclaim_gap ? c->gap : 0;
    uint64_t mgain = (carry + ceded) / c->U[X];
    uint64_t waste = (carry + ceded) % c->U[X];   /* bytes freed modulo the recipient unit */
    if (mgain == 0) return;               /* nothing whole to hand over: state untouched */

    c->fsm = ORC_REBALANCING;
    uint32_t newcap = c->cap[Y] - (uint32_t)n;

    /* The donor shrinks at the high end: slots >= newcap leave its free list (order kept). */
    uint32_t kept = 0;
    for (uint32_t i = 0; i < c->n_free[Y]; ++i)
        if (c->S[Y][i] < newcap) c->S[Y][kept++] = c->S[Y][i];
    c->n_free[Y] = kept;

    /* Live units in the ceded range move down, lowest first, and their handles are remapped. */
    for (uint32_t s = newcap; s < c->cap[Y]; ++s) {
        uint32_t v = c->OW[Y][s];
        if (v == ORC_INVALID) continue;
        uint32_t d = c->S[Y][--c->n_free[Y]];
        if (c->store[Y])
            memcpy(c->store[Y] + (uint64_t)d * c->U[Y], c->store[Y] + (uint64_t)s * c->U[Y], c->U[Y]);
        c->VT[Y][v] = d;
        c->OW[Y][d] = v;
        c->OW[Y][s] = ORC_INVALID;
        c->relocated_blocks += 1;
        c->relocated_bytes += c->U[Y];
    }
    c->cap[Y] = newcap;

    /* The recipient grows by whole units; the lowest new slot is handed out first. */
    for (uint64_t s = c->cap[X] + mgain; s-- > c->cap[X];)
        c->S[X][c->n_free[X]++] = (uint32_t)s;
    c->cap[X] += (uint32_t)mgain;

    c->gap = c->gap - carry + waste;
    if (!c->o.reclaim_gap) c->wasted_bytes += waste;   /* with reclaim nothing is lost for good */
    c->migrated_bytes += ceded;
    c->n_rebalance += 1;
    c->last_rebalance_op = c->op_counter;
    c->fsm = ORC_BALANCED;
}

static uint32_t do_alloc_op(orc_ctx *c, const orc_op *op)
{
    const uint32_t T = c->m.page_tokens, ns = c->m.n_ssm_layers;
    uint32_t r = op->req;
    uint32_t need_s = (op->kind == ORC_ADMIT) ? ns : 0;
    uint64_t new_len = (uint64_t)c->r_len[r] + op->tokens;
    uint64_t pages = (new_len + T - 1) / T;
    if (pages > c->o.max_pages_per_request || new_len > 0xFFFFFFFFull) return ORC_TOO_LONG;
    uint32_t need_k = (uint32_t)pages - c->r_npages[r];

    /* allocate() raises CapacityError when a pool cannot serve; SSM is tried first. */
    if (need_s > c->n_free[ORC_SSM]) capacity_error(c, ORC_SSM);
    if (need_k > c->n_free[ORC_KV]) capacity_error(c, ORC_KV);
    if (need_s > c->n_free[ORC_SSM] || need_k > c->n_free[ORC_KV]) {
        c->n_oom += 1;
        return ORC_OOM;                    /* nothing was taken */
    }
    for (uint32_t l = 0; l < need_s; ++l) c->r_ssm[(uint64_t)r * ns + l] = alloc_unit(c, ORC_SSM);
    for (uint32_t j = 0; j < need_k; ++j)
        c->r_chain[(uint64_t)r * c->o.max_pages_per_request + c->r_npages[r] + j] = alloc_unit(c, ORC_KV);
    c->r_npages[r] += need_k;
    c->r_len[r] = (uint32_t)new_len;
    c->r_state[r] = ORC_LIVE;
    return ORC_OK;
}

static uint32_t do_op(orc_ctx *c, const orc_op *op)
{
    c->op_counter += 1;                    /* every operation advances the logical clock */
    if (op->kind != ORC_ADMIT && op->kind != ORC_EXTEND && op->kind != ORC_FINISH) return ORC_BAD_ARG;
    if (op->req >= c->o.max_requests) return ORC_BAD_REQ;
    uint32_t r = op->req, st = c->r_state[r];
    const uint32_t ns = c->m.n_ssm_layers;

    if (op->kind == ORC_ADMIT) {
        if (op->tokens == 0) return ORC_BAD_ARG;
        if (op->flags & ORC_RESUME) { if (st != ORC_KV_ONLY) return ORC_BAD_REQ; }
        else if (st != ORC_EMPTY) return ORC_BAD_REQ;
        return do_alloc_op(c, op);
    }
    if (op->kind == ORC_EXTEND) {
        if (op->tokens == 0) return ORC_BAD_ARG;
        if (st != ORC_LIVE) return ORC_BAD_REQ;
        return do_alloc_op(c, op);
    }
    /* FINISH */
    if (st != ORC_LIVE && st != ORC_KV_ONLY) return ORC_BAD_REQ;
    int keep = (op->flags & ORC_KEEP_KV) != 0;
    if (!keep) {
        for (uint32_t j = 0; j < c->r_npages[r]; ++j)
            free_unit(c, c->r_chain[(uint64_t)r * c->o.max_pages_per_request + j]);
        c->r_npages[r] = 0;
        c->r_len[r] = 0;
    }
    if (st == ORC_LIVE)
        for (uint32_t l = 0; l < ns; ++l) free_unit(c, c->r_ssm[(uint64_t)r * ns + l]);
    c->r_state[r] = keep ? ORC_KV_ONLY : ORC_EMPTY;
    return ORC_OK;
}

void orc_step(orc_ctx *c, const orc_op *ops, uint32_t n, uint32_t *status)
{
    for (uint32_t i = 0; i < n; ++i) {
        uint32_t s = do_op(c, &ops[i]);
        if (s >= ORC_BAD_REQ) c->n_invalid += 1;
        status[i] = s;
    }
}

/* ---- Section 3.1 / Figure 1: handle -> (pool, physical offset in that pool's store) ---- */
static int resolve(const orc_ctx *c, uint32_t h, uint32_t *pool, uint32_t *slot)
{
    if (h == ORC_INVALID) return 0;
    uint32_t p = h >> 31, vid = h & 0x7FFFFFFFu;
    if (vid >= c->V[p]) return 0;
    uint32_t s = c->VT[p][vid];
    if (s == ORC_INVALID) return 0;
    *pool = p;
    *slot = s;
    return 1;
}

uint32_t orc_translate(const orc_ctx *c, const uint32_t *handles, uint32_t n, uint32_t *pool,
                       uint64_t *offset)
{
    uint32_t bad = 0;
    for (uint32_t i = 0; i < n; ++i) {
        uint32_t p, s;
        if (resolve(c, handles[i], &p, &s)) {
            pool[i] = p;
            offset[i] = (uint64_t)s * c->U[p];
        } else {
            pool[i] = ORC_INVALID;
            offset[i] = ORC_NONE64;
            ++bad;
        }
    }
    return bad;
}

/* ---- Section 2.2: paged scatter-gather for KV, contiguous access for SSM state ---- */
static int holds_kv(const orc_ctx *c, uint32_t r)
{
    return r < c->o.max_requests && (c->r_state[r] == ORC_LIVE || c->r_state[r] == ORC_KV_ONLY);
}

/* Address of token t's K (part 0) or V (part 1) row of `layer` for request r.
 * In-page order: [layer][K|V][token][head][dim]. */
static uint8_t *kv_row(const orc_ctx *c, uint32_t r, uint32_t layer, uint32_t part, uint32_t t)
{
    const uint32_t T = c->m.page_tokens;
    const uint64_t row = (uint64_t)c->m.kv_heads * c->m.head_dim * c->m.kv_elem_bytes;
    uint32_t h = c->r_chain[(uint64_t)r * c->o.max_pages_per_request + t / T];
    uint32_t p, slot;
    if (!resolve(c, h, &p, &slot) || p != ORC_KV) return NULL;
    return c->store[ORC_KV] + (uint64_t)slot * c->U[ORC_KV] + (uint64_t)layer * c->kv_layer_bytes +
           (uint64_t)part * T * row + (uint64_t)(t % T) * row;
}

uint32_t orc_gather_kv(const orc_ctx *c, uint32_t layer, const uint32_t *reqs, uint32_t n,
                       void *out_k, void *out_v, uint64_t capacity_tokens, uint32_t *cu_seqlens)
{
    const uint64_t row = (uint64_t)c->m.kv_heads * c->m.head_dim * c->m.kv_elem_bytes;
    uint32_t bad = 0;
    uint64_t cu = 0;
    cu_seqlens[0] = 0;
    if (!c->store[ORC_KV] || layer >= c->m.n_attn_layers) return n ? n : 1;
    for (uint32_t k = 0; k < n; ++k) {
        uint32_t r = reqs[k];
        uint32_t len = holds_kv(c, r) ? c->r_len[r] : 0;
        if (!holds_kv(c, r)) ++bad;
        else if (cu + len > capacity_tokens) ++bad;   /* a held request has len >= 1: ADMIT / EXTEND take tokens >= 1 */
        else
            for (uint32_t t = 0; t < len; ++t) {
                memcpy((uint8_t *)out_k + (cu + t) * row, kv_row(c, r, layer, 0, t), row);
                memcpy((uint8_t *)out_v + (cu + t) * row, kv_row(c, r, layer, 1, t), row);
            }
        cu += len;
        cu_seqlens[k + 1] = (uint32_t)cu;
    }
    return bad;
}

uint32_t orc_scatter_kv(orc_ctx *c, uint32_t layer, const uint32_t *reqs, const uint32_t *tok_start,
                        uint32_t n, const void *in_k, const void *in_v)
{
    const uint64_t row = (uint64_t)c->m.kv_heads * c->m.head_dim * c->m.kv_elem_bytes;
    uint32_t bad = 0;
    uint64_t cu = 0;
    if (!c->store[ORC_KV] || layer >= c->m.n_attn_layers) return n ? n : 1;
    for (uint32_t k = 0; k < n; ++k) {
        uint32_t r = reqs[k];
        uint32_t t0 = tok_start ? tok_start[k] : 0;
        if (!holds_kv(c, r) || t0 > c->r_len[r]) { ++bad; continue; }
        uint32_t len = c->r_len[r];
        for (uint32_t t = t0; t < len; ++t) {
            memcpy(kv_row(c, r, layer, 0, t), (const uint8_t *)in_k + (cu + t - t0) * row, row);
            memcpy(kv_row(c, r, layer, 1, t), (const uint8_t *)in_v + (cu + t - t0) * row, row);
        }
        cu += len - t0;
    }
    return bad;
}

static uint8_t *ssm_block(const orc_ctx *c, uint32_t r, uint32_t layer)
{
    if (r >= c->o.max_requests || c->r_state[r] != ORC_LIVE) return NULL;
    uint32_t p, slot;
    if (!resolve(c, c->r_ssm[(uint64_t)r * c->m.n_ssm_layers + layer], &p, &slot) || p != ORC_SSM)
        return NULL;
    return c->store[ORC_SSM] + (uint64_t)slot * c->U[ORC_SSM];
}

uint32_t orc_gather_ssm(const orc_ctx *c, uint32_t layer, const uint32_t *reqs, uint32_t n,
                        void *out_state, void *out_conv)
{
    const uint64_t sb = (uint64_t)c->m.ssm_state_elems * c->m.ssm_elem_bytes;
    const uint64_t cb = (uint64_t)c->m.ssm_conv_elems * c->m.ssm_elem_bytes;
    uint32_t bad = 0;
    if (!c->store[ORC_SSM] || layer >= c->m.n_ssm_layers) return n ? n : 1;
    for (uint32_t k = 0; k < n; ++k) {
        const uint8_t *b = ssm_block(c, reqs[k], layer);
        if (!b) { ++bad; continue; }
        memcpy((uint8_t *)out_state + k * sb, b, sb);
        memcpy((uint8_t *)out_conv + k * cb, b + sb, cb);
    }
    return bad;
}

uint32_t orc_scatter_ssm(orc_ctx *c, uint32_t layer, const uint32_t *reqs, uint32_t n,
                         const void *in_state, const void *in_conv)
{
    const uint64_t sb = (uint64_t)c->m.ssm_state_elems * c->m.ssm_elem_bytes;
    const uint64_t cb = (uint64_t)c->m.ssm_conv_elems * c->m.ssm_elem_bytes;
    uint32_t bad = 0;
    if (!c->store[ORC_SSM] || layer >= c->m.n_ssm_layers) return n ? n : 1;
    for (uint32_t k = 0; k < n; ++k) {
        uint8_t *b = ssm_block(c, reqs[k], layer);
        if (!b) { ++bad; continue; }
        memcpy(b, (const uint8_t *)in_state + k * sb, sb);
        memcpy(b + sb, (const uint8_t *)in_conv + k * cb, cb);
    }
    return bad;
}

void orc_get_stats(const orc_ctx *c, orc_stats *s)
{
    s->op_counter = c->op_counter;
    s->last_rebalance_op = c->last_rebalance_op;
    s->n_oom = c->n_oom;
    s->n_capacity_error = c->n_capacity_error;
    s->n_rebalance = c->n_rebalance;
    s->migrated_bytes = c->migrated_bytes;
    s->wasted_bytes = c->wasted_bytes;
    s->relocated_blocks = c->relocated_blocks;
    s->relocated_bytes = c->relocated_bytes;
    s->gap_bytes = c->gap;
    for (int p = 0; p < 2; ++p) {
        s->cap[p] = c->cap[p];
        s->free_units[p] = c->n_free[p];
        s->unit_bytes[p] = c->U[p];
        s->vid_space[p] = c->V[p];
    }
    s->fsm_state = c->fsm;
    s->n_invalid = c->n_invalid;
    s->pool_bytes_aligned = c->P_al;
}

const uint8_t *orc_store_bytes(const orc_ctx *c, int pool, uint64_t offset, uint64_t n)
{
    if (pool < 0 || pool > 1 || !c->store[pool]) return NULL;
    if (offset > c->store_bytes[pool] || n > c->store_bytes[pool] - offset) return NULL;
    return c->store[pool] + offset;
}

const uint32_t *orc_table(const orc_ctx *c, int which, uint64_t *count)
{
    uint64_t R = c->o.max_requests;
    switch (which) {
    case ORC_T_SLOT_STACK_KV:  *count = c->n_free[ORC_KV];   return c->S[ORC_KV];
    case ORC_T_SLOT_STACK_SSM: *count = c->n_free[ORC_SSM];  return c->S[ORC_SSM];
    case ORC_T_VID_STACK_KV:   *count = c->n_vfree[ORC_KV];  return c->W[ORC_KV];
    case ORC_T_VID_STACK_SSM:  *count = c->n_vfree[ORC_SSM]; return c->W[ORC_SSM];
    case ORC_T_VT_KV:          *count = c->V[ORC_KV];        return c->VT[ORC_KV];
    case ORC_T_VT_SSM:         *count = c->V[ORC_SSM];       return c->VT[ORC_SSM];
    case ORC_T_OW_KV:          *count = c->V[ORC_KV];        return c->OW[ORC_KV];
    case ORC_T_OW_SSM:         *count = c->V[ORC_SSM];       return c->OW[ORC_SSM];
    case ORC_T_REQ_STATE:      *count = R;                   return c->r_state;
    case ORC_T_REQ_LEN:        *count = R;                   return c->r_len;
    case ORC_T_REQ_NPAGES:     *count = R;                   return c->r_npages;
    case ORC_T_REQ_CHAIN:      *count = R * c->o.max_pages_per_request; return c->r_chain;
    case ORC_T_REQ_SSM:        *count = R * c->m.n_ssm_layers;          return c->r_ssm;
    default:                   *count = 0;                   return NULL;
    }
}
