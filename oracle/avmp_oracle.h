/*
 * AVMP CPU oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, single-threaded, sequential statement of Asymmetric Virtual Memory
 * Paging as the paper defines it (Section 3.1: virtual handles, the page table,
 * the two backing stores and their native unit sizes; Section 3.2: the
 * CapacityError-triggered rebalancer, its waste formula, its logical-operation
 * throttle; Section 4.6: failure modes and configuration validation), plus the
 * two access patterns the paper names for the stores (Section 2.2: paged
 * scatter-gather for KV, contiguous reads for SSM state).
 *
 * Only tests, the smoke check and the CPU-baseline leg of the benchmark may use
 * this code.  It shares nothing with the CUDA library: its own types, its own
 * constants, its own storage layout (two separate oversized stores, as the
 * paper's prototype has; Section 3.2).
 *
 * Pins (tests that tie this code to something other than itself): unit sizes and
 * capacities by closed form; fresh-pool allocation order; the migration
 * arithmetic of Section 3.2 by hand; a counts-only model and a static dual-pool
 * model written separately (the paper's static-equivalence claim, Section 1.1);
 * a naive list-based model on tiny inputs; structural invariants after every
 * operation; gathers against a payload that is a pure function of (request,
 * token); the position of every byte inside a unit ([layer][K, V][token][head][dim]
 * for a page, state then window for a block) read from the raw store bytes.  The free-list order, the choice of which live blocks move where and
 * the unit of migration_batch_size are policy the paper leaves open: for those
 * this file *is* the definition (parity unpinned by the paper).  The reclaim_gap
 * option is a variant of the waste rule that the paper does not have; it is pinned
 * by its own hand-worked trace, a closed-form case and the two separate models.
 */
#ifndef AVMP_ORACLE_H
#define AVMP_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ORC_INVALID 0xFFFFFFFFu
#define ORC_NONE64 0xFFFFFFFFFFFFFFFFull

enum { ORC_KV = 0, ORC_SSM = 1 };
enum { ORC_ADMIT = 1, ORC_EXTEND = 2, ORC_FINISH = 3 };
enum { ORC_KEEP_KV = 1, ORC_RESUME = 2 };
enum { ORC_OK = 0, ORC_OOM = 1, ORC_BAD_REQ = 2, ORC_TOO_LONG = 3, ORC_BAD_ARG = 4 };
enum { ORC_EMPTY = 0, ORC_LIVE = 1, ORC_KV_ONLY = 2 };
enum { ORC_BALANCED = 0, ORC_KV_PRESSURED = 1, ORC_SSM_PRESSURED = 2, ORC_REBALANCING = 3 };

typedef struct {
    uint32_t n_attn_layers, n_ssm_layers, page_tokens, kv_heads, head_dim, kv_elem_bytes;
    uint32_t ssm_state_elems, ssm_conv_elems, ssm_elem_bytes;
} orc_model;

typedef struct {
    uint32_t threshold_low_ppm, threshold_high_ppm;
    uint64_t min_rebalance_interval_ops;
    uint32_t migration_enabled;
    uint32_t max_requests, max_pages_per_request;
    uint32_t reclaim_gap;   /* 0 = waste is lost to the gap (Section 3.2 as written); 1 = see capacity_error */
} orc_options;

typedef struct {
    uint8_t kind, flags;
    uint16_t rsvd;
    uint32_t req, tokens;
} orc_op;

/* All counters of one context, in a fixed order (also read as uint64_t[ORC_N_STATS]). */
typedef struct {
    uint64_t op_counter;          /* logical operations seen (Section 3.2) */
    uint64_t last_rebalance_op;   /* ORC_NONE64 before the first migration */
    uint64_t n_oom;               /* operations that ended OOM (the paper's N_OOM) */
    uint64_t n_capacity_error;    /* handler invocations */
    uint64_t n_rebalance;         /* completed migrations */
    uint64_t migrated_bytes;      /* donor bytes ceded */
    uint64_t wasted_bytes;        /* sum of (donor bytes ceded mod recipient unit) */
    uint64_t relocated_blocks;    /* live units moved out of ceded regions */
    uint64_t relocated_bytes;
    uint64_t gap_bytes;           /* pool bytes in neither store */
    uint64_t cap[2];              /* capacity in units, KV then SSM */
    uint64_t free_units[2];
    uint64_t fsm_state;
    uint64_t n_invalid;           /* ops rejected with BAD_REQ / TOO_LONG / BAD_ARG */
    uint64_t unit_bytes[2];
    uint64_t vid_space[2];
    uint64_t pool_bytes_aligned;
} orc_stats;
#define ORC_N_STATS (sizeof(orc_stats) / sizeof(uint64_t))

typedef struct orc_ctx orc_ctx;

/* with_store != 0: own payload bytes for both stores (zero-filled, committed lazily). */
orc_ctx *orc_create(const orc_model *m, uint64_t pool_bytes, double initial_split,
                    uint32_t migration_batch_size, const orc_options *opt, int with_store);
void orc_destroy(orc_ctx *c);

/* Process ops[0..n) one at a time in array order (Section 3.2: deterministic, counter-driven). */
void orc_step(orc_ctx *c, const orc_op *ops, uint32_t n, uint32_t *status);

/* handle -> (pool, offset within its store).  Invalid: pool = ORC_INVALID, offset = ORC_NONE64.
 * Returns the number of invalid handles. */
uint32_t orc_translate(const orc_ctx *c, const uint32_t *handles, uint32_t n, uint32_t *pool,
                       uint64_t *offset);

/* Paged gather of one attention layer for a request list.  cu_seqlens[n+1] always gets the
 * prefix sums of the valid lengths.  Requests that are not held, or whose rows would pass
 * capacity_tokens, copy nothing and count as errors (return value). */
uint32_t orc_gather_kv(const orc_ctx *c, uint32_t layer, const uint32_t *reqs, uint32_t n,
                       void *out_k, void *out_v, uint64_t capacity_tokens, uint32_t *cu_seqlens);
uint32_t orc_gather_ssm(const orc_ctx *c, uint32_t layer, const uint32_t *reqs, uint32_t n,
                        void *out_state, void *out_conv);

/* Write side used to fill the stores: tokens [tok_start[i], len_i) of request i come from
 * rows cu[i].. of in_k / in_v, cu being the prefix sum of (len_i - tok_start[i]). */
uint32_t orc_scatter_kv(orc_ctx *c, uint32_t layer, const uint32_t *reqs, const uint32_t *tok_start,
                        uint32_t n, const void *in_k, const void *in_v);
uint32_t orc_scatter_ssm(orc_ctx *c, uint32_t layer, const uint32_t *reqs, uint32_t n,
                         const void *in_state, const void *in_conv);

void orc_get_stats(const orc_ctx *c, orc_stats *out);

/* Read-only view of n raw bytes of a store (pool ORC_KV or ORC_SSM) starting at byte `offset`
 * of that store, i.e. at the offsets orc_translate returns.  NULL without payload stores or when
 * the range leaves the store.  Lets a test look at where inside a unit each byte was put. */
const uint8_t *orc_store_bytes(const orc_ctx *c, int pool, uint64_t offset, uint64_t n);

/* Views of the internal tables (owned by the context; valid until the next call). */
enum {
    ORC_T_SLOT_STACK_KV = 0, ORC_T_SLOT_STACK_SSM, ORC_T_VID_STACK_KV, ORC_T_VID_STACK_SSM,
    ORC_T_VT_KV, ORC_T_VT_SSM, ORC_T_OW_KV, ORC_T_OW_SSM,
    ORC_T_REQ_STATE, ORC_T_REQ_LEN, ORC_T_REQ_NPAGES, ORC_T_REQ_CHAIN, ORC_T_REQ_SSM
};
const uint32_t *orc_table(const orc_ctx *c, int which, uint64_t *count);

#ifdef __cplusplus
}
#endif
#endif
