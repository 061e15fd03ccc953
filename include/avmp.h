/*
 * avmp.h -- C ABI of the B200-native AVMP hot path.
 *
 * AVMP (Asymmetric Virtual Memory Paging) keeps two physically different cache
 * stores for hybrid Mamba-Transformer inference -- fine-grained KV pages and
 * per-layer SSM state blocks -- behind one space of 32-bit virtual handles, and
 * moves capacity between them when an allocation would otherwise fail (paper
 * Sections 3.1 and 3.2).  This library holds all allocator state in device
 * memory and runs every step of the path as CUDA kernels on sm_100a:
 *
 *   avmp_step        batched admit / extend / finish in array order, including the
 *                    CapacityError handler, the migration (shrink donor, relocate
 *                    live units, remap handles, grow recipient) and the retry;
 *   avmp_translate   handle -> (pool, physical offset);
 *   avmp_gather_kv   paged gather of one attention layer into ragged batch buffers;
 *   avmp_gather_ssm  gather of one SSM layer's state blocks into batch buffers;
 *   avmp_scatter_*   the matching write side.
 *
 * Conventions
 *   - "d_" arguments are DEVICE pointers, "h_" arguments are HOST pointers.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Every call is ordered on that stream.  Calls with only device arguments never
 *     synchronise with the host; calls that take or fill host memory do, and say so.
 *   - The library never allocates device memory: the caller owns the arena and the
 *     workspace (e.g. two torch tensors) and must keep them alive until avmp_destroy.
 *   - Return value: AVMP_OK or a negative AVMP_E* code for misuse the host can see.
 *     What only the device can see (an invalid handle, a dead request in a gather
 *     list, an output buffer too small) never traps: the item is skipped, a sticky
 *     error code and an error count are recorded in the statistics block.
 *   - One context must not be used from two streams at once.
 */
#ifndef AVMP_H
#define AVMP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define AVMP_API __attribute__((visibility("default")))
#else
#define AVMP_API
#endif

#define AVMP_INVALID 0xFFFFFFFFu              /* no handle / no slot */
#define AVMP_NONE64 0xFFFFFFFFFFFFFFFFull     /* no offset / "never" */

enum { AVMP_OK = 0, AVMP_EINVAL = -1, AVMP_ENOSPC = -2, AVMP_ECUDA = -3, AVMP_ETOOBIG = -4 };
enum { AVMP_POOL_KV = 0, AVMP_POOL_SSM = 1 };

/* Operation kinds and flags (avmp_op). */
enum { AVMP_OP_ADMIT = 1, AVMP_OP_EXTEND = 2, AVMP_OP_FINISH = 3 };
enum {
    AVMP_FLAG_KEEP_KV = 1, /* FINISH: free only the SSM blocks, keep the KV chain (slot becomes KV_ONLY) */
    AVMP_FLAG_RESUME = 2   /* ADMIT: the slot is KV_ONLY; allocate SSM blocks and extend the kept chain */
};
/* Per-operation result written by avmp_step. */
enum {
    AVMP_ST_OK = 0,
    AVMP_ST_OOM = 1,      /* did not fit, even after the migration attempt; nothing was taken */
    AVMP_ST_BAD_REQ = 2,  /* slot out of range or in the wrong state for this kind */
    AVMP_ST_TOO_LONG = 3, /* chain would pass max_pages_per_request */
    AVMP_ST_BAD_ARG = 4   /* unknown kind, or zero tokens on ADMIT / EXTEND */
};
enum { AVMP_REQ_EMPTY = 0, AVMP_REQ_LIVE = 1, AVMP_REQ_KV_ONLY = 2 };
/* Rebalancer state label (paper Figure 2). */
enum { AVMP_FSM_BALANCED = 0, AVMP_FSM_KV_PRESSURED = 1, AVMP_FSM_SSM_PRESSURED = 2, AVMP_FSM_REBALANCING = 3 };
/* Sticky device-side error codes (avmp_stats.error_code keeps the first one). */
enum {
    AVMP_DEV_OK = 0,
    AVMP_DEV_BAD_HANDLE = 1,     /* translate: handle does not resolve */
    AVMP_DEV_BAD_REQUEST = 2,    /* gather / scatter: request slot out of range or holds nothing */
    AVMP_DEV_OUT_OVERFLOW = 3,   /* gather_kv: rows would pass out_capacity_tokens */
    AVMP_DEV_TIMEOUT = 4         /* a copy kernel gave up a bounded wait; the output is incomplete */
};

/* Model shape: what one KV page and one SSM block hold (paper Section 3.1).
 * KV page  = page_tokens tokens of {K, V} x kv_heads x head_dim x kv_elem_bytes for EVERY
 *            attention layer, laid out [layer][K|V][token][head][dim];
 * SSM block = one layer's ssm_state_elems then ssm_conv_elems elements of ssm_elem_bytes. */
typedef struct {
    uint32_t n_attn_layers, n_ssm_layers, page_tokens, kv_heads, head_dim, kv_elem_bytes;
    uint32_t ssm_state_elems, ssm_conv_elems, ssm_elem_bytes;
} avmp_model_spec;

/* Rebalancer and table-size options (paper Section 3.2; defaults from avmp_default_options). */
typedef struct {
    uint32_t threshold_low_ppm;           /* 50000: labels the PRESSURED states only */
    uint32_t threshold_high_ppm;          /* 300000: donor free fraction must exceed this */
    uint64_t min_rebalance_interval_ops;  /* 1000 logical operations between migrations; >= 1 */
    uint32_t migration_enabled;           /* 0 = static partition with AVMP handles */
    uint32_t max_requests;                /* request slots: op.req is in [0, max_requests) */
    uint32_t max_pages_per_request;       /* longest KV chain, in pages */
    uint32_t reclaim_gap;                 /* 0 (default): the paper's rule, recipient gains floor(n*U_donor /
                                             U_recipient) units and the remainder is lost to the gap between
                                             the pools.  1: a variant with no counterpart in the paper, the
                                             bytes already in the gap are offered again with the ceded ones:
                                             gain = floor((gap + n*U_donor) / U_recipient), gap = remainder,
                                             wasted_bytes stays 0 */
} avmp_options;

/* One allocator operation, 12 bytes. */
typedef struct {
    uint8_t kind, flags;
    uint16_t rsvd;
    uint32_t req;     /* caller-chosen dense slot id */
    uint32_t tokens;  /* ADMIT / EXTEND: tokens appended */
} avmp_op;

/* Sizes derived from the model and the pool (host-side arithmetic, no device access). */
typedef struct {
    uint64_t pool_bytes_aligned;  /* pool_bytes rounded down to 128 (slab alignment) */
    uint64_t unit_bytes[2];       /* KV page, SSM block; each rounded up to 16 */
    uint64_t vid_space[2];        /* virtual ids per pool = pool_bytes_aligned / unit */
    uint64_t cap0[2];             /* initial capacities in units */
    uint64_t gap0;                /* initial bytes in neither store */
    uint64_t kv_layer_bytes;      /* one attention layer inside a page (K then V) */
    uint64_t kv_row_bytes;        /* one token's K (or V) of one layer */
    uint64_t ssm_state_bytes, ssm_conv_bytes;
} avmp_layout;

/* All counters of a context (same order as uint64_t[AVMP_N_STATS]). */
typedef struct {
    uint64_t op_counter;          /* logical operations processed (Section 3.2) */
    uint64_t last_rebalance_op;   /* AVMP_NONE64 before the first migration */
    uint64_t n_oom;               /* operations that ended AVMP_ST_OOM (the paper's N_OOM) */
    uint64_t n_capacity_error;    /* CapacityError handler runs */
    uint64_t n_rebalance;         /* completed migrations */
    uint64_t migrated_bytes;      /* donor bytes ceded */
    uint64_t wasted_bytes;        /* sum of ceded bytes modulo the recipient unit */
    uint64_t relocated_blocks;    /* live units copied out of ceded regions */
    uint64_t relocated_bytes;
    uint64_t gap_bytes;
    uint64_t cap[2];
    uint64_t free_units[2];
    uint64_t fsm_state;
    uint64_t n_invalid;           /* operations rejected with BAD_REQ / TOO_LONG / BAD_ARG */
    uint64_t unit_bytes[2];
    uint64_t vid_space[2];
    uint64_t pool_bytes_aligned;
    uint64_t error_code;          /* first AVMP_DEV_* error seen, sticky */
    uint64_t error_count;         /* items skipped because of device-side errors */
    uint64_t relocation_ns_last;  /* device-clock duration of the last relocation copy (first CTA in, last out) */
    uint64_t relocation_ns_total; /* sum over all relocation copies: the time spent migrating payload */
    /* Time decomposition of the allocator kernel (paper Section 4.3), SM cycles at the nominal clock:
     * everything; the part spent handling CapacityErrors that ended OOM; the part spent planning
     * migrations.  The rest is service time. */
    uint64_t step_ns_total, step_ns_oom_retry, step_ns_migration_plan;
} avmp_stats;
#define AVMP_N_STATS (sizeof(avmp_stats) / sizeof(uint64_t))

/* Host copies of every table, for parity checks and snapshot / restore.  The caller
 * provides the arrays (sizes from avmp_layout and avmp_options); counts are filled by
 * export and read by import. */
typedef struct {
    uint32_t *slot_stack[2];  /* [vid_space[p]]  free physical slots, bottom first */
    uint32_t *vid_stack[2];   /* [vid_space[p]]  free virtual ids, bottom first */
    uint32_t *vt[2];          /* [vid_space[p]]  page table: vid -> slot or AVMP_INVALID */
    uint32_t *ow[2];          /* [vid_space[p]]  owner: slot -> vid or AVMP_INVALID */
    uint32_t *req_state;      /* [max_requests] */
    uint32_t *req_len;        /* [max_requests] tokens held */
    uint32_t *req_npages;     /* [max_requests] */
    uint32_t *req_chain;      /* [max_requests * max_pages_per_request] KV handles */
    uint32_t *req_ssm;        /* [max_requests * n_ssm_layers] SSM handles */
    uint32_t n_slot_stack[2], n_vid_stack[2];
    avmp_stats stats;
} avmp_tables;

typedef struct avmp_ctx avmp_ctx;

/* Fill *opt with the paper's defaults (thresholds 0.05 / 0.30, interval 1000, migration
 * on) and max_requests = 1024, max_pages_per_request = 4096. */
AVMP_API void avmp_default_options(avmp_options *opt);

/* Section 3.1 arithmetic.  initial_split is the fraction of the pool given to the SSM store
 * at start (the static systems' "mamba ratio").  Returns AVMP_EINVAL on zero units, a split
 * outside [0, 1], a pool too small for one unit, or an id space beyond 31 bits. */
AVMP_API int avmp_derive_layout(const avmp_model_spec *spec, uint64_t pool_bytes, double initial_split,
                       avmp_layout *out);

/* Bytes of workspace avmp_create needs (0 on invalid arguments). */
AVMP_API size_t avmp_workspace_bytes(const avmp_model_spec *spec, uint64_t pool_bytes, const avmp_options *opt);

/* Create a context over a caller-owned arena and workspace and initialise the tables on
 * `stream` (fresh pools hand out slot 0, 1, 2, ... and id 0, 1, 2, ...).
 *   d_arena      >= pool_bytes, 256-byte aligned.  KV slot i lives at byte i * U_kv; SSM slot j
 *                at pool_bytes_aligned - (j + 1) * U_ssm, so each store's high end faces the gap
 *                in the middle and ceded bytes are what the other store grows into.  The arena
 *                is never cleared.
 *   d_workspace  >= avmp_workspace_bytes(...), 256-byte aligned.
 *   migration_batch_size  B: upper bound, in donor units, on one migration (Section 3.1).
 *   opt          NULL = defaults.  threshold_low >= threshold_high is rejected (Section 4.6).
 *                max_requests * max_pages_per_request * max(page_tokens, copy pieces per page) must
 *                stay below 2^32: row offsets (cu_seqlens) and the gathers' piece counts are 32-bit.
 * Returns AVMP_EINVAL / AVMP_ENOSPC (workspace too small) / AVMP_ECUDA. */
AVMP_API int avmp_create(avmp_ctx **out, const avmp_model_spec *spec, void *d_arena, uint64_t pool_bytes,
                double initial_split, uint32_t migration_batch_size, const avmp_options *opt,
                void *d_workspace, size_t workspace_bytes, void *stream);
AVMP_API int avmp_destroy(avmp_ctx *ctx);

/* One engine step (Sections 3.1-3.2): process d_ops[0..n_ops) exactly as if they were applied
 * one at a time in array order -- each op advances the logical counter, allocations pop the
 * LIFO free lists, a shortage runs the CapacityError handler (SSM first, then KV), which may
 * migrate min(B, donor free) donor units when the donor's free fraction exceeds
 * threshold_high and the throttle allows, relocating live units out of the ceded range and
 * remapping their handles; the op is then retried once.  d_status[i] receives AVMP_ST_*.
 * Stream-ordered, no host synchronisation.  n_ops == 0 is a no-op. */
AVMP_API int avmp_step(avmp_ctx *ctx, const avmp_op *d_ops, uint32_t n_ops, uint32_t *d_status, void *stream);

/* avmp_step followed by avmp_translate of d_handles against the tables that step leaves (Sections 3.1-3.2
 * and Figure 1), with the translation riding on the step's relocation-copy launch: two launches per engine
 * step instead of three, which is most of what the allocator part of a step costs (lists of more than 32 768
 * handles, and contexts with migration disabled, take the wide translate kernel as a third launch).  Results
 * are exactly those of the two calls made one after the other.  n_handles == 0 is avmp_step; n_ops == 0 is avmp_translate. */
AVMP_API int avmp_step_translate(avmp_ctx *ctx, const avmp_op *d_ops, uint32_t n_ops, uint32_t *d_status,
                                 const uint32_t *d_handles, uint32_t n_handles, uint32_t *d_pool, uint64_t *d_offset,
                                 uint64_t *d_arena_offset, void *stream);

/* Same step, with the batch length read from device memory when the kernel runs (*d_n_ops, clamped
 * to max_ops): for batches that another kernel builds, so that a serving loop needs no host round
 * trip per step.  max_ops bounds the work the host queues (the number of migration rounds). */
AVMP_API int avmp_step_indirect(avmp_ctx *ctx, const avmp_op *d_ops, const uint32_t *d_n_ops, uint32_t max_ops,
                                uint32_t *d_status, void *stream);

/* Same step with HOST arrays: copies the ops in, runs the step, copies the statuses out
 * and waits for them.  n_ops is limited to 65536 per call. */
AVMP_API int avmp_step_host(avmp_ctx *ctx, const avmp_op *h_ops, uint32_t n_ops, uint32_t *h_status, void *stream);

/* Section 3.1 / Figure 1: resolve handles.  d_pool[i] = pool tag, d_offset[i] = slot * unit
 * bytes (offset inside that store), d_arena_offset[i] (may be NULL) = byte offset of the unit
 * from d_arena.  A handle that does not resolve gives AVMP_INVALID / AVMP_NONE64 and a sticky
 * AVMP_DEV_BAD_HANDLE. */
AVMP_API int avmp_translate(avmp_ctx *ctx, const uint32_t *d_handles, uint32_t n, uint32_t *d_pool,
                   uint64_t *d_offset, uint64_t *d_arena_offset, void *stream);

/* Paged KV gather (Section 2.2 "paged scatter-gather memory lookups") of attention layer
 * `attn_layer` for the request slots d_reqs[0..n_reqs), n_reqs <= max_requests.  Rows are one
 * token's kv_heads x head_dim elements; request k's rows start at d_cu_seqlens[k] (prefix sums
 * of the held lengths, n_reqs + 1 entries, always written).  Only valid tokens are copied
 * (the last page may be partial).  A slot that holds no chain contributes length 0 and a
 * sticky AVMP_DEV_BAD_REQUEST; a request whose rows would pass out_capacity_tokens copies
 * nothing (AVMP_DEV_OUT_OVERFLOW).  Output pointers must be 16-byte aligned.
 * Lists of up to 1024 requests are planned inside the copy kernel (one launch, no shared
 * scratch); longer lists are planned by a kernel of their own into the context's workspace, so
 * KV gathers / scatters with such lists must not overlap on the GPU (keep them on one stream). */
AVMP_API int avmp_gather_kv(avmp_ctx *ctx, uint32_t attn_layer, const uint32_t *d_reqs, uint32_t n_reqs,
                   void *d_out_k, void *d_out_v, uint64_t out_capacity_tokens,
                   uint32_t *d_cu_seqlens, void *stream);

/* SSM gather (Section 2.2 "contiguous read and write access") of SSM layer `ssm_layer`:
 * d_out_state[k] gets the state elements, d_out_conv[k] the convolution window of request
 * d_reqs[k].  Requests must be LIVE; others are skipped with AVMP_DEV_BAD_REQUEST. */
AVMP_API int avmp_gather_ssm(avmp_ctx *ctx, uint32_t ssm_layer, const uint32_t *d_reqs, uint32_t n_reqs,
                    void *d_out_state, void *d_out_conv, void *stream);

/* The two gathers for `n_layers` consecutive layers in ONE launch (same results as calling the
 * single-layer entry once per layer; one launch instead of n_layers removes the per-launch ramp
 * and tail, which is most of what separates a 250 MB gather from the HBM roofline).  Layer
 * first_layer + l writes to the given buffers advanced by l * stride bytes; strides are multiples
 * of 16 and at least one layer's worth (out_capacity_tokens rows for KV, n_reqs blocks for SSM).
 * d_cu_seqlens is shared by all layers. */
AVMP_API int avmp_gather_kv_layers(avmp_ctx *ctx, uint32_t first_layer, uint32_t n_layers, const uint32_t *d_reqs,
                                   uint32_t n_reqs, void *d_out_k, void *d_out_v, uint64_t layer_stride_bytes,
                                   uint64_t out_capacity_tokens, uint32_t *d_cu_seqlens, void *stream);
AVMP_API int avmp_gather_ssm_layers(avmp_ctx *ctx, uint32_t first_layer, uint32_t n_layers, const uint32_t *d_reqs,
                                    uint32_t n_reqs, void *d_out_state, uint64_t state_layer_stride_bytes,
                                    void *d_out_conv, uint64_t conv_layer_stride_bytes, void *stream);

/* Both gathers of an engine step in ONE launch (Section 2.2: the two access patterns, for the
 * same request list): attention layers [first_attn_layer, + n_attn_layers) exactly as
 * avmp_gather_kv_layers, then SSM layers [first_ssm_layer, + n_ssm_layers) exactly as
 * avmp_gather_ssm_layers -- same outputs, same error items (a slot that is KV_ONLY contributes
 * its rows to the KV part and one AVMP_DEV_BAD_REQUEST per SSM layer).  A step that moves only
 * tens of MB is bound by the ramp and tail of its launches; this pays them once.  Both layer
 * counts must be at least 1 (use the single-kind entry points otherwise). */
AVMP_API int avmp_gather_step(avmp_ctx *ctx, const uint32_t *d_reqs, uint32_t n_reqs,
                              uint32_t first_attn_layer, uint32_t n_attn_layers, void *d_out_k, void *d_out_v,
                              uint64_t kv_layer_stride_bytes, uint64_t out_capacity_tokens, uint32_t *d_cu_seqlens,
                              uint32_t first_ssm_layer, uint32_t n_ssm_layers, void *d_out_state,
                              uint64_t state_layer_stride_bytes, void *d_out_conv, uint64_t conv_layer_stride_bytes,
                              void *stream);

/* Write side of the two gathers (what the model's kernels do after a step).  Tokens
 * [d_tok_start[k], len_k) of request k are read from rows cu[k].. of d_in_k / d_in_v, cu being
 * the prefix sum of (len_k - d_tok_start[k]); d_tok_start == NULL means 0. */
AVMP_API int avmp_scatter_kv(avmp_ctx *ctx, uint32_t attn_layer, const uint32_t *d_reqs,
                    const uint32_t *d_tok_start, uint32_t n_reqs, const void *d_in_k,
                    const void *d_in_v, void *stream);
AVMP_API int avmp_scatter_ssm(avmp_ctx *ctx, uint32_t ssm_layer, const uint32_t *d_reqs, uint32_t n_reqs,
                     const void *d_in_state, const void *d_in_conv, void *stream);

/* (No counterpart in the paper: a deployment convenience.)  The same gather as avmp_gather_kv
 * for callers that can neither allocate device memory nor lend the library scratch of their
 * own -- e.g. code running after the process gave the whole card to a memory pool, or a
 * plug-in that is only ever handed device pointers.  Inputs and outputs are still the
 * caller's; the gather's planning arrays live in a fixed array inside the library
 * (about 33 KB per GPU, held until the process exits), which limits the request list to
 * AVMP_STATIC_GATHER_MAX_REQS entries: a longer list returns AVMP_ETOOBIG and does nothing
 * (and, as for avmp_gather_kv, a list longer than max_requests returns AVMP_EINVAL).
 * The context's device must be current.  The array's device address is resolved on the host,
 * once per device: by avmp_create (so that the driver loads the array onto the GPU while the
 * caller still has memory to spare), or else by the first call of this entry point on that
 * device -- make that call (n_reqs = 0 will do) before handing all memory away and before any
 * stream capture.  After a cudaDeviceReset create a new context before calling this again.
 * All calls on a device share the array: calls whose kernels may overlap on the GPU
 * (different streams) race -- keep them on one stream or order them with events.  Results,
 * error items and cu_seqlens are exactly those of avmp_gather_kv. */
#define AVMP_STATIC_GATHER_MAX_REQS 4096
AVMP_API int avmp_gather_kv_static(avmp_ctx *ctx, uint32_t attn_layer, const uint32_t *d_reqs, uint32_t n_reqs,
                                   void *d_out_k, void *d_out_v, uint64_t out_capacity_tokens,
                                   uint32_t *d_cu_seqlens, void *stream);

/* Write side for a range of layers in one launch (layer first_layer + l reads its rows from the
 * buffers advanced by l * stride bytes; rows of a layer are laid out as for the single-layer call). */
AVMP_API int avmp_scatter_kv_layers(avmp_ctx *ctx, uint32_t first_layer, uint32_t n_layers, const uint32_t *d_reqs,
                                    const uint32_t *d_tok_start, uint32_t n_reqs, const void *d_in_k,
                                    const void *d_in_v, uint64_t layer_stride_bytes, void *stream);
AVMP_API int avmp_scatter_ssm_layers(avmp_ctx *ctx, uint32_t first_layer, uint32_t n_layers, const uint32_t *d_reqs,
                                     uint32_t n_reqs, const void *d_in_state, uint64_t state_layer_stride_bytes,
                                     const void *d_in_conv, uint64_t conv_layer_stride_bytes, void *stream);

/* Counters -> host.  Synchronises the stream. */
AVMP_API int avmp_get_stats(avmp_ctx *ctx, avmp_stats *h_out, void *stream);
/* Clear the sticky device error code and count.  Stream-ordered. */
AVMP_API int avmp_clear_error(avmp_ctx *ctx, void *stream);

/* Tables <-> host (parity checks, snapshot / restore).  Both synchronise the stream.
 * Import checks the snapshot on the host first (capacities and pool-byte conservation, free lists
 * distinct and inside their stores, page table and owner table mutually inverse, every handle of
 * every request resolvable and owned once) and returns AVMP_EINVAL, with the context untouched, if
 * it does not hang together: the kernels index these tables without bounds checks. */
AVMP_API int avmp_export_tables(avmp_ctx *ctx, avmp_tables *h_out, void *stream);
AVMP_API int avmp_import_tables(avmp_ctx *ctx, const avmp_tables *h_in, void *stream);

/* ---- on-device closed loop (the paper's harness drives its traces from the host, Section 4.1) ----
 * A device-resident scheduler for queue-type traces: every avmp_driver_step builds the next batch
 * on the GPU (FINISH for requests whose decode is complete, EXTEND by one token for the other
 * running requests, ADMITs from the queue head into the lowest free slots within the concurrency
 * and a slow-start window), runs it through the allocator (avmp_step_indirect) and folds the
 * statuses back into the request slots -- three stream-ordered launches and no host round trip, so
 * a serving loop can be queued (or graph-captured) many steps ahead.  d_prompt / d_output are
 * device arrays of n_requests token counts; the driver's slots are the context's request slots.
 * The workspace (avmp_driver_workspace_bytes(max_requests), 256-byte aligned) is the caller's. */
typedef struct avmp_driver avmp_driver;
typedef struct {
    uint64_t steps, completed, dropped, preempted, n_oom_admit, n_oom_extend;
    uint64_t queue_next;      /* requests taken from the arrays so far */
    uint64_t requeued;        /* entries waiting at the queue head (failed admits, pre-empted requests) */
    uint64_t window;          /* current admission window */
    uint64_t last_batch_ops;
    uint64_t overflow;        /* 1 if the re-queue buffer ever overflowed (entries were lost) */
} avmp_driver_stats;
AVMP_API size_t avmp_driver_workspace_bytes(uint32_t max_requests);
AVMP_API int avmp_driver_create(avmp_driver **out, avmp_ctx *ctx, const uint32_t *d_prompt, const uint32_t *d_output,
                                uint32_t n_requests, uint32_t concurrency, void *d_workspace, size_t workspace_bytes,
                                void *stream);
AVMP_API int avmp_driver_destroy(avmp_driver *drv);
AVMP_API int avmp_driver_step(avmp_driver *drv, void *stream);
/* Both synchronise the stream.  Export copies the per-slot arrays (state 0 free / 1 running, request
 * index, tokens held, decode tokens left), max_requests entries each. */
AVMP_API int avmp_driver_get_stats(avmp_driver *drv, avmp_driver_stats *h_out, void *stream);
AVMP_API int avmp_driver_export(avmp_driver *drv, uint32_t *h_state, uint32_t *h_uid, uint32_t *h_len,
                                uint32_t *h_remaining, void *stream);

/* ---- the same loop for multi-turn sessions (the agentic-burst workload; the paper gives that
 * workload one sentence in Section 4.1 and no scheduler, so the policy is this library's) ----
 * Sessions arrive at d_arrival_step[i] (ascending); turn t of session i appends d_turn_prompt[i *
 * max_turns + t] prompt tokens and decodes d_turn_output[...] tokens; between turns the request
 * parks (FINISH with KEEP_KV) for d_turn_think[i * max_turns + t] steps and then resumes on its own
 * slot (ADMIT with RESUME); after turn d_n_turns[i] - 1 it finishes for good.  Each step admits, in
 * this order, re-queued entries, parked sessions whose think time is over (by ready step, then by
 * parking order) and newly arrived sessions, within the concurrency and the slow-start window;
 * a step that saw an OOM or ran out of free slots evicts the longest-parked chain (that session re-enters with its whole
 * context as the prompt), a step without any success pre-empts the most recently admitted
 * request, an admit that fails with nothing running and nothing parked is dropped.
 * All five arrays are device arrays of uint32 owned by the caller and must outlive the driver;
 * concurrency <= 1024.  The workspace (avmp_session_driver_workspace_bytes, 256-byte aligned) is
 * the caller's.  Each step is one launch plus the relocation copy (a few launches when a batch may
 * hold more than one migration), with no host round trip. */
typedef struct avmp_session_driver avmp_session_driver;
typedef struct {
    uint64_t steps, completed, dropped, preempted, evicted, n_oom_admit, n_oom_extend;
    uint64_t arrived;         /* sessions whose arrival step has passed */
    uint64_t arrival_queue;   /* of those, still waiting for their first admission */
    uint64_t requeued;        /* entries at the queue head (failed admits, pre-empted, found no slot) */
    uint64_t waiting;         /* parked or evicted sessions waiting for their ready step */
    uint64_t window, last_batch_ops;
    uint64_t forced_slot;     /* slot the next step will pre-empt or evict, ~0 if none */
} avmp_session_stats;
AVMP_API size_t avmp_session_driver_workspace_bytes(uint32_t max_requests, uint32_t n_sessions);
AVMP_API int avmp_session_driver_create(avmp_session_driver **out, avmp_ctx *ctx, const uint32_t *d_arrival_step,
                                        const uint32_t *d_n_turns, const uint32_t *d_turn_prompt,
                                        const uint32_t *d_turn_output, const uint32_t *d_turn_think,
                                        uint32_t n_sessions, uint32_t max_turns, uint32_t concurrency,
                                        void *d_workspace, size_t workspace_bytes, void *stream);
AVMP_API int avmp_session_driver_destroy(avmp_session_driver *drv);
AVMP_API int avmp_session_driver_step(avmp_session_driver *drv, void *stream);
/* Both synchronise the stream.  Export copies the per-slot arrays (state 0 free / 1 running / 2
 * parked, session index, tokens held, decode tokens left, turn), max_requests entries each, and the
 * session indices in the re-queued and the waiting queue, in order (room for n_sessions each). */
AVMP_API int avmp_session_driver_get_stats(avmp_session_driver *drv, avmp_session_stats *h_out, void *stream);
AVMP_API int avmp_session_driver_export(avmp_session_driver *drv, uint32_t *h_state, uint32_t *h_uid, uint32_t *h_len,
                                        uint32_t *h_remaining, uint32_t *h_turn, uint32_t *h_requeued,
                                        uint32_t *h_waiting, void *stream);

/* How many kernels this context has launched so far (host counter). */
AVMP_API uint64_t avmp_launch_count(const avmp_ctx *ctx);

AVMP_API const char *avmp_error_string(int code);

#ifdef __cplusplus
}
#endif
#endif
