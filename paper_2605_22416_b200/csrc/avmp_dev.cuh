// Device-side state, geometry and small block/warp primitives shared by the AVMP kernels.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

#include "avmp.h"

namespace avmp {

constexpr uint32_t kInvalid = 0xFFFFFFFFu;
constexpr unsigned long long kNone64 = 0xFFFFFFFFFFFFFFFFull;
constexpr uint32_t kStage = 16384;           // bytes per piece of a streaming copy (one ring stage)
constexpr uint32_t kLocalPlanMax = 1024;    // longest request list a KV copy plans inside its own CTAs
constexpr int kStepThreads = 1024;          // one CTA plans a step; one op per thread per window
constexpr uint32_t kHostStepMaxOps = 65536; // staging capacity of avmp_step_host

// Mutable allocator state, resident in the workspace (one instance per context).
struct DevState {
    unsigned long long op_counter, last_rebalance_op, n_oom, n_capacity_error, n_rebalance;
    unsigned long long migrated_bytes, wasted_bytes, relocated_blocks, relocated_bytes, gap_bytes;
    unsigned long long n_invalid, error_code, error_count;
    unsigned long long reloc_t0, reloc_t1, reloc_ns_total;   // device clock around relocation copies
    unsigned long long cyc_total, cyc_oom, cyc_mig;          // SM cycles of the step kernel, by bucket
    uint32_t cap[2], n_free[2], n_vfree[2], fsm;
    uint32_t resume_idx;     // ops of the batch in flight already applied (multi-round steps)
    uint32_t n_reloc;        // relocation list of the last round
    uint32_t reloc_pool;
    uint32_t g_total_items;  // work items of the gather / scatter being planned
    uint32_t reloc_pending;  // reloc_t0 / reloc_t1 hold a copy not yet added to reloc_ns_total
};

// Immutable geometry + table pointers, passed to kernels by value.
struct Geom {
    unsigned long long P_al, U[2], kv_layer_bytes, row_bytes, state_bytes, conv_bytes, min_interval;
    uint32_t V[2];
    uint32_t T, na, ns, R, max_pages, B, th_low, th_high, migration_enabled, reclaim_gap;
    uint8_t *arena;
    DevState *st;
    uint32_t *S[2], *W[2], *VT[2], *OW[2];
    uint32_t *r_state, *r_len, *r_npages, *r_chain, *r_ssm;
    uint32_t *reloc_src, *reloc_dst;
    uint32_t *g_cu_items, *g_cu_rows;   // gather scratch, R + 1 entries each
};

// Byte address of a unit: KV slots grow up from the arena base, SSM slots grow down
// from its end, so both stores shrink and grow at the gap between them.
__device__ __forceinline__ uint8_t *unit_ptr(const Geom &g, uint32_t pool, uint32_t slot)
{
    return pool == AVMP_POOL_KV ? g.arena + (unsigned long long)slot * g.U[0]
                                : g.arena + (g.P_al - ((unsigned long long)slot + 1ull) * g.U[1]);
}

__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void record_error(DevState *st, unsigned long long code)
{
    atomicCAS(&st->error_code, 0ull, code);
    atomicAdd(&st->error_count, 1ull);
}

// Table reads of the copy kernels (request list, request records, chains, page table): a few KB that every
// launch needs first, in the middle of GBs of payload streaming through L2.  They are read with an L2
// evict-last policy so that the next launch finds them in L2 instead of paying DRAM latency three or four
// times in a row before its first copy can be issued.
__device__ __forceinline__ unsigned long long l2_policy_evict_last()
{
    unsigned long long p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint32_t ld_keep(const uint32_t *ptr, unsigned long long policy)
{
    uint32_t v;
    asm volatile("ld.global.L2::cache_hint.u32 %0, [%1], %2;" : "=r"(v) : "l"(ptr), "l"(policy) : "memory");
    return v;
}

// ---- warp / block primitives (blockDim.x == kStepThreads for the block ones) ----
__device__ __forceinline__ unsigned long long warp_incl_scan(unsigned long long v)
{
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long n = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v += n;
    }
    return v;
}

// Inclusive scan over the whole block; *total receives the block sum.  `tmp` is 32
// words of shared memory; the call ends with a barrier so `tmp` can be reused at once.
__device__ __forceinline__ unsigned long long block_incl_scan(unsigned long long v, unsigned long long *tmp,
                                                              unsigned long long *total)
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    v = warp_incl_scan(v);
    if (lane == 31) tmp[wid] = v;
    __syncthreads();
    if (wid == 0) {
        unsigned long long w = (lane < (int)(blockDim.x >> 5)) ? tmp[lane] : 0ull;
        tmp[lane] = warp_incl_scan(w);
    }
    __syncthreads();
    const unsigned long long off = wid ? tmp[wid - 1] : 0ull;
    *total = tmp[31];
    __syncthreads();
    return v + off;
}

__device__ __forceinline__ uint32_t block_min(uint32_t v, uint32_t *tmp)
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    v = __reduce_min_sync(0xFFFFFFFFu, v);
    if (lane == 0) tmp[wid] = v;
    __syncthreads();
    uint32_t w = (lane < (int)(blockDim.x >> 5)) ? tmp[lane] : 0xFFFFFFFFu;
    w = __reduce_min_sync(0xFFFFFFFFu, w);
    __syncthreads();
    return w;
}

// Largest idx in [lo, hi) with a[idx] - base <= u   (a is non-decreasing, a[lo] - base <= u).
__device__ __forceinline__ uint32_t find_owner(const uint32_t *a, uint32_t lo, uint32_t hi, uint32_t base,
                                               uint32_t u)
{
    while (lo + 1 < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        if (a[mid] - base <= u) lo = mid; else hi = mid;
    }
    return lo;
}

// ---- programmatic dependent launch ------------------------------------------------------
// Every kernel of the library is launched through launch_pdl and starts with pdl_prologue(): it lets the next kernel in the stream
// be scheduled at once (its CTAs become resident as resources free up and its launch latency is
// hidden), then waits until everything before it in the stream has completed and is visible.
// No global memory is touched before the wait, so stream order is preserved exactly; launched
// without the attribute the two instructions do nothing.
// Because a kernel may be resident while its predecessor still writes, no kernel reads its inputs
// through the read-only (non-coherent) path: kernel pointer parameters are not `const __restrict__`.
// (A gather that read its plan that way saw the previous call's plan.)
__device__ __forceinline__ void pdl_prologue()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                              Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Pieces a KV copy cuts one page of one layer into: K slices, then V slices.
inline uint32_t kv_pieces_per_page(const avmp_layout &lay, uint32_t page_tokens)
{
    const unsigned long long part = (unsigned long long)page_tokens * lay.kv_row_bytes;
    return 2u * (uint32_t)((part + kStage - 1) / kStage);
}

// Host-side launch wrappers (defined next to their kernels).
struct Launch {
    cudaStream_t stream;
    int n_sms;
    int device;
};
cudaError_t launch_init(const Geom &g, const DevState &init, cudaStream_t s);
cudaError_t launch_step(const Geom &g, const avmp_op *d_ops, uint32_t n_ops, const uint32_t *d_n_ops,
                        uint32_t *d_status, int first_round, cudaStream_t s);
cudaError_t launch_relocate(const Geom &g, const Launch &l);
cudaError_t launch_relocate_translate(const Geom &g, const uint32_t *h, uint32_t n, uint32_t *pool,
                                      unsigned long long *off, unsigned long long *aoff, const Launch &l);
cudaError_t launch_translate(const Geom &g, const uint32_t *h, uint32_t n, uint32_t *pool,
                             unsigned long long *off, unsigned long long *aoff, const Launch &l);
cudaError_t launch_kv(const Geom &g, bool scatter, uint32_t layer0, uint32_t n_layers, const uint32_t *reqs,
                      const uint32_t *tok_start, uint32_t n, void *k, void *v, unsigned long long layer_stride,
                      unsigned long long cap_tokens, uint32_t *cu_out, const Launch &l);
cudaError_t launch_ssm(const Geom &g, bool scatter, uint32_t layer0, uint32_t n_layers, const uint32_t *reqs, uint32_t n,
                       void *state, unsigned long long state_stride, void *conv, unsigned long long conv_stride,
                       const Launch &l);
cudaError_t launch_step_gather(const Geom &g, const uint32_t *reqs, uint32_t n, uint32_t kv_layer0, uint32_t kv_layers,
                               void *k, void *v, unsigned long long kv_layer_stride, unsigned long long cap_tokens,
                               uint32_t *cu_out, uint32_t ssm_layer0, uint32_t ssm_layers, void *state,
                               unsigned long long state_stride, void *conv, unsigned long long conv_stride, const Launch &l);
// Resolves the in-library scratch of avmp_gather_kv_static on the current device (= dev).
cudaError_t static_gather_setup(int dev);

}  // namespace avmp

// The context behind the opaque avmp_ctx handle: a small host struct over the caller's arena
// and workspace (global namespace: it is the C ABI's handle type).
struct avmp_ctx {
    avmp::Geom g;
    avmp_model_spec spec;
    avmp_options opt;
    avmp_layout lay;
    uint32_t B;
    int n_sms;
    int device;
    int sm_khz;          // nominal SM clock, to turn the step kernel's cycle counts into time
    uint64_t launches;
    // staging for avmp_step_host, inside the workspace
    avmp_op *d_stage_ops;
    uint32_t *d_stage_status;
    size_t workspace_bytes;
    void *d_workspace;
};

