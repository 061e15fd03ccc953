// avmp_gather_kv_static: the paged KV gather with its planning scratch in a fixed device
// array that lives inside this library, for callers that cannot hand the library any
// scratch memory of their own and cannot allocate any.
//
// Who that is: code that runs after the process has given every byte of device memory to
// a pool it does not control (a serving engine's cache arena, a framework's caching
// allocator that was told to reserve the whole card), plug-ins that receive device pointers
// but are forbidden to call cudaMalloc, and loops that must not allocate because an
// allocation would stall the device mid-step.  They still pass their inputs (the request
// list) and outputs (the batch buffers, the row offsets); only the gather's own working
// arrays -- the per-request row and piece prefix sums that the plan pass hands to the copy
// pass -- come from here instead of from caller-provided scratch.
//
// The scratch is one file-scope __device__ array of a fixed, modest size (see
// AVMP_STATIC_GATHER_MAX_REQS); every GPU that loads this library carries it until the
// process exits.  All calls on a device share it.  The plan pass rewrites every word the
// copy pass reads, so stale contents from an earlier call are harmless and nothing needs
// clearing; but two calls whose kernels overlap on the GPU (different streams) would
// trample each other's scratch and race.
#include "avmp_dev.cuh"

using namespace avmp;

namespace {

constexpr uint32_t kMaxReqs = AVMP_STATIC_GATHER_MAX_REQS;
constexpr uint32_t kRowsOff = 0;                     // [0, kMaxReqs]           first output row per request
constexpr uint32_t kItemsOff = kMaxReqs + 1;         // [.., 2 * kMaxReqs + 1]  first work item per request
constexpr uint32_t kTotalOff = 2 * (kMaxReqs + 1);   // number of work items
constexpr uint32_t kScratchWords = kTotalOff + 2;

// In host code this name is only a stand-in for the symbol: never pass it to a kernel.
// The device address is fetched once per device with cudaGetSymbolAddress (below).
static __device__ __align__(256) uint32_t g_static_gather_scratch[kScratchWords];

constexpr int kThreads = 256;

// One CTA: held length of every request -> exclusive prefix sums of rows and of work items
// (an item is `tpi` consecutive rows of one request).
__global__ void __launch_bounds__(kStepThreads)
static_plan_kernel(const Geom g, uint32_t *scratch, const uint32_t *reqs,
                   uint32_t n, uint32_t tpi, uint32_t *cu_out)
{
    __shared__ unsigned long long tmp[32];
    unsigned long long run_rows = 0, run_items = 0, tot;
    const int tid = threadIdx.x;
    pdl_prologue();
    for (uint32_t b = 0; b < n; b += kStepThreads) {
        const uint32_t k = b + tid;
        uint32_t rows = 0;
        if (k < n) {
            const uint32_t r = reqs[k];
            const uint32_t st = r < g.R ? g.r_state[r] : AVMP_REQ_EMPTY;
            if (st == AVMP_REQ_EMPTY) record_error(g.st, AVMP_DEV_BAD_REQUEST);
            else rows = g.r_len[r];
        }
        const uint32_t items = (rows + tpi - 1) / tpi;
        const unsigned long long incl = block_incl_scan(((unsigned long long)items << 32) | rows, tmp, &tot);
        if (k < n) {
            const uint32_t ex_rows = (uint32_t)(run_rows + (uint32_t)incl - rows);
            scratch[kRowsOff + k] = ex_rows;
            scratch[kItemsOff + k] = (uint32_t)(run_items + (uint32_t)(incl >> 32) - items);
            cu_out[k] = ex_rows;
        }
        run_rows += (uint32_t)tot;
        run_items += (uint32_t)(tot >> 32);
    }
    if (tid == 0) {
        scratch[kRowsOff + n] = (uint32_t)run_rows;
        scratch[kItemsOff + n] = (uint32_t)run_items;
        scratch[kTotalOff] = (uint32_t)run_items;
        cu_out[n] = (uint32_t)run_rows;
    }
}

__device__ __forceinline__ void warp_copy_bytes(uint8_t *dst, const uint8_t *src, uint32_t bytes, int lane)
{
    if ((((uintptr_t)dst | (uintptr_t)src | bytes) & 15u) == 0) {
        const uint4 *s = reinterpret_cast<const uint4 *>(src);
        uint4 *d = reinterpret_cast<uint4 *>(dst);
        for (uint32_t i = lane; i < (bytes >> 4); i += 32u) d[i] = s[i];
    } else {
        for (uint32_t i = lane; i < bytes; i += 32u) dst[i] = src[i];
    }
}

// Warps walk the items grid-strided; rows of an item that share a page are one contiguous
// run in the page and in the batch buffer.
__global__ void __launch_bounds__(kThreads)
static_gather_kernel(const Geom g, const uint32_t *scratch, const uint32_t layer,
                     const uint32_t *reqs, const uint32_t n, const uint32_t tpi,
                     uint8_t *out_k, uint8_t *out_v, const unsigned long long cap_tokens)
{
    pdl_prologue();
    const uint32_t *cu_rows = scratch + kRowsOff, *cu_items = scratch + kItemsOff;
    const uint32_t total = scratch[kTotalOff];
    const int lane = threadIdx.x & 31;
    const uint32_t row = (uint32_t)g.row_bytes, T = g.T;
    const unsigned long long layer_off = (unsigned long long)layer * g.kv_layer_bytes;
    const unsigned long long v_off = (unsigned long long)T * row;
    const uint32_t nw = gridDim.x * (kThreads / 32);
    for (uint32_t it = (threadIdx.x >> 5) * gridDim.x + blockIdx.x; it < total; it += nw) {
        const uint32_t k = find_owner(cu_items, 0u, n, 0u, it);
        const uint32_t row0 = cu_rows[k], rows = cu_rows[k + 1] - row0;
        if ((unsigned long long)row0 + rows > cap_tokens) {
            if (it == cu_items[k] && lane == 0) record_error(g.st, AVMP_DEV_OUT_OVERFLOW);
            continue;
        }
        const uint32_t r = reqs[k];
        const uint32_t i0 = (it - cu_items[k]) * tpi;
        const uint32_t cnt = min(tpi, rows - i0);
        uint32_t done = 0;
        while (done < cnt) {
            const uint32_t t = i0 + done;
            const uint32_t in_page = min(cnt - done, T - t % T);
            const uint32_t h = g.r_chain[(unsigned long long)r * g.max_pages + t / T];
            const uint32_t slot = g.VT[0][h & 0x7FFFFFFFu];
            const uint8_t *pk = g.arena + (unsigned long long)slot * g.U[0] + layer_off + (unsigned long long)(t % T) * row;
            const unsigned long long o = ((unsigned long long)row0 + t) * row;
            warp_copy_bytes(out_k + o, pk, in_page * row, lane);
            warp_copy_bytes(out_v + o, pk + v_off, in_page * row, lane);
            done += in_page;
        }
    }
}

// Device address of the scratch array, per device.
uint32_t *g_scratch_addr[64] = {};

}  // namespace

// Resolve the array's address on the current device.  Under CUDA's lazy module loading this is
// also the moment the driver loads this file's code and the array onto the GPU, so it is done
// when a context is created -- while the caller can still spare the memory -- and again by the
// entry point if that did not happen.  Re-resolved at every avmp_create: after a cudaDeviceReset
// the old address is stale, and so is every context made before the reset.
cudaError_t avmp::static_gather_setup(int dev)
{
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    void *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_gather_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = static_cast<uint32_t *>(p);
    return cudaSuccess;
}

extern "C" AVMP_API int avmp_gather_kv_static(avmp_ctx *c, uint32_t layer, const uint32_t *d_reqs, uint32_t n,
                                              void *d_out_k, void *d_out_v, uint64_t cap_tokens,
                                              uint32_t *d_cu, void *stream)
{
    if (!c || layer >= c->spec.n_attn_layers || !d_cu) return AVMP_EINVAL;
    if (n > kMaxReqs) return AVMP_ETOOBIG;            // the fixed scratch cannot plan a longer list
    if (n > c->opt.max_requests) return AVMP_EINVAL;  // as avmp_gather_kv: a list is no longer than the slot table
    if (n && (!d_reqs || !d_out_k || !d_out_v)) return AVMP_EINVAL;
    if (((uintptr_t)d_out_k | (uintptr_t)d_out_v) & 15) return AVMP_EINVAL;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return AVMP_ECUDA;
    if (dev != c->device || dev < 0 || dev >= 64) return AVMP_EINVAL;   // the context's device must be current
    // Normally resolved by avmp_create; a context made on another device's turn gets it here.
    if (!g_scratch_addr[dev] && static_gather_setup(dev) != cudaSuccess) return AVMP_ECUDA;
    uint32_t *scratch = g_scratch_addr[dev];
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    uint32_t tpi = (uint32_t)(4096 / (c->g.row_bytes ? c->g.row_bytes : 1));
    if (tpi < 1) tpi = 1;
    if (tpi > c->g.T) tpi = c->g.T;
    if (launch_pdl(static_plan_kernel, dim3(1), dim3(kStepThreads), 0, s, c->g, scratch, d_reqs, n, tpi, d_cu) != cudaSuccess)
        return AVMP_ECUDA;
    if (launch_pdl(static_gather_kernel, dim3(c->n_sms * 4), dim3(kThreads), 0, s, c->g, (const uint32_t *)scratch, layer,
                   d_reqs, n, tpi, static_cast<uint8_t *>(d_out_k), static_cast<uint8_t *>(d_out_v),
                   (unsigned long long)cap_tokens) != cudaSuccess)
        return AVMP_ECUDA;
    c->launches += 2;
    return AVMP_OK;
}
