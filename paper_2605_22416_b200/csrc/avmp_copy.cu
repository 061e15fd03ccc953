// Bandwidth kernels of the AVMP path: handle translation, the relocation copy of a
// migration (paper Section 3.2; the paper's prototype copies nothing, this build keeps one
// arena and really moves live units), and the paged KV / contiguous SSM gathers and their
// write sides (Section 2.2).  No arithmetic on payload: bytes in, bytes out.
//
// All of them are HBM-bound streaming copies.  Work is cut into warp-sized items of a few
// KiB; consecutive warps take consecutive items, so a CTA streams one contiguous span.
// Every lane keeps several 16-byte loads in flight before the first store.
#include "avmp_dev.cuh"

namespace avmp {

namespace {

constexpr int kCopyThreads = 256;
constexpr int kCtasPerSm = 8;
constexpr uint32_t kChunk = 8192;      // bytes per warp item for contiguous copies

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4 *p, const uint4 &v)
{
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// One warp copies `bytes` (any size) from src to dst.  16-byte vectors when both ends and
// the size allow, single bytes otherwise (only toy shapes take that path).
template <int UNROLL>
__device__ __forceinline__ void warp_copy(uint8_t *dst, const uint8_t *src, uint32_t bytes, int lane)
{
    if ((((uintptr_t)dst | (uintptr_t)src | bytes) & 15u) == 0) {
        const uint4 *s = reinterpret_cast<const uint4 *>(src);
        uint4 *d = reinterpret_cast<uint4 *>(dst);
        const uint32_t nvec = bytes >> 4;
        uint32_t i = lane;
        for (; i + 32u * (UNROLL - 1) < nvec; i += 32u * UNROLL) {
            uint4 v[UNROLL];
#pragma unroll
            for (int k = 0; k < UNROLL; ++k) v[k] = ld_stream(s + i + 32u * k);
#pragma unroll
            for (int k = 0; k < UNROLL; ++k) st_stream(d + i + 32u * k, v[k]);
        }
        for (; i < nvec; i += 32u) st_stream(d + i, ld_stream(s + i));
    } else {
        for (uint32_t i = lane; i < bytes; i += 32u) dst[i] = src[i];
    }
}

// ---- a10: translate ------------------------------------------------------------------
__global__ void translate_kernel(const Geom g, const uint32_t *__restrict__ h, uint32_t n,
                                 uint32_t *__restrict__ pool, unsigned long long *__restrict__ off,
                                 unsigned long long *__restrict__ aoff)
{
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const uint32_t hv = h[i], p = hv >> 31, vid = hv & 0x7FFFFFFFu;
        uint32_t slot = kInvalid;
        if (hv != kInvalid && vid < g.V[p]) slot = g.VT[p][vid];
        if (slot == kInvalid) {
            pool[i] = kInvalid; off[i] = kNone64;
            if (aoff) aoff[i] = kNone64;
            record_error(g.st, AVMP_DEV_BAD_HANDLE);
        } else {
            pool[i] = p; off[i] = (unsigned long long)slot * g.U[p];
            if (aoff) aoff[i] = (unsigned long long)(unit_ptr(g, p, slot) - g.arena);
        }
    }
}

// ---- a7: relocation copy of the last migration -----------------------------------------
__global__ void __launch_bounds__(kCopyThreads) relocate_kernel(const Geom g)
{
    const uint32_t n = g.st->n_reloc;
    if (n == 0) return;
    const uint32_t pool = g.st->reloc_pool;
    const unsigned long long U = g.U[pool];
    const uint32_t per = (uint32_t)((U + kChunk - 1) / kChunk);
    const unsigned long long total = (unsigned long long)n * per;
    const int lane = threadIdx.x & 31;
    const unsigned long long nw = (unsigned long long)gridDim.x * (kCopyThreads / 32);
    for (unsigned long long it = (unsigned long long)blockIdx.x * (kCopyThreads / 32) + (threadIdx.x >> 5);
         it < total; it += nw) {
        const uint32_t k = (uint32_t)(it / per), c = (uint32_t)(it % per);
        const unsigned long long o = (unsigned long long)c * kChunk;
        const uint32_t bytes = (uint32_t)min((unsigned long long)kChunk, U - o);
        // dst < new capacity <= src: ranges never overlap
        warp_copy<8>(unit_ptr(g, pool, g.reloc_dst[k]) + o, unit_ptr(g, pool, g.reloc_src[k]) + o, bytes, lane);
    }
}

// ---- a11: KV gather / scatter ---------------------------------------------------------
// Plan: one CTA turns the request list into row prefix sums (cu_seqlens) and item prefix
// sums; an item is `tpi` consecutive rows of one request.
__global__ void __launch_bounds__(kStepThreads)
kv_plan_kernel(const Geom g, const uint32_t *__restrict__ reqs, const uint32_t *__restrict__ tok_start,
               uint32_t n, uint32_t tpi, uint32_t *__restrict__ cu_out)
{
    __shared__ unsigned long long tmp[32];
    unsigned long long run_rows = 0, run_items = 0, tot;
    const int tid = threadIdx.x;
    for (uint32_t b = 0; b < n; b += kStepThreads) {
        const uint32_t k = b + tid;
        uint32_t rows = 0;
        if (k < n) {
            const uint32_t r = reqs[k];
            const uint32_t st = r < g.R ? g.r_state[r] : AVMP_REQ_EMPTY;
            const uint32_t t0 = tok_start ? tok_start[k] : 0u;
            if (st == AVMP_REQ_EMPTY) record_error(g.st, AVMP_DEV_BAD_REQUEST);
            else {
                const uint32_t len = g.r_len[r];
                if (t0 > len) record_error(g.st, AVMP_DEV_BAD_REQUEST);
                else rows = len - t0;
            }
        }
        const uint32_t items = (rows + tpi - 1) / tpi;
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

template <bool SCATTER>
__global__ void __launch_bounds__(kCopyThreads)
kv_copy_kernel(const Geom g, const uint32_t layer, const uint32_t *__restrict__ reqs,
               const uint32_t *__restrict__ tok_start, const uint32_t n, const uint32_t tpi,
               uint8_t *__restrict__ buf_k, uint8_t *__restrict__ buf_v, const unsigned long long cap_tokens)
{
    const uint32_t total = g.st->g_total_items;
    const int lane = threadIdx.x & 31;
    const uint32_t row = (uint32_t)g.row_bytes, T = g.T;
    const unsigned long long layer_off = (unsigned long long)layer * g.kv_layer_bytes;
    const unsigned long long v_off = (unsigned long long)T * row;
    const uint32_t nw = gridDim.x * (kCopyThreads / 32);
    for (uint32_t it = blockIdx.x * (kCopyThreads / 32) + (threadIdx.x >> 5); it < total; it += nw) {
        // request of this item: largest k with cu_items[k] <= it
        const uint32_t k = find_owner(g.g_cu_items, 0u, n, 0u, it);
        const uint32_t r = reqs[k];
        const uint32_t row0 = g.g_cu_rows[k], rows = g.g_cu_rows[k + 1] - row0;
        if (!SCATTER && (unsigned long long)row0 + rows > cap_tokens) {
            if (it == g.g_cu_items[k] && lane == 0) record_error(g.st, AVMP_DEV_OUT_OVERFLOW);
            continue;
        }
        const uint32_t i0 = (it - g.g_cu_items[k]) * tpi;          // first row of the item, request-relative
        const uint32_t cnt = min(tpi, rows - i0);
        const uint32_t t0 = (tok_start ? tok_start[k] : 0u) + i0;  // its token index
        // rows of one item that share a page are contiguous in the page and in the buffer
        uint32_t done = 0;
        while (done < cnt) {
            const uint32_t t = t0 + done;
            const uint32_t in_page = min(cnt - done, T - t % T);
            const uint32_t h = g.r_chain[(unsigned long long)r * g.max_pages + t / T];
            const uint32_t slot = g.VT[0][h & 0x7FFFFFFFu];
            uint8_t *pk = g.arena + (unsigned long long)slot * g.U[0] + layer_off + (unsigned long long)(t % T) * row;
            uint8_t *bk = buf_k + ((unsigned long long)row0 + i0 + done) * row;
            uint8_t *bv = buf_v + ((unsigned long long)row0 + i0 + done) * row;
            const uint32_t bytes = in_page * row;
            if (SCATTER) { warp_copy<4>(pk, bk, bytes, lane); warp_copy<4>(pk + v_off, bv, bytes, lane); }
            else         { warp_copy<4>(bk, pk, bytes, lane); warp_copy<4>(bv, pk + v_off, bytes, lane); }
            done += in_page;
        }
    }
}

// ---- a12: SSM gather / scatter ----------------------------------------------------------
template <bool SCATTER>
__global__ void __launch_bounds__(kCopyThreads)
ssm_copy_kernel(const Geom g, const uint32_t layer, const uint32_t *__restrict__ reqs, const uint32_t n,
                uint8_t *__restrict__ buf_state, uint8_t *__restrict__ buf_conv)
{
    const unsigned long long sb = g.state_bytes, cb = g.conv_bytes;
    const uint32_t ps = (uint32_t)((sb + kChunk - 1) / kChunk), pc = (uint32_t)((cb + kChunk - 1) / kChunk);
    const uint32_t per = ps + pc;
    const unsigned long long total = (unsigned long long)n * per;
    const int lane = threadIdx.x & 31;
    const unsigned long long nw = (unsigned long long)gridDim.x * (kCopyThreads / 32);
    for (unsigned long long it = (unsigned long long)blockIdx.x * (kCopyThreads / 32) + (threadIdx.x >> 5);
         it < total; it += nw) {
        const uint32_t k = (uint32_t)(it / per), c = (uint32_t)(it % per);
        const uint32_t r = reqs[k];
        uint32_t slot = kInvalid;
        if (r < g.R && g.r_state[r] == AVMP_REQ_LIVE) {
            const uint32_t h = g.r_ssm[(unsigned long long)r * g.ns + layer];
            if (h != kInvalid) slot = g.VT[1][h & 0x7FFFFFFFu];
        }
        if (slot == kInvalid) {
            if (c == 0 && lane == 0) record_error(g.st, AVMP_DEV_BAD_REQUEST);
            continue;
        }
        uint8_t *blk = unit_ptr(g, AVMP_POOL_SSM, slot);
        uint8_t *p, *b;
        uint32_t bytes;
        if (c < ps) {
            const unsigned long long o = (unsigned long long)c * kChunk;
            p = blk + o; b = buf_state + (unsigned long long)k * sb + o;
            bytes = (uint32_t)min((unsigned long long)kChunk, sb - o);
        } else {
            const unsigned long long o = (unsigned long long)(c - ps) * kChunk;
            p = blk + sb + o; b = buf_conv + (unsigned long long)k * cb + o;
            bytes = (uint32_t)min((unsigned long long)kChunk, cb - o);
        }
        if (SCATTER) warp_copy<8>(p, b, bytes, lane);
        else         warp_copy<8>(b, p, bytes, lane);
    }
}

}  // namespace

cudaError_t launch_relocate(const Geom &g, const Launch &l)
{
    relocate_kernel<<<l.n_sms * kCtasPerSm, kCopyThreads, 0, l.stream>>>(g);
    return cudaGetLastError();
}

cudaError_t launch_translate(const Geom &g, const uint32_t *h, uint32_t n, uint32_t *pool,
                             unsigned long long *off, unsigned long long *aoff, const Launch &l)
{
    const int blocks = (int)min((unsigned long long)l.n_sms * 4, ((unsigned long long)n + 255) / 256);
    translate_kernel<<<blocks, 256, 0, l.stream>>>(g, h, n, pool, off, aoff);
    return cudaGetLastError();
}

cudaError_t launch_kv(const Geom &g, bool scatter, uint32_t layer, const uint32_t *reqs,
                      const uint32_t *tok_start, uint32_t n, void *k, void *v,
                      unsigned long long cap_tokens, uint32_t *cu_out, const Launch &l)
{
    // rows per warp item: about 4 KiB of K and as much of V
    uint32_t tpi = (uint32_t)(4096 / (g.row_bytes ? g.row_bytes : 1));
    if (tpi < 1) tpi = 1;
    if (tpi > g.T) tpi = g.T;
    kv_plan_kernel<<<1, kStepThreads, 0, l.stream>>>(g, reqs, tok_start, n, tpi, cu_out);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int grid = l.n_sms * kCtasPerSm;
    if (scatter)
        kv_copy_kernel<true><<<grid, kCopyThreads, 0, l.stream>>>(g, layer, reqs, tok_start, n, tpi,
                                                                 (uint8_t *)k, (uint8_t *)v, cap_tokens);
    else
        kv_copy_kernel<false><<<grid, kCopyThreads, 0, l.stream>>>(g, layer, reqs, tok_start, n, tpi,
                                                                  (uint8_t *)k, (uint8_t *)v, cap_tokens);
    return cudaGetLastError();
}

cudaError_t launch_ssm(const Geom &g, bool scatter, uint32_t layer, const uint32_t *reqs, uint32_t n,
                       void *state, void *conv, const Launch &l)
{
    const int grid = l.n_sms * kCtasPerSm;
    if (scatter)
        ssm_copy_kernel<true><<<grid, kCopyThreads, 0, l.stream>>>(g, layer, reqs, n, (uint8_t *)state, (uint8_t *)conv);
    else
        ssm_copy_kernel<false><<<grid, kCopyThreads, 0, l.stream>>>(g, layer, reqs, n, (uint8_t *)state, (uint8_t *)conv);
    return cudaGetLastError();
}

}  // namespace avmp
