// A caller of the C ABI that uses nothing but the CUDA runtime: cudaMalloc'd arena and workspace,
// a stream of its own, host arrays copied by hand.  It runs a few engine steps on a PR1-shaped cache
// small enough to force a migration that relocates live pages, writes a byte pattern through avmp_scatter_kv / avmp_scatter_ssm,
// gathers it back and prints statuses, counters and a hash of the gathered bytes, one "key=value" per
// line; the test compares them with the oracle fed the same ops and the same pattern.
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>

#include <cuda_runtime.h>

#include "avmp.h"

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("cuda_error=%s\n", cudaGetErrorString(e_)); return 2; } } while (0)
#define AV(x) do { int r_ = (x); if (r_ != AVMP_OK) { printf("avmp_error=%s at line %d\n", avmp_error_string(r_), __LINE__); return 3; } } while (0)

static uint64_t fnv(const std::vector<uint8_t> &v, uint64_t h = 1469598103934665603ull)
{
    for (uint8_t b : v) { h ^= b; h *= 1099511628211ull; }
    return h;
}

int main()
{
    avmp_model_spec m = {4, 12, 16, 8, 128, 2, 2048 * 16, 2048 * 3, 4};
    const uint64_t pool = 24ull << 20;
    avmp_options o;
    avmp_default_options(&o);
    o.max_requests = 16; o.max_pages_per_request = 48; o.min_rebalance_interval_ops = 4;
    avmp_layout lay;
    AV(avmp_derive_layout(&m, pool, 0.5, &lay));
    const size_t ws_bytes = avmp_workspace_bytes(&m, pool, &o);
    void *arena = nullptr, *ws = nullptr;
    CK(cudaMalloc(&arena, pool));
    CK(cudaMalloc(&ws, ws_bytes));
    cudaStream_t s;
    CK(cudaStreamCreate(&s));
    avmp_ctx *ctx = nullptr;
    AV(avmp_create(&ctx, &m, arena, pool, 0.5, 6, &o, ws, ws_bytes, s));

    // a long request fills the low KV slots and leaves; the next ones land on the top of the free
    // list, i.e. in the highest slots; then the SSM store runs dry and the KV store has to cede exactly
    // those slots: the migration relocates their live pages
    std::vector<std::vector<avmp_op>> batches = {
        {{AVMP_OP_ADMIT, 0, 0, 0, 736}, {AVMP_OP_ADMIT, 0, 0, 1, 16}},
        {{AVMP_OP_FINISH, 0, 0, 0, 0}, {AVMP_OP_ADMIT, 0, 0, 2, 16}, {AVMP_OP_ADMIT, 0, 0, 3, 20}, {AVMP_OP_ADMIT, 0, 0, 4, 5},
         {AVMP_OP_ADMIT, 0, 0, 5, 16}, {AVMP_OP_ADMIT, 0, 0, 6, 16}, {AVMP_OP_EXTEND, 0, 0, 9, 5}, {AVMP_OP_ADMIT, 0, 0, 6, 1}},
    };
    avmp_op *d_ops = nullptr;
    uint32_t *d_st = nullptr;
    CK(cudaMalloc(&d_ops, 64 * sizeof(avmp_op)));
    CK(cudaMalloc(&d_st, 64 * 4));
    printf("statuses=");
    for (auto &b : batches) {
        CK(cudaMemcpyAsync(d_ops, b.data(), b.size() * sizeof(avmp_op), cudaMemcpyHostToDevice, s));
        AV(avmp_step(ctx, d_ops, (uint32_t)b.size(), d_st, s));
        std::vector<uint32_t> st(b.size());
        CK(cudaMemcpyAsync(st.data(), d_st, b.size() * 4, cudaMemcpyDeviceToHost, s));
        CK(cudaStreamSynchronize(s));
        for (uint32_t x : st) printf("%u,", x);
    }
    printf("\n");

    // payload: request r, layer 1, token t, byte i of K = r * 131 + t * 7 + i (mod 256), V = K ^ 0x5A;
    // SSM layer 2: state byte i = r * 17 + i * 3, conv byte i = ~(r * 17 + i * 3)
    const uint32_t reqs_h[] = {3, 1, 2};
    const uint32_t lens_h[] = {20, 16, 16};
    const uint32_t n = 3, row = (uint32_t)lay.kv_row_bytes;
    uint32_t tot = 0;
    for (uint32_t l : lens_h) tot += l;
    std::vector<uint8_t> k((size_t)tot * row), v((size_t)tot * row);
    size_t off = 0;
    for (uint32_t q = 0; q < n; ++q)
        for (uint32_t t = 0; t < lens_h[q]; ++t)
            for (uint32_t i = 0; i < row; ++i, ++off) { k[off] = (uint8_t)(reqs_h[q] * 131 + t * 7 + i); v[off] = k[off] ^ 0x5A; }
    std::vector<uint8_t> st_bytes((size_t)n * lay.ssm_state_bytes), cv_bytes((size_t)n * lay.ssm_conv_bytes);
    for (uint32_t q = 0; q < n; ++q) {
        for (uint64_t i = 0; i < lay.ssm_state_bytes; ++i) st_bytes[q * lay.ssm_state_bytes + i] = (uint8_t)(reqs_h[q] * 17 + i * 3);
        for (uint64_t i = 0; i < lay.ssm_conv_bytes; ++i) cv_bytes[q * lay.ssm_conv_bytes + i] = (uint8_t)~(reqs_h[q] * 17 + i * 3);
    }
    uint32_t *d_reqs = nullptr, *d_zero = nullptr, *d_cu = nullptr;
    uint8_t *d_k = nullptr, *d_v = nullptr, *d_ok = nullptr, *d_ov = nullptr, *d_s = nullptr, *d_c = nullptr, *d_os = nullptr, *d_oc = nullptr;
    CK(cudaMalloc(&d_reqs, n * 4)); CK(cudaMalloc(&d_zero, n * 4)); CK(cudaMalloc(&d_cu, (n + 1) * 4));
    CK(cudaMalloc(&d_k, k.size())); CK(cudaMalloc(&d_v, v.size())); CK(cudaMalloc(&d_ok, k.size())); CK(cudaMalloc(&d_ov, v.size()));
    CK(cudaMalloc(&d_s, st_bytes.size())); CK(cudaMalloc(&d_c, cv_bytes.size()));
    CK(cudaMalloc(&d_os, st_bytes.size())); CK(cudaMalloc(&d_oc, cv_bytes.size()));
    CK(cudaMemcpyAsync(d_reqs, reqs_h, n * 4, cudaMemcpyHostToDevice, s));
    CK(cudaMemsetAsync(d_zero, 0, n * 4, s));
    CK(cudaMemcpyAsync(d_k, k.data(), k.size(), cudaMemcpyHostToDevice, s));
    CK(cudaMemcpyAsync(d_v, v.data(), v.size(), cudaMemcpyHostToDevice, s));
    CK(cudaMemcpyAsync(d_s, st_bytes.data(), st_bytes.size(), cudaMemcpyHostToDevice, s));
    CK(cudaMemcpyAsync(d_c, cv_bytes.data(), cv_bytes.size(), cudaMemcpyHostToDevice, s));
    AV(avmp_scatter_kv(ctx, 1, d_reqs, d_zero, n, d_k, d_v, s));
    AV(avmp_scatter_ssm(ctx, 2, d_reqs, n, d_s, d_c, s));
    // the step that migrates: request 7 needs 12 SSM blocks, 8 are free; the KV store cedes its top
    // 6 slots, three of which hold the pages written above
    std::vector<avmp_op> grow = {{AVMP_OP_ADMIT, 0, 0, 7, 30}, {AVMP_OP_EXTEND, 0, 0, 4, 100}, {AVMP_OP_ADMIT, 0, 0, 8, 16},
                                 {AVMP_OP_FINISH, AVMP_FLAG_KEEP_KV, 0, 5, 0}, {AVMP_OP_ADMIT, AVMP_FLAG_RESUME, 0, 5, 40}};
    CK(cudaMemcpyAsync(d_ops, grow.data(), grow.size() * sizeof(avmp_op), cudaMemcpyHostToDevice, s));
    AV(avmp_step(ctx, d_ops, (uint32_t)grow.size(), d_st, s));
    AV(avmp_gather_kv(ctx, 1, d_reqs, n, d_ok, d_ov, tot, d_cu, s));
    AV(avmp_gather_ssm(ctx, 2, d_reqs, n, d_os, d_oc, s));
    std::vector<uint32_t> cu(n + 1), st_last(grow.size());
    std::vector<uint8_t> ok(k.size()), ov(v.size()), os(st_bytes.size()), oc(cv_bytes.size());
    CK(cudaMemcpyAsync(st_last.data(), d_st, grow.size() * 4, cudaMemcpyDeviceToHost, s));
    CK(cudaMemcpyAsync(cu.data(), d_cu, (n + 1) * 4, cudaMemcpyDeviceToHost, s));
    CK(cudaMemcpyAsync(ok.data(), d_ok, ok.size(), cudaMemcpyDeviceToHost, s));
    CK(cudaMemcpyAsync(ov.data(), d_ov, ov.size(), cudaMemcpyDeviceToHost, s));
    CK(cudaMemcpyAsync(os.data(), d_os, os.size(), cudaMemcpyDeviceToHost, s));
    CK(cudaMemcpyAsync(oc.data(), d_oc, oc.size(), cudaMemcpyDeviceToHost, s));
    avmp_stats stt;
    AV(avmp_get_stats(ctx, &stt, s));
    printf("last_statuses="); for (uint32_t x : st_last) printf("%u,", x); printf("\n");
    printf("cu="); for (uint32_t x : cu) printf("%u,", x); printf("\n");
    printf("k_equal=%d v_equal=%d state_equal=%d conv_equal=%d\n", (int)(ok == k), (int)(ov == v), (int)(os == st_bytes), (int)(oc == cv_bytes));
    printf("hash_k=%llu hash_v=%llu hash_state=%llu hash_conv=%llu\n", (unsigned long long)fnv(ok), (unsigned long long)fnv(ov),
           (unsigned long long)fnv(os), (unsigned long long)fnv(oc));
    printf("op_counter=%llu n_oom=%llu n_rebalance=%llu relocated_blocks=%llu cap_kv=%llu cap_ssm=%llu free_kv=%llu free_ssm=%llu gap=%llu error_code=%llu\n",
           (unsigned long long)stt.op_counter, (unsigned long long)stt.n_oom, (unsigned long long)stt.n_rebalance,
           (unsigned long long)stt.relocated_blocks, (unsigned long long)stt.cap[0], (unsigned long long)stt.cap[1],
           (unsigned long long)stt.free_units[0], (unsigned long long)stt.free_units[1], (unsigned long long)stt.gap_bytes,
           (unsigned long long)stt.error_code);
    AV(avmp_destroy(ctx));
    cudaFree(arena); cudaFree(ws);
    printf("done=1\n");
    return 0;
}
