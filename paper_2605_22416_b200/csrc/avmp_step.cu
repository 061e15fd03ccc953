// avmp_step: the batched allocator update (paper Sections 3.1-3.2) as one planning CTA.
//
// The batch must behave exactly as if its ops were applied one at a time.  The CTA cuts
// the batch into windows of NT ops (one per thread; NT = 256, 512 or 1024 by batch length)
// and each window into maximal runs of ops that point the same way (all FINISH, or all
// ADMIT/EXTEND) and touch distinct request slots.  Inside a run the sequential result has a
// closed form:
//   * free run  -- an exclusive prefix sum of the units each op releases gives the stack
//                  position of every pushed slot and id;
//   * alloc run -- an exclusive prefix sum of the demands gives the stack entries every op
//                  pops, as long as every op before it fits.  The first op whose inclusive
//                  demand exceeds the free count is the first sequential failure: everything
//                  before it is committed, the CapacityError handler (Section 3.2) runs for
//                  that op alone (a migration with the whole CTA helping: stack compaction,
//                  relocation list, recipient growth), the op is retried once, and the scan
//                  resumes behind it.  A failed op takes nothing, so the same prefix sums
//                  stay valid.
// A window in an engine step's order (FINISH*, EXTEND*, ADMIT*, ascending slots inside a kind)
// is recognised with one ballot per warp and has exactly those two runs; any other window finds
// its runs through a shared-memory hash of the slots (avmp_step_body.cuh).
// Relocated payload is copied by a separate wide kernel after this one, so a launch performs
// at most one migration; if a second one is due, the launch stops before that op and the
// host-queued next round resumes there (the throttle bounds the number of rounds).
#include "avmp_step_body.cuh"

namespace avmp {

namespace {

using namespace stepimpl;

template <int NT>
__global__ void __launch_bounds__(NT, 1)
step_kernel(const Geom g, const avmp_op *ops, const uint32_t n_ops_max,
            const uint32_t *n_ops_dev, uint32_t *status, const int first_round)
{
    __shared__ Shared<NT> sh;
    pdl_prologue();
    // the batch length is a launch argument, or (device-built batches) a word in device memory
    const uint32_t n_ops = n_ops_dev ? min(*n_ops_dev, n_ops_max) : n_ops_max;
    step_body<NT>(g, sh, ops, n_ops, status, first_round);
}

// Fresh pools hand out slot 0, 1, 2, ... and id 0, 1, 2, ...: the lowest index is on top.
__global__ void init_kernel(const Geom g, const DevState init)
{
    const unsigned long long gid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    pdl_prologue();
    if (gid == 0) *g.st = init;
    for (int p = 0; p < 2; ++p) {
        const uint32_t V = g.V[p], cap = init.cap[p];
        for (unsigned long long i = gid; i < V; i += stride) {
            g.VT[p][i] = kInvalid;
            g.OW[p][i] = kInvalid;
            g.W[p][i] = V - 1u - (uint32_t)i;
            g.S[p][i] = i < cap ? cap - 1u - (uint32_t)i : kInvalid;
        }
    }
    for (unsigned long long i = gid; i < g.R; i += stride) {
        g.r_state[i] = AVMP_REQ_EMPTY; g.r_len[i] = 0; g.r_npages[i] = 0;
    }
    for (unsigned long long i = gid; i < (unsigned long long)g.R * g.max_pages; i += stride) g.r_chain[i] = kInvalid;
    for (unsigned long long i = gid; i < (unsigned long long)g.R * g.ns; i += stride) g.r_ssm[i] = kInvalid;
}

}  // namespace

cudaError_t launch_init(const Geom &g, const DevState &init, cudaStream_t s)
{
    return launch_pdl(init_kernel, dim3(296), dim3(512), 0, s, g, init);
}

cudaError_t launch_step(const Geom &g, const avmp_op *d_ops, uint32_t n_ops, const uint32_t *d_n_ops,
                        uint32_t *d_status, int first_round, cudaStream_t s)
{
    if (n_ops <= 256)
        return launch_pdl(step_kernel<256>, dim3(1), dim3(256), 0, s, g, d_ops, n_ops, d_n_ops, d_status, first_round);
    if (n_ops <= 512)
        return launch_pdl(step_kernel<512>, dim3(1), dim3(512), 0, s, g, d_ops, n_ops, d_n_ops, d_status, first_round);
    return launch_pdl(step_kernel<1024>, dim3(1), dim3(1024), 0, s, g, d_ops, n_ops, d_n_ops, d_status, first_round);
}

}  // namespace avmp
