"""B200-native AVMP hot path: batched allocator update, handle translation and paged
KV / SSM gathers as hand-written sm_100a CUDA kernels behind a C ABI."""
