// Launch interface of the tree-step kernel (internal to the library).
#pragma once

#include "common.cuh"

namespace mdraft {

constexpr int kTreeThreads = 128;  // channels per block, one thread each

struct TreeArgs {
    LayerDev L;
    PoolDev pool;
    const void *x, *z, *dt, *B, *C;
    void* out;
    int64_t ldx, ldz, lddt, ldb, ldc, ldo;
    const int32_t *parent_slot, *node_slot;
    int level_in_call;       // kernels this call has launched before this level (0 for the first)
    int lvl_begin, lvl_end;  // nodes [lvl_begin, lvl_end) form one tree level
    int32_t* dev_status;
};

cudaError_t launch_tree_step(const TreeArgs& p, int act, cudaStream_t st);

}  // namespace mdraft
