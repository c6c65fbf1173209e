// Launch interface of the tree step that forms its own step size, B and C (internal to the library).
#pragma once

#include "common.cuh"

namespace mdraft {

constexpr int kProjMaxRank = 256;     // largest dt_rank the kernel's shared-memory vectors hold
constexpr int kProjMaxCluster = 8;    // blocks per node: the portable cluster size limit

struct TreeProjArgs {
    LayerDev L;
    PoolDev pool;
    const void *x, *z;
    void* out;
    int64_t ldx, ldz, ldo;
    const void* W_x;   // (dt_rank + 2 N, D) row-major
    const void* W_dt;  // (D, dt_rank) row-major
    int dt_rank;
    int nodes_per_cluster;  // 0: chosen from the level's width; else 1, 2 or 4
    const int32_t *parent_slot, *node_slot;
    int n_nodes;
    int32_t* dev_status;
};

// Channels per block for a layer width, or 0 when no supported block width covers it with one cluster.
int tree_proj_block_channels(int d_inner);

cudaError_t launch_tree_proj(const TreeProjArgs& p, int act, cudaStream_t st);

}  // namespace mdraft
