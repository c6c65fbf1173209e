// Launch interface of the commit kernel (internal to the library).
#pragma once

#include "common.cuh"

namespace mdraft {

struct CommitArgs {
    char* ssm;    // byte view of the pool
    char* conv;
    int64_t ssm_layer_bytes, ssm_slot_bytes_stride, conv_layer_bytes, conv_slot_bytes_stride;
    int64_t ssm_bytes, conv_bytes;  // payload of one slot
    int n_layers, n_slots, n_commit;
    const int32_t *src_slot, *dst_slot;
    int32_t* dev_status;
};

cudaError_t launch_commit(const CommitArgs& p, cudaStream_t st);

}  // namespace mdraft
