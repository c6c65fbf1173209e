// Launch interface of the prefill kernels (internal to the library).
#pragma once

#include "common.cuh"

namespace mdraft {

constexpr int kPrefillThreads = 128;  // channels per block (one thread per channel)

struct PrefillArgs {
    LayerDev L;
    PoolDev pool;
    const void *x, *z, *dt, *B, *C;
    void* out;
    int64_t ldx, ldz, lddt, ldb, ldc, ldo;
    int T, n_seq, chunk_len, n_chunks_bound;
    const int32_t *cu, *init_slot, *final_slot;
    float* ws_h;    // [n_chunks_bound][D][N] chunk summaries, then incoming states
    float* ws_sd;   // [n_chunks_bound][D]    sum of Delta per chunk
    void* ws_conv;  // [n_seq][W-1][D]        starting conv windows (activation type)
    int32_t* dev_status;
    cudaEvent_t ev_state, ev_carry;  // optional profiling events (host side only)
};

cudaError_t launch_prefill(const PrefillArgs& p, int act, bool chunked, cudaStream_t st);

}  // namespace mdraft
