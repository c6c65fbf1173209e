// Launch interface of the prefill kernels (internal to the library).
#pragma once

#include <cuda.h>

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
    float* ws_q;    // [n_chunks_bound][N/4][D][4] zero-state result of each chunk; after the carry scan, entry c holds
                    //                             the state after chunk c = the incoming state of chunk c + 1
    float* ws_sd;   // [n_chunks_bound][D]         sum of Delta per chunk
    float* ws_h0;   // [n_seq][N/4][D][4]          starting state of each split sequence
    void* ws_conv;  // [n_seq][W-1][D]             starting conv window of each split sequence (activation type)
    int32_t* dev_status;
    int pdl_inputs_ready;  // set by the launcher: 1 if an earlier kernel of this call has already waited for the inputs
    cudaEvent_t ev_state, ev_carry;  // optional profiling events (host side only)
};

constexpr int kPrefillTileRowBytes = 32;  // a staged tile holds 32 / sizeof(activation) tokens: 16 (bf16) or 8 (fp32)

// TMA descriptors of the five activation matrices of one call: boxes of kPrefillThreads channels (x, dt, z) or
// 16 values (B, C) by one tile of tokens.  Built on the host for every call (they hold the base addresses).
struct PrefillMaps {
    CUtensorMap x, dt, z, B, C;
};

constexpr int kPrefillWideBoxes = 4;  // a wide block covers 4 x kPrefillThreads channels with 16 channel warps

// wide: one block of 512 channels per (channel block, chunk) instead of 128 — for plans that give every SM one block.
cudaError_t launch_prefill(const PrefillArgs& p, const PrefillMaps& maps, int act, bool chunked, bool wide, cudaStream_t st);

}  // namespace mdraft
