// Launch interface of the Mamba-2 (SSD) kernels (internal to the library).
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace mdraft {

constexpr int kSsdP = 64;      // channels per head handled by these kernels
constexpr int kSsdN = 128;     // state size handled by these kernels
constexpr int kSsdQ = 128;     // tokens per chunk of the context encode

// Per-layer constants of an SSD layer as the kernels take them.
struct SsdLayerDev {
    const float* A;        // (H)
    const float* D;        // (D) or NULL
    const float* conv_w;   // (D, W)
    const float* conv_b;   // (D) or NULL
    const float* dt_bias;  // (H) or NULL
    int d_inner;
    int n_heads;
    uint32_t flags;
};

// TMA descriptors of one context-encode call.
struct SsdMaps {
    CUtensorMap x, z;   // (T, D) activations, boxes of 64 channels x 128 tokens
    CUtensorMap Bs, Cs; // (T, N) activations in boxes of 64 states x 128 tokens, 128-byte swizzle (rows of 128 bytes: full sectors)
};

struct SsdPrefillArgs {
    SsdLayerDev L;
    PoolDev pool;               // slot = (D, 128) fp32 state + (W-1, D) window
    const __nv_bfloat16 *x, *z, *dt, *B, *C;
    __nv_bfloat16* out;
    int64_t ldx, ldz, lddt, ldb, ldc, ldo;
    int T, n_seq, n_chunks_bound;
    const int32_t *cu, *init_slot, *final_slot;
    float* ws_S;               // [chunk][H][P][N] fp32: what the chunk adds to a zero state
    float* ws_decay;           // [chunk][H]       fp32: sum over the chunk of Delta * A (log of the chunk's decay)
    __nv_bfloat16* ws_hin;     // [chunk][H][2][N/8][P][8] bf16: the chunk's incoming state (value, remainder), laid out as the tensor-core operand
    __nv_bfloat16* ws_xd;      // [chunk][H][P/8][Q (+1 unit of padding)][8] bf16: Delta * u in operand layout (kernel 1 -> kernel 3)
    __nv_bfloat16* ws_u;       // [T][D] bf16: conv + SiLU output, for the skip term (kernel 1 -> kernel 3)
    float* ws_csl;             // [chunk][H][Q] fp32: running log2-decay of the chunk's rows (kernel 1 -> kernel 3)
    int32_t* dev_status;
};

cudaError_t launch_ssd_prefill(const SsdPrefillArgs& p, const SsdMaps& maps, cudaStream_t st);

struct SsdStepArgs {
    SsdLayerDev L;
    PoolDev pool;
    const __nv_bfloat16 *x, *z, *dt, *B, *C;
    __nv_bfloat16* out;
    int64_t ldx, ldz, lddt, ldb, ldc, ldo;
    const int32_t *parent_slot, *node_slot;
    int lvl_begin, lvl_end;
    int32_t* dev_status;
};

cudaError_t launch_ssd_step(const SsdStepArgs& p, cudaStream_t st);

}  // namespace mdraft
