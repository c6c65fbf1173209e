// C ABI of the library: argument checks, launch planning, dispatch.  Nothing here allocates or keeps state between
// calls (the one exception in the library is the fixed scratch array of mdraft_conv_scan_prefill_noalloc, noalloc.cu).
#include <cudaTypedefs.h>
#include <limits.h>

#include <string.h>

#include "commit.cuh"
#include "common.cuh"
#include "prefill.cuh"
#include "ssd.cuh"
#include "tree_proj.cuh"
#include "tree_step.cuh"

using namespace mdraft;

namespace {

constexpr int kSmCountB200 = 148;

// SMs of the current device; the B200's count when no device can be asked (the workspace query also runs where there
// is none, and must then give the size the call will want on the B200 it is planned for).
int sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        (void)cudaGetLastError();
        return kSmCountB200;
    }
    return n;
}

inline size_t elem_size(int act) { return act == MDRAFT_BF16 ? 2 : 4; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

int check_layer(const mdraft_layer* L) {
    if (!L || !L->A || !L->conv_w) return MDRAFT_ERR_INVALID_ARG;
    if (L->d_inner <= 0) return MDRAFT_ERR_INVALID_ARG;
    if (L->d_state != kN || L->d_conv != kW || (L->d_inner % 8) != 0) return MDRAFT_ERR_UNSUPPORTED;
    if (L->act != MDRAFT_F32 && L->act != MDRAFT_BF16) return MDRAFT_ERR_UNSUPPORTED;
    if ((L->flags & MDRAFT_PRECONV) && (L->flags & MDRAFT_CONV_ONLY)) return MDRAFT_ERR_INVALID_ARG;
    if (!aligned16(L->A) || !aligned16(L->conv_w)) return MDRAFT_ERR_MISALIGNED;
    return MDRAFT_OK;
}

int check_cache(const mdraft_cache* c, int d_inner, int act, int layer_index, int d_state = kN) {
    if (!c || !c->ssm || !c->conv) return MDRAFT_ERR_INVALID_ARG;
    if (c->n_layers <= 0 || c->n_slots <= 0 || layer_index < 0 || layer_index >= c->n_layers) return MDRAFT_ERR_INVALID_ARG;
    const int64_t ssm_elems = (int64_t)d_inner * d_state, conv_elems = (int64_t)(kW - 1) * d_inner;
    if (c->ssm_slot_stride < ssm_elems || c->conv_slot_stride < conv_elems) return MDRAFT_ERR_INVALID_ARG;
    if (c->n_layers > 1 && (c->ssm_layer_stride < 0 || c->conv_layer_stride < 0)) return MDRAFT_ERR_INVALID_ARG;
    const size_t es = elem_size(act);
    if (!aligned16(c->ssm) || !aligned16(c->conv)) return MDRAFT_ERR_MISALIGNED;
    if ((c->ssm_slot_stride * 4) % 16 || (c->ssm_layer_stride * 4) % 16 || (c->conv_slot_stride * es) % 16 ||
        (c->conv_layer_stride * es) % 16)
        return MDRAFT_ERR_MISALIGNED;
    return MDRAFT_OK;
}

int check_matrix(const void* p, int64_t ld, int cols, int act, bool required) {
    if (!p) return required ? MDRAFT_ERR_INVALID_ARG : MDRAFT_OK;
    if (ld < cols) return MDRAFT_ERR_INVALID_ARG;
    if (!aligned16(p) || (ld * (int64_t)elem_size(act)) % 16) return MDRAFT_ERR_MISALIGNED;
    return MDRAFT_OK;
}

LayerDev layer_dev(const mdraft_layer* L) {
    LayerDev d;
    d.A = L->A; d.D = L->D; d.conv_w = L->conv_w; d.conv_b = L->conv_b; d.dt_bias = L->dt_bias;
    d.d_inner = L->d_inner; d.flags = L->flags;
    return d;
}

PoolDev pool_dev(const mdraft_cache* c, int act, int layer_index) {
    PoolDev p;
    p.ssm = c->ssm + (int64_t)layer_index * c->ssm_layer_stride;
    p.conv = static_cast<char*>(c->conv) + (int64_t)layer_index * c->conv_layer_stride * (int64_t)elem_size(act);
    p.ssm_slot_stride = c->ssm_slot_stride;
    p.conv_slot_stride = c->conv_slot_stride;
    p.n_slots = c->n_slots;
    return p;
}

struct PrefillPlan {
    int chunk_len;       // tokens per chunk (INT_MAX/2 when every sequence is one chunk)
    int n_chunks_bound;  // upper bound on the number of chunks
    bool chunked;
    bool wide;           // 512-channel blocks (one per SM) instead of 128-channel blocks
    size_t off_q, off_sd, off_h0, off_conv, bytes;
};

// Chunk length: split the token axis until every SM holds kBlocksPerSm blocks of kPrefillThreads channels (one
// resident wave, no tail), but never into chunks shorter than kMinChunk tokens (per-chunk set-up would dominate).
// When one wave would need chunks longer than kOneWaveMax tokens and the chunks would be uneven (packed batches) or the
// blocks narrow, several waves of short chunks do better: blocks are then handed out as SMs free up, which evens out
// uneven sequences and keeps every SM busy to the end (32 packed sequences of 1k-8k tokens: 1607 -> 1512 us).
constexpr int kBlocksPerSm = 4, kMinChunk = 32, kOneWaveMax = 256, kManyWavesChunk = 128, kManyWavesChunkBatched = 256;

PrefillPlan plan_prefill(const mdraft_layer* L, int T, int n_seq, int max_seqlen, const mdraft_prefill_opts* opts) {
    PrefillPlan pl;
    const int D = L->d_inner;
    const int wide_cols = kPrefillThreads * kPrefillWideBoxes;
    const int ch_blocks = (D + kPrefillThreads - 1) / kPrefillThreads;
    const int ch_blocks_wide = (D + wide_cols - 1) / wide_cols;
    const int forced = opts ? opts->block_channels : 0;
    // Wide blocks pay off when they fill the machine in one wave: every SM then runs ONE block whose 16 channel warps
    // advance together and finish together (four narrow blocks per SM finish one after another and leave the SM to
    // the last of them).  They need the channel count to (nearly) fill whole 512-channel blocks.
    bool wide = forced == wide_cols || (forced == 0 && (int64_t)ch_blocks_wide * wide_cols * 9 <= (int64_t)D * 10);
    int Lc;
    if (opts && opts->chunk_len > 0) {
        Lc = opts->chunk_len < 4 ? 4 : opts->chunk_len;
    } else {
        const int sms = sm_count();
        int want = wide ? sms / ch_blocks_wide : sms * kBlocksPerSm / ch_blocks;
        if (want < 1) want = 1;
        Lc = (T + want - 1) / want;
        if (Lc < kMinChunk) Lc = kMinChunk;
        // A single sequence in wide blocks stays in one wave at any length: 49 x 3 equal chunks finish together
        // (32768 tokens: 344 us against 372-376 for several waves of short chunks; 65536: 675 against 724).  Packed
        // batches, whose sequences differ in length, and widths that do not fill wide blocks take several waves of
        // short chunks in narrow blocks, four to an SM, so that a new block's set-up hides behind the others.
        if (Lc > kOneWaveMax && !(wide && n_seq == 1)) {
            Lc = n_seq > 1 ? kManyWavesChunkBatched : kManyWavesChunk;
            if (forced == 0) wide = false;
        }
    }
    pl.wide = wide;
    pl.chunked = Lc < max_seqlen;
    if (!pl.chunked) {
        pl.chunk_len = INT_MAX / 2;
        pl.n_chunks_bound = n_seq;
        pl.off_q = pl.off_sd = pl.off_h0 = pl.off_conv = 0;
        pl.bytes = 0;
        return pl;
    }
    pl.chunk_len = Lc;
    pl.n_chunks_bound = n_seq + T / Lc;
    const size_t Dz = (size_t)D;
    pl.off_q = 0;
    pl.off_sd = align_up(pl.off_q + (size_t)pl.n_chunks_bound * Dz * kN * sizeof(float), 256);
    pl.off_h0 = align_up(pl.off_sd + (size_t)pl.n_chunks_bound * Dz * sizeof(float), 256);
    pl.off_conv = align_up(pl.off_h0 + (size_t)n_seq * Dz * kN * sizeof(float), 256);
    pl.bytes = align_up(pl.off_conv + (size_t)n_seq * (kW - 1) * Dz * elem_size(L->act), 256);
    return pl;
}

// cuTensorMapEncodeTiled, fetched through the runtime so that the library has no link-time dependency on the
// driver (it can then be loaded, and its host-side checks exercised, on a machine without one).
PFN_cuTensorMapEncodeTiled tensor_map_encoder() {
    static PFN_cuTensorMapEncodeTiled fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) f = nullptr;
        return reinterpret_cast<PFN_cuTensorMapEncodeTiled>(f);
    }();
    return fn;
}

// Descriptor of a (rows x cols) row-major activation matrix with row stride ld, read in boxes of box_cols x tile rows.
bool encode_matrix(CUtensorMap* m, const void* base, int act, int64_t rows, int64_t cols, int64_t ld, int box_cols) {
    PFN_cuTensorMapEncodeTiled enc = tensor_map_encoder();
    if (!enc) return false;
    if (!base) {  // tensor not used by this mode: leave a recognisable empty descriptor
        memset(m, 0, sizeof(*m));
        return true;
    }
    const cuuint64_t es = elem_size(act);
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)ld * es};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)(kPrefillTileRowBytes / es)};
    cuuint32_t estride[2] = {1, 1};
    return enc(m, act == MDRAFT_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base),
               gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

__global__ void classify_A_kernel(const float* A, int D, int N, int32_t* res) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= D * N) return;
    int d = i / N, n = i % N;
    float a0 = A[(size_t)d * N], a = A[i];
    if (a != (float)(n + 1) * a0) atomicOr(res + 0, 1);
    if (!(a <= 0.0f)) atomicOr(res + 1, 1);
}

}  // namespace

extern "C" {

const char* mdraft_status_string(int status) {
    switch (status) {
        case MDRAFT_OK: return "ok";
        case MDRAFT_ERR_INVALID_ARG: return "invalid argument";
        case MDRAFT_ERR_UNSUPPORTED: return "unsupported shape or dtype (need d_state=16, d_conv=4, d_inner%8==0, fp32/bf16)";
        case MDRAFT_ERR_MISALIGNED: return "pointer or stride not a multiple of 16 bytes";
        case MDRAFT_ERR_WORKSPACE: return "workspace missing or too small";
        case MDRAFT_ERR_CUDA: return "CUDA runtime error";
        default: return "unknown status";
    }
}

int mdraft_version(void) { return 100; }

size_t mdraft_prefill_workspace_bytes(const mdraft_layer* layer, int32_t total_tokens, int32_t n_seq, int32_t max_seqlen,
                                      const mdraft_prefill_opts* opts) {
    if (check_layer(layer) != MDRAFT_OK || total_tokens <= 0 || n_seq <= 0 || max_seqlen <= 0) return 0;
    // No sequence is longer than the whole batch: a looser static bound must not change the plan.
    return plan_prefill(layer, total_tokens, n_seq, max_seqlen < total_tokens ? max_seqlen : total_tokens, opts).bytes;
}

int mdraft_conv_scan_prefill(const mdraft_layer* layer, const mdraft_cache* cache, int32_t layer_index,
                             const void* x, int64_t ldx, const void* z, int64_t ldz, const void* dt, int64_t lddt,
                             const void* B, int64_t ldb, const void* C, int64_t ldc, void* out, int64_t ldo,
                             int32_t total_tokens, int32_t n_seq, int32_t max_seqlen, const int32_t* cu_seqlens,
                             const int32_t* init_slot, const int32_t* final_slot, void* workspace, size_t workspace_bytes,
                             const mdraft_prefill_opts* opts, int32_t* dev_status, void* stream) {
    int rc = check_layer(layer);
    if (rc) return rc;
    if (total_tokens < 0 || n_seq < 0 || max_seqlen < 0) return MDRAFT_ERR_INVALID_ARG;
    if (opts) {
        if (opts->chunk_len < 0) return MDRAFT_ERR_INVALID_ARG;
        for (int i = 0; i < 2; ++i)
            if (opts->reserved[i]) return MDRAFT_ERR_INVALID_ARG;
        if (opts->block_channels != 0 && opts->block_channels != kPrefillThreads && opts->block_channels != kPrefillThreads * kPrefillWideBoxes)
            return MDRAFT_ERR_INVALID_ARG;
    }
    const bool needs_pool = init_slot || final_slot;
    if (needs_pool || cache) {
        rc = check_cache(cache, layer->d_inner, layer->act, layer_index);
        if (rc) return rc;
    }
    if (n_seq == 0) return MDRAFT_OK;
    if (!cu_seqlens && n_seq != 1) return MDRAFT_ERR_INVALID_ARG;  // offsets may be omitted for a single sequence only
    const bool conv_only = layer->flags & MDRAFT_CONV_ONLY;
    const int D = layer->d_inner, act = layer->act;
    const bool have_rows = total_tokens > 0;
    if ((rc = check_matrix(x, ldx, D, act, have_rows))) return rc;
    if ((rc = check_matrix(out, ldo, D, act, have_rows))) return rc;
    if ((rc = check_matrix(z, ldz, D, act, have_rows && !conv_only))) return rc;
    if ((rc = check_matrix(dt, lddt, D, act, have_rows && !conv_only))) return rc;
    if ((rc = check_matrix(B, ldb, kN, act, have_rows && !conv_only))) return rc;
    if ((rc = check_matrix(C, ldc, kN, act, have_rows && !conv_only))) return rc;
    // The same bound as in the workspace query: no sequence is longer than the whole batch.  A batch of empty
    // sequences therefore never takes the chunked path (and needs no workspace), whatever static bound was given.
    const int plan_tokens = total_tokens > 0 ? total_tokens : 1;
    if (max_seqlen > plan_tokens) max_seqlen = plan_tokens;
    if (max_seqlen < 1) max_seqlen = 1;

    PrefillPlan pl = plan_prefill(layer, plan_tokens, n_seq, max_seqlen, opts);
    if (pl.chunked) {
        if (!workspace || workspace_bytes < pl.bytes) return MDRAFT_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(workspace) & 255u) return MDRAFT_ERR_MISALIGNED;
    }
    PrefillArgs a;
    a.L = layer_dev(layer);
    if (cache) a.pool = pool_dev(cache, act, layer_index);
    else { a.pool.ssm = nullptr; a.pool.conv = nullptr; a.pool.ssm_slot_stride = 0; a.pool.conv_slot_stride = 0; a.pool.n_slots = 0; }
    a.x = x; a.z = z; a.dt = dt; a.B = B; a.C = C; a.out = out;
    a.ldx = ldx; a.ldz = ldz; a.lddt = lddt; a.ldb = ldb; a.ldc = ldc; a.ldo = ldo;
    a.T = total_tokens; a.n_seq = n_seq; a.chunk_len = pl.chunk_len; a.n_chunks_bound = pl.n_chunks_bound;
    a.cu = cu_seqlens; a.init_slot = init_slot; a.final_slot = final_slot;
    char* ws = static_cast<char*>(workspace);
    a.ws_q = pl.chunked ? reinterpret_cast<float*>(ws + pl.off_q) : nullptr;
    a.ws_sd = pl.chunked ? reinterpret_cast<float*>(ws + pl.off_sd) : nullptr;
    a.ws_h0 = pl.chunked ? reinterpret_cast<float*>(ws + pl.off_h0) : nullptr;
    a.ws_conv = pl.chunked ? static_cast<void*>(ws + pl.off_conv) : nullptr;
    a.dev_status = dev_status;
    if (a.n_chunks_bound > 65535) return MDRAFT_ERR_UNSUPPORTED;
    a.ev_state = opts ? static_cast<cudaEvent_t>(opts->event_after_chunk_state) : nullptr;
    a.ev_carry = opts ? static_cast<cudaEvent_t>(opts->event_after_carry_scan) : nullptr;
    PrefillMaps maps;  // with no tokens at all (only empty sequences) nothing is ever copied: empty descriptors
    if (!encode_matrix(&maps.x, have_rows ? x : nullptr, act, total_tokens, D, ldx, kPrefillThreads) ||
        !encode_matrix(&maps.dt, have_rows ? dt : nullptr, act, total_tokens, D, lddt, kPrefillThreads) ||
        !encode_matrix(&maps.z, have_rows ? z : nullptr, act, total_tokens, D, ldz, kPrefillThreads) ||
        !encode_matrix(&maps.B, have_rows ? B : nullptr, act, total_tokens, kN, ldb, kN) ||
        !encode_matrix(&maps.C, have_rows ? C : nullptr, act, total_tokens, kN, ldc, kN))
        return MDRAFT_ERR_CUDA;
    cudaError_t e = launch_prefill(a, maps, act, pl.chunked, pl.wide, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? MDRAFT_OK : MDRAFT_ERR_CUDA;
}

int mdraft_tree_step(const mdraft_layer* layer, const mdraft_cache* cache, int32_t layer_index, const void* x, int64_t ldx,
                     const void* z, int64_t ldz, const void* dt, int64_t lddt, const void* B, int64_t ldb, const void* C,
                     int64_t ldc, void* out, int64_t ldo, int32_t n_nodes, const int32_t* parent_slot,
                     const int32_t* node_slot, int32_t n_levels, const int32_t* level_offsets, int32_t* dev_status,
                     void* stream) {
    int rc = check_layer(layer);
    if (rc) return rc;
    if ((rc = check_cache(cache, layer->d_inner, layer->act, layer_index))) return rc;
    if (n_nodes < 0 || n_levels < 0) return MDRAFT_ERR_INVALID_ARG;
    if (n_nodes == 0) return MDRAFT_OK;
    if (!parent_slot || !node_slot) return MDRAFT_ERR_INVALID_ARG;
    if (!level_offsets && n_levels > 1) return MDRAFT_ERR_INVALID_ARG;
    if (level_offsets) {
        if (n_levels < 1 || level_offsets[0] != 0 || level_offsets[n_levels] != n_nodes) return MDRAFT_ERR_INVALID_ARG;
        for (int l = 0; l < n_levels; ++l)
            if (level_offsets[l + 1] < level_offsets[l]) return MDRAFT_ERR_INVALID_ARG;
    }
    const bool conv_only = layer->flags & MDRAFT_CONV_ONLY;
    const int D = layer->d_inner, act = layer->act;
    if ((rc = check_matrix(x, ldx, D, act, true))) return rc;
    if ((rc = check_matrix(out, ldo, D, act, true))) return rc;
    if ((rc = check_matrix(z, ldz, D, act, !conv_only))) return rc;
    if ((rc = check_matrix(dt, lddt, D, act, !conv_only))) return rc;
    if ((rc = check_matrix(B, ldb, kN, act, !conv_only))) return rc;
    if ((rc = check_matrix(C, ldc, kN, act, !conv_only))) return rc;

    TreeArgs a;
    a.L = layer_dev(layer);
    a.pool = pool_dev(cache, act, layer_index);
    a.x = x; a.z = z; a.dt = dt; a.B = B; a.C = C; a.out = out;
    a.ldx = ldx; a.ldz = ldz; a.lddt = lddt; a.ldb = ldb; a.ldc = ldc; a.ldo = ldo;
    a.parent_slot = parent_slot; a.node_slot = node_slot; a.dev_status = dev_status;
    const int levels = level_offsets ? n_levels : 1;
    int launched = 0;  // an empty level launches nothing and must not count: the chaining rules go by kernels ahead
    for (int l = 0; l < levels; ++l) {
        a.level_in_call = launched;
        a.lvl_begin = level_offsets ? level_offsets[l] : 0;
        a.lvl_end = level_offsets ? level_offsets[l + 1] : n_nodes;
        if (a.lvl_end == a.lvl_begin) continue;
        if (launch_tree_step(a, act, static_cast<cudaStream_t>(stream)) != cudaSuccess) return MDRAFT_ERR_CUDA;
        ++launched;
    }
    return MDRAFT_OK;
}

int mdraft_tree_step_proj(const mdraft_layer* layer, const mdraft_cache* cache, int32_t layer_index,
                          const mdraft_select_proj* proj, const void* x, int64_t ldx, const void* z, int64_t ldz, void* out,
                          int64_t ldo, int32_t n_nodes, const int32_t* parent_slot, const int32_t* node_slot,
                          int32_t* dev_status, void* stream) {
    int rc = check_layer(layer);
    if (rc) return rc;
    if ((rc = check_cache(cache, layer->d_inner, layer->act, layer_index))) return rc;
    if (layer->flags & (MDRAFT_PRECONV | MDRAFT_CONV_ONLY)) return MDRAFT_ERR_INVALID_ARG;
    if (!proj || !proj->W_x || !proj->W_dt || n_nodes < 0) return MDRAFT_ERR_INVALID_ARG;
    if (!aligned16(proj->W_x) || !aligned16(proj->W_dt)) return MDRAFT_ERR_MISALIGNED;
    if (proj->dt_rank < 8 || proj->dt_rank > kProjMaxRank || (proj->dt_rank % 8) != 0) return MDRAFT_ERR_UNSUPPORTED;
    if (tree_proj_block_channels(layer->d_inner) == 0) return MDRAFT_ERR_UNSUPPORTED;
    if (proj->nodes_per_cluster != 0 && proj->nodes_per_cluster != 1 && proj->nodes_per_cluster != 2 && proj->nodes_per_cluster != 4)
        return MDRAFT_ERR_INVALID_ARG;
    if (n_nodes == 0) return MDRAFT_OK;
    if (!parent_slot || !node_slot) return MDRAFT_ERR_INVALID_ARG;
    const int D = layer->d_inner, act = layer->act;
    if ((rc = check_matrix(x, ldx, D, act, true))) return rc;
    if ((rc = check_matrix(z, ldz, D, act, true))) return rc;
    if ((rc = check_matrix(out, ldo, D, act, true))) return rc;

    TreeProjArgs a;
    a.L = layer_dev(layer);
    a.pool = pool_dev(cache, act, layer_index);
    a.x = x; a.z = z; a.out = out;
    a.ldx = ldx; a.ldz = ldz; a.ldo = ldo;
    a.W_x = proj->W_x; a.W_dt = proj->W_dt; a.dt_rank = proj->dt_rank; a.nodes_per_cluster = proj->nodes_per_cluster;
    a.parent_slot = parent_slot; a.node_slot = node_slot; a.n_nodes = n_nodes; a.dev_status = dev_status;
    if (launch_tree_proj(a, act, static_cast<cudaStream_t>(stream)) != cudaSuccess) return MDRAFT_ERR_CUDA;
    return MDRAFT_OK;
}

int mdraft_state_commit(const mdraft_cache* cache, int32_t d_inner, int32_t d_state, int32_t d_conv, int32_t act,
                        int32_t n_commit, const int32_t* src_slot, const int32_t* dst_slot, int32_t* dev_status,
                        void* stream) {
    if (d_inner <= 0 || n_commit < 0) return MDRAFT_ERR_INVALID_ARG;
    if ((d_state != kN && d_state != kSsdN) || d_conv != kW || (d_inner % 8) != 0 || (act != MDRAFT_F32 && act != MDRAFT_BF16)) return MDRAFT_ERR_UNSUPPORTED;
    int rc = check_cache(cache, d_inner, act, 0, d_state);
    if (rc) return rc;
    if (n_commit == 0) return MDRAFT_OK;
    if (!src_slot || !dst_slot) return MDRAFT_ERR_INVALID_ARG;
    const int64_t es = (int64_t)elem_size(act);
    CommitArgs a;
    a.ssm = reinterpret_cast<char*>(cache->ssm);
    a.conv = static_cast<char*>(cache->conv);
    a.ssm_layer_bytes = cache->ssm_layer_stride * 4; a.ssm_slot_bytes_stride = cache->ssm_slot_stride * 4;
    a.conv_layer_bytes = cache->conv_layer_stride * es; a.conv_slot_bytes_stride = cache->conv_slot_stride * es;
    a.ssm_bytes = (int64_t)d_inner * d_state * 4; a.conv_bytes = (int64_t)(kW - 1) * d_inner * es;
    a.n_layers = cache->n_layers; a.n_slots = cache->n_slots; a.dev_status = dev_status;
    if (a.n_layers > 65535) return MDRAFT_ERR_UNSUPPORTED;
    for (int off = 0; off < n_commit; off += 65535) {
        a.n_commit = n_commit - off < 65535 ? n_commit - off : 65535;
        a.src_slot = src_slot + off; a.dst_slot = dst_slot + off;
        if (launch_commit(a, static_cast<cudaStream_t>(stream)) != cudaSuccess) return MDRAFT_ERR_CUDA;
    }
    return MDRAFT_OK;
}

int mdraft_classify_A(const float* A, int32_t d_inner, int32_t d_state, int32_t* scratch, int32_t* is_powers,
                      int32_t* is_nonpositive, void* stream) {
    if (!A || !scratch || !is_powers || d_inner <= 0 || d_state <= 0) return MDRAFT_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(scratch, 0, 2 * sizeof(int32_t), st) != cudaSuccess) return MDRAFT_ERR_CUDA;
    const int n = d_inner * d_state;
    classify_A_kernel<<<(n + 255) / 256, 256, 0, st>>>(A, d_inner, d_state, scratch);
    int32_t host[2] = {1, 1};
    if (cudaMemcpyAsync(host, scratch, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess) return MDRAFT_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return MDRAFT_ERR_CUDA;
    *is_powers = host[0] == 0;
    if (is_nonpositive) *is_nonpositive = host[1] == 0;
    return MDRAFT_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------- SSD layer
namespace {

int check_ssd_layer(const mdraft_ssd_layer* L) {
    if (!L || !L->A || !L->conv_w) return MDRAFT_ERR_INVALID_ARG;
    if (L->d_inner <= 0) return MDRAFT_ERR_INVALID_ARG;
    if (L->headdim != kSsdP || L->d_state != kSsdN || L->d_conv != kW || (L->d_inner % kSsdP) != 0 || L->act != MDRAFT_BF16)
        return MDRAFT_ERR_UNSUPPORTED;
    if (L->flags & ~(uint32_t)MDRAFT_DT_SOFTPLUS) return MDRAFT_ERR_INVALID_ARG;
    if (!aligned16(L->conv_w)) return MDRAFT_ERR_MISALIGNED;
    return MDRAFT_OK;
}

SsdLayerDev ssd_layer_dev(const mdraft_ssd_layer* L) {
    SsdLayerDev d;
    d.A = L->A; d.D = L->D; d.conv_w = L->conv_w; d.conv_b = L->conv_b; d.dt_bias = L->dt_bias;
    d.d_inner = L->d_inner; d.n_heads = L->d_inner / L->headdim; d.flags = L->flags;
    return d;
}

struct SsdPlan {
    int n_chunks_bound;
    size_t off_S, off_decay, off_hin, off_xd, off_u, off_csl, bytes;
};

SsdPlan plan_ssd(const mdraft_ssd_layer* L, int T, int n_seq) {
    SsdPlan pl;
    const size_t H = (size_t)(L->d_inner / L->headdim);
    pl.n_chunks_bound = n_seq + T / kSsdQ;
    const size_t per_chunk = H * kSsdP * kSsdN;
    pl.off_S = 0;
    pl.off_decay = align_up(pl.off_S + (size_t)pl.n_chunks_bound * per_chunk * sizeof(float), 256);
    pl.off_hin = align_up(pl.off_decay + (size_t)pl.n_chunks_bound * H * sizeof(float), 256);
    pl.off_xd = align_up(pl.off_hin + (size_t)pl.n_chunks_bound * per_chunk * 2 * 2, 256);   // bf16 value + bf16 remainder
    pl.off_u = align_up(pl.off_xd + (size_t)pl.n_chunks_bound * H * (kSsdP / 8) * (kSsdQ * 16 + 16), 256);
    pl.off_csl = align_up(pl.off_u + (size_t)T * L->d_inner * 2, 256);
    pl.bytes = align_up(pl.off_csl + (size_t)pl.n_chunks_bound * H * kSsdQ * sizeof(float), 256);
    return pl;
}

// Descriptor of a (rows x cols) row-major bf16 matrix read in boxes of box_cols x 128 rows.
bool encode_ssd_matrix(CUtensorMap* m, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_cols) {
    PFN_cuTensorMapEncodeTiled enc = tensor_map_encoder();
    if (!enc) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)kSsdQ};
    cuuint32_t estride[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Descriptor of a (rows x 128) row-major bf16 matrix read in boxes of 64 columns x 128 rows that land in shared memory as
// rows of 128 bytes, 16-byte units XOR-ed with the row index (the tensor core's 128-byte-swizzled K-major operand layout).
bool encode_ssd_swizzled(CUtensorMap* m, const void* base, int64_t rows, int64_t ld) {
    PFN_cuTensorMapEncodeTiled enc = tensor_map_encoder();
    if (!enc) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)kSsdN, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kSsdQ};
    cuuint32_t estride[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

extern "C" {

size_t mdraft_ssd_prefill_workspace_bytes(const mdraft_ssd_layer* layer, int32_t total_tokens, int32_t n_seq) {
    if (check_ssd_layer(layer) != MDRAFT_OK || total_tokens <= 0 || n_seq <= 0) return 0;
    return plan_ssd(layer, total_tokens, n_seq).bytes;
}

int mdraft_ssd_prefill(const mdraft_ssd_layer* layer, const mdraft_cache* cache, int32_t layer_index, const void* x, int64_t ldx,
                       const void* z, int64_t ldz, const void* dt, int64_t lddt, const void* B, int64_t ldb, const void* C,
                       int64_t ldc, void* out, int64_t ldo, int32_t total_tokens, int32_t n_seq, const int32_t* cu_seqlens,
                       const int32_t* init_slot, const int32_t* final_slot, void* workspace, size_t workspace_bytes,
                       int32_t* dev_status, void* stream) {
    int rc = check_ssd_layer(layer);
    if (rc) return rc;
    if (total_tokens < 0 || n_seq < 0) return MDRAFT_ERR_INVALID_ARG;
    if (init_slot || final_slot || cache) {
        rc = check_cache(cache, layer->d_inner, layer->act, layer_index, kSsdN);
        if (rc) return rc;
    }
    if (n_seq == 0) return MDRAFT_OK;
    if (!cu_seqlens && n_seq != 1) return MDRAFT_ERR_INVALID_ARG;
    const int D = layer->d_inner, H = D / layer->headdim;
    const bool have_rows = total_tokens > 0;
    if ((rc = check_matrix(x, ldx, D, MDRAFT_BF16, have_rows))) return rc;
    if ((rc = check_matrix(z, ldz, D, MDRAFT_BF16, have_rows))) return rc;
    if ((rc = check_matrix(out, ldo, D, MDRAFT_BF16, have_rows))) return rc;
    if ((rc = check_matrix(B, ldb, kSsdN, MDRAFT_BF16, have_rows))) return rc;
    if ((rc = check_matrix(C, ldc, kSsdN, MDRAFT_BF16, have_rows))) return rc;
    if (have_rows && (!dt || lddt < H)) return MDRAFT_ERR_INVALID_ARG;
    const SsdPlan pl = plan_ssd(layer, have_rows ? total_tokens : 1, n_seq);
    if (!workspace || workspace_bytes < pl.bytes) return MDRAFT_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return MDRAFT_ERR_MISALIGNED;
    if (pl.n_chunks_bound > 65535) return MDRAFT_ERR_UNSUPPORTED;

    SsdPrefillArgs a;
    a.L = ssd_layer_dev(layer);
    if (cache) a.pool = pool_dev(cache, MDRAFT_BF16, layer_index);
    else { a.pool.ssm = nullptr; a.pool.conv = nullptr; a.pool.ssm_slot_stride = 0; a.pool.conv_slot_stride = 0; a.pool.n_slots = 0; }
    a.x = static_cast<const __nv_bfloat16*>(x); a.z = static_cast<const __nv_bfloat16*>(z); a.dt = static_cast<const __nv_bfloat16*>(dt);
    a.B = static_cast<const __nv_bfloat16*>(B); a.C = static_cast<const __nv_bfloat16*>(C); a.out = static_cast<__nv_bfloat16*>(out);
    a.ldx = ldx; a.ldz = ldz; a.lddt = lddt; a.ldb = ldb; a.ldc = ldc; a.ldo = ldo;
    a.T = total_tokens; a.n_seq = n_seq; a.n_chunks_bound = pl.n_chunks_bound;
    a.cu = cu_seqlens; a.init_slot = init_slot; a.final_slot = final_slot;
    char* ws = static_cast<char*>(workspace);
    a.ws_S = reinterpret_cast<float*>(ws + pl.off_S);
    a.ws_decay = reinterpret_cast<float*>(ws + pl.off_decay);
    a.ws_hin = reinterpret_cast<__nv_bfloat16*>(ws + pl.off_hin);
    a.ws_xd = reinterpret_cast<__nv_bfloat16*>(ws + pl.off_xd);
    a.ws_u = reinterpret_cast<__nv_bfloat16*>(ws + pl.off_u);
    a.ws_csl = reinterpret_cast<float*>(ws + pl.off_csl);
    a.dev_status = dev_status;
    SsdMaps maps;
    memset(&maps, 0, sizeof(maps));
    if (have_rows) {
        if (!encode_ssd_matrix(&maps.x, x, total_tokens, D, ldx, kSsdP) || !encode_ssd_matrix(&maps.z, z, total_tokens, D, ldz, kSsdP) ||
            !encode_ssd_swizzled(&maps.Bs, B, total_tokens, ldb) ||
            !encode_ssd_swizzled(&maps.Cs, C, total_tokens, ldc))
            return MDRAFT_ERR_CUDA;
    }
    return launch_ssd_prefill(a, maps, static_cast<cudaStream_t>(stream)) == cudaSuccess ? MDRAFT_OK : MDRAFT_ERR_CUDA;
}

int mdraft_ssd_tree_step(const mdraft_ssd_layer* layer, const mdraft_cache* cache, int32_t layer_index, const void* x, int64_t ldx,
                         const void* z, int64_t ldz, const void* dt, int64_t lddt, const void* B, int64_t ldb, const void* C,
                         int64_t ldc, void* out, int64_t ldo, int32_t n_nodes, const int32_t* parent_slot, const int32_t* node_slot,
                         int32_t n_levels, const int32_t* level_offsets, int32_t* dev_status, void* stream) {
    int rc = check_ssd_layer(layer);
    if (rc) return rc;
    if ((rc = check_cache(cache, layer->d_inner, layer->act, layer_index, kSsdN))) return rc;
    if (n_nodes < 0 || n_levels < 0) return MDRAFT_ERR_INVALID_ARG;
    if (n_nodes == 0) return MDRAFT_OK;
    if (!parent_slot || !node_slot) return MDRAFT_ERR_INVALID_ARG;
    if (!level_offsets && n_levels > 1) return MDRAFT_ERR_INVALID_ARG;
    if (level_offsets) {
        if (n_levels < 1 || level_offsets[0] != 0 || level_offsets[n_levels] != n_nodes) return MDRAFT_ERR_INVALID_ARG;
        for (int l = 0; l < n_levels; ++l)
            if (level_offsets[l + 1] < level_offsets[l]) return MDRAFT_ERR_INVALID_ARG;
    }
    const int D = layer->d_inner, H = D / layer->headdim;
    if ((rc = check_matrix(x, ldx, D, MDRAFT_BF16, true))) return rc;
    if ((rc = check_matrix(z, ldz, D, MDRAFT_BF16, true))) return rc;
    if ((rc = check_matrix(out, ldo, D, MDRAFT_BF16, true))) return rc;
    if ((rc = check_matrix(B, ldb, kSsdN, MDRAFT_BF16, true))) return rc;
    if ((rc = check_matrix(C, ldc, kSsdN, MDRAFT_BF16, true))) return rc;
    if (!dt || lddt < H) return MDRAFT_ERR_INVALID_ARG;
    SsdStepArgs a;
    a.L = ssd_layer_dev(layer);
    a.pool = pool_dev(cache, MDRAFT_BF16, layer_index);
    a.x = static_cast<const __nv_bfloat16*>(x); a.z = static_cast<const __nv_bfloat16*>(z); a.dt = static_cast<const __nv_bfloat16*>(dt);
    a.B = static_cast<const __nv_bfloat16*>(B); a.C = static_cast<const __nv_bfloat16*>(C); a.out = static_cast<__nv_bfloat16*>(out);
    a.ldx = ldx; a.ldz = ldz; a.lddt = lddt; a.ldb = ldb; a.ldc = ldc; a.ldo = ldo;
    a.parent_slot = parent_slot; a.node_slot = node_slot; a.dev_status = dev_status;
    const int levels = level_offsets ? n_levels : 1;
    for (int l = 0; l < levels; ++l) {
        a.lvl_begin = level_offsets ? level_offsets[l] : 0;
        a.lvl_end = level_offsets ? level_offsets[l + 1] : n_nodes;
        if (launch_ssd_step(a, static_cast<cudaStream_t>(stream)) != cudaSuccess) return MDRAFT_ERR_CUDA;
    }
    return MDRAFT_OK;
}

}  // extern "C"
