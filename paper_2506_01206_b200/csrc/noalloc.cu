// Prefill entry point for callers that cannot allocate device memory: the chunk scratch lives in a fixed
// array inside the library image instead of a caller-supplied workspace.
#include <mutex>

#include "common.cuh"

namespace {

// Scratch for the chunked prefill.  Part of the loaded module: every device that loads the library holds
// these bytes until the process exits, whether or not the entry point below is ever called.
static __device__ __align__(256) unsigned char g_prefill_scratch[MDRAFT_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_lock;
void* g_scratch_addr[kMaxDevices];  // device address of g_prefill_scratch on each device, 0 = not resolved yet

// In host code `g_prefill_scratch` is only a handle for the runtime, not an address a kernel can use; the
// device address is looked up once per device (with that device current) and remembered.
int scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MDRAFT_ERR_CUDA;
    std::lock_guard<std::mutex> hold(g_lock);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_prefill_scratch) != cudaSuccess || !p) return MDRAFT_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return MDRAFT_OK;
}

}  // namespace

extern "C" int mdraft_conv_scan_prefill_noalloc(const mdraft_layer* layer, const mdraft_cache* cache, int32_t layer_index,
                                                const void* x, int64_t ldx, const void* z, int64_t ldz, const void* dt,
                                                int64_t lddt, const void* B, int64_t ldb, const void* C, int64_t ldc,
                                                void* out, int64_t ldo, int32_t total_tokens, int32_t n_seq,
                                                int32_t max_seqlen, const int32_t* cu_seqlens, const int32_t* init_slot,
                                                const int32_t* final_slot, const mdraft_prefill_opts* opts,
                                                int32_t* dev_status, void* stream) {
    // Size check first, on the host: an oversized problem is refused before CUDA is touched at all.
    size_t need = 0;
    if (layer && total_tokens > 0 && n_seq > 0)
        need = mdraft_prefill_workspace_bytes(layer, total_tokens, n_seq, max_seqlen > 0 ? max_seqlen : 1, opts);
    if (need > (size_t)MDRAFT_NOALLOC_SCRATCH_BYTES) return MDRAFT_ERR_WORKSPACE;
    void* scratch = nullptr;
    if (need > 0) {
        int rc = scratch_for_current_device(&scratch);
        if (rc != MDRAFT_OK) return rc;
    }
    return mdraft_conv_scan_prefill(layer, cache, layer_index, x, ldx, z, ldz, dt, lddt, B, ldb, C, ldc, out, ldo, total_tokens,
                                    n_seq, max_seqlen, cu_seqlens, init_slot, final_slot, scratch, need, opts, dev_status, stream);
}
