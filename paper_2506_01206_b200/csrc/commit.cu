// Accepted-path commit: slot dst <- slot src for every layer, as raw 128-bit words (bit-exact by construction).
#include "commit.cuh"

namespace mdraft {

namespace {

constexpr int kCommitThreads = 256;
constexpr int kWordsPerThread = 4;  // 4 x 16 bytes in flight per thread

__global__ void __launch_bounds__(kCommitThreads) commit_kernel(CommitArgs p) {
    const int j = blockIdx.z, layer = blockIdx.y;
    const int src = __ldg(p.src_slot + j), dst = __ldg(p.dst_slot + j);
    if (src < 0 || src >= p.n_slots || dst < 0 || dst >= p.n_slots) {
        if (threadIdx.x == 0 && blockIdx.x == 0 && layer == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
        return;
    }
    if (src == dst) return;
    const int64_t ssm_words = p.ssm_bytes / 16, conv_words = p.conv_bytes / 16, words = ssm_words + conv_words;
    const uint4* s_ssm = reinterpret_cast<const uint4*>(p.ssm + layer * p.ssm_layer_bytes + src * p.ssm_slot_bytes_stride);
    uint4* d_ssm = reinterpret_cast<uint4*>(p.ssm + layer * p.ssm_layer_bytes + dst * p.ssm_slot_bytes_stride);
    const uint4* s_conv = reinterpret_cast<const uint4*>(p.conv + layer * p.conv_layer_bytes + src * p.conv_slot_bytes_stride);
    uint4* d_conv = reinterpret_cast<uint4*>(p.conv + layer * p.conv_layer_bytes + dst * p.conv_slot_bytes_stride);
    const int64_t base = (int64_t)blockIdx.x * kCommitThreads * kWordsPerThread + threadIdx.x;
    uint4 v[kWordsPerThread];
#pragma unroll
    for (int i = 0; i < kWordsPerThread; ++i) {
        int64_t w = base + (int64_t)i * kCommitThreads;
        if (w < ssm_words) v[i] = s_ssm[w];
        else if (w < words) v[i] = s_conv[w - ssm_words];
    }
#pragma unroll
    for (int i = 0; i < kWordsPerThread; ++i) {
        int64_t w = base + (int64_t)i * kCommitThreads;
        if (w < ssm_words) d_ssm[w] = v[i];
        else if (w < words) d_conv[w - ssm_words] = v[i];
    }
}

}  // namespace

cudaError_t launch_commit(const CommitArgs& p, cudaStream_t st) {
    if (p.n_commit <= 0 || p.n_layers <= 0) return cudaSuccess;
    const int64_t words = (p.ssm_bytes + p.conv_bytes) / 16;
    const int64_t per_block = (int64_t)kCommitThreads * kWordsPerThread;
    dim3 grid((unsigned)((words + per_block - 1) / per_block), p.n_layers, p.n_commit);
    commit_kernel<<<grid, kCommitThreads, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace mdraft
