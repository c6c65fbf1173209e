// Draft-tree step of a Mamba-2 (SSD) layer: every node of a level takes one token from its parent's state.
//
// The state of a node is D x 128 fp32 (786 KB for the 130M shape), eight times that of the S6 layer, so the step is
// pure memory traffic: read the parent's state, one multiply-add per entry, write the child's.  A block takes 32
// channels of one node; a warp 4 channels, 8 lanes per channel, each lane 16 state entries as four 128-bit words
// (the 8 lanes of a channel read 128 contiguous bytes per word index).  The contraction with C is finished by three
// shuffles.  Forking is the gather itself: read slot parent_slot[i], write slot node_slot[i], no copy pass.
#include "common.cuh"
#include "ssd.cuh"

namespace mdraft {

namespace {

constexpr int kStepThreads = 256, kStepChannels = 32;

__device__ __forceinline__ float bfv(const __nv_bfloat16* p) { return __bfloat162float(*p); }

__global__ void __launch_bounds__(kStepThreads) ssd_step_kernel(const SsdStepArgs p) {
    const int D = p.L.d_inner;
    const int node = p.lvl_begin + blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d = blockIdx.y * kStepChannels + warp * 4 + (lane >> 3);
    const int j = lane & 7;                       // this lane's share of the channel's 128 states: n = 4 j + 32 i
    const int head = d / kSsdP;
    const int pslot = __ldg(p.parent_slot + node), nslot = __ldg(p.node_slot + node);
    if (pslot < -1 || pslot >= p.pool.n_slots || nslot < 0 || nslot >= p.pool.n_slots) {   // the node becomes a no-op
        if (tid == 0 && blockIdx.y == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
        return;
    }
    if (d >= D) return;
    const bool have_parent = pslot >= 0;
    const __nv_bfloat16* conv_parent = static_cast<const __nv_bfloat16*>(p.pool.conv) + (size_t)pslot * p.pool.conv_slot_stride + d;
    __nv_bfloat16* conv_child = static_cast<__nv_bfloat16*>(p.pool.conv) + (size_t)nslot * p.pool.conv_slot_stride + d;
    const float4* hp = reinterpret_cast<const float4*>(p.pool.ssm + (size_t)pslot * p.pool.ssm_slot_stride + (size_t)d * kSsdN) + j;
    float4* hc = reinterpret_cast<float4*>(p.pool.ssm + (size_t)nslot * p.pool.ssm_slot_stride + (size_t)d * kSsdN) + j;

    // the parent's state first: these are the loads the step waits for
    float4 h[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = have_parent ? hp[8 * i] : make_float4(0.f, 0.f, 0.f, 0.f);

    const float xv = bfv(p.x + (size_t)node * p.ldx + d);
    float w0 = 0.f, w1 = 0.f, w2 = 0.f;
    if (have_parent) { w0 = bfv(conv_parent); w1 = bfv(conv_parent + D); w2 = bfv(conv_parent + 2 * (size_t)D); }
    const float4 wv = __ldg(reinterpret_cast<const float4*>(p.L.conv_w + (size_t)d * kW));
    float acc = fmaf(wv.x, w0, p.L.conv_b ? __ldg(p.L.conv_b + d) : 0.f);
    acc = fmaf(wv.y, w1, acc);
    acc = fmaf(wv.z, w2, acc);
    acc = fmaf(wv.w, xv, acc);
    const float u = silu(acc);
    const float v = bfv(p.dt + (size_t)node * p.lddt + head) + (p.L.dt_bias ? __ldg(p.L.dt_bias + head) : 0.f);
    const float delta = (p.L.flags & MDRAFT_DT_SOFTPLUS) ? softplus(v) : v;
    const float decay = ex2(delta * __ldg(p.L.A + head) * kLog2e);
    const float du = delta * u;

    float y = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int n = 4 * j + 32 * i;
        const uint2 braw = *reinterpret_cast<const uint2*>(p.B + (size_t)node * p.ldb + n);
        const uint2 craw = *reinterpret_cast<const uint2*>(p.C + (size_t)node * p.ldc + n);
        const float b0 = __uint_as_float(braw.x << 16), b1 = __uint_as_float(braw.x & 0xffff0000u);
        const float b2 = __uint_as_float(braw.y << 16), b3 = __uint_as_float(braw.y & 0xffff0000u);
        const float c0 = __uint_as_float(craw.x << 16), c1 = __uint_as_float(craw.x & 0xffff0000u);
        const float c2 = __uint_as_float(craw.y << 16), c3 = __uint_as_float(craw.y & 0xffff0000u);
        h[i].x = fmaf(decay, h[i].x, du * b0); h[i].y = fmaf(decay, h[i].y, du * b1);
        h[i].z = fmaf(decay, h[i].z, du * b2); h[i].w = fmaf(decay, h[i].w, du * b3);
        y = fmaf(c0, h[i].x, y); y = fmaf(c1, h[i].y, y); y = fmaf(c2, h[i].z, y); y = fmaf(c3, h[i].w, y);
        hc[8 * i] = h[i];
    }
    y += __shfl_xor_sync(0xffffffffu, y, 1);
    y += __shfl_xor_sync(0xffffffffu, y, 2);
    y += __shfl_xor_sync(0xffffffffu, y, 4);
    if (j == 0) {
        const float zv = bfv(p.z + (size_t)node * p.ldz + d);
        const float dsk = p.L.D ? __ldg(p.L.D + d) : 0.f;
        p.out[(size_t)node * p.ldo + d] = __float2bfloat16_rn(fmaf(dsk, u, y) * silu(zv));
        conv_child[0] = __float2bfloat16_rn(w1);
        conv_child[D] = __float2bfloat16_rn(w2);
        conv_child[2 * (size_t)D] = __float2bfloat16_rn(xv);
    }
}

}  // namespace

cudaError_t launch_ssd_step(const SsdStepArgs& p, cudaStream_t st) {
    const int n = p.lvl_end - p.lvl_begin;
    if (n <= 0) return cudaSuccess;
    dim3 grid(n, (p.L.d_inner + kStepChannels - 1) / kStepChannels);
    ssd_step_kernel<<<grid, kStepThreads, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace mdraft
