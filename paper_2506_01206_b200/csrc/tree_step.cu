// Draft-tree step: every node of a tree level takes one token from its parent's state.
//
// One thread owns one channel of one node: it gathers the parent's 16 state entries (four 128-bit loads, all in
// flight together with the node's inputs, the conv window and the layer constants), advances the conv window and
// the state by one token, and writes the child's state straight from registers to the child's slot — forking
// costs no copy.  A block is 128 consecutive channels of one node; siblings are separate blocks that re-read the
// parent (the second reader finds it in L2), so a level's latency does not grow with its branching factor.
// The kernel is bound by HBM traffic: one state read and one state write per node and layer.
#include "common.cuh"
#include "tree_step.cuh"

namespace mdraft {

namespace {

// 16 consecutive activations (one row of B or C) as fp32.
template <typename AT> struct Row16;
template <> struct Row16<float> {
    __device__ static __forceinline__ void load(const float* p, float (&v)[kN]) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float4 t = __ldg(reinterpret_cast<const float4*>(p) + q);
            v[4 * q] = t.x; v[4 * q + 1] = t.y; v[4 * q + 2] = t.z; v[4 * q + 3] = t.w;
        }
    }
};
template <> struct Row16<__nv_bfloat16> {
    __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&v)[kN]) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const uint4 t = __ldg(reinterpret_cast<const uint4*>(p) + q);
            const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                v[8 * q + 2 * i] = __uint_as_float(w[i] << 16);
                v[8 * q + 2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
            }
        }
    }
};

template <typename AT, bool kPow>
__global__ void __launch_bounds__(kTreeThreads) tree_step_kernel(const TreeArgs p) {
    const int D = p.L.d_inner;
    const int node = p.lvl_begin + blockIdx.x;
    const int d = blockIdx.y * kTreeThreads + threadIdx.x;
    const int pslot = __ldg(p.parent_slot + node);
    const int nslot = __ldg(p.node_slot + node);
    if (pslot < -1 || pslot >= p.pool.n_slots || nslot < 0 || nslot >= p.pool.n_slots) {  // the node becomes a no-op
        if (threadIdx.x == 0 && blockIdx.y == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
        return;
    }
    if (d >= D) return;

    const uint32_t flags = p.L.flags;
    const bool preconv = flags & MDRAFT_PRECONV, conv_only = flags & MDRAFT_CONV_ONLY;
    const AT* x = static_cast<const AT*>(p.x);
    AT* out = static_cast<AT*>(p.out);
    AT* conv_pool = static_cast<AT*>(p.pool.conv);

    // ---- everything is requested before anything is used
    float4 hq[kN / 4];
#pragma unroll
    for (int q = 0; q < kN / 4; ++q) hq[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (!conv_only && pslot >= 0) {
        const float4* src = reinterpret_cast<const float4*>(p.pool.ssm + (size_t)pslot * p.pool.ssm_slot_stride + (size_t)d * kN);
#pragma unroll
        for (int q = 0; q < kN / 4; ++q) hq[q] = src[q];
    }
    float win[kW - 1] = {0.f, 0.f, 0.f};
    if (!preconv && pslot >= 0) {
#pragma unroll
        for (int j = 0; j < kW - 1; ++j) win[j] = Act<AT>::to_f32(conv_pool[(size_t)pslot * p.pool.conv_slot_stride + (size_t)j * D + d]);
    }
    const float xv = Act<AT>::load(x + (size_t)node * p.ldx + d);
    float zv = 0.f, dtv = 0.f, Bv[kN], Cv[kN], a2[kPow ? 1 : kN];
    float4 wv = make_float4(0.f, 0.f, 0.f, 0.f);
    float cb = 0.f, dtb = 0.f, dsk = 0.f;
    if (!preconv) {
        wv = __ldg(reinterpret_cast<const float4*>(p.L.conv_w + (size_t)d * kW));
        cb = p.L.conv_b ? __ldg(p.L.conv_b + d) : 0.f;
    }
    if (!conv_only) {
        zv = Act<AT>::load(static_cast<const AT*>(p.z) + (size_t)node * p.ldz + d);
        dtv = Act<AT>::load(static_cast<const AT*>(p.dt) + (size_t)node * p.lddt + d);
        Row16<AT>::load(static_cast<const AT*>(p.B) + (size_t)node * p.ldb, Bv);
        Row16<AT>::load(static_cast<const AT*>(p.C) + (size_t)node * p.ldc, Cv);
        if constexpr (kPow) {
            a2[0] = __ldg(p.L.A + (size_t)d * kN) * kLog2e;
        } else {
#pragma unroll
            for (int q = 0; q < kN / 4; ++q) {
                const float4 a = __ldg(reinterpret_cast<const float4*>(p.L.A + (size_t)d * kN) + q);
                a2[4 * q] = a.x * kLog2e; a2[4 * q + 1] = a.y * kLog2e; a2[4 * q + 2] = a.z * kLog2e; a2[4 * q + 3] = a.w * kLog2e;
            }
        }
        dtb = p.L.dt_bias ? __ldg(p.L.dt_bias + d) : 0.f;
        dsk = p.L.D ? __ldg(p.L.D + d) : 0.f;
    }

    // ---- conv window
    float u;
    if (preconv) {
        u = xv;
    } else {
        float acc = fmaf(wv.x, win[0], cb);
        acc = fmaf(wv.y, win[1], acc);
        acc = fmaf(wv.z, win[2], acc);
        acc = fmaf(wv.w, xv, acc);
        u = silu(acc);
        AT* dst = conv_pool + (size_t)nslot * p.pool.conv_slot_stride + d;
        dst[0] = Act<AT>::from_f32(win[1]);
        dst[(size_t)D] = Act<AT>::from_f32(win[2]);
        dst[(size_t)2 * D] = Act<AT>::from_f32(xv);
    }
    if (conv_only) {
        out[(size_t)node * p.ldo + d] = Act<AT>::from_f32(u);
        return;
    }

    // ---- one step of the recurrence
    const float v = dtv + dtb;
    const float delta = (flags & MDRAFT_DT_SOFTPLUS) ? softplus(v) : v;
    const float du = delta * u;
    float P[kN];
    if constexpr (kPow) {
        const float r1 = ex2(delta * a2[0]);
        const float r2 = r1 * r1, r4 = r2 * r2, r8 = r4 * r4;
        P[0] = r1; P[1] = r2; P[2] = r2 * r1; P[3] = r4;
        P[4] = r4 * r1; P[5] = r4 * r2; P[6] = r4 * P[2]; P[7] = r8;
#pragma unroll
        for (int n = 0; n < 8; ++n) P[8 + n] = r8 * P[n];
    } else {
#pragma unroll
        for (int n = 0; n < kN; ++n) P[n] = ex2(delta * a2[n]);
    }
    float h[kN];
#pragma unroll
    for (int q = 0; q < kN / 4; ++q) { h[4 * q] = hq[q].x; h[4 * q + 1] = hq[q].y; h[4 * q + 2] = hq[q].z; h[4 * q + 3] = hq[q].w; }
    float y0 = 0.f, y1 = 0.f;
#pragma unroll
    for (int n = 0; n < kN; ++n) {
        h[n] = fmaf(P[n], h[n], du * Bv[n]);
        if (n & 1) y1 = fmaf(Cv[n], h[n], y1); else y0 = fmaf(Cv[n], h[n], y0);
    }
    float4* dst = reinterpret_cast<float4*>(p.pool.ssm + (size_t)nslot * p.pool.ssm_slot_stride + (size_t)d * kN);
#pragma unroll
    for (int q = 0; q < kN / 4; ++q) dst[q] = make_float4(h[4 * q], h[4 * q + 1], h[4 * q + 2], h[4 * q + 3]);
    const float y = fmaf(dsk, u, y0 + y1);
    out[(size_t)node * p.ldo + d] = Act<AT>::from_f32(y * silu(zv));
}

}  // namespace

cudaError_t launch_tree_step(const TreeArgs& p, int act, cudaStream_t st) {
    const int n = p.lvl_end - p.lvl_begin;
    if (n <= 0) return cudaSuccess;
    const bool pow = p.L.flags & MDRAFT_A_POWERS;
    dim3 grid(n, (p.L.d_inner + kTreeThreads - 1) / kTreeThreads);
    if (act == MDRAFT_F32) {
        if (pow) tree_step_kernel<float, true><<<grid, kTreeThreads, 0, st>>>(p);
        else tree_step_kernel<float, false><<<grid, kTreeThreads, 0, st>>>(p);
    } else {
        if (pow) tree_step_kernel<__nv_bfloat16, true><<<grid, kTreeThreads, 0, st>>>(p);
        else tree_step_kernel<__nv_bfloat16, false><<<grid, kTreeThreads, 0, st>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace mdraft
