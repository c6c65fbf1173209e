// Draft-tree step: every node of a tree level takes one token from its parent's state.
//
// Mapping: 4 consecutive lanes share a channel, each owning 4 of the 16 state entries (one 128-bit load and one
// 128-bit store of fp32 state per lane; a warp touches 8 channels = 512 contiguous bytes of a slot).  The same 4
// lanes hold the 4 entries of the conv window (3 cached rows + the node's own input) and each multiplies one
// tap; window and y are summed across the 4 lanes with two xor-shuffles.  Consecutive nodes with the same
// parent slot ("a run" — siblings in breadth-first order) are handled by the first node's block, which reads the
// parent's state once and keeps it in registers for all of them.  The child's state goes straight from
// registers to the child's slot: forking costs no copy.
#include "common.cuh"
#include "tree_step.cuh"

namespace mdraft {

namespace {

constexpr int kChPerBlock = kTreeThreads / 4;

template <typename AT> struct Quad;  // 4 consecutive activations
template <> struct Quad<float> {
    __device__ static __forceinline__ void load(const float* p, float (&v)[4]) {
        float4 t = __ldg(reinterpret_cast<const float4*>(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
};
template <> struct Quad<__nv_bfloat16> {
    __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&v)[4]) {
        uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
        v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
        v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
    }
};

__device__ __forceinline__ float quad_sum(float v) {
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    return v;
}

template <typename AT>
__global__ void __launch_bounds__(kTreeThreads) tree_step_kernel(TreeArgs p) {
    const int D = p.L.d_inner;
    const int node0 = p.lvl_begin + blockIdx.x;
    const int q = threadIdx.x & 3;
    const int d = blockIdx.y * kChPerBlock + (threadIdx.x >> 2);
    const bool live = d < D;  // uniform within each group of 4 lanes

    const int pslot = __ldg(p.parent_slot + node0);
    if (node0 > p.lvl_begin && __ldg(p.parent_slot + node0 - 1) == pslot) return;  // handled by the head of its run
    if (pslot < -1 || pslot >= p.pool.n_slots) {  // bad parent: every node of the run becomes a no-op
        if (threadIdx.x == 0 && blockIdx.y == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
        return;
    }
    const uint32_t flags = p.L.flags;
    const bool preconv = flags & MDRAFT_PRECONV, conv_only = flags & MDRAFT_CONV_ONLY;
    const AT* x = static_cast<const AT*>(p.x);
    const AT* z = static_cast<const AT*>(p.z);
    const AT* dt = static_cast<const AT*>(p.dt);
    const AT* B = static_cast<const AT*>(p.B);
    const AT* C = static_cast<const AT*>(p.C);
    AT* out = static_cast<AT*>(p.out);
    AT* conv_pool = static_cast<AT*>(p.pool.conv);

    // Parent state and layer constants for this lane's (channel, quarter of the state).
    float hp[4] = {0.f, 0.f, 0.f, 0.f}, a2[4] = {0.f, 0.f, 0.f, 0.f};
    float wq = 0.f, winq = 0.f, cb = 0.f, dtb = 0.f, dsk = 0.f;
    if (live) {
        if (!conv_only) {
            if (pslot >= 0) {
                float4 t = *reinterpret_cast<const float4*>(p.pool.ssm + (size_t)pslot * p.pool.ssm_slot_stride + (size_t)d * kN + 4 * q);
                hp[0] = t.x; hp[1] = t.y; hp[2] = t.z; hp[3] = t.w;
            }
            float4 a = __ldg(reinterpret_cast<const float4*>(p.L.A + (size_t)d * kN + 4 * q));
            a2[0] = a.x * kLog2e; a2[1] = a.y * kLog2e; a2[2] = a.z * kLog2e; a2[3] = a.w * kLog2e;
            dtb = p.L.dt_bias ? __ldg(p.L.dt_bias + d) : 0.f;
            dsk = p.L.D ? __ldg(p.L.D + d) : 0.f;
        }
        if (!preconv) {
            wq = __ldg(p.L.conv_w + (size_t)d * kW + q);
            cb = p.L.conv_b ? __ldg(p.L.conv_b + d) : 0.f;
            if (q < kW - 1 && pslot >= 0)
                winq = Act<AT>::to_f32(conv_pool[(size_t)pslot * p.pool.conv_slot_stride + (size_t)q * D + d]);
        }
    }

    for (int node = node0; node < p.lvl_end; ++node) {
        if (node > node0 && __ldg(p.parent_slot + node) != pslot) break;
        const int nslot = __ldg(p.node_slot + node);
        if (nslot < 0 || nslot >= p.pool.n_slots) {
            if (threadIdx.x == 0 && blockIdx.y == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
            continue;
        }
        float xv = 0.f, o = 0.f;
        if (live) xv = Act<AT>::load(x + (size_t)node * p.ldx + d);
        float u;
        const float mine = (q < kW - 1) ? winq : xv;  // this lane's entry of the conv window
        if (preconv) {
            u = xv;
        } else {
            u = silu(quad_sum(wq * mine) + cb);
            if (live && q >= 1) conv_pool[(size_t)nslot * p.pool.conv_slot_stride + (size_t)(q - 1) * D + d] = Act<AT>::from_f32(mine);
        }
        if (conv_only) {
            o = u;
        } else {
            float bq[4] = {0.f, 0.f, 0.f, 0.f}, cq[4] = {0.f, 0.f, 0.f, 0.f}, dtv = 0.f, zv = 0.f;
            if (live) {
                Quad<AT>::load(B + (size_t)node * p.ldb + 4 * q, bq);
                Quad<AT>::load(C + (size_t)node * p.ldc + 4 * q, cq);
                dtv = Act<AT>::load(dt + (size_t)node * p.lddt + d);
                zv = Act<AT>::load(z + (size_t)node * p.ldz + d);
            }
            float v = dtv + dtb;
            float delta = (flags & MDRAFT_DT_SOFTPLUS) ? softplus(v) : v;
            float du = delta * u;
            float hn[4], yp = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                hn[i] = fmaf(ex2(delta * a2[i]), hp[i], du * bq[i]);
                yp = fmaf(cq[i], hn[i], yp);
            }
            float y = fmaf(dsk, u, quad_sum(yp));
            o = y * silu(zv);
            if (live)
                *reinterpret_cast<float4*>(p.pool.ssm + (size_t)nslot * p.pool.ssm_slot_stride + (size_t)d * kN + 4 * q) =
                    make_float4(hn[0], hn[1], hn[2], hn[3]);
        }
        if (live && q == 0) out[(size_t)node * p.ldo + d] = Act<AT>::from_f32(o);
    }
}

}  // namespace

cudaError_t launch_tree_step(const TreeArgs& p, int act, cudaStream_t st) {
    const int n = p.lvl_end - p.lvl_begin;
    if (n <= 0) return cudaSuccess;
    dim3 grid(n, (p.L.d_inner + kChPerBlock - 1) / kChPerBlock);
    if (act == MDRAFT_F32) tree_step_kernel<float><<<grid, kTreeThreads, 0, st>>>(p);
    else tree_step_kernel<__nv_bfloat16><<<grid, kTreeThreads, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace mdraft
