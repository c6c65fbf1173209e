// Draft-tree step: every node of a tree level takes one token from its parent's state.
//
// A block is 128 consecutive channels of one node.  Everything the block needs of that node is contiguous in
// memory — the parent's state slice (128 x 16 fp32 = 8 KB), three conv-window rows, the x / z / dt rows and the
// B / C rows — so one thread fetches it with a handful of bulk asynchronous copies (cp.async.bulk, completion
// counted on an mbarrier) into shared memory; each thread then advances its channel by one token in registers,
// puts the child's state, window and output back into the same shared-memory locations, and one thread sends
// them to the child's slot with bulk stores.  Forking therefore costs one read and one write of the state and
// no copy pass, all traffic is in multi-KB contiguous pieces, and the bytes in flight do not depend on how many
// registers a thread holds.  Siblings are separate blocks that re-read the parent (the second reader finds it in
// L2), so a level's latency does not grow with its branching factor.  The waits on the mbarriers are bounded: if one
// runs out the block raises MDRAFT_DEV_WAIT_EXPIRED, waits once more (bounded) for its copies, and returns.
//
// The levels of one call follow one another through programmatic dependent launch: a level's blocks start while the
// level before is still running, look up their slots, fetch the layer constants and the node's input
// rows, and only then wait for the kernel ahead, after which the parent's state and window are
// fetched.  Every block passes that wait on every path, so a level's completion implies the completion of everything
// before it.
#include "common.cuh"
#include "tree_step.cuh"

namespace mdraft {

namespace {

constexpr int kTB = kTreeThreads;            // channels per block

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes + kOverstateTx) : "memory");
}
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(kPollNs) : "memory");
        if (ok) return true;
    }
    return false;
}
// Bulk copies; addresses 16-byte aligned, sizes multiples of 16 bytes.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst)),
                 "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(__cvta_generic_to_global(dst)), "r"(smem_u32(src)),
                 "r"(bytes) : "memory");
}

__device__ __forceinline__ void swap4(float4& a, float4& b) { const float4 t = a; a = b; b = t; }
// t[i] <-> t[i ^ sw] for all i (sw in 0..3): turns "position i holds quad i ^ sw" into "position q holds quad q".
__device__ __forceinline__ void xor_permute(float4 (&t)[4], int sw) {
    if (sw & 1) { swap4(t[0], t[1]); swap4(t[2], t[3]); }
    if (sw & 2) { swap4(t[0], t[2]); swap4(t[1], t[3]); }
}

template <typename AT, bool kPow>
__global__ void __launch_bounds__(kTB) tree_step_kernel(const TreeArgs p, const int early_inputs, const int ordinary_launch) {
    __shared__ __align__(128) float4 s_h[kTB * (kN / 4)];  // state slice [channel][quad]
    __shared__ __align__(16) AT s_conv[kW - 1][kTB];
    __shared__ __align__(16) AT s_x[kTB];                 // the node's x row; receives the out row afterwards
    __shared__ __align__(16) AT s_z[kTB];
    __shared__ __align__(16) AT s_dt[kTB];
    __shared__ __align__(16) AT s_B[kN];
    __shared__ __align__(16) AT s_C[kN];
    __shared__ __align__(8) uint64_t bar, bar_in;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // the next level may begin its own look-ups
    // Launched the ordinary way nothing runs ahead of this kernel: the wait costs nothing, and passing it first lets
    // every copy be requested at once.
    if (ordinary_launch) asm volatile("griddepcontrol.wait;" ::: "memory");
    const int D = p.L.d_inner;
    const int node = p.lvl_begin + blockIdx.x;
    const int tid = threadIdx.x;
    const int d0 = blockIdx.y * kTB;
    const int cols = min(kTB, D - d0);
    const int d = d0 + tid;
    const bool live = tid < cols;
    const int pslot = __ldg(p.parent_slot + node);
    const int nslot = __ldg(p.node_slot + node);
    if (pslot < -1 || pslot >= p.pool.n_slots || nslot < 0 || nslot >= p.pool.n_slots) {  // the node becomes a no-op
        if (tid == 0 && blockIdx.y == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
        asm volatile("griddepcontrol.wait;" ::: "memory");
        return;
    }
    const uint32_t flags = p.L.flags;
    const bool preconv = flags & MDRAFT_PRECONV, conv_only = flags & MDRAFT_CONV_ONLY;
    const bool have_parent = pslot >= 0;
    const uint32_t row_bytes = (uint32_t)cols * sizeof(AT), bc_bytes = (uint32_t)kN * sizeof(AT), h_bytes = (uint32_t)cols * kN * 4u;
    float* h_parent = p.pool.ssm + (size_t)pslot * p.pool.ssm_slot_stride + (size_t)d0 * kN;
    float* h_child = p.pool.ssm + (size_t)nslot * p.pool.ssm_slot_stride + (size_t)d0 * kN;
    AT* conv_parent = static_cast<AT*>(p.pool.conv) + (size_t)pslot * p.pool.conv_slot_stride + d0;
    AT* conv_child = static_cast<AT*>(p.pool.conv) + (size_t)nslot * p.pool.conv_slot_stride + d0;

    // Inputs of the node (x, z, dt, B, C rows) go on one mbarrier, the parent's state and window on another: the
    // former may be requested before the kernel ahead has finished when the launch says they cannot be its work.
    auto issue_inputs = [&]() {
        uint32_t total = row_bytes;
        if (!conv_only) total += 2 * row_bytes + 2 * bc_bytes;
        mbar_expect_tx(&bar_in, total);
        bulk_load(s_x, static_cast<const AT*>(p.x) + (size_t)node * p.ldx + d0, row_bytes, &bar_in);
        if (!conv_only) {
            bulk_load(s_z, static_cast<const AT*>(p.z) + (size_t)node * p.ldz + d0, row_bytes, &bar_in);
            bulk_load(s_dt, static_cast<const AT*>(p.dt) + (size_t)node * p.lddt + d0, row_bytes, &bar_in);
            bulk_load(s_B, static_cast<const AT*>(p.B) + (size_t)node * p.ldb, bc_bytes, &bar_in);
            bulk_load(s_C, static_cast<const AT*>(p.C) + (size_t)node * p.ldc, bc_bytes, &bar_in);
        }
    };
    auto issue_state = [&]() {
        uint32_t total = 0;
        if (!conv_only && have_parent) total += h_bytes;
        if (!preconv && have_parent) total += (kW - 1) * row_bytes;
        mbar_expect_tx(&bar, total);
        if (!conv_only && have_parent) bulk_load(s_h, h_parent, h_bytes, &bar);
        if (!preconv && have_parent)
            for (int j = 0; j < kW - 1; ++j) bulk_load(s_conv[j], conv_parent + (size_t)j * D, row_bytes, &bar);
    };
    if (tid == 0) {
        mbar_init(&bar, 1);
        mbar_init(&bar_in, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (early_inputs || ordinary_launch) issue_inputs();
        if (ordinary_launch) issue_state();
    }

    // Layer constants travel by ordinary loads while the copies are in flight.
    float a2[kPow ? 1 : kN];
    float4 wv = make_float4(0.f, 0.f, 0.f, 0.f);
    float cb = 0.f, dtb = 0.f, dsk = 0.f;
    if (live) {
        if (!preconv) {
            wv = __ldg(reinterpret_cast<const float4*>(p.L.conv_w + (size_t)d * kW));
            cb = p.L.conv_b ? __ldg(p.L.conv_b + d) : 0.f;
        }
        if (!conv_only) {
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
    }
    if (!ordinary_launch) {
        asm volatile("griddepcontrol.wait;" ::: "memory");  // everything read from here on may be the work of the kernel ahead
        if (tid == 0) {
            if (!early_inputs) issue_inputs();
            issue_state();
        }
    }
    __syncthreads();  // the mbarriers are initialised for everyone
    const bool ok = mbar_wait_bounded(&bar_in, 0u) && mbar_wait_bounded(&bar, 0u);
    if (__syncthreads_or(!ok)) {
        if (tid == 0) {
            flag(p.dev_status, MDRAFT_DEV_WAIT_EXPIRED);
            mbar_wait_bounded(&bar_in, 0u); mbar_wait_bounded(&bar, 0u);
        }
        return;
    }

    if (live) {
        const float xv = Act<AT>::to_f32(s_x[tid]);
        // ---- conv window: (w0, w1, w2, x) -> (w1, w2, x)
        float u;
        if (preconv) {
            u = xv;
        } else {
            float win[kW - 1] = {0.f, 0.f, 0.f};
            if (have_parent) {
#pragma unroll
                for (int j = 0; j < kW - 1; ++j) win[j] = Act<AT>::to_f32(s_conv[j][tid]);
            }
            float acc = fmaf(wv.x, win[0], cb);
            acc = fmaf(wv.y, win[1], acc);
            acc = fmaf(wv.z, win[2], acc);
            acc = fmaf(wv.w, xv, acc);
            u = silu(acc);
            s_conv[0][tid] = Act<AT>::from_f32(win[1]);
            s_conv[1][tid] = Act<AT>::from_f32(win[2]);
            s_conv[2][tid] = Act<AT>::from_f32(xv);
        }
        float o = u;
        if (!conv_only) {
            // ---- one step of the recurrence.  The quads of a channel are visited in an order that differs between
            // neighbouring threads, which keeps the 128-bit shared-memory accesses free of bank conflicts.
            const int sw = (tid >> 1) & 3;
            float4 hq[kN / 4];
#pragma unroll
            for (int i = 0; i < kN / 4; ++i) hq[i] = have_parent ? s_h[tid * (kN / 4) + (i ^ sw)] : make_float4(0.f, 0.f, 0.f, 0.f);
            xor_permute(hq, sw);
            const float zv = Act<AT>::to_f32(s_z[tid]);
            const float v = Act<AT>::to_f32(s_dt[tid]) + dtb;
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
                h[n] = fmaf(P[n], h[n], du * Act<AT>::to_f32(s_B[n]));
                if (n & 1) y1 = fmaf(Act<AT>::to_f32(s_C[n]), h[n], y1); else y0 = fmaf(Act<AT>::to_f32(s_C[n]), h[n], y0);
            }
#pragma unroll
            for (int q = 0; q < kN / 4; ++q) hq[q] = make_float4(h[4 * q], h[4 * q + 1], h[4 * q + 2], h[4 * q + 3]);
            xor_permute(hq, sw);
#pragma unroll
            for (int i = 0; i < kN / 4; ++i) s_h[tid * (kN / 4) + (i ^ sw)] = hq[i];
            o = fmaf(dsk, u, y0 + y1) * silu(zv);
        }
        s_x[tid] = Act<AT>::from_f32(o);
    }
    // Shared-memory writes above must be visible to the copy engine before it reads them.
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (tid == 0) {
        if (!conv_only) bulk_store(h_child, s_h, h_bytes);
        if (!preconv)
            for (int j = 0; j < kW - 1; ++j) bulk_store(conv_child + (size_t)j * D, s_conv[j], row_bytes);
        bulk_store(static_cast<AT*>(p.out) + (size_t)node * p.ldo + d0, s_x, row_bytes);
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // shared memory stays valid until it has been read
    }
}

}  // namespace

// The first level of a call is launched the ordinary way: what runs ahead of it is usually somebody else's kernel (a
// projection), which never releases its dependents early, and behind such a kernel a programmatic launch was measured
// 0.8 us slower than an ordinary one.  Later levels follow a level of the same call and are launched programmatically.
template <typename K>
cudaError_t launch_level(K kernel, dim3 grid, cudaStream_t st, const TreeArgs& p, int early) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kTB);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.level_in_call > 0 ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, p, early, p.level_in_call > 0 ? 0 : 1);
}

cudaError_t launch_tree_step(const TreeArgs& p, int act, cudaStream_t st) {
    const int n = p.lvl_end - p.lvl_begin;
    if (n <= 0) return cudaSuccess;
    const bool pow = p.L.flags & MDRAFT_A_POWERS;
    // The first kernel of a call is an ordinary launch: it starts only after everything ahead of the call has finished.
    // A later level starts when the level before it does, so the only kernels that can still be running then are
    // levels of this call, which write states and `out` rows of other nodes only: the node's input rows cannot be
    // their work and are requested before the wait.
    const int early = p.level_in_call >= 1 ? 1 : 0;
    dim3 grid(n, (p.L.d_inner + kTB - 1) / kTB);
    if (act == MDRAFT_F32) {
        if (pow) return launch_level(tree_step_kernel<float, true>, grid, st, p, early);
        return launch_level(tree_step_kernel<float, false>, grid, st, p, early);
    }
    if (pow) return launch_level(tree_step_kernel<__nv_bfloat16, true>, grid, st, p, early);
    return launch_level(tree_step_kernel<__nv_bfloat16, false>, grid, st, p, early);
}

}  // namespace mdraft
