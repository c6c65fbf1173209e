// Draft-tree step of a whole Mamba block core: conv step, the block's two selection projections, recurrence, gate.
//
// In the drafter's block the step size, B and C of a token are linear functions of the conv output of ALL channels
// (s = W_x u; dt = W_dt s[0:R]; B = s[R:R+N]; C = s[R+N:R+2N]), so between the conv step and the recurrence sits a
// reduction over the channel axis.  Here the blocks of one node form a thread-block cluster along the channel axis:
// every block convolves its channels, multiplies them into its share of s (a partial sum per row of W_x), the
// cluster meets at its hardware barrier, every block adds the partial sums of all blocks out of their shared memory
// (distributed shared memory, fixed order, so all blocks hold the same bits), forms the step size of its own channels
// from its rows of W_dt and advances the recurrence.  One launch per tree level replaces the conv step, two
// matrix products, three slicing copies and the recurrence step of the split mode; nothing goes through global
// memory in between.
//
// The parent's state slice, window rows and the node's x / z rows arrive by bulk asynchronous copies counted on two
// mbarriers (window and x first, state and z later, so the projections overlap the 16-32 KB state fetch); the child's
// state, window and output leave by bulk stores.  All waits on the mbarriers are bounded.  The cluster barrier is
// executed unconditionally by every thread of every block of the cluster (a block that gave up on its copies still
// takes part), so no block can wait for one that left.
#include "common.cuh"
#include "tree_proj.cuh"

namespace mdraft {

namespace {

constexpr int kMaxRows = kProjMaxRank + 2 * kN;

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
// Bulk copies; addresses 16-byte aligned, sizes multiples of 16 bytes.  The destination and the mbarrier are this
// block's own shared memory (a block's own addresses are valid in the cluster window).
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst)),
                 "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(__cvta_generic_to_global(dst)), "r"(smem_u32(src)),
                 "r"(bytes) : "memory");
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_size() {
    uint32_t n;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(n));
    return n;
}
// The float that block `rank` of this cluster keeps at the place where this block keeps *local.
__device__ __forceinline__ float peer_block_float(const float* local, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local)), "r"(rank));
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

__device__ __forceinline__ void swap4(float4& a, float4& b) { const float4 t = a; a = b; b = t; }
__device__ __forceinline__ void xor_permute(float4 (&t)[4], int sw) {
    if (sw & 1) { swap4(t[0], t[1]); swap4(t[2], t[3]); }
    if (sw & 2) { swap4(t[0], t[2]); swap4(t[1], t[3]); }
}

// Four consecutive weights as floats.
__device__ __forceinline__ float4 load_w4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float4 load_w4(const __nv_bfloat16* p) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u), __uint_as_float(v.y << 16),
                       __uint_as_float(v.y & 0xffff0000u));
}
// Eight consecutive weights, kept as loaded until they are used.
template <typename AT> struct Raw8;
template <> struct Raw8<float> {
    float4 a, b;
    __device__ __forceinline__ void load(const float* p) { a = load_w4(p); b = load_w4(p + 4); }
    __device__ __forceinline__ float4 lo() const { return a; }
    __device__ __forceinline__ float4 hi() const { return b; }
};
template <> struct Raw8<__nv_bfloat16> {
    uint4 v;
    __device__ __forceinline__ void load(const __nv_bfloat16* p) { v = __ldg(reinterpret_cast<const uint4*>(p)); }
    __device__ __forceinline__ float4 lo() const {
        return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u), __uint_as_float(v.y << 16),
                           __uint_as_float(v.y & 0xffff0000u));
    }
    __device__ __forceinline__ float4 hi() const {
        return make_float4(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xffff0000u), __uint_as_float(v.w << 16),
                           __uint_as_float(v.w & 0xffff0000u));
    }
};
// Four consecutive weights as loaded (8 or 16 bytes).
template <typename AT> struct Raw4;
template <> struct Raw4<float> {
    float4 v;
    __device__ __forceinline__ void load(const float* p) { v = load_w4(p); }
    __device__ __forceinline__ float4 get() const { return v; }
};
template <> struct Raw4<__nv_bfloat16> {
    uint2 v;
    __device__ __forceinline__ void load(const __nv_bfloat16* p) { v = __ldg(reinterpret_cast<const uint2*>(p)); }
    __device__ __forceinline__ float4 get() const {
        return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u), __uint_as_float(v.y << 16),
                           __uint_as_float(v.y & 0xffff0000u));
    }
};
__device__ __forceinline__ float dot4(const float4& a, const float4& b, float acc) {
    acc = fmaf(a.x, b.x, acc); acc = fmaf(a.y, b.y, acc); acc = fmaf(a.z, b.z, acc); acc = fmaf(a.w, b.w, acc);
    return acc;
}

// Shared-memory layout of a block: NT nodes x CB channels.  Byte offsets into the dynamic array; all multiples of 16.
template <typename AT, int CB, int NT>
struct ProjSmem {
    static constexpr int kH = 0;                                           // [NT][CB][16] fp32 state slices
    static constexpr int kConv = kH + NT * CB * kN * 4;                    // [NT][W-1][CB] window rows
    static constexpr int kX = kConv + NT * (kW - 1) * CB * (int)sizeof(AT);  // [NT][CB] x rows; receive the out rows
    static constexpr int kZ = kX + NT * CB * (int)sizeof(AT);              // [NT][CB] z rows
    static constexpr int kU = kZ + NT * CB * (int)sizeof(AT);              // [NT][CB] fp32 conv outputs
    static constexpr int kPart = kU + NT * CB * 4;                         // [NT][kMaxRows] this block's share of s
    static constexpr int kS = kPart + NT * kMaxRows * 4;                   // [NT][kMaxRows] s, summed over the cluster
    static constexpr int kBars = kS + NT * kMaxRows * 4;                   // [NT][2] mbarriers
    static constexpr int kTotal = kBars + NT * 2 * 8;
};

// A block is CB channels of NT consecutive nodes of the level; the blocks that cover one such group of nodes form
// the cluster.  With NT > 1 the rows of W_x and W_dt a thread holds serve NT nodes, which is what wide levels need
// (every node otherwise re-reads both matrices out of L2).
template <typename AT, int CB, int NT, bool kPow>
__global__ void __launch_bounds__(CB) tree_proj_kernel(const TreeProjArgs p) {
    constexpr int NW = CB / 32;    // warps
    constexpr int NP = CB / 128;   // a lane owns 4 consecutive channels in each of NP 128-channel spans
    using S = ProjSmem<AT, CB, NT>;
    extern __shared__ __align__(128) unsigned char s_dyn[];
    float4* const s_h = reinterpret_cast<float4*>(s_dyn + S::kH);
    AT* const s_conv = reinterpret_cast<AT*>(s_dyn + S::kConv);
    AT* const s_x = reinterpret_cast<AT*>(s_dyn + S::kX);
    AT* const s_z = reinterpret_cast<AT*>(s_dyn + S::kZ);
    float* const s_u = reinterpret_cast<float*>(s_dyn + S::kU);
    float* const s_part = reinterpret_cast<float*>(s_dyn + S::kPart);
    float* const s_s = reinterpret_cast<float*>(s_dyn + S::kS);
    uint64_t* const bars = reinterpret_cast<uint64_t*>(s_dyn + S::kBars);  // [i][0]: x + window, [i][1]: z + state

    const int D = p.L.d_inner, R = p.dt_rank, rows = R + 2 * kN;
    const int node0 = blockIdx.x * NT;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d0 = blockIdx.y * CB;
    const int cols = min(CB, D - d0);
    const int d = d0 + tid;
    const bool live = tid < cols;
    const uint32_t flags = p.L.flags;
    const uint32_t row_bytes = (uint32_t)cols * sizeof(AT), h_bytes = (uint32_t)cols * kN * 4u;

    // Slots of this block's nodes.  They are the nodes', not the block's, so every block of the cluster decides
    // alike; a node with a slot out of range is skipped (nothing loaded, nothing stored) but nobody leaves early.
    int pslot[NT], nslot[NT];
    bool valid[NT];
#pragma unroll
    for (int i = 0; i < NT; ++i) {
        valid[i] = node0 + i < p.n_nodes;
        pslot[i] = valid[i] ? __ldg(p.parent_slot + node0 + i) : -1;
        nslot[i] = valid[i] ? __ldg(p.node_slot + node0 + i) : 0;
        if (valid[i] && (pslot[i] < -1 || pslot[i] >= p.pool.n_slots || nslot[i] < 0 || nslot[i] >= p.pool.n_slots)) {
            valid[i] = false;
            if (tid == 0 && blockIdx.y == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
        }
    }

    if (tid == 0) {
#pragma unroll
        for (int i = 0; i < 2 * NT; ++i) mbar_init(&bars[i], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
#pragma unroll
        for (int i = 0; i < NT; ++i) {
            if (!valid[i]) continue;
            const bool have_parent = pslot[i] >= 0;
            const AT* conv_parent = static_cast<const AT*>(p.pool.conv) + (size_t)pslot[i] * p.pool.conv_slot_stride + d0;
            mbar_expect_tx(&bars[2 * i], row_bytes + (have_parent ? (kW - 1) * row_bytes : 0u));
            bulk_load(s_x + i * CB, static_cast<const AT*>(p.x) + (size_t)(node0 + i) * p.ldx + d0, row_bytes, &bars[2 * i]);
            if (have_parent)
                for (int j = 0; j < kW - 1; ++j) bulk_load(s_conv + (i * (kW - 1) + j) * CB, conv_parent + (size_t)j * D, row_bytes, &bars[2 * i]);
        }
#pragma unroll
        for (int i = 0; i < NT; ++i) {
            if (!valid[i]) continue;
            const bool have_parent = pslot[i] >= 0;
            mbar_expect_tx(&bars[2 * i + 1], row_bytes + (have_parent ? h_bytes : 0u));
            if (have_parent)
                bulk_load(s_h + i * CB * (kN / 4), p.pool.ssm + (size_t)pslot[i] * p.pool.ssm_slot_stride + (size_t)d0 * kN, h_bytes, &bars[2 * i + 1]);
            bulk_load(s_z + i * CB, static_cast<const AT*>(p.z) + (size_t)(node0 + i) * p.ldz + d0, row_bytes, &bars[2 * i + 1]);
        }
    }

    // Layer constants travel by ordinary loads while the copies are in flight.
    float a2[kPow ? 1 : kN];
    float4 wv = make_float4(0.f, 0.f, 0.f, 0.f);
    float cb = 0.f, dtb = 0.f, dsk = 0.f;
    if (live) {
        wv = __ldg(reinterpret_cast<const float4*>(p.L.conv_w + (size_t)d * kW));
        cb = p.L.conv_b ? __ldg(p.L.conv_b + d) : 0.f;
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
    // The weights depend on nothing that is still in flight: the first rows of this warp's share of W_x and the
    // head of this channel's row of W_dt are requested now, ahead of the waits they would otherwise queue behind.
    // (Giving the registers up for more resident blocks on wide levels was measured: it is slower at every width.)
    constexpr int kPreRows = NP == 4 ? (sizeof(AT) == 4 ? 3 : 5) : 10;  // rows of W_x held in registers per warp
    constexpr int kPreDt = sizeof(AT) == 4 ? 3 : 6;  // groups of eight weights of W_dt held in registers per thread
    const AT* wx = static_cast<const AT*>(p.W_x) + d0 + 4 * lane;
    bool in[NP];
#pragma unroll
    for (int q = 0; q < NP; ++q) in[q] = q * 128 + 4 * lane < cols;  // cols is a multiple of 8: a group of four is all in or all out
    Raw4<AT> wpre[kPreRows][NP];
#pragma unroll
    for (int j = 0; j < kPreRows; ++j) {
        const int r = warp + j * NW;
#pragma unroll
        for (int q = 0; q < NP; ++q) {
            wpre[j][q].load(wx);  // a valid address; replaced below when the row and the channels exist
            if (r < rows && in[q]) wpre[j][q].load(wx + (size_t)r * D + q * 128);
        }
    }
    const AT* wr = static_cast<const AT*>(p.W_dt) + (size_t)(live ? d : d0) * R;
    Raw8<AT> dpre[kPreDt];
#pragma unroll
    for (int j = 0; j < kPreDt; ++j)
        dpre[j].load(wr + (8 * j < R ? 8 * j : 0));

    __syncthreads();  // the mbarriers are initialised for everyone
    bool waited = true;
#pragma unroll
    for (int i = 0; i < NT; ++i)
        if (valid[i]) waited = mbar_wait_bounded(&bars[2 * i], 0u) && waited;
    bool bad = __syncthreads_or(!waited);

    // ---- conv window of every node: (w0, w1, w2, x) -> (w1, w2, x)
    float u[NT];
#pragma unroll
    for (int i = 0; i < NT; ++i) {
        u[i] = 0.f;
        if (live && !bad && valid[i]) {
            AT* cw = s_conv + i * (kW - 1) * CB + tid;
            const float xv = Act<AT>::to_f32(s_x[i * CB + tid]);
            float win[kW - 1] = {0.f, 0.f, 0.f};
            if (pslot[i] >= 0) {
#pragma unroll
                for (int j = 0; j < kW - 1; ++j) win[j] = Act<AT>::to_f32(cw[j * CB]);
            }
            float acc = fmaf(wv.x, win[0], cb);
            acc = fmaf(wv.y, win[1], acc);
            acc = fmaf(wv.z, win[2], acc);
            acc = fmaf(wv.w, xv, acc);
            u[i] = silu(acc);
            cw[0] = Act<AT>::from_f32(win[1]);
            cw[CB] = Act<AT>::from_f32(win[2]);
            cw[2 * CB] = Act<AT>::from_f32(xv);
        }
        s_u[i * CB + tid] = u[i];
    }
    __syncthreads();

    // ---- this block's share of s = W_x u per node: a warp takes every NW-th row, a lane 4 NP channels of it.
    {
        float4 uu[NT][NP];
#pragma unroll
        for (int i = 0; i < NT; ++i)
#pragma unroll
            for (int q = 0; q < NP; ++q) uu[i][q] = *reinterpret_cast<const float4*>(&s_u[i * CB + q * 128 + 4 * lane]);
        float acc[NT][kPreRows];
#pragma unroll
        for (int j = 0; j < kPreRows; ++j) {
            float4 wq[NP];
#pragma unroll
            for (int q = 0; q < NP; ++q) wq[q] = wpre[j][q].get();
#pragma unroll
            for (int i = 0; i < NT; ++i) {
                acc[i][j] = 0.f;
#pragma unroll
                for (int q = 0; q < NP; ++q)
                    if (in[q]) acc[i][j] = dot4(wq[q], uu[i][q], acc[i][j]);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
            for (int i = 0; i < NT; ++i)
#pragma unroll
                for (int j = 0; j < kPreRows; ++j) acc[i][j] += __shfl_xor_sync(0xffffffffu, acc[i][j], o);
        }
        if (lane == 0) {
#pragma unroll
            for (int i = 0; i < NT; ++i)
#pragma unroll
                for (int j = 0; j < kPreRows; ++j)
                    if (warp + j * NW < rows) s_part[i * kMaxRows + warp + j * NW] = acc[i][j];
        }
        // Rows beyond the prefetched ones (large dt_rank), four rows of W_x in flight per warp.
        constexpr int kBatch = 4;
        for (int r0 = warp + kPreRows * NW; r0 < rows; r0 += kBatch * NW) {
            float4 wq[kBatch][NP];
#pragma unroll
            for (int j = 0; j < kBatch; ++j)
#pragma unroll
                for (int q = 0; q < NP; ++q)
                    wq[j][q] = (r0 + j * NW < rows && in[q]) ? load_w4(wx + (size_t)(r0 + j * NW) * D + q * 128) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int i = 0; i < NT; ++i) {
                float a4[kBatch];
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    a4[j] = 0.f;
#pragma unroll
                    for (int q = 0; q < NP; ++q) a4[j] = dot4(wq[j][q], uu[i][q], a4[j]);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                    for (int j = 0; j < kBatch; ++j) a4[j] += __shfl_xor_sync(0xffffffffu, a4[j], o);
                }
                if (lane == 0) {
#pragma unroll
                    for (int j = 0; j < kBatch; ++j)
                        if (r0 + j * NW < rows) s_part[i * kMaxRows + r0 + j * NW] = a4[j];
                }
            }
        }
    }
    // Every block's share is complete and visible to the cluster after this barrier.
    cluster_arrive();
    cluster_wait();
    {
        const uint32_t nblk = cluster_size();
        if constexpr (NT == 1) {
            // Narrow level, latency counts: all remote reads of an entry are in flight together; the additions keep
            // the blocks' order.
            for (int r = tid; r < rows; r += CB) {
                float part[kProjMaxCluster];
#pragma unroll
                for (int c = 0; c < kProjMaxCluster; ++c) part[c] = (uint32_t)c < nblk ? peer_block_float(&s_part[r], c) : 0.f;
                float sum = 0.f;
#pragma unroll
                for (int c = 0; c < kProjMaxCluster; ++c)
                    if ((uint32_t)c < nblk) sum += part[c];
                s_s[r] = sum;
            }
        } else {
            // Wide level: the registers are better spent elsewhere (measured), other blocks cover the waits.
            for (int idx = tid; idx < NT * rows; idx += CB) {
                const int i = idx / rows, r = idx - i * rows;
                float sum = 0.f;
                for (uint32_t c = 0; c < nblk; ++c) sum += peer_block_float(&s_part[i * kMaxRows + r], c);
                s_s[i * kMaxRows + r] = sum;
            }
        }
    }
    cluster_arrive();  // this block no longer reads its neighbours; the matching wait is the last thing it does
    __syncthreads();

    // ---- step size of this thread's channel in every node: dt = W_dt[d][:] . s[0:R]  (R is a multiple of 8)
    float dtv[NT];
#pragma unroll
    for (int i = 0; i < NT; ++i) dtv[i] = 0.f;
    if (live) {
        float acc0[NT], acc1[NT];
#pragma unroll
        for (int i = 0; i < NT; ++i) { acc0[i] = 0.f; acc1[i] = 0.f; }
#pragma unroll
        for (int j = 0; j < kPreDt; ++j) {
            if (8 * j < R) {
                const float4 w0 = dpre[j].lo(), w1 = dpre[j].hi();
#pragma unroll
                for (int i = 0; i < NT; ++i) {
                    acc0[i] = dot4(w0, *reinterpret_cast<const float4*>(&s_s[i * kMaxRows + 8 * j]), acc0[i]);
                    acc1[i] = dot4(w1, *reinterpret_cast<const float4*>(&s_s[i * kMaxRows + 8 * j + 4]), acc1[i]);
                }
            }
        }
#pragma unroll 2
        for (int r = 8 * kPreDt; r < R; r += 8) {
            const float4 w0 = load_w4(wr + r), w1 = load_w4(wr + r + 4);
#pragma unroll
            for (int i = 0; i < NT; ++i) {
                acc0[i] = dot4(w0, *reinterpret_cast<const float4*>(&s_s[i * kMaxRows + r]), acc0[i]);
                acc1[i] = dot4(w1, *reinterpret_cast<const float4*>(&s_s[i * kMaxRows + r + 4]), acc1[i]);
            }
        }
#pragma unroll
        for (int i = 0; i < NT; ++i) dtv[i] = acc0[i] + acc1[i];
    }

    waited = true;
#pragma unroll
    for (int i = 0; i < NT; ++i)
        if (valid[i]) waited = mbar_wait_bounded(&bars[2 * i + 1], 0u) && waited;
    bad = __syncthreads_or(bad || !waited);

#pragma unroll
    for (int i = 0; i < NT; ++i) {
        if (!(live && !bad && valid[i])) continue;
        // ---- one step of the recurrence.  The quads of a channel are visited in an order that differs between
        // neighbouring threads, which keeps the 128-bit shared-memory accesses free of bank conflicts.
        float4* hs = s_h + (i * CB + tid) * (kN / 4);
        const float* ss = s_s + i * kMaxRows;
        const int sw = (tid >> 1) & 3;
        float4 hq[kN / 4];
#pragma unroll
        for (int k = 0; k < kN / 4; ++k) hq[k] = pslot[i] >= 0 ? hs[k ^ sw] : make_float4(0.f, 0.f, 0.f, 0.f);
        xor_permute(hq, sw);
        const float zv = Act<AT>::to_f32(s_z[i * CB + tid]);
        const float v = dtv[i] + dtb;
        const float delta = (flags & MDRAFT_DT_SOFTPLUS) ? softplus(v) : v;
        const float du = delta * u[i];
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
        float h[kN], Bv[kN], Cv[kN];
#pragma unroll
        for (int q = 0; q < kN / 4; ++q) {
            h[4 * q] = hq[q].x; h[4 * q + 1] = hq[q].y; h[4 * q + 2] = hq[q].z; h[4 * q + 3] = hq[q].w;
            const float4 b = *reinterpret_cast<const float4*>(&ss[R + 4 * q]);
            const float4 c = *reinterpret_cast<const float4*>(&ss[R + kN + 4 * q]);
            Bv[4 * q] = b.x; Bv[4 * q + 1] = b.y; Bv[4 * q + 2] = b.z; Bv[4 * q + 3] = b.w;
            Cv[4 * q] = c.x; Cv[4 * q + 1] = c.y; Cv[4 * q + 2] = c.z; Cv[4 * q + 3] = c.w;
        }
        float y0 = 0.f, y1 = 0.f;
#pragma unroll
        for (int n = 0; n < kN; ++n) {
            h[n] = fmaf(P[n], h[n], du * Bv[n]);
            if (n & 1) y1 = fmaf(Cv[n], h[n], y1); else y0 = fmaf(Cv[n], h[n], y0);
        }
#pragma unroll
        for (int q = 0; q < kN / 4; ++q) hq[q] = make_float4(h[4 * q], h[4 * q + 1], h[4 * q + 2], h[4 * q + 3]);
        xor_permute(hq, sw);
#pragma unroll
        for (int k = 0; k < kN / 4; ++k) hs[k ^ sw] = hq[k];
        s_x[i * CB + tid] = Act<AT>::from_f32(fmaf(dsk, u[i], y0 + y1) * silu(zv));
    }
    // Shared-memory writes above must be visible to the copy engine before it reads them.
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (tid == 0) {
        if (bad) {
            // Nothing of these nodes is stored.  The copies target this block's shared memory: give them one more
            // bounded chance to land before the block ends.
            flag(p.dev_status, MDRAFT_DEV_WAIT_EXPIRED);
#pragma unroll
            for (int i = 0; i < NT; ++i)
                if (valid[i]) { mbar_wait_bounded(&bars[2 * i], 0u); mbar_wait_bounded(&bars[2 * i + 1], 0u); }
        } else {
#pragma unroll
            for (int i = 0; i < NT; ++i) {
                if (!valid[i]) continue;
                bulk_store(p.pool.ssm + (size_t)nslot[i] * p.pool.ssm_slot_stride + (size_t)d0 * kN, s_h + i * CB * (kN / 4), h_bytes);
                AT* conv_child = static_cast<AT*>(p.pool.conv) + (size_t)nslot[i] * p.pool.conv_slot_stride + d0;
                for (int j = 0; j < kW - 1; ++j) bulk_store(conv_child + (size_t)j * D, s_conv + (i * (kW - 1) + j) * CB, row_bytes);
                bulk_store(static_cast<AT*>(p.out) + (size_t)(node0 + i) * p.ldo + d0, s_x + i * CB, row_bytes);
            }
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // shared memory stays valid until it has been read
        }
    }
    __syncwarp();
    cluster_wait();  // no block of the cluster leaves while a neighbour may still read its share of s
}

template <typename AT, int CB, int NT>
cudaError_t launch_nt(const TreeProjArgs& p, int n_blocks, cudaStream_t st) {
    constexpr int kSmem = ProjSmem<AT, CB, NT>::kTotal;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((p.n_nodes + NT - 1) / NT), (unsigned)n_blocks, 1);
    cfg.blockDim = dim3(CB, 1, 1);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 1;
    at[0].val.clusterDim.y = (unsigned)n_blocks;  // the blocks of one group of nodes
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    const bool pow = p.L.flags & MDRAFT_A_POWERS;
    auto kernel = pow ? tree_proj_kernel<AT, CB, NT, true> : tree_proj_kernel<AT, CB, NT, false>;
    if (kSmem > 48 * 1024) {  // a property of the loaded function, not an allocation
        const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
        if (e != cudaSuccess) return e;
    }
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

template <typename AT>
cudaError_t launch_act(const TreeProjArgs& p, cudaStream_t st) {
    const int cb = tree_proj_block_channels(p.L.d_inner);
    const int n_blocks = (p.L.d_inner + cb - 1) / cb;
    // Nodes per cluster: one while the level is narrow (latency is what counts and every node gets its own SMs);
    // two or four once the level is wide enough that re-reading the two matrices per node is what costs.
    int nt = p.nodes_per_cluster;
    if (nt <= 0) nt = p.n_nodes * n_blocks <= 2 * 148 ? 1 : (p.n_nodes * n_blocks <= 4 * 148 ? 2 : 4);
    if (cb == 512) nt = 1;  // the widest block has no registers to spare for a second node
    switch (cb) {
        case 128: return nt == 1 ? launch_nt<AT, 128, 1>(p, n_blocks, st) : nt == 2 ? launch_nt<AT, 128, 2>(p, n_blocks, st) : launch_nt<AT, 128, 4>(p, n_blocks, st);
        case 256: return nt == 1 ? launch_nt<AT, 256, 1>(p, n_blocks, st) : nt == 2 ? launch_nt<AT, 256, 2>(p, n_blocks, st) : launch_nt<AT, 256, 4>(p, n_blocks, st);
        case 512: return launch_nt<AT, 512, 1>(p, n_blocks, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

int tree_proj_block_channels(int d_inner) {
    for (int cb = 128; cb <= 512; cb *= 2)
        if ((d_inner + cb - 1) / cb <= kProjMaxCluster) return cb;
    return 0;
}

cudaError_t launch_tree_proj(const TreeProjArgs& p, int act, cudaStream_t st) {
    if (p.n_nodes <= 0) return cudaSuccess;
    return act == MDRAFT_F32 ? launch_act<float>(p, st) : launch_act<__nv_bfloat16>(p, st);
}

}  // namespace mdraft
