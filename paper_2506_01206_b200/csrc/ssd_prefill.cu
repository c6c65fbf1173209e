// Context encode of a Mamba-2 (SSD) layer: conv1d+SiLU -> Delta -> recurrence with one scalar A per head -> gate.
//
// With a scalar decay per head the recurrence of a chunk of Q tokens turns into matrix products (the "state-space
// duality" form).  With cs_t = sum_{r <= t} Delta_r A (the running log-decay inside the chunk), for a head of P channels:
//
//     y_t = sum_{s <= t} (C_t . B_s) exp(cs_t - cs_s) Delta_s u_s      (inside the chunk:  (G o L) Xd,  G = C B^T)
//           + exp(cs_t) C_t . h_in                                      (from the incoming state:  C H_in^T, row-scaled)
//     S   = sum_s exp(cs_end - cs_s) Delta_s u_s (x) B_s                (what the chunk adds to a zero state)
//     h_out = exp(cs_end) h_in + S
//
// Three kernels, none waiting on another block, chained by programmatic dependent launch: the first waits for everything
// ahead of the call and then lets the others start, so that they may read the call's inputs before their own wait.
//   1. ssd_chunk_state: per (head, chunk) conv + SiLU, step sizes and running decays, then S^T = B^T Xw on the tensor
//      cores (tcgen05.mma, bf16 operands, fp32 accumulator in tensor memory); Xw is split into a bf16 value and a bf16
//      remainder (two products into one accumulator) so that the state keeps fp32-level accuracy.  What kernel 3 needs
//      of this work is handed over through the workspace: Xd = Delta u already in operand layout, u, and the running
//      log-decays of the chunk's rows; the sequence's last chunk also leaves the conv window.
//   2. ssd_state_passing: per (channel, 4 states) the chunk states of a sequence are chained in token order; every
//      chunk's incoming state is left in the operand layout the next kernel wants, the final state goes to its slot.
//   3. ssd_chunk_scan: per (head, chunk) G = C B^T (issued before the kernel's wait: inputs only), the causal decay mask applied to G on its way from tensor memory to
//      shared memory, Y = (G o L) Xd and C H_in^T on the tensor cores, then skip term, gate and store.  It touches no
//      x, dt or conv weight: its shared memory is three operand tiles, so that two blocks share an SM.
//
// Operands live in shared memory in the tensor core's canonical un-swizzled layout: 16-byte units of 8 bf16 values,
// 8 units = one 8 x 8 "core matrix" of 128 contiguous bytes; one descriptor field gives the byte step between core
// matrices along the contraction index, the other along the row index.  That is the layout of the operands that threads
// write (Xw, Xd, the masked G) and of the incoming state.  The B and C rows come by TMA in boxes of 64 states x 128 tokens
// with the 128-byte swizzle (rows of 128 bytes, 16-byte units XOR-ed with the row index: full sectors on the way in and the
// tensor core's swizzled operand layout in shared memory), so they arrive in operand form without a pass over them, both as
// "K-major" (G: contraction over the state index) and as "MN-major" (S: contraction over tokens) - same bytes, two descriptors.
// All waits on mbarriers are bounded (MDRAFT_DEV_WAIT_EXPIRED); tensor memory is freed on every path.
#include "chunk_map.cuh"
#include "common.cuh"
#include "ssd.cuh"

namespace mdraft {

namespace {

constexpr int P = kSsdP, N = kSsdN, Q = kSsdQ;
constexpr int kThreads = 256;                 // two warps per 32 accumulator lanes: warps w and w + 4 share rows 32 (w % 4) .. and split the columns
constexpr int kRowsPerWarp = Q / (kThreads / 32);   // rows of the chunk a warp convolves and stores
constexpr uint32_t kColBytes = Q * 16;        // one 8-wide column of core matrices over 128 rows: 2048 bytes
constexpr uint32_t kXdColBytes = Q * 16 + 16; // the same for the thread-written Xd / Xw operand, padded against bank conflicts
constexpr uint32_t kHinColBytes = P * 16;     // H_in: 64 rows

// ---------------------------------------------------------------- PTX helpers
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
__device__ __forceinline__ void tma_box(void* dst, const CUtensorMap* map, int col, int row, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(smem_u32(dst)),
                 "l"(reinterpret_cast<uint64_t>(map)), "r"(col), "r"(row), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst)),
                 "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// Tensor memory: allocation (one warp), release, and the accumulator loads (a warp reads the 32 lanes it owns).
__device__ __forceinline__ void tmem_alloc(uint32_t* slot_in_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot_in_smem)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free(uint32_t base, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory operand descriptor, un-swizzled canonical layout.  `lead` / `stride` are the two byte steps between core
// matrices: for a K-major operand lead = along the contraction index, stride = along rows; for an MN-major operand
// lead = along the contraction index (groups of 8), stride = along the row index (groups of 8).
__device__ __forceinline__ uint64_t operand_desc(uint32_t saddr, uint32_t lead, uint32_t stride) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lead >> 4) & 0x3FFFu) << 16) | ((uint64_t)((stride >> 4) & 0x3FFFu) << 32) |
           (1ull << 46);
}
// The same for a K-major operand in the 128-byte-swizzled layout (rows of 64 values = 128 bytes, 8 rows = one 1024-byte
// group, 16-byte units XOR-ed with the row index; the tile starts on a 1024-byte boundary): the stride field is the step
// between groups of 8 rows, the leading field is not used, and a step of 16 values along the contraction index is 32 bytes
// added to the start address.
__device__ __forceinline__ uint64_t operand_desc_sw128(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// The same layout read as an MN-major operand (rows of 64 MN-values, one row per contraction index): `lead` is the step
// between blocks of 64 MN-values, `stride` the step between groups of 8 contraction indices.
__device__ __forceinline__ uint64_t operand_desc_sw128_mn(uint32_t saddr, uint32_t lead, uint32_t stride) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lead >> 4) & 0x3FFFu) << 16) | ((uint64_t)((stride >> 4) & 0x3FFFu) << 32) | (1ull << 46) |
           (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = n; bit 15 / 16 = A / B operand is MN-major.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool a_mn, bool b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}
// D (tensor memory) (+)= A (smem) * B (smem), one instruction of contraction length 16; issued by ONE thread.
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate ? 1u : 0u), "r"(0u)
        : "memory");
}
// All tensor-core work issued so far by this thread arrives on the mbarrier when it has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Programmatic dependent launch: the kernels of a call (and the first kernel of the next call on the stream) may start
// before the kernel ahead of them has finished.  A kernel passes grid_wait() before it touches anything a kernel ahead
// of it writes, or overwrites anything one reads; every block passes it on every path, so that a kernel's completion
// implies the completion of everything before it.
__device__ __forceinline__ void grid_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// SiLU of the gate input with one special-function instruction instead of two: z sigmoid(z) = 0.5 z (1 + tanh(z / 2)); the
// approximate tanh is good to about 2^-11, an order below the bf16 rounding of `out`.
__device__ __forceinline__ float silu_gate(float v) {
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * v));
    const float h = 0.5f * v;
    return fmaf(h, t, h);
}
__device__ __forceinline__ float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// ---------------------------------------------------------------- what both tensor-core kernels share
// Per-row scalars of a chunk: step size and running log-decay.  Thread t = row t; rows past the chunk's end get a
// step size of 0 (no decay, no input).  Leaves delta[t], cs[t] (natural log) and csl[t] = cs[t] * log2(e) in shared memory.
struct RowScalars {
    float delta[Q];
    float cs[Q];
    float csl[Q];
    float warp_sum[4];
};

__device__ __forceinline__ void row_scalars(RowScalars& rs, const SsdPrefillArgs& p, int head, int t0, int rows) {
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const bool owner = t < Q;   // threads Q.. only take part in the barriers
    float delta = 0.0f;
    if (owner && t < rows) {
        const float v = __bfloat162float(p.dt[(size_t)(t0 + t) * p.lddt + head]) + (p.L.dt_bias ? __ldg(p.L.dt_bias + head) : 0.0f);
        delta = (p.L.flags & MDRAFT_DT_SOFTPLUS) ? softplus(v) : v;
    }
    float la = delta * __ldg(p.L.A + head);
    // inclusive scan over the 128 rows: inside the warp by shuffles, across the four warps through shared memory
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float up = __shfl_up_sync(0xffffffffu, la, o);
        if (lane >= o) la += up;
    }
    if (owner && lane == 31) rs.warp_sum[warp] = la;
    __syncthreads();
    if (owner) {
        float before = 0.0f;
        for (int w = 0; w < warp; ++w) before += rs.warp_sum[w];
        la += before;
        rs.delta[t] = delta;
        rs.cs[t] = la;
        rs.csl[t] = la * kLog2e;
    }
    __syncthreads();
}

// The three rows before the chunk, as rows 0..2 of the extended x tile (rows 3.. are the TMA box): the sequence's own
// tokens, or the window of its starting slot, or zeros.  Threads 0..95, one bf16 pair each.
__device__ __forceinline__ void load_halo(__nv_bfloat16* xs_ext, const SsdPrefillArgs& p, const ChunkInfo& ci, int head, int islot) {
    const int t = threadIdx.x;
    if (t >= 3 * 32) return;
    const int j = t >> 5, lane = t & 31;
    const int d = head * P + 2 * lane;
    uint32_t v = 0u;
    if (ci.k > 0) v = *reinterpret_cast<const uint32_t*>(p.x + (size_t)(ci.t0 - 3 + j) * p.ldx + d);
    else if (islot >= 0) v = *reinterpret_cast<const uint32_t*>(static_cast<const __nv_bfloat16*>(p.pool.conv) + (size_t)islot * p.pool.conv_slot_stride + (size_t)j * p.L.d_inner + d);
    *reinterpret_cast<uint32_t*>(xs_ext + j * P + 2 * lane) = v;
}

// The warp's rows of the extended x tile (its kRowsPerWarp rows and the three before them) for this lane's channel pair.
__device__ __forceinline__ void load_rows(const __nv_bfloat16* xs_ext, uint32_t (&xr)[kRowsPerWarp + 3]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t* col = reinterpret_cast<const uint32_t*>(xs_ext) + lane;   // row r of the chunk is extended row r + 3
    const int r0 = warp * kRowsPerWarp;
#pragma unroll
    for (int i = 0; i < kRowsPerWarp + 3; ++i) xr[i] = col[(r0 + i) * (P / 2)];
}

// conv + SiLU of those rows; calls f(row, index in the warp, u_lo, u_hi).
template <typename F>
__device__ __forceinline__ void conv_rows(const uint32_t (&xr)[kRowsPerWarp + 3], const SsdLayerDev& L, int head, F&& f) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d = head * P + 2 * lane;
    const float4 wa = __ldg(reinterpret_cast<const float4*>(L.conv_w + (size_t)d * kW));
    const float4 wb = __ldg(reinterpret_cast<const float4*>(L.conv_w + (size_t)(d + 1) * kW));
    const float ba = L.conv_b ? __ldg(L.conv_b + d) : 0.0f, bb = L.conv_b ? __ldg(L.conv_b + d + 1) : 0.0f;
    const int r0 = warp * kRowsPerWarp;
#pragma unroll
    for (int i = 0; i < kRowsPerWarp; ++i) {
        const uint32_t w0 = xr[i], w1 = xr[i + 1], w2 = xr[i + 2], xv = xr[i + 3];
        float a = fmaf(wa.x, bf_lo(w0), ba), b = fmaf(wb.x, bf_hi(w0), bb);
        a = fmaf(wa.y, bf_lo(w1), a); b = fmaf(wb.y, bf_hi(w1), b);
        a = fmaf(wa.z, bf_lo(w2), a); b = fmaf(wb.z, bf_hi(w2), b);
        a = fmaf(wa.w, bf_lo(xv), a); b = fmaf(wb.w, bf_hi(xv), b);
        f(r0 + i, i, silu(a), silu(b));
    }
}

// ---------------------------------------------------------------- kernel 1: what a chunk adds to a zero state
struct StateSmem {
    unsigned char Bt[Q * N * 2];                          // B rows of the chunk [2][Q][64] bf16, 128-byte swizzle (MN-major operand)
    unsigned char xw_hi[(P / 8) * kXdColBytes];           // Xw = Delta exp(cs_end - cs) u, bf16 value ...
    // ... and bf16 remainder, which takes the place of the x tile (3 rows before the chunk + the x box) once every thread
    // holds its rows of x in registers
    unsigned char xs_or_lo[(Q + 3) * P * 2];
    RowScalars rs;
    uint64_t bar_tma, bar_mma;
    uint32_t tmem_base;
};
static_assert((Q + 3) * P * 2 >= (P / 8) * kXdColBytes, "the remainder operand must fit the x tile it replaces");
static_assert(3 * (sizeof(StateSmem) + 1024 + 1024) <= 227 * 1024, "three blocks per SM");

__global__ void __launch_bounds__(kThreads, 3) ssd_chunk_state_kernel(const SsdPrefillArgs p, const __grid_constant__ SsdMaps maps) {
    extern __shared__ __align__(1024) unsigned char s_raw[];
    StateSmem& sm = *reinterpret_cast<StateSmem*>(s_raw + ((1024u - (smem_u32(s_raw) & 1023u)) & 1023u));   // the swizzled tile starts on a 1024-byte boundary
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int head = blockIdx.x, cidx = blockIdx.y, H = p.L.n_heads;
    // The inputs may be the work of the kernel ahead of this call, and the workspace is still being read by the call
    // before this one: nothing is touched before that kernel is complete.  Only then may the next kernels start, which
    // lets them read the call's inputs without a wait of their own.
    grid_wait();
    grid_release_dependents();
    const ChunkInfo ci = find_chunk(p.cu, p.n_seq, p.T, Q, cidx);
    if (ci.seq < 0) return;
    const int islot = load_slot(p.init_slot, ci.seq), fslot = load_slot(p.final_slot, ci.seq);
    if (islot >= p.pool.n_slots || fslot >= p.pool.n_slots) return;   // reported by the state-passing kernel
    const int rows = ci.t1 - ci.t0;
    __nv_bfloat16* xs_ext = reinterpret_cast<__nv_bfloat16*>(sm.xs_or_lo);
    unsigned char* xw_lo = sm.xs_or_lo;

    if (tid == 0) {
        mbar_init(&sm.bar_tma, 1);
        mbar_init(&sm.bar_mma, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(&sm.bar_tma, Q * P * 2 + Q * N * 2);
        tma_box(xs_ext + 3 * P, &maps.x, head * P, ci.t0, &sm.bar_tma);
        tma_box(sm.Bt, &maps.Bs, 0, ci.t0, &sm.bar_tma);
        tma_box(sm.Bt + Q * 128, &maps.Bs, 64, ci.t0, &sm.bar_tma);
    }
    if (warp == 0) { tmem_alloc(&sm.tmem_base, 64); tc_fence_before(); }
    load_halo(xs_ext, p, ci, head, islot);
    row_scalars(sm.rs, p, head, ci.t0, rows);   // two block-wide barriers inside: barrier init and tmem_base are visible after it
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    bool ok = mbar_wait_bounded(&sm.bar_tma, 0u);
    uint32_t xr[kRowsPerWarp + 3];
    if (ok) {
        load_rows(xs_ext, xr);
        // the sequence's last chunk leaves the window: the last three raw inputs (extended rows rows .. rows + 2)
        if (ci.k == ci.nck - 1 && fslot >= 0 && warp < 3) {
            __nv_bfloat16* dc = static_cast<__nv_bfloat16*>(p.pool.conv) + (size_t)fslot * p.pool.conv_slot_stride + (size_t)warp * p.L.d_inner + head * P + 2 * lane;
            *reinterpret_cast<uint32_t*>(dc) = reinterpret_cast<const uint32_t*>(xs_ext)[(rows + warp) * (P / 2) + lane];
        }
    }
    __syncthreads();   // every thread holds its rows: the x tile may be overwritten
    if (ok) {
        const float cs_end_l = sm.rs.csl[Q - 1];
        unsigned char* xd_g = reinterpret_cast<unsigned char*>(p.ws_xd) + ((size_t)cidx * H + head) * ((P / 8) * kXdColBytes);
        conv_rows(xr, p.L, head, [&](int r, int, float ua, float ub) {
            const float wgt = r < rows ? sm.rs.delta[r] * ex2(cs_end_l - sm.rs.csl[r]) : 0.0f;
            const float va = r < rows ? wgt * ua : 0.0f, vb = r < rows ? wgt * ub : 0.0f;
            const uint32_t hi = pack_bf(va, vb);
            const uint32_t lo = pack_bf(va - bf_lo(hi), vb - bf_hi(hi));
            const uint32_t off = (uint32_t)(lane >> 2) * kXdColBytes + (uint32_t)r * 16u + (uint32_t)(lane & 3) * 4u;
            *reinterpret_cast<uint32_t*>(sm.xw_hi + off) = hi;
            *reinterpret_cast<uint32_t*>(xw_lo + off) = lo;
            // Xd = Delta u goes straight to the workspace, in the layout of the chunk-scan kernel's operand
            const float dl = r < rows ? sm.rs.delta[r] : 0.0f;
            *reinterpret_cast<uint32_t*>(xd_g + off) = r < rows ? pack_bf(dl * ua, dl * ub) : 0u;
            if (r < rows) *reinterpret_cast<uint32_t*>(p.ws_u + (size_t)(ci.t0 + r) * p.L.d_inner + head * P + 2 * lane) = pack_bf(ua, ub);
        });
        if (tid < Q) p.ws_csl[((size_t)cidx * H + head) * Q + tid] = sm.rs.csl[tid];
    }
    fence_async_smem();   // the operands written by threads must be visible to the tensor core's reads
    const bool all_ok = !__syncthreads_or(!ok);
    if (all_ok && tid == 0) {
        tc_fence_after();
        // S^T (n x p) = sum over tokens: A operand = B^T read MN-major out of the TMA boxes, B operand = Xw MN-major.
        constexpr uint32_t idesc = instr_desc(P, true, true);
        const uint32_t bh = smem_u32(sm.xw_hi), bl = smem_u32(xw_lo);
        // B^T: two blocks of 64 states (16 KB apart), 16 tokens per instruction = two groups of 8 rows of 128 bytes
        const uint64_t dA = operand_desc_sw128_mn(smem_u32(sm.Bt), Q * 128, 1024);
#pragma unroll
        for (int k = 0; k < Q / 16; ++k)
            mma_bf16(tmem, dA + (uint64_t)(k * 2048 >> 4), operand_desc(bh + k * 256, 128, kXdColBytes), idesc, k > 0);
#pragma unroll
        for (int k = 0; k < Q / 16; ++k)
            mma_bf16(tmem, dA + (uint64_t)(k * 2048 >> 4), operand_desc(bl + k * 256, 128, kXdColBytes), idesc, true);
        mma_commit(&sm.bar_mma);
    }
    bool done = all_ok && mbar_wait_bounded(&sm.bar_mma, 0u);
    if (done) {
        tc_fence_after();
        // a thread holds half a row of S^T (state n = its accumulator lane): 32 of the head's channels; stores are
        // contiguous across the threads of a warp
        const int n = (warp & 3) * 32 + lane, half = warp >> 2;
        float* dst = p.ws_S + ((size_t)cidx * H + head) * P * N + n;
        {
            float v[32];
            tmem_ld32(tmem + ((uint32_t)((warp & 3) * 32) << 16) + half * 32, v);
#pragma unroll
            for (int j = 0; j < 32; ++j) dst[(size_t)(half * 32 + j) * N] = v[j];
        }
        if (tid == 0) p.ws_decay[(size_t)cidx * H + head] = sm.rs.cs[Q - 1];
    } else if (tid == 0) {
        flag(p.dev_status, MDRAFT_DEV_WAIT_EXPIRED);
        if (!ok) mbar_wait_bounded(&sm.bar_tma, 0u);   // the copies target this block's shared memory: one more bounded chance
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_free(tmem, 64);
}

// ---------------------------------------------------------------- kernel 2: chain the chunk states of a sequence
// Thread = (channel d, 4 states); a lane pair covers one 16-byte unit of the operand.  Walks the sequence's chunks in order:
// writes the chunk's incoming state as bf16 (a value and a remainder) in the operand layout [state group][channel of the
// head][8], then h <- exp(chunk decay) h + S.
constexpr int kPassThreads = 256;
constexpr int kPassBatch = 16;   // chunks whose summaries are in flight together

__global__ void __launch_bounds__(kPassThreads) ssd_state_passing_kernel(const SsdPrefillArgs p) {
    const int D = p.L.d_inner, H = p.L.n_heads;
    const int s = blockIdx.y;
    const int idx = blockIdx.x * kPassThreads + threadIdx.x;
    grid_release_dependents();
    // Sequence offsets, slots and the starting state are inputs of the call: the kernel ahead let this one start only
    // after everything before the call had finished, so they are read before the wait below.
    int first, nck;
    seq_chunks(p.cu, p.n_seq, p.T, Q, s, first, nck);   // whole warps call this
    // malformed offsets: the sequence has no chunk and is skipped
    if (p.cu && blockIdx.x == 0 && threadIdx.x == 0) {
        const int lo = __ldg(p.cu + s), hi = __ldg(p.cu + s + 1);
        if (lo < 0 || hi < lo || hi > p.T) flag(p.dev_status, MDRAFT_DEV_BAD_SEQLENS);
    }
    const int islot = load_slot(p.init_slot, s), fslot = load_slot(p.final_slot, s);
    const bool slots_ok = islot < p.pool.n_slots && fslot < p.pool.n_slots;
    if (!slots_ok && blockIdx.x == 0 && threadIdx.x == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
    const bool mine = slots_ok && idx < D * (N / 4);
    // consecutive lanes: the two halves of a unit, then consecutive channels of one head and one state group, so that the
    // 16-byte operand units a warp writes are contiguous (its 32-byte reads of the chunk states each fill a sector)
    const int sub = idx & 1, ch = (idx >> 1) % P, g = (idx / (2 * P)) % (N / 8), head = mine ? idx / (2 * P * (N / 8)) : 0, d = head * P + ch;
    const int n0 = g * 8 + sub * 4;
    float4 h = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    if (mine && islot >= 0) h = *reinterpret_cast<const float4*>(p.pool.ssm + (size_t)islot * p.pool.ssm_slot_stride + (size_t)d * N + n0);
    grid_wait();   // the chunk states are the work of the kernel just before
    if (!mine) return;
    const int end = first + nck;
    for (int c0 = first; c0 < end; c0 += kPassBatch) {
        float4 sv[kPassBatch];
        float decay[kPassBatch];
#pragma unroll
        for (int i = 0; i < kPassBatch; ++i) {
            if (c0 + i < end) {
                const size_t ch_head = (size_t)(c0 + i) * H + head;
                sv[i] = *reinterpret_cast<const float4*>(p.ws_S + (ch_head * P + ch) * N + n0);
                decay[i] = __ldg(p.ws_decay + ch_head);
            }
        }
#pragma unroll
        for (int i = 0; i < kPassBatch; ++i) {
            if (c0 + i < end) {
                const size_t ch_head = (size_t)(c0 + i) * H + head;
                // bf16 value and bf16 remainder of the incoming state: two operands, so that the product with C sees ~16 mantissa bits
                uint2 hi2, lo2;
                hi2.x = pack_bf(h.x, h.y); hi2.y = pack_bf(h.z, h.w);
                lo2.x = pack_bf(h.x - bf_lo(hi2.x), h.y - bf_hi(hi2.x)); lo2.y = pack_bf(h.z - bf_lo(hi2.y), h.w - bf_hi(hi2.y));
                __nv_bfloat16* blob = p.ws_hin + ch_head * 2 * N * P + ((size_t)g * P + ch) * 8 + sub * 4;
                *reinterpret_cast<uint2*>(blob) = hi2;
                *reinterpret_cast<uint2*>(blob + (size_t)N * P) = lo2;
                const float dk = ex2(decay[i] * kLog2e);
                h = make_float4(fmaf(dk, h.x, sv[i].x), fmaf(dk, h.y, sv[i].y), fmaf(dk, h.z, sv[i].z), fmaf(dk, h.w, sv[i].w));
            }
        }
    }
    if (fslot < 0) return;
    if (nck > 0 || fslot != islot) *reinterpret_cast<float4*>(p.pool.ssm + (size_t)fslot * p.pool.ssm_slot_stride + (size_t)d * N + n0) = h;
    if (nck == 0 && fslot != islot && g == 0 && sub == 0) {   // a sequence without tokens: its window moves with its state
        __nv_bfloat16* dc = static_cast<__nv_bfloat16*>(p.pool.conv) + (size_t)fslot * p.pool.conv_slot_stride;
        const __nv_bfloat16* sc = islot >= 0 ? static_cast<const __nv_bfloat16*>(p.pool.conv) + (size_t)islot * p.pool.conv_slot_stride : nullptr;
        for (int j = 0; j < kW - 1; ++j) dc[(size_t)j * D + d] = sc ? sc[(size_t)j * D + d] : __float2bfloat16_rn(0.0f);
    }
}

// ---------------------------------------------------------------- kernel 3: outputs of a chunk
// Shared memory is three operand tiles that are re-used as the phases go by:
//   region A: C rows (operand of G and of C H_in^T)  ->  Xd (fetched from the workspace once those products are done)
//   region B: B rows (operand of G)                   ->  masked G (operand of Y)
//   region H: incoming state, value + remainder        ->  the z box (fetched once C H_in^T is done)
//   regions A + B                                       ->  y rows on their way from accumulator lanes to channel-contiguous stores
struct ScanSmem {
    unsigned char regA[N / 8 * Q * 16];   // C rows [2][Q][64] bf16, 128-byte swizzle (K-major operand)  ->  Xd [(P/8)][Q + 1 unit][8] (MN-major operand, from kernel 1)
    unsigned char regB[N / 8 * Q * 16];   // B rows [2][Q][64] bf16, 128-byte swizzle (K-major operand)  ->  masked G [Q/8][Q][8] (K-major over the source token)
    unsigned char regH[2 * N * P * 2];    // incoming state [2][N/8][P][8] bf16 (value, remainder; K-major operands)  ->  z box [Q][P] bf16
    float csl[Q];                         // running log2-decay of the chunk's rows (from kernel 1)
    uint64_t bar_cb, bar_in, bar_late, bar_g, bar_x, bar_y;
    uint32_t tmem_base;
};
static_assert(sizeof(float) * Q * (P + 1) <= 2 * (N / 8 * Q * 16), "the y staging rows must fit the two operand tiles they lie over");
static_assert((P / 8) * kXdColBytes <= N / 8 * Q * 16 && Q * P * 2 <= 2 * N * P * 2, "re-used regions too small");

__global__ void __launch_bounds__(kThreads, 2) ssd_chunk_scan_kernel(const SsdPrefillArgs p, const __grid_constant__ SsdMaps maps) {
    extern __shared__ __align__(1024) unsigned char s_raw[];
    ScanSmem& sm = *reinterpret_cast<ScanSmem*>(s_raw + ((1024u - (smem_u32(s_raw) & 1023u)) & 1023u));   // swizzled tiles start on 1024-byte boundaries
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int head = blockIdx.x, cidx = blockIdx.y, H = p.L.n_heads;
    grid_release_dependents();
    // Offsets, slots and the C / B rows are inputs of the call (complete before its first kernel let the others start): the
    // look-ups and the copies of C and B run while the kernels ahead are still at work.
    const ChunkInfo ci = find_chunk(p.cu, p.n_seq, p.T, Q, cidx);
    if (ci.seq < 0) { grid_wait(); return; }
    const int islot = load_slot(p.init_slot, ci.seq), fslot = load_slot(p.final_slot, ci.seq);
    if (islot >= p.pool.n_slots || fslot >= p.pool.n_slots) { grid_wait(); return; }
    const int rows = ci.t1 - ci.t0;
    const size_t ch_head = (size_t)cidx * H + head;
    __nv_bfloat16 (*Mt)[Q][8] = reinterpret_cast<__nv_bfloat16 (*)[Q][8]>(sm.regB);
    unsigned char* xd = sm.regA;
    constexpr uint32_t kXdBytes = (P / 8) * kXdColBytes;
    __nv_bfloat16* hin = reinterpret_cast<__nv_bfloat16*>(sm.regH);
    __nv_bfloat16* zs = reinterpret_cast<__nv_bfloat16*>(sm.regH);
    float (*ystage)[P + 1] = reinterpret_cast<float (*)[P + 1]>(sm.regA);   // runs on into regB

    if (tid == 0) {
        mbar_init(&sm.bar_cb, 1); mbar_init(&sm.bar_in, 1); mbar_init(&sm.bar_late, 1); mbar_init(&sm.bar_g, 1); mbar_init(&sm.bar_x, 1); mbar_init(&sm.bar_y, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(&sm.bar_cb, 2 * Q * N * 2);
        // two boxes of 64 states x 128 tokens per matrix
        tma_box(sm.regA, &maps.Cs, 0, ci.t0, &sm.bar_cb);
        tma_box(sm.regA + Q * 128, &maps.Cs, 64, ci.t0, &sm.bar_cb);
        tma_box(sm.regB, &maps.Bs, 0, ci.t0, &sm.bar_cb);
        tma_box(sm.regB + Q * 128, &maps.Bs, 64, ci.t0, &sm.bar_cb);
    }
    if (warp == 0) { tmem_alloc(&sm.tmem_base, 256); tc_fence_before(); }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const uint32_t tG = tmem, tYi = tmem + 128, tYx = tmem + 192;   // accumulator columns: G, Y inside the chunk, C H_in^T
    // Operand descriptors are built once; an instruction's descriptor is a base plus the step along the contraction index
    // (the start-address field counts 16-byte units and cannot carry out of its 14 bits: shared memory ends below 256 KB).
    // C and B rows: swizzled tiles; contraction step k (16 states) starts 32 bytes further on inside a half of 64 states,
    // the second half lies one 16 KB box further on.  The masked G that replaces the B rows is un-swizzled.
    const uint64_t dC = operand_desc_sw128(smem_u32(sm.regA)), dB = operand_desc_sw128(smem_u32(sm.regB));
    const uint64_t dM = operand_desc(smem_u32(sm.regB), kColBytes, 128);
    const uint64_t dH = operand_desc(smem_u32(hin), kHinColBytes, 128), dX = operand_desc(smem_u32(xd), 128, kXdColBytes);
    auto kstep = [](int k) { return (uint64_t)(((k >> 2) * (Q * 128) + (k & 3) * 32) >> 4); };

    // G = C B^T needs inputs of the call only: it is issued while the kernels ahead are still at work.
    const bool cb_ok = mbar_wait_bounded(&sm.bar_cb, 0u);
    if (cb_ok && tid == 0) {
        tc_fence_after();
        constexpr uint32_t idG = instr_desc(Q, false, false);
#pragma unroll
        for (int k = 0; k < N / 16; ++k)   // G[t][s] = sum_n C[t][n] B[s][n]
            mma_bf16(tG, dC + kstep(k), dB + kstep(k), idG, k > 0);
        mma_commit(&sm.bar_g);
    }
    grid_wait();   // the incoming states and the running decays are the work of the kernels just before
    if (tid == 0) {
        mbar_expect_tx(&sm.bar_in, 2 * N * P * 2 + Q * 4);
        bulk_load(hin, p.ws_hin + ch_head * 2 * N * P, 2 * N * P * 2, &sm.bar_in);
        bulk_load(sm.csl, p.ws_csl + ch_head * Q, Q * 4, &sm.bar_in);
    }
    // skip term inputs of the warp's rows (u of this lane's channel pair, from kernel 1): requested now, used at the very end
    const int d = head * P + 2 * lane;
    uint32_t uraw[kRowsPerWarp];
#pragma unroll
    for (int i = 0; i < kRowsPerWarp; ++i) {
        const int r = warp * kRowsPerWarp + i;
        uraw[i] = r < rows ? *reinterpret_cast<const uint32_t*>(p.ws_u + (size_t)(ci.t0 + r) * p.L.d_inner + d) : 0u;
    }

    const bool ok = cb_ok && mbar_wait_bounded(&sm.bar_in, 0u);
    if (ok && tid == 0) {
        tc_fence_after();
        constexpr uint32_t idX = instr_desc(P, false, false);
#pragma unroll
        for (int k = 0; k < 2 * (N / 16); ++k) {   // Yx[t][p] = sum_n C[t][n] h_in[p][n], value then remainder
            const int kk = k % (N / 16), part = k / (N / 16);
            mma_bf16(tYx, dC + kstep(kk), dH + (uint64_t)((part * (N * P * 2) + kk * 2 * kHinColBytes) >> 4), idX, k > 0);
        }
        mma_commit(&sm.bar_x);
    }
    // The mask needs G and the decays only: it is written while C H_in^T runs.
    const bool g_ok = ok && mbar_wait_bounded(&sm.bar_g, 0u);
    if (g_ok) {
        tc_fence_after();
        // row t of G, masked: M[t][s] = G[t][s] exp(cs_t - cs_s) for s <= t, else 0; written over the B boxes (G is complete).
        // Warps w and w + 4 own rows 32 (w % 4) ..: the first takes column blocks 0 and 3, the second 1 and 2 (five
        // non-zero blocks of 32 x 32 on each side of the split).
        const int rb = warp & 3, row = rb * 32 + lane;
        const float my = sm.csl[row];
#pragma unroll 1
        for (int q = 0; q < 2; ++q) {
            const int cb = warp < 4 ? (q == 0 ? 0 : 3) : (q == 0 ? 1 : 2);
            uint32_t packed[16];
            if (cb <= rb) {   // column blocks right of the warp's rows are all zero
                float g[32];
                tmem_ld32(tG + ((uint32_t)(rb * 32) << 16) + cb * 32, g);
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const int s0 = cb * 32 + j;
                    const float m0 = s0 <= row ? g[j] * ex2(my - sm.csl[s0]) : 0.0f;
                    const float m1 = s0 + 1 <= row ? g[j + 1] * ex2(my - sm.csl[s0 + 1]) : 0.0f;
                    packed[j >> 1] = pack_bf(m0, m1);
                }
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) packed[j] = 0u;
            }
#pragma unroll
            for (int u4 = 0; u4 < 4; ++u4)
                *reinterpret_cast<uint4*>(&Mt[cb * 4 + u4][row][0]) = make_uint4(packed[4 * u4], packed[4 * u4 + 1], packed[4 * u4 + 2], packed[4 * u4 + 3]);
        }
    }
    // Warp 4 has only zeros to write above.  Once C H_in^T is complete, the tiles it read take Xd and the z box.
    if (warp == 4 && g_ok && mbar_wait_bounded(&sm.bar_x, 0u) && lane == 0) {
        mbar_expect_tx(&sm.bar_late, kXdBytes + Q * P * 2);
        bulk_load(xd, p.ws_xd + ch_head * (kXdBytes / 2), kXdBytes, &sm.bar_late);
        tma_box(zs, &maps.z, head * P, ci.t0, &sm.bar_late);
    }
    const bool late_ok = g_ok && mbar_wait_bounded(&sm.bar_late, 0u);
    fence_async_smem();
    tc_fence_before();
    const bool all_ok = !__syncthreads_or(!late_ok);
    if (all_ok && tid == 0) {
        tc_fence_after();
        constexpr uint32_t idY = instr_desc(P, false, true);
#pragma unroll
        for (int k = 0; k < Q / 16; ++k)   // Yi[t][p] = sum_s M[t][s] Xd[s][p]; the masked G lies where the B rows were
            mma_bf16(tYi, dM + (uint64_t)(k * 2 * kColBytes >> 4), dX + (uint64_t)(k * 256 >> 4), idY, k > 0);
        mma_commit(&sm.bar_y);
    }
    bool y_ok = all_ok && mbar_wait_bounded(&sm.bar_y, 0u);
    if (y_ok) {
        tc_fence_after();
        const int rb = warp & 3, row = rb * 32 + lane, half = warp >> 2;
        const float scale = ex2(sm.csl[row]);   // decay from the chunk's start through this row
        float yi[32], yx[32];
        tmem_ld32(tYi + ((uint32_t)(rb * 32) << 16) + half * 32, yi);
        tmem_ld32(tYx + ((uint32_t)(rb * 32) << 16) + half * 32, yx);
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 32; ++j) yi[j] = fmaf(scale, yx[j], yi[j]);
        // the staging rows lie over the operand tiles of the product that has just completed
#pragma unroll
        for (int j = 0; j < 32; ++j) ystage[row][half * 32 + j] = yi[j];
    }
    y_ok = !__syncthreads_or(!y_ok);
    if (y_ok) {
        // skip term, gate, store: the warp's rows, this lane's channel pair (128 contiguous bytes per row and warp)
        const float da = p.L.D ? __ldg(p.L.D + d) : 0.0f, db = p.L.D ? __ldg(p.L.D + d + 1) : 0.0f;
        const uint32_t* zc = reinterpret_cast<const uint32_t*>(zs) + lane;
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) {
            const int r = warp * kRowsPerWarp + i;
            if (r < rows) {
                const uint32_t zv = zc[r * (P / 2)];
                const float oa = fmaf(da, bf_lo(uraw[i]), ystage[r][2 * lane]) * silu_gate(bf_lo(zv));
                const float ob = fmaf(db, bf_hi(uraw[i]), ystage[r][2 * lane + 1]) * silu_gate(bf_hi(zv));
                *reinterpret_cast<uint32_t*>(p.out + (size_t)(ci.t0 + r) * p.ldo + d) = pack_bf(oa, ob);
            }
        }
    } else if (tid == 0) {
        flag(p.dev_status, MDRAFT_DEV_WAIT_EXPIRED);
        if (!cb_ok) mbar_wait_bounded(&sm.bar_cb, 0u);   // copies target this block's shared memory: one more bounded chance
        if (!ok) mbar_wait_bounded(&sm.bar_in, 0u);
        if (g_ok && !late_ok) mbar_wait_bounded(&sm.bar_late, 0u);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_free(tmem, 256);
}

template <typename K>
cudaError_t allow_smem(K kernel, size_t bytes) {
    // two blocks of ~100 KB per SM: ask for the largest shared-memory carve-out up front, so that the second block of
    // an SM does not wait for the split to be changed
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

// Launch with programmatic stream serialisation: the kernel may begin before the one ahead of it has finished.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, int threads, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

}  // namespace

cudaError_t launch_ssd_prefill(const SsdPrefillArgs& p, const SsdMaps& maps, cudaStream_t st) {
    const int H = p.L.n_heads;
    cudaError_t e;
    constexpr size_t smem1 = sizeof(StateSmem) + 1024, smem3 = sizeof(ScanSmem) + 1024;
    if ((e = allow_smem(ssd_chunk_state_kernel, smem1)) != cudaSuccess) return e;
    if ((e = allow_smem(ssd_chunk_scan_kernel, smem3)) != cudaSuccess) return e;
    dim3 grid(H, p.n_chunks_bound);
    if ((e = launch_pdl(ssd_chunk_state_kernel, grid, kThreads, smem1, st, p, maps)) != cudaSuccess) return e;
    dim3 g2((p.L.d_inner * (N / 4) + kPassThreads - 1) / kPassThreads, p.n_seq);
    if ((e = launch_pdl(ssd_state_passing_kernel, g2, kPassThreads, 0, st, p)) != cudaSuccess) return e;
    if ((e = launch_pdl(ssd_chunk_scan_kernel, grid, kThreads, smem3, st, p, maps)) != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace mdraft
