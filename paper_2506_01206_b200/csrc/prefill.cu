// Context encode: conv1d+SiLU -> Delta -> S6 scan -> gate, chunked over tokens.
//
// The recurrence h_t = a_t h_{t-1} + b_t is first-order linear, so a chunk of tokens acts on the incoming
// state as h_out = P h_in + q with P = prod a_t = exp(A * sum Delta_t) and q = the chunk's result from a zero
// state.  Three stream-ordered kernels, none of which waits on another block:
//   1. summary pass (chunk_kernel, kOut = false): every chunk but the last of a sequence computes (sum Delta, q)
//      from a zero state; the first chunk of a split sequence also stashes the sequence's starting conv window.
//   2. carry scan: per (channel, state) the (P, q) pairs of a sequence are combined in token order (eight groups
//      of chunks folded side by side, group results exchanged through shared memory); entry c of the summary
//      array is overwritten with the state after chunk c, and the starting state is stashed, so that the final
//      state may later be written to the slot the starting state came from.
//   3. output pass (chunk_kernel, kOut = true): every chunk starts from its incoming state, runs its tokens and
//      writes the outputs; the last chunk stores the final state and conv window.
// A call in which every sequence fits one chunk runs the output pass only.
//
// Data movement.  One thread owns one channel and keeps its 16 state entries in registers as 8 packed pairs
// (fma.rn.f32x2 / mul.rn.f32x2: one instruction per two entries).  A block of 128 or 512 channels walks its chunk in
// tiles of 16 (bf16) or 8 (fp32) tokens; the x / dt / z boxes (tile x 128 channels) and the B / C boxes of a tile
// are brought into a ring of shared-memory stages by TMA (cp.async.bulk.tensor, one instruction per matrix and
// tile, completion counted on an mbarrier), two tiles ahead of the arithmetic.  The block is warp-specialised: one extra
// warp queues the copies, widens each landed B / C tile to fp32 (read afterwards as 128-bit broadcasts) and hands it
// to the 4 or 16 channel warps through a "ready" mbarrier; each channel warp releases a stage through an "empty" mbarrier
// when it is done, so the channel warps never wait for one another.  Every wait on an mbarrier is bounded: if
// it runs out, the warp raises MDRAFT_DEV_WAIT_EXPIRED and stops; the copy warp first gives the copies it still
// has in flight a bounded chance to land (they target this block's shared memory).
#include "common.cuh"
#include "chunk_map.cuh"
#include "prefill.cuh"

namespace mdraft {

namespace {

constexpr int kBoxCols = kPrefillThreads;  // channels of one TMA box (and of one group of four channel warps)
constexpr int kStages = 3;              // shared-memory ring depth
constexpr int kTileBytes = 4096;        // one staged x / dt / z box: kTT rows of kBoxCols activations
constexpr int kBCBytes = 512;           // one staged B or C tile: kTT rows of 16 activations
// A block covers SUB boxes of channels (SUB = 1: 128 channels, 4 channel warps; SUB = 4: 512 channels, 16 channel
// warps that share the block's B / C tiles and advance tile by tile together).  Stage layout: x boxes, dt boxes,
// z boxes, B, C.
__host__ __device__ constexpr int stage_bytes(int sub) { return 3 * sub * kTileBytes + 2 * kBCBytes; }
__host__ __device__ constexpr int off_x(int) { return 0; }
__host__ __device__ constexpr int off_dt(int sub) { return sub * kTileBytes; }
__host__ __device__ constexpr int off_z(int sub) { return 2 * sub * kTileBytes; }
__host__ __device__ constexpr int off_b(int sub) { return 3 * sub * kTileBytes; }
__host__ __device__ constexpr int off_c(int sub) { return 3 * sub * kTileBytes + kBCBytes; }
__host__ __device__ constexpr int smem_bytes(int sub) { return kStages * (stage_bytes(sub) + 2 * kBCBytes * 2); }  // + fp32 B, C
constexpr int kFmaPairs = 1;            // pairs of decays per token computed on the FMA pipe when A is general (measured: 0 -> 43.8, 1 -> 42.5, 2 -> 43.0, 3 -> 45.6 us per 2048x1536 call)
constexpr int GRP = 4;                  // tokens whose state-independent part is computed together (measured: 2 % faster than one by one)

template <typename AT> struct TileTokens { static constexpr int v = kPrefillTileRowBytes / (int)sizeof(AT); };  // 16 (bf16) or 8 (fp32)

typedef unsigned long long u64;

// ---------------------------------------------------------------- packed fp32 pairs
__device__ __forceinline__ u64 pk(float lo, float hi) {
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpk(u64 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ float hi_of(u64 v) {
    float lo, hi;
    unpk(v, lo, hi);
    return hi;
}
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ u64 mul2(u64 a, u64 b) {
    u64 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

__device__ __forceinline__ u64 add2(u64 a, u64 b) {
    u64 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// 2^x for a pair of arguments x <= 0 on the FMA pipe instead of the special-function unit (which a general A keeps
// busy with 16 exponentials per token, channel and pass).  x = j + f with j = round(x) taken from the mantissa of
// x + 1.5*2^23 and f in [-0.5, 0.5]; 2^f = 1 + f g(f) with g of degree 4 interpolated at Chebyshev nodes (relative error
// 2.8e-7 at most, 1e-8 on average: the accuracy of ex2.approx, and exactly 1 at 0); the result's exponent field then takes j.  Arguments below -126 are raised to -126
// (the true value is below 1.2e-38 there and the product with the state flushes to zero either way).
__device__ __forceinline__ u64 exp2_pair_fma(u64 x) {
    float lo, hi;
    unpk(x, lo, hi);
    x = pk(fmaxf(lo, -126.0f), fmaxf(hi, -126.0f));
    const u64 magic = pk(12582912.0f, 12582912.0f);
    const u64 t = add2(x, magic);                                   // integer part in the low mantissa bits
    const u64 r = add2(t, pk(-12582912.0f, -12582912.0f));          // round(x) as a float
    const u64 f = fma2(r, pk(-1.0f, -1.0f), x);                     // x - round(x)
    u64 q = pk(0.0013381302f, 0.0013381302f);                      // (2^f - 1) / f ...
    q = fma2(q, f, pk(0.009666368f, 0.009666368f));
    q = fma2(q, f, pk(0.05550381f, 0.05550381f));
    q = fma2(q, f, pk(0.2402235f, 0.2402235f));
    q = fma2(q, f, pk(0.6931472f, 0.6931472f));
    q = fma2(q, f, pk(1.0f, 1.0f));                                 // ... so that 2^0 is exactly 1
    float qlo, qhi, tlo, thi;
    unpk(q, qlo, qhi);
    unpk(t, tlo, thi);
    qlo = __int_as_float(__float_as_int(qlo) + (__float_as_int(tlo) << 23));
    qhi = __int_as_float(__float_as_int(qhi) + (__float_as_int(thi) << 23));
    return pk(qlo, qhi);
}

// ---------------------------------------------------------------- mbarrier + bulk copy
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes + kOverstateTx) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(kPollNs)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// One 2-D box of a matrix -> shared memory (TMA).  `col` times the element size must be a multiple of 16 bytes;
// rows or columns of the box that fall outside the matrix arrive as zeros and still count towards the
// transaction bytes.
__device__ __forceinline__ void tma_box(void* dst, const CUtensorMap* map, int col, int row, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(smem_u32(dst)),
                 "l"(reinterpret_cast<uint64_t>(map)), "r"(col), "r"(row), "r"(smem_u32(bar))
                 : "memory");
}

// ---------------------------------------------------------------- programmatic dependent launch
// The three kernels of a call (and the first kernel of the next call on the stream) are launched with programmatic
// stream serialisation: a kernel may start while its predecessor is still running, and must pass grid_wait() before
// it touches anything the predecessor (or a kernel before that) writes, or overwrites anything it reads.  Every block
// passes grid_wait() on every path, so that a kernel's completion implies that of all its predecessors.
__device__ __forceinline__ void grid_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---------------------------------------------------------------- one channel's running computation
template <typename AT, bool kPow, bool kOut, bool kFast>
struct ChannelScan {
    u64 h[kN / 2];        // state, entries (2k, 2k+1) packed
    u64 a2[kN / 2];       // general A: A[d][n] * log2(e), packed;  structured A: only a20 is used
    float a20;
    float w[kW];
    float win[kW - 1];    // previous raw inputs, oldest first
    float cb, dtb, dsk, sum_delta;
    uint32_t flags;

    __device__ __forceinline__ void init(const LayerDev& L, int d) {
        const float4* Ap = reinterpret_cast<const float4*>(L.A + (size_t)d * kN);
#pragma unroll
        for (int q = 0; q < kN / 4; ++q) {
            float4 a = __ldg(Ap + q);
            a2[2 * q] = pk(a.x * kLog2e, a.y * kLog2e);
            a2[2 * q + 1] = pk(a.z * kLog2e, a.w * kLog2e);
            if (q == 0) a20 = a.x * kLog2e;
        }
        float4 wv = __ldg(reinterpret_cast<const float4*>(L.conv_w + (size_t)d * kW));
        w[0] = wv.x; w[1] = wv.y; w[2] = wv.z; w[3] = wv.w;
        cb = L.conv_b ? __ldg(L.conv_b + d) : 0.0f;
        dtb = L.dt_bias ? __ldg(L.dt_bias + d) : 0.0f;
        dsk = L.D ? __ldg(L.D + d) : 0.0f;
        sum_delta = 0.0f;
        flags = kFast ? (uint32_t)MDRAFT_DT_SOFTPLUS : L.flags;
#pragma unroll
        for (int k = 0; k < kN / 2; ++k) h[k] = pk(0.0f, 0.0f);
    }

    // The 16 decays exp(A[d][n] * delta) as 8 packed pairs.
    __device__ __forceinline__ void decays(float delta, u64 (&P)[kN / 2]) const {
        if (kPow) {
            const float r1 = ex2(delta * a20);
            const float r2 = r1 * r1;
            P[0] = pk(r1, r2);
            P[1] = mul2(P[0], pk(r2, r2));
            const float r4 = hi_of(P[1]);
            const u64 R4 = pk(r4, r4);
            P[2] = mul2(P[0], R4);
            P[3] = mul2(P[1], R4);
            const float r8 = hi_of(P[3]);
            const u64 R8 = pk(r8, r8);
#pragma unroll
            for (int k = 0; k < 4; ++k) P[4 + k] = mul2(P[k], R8);
        } else {
            const u64 dd = pk(delta, delta);
            // With a step size known to be >= 0 (softplus) the arguments are <= 0 and the last kFmaPairs pairs go to
            // the FMA pipe, which takes a little load off the special-function unit.
            constexpr int kMufuPairs = kFast ? kN / 2 - kFmaPairs : kN / 2;
#pragma unroll
            for (int k = 0; k < kN / 2; ++k) {
                if (k < kMufuPairs) {
                    float lo, hi;
                    unpk(mul2(dd, a2[k]), lo, hi);
                    P[k] = pk(ex2(lo), ex2(hi));
                } else {
                    P[k] = exp2_pair_fma(mul2(dd, a2[k]));
                }
            }
        }
    }

    // A token is processed in two steps, so that the first, which has no dependence between tokens, can be run for a
    // group of tokens at once (their special-function latencies overlap) before the second walks the state forward.
    struct Pre { float u, delta, du, gate; };  // conv+SiLU output, step size, their product, SiLU(z)
    // Step 1: everything that does not touch the state.
    __device__ __forceinline__ void pre(float xv, float zv, float dtv, Pre& e) {
        if (flags & MDRAFT_PRECONV) {
            e.u = xv;
        } else {
            float acc = fmaf(w[0], win[0], cb);
            acc = fmaf(w[1], win[1], acc);
            acc = fmaf(w[2], win[2], acc);
            acc = fmaf(w[3], xv, acc);
            win[0] = win[1]; win[1] = win[2]; win[2] = xv;
            e.u = silu(acc);
        }
        e.delta = 0.f; e.du = 0.f; e.gate = 0.f;
        if (flags & MDRAFT_CONV_ONLY) return;
        const float v = dtv + dtb;
        e.delta = (flags & MDRAFT_DT_SOFTPLUS) ? softplus(v) : v;
        if (!kOut) sum_delta += e.delta;
        e.du = e.delta * e.u;
        if (kOut) e.gate = silu(zv);
    }
    // Step 2: state update and output.  Bt / Ct point at 16 fp32 values in shared memory.  Returns the output (kOut),
    // or u in conv-only mode.
    __device__ __forceinline__ float post(const Pre& e, const float* Bt, const float* Ct) {
        if (flags & MDRAFT_CONV_ONLY) return e.u;
        u64 P[kN / 2];
        decays(e.delta, P);
        const u64 DU = pk(e.du, e.du);
        u64 y0 = pk(0.0f, 0.0f), y1 = pk(0.0f, 0.0f);
        const ulonglong2* B2 = reinterpret_cast<const ulonglong2*>(Bt);
        const ulonglong2* C2 = reinterpret_cast<const ulonglong2*>(Ct);
#pragma unroll
        for (int q = 0; q < kN / 4; ++q) {
            const ulonglong2 b = B2[q];
            h[2 * q] = fma2(P[2 * q], h[2 * q], mul2(DU, b.x));
            h[2 * q + 1] = fma2(P[2 * q + 1], h[2 * q + 1], mul2(DU, b.y));
            if (kOut) {
                const ulonglong2 c = C2[q];
                y0 = fma2(c.x, h[2 * q], y0);
                y1 = fma2(c.y, h[2 * q + 1], y1);
            }
        }
        if (!kOut) return 0.0f;
        float ya, yb, yc, yd;
        unpk(y0, ya, yb);
        unpk(y1, yc, yd);
        return fmaf(dsk, e.u, (ya + yb) + (yc + yd)) * e.gate;
    }
};

// Conv window at the start of a chunk: the W-1 rows before t0, taken from the sequence itself, or (chunk 0)
// from `src_rows` = (W-1, D) activations, or zeros.
template <typename AT>
__device__ __forceinline__ void load_window(float* win, const AT* x, int64_t ldx, int d, int t0, int k, const AT* src_rows, int D) {
#pragma unroll
    for (int j = 0; j < kW - 1; ++j) {
        if (k > 0) win[j] = Act<AT>::load(x + (size_t)(t0 - (kW - 1) + j) * ldx + d);
        else win[j] = src_rows ? Act<AT>::load(src_rows + (size_t)j * D + d) : 0.0f;
    }
}

// One lane queues the copies of one tile: per matrix one box for every 128 channels of the block that exist.
// `mask`: bit 0 = dt, bit 1 = z, bit 2 = B, bit 3 = C (x is always copied).  Every box is full size whatever part
// of it lies inside the matrix.
template <int SUB>
__device__ __forceinline__ void issue_tile(unsigned char* stage, uint64_t* bar, const PrefillMaps& m, int t, int d0, int D, uint32_t mask) {
    const uint32_t n_wide = 1u + (mask & 1u) + ((mask >> 1) & 1u), n_bc = ((mask >> 2) & 1u) + ((mask >> 3) & 1u);
    const uint32_t subs = (uint32_t)min(SUB, (D - d0 + kBoxCols - 1) / kBoxCols);
    mbar_expect_tx(bar, subs * n_wide * kTileBytes + n_bc * kBCBytes);
#pragma unroll
    for (int sb = 0; sb < SUB; ++sb) {
        if (sb < (int)subs) {
            const int c = d0 + sb * kBoxCols;
            tma_box(stage + off_x(SUB) + sb * kTileBytes, &m.x, c, t, bar);
            if (mask & 1u) tma_box(stage + off_dt(SUB) + sb * kTileBytes, &m.dt, c, t, bar);
            if (mask & 2u) tma_box(stage + off_z(SUB) + sb * kTileBytes, &m.z, c, t, bar);
        }
    }
    if (mask & 4u) tma_box(stage + off_b(SUB), &m.B, 0, t, bar);
    if (mask & 8u) tma_box(stage + off_c(SUB), &m.C, 0, t, bar);
}

// ---------------------------------------------------------------------------------------------------
template <typename AT, int SUB, bool kPow, bool kOut, bool kFast>
__global__ void __launch_bounds__(SUB * kBoxCols + 32, SUB == 1 ? 4 : 1) chunk_kernel(const PrefillArgs p, const __grid_constant__ PrefillMaps maps) {
    constexpr int TT = TileTokens<AT>::v;
    constexpr int kCB = SUB * kBoxCols;          // channels per block, one thread each
    constexpr int kStageBytes = stage_bytes(SUB);
    extern __shared__ __align__(128) unsigned char s_dyn[];
    unsigned char (*s_stage)[kStageBytes] = reinterpret_cast<unsigned char (*)[kStageBytes]>(s_dyn);
    float (*sBf)[TT][kN] = reinterpret_cast<float (*)[TT][kN]>(s_dyn + kStages * kStageBytes);
    float (*sCf)[TT][kN] = reinterpret_cast<float (*)[TT][kN]>(s_dyn + kStages * kStageBytes + kStages * TT * kN * 4);
    __shared__ __align__(8) uint64_t bar_raw[kStages];    // copies of a tile have landed (transaction count)
    __shared__ __align__(8) uint64_t bar_ready[kStages];  // ... and its B / C are widened: channel warps may start
    __shared__ __align__(8) uint64_t bar_empty[kStages];  // all channel warps are done with the stage

    const int D = p.L.d_inner;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d0 = blockIdx.x * kCB;
    const int cols = min(kCB, D - d0);
    const int d = d0 + tid;
    const bool live = tid < cols;            // false for the copy warp (tid >= kCB) as well
    const bool copy_warp = warp == kCB / 32;
    const int cidx = blockIdx.y;
    const uint32_t flags = kFast ? (uint32_t)MDRAFT_DT_SOFTPLUS : p.L.flags;
    const bool conv_only = flags & MDRAFT_CONV_ONLY, preconv = flags & MDRAFT_PRECONV;

    // Layer constants first: they depend on nothing but the channel and are never written by a kernel of this
    // library, so they may be read before the predecessor on the stream has finished.
    ChannelScan<AT, kPow, kOut, kFast> cs;
    if (live) cs.init(p.L, d);

    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&bar_raw[s], 1);
            mbar_init(&bar_ready[s], 1);
            mbar_init(&bar_empty[s], kCB / 32);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (!kOut) {
        // Summary pass: the inputs may be the work of the kernel before this call, so nothing else is read before
        // that kernel is known to be complete; only then may the kernels after this one start.
        grid_wait();
        grid_release_dependents();
    } else {
        grid_release_dependents();
        if (!p.pdl_inputs_ready) grid_wait();  // unsplit call: no summary pass has waited for the inputs yet
    }

    if (kOut) {
        // Sequences without tokens have no chunk: their final state is their starting state.
        if (cidx == 0 && p.final_slot) {
            grid_wait();  // the state pool may be the work of the kernels before
            for (int s = 0; s < p.n_seq; ++s) {
                int lo = p.cu ? __ldg(p.cu + s) : 0, hi = p.cu ? __ldg(p.cu + s + 1) : p.T;
                bool bad = (lo < 0) || (hi < lo) || (hi > p.T);
                if (bad && blockIdx.x == 0 && tid == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SEQLENS);
                if (bad || hi != lo) continue;
                int fs = __ldg(p.final_slot + s), is = load_slot(p.init_slot, s);
                if (fs < 0 || fs == is) continue;
                if (fs >= p.pool.n_slots || is >= p.pool.n_slots) {
                    if (blockIdx.x == 0 && tid == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
                    continue;
                }
                if (live) {
                    float* dh = p.pool.ssm + (size_t)fs * p.pool.ssm_slot_stride + (size_t)d * kN;
                    AT* dc = static_cast<AT*>(p.pool.conv) + (size_t)fs * p.pool.conv_slot_stride;
                    const float* sh = is >= 0 ? p.pool.ssm + (size_t)is * p.pool.ssm_slot_stride + (size_t)d * kN : nullptr;
                    const AT* sc = is >= 0 ? static_cast<const AT*>(p.pool.conv) + (size_t)is * p.pool.conv_slot_stride : nullptr;
                    for (int n = 0; n < kN; ++n) dh[n] = sh ? sh[n] : 0.0f;
                    for (int j = 0; j < kW - 1; ++j) dc[(size_t)j * D + d] = sc ? sc[(size_t)j * D + d] : Act<AT>::from_f32(0.0f);
                }
            }
        } else if (cidx == 0 && blockIdx.x == 0 && tid < 32 && p.cu) {
            for (int s = tid; s < p.n_seq; s += 32) {
                int lo = __ldg(p.cu + s), hi = __ldg(p.cu + s + 1);
                if ((lo < 0) || (hi < lo) || (hi > p.T)) flag(p.dev_status, MDRAFT_DEV_BAD_SEQLENS);
            }
        }
    }

    const ChunkInfo ci = find_chunk(p.cu, p.n_seq, p.T, p.chunk_len, cidx);
    if (ci.seq < 0) { if (kOut) grid_wait(); return; }
    if (!kOut) {
        // No summary is needed for an unsplit sequence or for a sequence's last chunk; in conv-only mode the only
        // job left is the first chunk's stash of the starting window.
        if (ci.nck == 1 || ci.k == ci.nck - 1) return;
        if ((flags & MDRAFT_CONV_ONLY) && ci.k > 0) return;
    }

    const AT* x = static_cast<const AT*>(p.x);
    AT* out = static_cast<AT*>(p.out);

    // In conv-only mode the summary pass computes nothing (it only stashes, below).
    const bool compute = kOut || !conv_only;
    const int ntiles = compute ? (ci.t1 - ci.t0 + TT - 1) / TT : 0;
    uint32_t mask = 0;
    if (!conv_only) mask = kOut ? 15u : 5u;  // summary pass: x, dt, B

    const bool want_c = kOut && !conv_only;
    const int pre = min(kStages - 1, ntiles);
    if (copy_warp && lane == 0)  // the first tiles go out before anything else is looked up
        for (int j = 0; j < pre; ++j) issue_tile<SUB>(s_stage[j], &bar_raw[j], maps, ci.t0 + j * TT, d0, D, mask);

    const int islot = load_slot(p.init_slot, ci.seq);
    const int fslot = load_slot(p.final_slot, ci.seq);
    if (islot >= p.pool.n_slots || fslot >= p.pool.n_slots) {  // whole sequence becomes a no-op
        if (kOut && tid == 0 && blockIdx.x == 0 && ci.k == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
        if (copy_warp)  // the tiles already queued still land in this block's shared memory: see them in first
            for (int j = 0; j < pre; ++j) mbar_wait_bounded(&bar_raw[j], 0u);
        if (kOut) grid_wait();
        return;
    }

    if (copy_warp) {
        // ---- copy warp: keep two tiles in flight, widen B / C of each landed tile, hand it over.
        int landed = 0, queued = pre;  // tiles [landed, queued) are in flight
        bool ok = true;
        for (int j = 0; j < ntiles && ok; ++j) {
            const int s = j % kStages;
            ok = mbar_wait_bounded(&bar_raw[s], (uint32_t)(j / kStages) & 1u);
            if (!ok) break;
            landed = j + 1;
            if (!conv_only) {
                const int rows = min(TT, ci.t1 - (ci.t0 + j * TT));
                const AT* rb = reinterpret_cast<const AT*>(s_stage[s] + off_b(SUB));
                const AT* rc = reinterpret_cast<const AT*>(s_stage[s] + off_c(SUB));
                for (int i = lane; i < rows * kN; i += 32) {
                    (&sBf[s][0][0])[i] = Act<AT>::to_f32(rb[i]);
                    if (want_c) (&sCf[s][0][0])[i] = Act<AT>::to_f32(rc[i]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_ready[s]);
            const int nxt = j + kStages - 1;  // goes into the stage that tile j - 1 occupied
            if (nxt < ntiles) {
                if (nxt >= kStages) ok = mbar_wait_bounded(&bar_empty[nxt % kStages], (uint32_t)(nxt / kStages - 1) & 1u);
                if (!ok) break;
                if (lane == 0) issue_tile<SUB>(s_stage[nxt % kStages], &bar_raw[nxt % kStages], maps, ci.t0 + nxt * TT, d0, D, mask);
                queued = nxt + 1;
            }
        }
        if (!ok) {
            if (lane == 0) flag(p.dev_status, MDRAFT_DEV_WAIT_EXPIRED);
            for (int j = landed; j < queued; ++j) mbar_wait_bounded(&bar_raw[j % kStages], (uint32_t)(j / kStages) & 1u);
        }
        if (kOut) grid_wait();
        return;
    }

    // Output pass: everything read from here on (workspace, state pool) may be the work of the kernels just before.
    if (kOut) grid_wait();
    if (live) {
        const bool split = ci.nck > 1;
        if (!preconv) {
            const AT* rows = nullptr;
            if (ci.k == 0) {
                if (kOut && split) rows = static_cast<const AT*>(p.ws_conv) + (size_t)ci.seq * (kW - 1) * D;
                else if (islot >= 0) rows = static_cast<const AT*>(p.pool.conv) + (size_t)islot * p.pool.conv_slot_stride;
            }
            load_window<AT>(cs.win, x, p.ldx, d, ci.t0, ci.k, rows, D);
        }
        if (!kOut) {
            if (ci.k == 0 && !preconv) {  // stash the starting window where the output pass will look for it
                AT* stash = static_cast<AT*>(p.ws_conv) + (size_t)ci.seq * (kW - 1) * D;
#pragma unroll
                for (int j = 0; j < kW - 1; ++j) stash[(size_t)j * D + d] = Act<AT>::from_f32(cs.win[j]);
            }
        } else if (!conv_only) {
            // Incoming state: the slot itself for an unsplit sequence, else what the carry scan left.
            const float4* src = nullptr;
            size_t step = 1;
            if (!split) {
                if (islot >= 0) src = reinterpret_cast<const float4*>(p.pool.ssm + (size_t)islot * p.pool.ssm_slot_stride + (size_t)d * kN);
            } else if (ci.k == 0) {
                src = reinterpret_cast<const float4*>(p.ws_h0) + ((size_t)ci.seq * (kN / 4)) * D + d;
                step = D;
            } else {
                src = reinterpret_cast<const float4*>(p.ws_q) + ((size_t)(cidx - 1) * (kN / 4)) * D + d;
                step = D;
            }
            if (src) {
#pragma unroll
                for (int q = 0; q < kN / 4; ++q) {
                    const float4 v = src[(size_t)q * step];
                    cs.h[2 * q] = pk(v.x, v.y); cs.h[2 * q + 1] = pk(v.z, v.w);
                }
            }
        }
    }

    // ---- channel warps
    for (int j = 0; j < ntiles; ++j) {
        const int s = j % kStages;
        const int t = ci.t0 + j * TT;
        const int rows = min(TT, ci.t1 - t);
        const uint32_t parity = (uint32_t)(j / kStages) & 1u;
        if (!mbar_wait_bounded(&bar_ready[s], parity) || !mbar_wait_bounded(&bar_raw[s], parity)) {
            if (lane == 0) flag(p.dev_status, MDRAFT_DEV_WAIT_EXPIRED);  // the outputs of this chunk are invalid
            return;
        }
        if (live) {
            const unsigned char* st = s_stage[s];
            const int box = (tid / kBoxCols) * kTileBytes, col = tid % kBoxCols;  // this thread's box of 128 channels and its column in it
            const AT* sx = reinterpret_cast<const AT*>(st + off_x(SUB) + box) + col;
            const AT* sdt = reinterpret_cast<const AT*>(st + off_dt(SUB) + box) + col;
            const AT* sz = reinterpret_cast<const AT*>(st + off_z(SUB) + box) + col;
            AT* orow = out + (size_t)t * p.ldo + d;
            typedef typename ChannelScan<AT, kPow, kOut, kFast>::Pre Pre;
            int r = 0;
            for (; r + GRP <= rows; r += GRP) {
                Pre e[GRP];
                float o[GRP];
#pragma unroll
                for (int g = 0; g < GRP; ++g) {
                    const float xv = Act<AT>::to_f32(sx[(r + g) * kBoxCols]);
                    const float dtv = conv_only ? 0.0f : Act<AT>::to_f32(sdt[(r + g) * kBoxCols]);
                    const float zv = want_c ? Act<AT>::to_f32(sz[(r + g) * kBoxCols]) : 0.0f;
                    cs.pre(xv, zv, dtv, e[g]);
                }
#pragma unroll
                for (int g = 0; g < GRP; ++g) o[g] = cs.post(e[g], sBf[s][r + g], sCf[s][r + g]);
                if (kOut) {
#pragma unroll
                    for (int g = 0; g < GRP; ++g) orow[(size_t)(r + g) * p.ldo] = Act<AT>::from_f32(o[g]);
                }
            }
            for (; r < rows; ++r) {
                Pre e;
                const float xv = Act<AT>::to_f32(sx[r * kBoxCols]);
                const float dtv = conv_only ? 0.0f : Act<AT>::to_f32(sdt[r * kBoxCols]);
                const float zv = want_c ? Act<AT>::to_f32(sz[r * kBoxCols]) : 0.0f;
                cs.pre(xv, zv, dtv, e);
                const float o = cs.post(e, sBf[s][r], sCf[s][r]);
                if (kOut) orow[(size_t)r * p.ldo] = Act<AT>::from_f32(o);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar_empty[s]);
    }

    if (!live) return;
    if (!kOut) {
        if (compute) {
            float4* dst = reinterpret_cast<float4*>(p.ws_q) + ((size_t)cidx * (kN / 4)) * D + d;
#pragma unroll
            for (int q = 0; q < kN / 4; ++q) {
                float a, b, c, e;
                unpk(cs.h[2 * q], a, b);
                unpk(cs.h[2 * q + 1], c, e);
                dst[(size_t)q * D] = make_float4(a, b, c, e);
            }
            p.ws_sd[(size_t)cidx * D + d] = cs.sum_delta;
        }
        return;
    }
    if (ci.k == ci.nck - 1 && fslot >= 0) {
        if (!conv_only) {
            float4* dst = reinterpret_cast<float4*>(p.pool.ssm + (size_t)fslot * p.pool.ssm_slot_stride + (size_t)d * kN);
#pragma unroll
            for (int q = 0; q < kN / 4; ++q) {
                float a, b, c, e;
                unpk(cs.h[2 * q], a, b);
                unpk(cs.h[2 * q + 1], c, e);
                dst[q] = make_float4(a, b, c, e);
            }
        }
        if (!preconv) {
            AT* dc = static_cast<AT*>(p.pool.conv) + (size_t)fslot * p.pool.conv_slot_stride;
#pragma unroll
            for (int j = 0; j < kW - 1; ++j) dc[(size_t)j * D + d] = Act<AT>::from_f32(cs.win[j]);
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// Carry scan.  Block = 8 warps; a thread owns one state quad (4 entries of one channel), a warp's lanes are 32
// consecutive channels of that quad, so every load and store of a warp is 512 contiguous bytes.  Per round,
// warp g takes kCarryPer consecutive chunks: it loads their summaries at once, folds them into one (P, q) pair,
// publishes the pair, folds the pairs of the warps before it into its starting state, and then replays its own
// chunks to write the state after each.  Rounds carry the running state forward past 48 chunks.
constexpr int kCarryGroups = 8, kCarryPer = 6;

__device__ __forceinline__ float4 fold4(const float4& a, const float4& h, const float4& q) {
    return make_float4(fmaf(a.x, h.x, q.x), fmaf(a.y, h.y, q.y), fmaf(a.z, h.z, q.z), fmaf(a.w, h.w, q.w));
}

__global__ void __launch_bounds__(kCarryGroups * 32) carry_kernel(const PrefillArgs p) {
    __shared__ float4 sP[kCarryGroups][32];
    __shared__ float4 sQ[kCarryGroups][32];
    const int D = p.L.d_inner;
    const int lane = threadIdx.x & 31, g = threadIdx.x >> 5;
    const int quad = blockIdx.y, s = blockIdx.z;
    const int d = blockIdx.x * 32 + lane;
    const bool live = d < D;
    const int dd = live ? d : 0;  // dead lanes shadow channel 0 and write nothing
    float4 a2 = __ldg(reinterpret_cast<const float4*>(p.L.A + (size_t)dd * kN) + quad);
    a2.x *= kLog2e; a2.y *= kLog2e; a2.z *= kLog2e; a2.w *= kLog2e;
    grid_release_dependents();
    // Sequence offsets, slots and the starting state are inputs of the call: the summary pass ahead of this kernel
    // let it start only after everything before the call had finished, so they may be read before the wait below.
    int first, nck;
    seq_chunks(p.cu, p.n_seq, p.T, p.chunk_len, s, first, nck);
    const int islot = load_slot(p.init_slot, s), fslot = load_slot(p.final_slot, s);
    const bool slots_ok = islot < p.pool.n_slots && fslot < p.pool.n_slots;
    float4 carry = make_float4(0.f, 0.f, 0.f, 0.f);
    if (nck > 1 && slots_ok && islot >= 0)
        carry = *(reinterpret_cast<const float4*>(p.pool.ssm + (size_t)islot * p.pool.ssm_slot_stride + (size_t)dd * kN) + quad);
    grid_wait();  // the summaries are the work of the kernel just before
    if (nck <= 1) return;
    if (!slots_ok) return;  // the output pass reports it
    const size_t per_chunk = (size_t)D * (kN / 4);  // float4s in one chunk's [N/4][D] block
    const size_t col = (size_t)quad * D + dd;        // this thread's float4 inside such a block
    float4* wsq = reinterpret_cast<float4*>(p.ws_q);
    if (g == 0 && live) reinterpret_cast<float4*>(p.ws_h0)[(size_t)s * per_chunk + col] = carry;

    const int nsum = nck - 1;  // summaries of chunks 0 .. nck-2
    for (int base = 0; base < nsum; base += kCarryGroups * kCarryPer) {
        const int c0 = base + g * kCarryPer;
        const int cnt = min(kCarryPer, nsum - c0);  // may be <= 0
        float4 q[kCarryPer], a[kCarryPer];
        const float4* qp = wsq + (size_t)(first + c0) * per_chunk + col;
        const float* sp = p.ws_sd + (size_t)(first + c0) * D + dd;
#pragma unroll
        for (int i = 0; i < kCarryPer; ++i) {
            q[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            float sd = 0.0f;  // padding past nsum: decay 1, nothing added
            if (i < cnt) { q[i] = qp[(size_t)i * per_chunk]; sd = sp[(size_t)i * D]; }
            a[i] = make_float4(ex2(a2.x * sd), ex2(a2.y * sd), ex2(a2.z * sd), ex2(a2.w * sd));  // decay of the whole chunk
        }
        float4 Pg = make_float4(1.f, 1.f, 1.f, 1.f), qg = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < kCarryPer; ++i) {
            qg = fold4(a[i], qg, q[i]);
            Pg.x *= a[i].x; Pg.y *= a[i].y; Pg.z *= a[i].z; Pg.w *= a[i].w;
        }
        sP[g][lane] = Pg;
        sQ[g][lane] = qg;
        __syncthreads();
        float4 h = carry;
        for (int gg = 0; gg < g; ++gg) h = fold4(sP[gg][lane], h, sQ[gg][lane]);
        float4 after = h;  // running state after the whole round, the same in every warp
        for (int gg = g; gg < kCarryGroups; ++gg) after = fold4(sP[gg][lane], after, sQ[gg][lane]);
        float4* op = wsq + (size_t)(first + c0) * per_chunk + col;
#pragma unroll
        for (int i = 0; i < kCarryPer; ++i) {
            if (i < cnt) {
                h = fold4(a[i], h, q[i]);
                if (live) op[(size_t)i * per_chunk] = h;
            }
        }
        carry = after;
        __syncthreads();
    }
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

// The wide block needs more dynamic shared memory than a kernel gets by default; the limit is raised once per
// kernel and device (a property of the loaded function, not an allocation).
template <typename K>
cudaError_t allow_smem(K kernel, int bytes) {
    if (bytes <= 48 * 1024) return cudaSuccess;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

template <typename AT, int SUB, bool kPow, bool kFast>
cudaError_t launch_typed(PrefillArgs p, const PrefillMaps& maps, bool chunked, cudaStream_t st) {
    const int D = p.L.d_inner;
    constexpr int kCB = SUB * kBoxCols, kThreads = kCB + 32, kSmem = smem_bytes(SUB);
    dim3 grid((D + kCB - 1) / kCB, p.n_chunks_bound);
    const bool recur = !(p.L.flags & MDRAFT_CONV_ONLY);
    p.pdl_inputs_ready = chunked ? 1 : 0;  // the summary pass waits for the producer of the inputs on behalf of all three
    cudaError_t e = cudaSuccess;
    if (chunked) {
        if ((e = allow_smem(chunk_kernel<AT, SUB, kPow, false, kFast>, kSmem)) != cudaSuccess) return e;
        e = launch_pdl(chunk_kernel<AT, SUB, kPow, false, kFast>, grid, kThreads, kSmem, st, p, maps);
    }
    if (e != cudaSuccess) return e;
    if (p.ev_state) cudaEventRecord(p.ev_state, st);
    if (chunked && recur) {
        dim3 g2((D + 31) / 32, kN / 4, p.n_seq);
        e = launch_pdl(carry_kernel, g2, kCarryGroups * 32, 0, st, p);
        if (e != cudaSuccess) return e;
    }
    if (p.ev_carry) cudaEventRecord(p.ev_carry, st);
    if ((e = allow_smem(chunk_kernel<AT, SUB, kPow, true, kFast>, kSmem)) != cudaSuccess) return e;
    e = launch_pdl(chunk_kernel<AT, SUB, kPow, true, kFast>, grid, kThreads, kSmem, st, p, maps);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

template <typename AT, int SUB>
cudaError_t launch_act(const PrefillArgs& p, const PrefillMaps& maps, bool chunked, cudaStream_t st) {
    const bool pow = p.L.flags & MDRAFT_A_POWERS;
    const bool fast = (p.L.flags & ~(uint32_t)MDRAFT_A_POWERS) == (uint32_t)MDRAFT_DT_SOFTPLUS;
    if (fast) return pow ? launch_typed<AT, SUB, true, true>(p, maps, chunked, st) : launch_typed<AT, SUB, false, true>(p, maps, chunked, st);
    return pow ? launch_typed<AT, SUB, true, false>(p, maps, chunked, st) : launch_typed<AT, SUB, false, false>(p, maps, chunked, st);
}

}  // namespace

cudaError_t launch_prefill(const PrefillArgs& p, const PrefillMaps& maps, int act, bool chunked, bool wide, cudaStream_t st) {
    if (wide) return act == MDRAFT_F32 ? launch_act<float, kPrefillWideBoxes>(p, maps, chunked, st) : launch_act<__nv_bfloat16, kPrefillWideBoxes>(p, maps, chunked, st);
    return act == MDRAFT_F32 ? launch_act<float, 1>(p, maps, chunked, st) : launch_act<__nv_bfloat16, 1>(p, maps, chunked, st);
}

}  // namespace mdraft
