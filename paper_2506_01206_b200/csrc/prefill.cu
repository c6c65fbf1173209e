// Context encode: conv1d+SiLU -> Delta -> S6 scan -> gate, chunked over tokens.
//
// The recurrence h_t = a_t h_{t-1} + b_t is first-order linear, so a chunk of tokens acts on the incoming
// state as h_out = P h_in + q with P = prod a_t = exp(A * sum Delta_t) and q = the chunk's result from a zero
// state.  Three stream-ordered kernels, none of which waits on another block:
//   1. chunk_state : every chunk but the last of a sequence computes (sum Delta, q) from a zero state.
//   2. carry_scan  : per (channel, state) the (P, q) pairs of a sequence are combined in token order with a
//                    warp-shuffle inclusive scan (lanes = chunks); the result is each chunk's incoming state.
//   3. chunk_scan  : every chunk re-runs its tokens from the true incoming state and writes the outputs.
// A sequence that fits one chunk skips 1 and 2.
#include "common.cuh"
#include "prefill.cuh"

namespace mdraft {

namespace {

constexpr int kTT = 32;  // tokens per shared-memory tile of B / C

struct ChunkInfo {
    int seq;     // sequence index, -1 if this chunk id is past the last chunk
    int k;       // chunk index within the sequence
    int nck;     // chunks in the sequence
    int t0, t1;  // token rows of this chunk
    int s0;      // first token row of the sequence
};

// Chunks per sequence: ceil(len / Lc); a sequence whose cu_seqlens entries are out of order or out of range
// gets none.  Global chunk ids number the chunks of sequence 0, then 1, ...  Called by whole warps.
__device__ __forceinline__ void seq_span(const int32_t* cu, int n_seq, int T, int s, int& a, int& len, bool& bad) {
    a = 0; len = 0; bad = false;
    if (s < n_seq) {
        int lo = __ldg(cu + s), hi = __ldg(cu + s + 1);
        bad = (lo < 0) || (hi < lo) || (hi > T);
        if (!bad) { a = lo; len = hi - lo; }
    }
}

__device__ ChunkInfo find_chunk(const int32_t* cu, int n_seq, int T, int Lc, int cidx) {
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    ChunkInfo ci;
    ci.seq = -1; ci.k = 0; ci.nck = 0; ci.t0 = 0; ci.t1 = 0; ci.s0 = 0;
    int base = 0;
    for (int sb = 0; sb < n_seq; sb += 32) {
        int a, len; bool bad;
        seq_span(cu, n_seq, T, sb + lane, a, len, bad);
        int nc = (len + Lc - 1) / Lc;
        int incl = nc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int v = __shfl_up_sync(full, incl, o);
            if (lane >= o) incl += v;
        }
        int total = __shfl_sync(full, incl, 31);
        if (cidx < base + total) {
            unsigned m = __ballot_sync(full, cidx < base + incl);
            int l = __ffs(m) - 1;
            int first = base + __shfl_sync(full, incl, l) - __shfl_sync(full, nc, l);
            int sa = __shfl_sync(full, a, l), sl = __shfl_sync(full, len, l);
            ci.seq = sb + l;
            ci.k = cidx - first;
            ci.nck = __shfl_sync(full, nc, l);
            ci.s0 = sa;
            ci.t0 = sa + ci.k * Lc;
            ci.t1 = min(ci.t0 + Lc, sa + sl);
            return ci;
        }
        base += total;
    }
    return ci;
}

// First global chunk id and chunk count of sequence s.  Called by whole warps.
__device__ void seq_chunks(const int32_t* cu, int n_seq, int T, int Lc, int s, int& first, int& nck) {
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    int base = 0;
    first = 0; nck = 0;
    for (int sb = 0; sb <= s; sb += 32) {
        int a, len; bool bad;
        seq_span(cu, n_seq, T, sb + lane, a, len, bad);
        int nc = (len + Lc - 1) / Lc;
        int incl = nc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int v = __shfl_up_sync(full, incl, o);
            if (lane >= o) incl += v;
        }
        if (s < sb + 32) {
            int l = s - sb;
            nck = __shfl_sync(full, nc, l);
            first = base + __shfl_sync(full, incl, l) - nck;
            return;
        }
        base += __shfl_sync(full, incl, 31);
    }
}

__device__ __forceinline__ int load_slot(const int32_t* slots, int s) { return slots ? __ldg(slots + s) : -1; }

// ---------------------------------------------------------------------------------------------------
// Per-channel running computation shared by chunk_state (kOut = false) and chunk_scan (kOut = true).
template <typename AT, bool kPow, bool kOut>
struct ChannelScan {
    float h[kN];
    float a2[kN];      // general A: A[d][n] * log2(e);   powers: only a2[0] is used
    float w[kW];
    float win[kW - 1]; // previous raw inputs, oldest first
    float cb, dtb, dsk, sum_delta;
    uint32_t flags;

    __device__ __forceinline__ void init(const LayerDev& L, int d) {
#pragma unroll
        for (int n = 0; n < kN; ++n) a2[n] = __ldg(L.A + (size_t)d * kN + n) * kLog2e;
#pragma unroll
        for (int k = 0; k < kW; ++k) w[k] = __ldg(L.conv_w + (size_t)d * kW + k);
        cb = L.conv_b ? __ldg(L.conv_b + d) : 0.0f;
        dtb = L.dt_bias ? __ldg(L.dt_bias + d) : 0.0f;
        dsk = L.D ? __ldg(L.D + d) : 0.0f;
        sum_delta = 0.0f;
        flags = L.flags;
    }

    // One token.  Bt / Ct point at 16 fp32 values in shared memory.  Returns out (kOut) or is unused.
    __device__ __forceinline__ float token(float xv, float zv, float dtv, const float* Bt, const float* Ct) {
        float u;
        if (flags & MDRAFT_PRECONV) {
            u = xv;
        } else {
            float acc = cb;
            acc = fmaf(w[0], win[0], acc);
            acc = fmaf(w[1], win[1], acc);
            acc = fmaf(w[2], win[2], acc);
            acc = fmaf(w[3], xv, acc);
            win[0] = win[1]; win[1] = win[2]; win[2] = xv;
            u = silu(acc);
        }
        if (flags & MDRAFT_CONV_ONLY) return u;
        float v = dtv + dtb;
        float delta = (flags & MDRAFT_DT_SOFTPLUS) ? softplus(v) : v;
        sum_delta += delta;
        float du = delta * u;
        float dA[kN];
        if (kPow) {
            float r1 = ex2(delta * a2[0]);
            float r2 = r1 * r1, r4 = r2 * r2, r8 = r4 * r4;
            dA[0] = r1; dA[1] = r2; dA[2] = r2 * r1; dA[3] = r4;
            dA[4] = r4 * r1; dA[5] = r4 * r2; dA[6] = r4 * dA[2]; dA[7] = r8;
#pragma unroll
            for (int n = 0; n < 8; ++n) dA[8 + n] = r8 * dA[n];
        } else {
#pragma unroll
            for (int n = 0; n < kN; ++n) dA[n] = ex2(delta * a2[n]);
        }
        float y0 = 0.0f, y1 = 0.0f;
#pragma unroll
        for (int q = 0; q < kN / 4; ++q) {
            float4 b4 = *reinterpret_cast<const float4*>(Bt + 4 * q);
            float bb[4] = {b4.x, b4.y, b4.z, b4.w};
            float cc[4] = {0.f, 0.f, 0.f, 0.f};
            if (kOut) {
                float4 c4 = *reinterpret_cast<const float4*>(Ct + 4 * q);
                cc[0] = c4.x; cc[1] = c4.y; cc[2] = c4.z; cc[3] = c4.w;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int n = 4 * q + j;
                h[n] = fmaf(dA[n], h[n], du * bb[j]);
                if (kOut) {
                    if (j & 1) y1 = fmaf(cc[j], h[n], y1); else y0 = fmaf(cc[j], h[n], y0);
                }
            }
        }
        if (!kOut) return 0.0f;
        float y = fmaf(dsk, u, y0 + y1);
        return y * silu(zv);
    }
};

template <typename AT>
__device__ __forceinline__ void stage_bc(float (*sB)[kN], float (*sC)[kN], const AT* B, const AT* C, int64_t ldb, int64_t ldc,
                                         int t, int rows, bool want_c) {
    for (int i = threadIdx.x; i < rows * kN; i += blockDim.x) {
        int r = i / kN, n = i % kN;
        sB[r][n] = Act<AT>::load(B + (size_t)(t + r) * ldb + n);
        if (want_c) sC[r][n] = Act<AT>::load(C + (size_t)(t + r) * ldc + n);
    }
}

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

// ---------------------------------------------------------------------------------------------------
template <typename AT, bool kPow>
__global__ void __launch_bounds__(kPrefillThreads) chunk_state_kernel(PrefillArgs p) {
    __shared__ __align__(16) float sB[kTT][kN];
    const int D = p.L.d_inner;
    const int d = blockIdx.x * blockDim.x + threadIdx.x;
    const bool live = d < D;
    const int cidx = blockIdx.y;
    ChunkInfo ci = find_chunk(p.cu, p.n_seq, p.T, p.chunk_len, cidx);
    if (ci.seq < 0 || ci.k == ci.nck - 1) return;  // the last chunk's summary is never used

    const AT* x = static_cast<const AT*>(p.x);
    const AT* dt = static_cast<const AT*>(p.dt);
    const AT* B = static_cast<const AT*>(p.B);

    ChannelScan<AT, kPow, false> cs;
    if (live) {
        cs.init(p.L, d);
        const AT* rows = nullptr;
        if (ci.k == 0) {
            int slot = load_slot(p.init_slot, ci.seq);
            if (slot >= 0 && slot < p.pool.n_slots) rows = static_cast<const AT*>(p.pool.conv) + (size_t)slot * p.pool.conv_slot_stride;
        }
        load_window<AT>(cs.win, x, p.ldx, d, ci.t0, ci.k, rows, D);
        if (ci.k == 0) {  // keep the sequence's starting window where chunk_scan can read it even if the slot is overwritten
            AT* stash = static_cast<AT*>(p.ws_conv) + (size_t)ci.seq * (kW - 1) * D;
#pragma unroll
            for (int j = 0; j < kW - 1; ++j) stash[(size_t)j * D + d] = Act<AT>::from_f32(cs.win[j]);
        }
#pragma unroll
        for (int n = 0; n < kN; ++n) cs.h[n] = 0.0f;
    }
    if (p.L.flags & MDRAFT_CONV_ONLY) return;  // no recurrence: the stash was all this kernel had to do
    for (int t = ci.t0; t < ci.t1; t += kTT) {
        int rows = min(kTT, ci.t1 - t);
        __syncthreads();
        stage_bc<AT>(sB, sB, B, B, p.ldb, p.ldb, t, rows, false);
        __syncthreads();
        if (live) {
#pragma unroll 4
            for (int r = 0; r < rows; ++r) {
                float xv = Act<AT>::load(x + (size_t)(t + r) * p.ldx + d);
                float dtv = Act<AT>::load(dt + (size_t)(t + r) * p.lddt + d);
                cs.token(xv, 0.0f, dtv, sB[r], sB[r]);
            }
        }
    }
    if (live) {
        float4* dst = reinterpret_cast<float4*>(p.ws_h + ((size_t)cidx * D + d) * kN);
#pragma unroll
        for (int q = 0; q < kN / 4; ++q) dst[q] = make_float4(cs.h[4 * q], cs.h[4 * q + 1], cs.h[4 * q + 2], cs.h[4 * q + 3]);
        p.ws_sd[(size_t)cidx * D + d] = cs.sum_delta;
    }
}

// ---------------------------------------------------------------------------------------------------
// Block = 32 warps.  Tile = 32 consecutive (d, n) elements x 32 consecutive chunks of one sequence.
// Load: warp j reads chunk j's 32 elements (one 128-byte line).  Scan: warp j owns element j, lanes = chunks,
// Hillis-Steele inclusive scan of (P, q) under (P2,q2)o(P1,q1) = (P1*P2, P2*q1 + q2).  The incoming state of
// chunk k+1 is stored where chunk k's summary was.
__global__ void __launch_bounds__(1024) carry_scan_kernel(PrefillArgs p) {
    __shared__ float sP[32][33];
    __shared__ float sQ[32][33];
    __shared__ float carry[32];
    const unsigned full = 0xffffffffu;
    const int D = p.L.d_inner;
    const int E = D * kN;
    const int lane = threadIdx.x & 31, wj = threadIdx.x >> 5;
    const int e0 = blockIdx.x * 32;
    const int s = blockIdx.y;
    int first, nck;
    seq_chunks(p.cu, p.n_seq, p.T, p.chunk_len, s, first, nck);
    if (nck <= 1) return;

    if (wj == 0) {
        int e = e0 + lane;
        float h0 = 0.0f;
        int slot = load_slot(p.init_slot, s);
        if (e < E && slot >= 0 && slot < p.pool.n_slots) h0 = p.pool.ssm[(size_t)slot * p.pool.ssm_slot_stride + e];
        carry[lane] = h0;
    }
    const int n_sum = nck - 1;  // summaries of chunks 0 .. nck-2
    for (int b0 = 0; b0 < n_sum; b0 += 32) {
        __syncthreads();
        {
            int k = b0 + wj, e = e0 + lane;
            float P = 1.0f, q = 0.0f;
            if (k < n_sum && e < E) {
                size_t c = (size_t)(first + k);
                q = p.ws_h[c * E + e];
                float sd = p.ws_sd[c * D + e / kN];
                P = ex2(__ldg(p.L.A + e) * kLog2e * sd);
            }
            sP[wj][lane] = P;
            sQ[wj][lane] = q;
        }
        __syncthreads();
        {
            float P = sP[lane][wj], q = sQ[lane][wj];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                float Pp = __shfl_up_sync(full, P, o);
                float qp = __shfl_up_sync(full, q, o);
                if (lane >= o) { q = fmaf(P, qp, q); P = P * Pp; }
            }
            float hin = fmaf(P, carry[wj], q);  // state after chunk b0+lane = incoming state of chunk b0+lane+1
            sQ[lane][wj] = hin;
            __syncwarp();
            if (lane == 31) carry[wj] = hin;
        }
        __syncthreads();
        {
            int k = b0 + wj, e = e0 + lane;
            if (k < n_sum && e < E) p.ws_h[(size_t)(first + k) * E + e] = sQ[wj][lane];
        }
    }
}

// ---------------------------------------------------------------------------------------------------
template <typename AT, bool kPow>
__global__ void __launch_bounds__(kPrefillThreads) chunk_scan_kernel(PrefillArgs p) {
    __shared__ __align__(16) float sB[kTT][kN];
    __shared__ __align__(16) float sC[kTT][kN];
    const int D = p.L.d_inner;
    const int d = blockIdx.x * blockDim.x + threadIdx.x;
    const bool live = d < D;
    const int cidx = blockIdx.y;

    // Sequences without tokens have no chunk: their final state is their starting state.
    if (cidx == 0 && p.final_slot) {
        for (int s = 0; s < p.n_seq; ++s) {
            int lo = __ldg(p.cu + s), hi = __ldg(p.cu + s + 1);
            bool bad = (lo < 0) || (hi < lo) || (hi > p.T);
            if (bad && blockIdx.x == 0 && threadIdx.x == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SEQLENS);
            if (bad || hi != lo) continue;
            int fs = __ldg(p.final_slot + s), is = load_slot(p.init_slot, s);
            if (fs < 0 || fs == is) continue;
            if (fs >= p.pool.n_slots || is >= p.pool.n_slots) {
                if (blockIdx.x == 0 && threadIdx.x == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
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
    } else if (cidx == 0 && blockIdx.x == 0 && threadIdx.x < 32) {
        for (int s = threadIdx.x; s < p.n_seq; s += 32) {
            int lo = __ldg(p.cu + s), hi = __ldg(p.cu + s + 1);
            if ((lo < 0) || (hi < lo) || (hi > p.T)) flag(p.dev_status, MDRAFT_DEV_BAD_SEQLENS);
        }
    }

    ChunkInfo ci = find_chunk(p.cu, p.n_seq, p.T, p.chunk_len, cidx);
    if (ci.seq < 0) return;

    const AT* x = static_cast<const AT*>(p.x);
    const AT* z = static_cast<const AT*>(p.z);
    const AT* dt = static_cast<const AT*>(p.dt);
    const AT* B = static_cast<const AT*>(p.B);
    const AT* C = static_cast<const AT*>(p.C);
    AT* out = static_cast<AT*>(p.out);

    int islot = load_slot(p.init_slot, ci.seq);
    int fslot = load_slot(p.final_slot, ci.seq);
    if (islot >= p.pool.n_slots || fslot >= p.pool.n_slots) {  // whole sequence becomes a no-op
        if (threadIdx.x == 0 && blockIdx.x == 0 && ci.k == 0) flag(p.dev_status, MDRAFT_DEV_BAD_SLOT);
        return;
    }

    ChannelScan<AT, kPow, true> cs;
    if (live) {
        cs.init(p.L, d);
        const AT* rows = nullptr;
        if (ci.k == 0) {
            if (ci.nck > 1 && !(p.L.flags & MDRAFT_PRECONV)) rows = static_cast<const AT*>(p.ws_conv) + (size_t)ci.seq * (kW - 1) * D;
            else if (islot >= 0) rows = static_cast<const AT*>(p.pool.conv) + (size_t)islot * p.pool.conv_slot_stride;
        }
        load_window<AT>(cs.win, x, p.ldx, d, ci.t0, ci.k, rows, D);
        const float* hsrc = nullptr;
        if (ci.k > 0) hsrc = p.ws_h + ((size_t)(cidx - 1) * D + d) * kN;
        else if (islot >= 0) hsrc = p.pool.ssm + (size_t)islot * p.pool.ssm_slot_stride + (size_t)d * kN;
#pragma unroll
        for (int q = 0; q < kN / 4; ++q) {
            float4 v = hsrc ? *reinterpret_cast<const float4*>(hsrc + 4 * q) : make_float4(0.f, 0.f, 0.f, 0.f);
            cs.h[4 * q] = v.x; cs.h[4 * q + 1] = v.y; cs.h[4 * q + 2] = v.z; cs.h[4 * q + 3] = v.w;
        }
    }
    const bool conv_only = p.L.flags & MDRAFT_CONV_ONLY;
    for (int t = ci.t0; t < ci.t1; t += kTT) {
        int rows = min(kTT, ci.t1 - t);
        __syncthreads();
        if (!conv_only) stage_bc<AT>(sB, sC, B, C, p.ldb, p.ldc, t, rows, true);
        __syncthreads();
        if (live) {
#pragma unroll 4
            for (int r = 0; r < rows; ++r) {
                float xv = Act<AT>::load(x + (size_t)(t + r) * p.ldx + d);
                float zv = conv_only ? 0.0f : Act<AT>::load(z + (size_t)(t + r) * p.ldz + d);
                float dtv = conv_only ? 0.0f : Act<AT>::load(dt + (size_t)(t + r) * p.lddt + d);
                float o = cs.token(xv, zv, dtv, sB[r], sC[r]);
                out[(size_t)(t + r) * p.ldo + d] = Act<AT>::from_f32(o);
            }
        }
    }
    if (live && ci.k == ci.nck - 1 && fslot >= 0) {
        if (!conv_only) {
            float4* dst = reinterpret_cast<float4*>(p.pool.ssm + (size_t)fslot * p.pool.ssm_slot_stride + (size_t)d * kN);
#pragma unroll
            for (int q = 0; q < kN / 4; ++q) dst[q] = make_float4(cs.h[4 * q], cs.h[4 * q + 1], cs.h[4 * q + 2], cs.h[4 * q + 3]);
        }
        if (!(p.L.flags & MDRAFT_PRECONV)) {
            AT* dc = static_cast<AT*>(p.pool.conv) + (size_t)fslot * p.pool.conv_slot_stride;
#pragma unroll
            for (int j = 0; j < kW - 1; ++j) dc[(size_t)j * D + d] = Act<AT>::from_f32(cs.win[j]);
        }
    }
}

template <typename AT, bool kPow>
cudaError_t launch_typed(const PrefillArgs& p, bool chunked, cudaStream_t st) {
    const int D = p.L.d_inner;
    dim3 grid((D + kPrefillThreads - 1) / kPrefillThreads, p.n_chunks_bound);
    const bool recur = !(p.L.flags & MDRAFT_CONV_ONLY);
    if (chunked) {
        chunk_state_kernel<AT, kPow><<<grid, kPrefillThreads, 0, st>>>(p);
        if (p.ev_state) cudaEventRecord(p.ev_state, st);
        if (recur) {
            dim3 g2((D * kN + 31) / 32, p.n_seq);
            carry_scan_kernel<<<g2, 1024, 0, st>>>(p);
        }
        if (p.ev_carry) cudaEventRecord(p.ev_carry, st);
    } else {
        if (p.ev_state) cudaEventRecord(p.ev_state, st);
        if (p.ev_carry) cudaEventRecord(p.ev_carry, st);
    }
    chunk_scan_kernel<AT, kPow><<<grid, kPrefillThreads, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prefill(const PrefillArgs& p, int act, bool chunked, cudaStream_t st) {
    const bool pow = p.L.flags & MDRAFT_A_POWERS;
    if (act == MDRAFT_F32) return pow ? launch_typed<float, true>(p, chunked, st) : launch_typed<float, false>(p, chunked, st);
    return pow ? launch_typed<__nv_bfloat16, true>(p, chunked, st) : launch_typed<__nv_bfloat16, false>(p, chunked, st);
}

}  // namespace mdraft
