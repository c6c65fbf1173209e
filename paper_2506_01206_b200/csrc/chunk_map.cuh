// Which tokens a chunk of a packed batch covers (shared by the S6 and the SSD context-encode kernels).
#pragma once

#include <stdint.h>

namespace mdraft {

// ---------------------------------------------------------------- chunk bookkeeping
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
    if (!cu) {  // no offsets given: one sequence that is all T rows (nothing to look up in memory)
        if (s == 0) len = T;
        return;
    }
    if (s < n_seq) {
        int lo = __ldg(cu + s), hi = __ldg(cu + s + 1);
        bad = (lo < 0) || (hi < lo) || (hi > T);
        if (!bad) { a = lo; len = hi - lo; }
    }
}

__device__ inline ChunkInfo find_chunk(const int32_t* cu, int n_seq, int T, int Lc, int cidx) {
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
__device__ inline void seq_chunks(const int32_t* cu, int n_seq, int T, int Lc, int s, int& first, int& nck) {
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

}  // namespace mdraft
