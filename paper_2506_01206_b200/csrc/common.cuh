// Shared device helpers for the mdraft kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mdraft.h"

namespace mdraft {

constexpr int kN = 16;            // d_state handled by these kernels
constexpr int kW = 4;             // d_conv handled by these kernels
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Every wait on an mbarrier polls at most this often before the block gives up, raises MDRAFT_DEV_WAIT_EXPIRED
// and returns.  One poll is a try_wait that may suspend the thread for at most kPollNs nanoseconds (a stated limit
// instead of the system's own), so a wait that never completes ends after about a second.  The two macros exist for the failure-path tests only: a second build of the library with a short
// limit and with every copy barrier told to expect a few bytes more than will ever arrive, so that each bounded
// wait runs out (the copies themselves still land) and the give-up paths execute on a healthy GPU.
#ifndef MDRAFT_SPIN_LIMIT
#define MDRAFT_SPIN_LIMIT (1u << 20)
#endif
#ifndef MDRAFT_TEST_OVERSTATE_TX
#define MDRAFT_TEST_OVERSTATE_TX 0u
#endif
constexpr uint32_t kSpinLimit = MDRAFT_SPIN_LIMIT;
constexpr uint32_t kOverstateTx = MDRAFT_TEST_OVERSTATE_TX;
constexpr uint32_t kPollNs = 1000u;

// ---------------------------------------------------------------- scalar math
__device__ __forceinline__ float ex2(float v) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ float lg2(float v) {
    float r;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ float rcp(float v) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}

// SiLU(v) = v / (1 + exp(-v)).  exp(-v) overflows to +inf for v < -88 and the quotient is then -0.
__device__ __forceinline__ float silu(float v) { return v * rcp(1.0f + ex2(-kLog2e * v)); }

// softplus(v) = log(1 + exp(v)).  For small e = exp(v) the series e - e^2/2 + e^3/3 - e^4/4 avoids the
// cancellation in 1 + e; for large v the result is v itself.
__device__ __forceinline__ float softplus(float v) {
    float e = ex2(kLog2e * v);
    float series = e * (1.0f - e * (0.5f - e * (0.33333334f - 0.25f * e)));
    float full = kLn2 * lg2(1.0f + e);
    float r = (e < 0.03125f) ? series : full;
    return (v > 20.0f) ? v : r;
}

// ---------------------------------------------------------------- activation dtype
template <typename T> struct Act;
template <> struct Act<float> {
    static constexpr int kDtype = MDRAFT_F32;
    __device__ static __forceinline__ float load(const float* p) { return __ldg(p); }
    __device__ static __forceinline__ float to_f32(float v) { return v; }
    __device__ static __forceinline__ float from_f32(float v) { return v; }
};
template <> struct Act<__nv_bfloat16> {
    static constexpr int kDtype = MDRAFT_BF16;
    __device__ static __forceinline__ float load(const __nv_bfloat16* p) {
        return __uint_as_float(((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
    }
    __device__ static __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
    __device__ static __forceinline__ __nv_bfloat16 from_f32(float v) { return __float2bfloat16_rn(v); }
};

// Per-layer constants as the kernels take them (by value).
struct LayerDev {
    const float* A;
    const float* D;
    const float* conv_w;
    const float* conv_b;
    const float* dt_bias;
    int d_inner;
    uint32_t flags;
};

// One layer's view of the state pool.
struct PoolDev {
    float* ssm;            // slot s: ssm + s * ssm_slot_stride, (D, N) fp32
    void* conv;            // slot s: conv + s * conv_slot_stride elements, (W-1, D) activations
    int64_t ssm_slot_stride;
    int64_t conv_slot_stride;
    int n_slots;
};

__device__ __forceinline__ void flag(int32_t* dev_status, int bit) {
    if (dev_status) atomicOr(dev_status, bit);
}

}  // namespace mdraft
