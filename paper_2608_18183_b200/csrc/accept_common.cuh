// Small device helpers shared by the verification kernels (probability pipeline, accept test, sampling).
#pragma once
#include "common.cuh"

namespace hbsjd {

// Codes written to counters[CNT_ERROR] when a kernel meets rollout state that cannot be valid (the access is
// skipped and the draft treated as rejected, so nothing faults).  Codes below 16 are bounded-wait time-outs.
enum { ERR_BAD_CURSOR = 16, ERR_BAD_TOKEN = 17, ERR_BAD_PROPOSAL_ROW = 18 };

// Monotone map of a float to an unsigned key (larger float, larger key).
__device__ __forceinline__ unsigned int float_key(float x) {
    const unsigned int u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_float(unsigned int k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// Fixed-point weight of the categorical sampler: floor(a * 2^30).
__device__ __forceinline__ unsigned int fixed_weight(float a) { return __float2uint_rd(a * 1073741824.0f); }

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Selection histogram of the exact top-k threshold: bins, and the capacity of the candidate list of one bin.
constexpr int SEL_BINS = 1024;
constexpr int SEL_CAP = 1536;

// A value below the k-th largest of V entries with the given mean and standard deviation, from a normal fit:
// the upper-tail quantile of (1.5 k + 16) / V by the rational approximation of Abramowitz & Stegun 26.2.23.
// Only a guess: the selection verifies it by counting and falls back to the whole range.
__device__ __forceinline__ float topk_guess(float mean, float sd, int top_k, int V) {
    const float f = fminf(0.5f, (1.5f * (float)top_k + 16.f) / (float)V);
    const float tq = sqrtf(-2.0f * __logf(f));
    const float zq = tq - (2.515517f + tq * (0.802853f + tq * 0.010328f)) /
                              (1.0f + tq * (1.432788f + tq * (0.189269f + tq * 0.001308f)));
    return mean + zq * sd;
}

}  // namespace hbsjd
