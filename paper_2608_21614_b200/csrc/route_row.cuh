// The gate of one token, shared by the routing kernels and the fused decode kernels: one warp routes
// one token (Background, "Mixture-of-Experts Inference": the router selects the top-k experts).
// Each lane keeps up to four logits in registers (experts lane, lane+32, ...); k rounds of a
// warp-wide arg-max by shuffles on a packed 64-bit key whose high word orders the logit and whose
// low word prefers the lower expert id; softmax over the k winners in registers.
#ifndef SAEM_ROUTE_ROW_CUH_
#define SAEM_ROUTE_ROW_CUH_

#include <math_constants.h>

#include "saem_internal.h"

namespace saem {

constexpr int kPerLane = SAEM_MAX_EXPERTS / 32;

// Order-preserving map float -> uint32: larger float <=> larger key.  NaN -> key of -inf,
// -0 -> key of +0 so that the two zeros tie.
__device__ __forceinline__ uint32_t order_key(float v) {
    if (v != v) v = -CUDART_INF_F;
    if (v == 0.0f) v = 0.0f;
    uint32_t b = __float_as_uint(v);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_value(uint32_t k) {
    uint32_t b = (k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k;
    return __uint_as_float(b);
}

// One warp routes one token: `row` holds the token's E logits (global or shared memory).
__device__ __forceinline__ void route_row(const float* __restrict__ row, int E, int k, int renorm, int lane,
                                          int32_t* __restrict__ idx_out, float* __restrict__ w_out) {
    unsigned long long key[kPerLane];
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
        int e = lane + 32 * i;
        key[i] = 0ull;                                    // below every real key (a real key's high word is never 0)
        if (e < E) key[i] = ((unsigned long long)order_key(row[e]) << 32) | (uint32_t)(~(uint32_t)e);
    }

    // winners: slot j lives in lane j & 31, register j >> 5
    float win_v[kPerLane];
    float denom_all = 0.f;
    float vmax = 0.f;
    for (int j = 0; j < k; ++j) {
        unsigned long long best = key[0];
#pragma unroll
        for (int i = 1; i < kPerLane; ++i) best = key[i] > best ? key[i] : best;
        // warp-wide maximum of the 64-bit key in two 32-bit reductions: the largest value word, then
        // the largest ~id (the lowest expert id) among the lanes that hold that value
        const uint32_t hi = (uint32_t)(best >> 32);
        const uint32_t hi_max = __reduce_max_sync(0xffffffffu, hi);
        const uint32_t lo_max = __reduce_max_sync(0xffffffffu, hi == hi_max ? (uint32_t)best : 0u);
        best = ((unsigned long long)hi_max << 32) | lo_max;
        int e = (int)(~(uint32_t)best);
        float v = key_value((uint32_t)(best >> 32));
        if (j == 0) {
            vmax = v;
            if (!renorm) {                                // denominator over all experts, before any key is cleared
                float s = 0.f;
#pragma unroll
                for (int i = 0; i < kPerLane; ++i)
                    if (lane + 32 * i < E) s += expf(key_value((uint32_t)(key[i] >> 32)) - vmax);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                denom_all = s;
            }
        }
#pragma unroll
        for (int i = 0; i < kPerLane; ++i)
            if (lane + 32 * i == e) key[i] = 0ull;        // taken
        if (lane == 0) idx_out[j] = e;
#pragma unroll
        for (int i = 0; i < kPerLane; ++i)
            if ((j >> 5) == i && (j & 31) == lane) win_v[i] = v;
    }

    // softmax over the winners
    float z[kPerLane];
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
        int j = lane + 32 * i;
        z[i] = 0.f;
        if (j < k) {
            if (vmax == CUDART_INF_F) {
                z[i] = (win_v[i] == CUDART_INF_F) ? 1.f : 0.f;
            } else if (vmax == -CUDART_INF_F) {
                z[i] = 1.f;
            } else {
                z[i] = expf(win_v[i] - vmax);
            }
            s += z[i];
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    float denom = s;
    if (!renorm && vmax != CUDART_INF_F && vmax != -CUDART_INF_F) denom = denom_all;
#pragma unroll
    for (int i = 0; i < kPerLane; ++i) {
        int j = lane + 32 * i;
        if (j < k) w_out[j] = z[i] / denom;
    }
}

}  // namespace saem

#endif  // SAEM_ROUTE_ROW_CUH_
