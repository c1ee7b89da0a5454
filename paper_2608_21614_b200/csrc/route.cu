// Top-k gating (Background, "Mixture-of-Experts Inference": the router selects the top-k experts
// per token).  One warp per token; each lane keeps up to four logits in registers (experts lane,
// lane+32, ...); k rounds of a warp-wide arg-max by shuffles on a packed 64-bit key whose high
// word orders the logit and whose low word prefers the lower expert id; softmax over the k
// winners in registers.
#include "route_row.cuh"

namespace saem {

constexpr int kRouteWarps = 4;

__global__ void __launch_bounds__(kRouteWarps * 32)
route_kernel(const float* __restrict__ logits, int T, int E, int k, int renorm, int32_t* __restrict__ idx,
             float* __restrict__ w) {
    pdl_wait();
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * kRouteWarps + (threadIdx.x >> 5);
    if (t >= T) return;
    route_row(logits + (size_t)t * E, E, k, renorm, lane, idx + (size_t)t * k, w + (size_t)t * k);
}

// Router projection fused with the gate: one CTA per token computes logits[e] = <x_t, W_r[e]> in
// fp32 (16-byte loads of bf16, one warp per expert in turn, warp-shuffle reduction), keeps the
// row in shared memory and lets warp 0 run the same top-k / softmax.  Saves a launch and the
// logits' round trip through HBM on the latency-bound decode shapes.
constexpr int kRouterWarps = 8;

__global__ void __launch_bounds__(kRouterWarps * 32)
route_fused_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ w_router, int T, int E, int d, int k,
                   int renorm, float* __restrict__ logits_out, int32_t* __restrict__ idx, float* __restrict__ w) {
    __shared__ float row[SAEM_MAX_EXPERTS];
    pdl_wait();
    pdl_launch_dependents();
    const int t = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)t * d);
    for (int e = warp; e < E; e += kRouterWarps) {
        const uint4* wr = reinterpret_cast<const uint4*>(w_router + (size_t)e * d);
        float acc = 0.f;
        for (int c = lane; c < d / 8; c += 32) {
            const uint4 a = xr[c], b = wr[c];
            const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                acc = fmaf(__uint_as_float(av[q] << 16), __uint_as_float(bv[q] << 16), acc);
                acc = fmaf(__uint_as_float(av[q] & 0xFFFF0000u), __uint_as_float(bv[q] & 0xFFFF0000u), acc);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) {
            row[e] = acc;
            if (logits_out) logits_out[(size_t)t * E + e] = acc;
        }
    }
    __syncthreads();
    if (warp == 0) route_row(row, E, k, renorm, lane, idx + (size_t)t * k, w + (size_t)t * k);
}

cudaError_t launch_route(const float* logits, int T, int E, int k, int renorm, int32_t* idx, float* w,
                         cudaStream_t st) {
    int blocks = (T + kRouteWarps - 1) / kRouteWarps;
    return launch_pdl(route_kernel, dim3(blocks), dim3(kRouteWarps * 32), 0, st, logits, T, E, k, renorm, idx, w);
}

}  // namespace saem

namespace saem {
cudaError_t launch_route_fused(const uint16_t* x, const uint16_t* w_router, int T, int E, int d, int k, int renorm,
                               float* logits_out, int32_t* idx, float* w, cudaStream_t st) {
    return launch_pdl(route_fused_kernel, dim3(T), dim3(kRouterWarps * 32), 0, st, x, w_router, T, E, d, k, renorm,
                      logits_out, idx, w);
}
}  // namespace saem
