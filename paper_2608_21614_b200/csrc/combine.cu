// Weighted merge of the expert outputs back to token order (Sec. IV-D, last paragraph: outputs
// are merged before the next layer).  Gather-based: each output element is produced by exactly
// one thread that sums its k contributions in slot order j = 0..k-1 and adds the shared-expert
// output last, so the result does not depend on scheduling (the atomic accumulation the paper's
// Sec. VI-D mentions as a source of run-to-run differences is avoided).
#include <cuda_bf16.h>

#include "saem_internal.h"

namespace saem {

__global__ void __launch_bounds__(256)
combine_kernel(const float* __restrict__ y, const int32_t* __restrict__ inv_perm, const float* __restrict__ w,
               int T, int k, int S, int d, const float* __restrict__ shared_y, void* __restrict__ out, int out_bf16) {
    pdl_wait();
    pdl_launch_dependents();
    const int vec_per_row = d >> 2;
    const long long total = (long long)T * vec_per_row;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int t = (int)(i / vec_per_row), c4 = (int)(i % vec_per_row);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j = 0; j < k; ++j) {
            const int r = inv_perm[(size_t)t * k + j];
            if (r < 0) continue;                       // pair dropped by repack (invalid expert id)
            const float wj = w[(size_t)t * k + j];
            const float4 v = *reinterpret_cast<const float4*>(y + (size_t)r * d + (size_t)c4 * 4);
            acc.x = fmaf(wj, v.x, acc.x);
            acc.y = fmaf(wj, v.y, acc.y);
            acc.z = fmaf(wj, v.z, acc.z);
            acc.w = fmaf(wj, v.w, acc.w);
        }
        for (int sh = 0; sh < S; ++sh) {               // in-layer shared experts: rows after the T*k pairs
            const float4 v = *reinterpret_cast<const float4*>(y + ((size_t)T * k + (size_t)sh * T + t) * d + (size_t)c4 * 4);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        if (shared_y) {
            const float4 s = *reinterpret_cast<const float4*>(shared_y + (size_t)t * d + (size_t)c4 * 4);
            acc.x += s.x; acc.y += s.y; acc.z += s.z; acc.w += s.w;
        }
        if (out_bf16) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&lo);
            pk.y = *reinterpret_cast<uint32_t*>(&hi);
            *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(out) + (size_t)t * d + (size_t)c4 * 4) = pk;
        } else {
            *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + (size_t)t * d + (size_t)c4 * 4) = acc;
        }
    }
}

cudaError_t launch_combine(const float* y, const int32_t* inv_perm, const float* w, int T, int k, int S, int d,
                           const float* shared_y, void* out, int out_bf16, cudaStream_t st) {
    long long total = (long long)T * (d / 4);
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    return launch_pdl(combine_kernel, dim3((unsigned)blocks), dim3(256), 0, st, y, inv_perm, w, T, k, S, d, shared_y, out,
                      out_bf16);
}

}  // namespace saem
