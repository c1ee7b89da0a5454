// Plain scalar (FMA) version of the grouped SwiGLU expert FFN over the repacked segments
// (Sec. IV-E: each expert runs once over its contiguous segment).  Kept for triage: it reads the
// same packed slot layout as the tensor-core kernels but uses no shared memory, no asynchronous
// copies and no tensor cores, so a disagreement between the two isolates the fast path.
// One thread per weight row of a 128-row tile; eight packed rows of activations at a time.
#include <cuda_bf16.h>

#include "saem_internal.h"

namespace saem {

constexpr int kRowsPerPass = 8;

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

__device__ __forceinline__ bool segment_of(const int32_t* offsets, int max_rows, int e, int& r0, int& r1) {
    if (offsets) { r0 = offsets[e]; r1 = offsets[e + 1]; } else { r0 = 0; r1 = max_rows; }
    if (r1 > max_rows) r1 = max_rows;
    return r1 > r0;
}

// phase 0: h = silu(Wg x) * (Wu x);  phase 1: y = Wd h
template <int PHASE>
__global__ void __launch_bounds__(kTileRows)
ffn_scalar_kernel(FfnArgs a, const __grid_constant__ SlotTable tab) {
    const int rb = blockIdx.x, e = blockIdx.y, i = threadIdx.x;
    int r0, r1;
    if (!tab.in_subset[e] || !segment_of(a.offsets, a.max_rows, e, r0, r1)) return;
    if (tab.slot[e] < 0) {
        if (rb == 0 && i == 0) atomicExch(a.status, SAEM_ERR_NOT_RESIDENT);
        return;
    }
    const int K = PHASE == 0 ? a.d : a.f;             // reduction length
    const int KC = K / kTileK;
    const uint8_t* slot = a.slot_region + (size_t)tab.slot[e] * a.slot_bytes;
    const uint8_t* base = PHASE == 0 ? slot : slot + (size_t)2 * a.d * a.f * 2;
    const size_t chunk_bytes = PHASE == 0 ? 2 * kTileBytes : kTileBytes;
    const uint16_t* act = PHASE == 0 ? a.x_packed : a.h;

    for (int row = r0; row < r1; row += kRowsPerPass) {
        const int nr = min(kRowsPerPass, r1 - row);
        float acc0[kRowsPerPass], acc1[kRowsPerPass];
#pragma unroll
        for (int n = 0; n < kRowsPerPass; ++n) acc0[n] = acc1[n] = 0.f;
        for (int kc = 0; kc < KC; ++kc) {
            const uint8_t* tile = base + ((size_t)rb * KC + kc) * chunk_bytes;
#pragma unroll 2
            for (int ch = 0; ch < 8; ++ch) {
                const int pos = i * 128 + ((ch ^ (i & 7)) << 4);
                float w0[8], w1[8];
                unpack8(*reinterpret_cast<const uint4*>(tile + pos), w0);
                if (PHASE == 0) unpack8(*reinterpret_cast<const uint4*>(tile + kTileBytes + pos), w1);
#pragma unroll
                for (int n = 0; n < kRowsPerPass; ++n) {
                    if (n < nr) {
                        float xv[8];
                        unpack8(*reinterpret_cast<const uint4*>(act + (size_t)(row + n) * K + kc * kTileK + ch * 8), xv);
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            acc0[n] = fmaf(w0[q], xv[q], acc0[n]);
                            if (PHASE == 0) acc1[n] = fmaf(w1[q], xv[q], acc1[n]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int n = 0; n < kRowsPerPass; ++n) {
            if (n < nr) {
                if (PHASE == 0) {
                    const float g = acc0[n];
                    const float hv = g / (1.f + expf(-g)) * acc1[n];
                    reinterpret_cast<__nv_bfloat16*>(a.h)[(size_t)(row + n) * a.f + rb * kTileRows + i] = __float2bfloat16_rn(hv);
                } else {
                    a.y_packed[(size_t)(row + n) * a.d + rb * kTileRows + i] = acc0[n];
                }
            }
        }
    }
}

cudaError_t launch_ffn_scalar(const FfnArgs& a, const SlotTable& tab, cudaStream_t st, int* n_launch) {
    dim3 g0(a.f / kTileRows, a.E), g1(a.d / kTileRows, a.E);
    ffn_scalar_kernel<0><<<g0, kTileRows, 0, st>>>(a, tab);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    ffn_scalar_kernel<1><<<g1, kTileRows, 0, st>>>(a, tab);
    *n_launch = 2;
    return cudaGetLastError();
}

}  // namespace saem
