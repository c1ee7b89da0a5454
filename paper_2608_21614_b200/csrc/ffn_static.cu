// saem_expert_ffn_static: the grouped SwiGLU expert FFN for callers that cannot allocate device
// memory -- code running where cudaMalloc is forbidden or unavailable (a plugin inside a host
// application that owns the memory pool, a real-time loop, a process whose pool is exhausted).
// The only scratch the FFN needs, the hidden activations h[rows, d_ff], lives in a file-scope
// device array of fixed size instead of a caller-provided workspace; the function needs no
// context object (creating one allocates pinned memory and events).
//
// Host code must not hand the array's name to a kernel: on the host that name is only a stand-in,
// not a device address.  The address is obtained once per device with cudaGetSymbolAddress while
// that device is current, and passed to the kernels as an ordinary pointer.
#include <cuda_bf16.h>
#include <mutex>

#include "saem_internal.h"

namespace saem {

// 1 Mi bf16 elements = 2 MiB, held by every GPU that loads the library until the process exits.
static __device__ __align__(256) uint16_t g_static_h[SAEM_STATIC_SCRATCH_ELEMS];

constexpr int kStaticMaxDevices = 64;
static uint16_t* g_static_h_ptr[kStaticMaxDevices];
static bool g_static_ready[kStaticMaxDevices];
static std::mutex g_static_mutex;

// Device address of the scratch array on the current device (set up on the first call there).
static cudaError_t static_scratch(uint16_t** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kStaticMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ready[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_h);
        if (e != cudaSuccess) return e;
        g_static_h_ptr[dev] = (uint16_t*)p;
        g_static_ready[dev] = true;
    }
    *out = g_static_h_ptr[dev];
    return cudaSuccess;
}

__device__ __forceinline__ void widen8(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

// One thread per weight row of a 128-row tile of the packed slot layout, four packed rows of
// activations at a time.  PHASE 0: h = silu(Wg x) * (Wu x);  PHASE 1: y = Wd h.
template <int PHASE>
__global__ void __launch_bounds__(kTileRows)
ffn_static_kernel(const uint16_t* __restrict__ x_packed, const int32_t* __restrict__ offsets, int max_rows, int d,
                  int f, const uint8_t* __restrict__ experts, uint16_t* __restrict__ h, float* __restrict__ y) {
    constexpr int R = 4;
    const int rb = blockIdx.x, e = blockIdx.y, i = threadIdx.x;
    int r0 = offsets[e], r1 = offsets[e + 1];
    if (r1 > max_rows) r1 = max_rows;
    if (r1 <= r0) return;
    const int K = PHASE == 0 ? d : f, KC = K / kTileK;
    const uint8_t* slot = experts + (size_t)e * 3 * d * f * 2;
    const uint8_t* base = PHASE == 0 ? slot : slot + (size_t)2 * d * f * 2;
    const size_t chunk = PHASE == 0 ? 2 * kTileBytes : kTileBytes;
    const uint16_t* act = PHASE == 0 ? x_packed : h;
    for (int row = r0; row < r1; row += R) {
        const int nr = min(R, r1 - row);
        float a0[R], a1[R];
#pragma unroll
        for (int n = 0; n < R; ++n) a0[n] = a1[n] = 0.f;
        for (int kc = 0; kc < KC; ++kc) {
            const uint8_t* tile = base + ((size_t)rb * KC + kc) * chunk;
            for (int ch = 0; ch < 8; ++ch) {
                const int pos = i * 128 + ((ch ^ (i & 7)) << 4);
                float w0[8], w1[8];
                widen8(*reinterpret_cast<const uint4*>(tile + pos), w0);
                if (PHASE == 0) widen8(*reinterpret_cast<const uint4*>(tile + kTileBytes + pos), w1);
#pragma unroll
                for (int n = 0; n < R; ++n) {
                    if (n < nr) {
                        float xv[8];
                        widen8(*reinterpret_cast<const uint4*>(act + (size_t)(row + n) * K + kc * kTileK + ch * 8), xv);
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            a0[n] = fmaf(w0[q], xv[q], a0[n]);
                            if (PHASE == 0) a1[n] = fmaf(w1[q], xv[q], a1[n]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int n = 0; n < R; ++n) {
            if (n < nr) {
                if (PHASE == 0) {
                    const float hv = a0[n] / (1.f + expf(-a0[n])) * a1[n];
                    reinterpret_cast<__nv_bfloat16*>(h)[(size_t)(row + n) * f + rb * kTileRows + i] = __float2bfloat16_rn(hv);
                } else {
                    y[(size_t)(row + n) * d + rb * kTileRows + i] = a0[n];
                }
            }
        }
    }
}

}  // namespace saem

extern "C" int saem_expert_ffn_static(const void* x_packed, const int32_t* offsets, int n_experts, int max_rows,
                                      int d_model, int d_ff, const void* packed_experts, float* y_packed,
                                      void* stream) {
    using namespace saem;
    if (!x_packed || !offsets || !packed_experts || !y_packed) return SAEM_ERR_INVALID_ARG;
    if (n_experts < 1 || n_experts > SAEM_MAX_EXPERTS || max_rows < 0) return SAEM_ERR_SHAPE;
    if (d_model <= 0 || d_ff <= 0 || d_model % 128 || d_ff % 128) return SAEM_ERR_SHAPE;
    if (((uintptr_t)x_packed | (uintptr_t)y_packed | (uintptr_t)packed_experts) & 15) return SAEM_ERR_ALIGNMENT;
    if ((long long)max_rows * d_ff > (long long)SAEM_STATIC_SCRATCH_ELEMS) return SAEM_ERR_WORKSPACE;
    if (max_rows == 0) return SAEM_OK;
    uint16_t* h = nullptr;
    if (static_scratch(&h) != cudaSuccess) return SAEM_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    // every h row that phase 1 reads is written by phase 0 of this same call: nothing needs clearing
    dim3 g0(d_ff / kTileRows, n_experts), g1(d_model / kTileRows, n_experts);
    ffn_static_kernel<0><<<g0, kTileRows, 0, st>>>((const uint16_t*)x_packed, offsets, max_rows, d_model, d_ff,
                                                   (const uint8_t*)packed_experts, h, y_packed);
    if (cudaGetLastError() != cudaSuccess) return SAEM_ERR_CUDA;
    ffn_static_kernel<1><<<g1, kTileRows, 0, st>>>((const uint16_t*)x_packed, offsets, max_rows, d_model, d_ff,
                                                   (const uint8_t*)packed_experts, h, y_packed);
    if (cudaGetLastError() != cudaSuccess) return SAEM_ERR_CUDA;
    return SAEM_OK;
}
