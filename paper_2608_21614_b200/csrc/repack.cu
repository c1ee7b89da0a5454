// Expert-aligned token repacking (Sec. IV-E): histogram of (token, slot) pairs per expert,
// exclusive scan, and a stable scatter into per-expert contiguous segments -- a counting sort
// that keeps ascending pair id inside a segment, so the permutation is unique and no atomics
// decide an order.  The row gather moves 16 bytes per thread per access.
//
// Index phase, one CTA: warps take consecutive 32-pair chunks; within a chunk __match_any_sync
// groups equal expert ids and a lane's rank is the number of lower lanes in its group; an
// [expert][chunk] table of 16-bit counts is scanned down the chunks by one warp per expert;
// a scan over the expert totals gives the segment offsets.
//
// Small problems (pairs <= kFusedPairs): every CTA of the grid repeats the index phase in its own
// shared memory (only CTA 0 writes the index outputs) and then copies its share of the rows, so
// the whole repack is one launch.  Larger problems: one index CTA, then a grid-wide gather.
#include "saem_internal.h"

namespace saem {

constexpr int kRepackThreads = 512;
constexpr int kFusedPairs = 2048;

struct RepackSmem {
    int counts[SAEM_MAX_EXPERTS];
    int offsets[SAEM_MAX_EXPERTS + 1];
    int bad;
};

// Shared-memory carve: [RepackSmem][chunk table uint16 n_chunks*E][rank uint8 P_padded][perm int32 P (fused only)]
__device__ __forceinline__ void index_phase(const int32_t* __restrict__ idx, int P, int E, int S, int T, RepackSmem& sm,
                                            uint16_t* table, uint8_t* rank, int32_t* perm_s, bool write_global,
                                            int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                                            int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
                                            int* __restrict__ status) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = blockDim.x >> 5;
    const int n_chunks = (P + 31) >> 5;
    // table[e * n_chunks + c]: pairs of chunk c routed to expert e (expert-major, so that the scan
    // down the chunks of one expert reads consecutive shared-memory words)
    for (int i = tid; i < n_chunks * E; i += blockDim.x) table[i] = 0;
    if (tid == 0) sm.bad = 0;
    __syncthreads();
    for (int c = warp; c < n_chunks; c += n_warps) {
        int p = c * 32 + lane;
        int e = p < P ? idx[p] : -1;
        if (p < P && (e < 0 || e >= E)) { e = -1; sm.bad = 1; }
        unsigned grp = __match_any_sync(0xffffffffu, e);
        int r = __popc(grp & ((1u << lane) - 1u));
        if (e >= 0) {
            rank[p] = (uint8_t)r;
            if (r == 0) table[e * n_chunks + c] = (uint16_t)__popc(grp);
        }
    }
    __syncthreads();
    // chunk counts -> exclusive running base per expert: one warp per expert, 32 chunks per step
    for (int e = warp; e < E; e += n_warps) {
        int run = 0;
        for (int c0 = 0; c0 < n_chunks; c0 += 32) {
            const int c = c0 + lane;
            const int v = c < n_chunks ? table[e * n_chunks + c] : 0;
            int inc = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += n;
            }
            if (c < n_chunks) table[e * n_chunks + c] = (uint16_t)(run + inc - v);
            run += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) sm.counts[e] = run;
    }
    __syncthreads();
    if (warp == 0) {                                 // exclusive scan over the expert totals
        int carry = 0;
        for (int base = 0; base < E; base += 32) {
            int e = base + lane;
            int v = e < E ? sm.counts[e] : 0;
            int inc = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int n = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += n;
            }
            if (e < E) sm.offsets[e] = carry + inc - v;
            carry += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) sm.offsets[E] = carry;
    }
    __syncthreads();
    if (write_global) {
        for (int e = tid; e < E; e += blockDim.x) counts[e] = sm.counts[e];
        for (int e = tid; e <= E; e += blockDim.x) offsets[e] = sm.offsets[e];
        // in-layer shared experts: one segment of all T tokens each, after the T*k pair rows
        if (S > 0 && tid == 0) offsets[E] = P;
        for (int sh = tid; sh < S; sh += blockDim.x) { counts[E + sh] = T; offsets[E + sh + 1] = P + (sh + 1) * T; }
        if (tid == 0 && sm.bad) atomicExch(status, SAEM_ERR_INVALID_ARG);
    }
    for (int p = tid; p < P; p += blockDim.x) {
        int e = idx[p];
        if (e < 0 || e >= E) { if (write_global) inv_perm[p] = -1; continue; }
        int r = sm.offsets[e] + table[e * n_chunks + (p >> 5)] + rank[p];
        if (perm_s) perm_s[r] = p;
        if (write_global) { perm[r] = p; inv_perm[p] = r; }
    }
    __syncthreads();
}

__device__ __forceinline__ void copy_row(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int d,
                                         int tid, int nthreads) {
    const uint4* s = reinterpret_cast<const uint4*>(src);
    uint4* o = reinterpret_cast<uint4*>(dst);
    for (int i = tid; i < d / 8; i += nthreads) o[i] = s[i];
}

__global__ void __launch_bounds__(kRepackThreads)
repack_fused_kernel(const int32_t* __restrict__ idx, const uint16_t* __restrict__ x, int T, int E, int S, int k, int d,
                    int32_t* __restrict__ counts, int32_t* __restrict__ offsets, int32_t* __restrict__ perm,
                    int32_t* __restrict__ inv_perm, uint16_t* __restrict__ x_packed, int* __restrict__ status) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    pdl_wait();
    pdl_launch_dependents();
    const int P = T * k, n_chunks = (P + 31) >> 5;
    RepackSmem& sm = *reinterpret_cast<RepackSmem*>(smem_raw);
    uint16_t* table = reinterpret_cast<uint16_t*>(smem_raw + sizeof(RepackSmem));
    size_t off = sizeof(RepackSmem) + (((size_t)n_chunks * E * 2 + 15) & ~(size_t)15);
    int32_t* perm_s = reinterpret_cast<int32_t*>(smem_raw + off);
    uint8_t* rank = smem_raw + off + (size_t)n_chunks * 32 * 4;
    for (int i = threadIdx.x; i < n_chunks * 32; i += blockDim.x) perm_s[i] = -1;
    index_phase(idx, P, E, S, T, sm, table, rank, perm_s, blockIdx.x == 0, counts, offsets, perm, inv_perm, status);
    const int total = sm.offsets[E];                 // rows actually packed (pairs with a valid expert)
    // each CTA copies rows r = blockIdx.x, blockIdx.x + gridDim.x, ...; 128 threads per row
    const int sub = threadIdx.x >> 7, nsub = blockDim.x >> 7;
    for (int r = blockIdx.x * nsub + sub; r < total; r += gridDim.x * nsub) {
        int p = perm_s[r];
        copy_row(x + (size_t)(p / k) * d, x_packed + (size_t)r * d, d, threadIdx.x & 127, 128);
    }
    for (int r = blockIdx.x * nsub + sub; r < S * T; r += gridDim.x * nsub)      // shared segments: x itself
        copy_row(x + (size_t)(r % T) * d, x_packed + (size_t)(P + r) * d, d, threadIdx.x & 127, 128);
}

__global__ void __launch_bounds__(1024)
repack_index_kernel(const int32_t* __restrict__ idx, int T, int E, int S, int k, int32_t* __restrict__ counts,
                    int32_t* __restrict__ offsets, int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
                    int* __restrict__ status) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    pdl_wait();
    pdl_launch_dependents();
    const int P = T * k, n_chunks = (P + 31) >> 5;
    RepackSmem& sm = *reinterpret_cast<RepackSmem*>(smem_raw);
    uint16_t* table = reinterpret_cast<uint16_t*>(smem_raw + sizeof(RepackSmem));
    uint8_t* rank = smem_raw + sizeof(RepackSmem) + (((size_t)n_chunks * E * 2 + 15) & ~(size_t)15);
    index_phase(idx, P, E, S, T, sm, table, rank, nullptr, true, counts, offsets, perm, inv_perm, status);
}

__global__ void __launch_bounds__(256)
repack_gather_kernel(const uint16_t* __restrict__ x, const int32_t* __restrict__ perm,
                     const int32_t* __restrict__ offsets, int T, int E, int S, int k, int d,
                     uint16_t* __restrict__ x_packed) {
    pdl_wait();
    pdl_launch_dependents();
    const int total = S > 0 ? T * k : offsets[E];
    const int sub = threadIdx.x >> 6, nsub = blockDim.x >> 6;     // 64 threads per row
    for (int r = blockIdx.x * nsub + sub; r < total; r += gridDim.x * nsub) {
        int p = perm[r];
        copy_row(x + (size_t)(p / k) * d, x_packed + (size_t)r * d, d, threadIdx.x & 63, 64);
    }
    for (int r = blockIdx.x * nsub + sub; r < S * T; r += gridDim.x * nsub)      // shared segments: x itself
        copy_row(x + (size_t)(r % T) * d, x_packed + (size_t)(T * k + r) * d, d, threadIdx.x & 63, 64);
}

cudaError_t launch_repack(const int32_t* idx, const uint16_t* x, int T, int E, int S, int k, int d, int32_t* counts,
                          int32_t* offsets, int32_t* perm, int32_t* inv_perm, uint16_t* x_packed, int* status,
                          int n_sm, cudaStream_t st, int* n_launch) {
    const int P = T * k, n_chunks = (P + 31) >> 5;
    size_t base = sizeof(RepackSmem) + (((size_t)n_chunks * E * 2 + 15) & ~(size_t)15);
    static bool attr_done[64];
    if (first_call_on_device(attr_done)) {
        cudaError_t e = cudaFuncSetAttribute(repack_index_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(repack_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
        if (e != cudaSuccess) return e;
    }
    if (P <= kFusedPairs) {
        size_t smem = base + (size_t)n_chunks * 32 * 4 + (size_t)n_chunks * 32;
        int rows_per_cta = kRepackThreads / 128;
        int grid = (P + S * T + rows_per_cta - 1) / rows_per_cta;
        if (grid < 1) grid = 1;
        if (grid > n_sm) grid = n_sm;
        *n_launch = 1;
        return launch_pdl(repack_fused_kernel, dim3(grid), dim3(kRepackThreads), smem, st, idx, x, T, E, S, k, d,
                          counts, offsets, perm, inv_perm, x_packed, status);
    }
    size_t smem = base + (size_t)n_chunks * 32;
    cudaError_t e = launch_pdl(repack_index_kernel, dim3(1), dim3(1024), smem, st, idx, T, E, S, k, counts, offsets, perm,
                               inv_perm, status);
    if (e != cudaSuccess) return e;
    *n_launch = 2;
    return launch_pdl(repack_gather_kernel, dim3(n_sm * 4), dim3(256), 0, st, x, perm, offsets, T, E, S, k, d, x_packed);
}

}  // namespace saem
