// Expert-aligned token repacking (Sec. IV-E): histogram of (token, slot) pairs per expert,
// exclusive scan, and a stable scatter into per-expert contiguous segments -- a counting sort
// that keeps ascending pair id inside a segment, so the permutation is unique and no atomics
// decide an order.  The row gather moves 16 bytes per thread per access.
//
// Index phase, one CTA: warps take consecutive 32-pair chunks; within a chunk one ballot per bit of
// the expert id groups equal ids and a lane's rank is the number of lower lanes in its group; an
// [expert][chunk] table of 16-bit counts is scanned down the chunks by one warp per expert;
// a scan over the expert totals gives the segment offsets.
//
// Small problems (pairs <= kFusedPairs): every CTA of the grid repeats the index phase in its own
// shared memory (only CTA 0 writes the index outputs) and then copies its share of the rows, so
// the whole repack is one launch.  Larger problems: the index phase runs on one CTA per 1024 pairs in
// two passes (per-block histograms and ranks; offsets and scatter), then a grid-wide gather.
#include "saem_internal.h"

namespace saem {

constexpr int kRepackThreads = 512;
constexpr int kFusedPairs = 2048;

// Row length (in 16-bit entries) of the [expert][chunk] table: at least n_chunks, and an odd number of
// 32-bit words, so that the lanes of a warp, which touch the same chunk of different experts, fall
// into different shared-memory banks (with a row of 384 entries all 32 lanes hit one bank).
__host__ __device__ __forceinline__ int table_stride(int n_chunks) {
    int s = (n_chunks + 1) & ~1;
    if (((s >> 1) & 1) == 0) s += 2;
    return s;
}

struct RepackSmem {
    int counts[SAEM_MAX_EXPERTS];
    int offsets[SAEM_MAX_EXPERTS + 1];
    int bad;
    int pad_[2];            // sizeof is a multiple of 16: the chunk table behind it is cleared with 16-byte stores
};
static_assert(sizeof(RepackSmem) % 16 == 0, "the chunk table must start 16-byte aligned");

// Shared-memory carve: [RepackSmem][chunk table uint16 n_chunks*E][perm int32 P][rank uint8 P_padded]
__device__ __forceinline__ void index_phase(const int32_t* __restrict__ idx, int P, int E, int S, int T, RepackSmem& sm,
                                            uint16_t* table, uint8_t* rank, int32_t* perm_s, bool write_global,
                                            int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                                            int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
                                            int* __restrict__ status) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = blockDim.x >> 5;
    const int n_chunks = (P + 31) >> 5, tstride = table_stride(n_chunks);
    const int id_bits = E > 1 ? 32 - __clz(E - 1) : 0;
    // table[e * tstride + c]: pairs of chunk c routed to expert e (expert-major, so that the scan
    // down the chunks of one expert reads consecutive shared-memory words)
    {   // the table starts 16-byte aligned; clear it with wide stores (the tail may spill into the rank
        // array behind it, which is written later)
        uint4* t4 = reinterpret_cast<uint4*>(table);
        const int n16 = (tstride * E * 2 + 15) >> 4;
        for (int i = tid; i < n16; i += blockDim.x) t4[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    if (tid == 0) sm.bad = 0;
    __syncthreads();
    for (int c = warp; c < n_chunks; c += n_warps) {
        int p = c * 32 + lane;
        int e = p >= P ? -1 : idx[p];
        if (p < P && (e < 0 || e >= E)) { e = -1; sm.bad = 1; }
        // lanes with the same expert id: one ballot per bit of the id (the index phase runs on one SM
        // and is bound by its instruction issue, so only the bits that E needs); invalid pairs are
        // masked out and never use their rank
        unsigned grp = __ballot_sync(0xffffffffu, e >= 0);
        for (int b = 0; b < id_bits; ++b) {
            const unsigned bal = __ballot_sync(0xffffffffu, (e >> b) & 1);
            grp &= ((e >> b) & 1) ? bal : ~bal;
        }
        int r = __popc(grp & ((1u << lane) - 1u));
        if (e >= 0) {
            rank[p] = (uint8_t)r;
            if (r == 0) table[e * tstride + c] = (uint16_t)__popc(grp);
        }
    }
    __syncthreads();
    // chunk counts -> exclusive running base per expert: one warp per expert, 32 chunks per step
    for (int e = warp; e < E; e += n_warps) {
        int run = 0;
        for (int c0 = 0; c0 < n_chunks; c0 += 32) {
            const int c = c0 + lane;
            const int v = c < n_chunks ? table[e * tstride + c] : 0;
            int inc = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += n;
            }
            if (c < n_chunks) table[e * tstride + c] = (uint16_t)(run + inc - v);
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
        int r = sm.offsets[e] + table[e * tstride + (p >> 5)] + rank[p];
        if (perm_s) perm_s[r] = p;
        else if (write_global) perm[r] = p;
        if (write_global) inv_perm[p] = r;
    }
    __syncthreads();
    if (perm_s && write_global)                      // the permutation leaves through shared memory: coalesced stores
        for (int r = tid; r < sm.offsets[E]; r += blockDim.x) perm[r] = perm_s[r];
    // pairs with an invalid expert id were dropped: the rows behind the last segment hold no pair
    if (write_global)
        for (int r = sm.offsets[E] + tid; r < P; r += blockDim.x) perm[r] = -1;
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
    size_t off = sizeof(RepackSmem) + (((size_t)table_stride(n_chunks) * E * 2 + 15) & ~(size_t)15);
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

// ---- larger problems: the index phase on many CTAs ----
// Block b owns pairs [b * kBlockPairs, (b + 1) * kBlockPairs).  Pass 1: per block and expert the number of
// pairs (hist[b][e]) and every pair's rank among the block's pairs of the same expert (rank16[p]), both by
// the chunk rule of the one-CTA phase (ballots inside a 32-pair chunk, a scan down the block's 32 chunks).
// Pass 2: every block adds up the columns of hist (segment offsets = scan over the expert totals; its own
// base per expert = offset + the blocks before it) and writes perm / inv_perm for its pairs.  Ascending
// pair id inside a segment holds by construction: blocks in order, ranks in order.
constexpr int kBlockPairs = 1024;
constexpr int kBlockChunks = kBlockPairs / 32;

__global__ void __launch_bounds__(kBlockPairs)
repack_hist_kernel(const int32_t* __restrict__ idx, int P, int E, int32_t* __restrict__ hist, uint16_t* __restrict__ rank16,
                   int* __restrict__ status) {
    __shared__ uint16_t table[SAEM_MAX_EXPERTS][kBlockChunks + 2];      // [expert][chunk], padded against bank conflicts
    __shared__ int bad;
    pdl_wait();
    pdl_launch_dependents();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int id_bits = E > 1 ? 32 - __clz(E - 1) : 0;
    for (int i = tid; i < SAEM_MAX_EXPERTS * (kBlockChunks + 2); i += kBlockPairs) (&table[0][0])[i] = 0;
    if (tid == 0) bad = 0;
    __syncthreads();
    const int p = blockIdx.x * kBlockPairs + tid;
    int e = p < P ? idx[p] : -1;
    if (p < P && (e < 0 || e >= E)) { e = -1; bad = 1; }
    unsigned grp = __ballot_sync(0xffffffffu, e >= 0);
    for (int b = 0; b < id_bits; ++b) {
        const unsigned bal = __ballot_sync(0xffffffffu, (e >> b) & 1);
        grp &= ((e >> b) & 1) ? bal : ~bal;
    }
    const int r = __popc(grp & ((1u << lane) - 1u));
    if (e >= 0 && r == 0) table[e][warp] = (uint16_t)__popc(grp);
    __syncthreads();
    for (int x = warp; x < E; x += kBlockChunks) {                      // exclusive scan down the 32 chunks of expert x
        const int v = table[x][lane];
        int inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += n;
        }
        table[x][lane] = (uint16_t)(inc - v);
        if (lane == 31) hist[(size_t)blockIdx.x * E + x] = inc;
    }
    __syncthreads();
    if (e >= 0) rank16[p] = (uint16_t)(table[e][warp] + r);
    if (tid == 0 && bad) atomicExch(status, SAEM_ERR_INVALID_ARG);
}

__global__ void __launch_bounds__(kBlockPairs)
repack_scatter_kernel(const int32_t* __restrict__ idx, int T, int E, int S, int k, const int32_t* __restrict__ hist,
                      const uint16_t* __restrict__ rank16, int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                      int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm) {
    __shared__ int total[SAEM_MAX_EXPERTS], base[SAEM_MAX_EXPERTS], seg[SAEM_MAX_EXPERTS + 1];
    pdl_wait();
    pdl_launch_dependents();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int P = T * k, n_blocks = (P + kBlockPairs - 1) / kBlockPairs;
    if (tid < E) {
        int before = 0, all = 0;
        for (int b = 0; b < n_blocks; ++b) {
            const int v = hist[(size_t)b * E + tid];
            if (b < (int)blockIdx.x) before += v;
            all += v;
        }
        total[tid] = all;
        base[tid] = before;
    }
    __syncthreads();
    if (warp == 0) {                                   // exclusive scan over the expert totals
        int carry = 0;
        for (int b0 = 0; b0 < E; b0 += 32) {
            const int x = b0 + lane;
            const int v = x < E ? total[x] : 0;
            int inc = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += n;
            }
            if (x < E) seg[x] = carry + inc - v;
            carry += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) seg[E] = carry;
    }
    __syncthreads();
    const int p = blockIdx.x * kBlockPairs + tid;
    if (p < P) {
        const int e = idx[p];
        if (e < 0 || e >= E) {
            inv_perm[p] = -1;
        } else {
            const int r = seg[e] + base[e] + rank16[p];
            perm[r] = p;
            inv_perm[p] = r;
        }
    }
    // rows behind the last segment hold no pair (pairs with an invalid expert id were dropped)
    for (int r = seg[E] + (int)blockIdx.x * kBlockPairs + tid; r < P; r += (int)gridDim.x * kBlockPairs) perm[r] = -1;
    if (blockIdx.x == 0) {
        for (int x = tid; x < E; x += kBlockPairs) counts[x] = total[x];
        for (int x = tid; x <= E; x += kBlockPairs) offsets[x] = seg[x];
        if (S > 0 && tid == 0) offsets[E] = P;         // in-layer shared experts: one segment of all T tokens each
        for (int sh = tid; sh < S; sh += kBlockPairs) { counts[E + sh] = T; offsets[E + sh + 1] = P + (sh + 1) * T; }
    }
}

__global__ void __launch_bounds__(256)
repack_gather_kernel(const uint16_t* __restrict__ x, const int32_t* __restrict__ perm,
                     const int32_t* __restrict__ offsets, int T, int E, int S, int k, int d,
                     uint16_t* __restrict__ x_packed) {
    pdl_wait();
    pdl_launch_dependents();
    // with shared experts offsets[E] is T*k whatever was dropped; rows without a pair have perm -1
    const int total = S > 0 ? T * k : offsets[E];
    const int sub = threadIdx.x >> 6, nsub = blockDim.x >> 6;     // 64 threads per row
    for (int r = blockIdx.x * nsub + sub; r < total; r += gridDim.x * nsub) {
        int p = perm[r];
        if (p < 0) continue;
        copy_row(x + (size_t)(p / k) * d, x_packed + (size_t)r * d, d, threadIdx.x & 63, 64);
    }
    for (int r = blockIdx.x * nsub + sub; r < S * T; r += gridDim.x * nsub)      // shared segments: x itself
        copy_row(x + (size_t)(r % T) * d, x_packed + (size_t)(T * k + r) * d, d, threadIdx.x & 63, 64);
}

cudaError_t launch_repack(const int32_t* idx, const uint16_t* x, int T, int E, int S, int k, int d, int32_t* counts,
                          int32_t* offsets, int32_t* perm, int32_t* inv_perm, uint16_t* x_packed, int* status,
                          int32_t* hist, uint16_t* rank16, int n_sm, cudaStream_t st, int* n_launch) {
    const int P = T * k, n_chunks = (P + 31) >> 5;
    static bool attr_done[64];
    if (first_call_on_device(attr_done)) {
        cudaError_t e = cudaFuncSetAttribute(repack_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
        if (e != cudaSuccess) return e;
    }
    if (P <= kFusedPairs) {
        size_t base = sizeof(RepackSmem) + (((size_t)table_stride(n_chunks) * E * 2 + 15) & ~(size_t)15);
        size_t smem = base + (size_t)n_chunks * 32 * 4 + (size_t)n_chunks * 32;
        int rows_per_cta = kRepackThreads / 128;
        int grid = (P + S * T + rows_per_cta - 1) / rows_per_cta;
        if (grid < 1) grid = 1;
        if (grid > n_sm) grid = n_sm;
        *n_launch = 1;
        return launch_pdl(repack_fused_kernel, dim3(grid), dim3(kRepackThreads), smem, st, idx, x, T, E, S, k, d,
                          counts, offsets, perm, inv_perm, x_packed, status);
    }
    const int n_blocks = (P + kBlockPairs - 1) / kBlockPairs;
    cudaError_t e = launch_pdl(repack_hist_kernel, dim3(n_blocks), dim3(kBlockPairs), 0, st, idx, P, E, hist, rank16, status);
    if (e != cudaSuccess) return e;
    e = launch_pdl(repack_scatter_kernel, dim3(n_blocks), dim3(kBlockPairs), 0, st, idx, T, E, S, k, (const int32_t*)hist,
                   (const uint16_t*)rank16, counts, offsets, perm, inv_perm);
    if (e != cudaSuccess) return e;
    *n_launch = 3;
    return launch_pdl(repack_gather_kernel, dim3(n_sm * 4), dim3(256), 0, st, x, perm, offsets, T, E, S, k, d, x_packed);
}

}  // namespace saem
