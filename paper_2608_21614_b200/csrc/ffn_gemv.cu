// Grouped SwiGLU expert FFN for the tiniest decode batches: every segment has at most 8 rows
// (Sec. IV-E: the expert still runs once over its contiguous rows; at batch 1-8 that is a
// matrix-vector product per expert and pure weight streaming).
//
// GEMV-style, shaped by bytes: a CTA owns 16 weight rows of one ACTIVE expert over the whole
// reduction length, so nothing is split across CTAs and nothing has to be added up afterwards
// through global memory; the grid covers (16-row group) x (active-expert rank) and the CTAs of
// ranks beyond the number of active experts exit at once (inactive experts are never read).
// Weights go straight from global memory to registers with 16-byte loads -- the packed slot
// layout keeps a tile row's 128 bytes contiguous, so a warp reads 16 rows x 64 reduction elements
// as 2 KB of full 32-byte sectors -- several k-chunks per warp in flight, no shared-memory
// staging, no mbarriers, no tensor memory: the fixed cost per launch is a few microseconds.
// The arithmetic uses mma.sync m16n8k16 (16 weight rows x up to 8 tokens): at 8 tokens the fp32
// pipes could not keep up with the weight stream.  Both operands take the SAME register-to-k
// assignment (a lane's 16-byte chunk supplies k-slots {2t, 2t+1, 2t+8, 2t+9} of two MMAs), so the
// contraction is exact without any shuffling of the loaded data.  The 8 warps of a CTA split the
// k-chunks (and, when the reduction length is short, several 16-row groups) among themselves and
// their partial tiles are added in a fixed order through shared memory (deterministic).
#include <cuda_bf16.h>

#include "saem_internal.h"

namespace saem {

constexpr int kGvThreads = 256;
constexpr int kGvWarps = kGvThreads / 32;
constexpr int kGvRows = 16;                // weight rows per CTA
constexpr int kGvMaxTokens = 8;            // rows per segment this path accepts (MMA N)

__device__ __forceinline__ void mma_16816(float* c, const uint32_t a0, const uint32_t a1, const uint32_t a2,
                                          const uint32_t a3, const uint32_t b0, const uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// PHASE 0: h = silu(Wg x) * (Wu x);  PHASE 1: y = Wd h
template <int PHASE>
__global__ void __launch_bounds__(kGvThreads, 3)
ffn_gemv_kernel(FfnArgs a, const __grid_constant__ SlotTable tab, int gpc) {
    __shared__ int s_cnt[4];
    __shared__ int s_expert, s_row0, s_rows;
    __shared__ float red[kGvWarps][2][kGvRows][kGvMaxTokens];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_wait();
    pdl_launch_dependents();

    // ---- which expert is the blockIdx.y-th active one? (one thread per expert, ballots) ----
    {
        int rows = 0, r0 = 0;
        const int e = tid;
        if (e < a.E) {
            int r1 = a.max_rows;
            if (a.offsets) { r0 = a.offsets[e]; r1 = a.offsets[e + 1]; }
            if (r1 > a.max_rows) r1 = a.max_rows;
            rows = r1 > r0 ? r1 - r0 : 0;
            if (!tab.in_subset[e]) rows = 0;
            if (rows > 0 && tab.slot[e] == -1) {
                if (blockIdx.x == 0 && blockIdx.y == 0) atomicExch(a.status, SAEM_ERR_NOT_RESIDENT);
                rows = 0;
            }
        }
        const unsigned act = __ballot_sync(0xffffffffu, rows > 0);
        if (tid == 0) s_expert = -1;
        if (warp < 4 && lane == 0) s_cnt[warp] = __popc(act);
        __syncthreads();
        if (warp < 4 && rows > 0) {
            int before = __popc(act & ((1u << lane) - 1u));
            for (int w = 0; w < warp; ++w) before += s_cnt[w];
            if (before == (int)blockIdx.y) { s_expert = e; s_row0 = r0; s_rows = rows; }
        }
        __syncthreads();
    }
    const int e = s_expert;
    if (e < 0) return;
    const int row0 = s_row0;
    int m = s_rows;
    if (m > kGvMaxTokens) {                    // the host only sends batches of at most 8 tokens here
        if (blockIdx.x == 0 && tid == 0) atomicExch(a.status, SAEM_ERR_SHAPE);
        m = kGvMaxTokens;
    }

    const int K = PHASE == 0 ? a.d : a.f;
    const int KC = K / kTileK;
    // A CTA owns gpc consecutive 16-row groups (more when the reduction length is short, so that every
    // CTA still moves tens of KB); warp w works on group w % gpc and takes every (8 / gpc)-th k-chunk.
    const int wpg = kGvWarps / gpc;            // warps per row group
    const int rg = blockIdx.x * gpc + (warp % gpc);
    const int kslice = warp / gpc;
    const int rb = rg >> 3, r_in = (rg & 7) * kGvRows;
    const int g = lane >> 2, t = lane & 3;     // MMA fragment coordinates
    // an HBM slot, or a packed expert in mapped pinned host memory read in place over the host link
    const int si = tab.slot[e];
    const uint8_t* slot = si >= 0 ? a.slot_region + (size_t)si * a.slot_bytes : tab.host[-(si + 2)];
    const uint8_t* wbase = PHASE == 0 ? slot + (size_t)rb * KC * (2 * kTileBytes)
                                      : slot + (size_t)2 * a.d * a.f * 2 + (size_t)rb * KC * kTileBytes;
    const size_t chunk_stride = PHASE == 0 ? 2 * kTileBytes : kTileBytes;
    const uint16_t* act = PHASE == 0 ? a.x_packed : a.h;
    // byte offset of this lane's 16-byte chunk (k-chunk position 4 b + t) in tile rows r_in + g and r_in + g + 8
    const uint32_t off_lo0 = (uint32_t)(r_in + g) * 128u + (uint32_t)((t ^ g) << 4);
    const uint32_t off_lo1 = (uint32_t)(r_in + g) * 128u + (uint32_t)(((4 + t) ^ g) << 4);
    const uint32_t off_hi0 = off_lo0 + 8u * 128u, off_hi1 = off_lo1 + 8u * 128u;
    const uint16_t* xrow = act + (size_t)(row0 + (g < m ? g : 0)) * K + t * 8;
    const bool x_valid = g < m;

    float cg[4] = {0.f, 0.f, 0.f, 0.f}, cu[4] = {0.f, 0.f, 0.f, 0.f};
    constexpr int UN = PHASE == 0 ? 1 : 2;     // k-chunks of loads in flight per warp (three CTAs per SM)
    for (int kc0 = kslice; kc0 < KC; kc0 += wpg * UN) {
        uint4 wl[UN][2], wh[UN][2], ul[UN][2], uh[UN][2], xv[UN][2];
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int kc = kc0 + u * wpg;
            if (kc < KC) {
                const uint8_t* tile = wbase + (size_t)kc * chunk_stride;
                wl[u][0] = *reinterpret_cast<const uint4*>(tile + off_lo0);
                wl[u][1] = *reinterpret_cast<const uint4*>(tile + off_lo1);
                wh[u][0] = *reinterpret_cast<const uint4*>(tile + off_hi0);
                wh[u][1] = *reinterpret_cast<const uint4*>(tile + off_hi1);
                if (PHASE == 0) {
                    ul[u][0] = *reinterpret_cast<const uint4*>(tile + kTileBytes + off_lo0);
                    ul[u][1] = *reinterpret_cast<const uint4*>(tile + kTileBytes + off_lo1);
                    uh[u][0] = *reinterpret_cast<const uint4*>(tile + kTileBytes + off_hi0);
                    uh[u][1] = *reinterpret_cast<const uint4*>(tile + kTileBytes + off_hi1);
                }
                const uint4 z = make_uint4(0u, 0u, 0u, 0u);
                xv[u][0] = x_valid ? *reinterpret_cast<const uint4*>(xrow + (size_t)kc * kTileK) : z;
                xv[u][1] = x_valid ? *reinterpret_cast<const uint4*>(xrow + (size_t)kc * kTileK + 32) : z;
            }
        }
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            if (kc0 + u * wpg < KC) {
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    mma_16816(cg, wl[u][b].x, wh[u][b].x, wl[u][b].y, wh[u][b].y, xv[u][b].x, xv[u][b].y);
                    mma_16816(cg, wl[u][b].z, wh[u][b].z, wl[u][b].w, wh[u][b].w, xv[u][b].z, xv[u][b].w);
                    if (PHASE == 0) {
                        mma_16816(cu, ul[u][b].x, uh[u][b].x, ul[u][b].y, uh[u][b].y, xv[u][b].x, xv[u][b].y);
                        mma_16816(cu, ul[u][b].z, uh[u][b].z, ul[u][b].w, uh[u][b].w, xv[u][b].z, xv[u][b].w);
                    }
                }
            }
        }
    }
    // accumulator fragment: c0,c1 -> (row g, tokens 2t, 2t+1); c2,c3 -> (row g + 8, same tokens)
    red[warp][0][g][2 * t] = cg[0];
    red[warp][0][g][2 * t + 1] = cg[1];
    red[warp][0][g + 8][2 * t] = cg[2];
    red[warp][0][g + 8][2 * t + 1] = cg[3];
    if (PHASE == 0) {
        red[warp][1][g][2 * t] = cu[0];
        red[warp][1][g][2 * t + 1] = cu[1];
        red[warp][1][g + 8][2 * t] = cu[2];
        red[warp][1][g + 8][2 * t + 1] = cu[3];
    }
    __syncthreads();
    // red[w] holds the partial tile of warp w = kslice * gpc + group; add a group's wpg slices in order
    for (int o = tid; o < gpc * kGvRows * kGvMaxTokens; o += kGvThreads) {
        const int grp = o >> 7, n = (o >> 4) & 7, r = o & 15;   // 16 consecutive threads: 16 consecutive columns of a token row
        if (n < m) {
            float sg = 0.f, su = 0.f;
            for (int ks = 0; ks < wpg; ++ks) {            // fixed order
                sg += red[ks * gpc + grp][0][r][n];
                if (PHASE == 0) su += red[ks * gpc + grp][1][r][n];
            }
            const size_t row = (size_t)(row0 + n);
            const size_t col = (size_t)(blockIdx.x * gpc + grp) * kGvRows + r;
            if (PHASE == 0) {
                const float hv = sg / (1.f + expf(-sg)) * su;
                reinterpret_cast<__nv_bfloat16*>(a.h)[row * a.f + col] = __float2bfloat16_rn(hv);
            } else {
                a.y_packed[row * a.d + col] = sg;
            }
        }
    }
}

// Row groups per CTA: enough that a CTA moves about 64 KB of weights, a power of two that divides
// both the warp count and the number of row groups.
static int groups_per_cta(int rows, int K, int matrices) {
    const int n_groups = rows / kGvRows;
    const long long bytes_per_group = (long long)kGvRows * K * 2 * matrices;
    int gpc = 1;
    while (gpc < kGvWarps && bytes_per_group * gpc < 64 * 1024 && n_groups % (gpc * 2) == 0) gpc *= 2;
    return gpc;
}

cudaError_t launch_ffn_gemv(const FfnArgs& a, const SlotTable& tab, cudaStream_t st, int* n_launch) {
    const int max_active = a.max_active < 1 ? 1 : a.max_active;
    const int gpc0 = groups_per_cta(a.f, a.d, 2), gpc1 = groups_per_cta(a.d, a.f, 1);
    const dim3 g0((unsigned)(a.f / kGvRows / gpc0), (unsigned)max_active), g1((unsigned)(a.d / kGvRows / gpc1), (unsigned)max_active);
    cudaError_t e = launch_pdl(ffn_gemv_kernel<0>, g0, dim3(kGvThreads), 0, st, a, tab, gpc0);
    if (e != cudaSuccess) return e;
    e = launch_pdl(ffn_gemv_kernel<1>, g1, dim3(kGvThreads), 0, st, a, tab, gpc1);
    *n_launch = 2;
    return e;
}

}  // namespace saem
