// The whole MoE layer step for the smallest decode batches (at most 8 tokens, top-k at most 8) in ONE
// launch instead of five.  At batch 1-8 the step moves a few tens of megabytes, so a launch's fixed
// cost (start-up, finding the active experts, the last partial wave) is as large as its streaming
// time; the paper's operating point is exactly this regime (batch 1-8 decode).
//
// One persistent CTA per SM, 16 warps.  Every CTA repeats the tiny gate (top-k of E logits for <= 8
// tokens; Background "Mixture-of-Experts Inference") and the expert-aligned repack indices (Sec. IV-E:
// counts, exclusive scan, stable permutation) in its own shared memory -- CTA 0 also writes them out,
// so they stay inspectable and bit-exact -- and then the grid runs two streaming phases:
//
//   phase A  h = silu(Wg x) * (Wu x).  A warp's unit is 16 hidden units of one ACTIVE expert over the
//            whole reduction length: an MMA's 16 rows are 8 gate rows and the 8 matching up rows, so
//            SiLU*mul happens in the accumulator registers of one thread and nothing is exchanged
//            between warps.  Token rows are read straight from x through the permutation (no x_packed).
//   phase B  y = Wd h for 32 output columns of one active expert per warp unit, then the merge (Sec.
//            IV-D): each (group of 32 columns, token) has a ticket counter, and the warp that delivers
//            a token's last contribution adds the token's k contributions in slot order j = 0..k-1,
//            shared experts last, with the arithmetic of the combine kernel (deterministic whoever
//            does it; nobody waits for anybody; the merges are spread over the whole phase).  With at
//            most 16 active experts a CTA owns 16 columns of every expert instead and merges them in
//            its own shared memory.
//
// Between the phases the grid meets at a barrier (a cooperative launch guarantees that all CTAs are
// resident; the wait is bounded and gives up with SAEM_ERR_TIMEOUT).  Before it arrives, every warp
// has already requested the first weight stages of its phase-B unit, so the barrier and the L2 round
// trip of h hide behind loads in flight.  Where a cooperative launch is not available the same kernel
// runs as two launches (phase A, phase B), the second waiting for the first by programmatic dependent
// launch after it has requested its first weights.
//
// Shaped by bytes (decode is weight streaming): a chunk of a unit is 4 KB of consecutive rows of the
// packed slot layout's tiles, fetched by one cp.async.bulk into the warp's own ring of shared-memory
// stages (three in flight per warp, 192 KB per SM, no registers spent on loads in flight; 16-byte
// cp.async per lane was tried first and was bound by the SM's memory-instruction queue);
// mma.sync m16n8k16 is the arithmetic unit (16 weight rows x up to 8 tokens, fp32 accumulation),
// reading the XOR-swizzled rows without bank conflicts; activation pieces come from L1 / L2 into
// registers one chunk ahead.  Every warp gets one contiguous range of k-chunks; when a range cuts a
// unit, the partial tiles are added in warp order through shared memory.
#include <cuda_bf16.h>

#include "route_row.cuh"
#include "tc_common.cuh"

namespace saem {

constexpr int kDfMaxTokens = 8;
constexpr int kDfMaxK = 8;
constexpr int kDfMaxPairs = kDfMaxTokens * kDfMaxK;
constexpr int kDfWarps = 16;
constexpr int kDfThreads = kDfWarps * 32;
constexpr int kDfStages = 3;                  // stages of a warp's ring (the launch uses two of them beyond 4 tokens)
constexpr int kDfStageBytes = 4096;              // per warp and stage: the 32 weight rows of one chunk of a unit
constexpr int kDfRingBytes = kDfWarps * kDfStages * kDfStageBytes + 128;
constexpr unsigned long long kDfBarrierLimitNs = 200000000ull;   // 0.2 s
constexpr int kDfTicketOff = 64;               // the step's synchronisation words: barrier counter, then the merge's tickets

struct DecodeIndex {
    int32_t idx[kDfMaxPairs];
    float w[kDfMaxPairs];
    int32_t perm[kDfMaxPairs];
    int32_t inv[kDfMaxPairs];
    int32_t counts[SAEM_MAX_EXPERTS];
    int32_t offsets[SAEM_MAX_EXPERTS + 1];
    int16_t act[SAEM_MAX_EXPERTS];          // experts with rows AND a slot, ascending id
    int warp_act[4];
    int need[kDfMaxTokens];                 // contributions a token's merge waits for: its resident experts + resident shared ones
    int n_active;
    int absent;                             // an expert with rows has no slot
};

__device__ __forceinline__ void mma_16816(float* c, const uint32_t a0, const uint32_t a1, const uint32_t a2,
                                          const uint32_t a3, const uint32_t b0, const uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
// Activation pieces come through L1: the 16 warps of a CTA read the same few token rows over and over (x is an
// input; h is first touched by this CTA after the grid barrier, so no stale line can be in L1).
__device__ __forceinline__ uint4 ld_act(const uint16_t* p) {
    uint4 v;
    asm volatile("ld.global.ca.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
// Gate and repack indices of the whole (tiny) batch in shared memory; every thread of the CTA calls it.
// Same arithmetic and tie rules as route_kernel / the repack kernels: slots in descending logit order,
// segments in ascending expert id, ascending pair id inside a segment, one segment of all T tokens per
// in-layer shared expert behind the T*k pair rows.  counts[e] = #{p: idx[p] == e} and offsets[e] =
// #{p: idx[p] < e} come from one sweep over the (at most 64) pairs: no scan is needed.
__device__ __forceinline__ void build_index(const DecodeArgs& a, const SlotTable& tab, DecodeIndex& sm) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int P = a.T * a.k, ES = a.E + a.S;
    if (warp < a.T)
        route_row(a.logits + (size_t)warp * a.E, a.E, a.k, a.renorm, lane, &sm.idx[warp * a.k], &sm.w[warp * a.k]);
    if (tid == 0) sm.absent = 0;
    __syncthreads();
    if (tid < SAEM_MAX_EXPERTS) {                     // four whole warps: the ballots below need them
        int c = 0, o = 0;
        if (tid < a.E) {
            for (int p = 0; p < P; ++p) {
                const int e = sm.idx[p];
                c += e == tid ? 1 : 0;
                o += e < tid ? 1 : 0;
            }
        } else if (tid < ES) {
            c = a.T;
            o = P + (tid - a.E) * a.T;
        }
        if (tid < ES) { sm.counts[tid] = c; sm.offsets[tid] = o; }
        if (tid == ES) sm.offsets[ES] = P + a.S * a.T;
        const bool has_rows = tid < ES && c > 0;
        if (has_rows && tab.slot[tid] < 0) sm.absent = 1;
        const unsigned actm = __ballot_sync(0xffffffffu, has_rows && tab.slot[tid] >= 0);
        if (lane == 0) sm.warp_act[warp] = __popc(actm);
    }
    if (tid == SAEM_MAX_EXPERTS && ES == SAEM_MAX_EXPERTS) sm.offsets[ES] = P + a.S * a.T;
    __syncthreads();
    if (tid < SAEM_MAX_EXPERTS) {
        const bool act = tid < ES && sm.counts[tid] > 0 && tab.slot[tid] >= 0;
        const unsigned actm = __ballot_sync(0xffffffffu, act);
        int before = __popc(actm & ((1u << lane) - 1u));
        for (int w = 0; w < warp; ++w) before += sm.warp_act[w];
        if (act) sm.act[before] = (int16_t)tid;
        if (tid == 0) sm.n_active = sm.warp_act[0] + sm.warp_act[1] + sm.warp_act[2] + sm.warp_act[3];
    }
    if (tid < P) {
        const int e = sm.idx[tid];
        int rank = 0;
        for (int q = 0; q < tid; ++q) rank += sm.idx[q] == e ? 1 : 0;
        const int r = sm.offsets[e] + rank;
        sm.perm[r] = tid;
        sm.inv[tid] = r;
    }
    if (tid >= kDfThreads - a.T) {
        const int tok = kDfThreads - 1 - tid;
        int n = 0;
        for (int j = 0; j < a.k; ++j) n += tab.slot[sm.idx[tok * a.k + j]] >= 0 ? 1 : 0;
        for (int sh = 0; sh < a.S; ++sh) n += tab.slot[a.E + sh] >= 0 ? 1 : 0;
        sm.need[tok] = n;
    }
    __syncthreads();
}

// How a phase's units are dealt to the grid's warps: every warp gets ONE contiguous range of k-chunks.
//   few units (fewer than 8 per CTA): ks adjacent warps of a CTA share one unit and cut its k-chunks
//     into ks contiguous parts; warp group wg of CTA b takes unit b + gridDim * wg, so that consecutive
//     units land in different CTAs and every busy warp has the same amount of work (more than half of
//     the warps are busy, which is enough requests in flight to keep HBM busy);
//   many units: CTA b takes the units b, b + G, b + 2 G, ... (every CTA gets a share of every expert, so
//     an expert that streams faster or slower than the others -- its weights partly in L2, more rows --
//     does not unbalance the grid) and its 16 warps cut that unit-major chunk list into 16 equal
//     contiguous ranges (CTAs differ by at most one unit in 8).
// A range that starts inside a unit yields a "head" partial tile (left in shared memory), one that
// starts a unit but does not finish it a "tail" (kept in registers): after the phase's streaming the
// warp that holds a unit's tail adds the heads of the following warps in warp order.
struct WarpWork {
    int u0, kc0, n;       // first unit, first chunk inside it, number of chunks
    int ustep;            // distance between consecutive units of this warp's range
};
__device__ __forceinline__ WarpWork deal_units(int n_units, int KC, int warp) {
    const int G = (int)gridDim.x, b = (int)blockIdx.x;
    WarpWork w;
    if (n_units < 8 * G) {
        int ks = 1;
        while (ks < kDfWarps && ks * 2 <= KC && (long long)n_units * ks * 2 <= (long long)G * kDfWarps) ks *= 2;   // every warp of a group gets a chunk
        const int u = b + G * (warp / ks), s = warp % ks;
        const int c0 = KC * s / ks, c1 = KC * (s + 1) / ks;
        w.u0 = u;
        w.kc0 = c0;
        w.n = u < n_units ? c1 - c0 : 0;
        w.ustep = 1;
    } else {
        const int mine = (n_units - b + G - 1) / G;    // units b, b + G, b + 2 G, ...
        const long long n = (long long)mine * KC;
        const long long q0 = n * warp / kDfWarps, q1 = n * (warp + 1) / kDfWarps;
        w.u0 = b + G * (int)(q0 / KC);
        w.kc0 = (int)(q0 % KC);
        w.n = (int)(q1 - q0);
        w.ustep = G;
    }
    return w;
}

// A unit's address arithmetic.  PHASE 0: unit = hidden units 16j..16j+15 of expert act[ai]: 16 gate rows and the
// 16 matching up rows, 2 KB each, contiguous in the packed tiles (the up tile follows the gate tile); activations are
// token rows of x.  PHASE 1: unit = output columns 32j..32j+31: 32 consecutive rows of a down-matrix tile (4 KB
// contiguous); activations are the segment's rows of h.  A chunk (64 reduction elements) of a unit is 4 KB of
// weights: one stage.
template <int PHASE>
struct Unit {
    static constexpr uint32_t kStride = PHASE == 0 ? 2u * kTileBytes : (uint32_t)kTileBytes;    // bytes between chunks
    // first chunk's weights of unit u (the tile rows of chunk kc are + kc * kStride)
    static __device__ __forceinline__ const uint8_t* weights(const DecodeArgs& a, const SlotTable& tab, const DecodeIndex& sm,
                                                             int u, int upe, int KC) {
        const int ai = u / upe, j = u - ai * upe;
        const uint8_t* slot = a.slot_region + (size_t)tab.slot[sm.act[ai]] * a.slot_bytes;
        if (PHASE == 0) return slot + (size_t)(j >> 3) * KC * kStride + (size_t)((j & 7) << 4) * 128u;
        return slot + (size_t)2 * a.d * a.f * 2 + (size_t)(j >> 2) * KC * kStride + (size_t)((j & 3) << 5) * 128u;
    }
    // this lane's activation row (MMA column g = the segment's g-th row) at reduction element 8 t; nullptr beyond the segment
    static __device__ __forceinline__ const uint16_t* acts(const DecodeArgs& a, const DecodeIndex& sm, int u, int upe, int g, int t) {
        const int e = sm.act[u / upe];
        if (g >= sm.counts[e]) return nullptr;
        if (PHASE == 0) {
            const int token = e < a.E ? sm.perm[sm.offsets[e] + g] / a.k : g;
            return a.x + (size_t)token * a.d + t * 8;
        }
        return a.h + (size_t)(sm.offsets[e] + g) * a.f + t * 8;
    }
};

// phase_mask: 1 = phase A, 2 = phase B, 3 = both in this launch with the grid barrier in between.
__global__ void __launch_bounds__(kDfThreads, 1)
decode_step_kernel(DecodeArgs a, const __grid_constant__ SlotTable tab, int phase_mask) {
    extern __shared__ __align__(16) uint8_t ring_raw[];
    __shared__ DecodeIndex sm;
    __shared__ float red[kDfWarps][8][32];
    __shared__ int head_units[2][kDfWarps];           // per phase
    __shared__ __align__(8) uint64_t stage_bar[kDfWarps][kDfStages];
    __shared__ int barrier_ok, abort_flag;
    __shared__ unsigned long long barrier_target;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;            // MMA fragment coordinates
    const int P = a.T * a.k, ES = a.E + a.S;
    const uint32_t ring = (smem_u32(ring_raw) + 127u & ~127u) + (uint32_t)(warp * kDfStages) * kDfStageBytes;
    const uint32_t bars = smem_u32(&stage_bar[warp][0]);
    // Requests in flight per warp.  Up to 4 tokens the ring also holds the phase-B weights that a warp requests while it
    // waits at the grid barrier, and three stages are faster; beyond that the phases stream long enough that two are
    // (measured: Qwen3 shape at 8 tokens 67.2 -> 66.7 us, ERNIE shape 116.5 -> 114.0; at 1 token 30.7 -> 31.2 on c4).
    const int n_st = a.T > 4 ? 2 : kDfStages;
    if (tid == 0) {
        abort_flag = 0;
        barrier_ok = 1;
        for (int i = 0; i < kDfWarps * kDfStages; ++i) mbar_init(smem_u32(&stage_bar[0][0]) + 8u * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // A launch that starts with phase A may run ahead of the kernel that produces logits and x.  A
    // phase-B-only launch follows the phase-A launch, which passed this very wait before it let
    // dependents start: logits and x are final, weights are never written by a kernel, so everything
    // up to the wait for h further down may overlap the phase-A launch.
    if (phase_mask & 1) {
        pdl_wait();
        pdl_launch_dependents();
    }
    // Before this CTA arrives, the barrier counter cannot pass the next multiple of G.  The last warp reads it (warp 0
    // is on the critical path: it routes token 0) and leaves the target in shared memory for thread 0.
    if (phase_mask == 3 && tid == kDfThreads - 32) {
        unsigned long long c;
        asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(c) : "l"(a.sync) : "memory");
        barrier_target = (c / gridDim.x + 1ull) * gridDim.x;
    }
    build_index(a, tab, sm);
    const int n_active = sm.n_active;
    if (blockIdx.x == 0 && (phase_mask & 1)) {        // the index outputs of the step, for the caller and for inspection
        for (int p = tid; p < P; p += kDfThreads) {
            a.topk_idx[p] = sm.idx[p];
            a.topk_w[p] = sm.w[p];
            a.perm[p] = sm.perm[p];
            a.inv_perm[p] = sm.inv[p];
        }
        for (int e = tid; e < ES; e += kDfThreads) a.counts[e] = sm.counts[e];
        for (int e = tid; e <= ES; e += kDfThreads) a.offsets[e] = sm.offsets[e];
        if (tid == 0 && sm.absent) atomicExch(a.status, SAEM_ERR_NOT_RESIDENT);
    }
    // byte offsets of this lane's two 16-byte pieces (k positions 8t.. and 32 + 8t.. of the chunk) in a tile row whose
    // index is g modulo 8
    const uint32_t piece0 = (uint32_t)((t ^ g) << 4), piece1 = (uint32_t)(((4 + t) ^ g) << 4);

    // A warp has the complete tiles of a unit: two MMA row sets s = 0, 1, four accumulators each.  Accumulator
    // fragment: c0, c1 -> (row g, tokens 2t, 2t + 1); c2, c3 -> (row g + 8, same tokens).
    auto finish_a = [&](int u, const float* acc) {    // set s: rows g = gate rows 8s + g, rows g + 8 = the matching up rows
        const int upe = a.f / 16;
        const int ai = u / upe, j = u - ai * upe;
        const int e = sm.act[ai], row0 = sm.offsets[e], m = sm.counts[e];
        __nv_bfloat16* hb = reinterpret_cast<__nv_bfloat16*>(a.h);
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const float* c = acc + 4 * s;
            const int col = j * 16 + 8 * s + g;
            if (2 * t < m) hb[(size_t)(row0 + 2 * t) * a.f + col] = __float2bfloat16_rn(c[0] / (1.f + expf(-c[0])) * c[2]);
            if (2 * t + 1 < m) hb[(size_t)(row0 + 2 * t + 1) * a.f + col] = __float2bfloat16_rn(c[1] / (1.f + expf(-c[1])) * c[3]);
        }
    };
    auto finish_b = [&](int u, const float* acc) {    // store y, take the tokens' tickets for the 32 columns, merge what is complete
        const int upe = a.d / 32;
        const int ai = u / upe, j = u - ai * upe;
        const int e = sm.act[ai], row0 = sm.offsets[e], m = sm.counts[e];
        float* y = a.y_packed;
#pragma unroll
        for (int s = 0; s < 2; ++s) {                  // set s: rows 16 s + g and 16 s + g + 8 of the unit
            const float* c = acc + 4 * s;
            const int col = j * 32 + 16 * s + g;
            if (2 * t < m) {
                y[(size_t)(row0 + 2 * t) * a.d + col] = c[0];
                y[(size_t)(row0 + 2 * t) * a.d + col + 8] = c[2];
            }
            if (2 * t + 1 < m) {
                y[(size_t)(row0 + 2 * t + 1) * a.d + col] = c[1];
                y[(size_t)(row0 + 2 * t + 1) * a.d + col + 8] = c[3];
            }
        }
        __threadfence();
        __syncwarp();
        // One ticket per (column group, token): lane r < m speaks for the token of the segment's row r.  The warp that
        // delivers a token's last contribution merges that token's 32 columns (lane = column): the k values are
        // requested together, then added in slot order with fused multiply-adds, shared experts last -- the combine
        // kernel's arithmetic, whoever does it.
        int tok = 0;
        bool last = false;
        if (lane < m) {
            tok = e < a.E ? sm.perm[row0 + lane] / a.k : lane;
            int* ticket = a.sync + kDfTicketOff + j * kDfMaxTokens + tok;
            last = atomicAdd(ticket, 1) == sm.need[tok] - 1;
            if (last) *ticket = 0;                     // every contributor has arrived: ready for the next step
        }
        unsigned done = __ballot_sync(0xffffffffu, last);
        if (!done) return;
        __threadfence();
        const float* yc = y + j * 32 + lane;
        while (done) {
            const int tk = __shfl_sync(0xffffffffu, tok, __ffs(done) - 1);
            done &= done - 1;
            float v[kDfMaxK];
            unsigned present = 0;
#pragma unroll
            for (int jj = 0; jj < kDfMaxK; ++jj) {
                v[jj] = 0.f;
                if (jj < a.k && tab.slot[sm.idx[tk * a.k + jj]] >= 0) {
                    v[jj] = __ldcg(yc + (size_t)sm.inv[tk * a.k + jj] * a.d);
                    present |= 1u << jj;
                }
            }
            float s = 0.f;
#pragma unroll
            for (int jj = 0; jj < kDfMaxK; ++jj)
                if (present >> jj & 1u) s = fmaf(sm.w[tk * a.k + jj], v[jj], s);
            for (int sh = 0; sh < a.S; ++sh)
                if (tab.slot[a.E + sh] >= 0) s += __ldcg(yc + (size_t)(P + sh * a.T + tk) * a.d);
            const size_t at = (size_t)tk * a.d + j * 32 + lane;
            if (a.out_bf16) reinterpret_cast<__nv_bfloat16*>(a.out)[at] = __float2bfloat16_rn(s);
            else reinterpret_cast<float*>(a.out)[at] = s;
        }
    };

    // The streaming loop of one phase over this warp's chunk range ww.  Lane 0 keeps kDfStages bulk copies of 4 KB
    // in flight (request for chunk i + kDfStages goes out when chunk i has been consumed); every lane loads its own
    // activation pieces of the NEXT chunk from L2 into registers while the current chunk's weights are awaited.
    // `requested` chunks have been requested by the caller already.  Complete tiles are delivered through `finish`,
    // partial ones parked.  Returns false if a wait ran out.
    uint32_t parity = 0;                               // bit s: the phase of stage s's barrier to wait for next
    auto stream = [&](auto unit_tag, const WarpWork& ww, int KC, int upe, auto& finish, int requested, int* head_unit,
                      auto&& after_loop) -> bool {
        using U = decltype(unit_tag);
        // ---- producer state (lane 0 issues) ----
        int pu = ww.u0, pkc = ww.kc0, pleft = ww.n;
        const uint8_t* wp = nullptr;
        if (pleft > 0) wp = U::weights(a, tab, sm, pu, upe, KC) + (size_t)pkc * U::kStride;
        auto request = [&](int stage) {               // the next chunk's 4 KB into `stage`
            if (lane == 0) {
                const uint32_t dst = ring + (uint32_t)stage * kDfStageBytes, bar = bars + 8u * stage;
                mbar_expect_tx(bar, 4096u);
                if (U::kStride == 2u * kTileBytes) {   // gate rows, then the up rows of the tile behind
                    bulk_g2s(dst, wp, 2048, bar);
                    bulk_g2s(dst + 2048, wp + kTileBytes, 2048, bar);
                } else {
                    bulk_g2s(dst, wp, 4096, bar);
                }
            }
            wp += U::kStride;
            --pleft;
            if (++pkc == KC && pleft > 0) {
                pu += ww.ustep;
                pkc = 0;
                wp = U::weights(a, tab, sm, pu, upe, KC);
            }
        };
        // `requested` chunks are in flight already: move the producer past them, then fill the remaining stages
        for (int s = 0; s < n_st; ++s) {
            if (pleft <= 0) break;
            if (s < requested) {
                wp += U::kStride;
                --pleft;
                if (++pkc == KC && pleft > 0) { pu += ww.ustep; pkc = 0; wp = U::weights(a, tab, sm, pu, upe, KC); }
            } else {
                request(s);
            }
        }
        // ---- consumer state ----
        float acc[8], tail[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = tail[i] = 0.f;
        int tail_unit = -1;
        int u = ww.u0, kc_begin = ww.kc0, left = ww.n;
        int in_unit = KC - kc_begin < left ? KC - kc_begin : left;     // chunks of this range inside the current unit
        int run = in_unit;
        int stage = 0;
        bool ok = true;
        const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
        // Activation pieces travel through registers, fetched two chunks ahead of the MMAs that use them: the fetch
        // cursor (unit, chunks left in it, chunks left in the range) runs ahead of the consumer's own.
        const uint16_t* xq = nullptr;                  // this lane's activation row at the chunk to be fetched next
        int au = u, a_run = KC - kc_begin, a_left = left;
        if (left > 0) {
            xq = U::acts(a, sm, u, upe, g, t);
            if (xq) xq += (size_t)kc_begin * kTileK;
        }
        auto fetch = [&](uint4& pa, uint4& pb) {
            pa = zero4;
            pb = zero4;
            if (a_left <= 0) return;
            if (a_run == 0) {                          // the next chunk opens the range's next unit
                au += ww.ustep;
                xq = U::acts(a, sm, au, upe, g, t);
                a_run = KC;
            }
            if (xq) {
                pa = ld_act(xq);
                pb = ld_act(xq + 32);
                xq += kTileK;
            }
            --a_run;
            --a_left;
        };
        uint4 xa, xb, na, nb;                          // pieces of the current chunk and of the one after it
        fetch(xa, xb);
        fetch(na, nb);
        // this lane's weight pieces inside a stage: rows g (+ 8 per set) of the first 2 KB, the matching rows 2 KB further
        // (up rows in phase A; rows + 16 ... in phase B the second set is 2 KB further and the + 8 rows 1 KB further)
        const uint32_t w_lo = ring + (uint32_t)g * 128u;
        constexpr uint32_t kSetStep = U::kStride == 2u * kTileBytes ? 1024u : 2048u;     // bytes from set 0's rows g to set 1's
        constexpr uint32_t kHiStep = U::kStride == 2u * kTileBytes ? 2048u : 1024u;      // bytes from rows g to the set's rows g + 8
        while (left > 0) {
            uint4 ma, mb;                              // pieces of the chunk after the next one
            fetch(ma, mb);
            ok = mbar_wait(bars + 8u * stage, (parity >> stage) & 1u, &abort_flag, a.status, kDfBarrierLimitNs);
            if (!ok) break;
            parity ^= 1u << stage;
            const uint32_t base = w_lo + (uint32_t)stage * kDfStageBytes;
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                const uint32_t lo = base + (uint32_t)s * kSetStep, hi = lo + kHiStep;
                const uint4 w00 = ld_shared_v4(lo + piece0), w01 = ld_shared_v4(lo + piece1);
                const uint4 w10 = ld_shared_v4(hi + piece0), w11 = ld_shared_v4(hi + piece1);
                mma_16816(acc + 4 * s, w00.x, w10.x, w00.y, w10.y, xa.x, xa.y);
                mma_16816(acc + 4 * s, w00.z, w10.z, w00.w, w10.w, xa.z, xa.w);
                mma_16816(acc + 4 * s, w01.x, w11.x, w01.y, w11.y, xb.x, xb.y);
                mma_16816(acc + 4 * s, w01.z, w11.z, w01.w, w11.w, xb.z, xb.w);
            }
            __syncwarp();                              // every lane has read the stage (its MMAs issued) before it is refilled
            if (pleft > 0) request(stage);
            if (++stage == n_st) stage = 0;
            xa = na;
            xb = nb;
            na = ma;
            nb = mb;
            --left;
            if (--run == 0) {                          // this range's share of unit u is complete
                if (kc_begin > 0) {                    // started inside the unit: a head partial
#pragma unroll
                    for (int i = 0; i < 8; ++i) red[warp][i][lane] = acc[i];
                    if (lane == 0) head_unit[warp] = u;
                } else if (in_unit < KC) {             // started the unit but does not finish it: the tail
#pragma unroll
                    for (int i = 0; i < 8; ++i) tail[i] = acc[i];
                    tail_unit = u;
                } else {
                    finish(u, acc);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[i] = 0.f;
                u += ww.ustep;
                kc_begin = 0;
                in_unit = KC < left ? KC : left;
                run = in_unit;
            }
        }
        after_loop();                                  // this warp's ring is free again
        __syncthreads();
        if (ok && tail_unit >= 0 && !abort_flag) {     // add the following warps' heads in warp order
            for (int w2 = warp + 1; w2 < kDfWarps && head_unit[w2] == tail_unit; ++w2)
#pragma unroll
                for (int i = 0; i < 8; ++i) tail[i] += red[w2][i][lane];
            finish(tail_unit, tail);
        }
        return ok;
    };

    // Phase B's deal and the request of its first weight stages: a warp does this the moment its own phase-A
    // loop is over (or at once in a phase-B-only launch), before it meets its CTA and the grid.
    const int KC_b = a.f / kTileK, upe_b = a.d / 32;
    WarpWork ww_b = {0, 0, 0, 1};
    int requested_b = 0;
    // Column form of phase B, for the very smallest steps (at most 16 active experts, d_model / 16 <= grid): CTA j
    // owns output columns 16 j .. 16 j + 15 of EVERY active expert, a warp is (expert, part of the reduction
    // length), and the merge over a token's experts happens in this CTA's shared memory: no ticket, no read-back of
    // y through L2 (two to three dependent L2 round trips at the end of a step that is all latency).  A stage holds
    // the unit's 16 rows of two consecutive chunks (2 KB each).
    const int n_pairs_b = KC_b >> 1;
    const bool columns_b = n_active <= kDfWarps && (a.d >> 4) <= (int)gridDim.x;     // (d_ff is a multiple of 128: KC_b is even)
    int cw_ks = 1, cw_ai = 0, cw_p0 = 0, cw_n = 0, cw_left = 0;     // warps per expert; this warp's expert, first pair, pairs; pairs not requested yet
    const uint8_t* cw_wp = nullptr;                                 // weights of the next pair to request
    auto request_pair = [&](int stage) {
        if (lane == 0) {
            const uint32_t dst = ring + (uint32_t)stage * kDfStageBytes, bar = bars + 8u * stage;
            mbar_expect_tx(bar, 4096u);
            bulk_g2s(dst, cw_wp, 2048, bar);
            bulk_g2s(dst + 2048, cw_wp + kTileBytes, 2048, bar);
        }
        cw_wp += 2 * (size_t)kTileBytes;
        --cw_left;
    };
    auto prefetch_b = [&]() {
        if (columns_b) {
            while (n_active * cw_ks * 2 <= kDfWarps && cw_ks * 2 <= n_pairs_b) cw_ks *= 2;
            cw_ai = warp / cw_ks;
            const int part = warp % cw_ks, j = (int)blockIdx.x;
            if (cw_ai < n_active && j < (a.d >> 4)) {
                cw_p0 = n_pairs_b * part / cw_ks;
                cw_n = n_pairs_b * (part + 1) / cw_ks - cw_p0;
                cw_wp = a.slot_region + (size_t)tab.slot[sm.act[cw_ai]] * a.slot_bytes + (size_t)2 * a.d * a.f * 2 +
                        ((size_t)(j >> 3) * KC_b + 2 * cw_p0) * kTileBytes + (size_t)(j & 7) * 2048u;
            }
            cw_left = cw_n;
            for (; requested_b < n_st && requested_b < cw_n; ++requested_b) request_pair(requested_b);
            return;
        }
        ww_b = deal_units(n_active * upe_b, KC_b, warp);
        if (lane == 0) head_units[1][warp] = -1;
        int pu = ww_b.u0, pkc = ww_b.kc0;
        for (; requested_b < n_st && requested_b < ww_b.n; ++requested_b) {
            if (lane == 0) {
                const uint32_t dst = ring + (uint32_t)requested_b * kDfStageBytes, bar = bars + 8u * requested_b;
                mbar_expect_tx(bar, 4096u);
                bulk_g2s(dst, Unit<1>::weights(a, tab, sm, pu, upe_b, KC_b) + (size_t)pkc * Unit<1>::kStride, 4096, bar);
            }
            if (++pkc == KC_b) { pu += ww_b.ustep; pkc = 0; }
        }
    };
    // The column form's streaming and merge; every thread of the CTA calls it.  Returns false if a wait ran out.
    auto columns_phase_b = [&]() -> bool {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        bool ok = true;
        if (cw_n > 0) {
            const int e = sm.act[cw_ai];
            const uint16_t* hq = g < sm.counts[e] ? a.h + (size_t)(sm.offsets[e] + g) * a.f + (size_t)cw_p0 * (2 * kTileK) + t * 8
                                                  : nullptr;
            const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
            uint4 x[4] = {zero4, zero4, zero4, zero4};             // pieces of the current pair: k 8t.., 32 + 8t.., 64 + 8t.., 96 + 8t..
            if (hq) {
#pragma unroll
                for (int q = 0; q < 4; ++q) x[q] = ld_act(hq + 32 * q);
                hq += 2 * kTileK;
            }
            const uint32_t w_lo = ring + (uint32_t)g * 128u;
            int stage = 0;
            for (int i = 0; i < cw_n; ++i) {
                uint4 nx[4] = {zero4, zero4, zero4, zero4};
                if (i + 1 < cw_n && hq) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) nx[q] = ld_act(hq + 32 * q);
                    hq += 2 * kTileK;
                }
                ok = mbar_wait(bars + 8u * stage, (parity >> stage) & 1u, &abort_flag, a.status, kDfBarrierLimitNs);
                if (!ok) break;
                parity ^= 1u << stage;
                const uint32_t base = w_lo + (uint32_t)stage * kDfStageBytes;
#pragma unroll
                for (int c = 0; c < 2; ++c) {                        // the pair's two chunks: rows g and g + 8 of each
                    const uint32_t lo = base + (uint32_t)c * 2048u, hi = lo + 1024u;
                    const uint4 w00 = ld_shared_v4(lo + piece0), w01 = ld_shared_v4(lo + piece1);
                    const uint4 w10 = ld_shared_v4(hi + piece0), w11 = ld_shared_v4(hi + piece1);
                    mma_16816(acc, w00.x, w10.x, w00.y, w10.y, x[2 * c].x, x[2 * c].y);
                    mma_16816(acc, w00.z, w10.z, w00.w, w10.w, x[2 * c].z, x[2 * c].w);
                    mma_16816(acc, w01.x, w11.x, w01.y, w11.y, x[2 * c + 1].x, x[2 * c + 1].y);
                    mma_16816(acc, w01.z, w11.z, w01.w, w11.w, x[2 * c + 1].z, x[2 * c + 1].w);
                }
                __syncwarp();
                if (cw_left > 0) request_pair(stage);
                if (++stage == n_st) stage = 0;
#pragma unroll
                for (int q = 0; q < 4; ++q) x[q] = nx[q];
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) red[warp][i][lane] = acc[i];
        __syncthreads();
        if (abort_flag || (int)blockIdx.x >= (a.d >> 4)) return ok && !abort_flag;
        // Merge: thread (token, column) adds the token's experts in slot order, shared experts last (the combine
        // kernel's arithmetic); an expert's value is the sum of its warps' partial tiles in warp order.  Accumulator
        // fragment: element 2 * (column / 8) + (row & 1) of lane 4 * (column & 7) + row / 2, row = the token's row
        // inside the expert's segment.
        for (int o = tid; o < a.T * 16; o += kDfThreads) {
            const int tok = o >> 4, c = o & 15, col = (int)blockIdx.x * 16 + c;
            auto value = [&](int e, int r) -> float {
                int ai = 0;
                while (sm.act[ai] != e) ++ai;
                const int ln = (c & 7) * 4 + (r >> 1), fi = (c >> 3) * 2 + (r & 1);
                float v = red[ai * cw_ks][fi][ln];
                for (int q = 1; q < cw_ks; ++q) v += red[ai * cw_ks + q][fi][ln];
                a.y_packed[(size_t)(sm.offsets[e] + r) * a.d + col] = v;
                return v;
            };
            float s = 0.f;
            for (int jj = 0; jj < a.k; ++jj) {
                const int e = sm.idx[tok * a.k + jj];
                if (tab.slot[e] < 0) continue;
                s = fmaf(sm.w[tok * a.k + jj], value(e, sm.inv[tok * a.k + jj] - sm.offsets[e]), s);
            }
            for (int sh = 0; sh < a.S; ++sh)
                if (tab.slot[a.E + sh] >= 0) s += value(a.E + sh, tok);
            const size_t at = (size_t)tok * a.d + col;
            if (a.out_bf16) reinterpret_cast<__nv_bfloat16*>(a.out)[at] = __float2bfloat16_rn(s);
            else reinterpret_cast<float*>(a.out)[at] = s;
        }
        return ok;
    };

    // ================================ phase A: gate/up + SiLU*mul ================================
    if (phase_mask & 1) {
        const int KC = a.d / kTileK, upe = a.f / 16;
        const WarpWork ww = deal_units(n_active * upe, KC, warp);
        if (lane == 0) head_units[0][warp] = -1;
        stream(Unit<0>(), ww, KC, upe, finish_a, 0, head_units[0], [&]() { if (phase_mask & 2) prefetch_b(); });
    }

    // ================================ phase B: down + merge ================================
    if (phase_mask & 2) {
        if (!(phase_mask & 1)) prefetch_b();
        bool ok = true;
        if (phase_mask == 3) {
            // Grid barrier: every h store of phase A is visible device-wide before anyone reads h.  The CTA's
            // stores are ordered before thread 0's release by the CTA barrier (release / acquire are cumulative).
            // The arrival counter only ever grows: G arrivals per launch, so this launch is complete when the
            // counter reaches the next multiple of G above what thread 0 saw when the kernel started.
            __syncthreads();
            if (tid == 0) {
                int good = abort_flag ? 0 : 1;
                unsigned long long* counter = reinterpret_cast<unsigned long long*>(a.sync);
                asm volatile("red.release.gpu.global.add.u64 [%0], 1;" ::"l"(counter) : "memory");
                const unsigned long long target = barrier_target;
                unsigned long long t0 = 0;
                for (uint32_t i = 0;; ++i) {
                    unsigned long long c;
                    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(c) : "l"(counter) : "memory");
                    if (c >= target) break;
                    if ((i & 255u) == 255u) {
                        const unsigned long long now = globaltimer_ns();
                        if (t0 == 0) t0 = now;
                        else if (now - t0 > kDfBarrierLimitNs) { good = 0; atomicExch(a.status, SAEM_ERR_TIMEOUT); break; }
                    }
                }
                barrier_ok = good;
            }
            __syncthreads();
            ok = barrier_ok != 0;
        } else {
            pdl_wait();                                // h is complete from here on
            pdl_launch_dependents();
        }
        if (ok) {
            if (columns_b) {
                columns_phase_b();
            } else {
                if (blockIdx.x == 0) {                 // a token without any resident expert gets no ticket: its output is zero
                    for (int tok = 0; tok < a.T; ++tok) {
                        if (sm.need[tok] > 0) continue;
                        for (int c = tid; c < a.d; c += kDfThreads) {
                            if (a.out_bf16) reinterpret_cast<__nv_bfloat16*>(a.out)[(size_t)tok * a.d + c] = __float2bfloat16_rn(0.f);
                            else reinterpret_cast<float*>(a.out)[(size_t)tok * a.d + c] = 0.f;
                        }
                    }
                }
                stream(Unit<1>(), ww_b, KC_b, upe_b, finish_b, requested_b, head_units[1], []() {});
            }
        }
    }
    // Copies still in flight (a wait that ran out, a barrier that was not met) must land before the CTA's shared
    // memory goes away.
    if (abort_flag || (phase_mask == 3 && !barrier_ok)) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) {}
    }
}

bool decode_fused_supported(int T, int k) { return T >= 1 && T <= kDfMaxTokens && k <= kDfMaxK; }

// mode per device: 0 not decided, 1 cooperative + programmatic serialization, 2 cooperative, 3 two launches
static int g_mode[64];

static cudaError_t launch_step(const DecodeArgs& a, const SlotTable& tab, int grid, cudaStream_t st, int phase_mask,
                               bool cooperative, bool pdl) {
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (pdl) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (cooperative) {
        attr[n].id = cudaLaunchAttributeCooperative;
        attr[n].val.cooperative = 1;
        ++n;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kDfThreads);
    cfg.dynamicSmemBytes = kDfRingBytes;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, decode_step_kernel, a, tab, phase_mask);
}

cudaError_t launch_decode_fused(const DecodeArgs& a, const SlotTable& tab, int n_sm, cudaStream_t st, int* n_launch) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    static bool attr_done[64];
    if (first_call_on_device(attr_done)) {
        e = cudaFuncSetAttribute(decode_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDfRingBytes);
        if (e != cudaSuccess) return e;
        int coop = 0, per_sm = 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) coop = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_step_kernel, kDfThreads, kDfRingBytes) != cudaSuccess)
            per_sm = 0;
        g_mode[dev] = (coop && per_sm >= 1) ? 0 : 3;
    }
    const int grid = n_sm;                     // one CTA per SM
    if (g_mode[dev] == 0) {                    // first step on this device: find out what the driver accepts
        e = launch_step(a, tab, grid, st, 3, true, true);
        if (e == cudaSuccess) { g_mode[dev] = 1; *n_launch = 1; return e; }
        (void)cudaGetLastError();
        e = launch_step(a, tab, grid, st, 3, true, false);
        if (e == cudaSuccess) { g_mode[dev] = 2; *n_launch = 1; return e; }
        (void)cudaGetLastError();
        g_mode[dev] = 3;
    }
    if (g_mode[dev] == 1 || g_mode[dev] == 2) {
        *n_launch = 1;
        return launch_step(a, tab, grid, st, 3, true, g_mode[dev] == 1);
    }
    e = launch_step(a, tab, grid, st, 1, false, true);
    if (e != cudaSuccess) return e;
    *n_launch = 2;
    return launch_step(a, tab, grid, st, 2, false, true);
}

int decode_fused_mode() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    return g_mode[dev];
}

}  // namespace saem
