// The whole MoE layer step for the smallest decode batches (at most 8 tokens, top-k at most 8) in
// two launches instead of five.  At batch 1-8 the step moves a few tens of megabytes, so a launch's
// fixed cost (start-up, finding the active experts, the last partial wave) is as large as its
// streaming time; the paper's operating point is exactly this regime (batch 1-8 decode).
//
//   decode_gateup_kernel        every CTA repeats the tiny gate (top-k of E logits for <= 8 tokens,
//                               Background "Mixture-of-Experts Inference") and the expert-aligned
//                               repack indices (Sec. IV-E: counts, exclusive scan, stable
//                               permutation) in its own shared memory, then streams its share of the
//                               ACTIVE experts' gate/up rows and writes h = silu(Wg x) * (Wu x).
//                               Token rows are read straight from x through the permutation: no
//                               x_packed round trip.  CTA 0 also writes the index outputs, so they
//                               stay inspectable and bit-exact.
//   decode_down_combine_kernel  a CTA owns 16 output columns for ALL active experts: it streams those
//                               16 rows of every active expert's down matrix, keeps the per-pair
//                               results in shared memory and merges them per token in slot order
//                               j = 0..k-1, shared experts last (Sec. IV-D merge; deterministic, no
//                               atomics): no y_packed round trip and no combine launch.  It repeats
//                               the gate from the logits itself and starts streaming weights BEFORE
//                               it waits for the first kernel (programmatic dependent launch), so its
//                               start-up hides behind the first kernel's tail.
//
// Both kernels are shaped by bytes (decode is weight streaming): 16-byte loads of the packed slot
// layout's 128-byte tile rows, mma.sync m16n8k16 as the arithmetic unit (16 weight rows x up to 8
// tokens), fp32 accumulation, fixed summation orders.  The second kernel keeps a deep queue of loads
// in flight without spending registers on it: every warp owns a ring of shared-memory stages that
// its lanes fill with cp.async (each lane copies exactly the bytes its own MMA fragments need, so no
// barrier is involved), because with one CTA per 16 output columns there are only d_model / 16 CTAs.
#include <cuda_bf16.h>

#include "route_row.cuh"

namespace saem {

constexpr int kDfMaxTokens = 8;
constexpr int kDfMaxK = 8;
constexpr int kDfMaxPairs = kDfMaxTokens * kDfMaxK;
constexpr int kDfMaxRows = kDfMaxTokens * (kDfMaxK + 16);      // pair rows, then T rows per shared expert
constexpr int kDfThreadsA = 256;
constexpr int kDfWarpsA = kDfThreadsA / 32;
constexpr int kDfRows = 16;                                    // weight rows per MMA

struct DecodeIndex {
    int32_t idx[kDfMaxPairs];
    float w[kDfMaxPairs];
    int32_t perm[kDfMaxPairs];
    int32_t inv[kDfMaxPairs];
    int32_t counts[SAEM_MAX_EXPERTS];
    int32_t offsets[SAEM_MAX_EXPERTS + 1];
    int16_t act[SAEM_MAX_EXPERTS];          // experts with rows, ascending id
    int n_active;
};

__device__ __forceinline__ void mma_16816(float* c, const uint32_t a0, const uint32_t a1, const uint32_t a2,
                                          const uint32_t a3, const uint32_t b0, const uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Gate and repack indices of the whole (tiny) batch in shared memory; every thread of the CTA calls
// it (at least 8 warps).  Same arithmetic and tie rules as route_kernel / the repack kernels: slots
// in descending logit order, segments in ascending expert id, ascending pair id inside a segment,
// one segment of all T tokens per in-layer shared expert behind the T*k pair rows.
__device__ __forceinline__ void build_index(const DecodeArgs& a, DecodeIndex& sm) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int P = a.T * a.k, ES = a.E + a.S;
    if (warp < a.T)
        route_row(a.logits + (size_t)warp * a.E, a.E, a.k, a.renorm, lane, &sm.idx[warp * a.k], &sm.w[warp * a.k]);
    __syncthreads();
    if (tid < ES) {
        int c = a.T;
        if (tid < a.E) {
            c = 0;
            for (int p = 0; p < P; ++p) c += sm.idx[p] == tid ? 1 : 0;
        }
        sm.counts[tid] = c;
    }
    __syncthreads();
    if (warp == 0) {
        int carry = 0, carry_act = 0;
        for (int base = 0; base < ES; base += 32) {
            const int e = base + lane;
            const int v = e < ES ? sm.counts[e] : 0;
            int inc = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += n;
            }
            const unsigned actm = __ballot_sync(0xffffffffu, v > 0);
            if (e < ES) sm.offsets[e] = carry + inc - v;
            if (v > 0) sm.act[carry_act + __popc(actm & ((1u << lane) - 1u))] = (int16_t)e;
            carry += __shfl_sync(0xffffffffu, inc, 31);
            carry_act += __popc(actm);
        }
        if (lane == 0) { sm.offsets[ES] = carry; sm.n_active = carry_act; }
    }
    __syncthreads();
    if (tid < P) {
        const int e = sm.idx[tid];
        int rank = 0;
        for (int q = 0; q < tid; ++q) rank += sm.idx[q] == e ? 1 : 0;
        const int r = sm.offsets[e] + rank;
        sm.perm[r] = tid;
        sm.inv[tid] = r;
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------ gate/up + SiLU*mul
// Work unit: gpc consecutive 16-row groups of one active expert's gate and up matrices over the whole
// reduction length d_model (gpc > 1 when d_model is short, so that a unit still moves tens of KB).
// The 8 warps of a CTA split the unit's k-chunks; their partial tiles are added in warp order.
__global__ void __launch_bounds__(kDfThreadsA, 3)
decode_gateup_kernel(DecodeArgs a, const __grid_constant__ SlotTable tab, int gpc) {
    __shared__ DecodeIndex sm;
    __shared__ float red[kDfWarpsA][2][kDfRows][kDfMaxTokens];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_wait();                       // logits and x may come from the kernel before
    pdl_launch_dependents();
    build_index(a, sm);
    const int P = a.T * a.k, ES = a.E + a.S;
    if (blockIdx.x == 0) {            // the index outputs of the step, for the caller and for inspection
        for (int p = tid; p < P; p += kDfThreadsA) {
            a.topk_idx[p] = sm.idx[p];
            a.topk_w[p] = sm.w[p];
            a.perm[p] = sm.perm[p];
            a.inv_perm[p] = sm.inv[p];
        }
        for (int e = tid; e < ES; e += kDfThreadsA) a.counts[e] = sm.counts[e];
        for (int e = tid; e <= ES; e += kDfThreadsA) a.offsets[e] = sm.offsets[e];
    }

    const int KC = a.d / kTileK;
    const int units_per_expert = a.f / kDfRows / gpc;
    const int total_units = sm.n_active * units_per_expert;
    const int wpg = kDfWarpsA / gpc;              // warps per row group
    const int grp = warp % gpc, kslice = warp / gpc;
    const int g = lane >> 2, t = lane & 3;        // MMA fragment coordinates
    for (int unit = blockIdx.x; unit < total_units; unit += gridDim.x) {
        const int ai = unit / units_per_expert, cb = unit - ai * units_per_expert;
        const int e = sm.act[ai];
        const int slot = tab.slot[e];
        if (slot < 0) {                            // routed to an expert that has no slot: rows left untouched
            if (cb == 0 && tid == 0) atomicExch(a.status, SAEM_ERR_NOT_RESIDENT);
            continue;
        }
        const int row0 = sm.offsets[e], m = sm.counts[e];
        const int rg = cb * gpc + grp;
        const int rb = rg >> 3, r_in = (rg & 7) * kDfRows;
        const uint8_t* wbase = a.slot_region + (size_t)slot * a.slot_bytes + (size_t)rb * KC * (2 * kTileBytes);
        // byte offset of this lane's 16-byte chunk (k positions 4 b + t) in tile rows r_in + g and r_in + g + 8
        const uint32_t off_lo0 = (uint32_t)(r_in + g) * 128u + (uint32_t)((t ^ g) << 4);
        const uint32_t off_lo1 = (uint32_t)(r_in + g) * 128u + (uint32_t)(((4 + t) ^ g) << 4);
        const uint32_t off_hi0 = off_lo0 + 8u * 128u, off_hi1 = off_lo1 + 8u * 128u;
        const bool x_valid = g < m;
        // MMA column g is the segment's g-th row: the token of pair perm[row0 + g], or token g of a shared expert
        const int token = !x_valid ? 0 : (e < a.E ? sm.perm[row0 + g] / a.k : g);
        const uint16_t* xrow = a.x + (size_t)token * a.d + t * 8;

        float cg[4] = {0.f, 0.f, 0.f, 0.f}, cu[4] = {0.f, 0.f, 0.f, 0.f};
        for (int kc = kslice; kc < KC; kc += wpg) {
            const uint8_t* tile = wbase + (size_t)kc * (2 * kTileBytes);
            const uint4 z = make_uint4(0u, 0u, 0u, 0u);
            const uint4 wl0 = *reinterpret_cast<const uint4*>(tile + off_lo0);
            const uint4 wl1 = *reinterpret_cast<const uint4*>(tile + off_lo1);
            const uint4 wh0 = *reinterpret_cast<const uint4*>(tile + off_hi0);
            const uint4 wh1 = *reinterpret_cast<const uint4*>(tile + off_hi1);
            const uint4 ul0 = *reinterpret_cast<const uint4*>(tile + kTileBytes + off_lo0);
            const uint4 ul1 = *reinterpret_cast<const uint4*>(tile + kTileBytes + off_lo1);
            const uint4 uh0 = *reinterpret_cast<const uint4*>(tile + kTileBytes + off_hi0);
            const uint4 uh1 = *reinterpret_cast<const uint4*>(tile + kTileBytes + off_hi1);
            const uint4 x0 = x_valid ? *reinterpret_cast<const uint4*>(xrow + (size_t)kc * kTileK) : z;
            const uint4 x1 = x_valid ? *reinterpret_cast<const uint4*>(xrow + (size_t)kc * kTileK + 32) : z;
            mma_16816(cg, wl0.x, wh0.x, wl0.y, wh0.y, x0.x, x0.y);
            mma_16816(cg, wl0.z, wh0.z, wl0.w, wh0.w, x0.z, x0.w);
            mma_16816(cu, ul0.x, uh0.x, ul0.y, uh0.y, x0.x, x0.y);
            mma_16816(cu, ul0.z, uh0.z, ul0.w, uh0.w, x0.z, x0.w);
            mma_16816(cg, wl1.x, wh1.x, wl1.y, wh1.y, x1.x, x1.y);
            mma_16816(cg, wl1.z, wh1.z, wl1.w, wh1.w, x1.z, x1.w);
            mma_16816(cu, ul1.x, uh1.x, ul1.y, uh1.y, x1.x, x1.y);
            mma_16816(cu, ul1.z, uh1.z, ul1.w, uh1.w, x1.z, x1.w);
        }
        // accumulator fragment: c0,c1 -> (row g, tokens 2t, 2t+1); c2,c3 -> (row g + 8, same tokens)
        red[warp][0][g][2 * t] = cg[0];
        red[warp][0][g][2 * t + 1] = cg[1];
        red[warp][0][g + 8][2 * t] = cg[2];
        red[warp][0][g + 8][2 * t + 1] = cg[3];
        red[warp][1][g][2 * t] = cu[0];
        red[warp][1][g][2 * t + 1] = cu[1];
        red[warp][1][g + 8][2 * t] = cu[2];
        red[warp][1][g + 8][2 * t + 1] = cu[3];
        __syncthreads();
        // red[w] is the partial tile of warp w = kslice * gpc + group; a group's slices are added in order
        for (int o = tid; o < gpc * kDfRows * kDfMaxTokens; o += kDfThreadsA) {
            const int gq = o >> 7, n = (o >> 4) & 7, r = o & 15;
            if (n < m) {
                float sg = 0.f, su = 0.f;
                for (int ks = 0; ks < wpg; ++ks) {
                    sg += red[ks * gpc + gq][0][r][n];
                    su += red[ks * gpc + gq][1][r][n];
                }
                const float hv = sg / (1.f + expf(-sg)) * su;
                const size_t col = (size_t)(cb * gpc + gq) * kDfRows + r;
                reinterpret_cast<__nv_bfloat16*>(a.h)[(size_t)(row0 + n) * a.f + col] = __float2bfloat16_rn(hv);
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------- down + combine
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

constexpr int kDfStageBytes = 6 * 32 * 16;       // per warp and stage: 4 weight pieces + 2 activation pieces per lane

// One CTA per 16 output columns (16 rows of every expert's down matrix), W warps, D stages per warp.
// With fewer active experts than warps, wpe warps share an expert and split its k-chunks (their
// partial tiles are added in warp order); otherwise every warp walks its own experts a, a + W, ...
// over the whole reduction length d_ff and no partial tiles exist.
template <int W, int D>
__global__ void __launch_bounds__(W * 32, W <= 8 ? 2 : 1)
decode_down_combine_kernel(DecodeArgs a, const __grid_constant__ SlotTable tab) {
    extern __shared__ __align__(16) uint8_t ring_raw[];
    __shared__ DecodeIndex sm;
    __shared__ float y_s[kDfMaxRows][kDfRows];
    __shared__ float red[W][kDfRows][kDfMaxTokens];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // The kernel before this one in the stream (the gate/up kernel) waited for ITS predecessors
    // before it let this kernel start, so the step's inputs (logits, x) are final here and the
    // expert weights are never written by a kernel: everything up to the wait below may run while
    // the gate/up kernel is still streaming.
    for (int o = tid; o < kDfMaxRows * kDfRows; o += W * 32) (&y_s[0][0])[o] = 0.f;
    for (int o = tid; o < W * kDfRows * kDfMaxTokens; o += W * 32) (&red[0][0][0])[o] = 0.f;   // a warp may have no chunk
    build_index(a, sm);

    const int KC = a.f / kTileK;
    const int n_active = sm.n_active;
    int wpe = 1;
    while (wpe * 2 * n_active <= W) wpe *= 2;
    const int a_step = W / wpe, kslice = warp % wpe;
    const int rg = blockIdx.x, rb = rg >> 3, r_in = (rg & 7) * kDfRows;
    const int g = lane >> 2, t = lane & 3;
    const uint32_t off_lo0 = (uint32_t)(r_in + g) * 128u + (uint32_t)((t ^ g) << 4);
    const uint32_t off_lo1 = (uint32_t)(r_in + g) * 128u + (uint32_t)(((4 + t) ^ g) << 4);
    const uint32_t off_hi0 = off_lo0 + 8u * 128u, off_hi1 = off_lo1 + 8u * 128u;
    const size_t down_region = (size_t)2 * a.d * a.f * 2 + (size_t)rb * KC * kTileBytes;
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(ring_raw) + (uint32_t)(warp * D) * kDfStageBytes + (uint32_t)lane * 16u;

    // A cursor over this warp's chunk sequence: experts ai = warp / wpe, + a_step, ...; chunks kslice, + wpe, ...
    // Experts without a slot are skipped (their rows contribute zero and the status word is set).
    struct Cursor { int ai, kc; };
    auto settle = [&](Cursor& c) {               // move to the next expert that has work for this warp
        while (c.ai < n_active && (c.kc >= KC || tab.slot[sm.act[c.ai]] < 0)) { c.ai += a_step; c.kc = kslice; }
    };
    auto advance = [&](Cursor& c) { c.kc += wpe; settle(c); };
    Cursor pw = {warp / wpe, kslice};            // next chunk whose weights are to be requested
    settle(pw);
    Cursor ph = pw, cc = pw;                     // ... whose activations are to be requested; next chunk to consume

    auto issue_w = [&](const Cursor& c, int stage) {
        const uint8_t* tile = a.slot_region + (size_t)tab.slot[sm.act[c.ai]] * a.slot_bytes + down_region +
                              (size_t)c.kc * kTileBytes;
        const uint32_t dst = ring + (uint32_t)stage * kDfStageBytes;
        cp_async16(dst, tile + off_lo0, 16);
        cp_async16(dst + 512, tile + off_lo1, 16);
        cp_async16(dst + 1024, tile + off_hi0, 16);
        cp_async16(dst + 1536, tile + off_hi1, 16);
    };
    auto issue_h = [&](const Cursor& c, int stage) {
        const int e = sm.act[c.ai];
        const bool valid = g < sm.counts[e];
        const uint16_t* hrow = a.h + (size_t)(sm.offsets[e] + (valid ? g : 0)) * a.f + (size_t)c.kc * kTileK + t * 8;
        const uint32_t dst = ring + (uint32_t)stage * kDfStageBytes;
        cp_async16(dst + 2048, hrow, valid ? 16u : 0u);          // lanes beyond the segment's rows: zero fill
        cp_async16(dst + 2560, hrow + 32, valid ? 16u : 0u);
    };

    // weights of the first D chunks go out before the dependency wait
#pragma unroll
    for (int s = 0; s < D; ++s) {
        if (pw.ai < n_active) { issue_w(pw, s); advance(pw); }
        cp_async_commit();
    }
    pdl_wait();                                  // h is complete from here on
    pdl_launch_dependents();
#pragma unroll
    for (int s = 0; s < D; ++s) {
        if (ph.ai < n_active) { issue_h(ph, s); advance(ph); }
        cp_async_commit();
    }

    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    int stage = 0;
    auto flush = [&](int ai) {                   // this warp's tile of expert ai is complete
        const int e = sm.act[ai], row0 = sm.offsets[e], m = sm.counts[e];
        if (wpe == 1) {
            if (2 * t < m) { y_s[row0 + 2 * t][g] = acc[0]; y_s[row0 + 2 * t][g + 8] = acc[2]; }
            if (2 * t + 1 < m) { y_s[row0 + 2 * t + 1][g] = acc[1]; y_s[row0 + 2 * t + 1][g + 8] = acc[3]; }
        } else {
            red[warp][g][2 * t] = acc[0];
            red[warp][g][2 * t + 1] = acc[1];
            red[warp][g + 8][2 * t] = acc[2];
            red[warp][g + 8][2 * t + 1] = acc[3];
        }
        acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
    };
    while (cc.ai < n_active) {
        cp_async_wait<D - 1>();                  // the oldest outstanding stage has landed (own bytes only)
        const uint32_t src = ring + (uint32_t)stage * kDfStageBytes;
        const uint4 wl0 = ld_shared_v4(src), wl1 = ld_shared_v4(src + 512);
        const uint4 wh0 = ld_shared_v4(src + 1024), wh1 = ld_shared_v4(src + 1536);
        const uint4 x0 = ld_shared_v4(src + 2048), x1 = ld_shared_v4(src + 2560);
        mma_16816(acc, wl0.x, wh0.x, wl0.y, wh0.y, x0.x, x0.y);
        mma_16816(acc, wl0.z, wh0.z, wl0.w, wh0.w, x0.z, x0.w);
        mma_16816(acc, wl1.x, wh1.x, wl1.y, wh1.y, x1.x, x1.y);
        mma_16816(acc, wl1.z, wh1.z, wl1.w, wh1.w, x1.z, x1.w);
        const int ai_done = cc.ai;
        advance(cc);
        if (cc.ai != ai_done) flush(ai_done);
        // refill the stage just consumed (the MMAs above have read it: they issued before this point)
        if (pw.ai < n_active) { issue_w(pw, stage); issue_h(pw, stage); advance(pw); }
        cp_async_commit();
        if (++stage == D) stage = 0;
    }
    cp_async_wait<0>();
    __syncthreads();
    if (wpe > 1) {                               // add the k-slices of every expert in warp order
        for (int o = tid; o < n_active * kDfRows * kDfMaxTokens; o += W * 32) {
            const int ai = o >> 7, n = (o >> 4) & 7, r = o & 15;
            const int e = sm.act[ai];
            if (n < sm.counts[e] && tab.slot[e] >= 0) {
                float s = 0.f;
                for (int ks = 0; ks < wpe; ++ks) s += red[ai * wpe + ks][r][n];
                y_s[sm.offsets[e] + n][r] = s;
            }
        }
        __syncthreads();
    }
    if (blockIdx.x == 0 && tid < n_active && tab.slot[sm.act[tid]] < 0) atomicExch(a.status, SAEM_ERR_NOT_RESIDENT);
    // merge: slot order j = 0..k-1 with fused multiply-adds, then the shared experts with weight 1
    const int P = a.T * a.k;
    for (int o = tid; o < a.T * kDfRows; o += W * 32) {
        const int tok = o >> 4, c = o & 15;
        float s = 0.f;
        for (int j = 0; j < a.k; ++j) s = fmaf(sm.w[tok * a.k + j], y_s[sm.inv[tok * a.k + j]][c], s);
        for (int sh = 0; sh < a.S; ++sh) s += y_s[P + sh * a.T + tok][c];
        const size_t at = (size_t)tok * a.d + (size_t)rg * kDfRows + c;
        if (a.out_bf16) reinterpret_cast<__nv_bfloat16*>(a.out)[at] = __float2bfloat16_rn(s);
        else reinterpret_cast<float*>(a.out)[at] = s;
    }
}

// Row groups per unit of the gate/up kernel: enough that a unit moves about 64 KB of weights, a power
// of two that divides both the warp count and the number of row groups.
static int groups_per_unit(int rows, int K) {
    const int n_groups = rows / kDfRows;
    const long long bytes_per_group = (long long)kDfRows * K * 2 * 2;
    int gpc = 1;
    while (gpc < kDfWarpsA && bytes_per_group * gpc < 64 * 1024 && n_groups % (gpc * 2) == 0) gpc *= 2;
    return gpc;
}

bool decode_fused_supported(int T, int k) { return T >= 1 && T <= kDfMaxTokens && k <= kDfMaxK; }

cudaError_t launch_decode_fused(const DecodeArgs& a, const SlotTable& tab, int n_sm, cudaStream_t st, int* n_launch) {
    constexpr int kBigSmem = 16 * 4 * kDfStageBytes, kSmallSmem = 8 * 3 * kDfStageBytes;
    static bool attr_done[64];
    if (first_call_on_device(attr_done)) {
        cudaError_t e = cudaFuncSetAttribute(decode_down_combine_kernel<16, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kBigSmem);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(decode_down_combine_kernel<8, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmallSmem);
        if (e != cudaSuccess) return e;
    }
    const int gpc = groups_per_unit(a.f, a.d);
    const int units_per_expert = a.f / kDfRows / gpc;
    const long long bound_active = (long long)a.T * a.k + a.S < a.E + a.S ? (long long)a.T * a.k + a.S : a.E + a.S;
    long long grid_a = bound_active * units_per_expert;
    if (grid_a > 3LL * n_sm) grid_a = 3LL * n_sm;
    if (grid_a < 1) grid_a = 1;
    cudaError_t e = launch_pdl(decode_gateup_kernel, dim3((unsigned)grid_a), dim3(kDfThreadsA), 0, st, a, tab, gpc);
    if (e != cudaSuccess) return e;
    const int grid_b = a.d / kDfRows;
    // one CTA per SM with 16 warps and four stages each when the column groups fit one wave; otherwise
    // two smaller CTAs per SM
    if (grid_b <= n_sm)
        e = launch_pdl(decode_down_combine_kernel<16, 4>, dim3((unsigned)grid_b), dim3(16 * 32), (size_t)kBigSmem, st, a, tab);
    else
        e = launch_pdl(decode_down_combine_kernel<8, 3>, dim3((unsigned)grid_b), dim3(8 * 32), (size_t)kSmallSmem, st, a, tab);
    *n_launch = 2;
    return e;
}

}  // namespace saem
