// Grouped SwiGLU expert FFN for large segments on CTA PAIRS (Sec. IV-E: one dense batched execution
// per expert over its contiguous rows).  Same contraction as ffn_prefill.cu, different machine
// mapping: the two CTAs of a cluster (two SMs of one TPC) run ONE tcgen05.mma.cta_group::2 of
// 256 tokens x 256 weight rows together.
//
//   * Why pairs.  With one SM per tile, a 256 x 256 tile needs 64 KB of operands per 1024 tensor
//     clocks; three such stages fit in shared memory, and when the loads take about two
//     microseconds (weights arriving from HBM next to L2 hits) the MMA waits for data 40 % of the
//     time.  In a pair each CTA loads its own 128 tokens (A) but only HALF of the weight rows (B);
//     the hardware reads the other half from the partner's shared memory.  An item here is
//     256 tokens x 512 weight rows (two weight blocks): 48 KB of operands per CTA for the same 1024
//     clocks, four stages instead of three.
//   * Item: (expert, pair of weight blocks, 256-token tile), dealt round-robin to the pairs with
//     the token tile fastest, so the pairs that run together share weight blocks through L2.
//     CTA r of the pair owns tokens [128 r, 128 r + 128) of the tile; its accumulators (one
//     256-column unit per weight block, 512 TMEM columns in all) hold those tokens' outputs, so the
//     epilogue is the single-CTA one: drain to registers, release, SiLU*mul (gate/up) or nothing
//     (down), stage in shared memory, TMA tile store; ragged last rows are stored directly.
//   * For gate/up a weight block is one f-block: CTA 0 holds its gate tile, CTA 1 its up tile, so
//     gate lands in accumulator columns 0..127 and up in 128..255 as in the single-CTA kernel.
//     For the down projection a weight block is two adjacent 128-row d-blocks, one per CTA.
//   * Barriers.  full[stage] lives in the leader (CTA 0): its copy warp arms it with the byte count
//     of both CTAs and both CTAs' TMA loads complete on it (cp.async.bulk.tensor ... cta_group::2,
//     no multicast).  empty[stage] and acc_full[unit] exist in both CTAs and are signalled in both
//     by one multicast tcgen05.commit.  acc_empty[unit] lives in the leader; the partner's
//     epilogue warps arrive on it remotely.  Every wait is bounded; the kernel ends with a
//     cluster barrier so that neither CTA leaves while the other may still touch its memory.
//   * Weights are fetched with a tensor map that views the slot region as rows of 128 bytes
//     (a box of 128 rows is one packed, pre-swizzled 16 KB tile, copied verbatim): the untiled bulk
//     copy cannot signal a barrier in the other CTA.
#include "tc_common.cuh"

namespace saem {

constexpr int kPrThreads = 320;            // warp 0 copies, warp 1 MMA (leader only), warps 2..9 epilogue
constexpr int kPrStage = 3 * kTileBytes;   // this CTA's half of two weight blocks + its 128 tokens x 64 k
constexpr int kPrStages = 4;
constexpr int kPrStageArea = kPrStages * kPrStage;
constexpr int kPrStoreBuf = 2048;          // per epilogue warp: 32 rows x 64 bytes on their way out
constexpr int kPrSmem = kPrStageArea + 8 * kPrStoreBuf + 1024;

struct PrPlan {
    int n_active;
    int total_items;
    int slot[SAEM_MAX_EXPERTS];
    int row0[SAEM_MAX_EXPERTS];
    int rows[SAEM_MAX_EXPERTS];
    int item_base[SAEM_MAX_EXPERTS + 1];
};

struct PrItem {
    int a, pb, mb;
    int row_start, rows_here;
    int n_wb;               // weight blocks in this item (2, or 1 for the odd last one)
};

// item -> (active expert, pair of weight blocks, 256-token tile); token tile fastest
__device__ __forceinline__ void pr_decode(const PrPlan& plan, int it, int& cursor, int WB, PrItem& o) {
    while (cursor + 1 < plan.n_active && plan.item_base[cursor + 1] <= it) ++cursor;
    o.a = cursor;
    const int local = it - plan.item_base[cursor];
    const int m_blocks = (plan.rows[cursor] + 255) >> 8;
    o.pb = local / m_blocks;
    o.mb = local - o.pb * m_blocks;
    o.row_start = plan.row0[cursor] + o.mb * 256;
    const int left = plan.rows[cursor] - o.mb * 256;
    o.rows_here = left < 256 ? left : 256;
    o.n_wb = 2 * o.pb + 1 < WB ? 2 : 1;
}

// PHASE 0: h = silu(x Wg^T) * (x Wu^T);  PHASE 1: y = h Wd^T
template <int PHASE>
__global__ void __launch_bounds__(kPrThreads, 1)
ffn_pair_kernel(FfnArgs a, const __grid_constant__ SlotTable tab, const __grid_constant__ CUtensorMap act_map,
                const __grid_constant__ CUtensorMap act_map128, const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap out_map) {
    extern __shared__ uint8_t dyn_smem[];
    __shared__ PrPlan plan;
    __shared__ __align__(8) uint64_t bar_full[kPrStages], bar_empty[kPrStages], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    __shared__ int s_warp_act[kPrThreads / 32], s_warp_t2[kPrThreads / 32];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();          // 0: leader (issues the MMAs)
    const int K = PHASE == 0 ? a.d : a.f;
    const int KC = K / kTileK;
    // weight blocks of 256 output columns: gate/up -> one f-block (gate tile + up tile); down -> two d-blocks
    const int WB = PHASE == 0 ? a.f / kTileRows : a.d / (2 * kTileRows);
    const int PB = (WB + 1) / 2;
    const uint32_t smem_base = (smem_u32(dyn_smem) + 1023u) & ~1023u;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < kPrStages; ++s) { mbar_init(smem_u32(&bar_full[s]), 1); mbar_init(smem_u32(&bar_empty[s]), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&bar_acc_full[s]), 1); mbar_init(smem_u32(&bar_acc_empty[s]), 16); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync_all();            // barriers of both CTAs exist before anyone arrives remotely
    tc_fence_after();
    pdl_wait();
    pdl_launch_dependents();

    // ---- plan (one thread per expert, block-wide prefix sums); identical in both CTAs ----
    {
        const int e = tid;
        int rows = 0, r0 = 0;
        if (e < a.E) {
            int r1 = a.max_rows;
            if (a.offsets) { r0 = a.offsets[e]; r1 = a.offsets[e + 1]; }
            if (r1 > a.max_rows) r1 = a.max_rows;
            rows = r1 > r0 ? r1 - r0 : 0;
            if (!tab.in_subset[e]) rows = 0;
            if (rows > 0 && tab.slot[e] < 0) {
                if (blockIdx.x == 0) atomicExch(a.status, SAEM_ERR_NOT_RESIDENT);
                rows = 0;
            }
        }
        const int t2 = rows > 0 ? (rows + 255) >> 8 : 0;
        int act_inc = rows > 0 ? 1 : 0, t2_inc = t2;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int na = __shfl_up_sync(0xffffffffu, act_inc, o), n2 = __shfl_up_sync(0xffffffffu, t2_inc, o);
            if (lane >= o) { act_inc += na; t2_inc += n2; }
        }
        if (lane == 31) { s_warp_act[warp] = act_inc; s_warp_t2[warp] = t2_inc; }
        __syncthreads();
        int base_act = 0, base_t2 = 0, tot_act = 0, tot_t2 = 0;
#pragma unroll
        for (int w = 0; w < kPrThreads / 32; ++w) {
            if (w < warp) { base_act += s_warp_act[w]; base_t2 += s_warp_t2[w]; }
            tot_act += s_warp_act[w];
            tot_t2 += s_warp_t2[w];
        }
        if (rows > 0) {
            const int n = base_act + act_inc - 1;
            plan.slot[n] = tab.slot[e];
            plan.row0[n] = r0;
            plan.rows[n] = rows;
            plan.item_base[n] = (base_t2 + t2_inc - t2) * PB;
        }
        if (tid == 0) {
            plan.item_base[tot_act] = tot_t2 * PB;
            plan.n_active = tot_act;
            plan.total_items = tot_t2 * PB;
        }
        __syncthreads();
    }
    const uint32_t tmem_base = tmem_base_s;
    const int total_items = plan.total_items;
    const int NC = gridDim.x >> 1, cid = blockIdx.x >> 1;      // pairs in the grid, this pair
    volatile int* abort_p = &abort_flag;

    if (warp == 0) {
        // =============================== copy warp (both CTAs) ===============================
        int stage = 0, cursor = 0;
        uint32_t phase = 0;
        bool ok = true;
        int issued = 0;
        PrItem it;
        for (int item = cid; ok && item < total_items; item += NC) {
            pr_decode(plan, item, cursor, WB, it);
            // this CTA's tiles, as row numbers of the 128-byte-row view of the slot region
            const size_t slot_off = (size_t)plan.slot[it.a] * a.slot_bytes;
            int w_row[2], w_row_step;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int wb = 2 * it.pb + j;
                const size_t off = PHASE == 0 ? slot_off + ((size_t)wb * KC) * (2 * kTileBytes) + (size_t)rank * kTileBytes
                                              : slot_off + (size_t)2 * a.d * a.f * 2 + ((size_t)(2 * wb + (int)rank) * KC) * kTileBytes;
                w_row[j] = (int)(off >> 7);
            }
            w_row_step = PHASE == 0 ? (2 * kTileBytes) >> 7 : kTileBytes >> 7;
            const int my_rows = it.rows_here - 128 * (int)rank;                    // valid tokens of this CTA's half
            const int n_boxes = my_rows <= 0 ? 0 : (my_rows >= 128 ? 4 : (my_rows + 31) >> 5);
            // bytes of BOTH CTAs per stage: the leader alone arms the barrier (the partner's copies may
            // complete on it first; a transaction count may run negative inside a phase)
            const uint32_t bytes = 2u * (uint32_t)it.n_wb * kTileBytes + (uint32_t)((it.rows_here + 31) >> 5) * 4096u;
            for (int kc = 0; kc < KC; ++kc) {
                ok = mbar_wait(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_p, a.status);
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t full = mapa_u32(smem_u32(&bar_full[stage]), 0);     // the leader's barrier
                    const uint32_t ws = smem_base + (uint32_t)stage * kPrStage;
                    if (rank == 0) mbar_expect_tx(smem_u32(&bar_full[stage]), bytes);
                    for (int j = 0; j < it.n_wb; ++j)
                        tma_2d_pair(ws + (uint32_t)j * kTileBytes, &w_map, 0, w_row[j] + kc * w_row_step, full);
                    if (n_boxes == 4) {     // a whole 128-token tile in one copy
                        tma_2d_pair(ws + 2u * kTileBytes, &act_map128, kc * kTileK, it.row_start + 128 * (int)rank, full);
                    } else {
                        for (int b = 0; b < n_boxes; ++b)
                            tma_2d_pair(ws + 2u * kTileBytes + (uint32_t)b * 4096u, &act_map, kc * kTileK,
                                        it.row_start + 128 * (int)rank + b * 32, full);
                    }
                }
                ++issued;
                if (++stage == kPrStages) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok && issued > 0) {     // let copies already in flight land before the CTA's memory goes away
            unsigned long long t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 200000ull) {}
        }
    } else if (warp == 1) {
        // =============================== MMA issuer (leader CTA only) ===============================
        if (rank == 0) {
            int stage = 0, acc = 0, cursor = 0;
            uint32_t phase = 0, acc_phase[2] = {0u, 0u};
            bool ok = true;
            PrItem it;
            const uint32_t idesc = idesc_bf16_pair(256);
            for (int item = cid; ok && item < total_items; item += NC) {
                pr_decode(plan, item, cursor, WB, it);
                const int acc0 = acc, acc1 = acc ^ 1;             // accumulator units of the item's first / second weight block
                for (int kc = 0; ok && kc < KC; ++kc) {
                    ok = mbar_wait_cluster(smem_u32(&bar_full[stage]), phase, abort_p, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t ws = smem_base + (uint32_t)stage * kPrStage;
                    const uint32_t xs = ws + 2u * kTileBytes;
                    for (int j = 0; j < it.n_wb; ++j) {
                        const int ac = j == 0 ? acc0 : acc1;
                        if (kc == 0) {      // both CTAs' epilogues must have drained this unit
                            ok = mbar_wait_cluster(smem_u32(&bar_acc_empty[ac]), acc_phase[ac] ^ 1u, abort_p, a.status);
                            if (!ok) break;
                            tc_fence_after();
                        }
                        if (lane == 0) {
                            const uint32_t d_tmem = tmem_base + (uint32_t)(ac * 256);
#pragma unroll
                            for (int k4 = 0; k4 < kTileK / 16; ++k4)
                                tc_mma_bf16_pair(d_tmem, smem_desc_sw128(xs + k4 * 32),
                                                 smem_desc_sw128(ws + (uint32_t)j * kTileBytes + k4 * 32), idesc,
                                                 (kc > 0 || k4 > 0) ? 1u : 0u);
                        }
                    }
                    if (!ok) break;
                    if (lane == 0) tc_commit_pair(smem_u32(&bar_empty[stage]));
                    __syncwarp();
                    if (++stage == kPrStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (lane == 0) {
                    tc_commit_pair(smem_u32(&bar_acc_full[acc0]));
                    if (it.n_wb == 2) tc_commit_pair(smem_u32(&bar_acc_full[acc1]));
                }
                __syncwarp();
                acc_phase[acc0] ^= 1u;
                if (it.n_wb == 2) acc_phase[acc1] ^= 1u;
                else acc ^= 1;                                    // a one-block item takes one unit of the ring
            }
        }
    } else {
        // =============================== epilogue (warps 2..9, both CTAs) ===============================
        const int q = warp & 3;                 // TMEM lane quarter = token rows 32q .. 32q+31 of this CTA's 128
        const int half = (warp - 2) >> 2;       // which half of the unit's columns
        const int i = q * 32 + lane;
        const uint32_t store_buf = smem_base + (uint32_t)kPrStageArea + (uint32_t)(warp - 2) * kPrStoreBuf;
        const uint32_t my_buf = store_buf + (uint32_t)lane * 64u;
        const uint32_t sw = (uint32_t)((lane >> 1) & 3);
        int acc = 0, cursor = 0;
        uint32_t acc_phase[2] = {0u, 0u};
        bool ok = true;
        PrItem it;
        for (int item = cid; ok && item < total_items; item += NC) {
            pr_decode(plan, item, cursor, WB, it);
            for (int j = 0; ok && j < it.n_wb; ++j) {
                const int ac = j == 0 ? acc : acc ^ 1;
                const int wb = 2 * it.pb + j;
                ok = mbar_wait(smem_u32(&bar_acc_full[ac]), acc_phase[ac], abort_p, a.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ac * 256);
                uint32_t v[128];
                tc_ld32_issue(t_row + (uint32_t)(PHASE == 0 ? half * 64 : half * 128), v);
                tc_ld32_issue(t_row + (uint32_t)(PHASE == 0 ? half * 64 + 32 : half * 128 + 32), v + 32);
                tc_ld32_issue(t_row + (uint32_t)(PHASE == 0 ? 128 + half * 64 : half * 128 + 64), v + 64);
                tc_ld32_issue(t_row + (uint32_t)(PHASE == 0 ? 128 + half * 64 + 32 : half * 128 + 96), v + 96);
                tc_wait_ld();
#pragma unroll
                for (int g16 = 0; g16 < 8; ++g16) tc_reg_fence16(v + 16 * g16);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(mapa_u32(smem_u32(&bar_acc_empty[ac]), 0));
                acc_phase[ac] ^= 1u;

                const int r = 128 * (int)rank + i;                            // token row inside the 256-token tile
                const bool valid = r < it.rows_here;
                const bool full_box = 128 * (int)rank + q * 32 + 32 <= it.rows_here;
                const int box_row = it.row_start + 128 * (int)rank + q * 32;
                const size_t row = (size_t)(it.row_start + r);
                if (PHASE == 0) {
                    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.h) + row * a.f + (size_t)wb * kTileRows + half * 64;
#pragma unroll
                    for (int bx = 0; bx < 2; ++bx) {          // two boxes of 32 h columns
                        uint32_t pk[16];
#pragma unroll
                        for (int n = 0; n < 16; ++n) {
                            const float g0 = __uint_as_float(v[32 * bx + 2 * n]), g1 = __uint_as_float(v[32 * bx + 2 * n + 1]);
                            const float u0 = __uint_as_float(v[64 + 32 * bx + 2 * n]), u1 = __uint_as_float(v[64 + 32 * bx + 2 * n + 1]);
                            const float h0 = __fdividef(g0, 1.f + __expf(-g0)) * u0;
                            const float h1 = __fdividef(g1, 1.f + __expf(-g1)) * u1;
                            __nv_bfloat162 p2 = __floats2bfloat162_rn(h0, h1);
                            pk[n] = *reinterpret_cast<uint32_t*>(&p2);
                        }
                        if (full_box) {
                            if (lane == 0) bulk_wait_read();
                            __syncwarp();
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                st_shared_v4(my_buf + ((((uint32_t)c) ^ sw) << 4), pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                            fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0) {
                                tma_store_2d(&out_map, wb * kTileRows + half * 64 + 32 * bx, box_row, store_buf);
                                bulk_commit();
                            }
                        } else if (valid) {
                            uint4* o = reinterpret_cast<uint4*>(dst + 32 * bx);
#pragma unroll
                            for (int c = 0; c < 4; ++c) o[c] = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                        }
                    }
                } else {
                    float* dst = a.y_packed + row * a.d + (size_t)wb * 256 + half * 128;
#pragma unroll
                    for (int bx = 0; bx < 8; ++bx) {          // boxes of 16 y columns
                        if (full_box) {
                            if (lane == 0) bulk_wait_read();
                            __syncwarp();
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                st_shared_v4(my_buf + ((((uint32_t)c) ^ sw) << 4), v[16 * bx + 4 * c], v[16 * bx + 4 * c + 1],
                                             v[16 * bx + 4 * c + 2], v[16 * bx + 4 * c + 3]);
                            fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0) {
                                tma_store_2d(&out_map, wb * 256 + half * 128 + 16 * bx, box_row, store_buf);
                                bulk_commit();
                            }
                        } else if (valid) {
                            uint4* o = reinterpret_cast<uint4*>(dst + 16 * bx);
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                o[c] = make_uint4(v[16 * bx + 4 * c], v[16 * bx + 4 * c + 1], v[16 * bx + 4 * c + 2], v[16 * bx + 4 * c + 3]);
                        }
                    }
                }
            }
            if (it.n_wb == 1) acc ^= 1;
        }
        if (lane == 0) bulk_wait_all();         // this warp's tile stores have landed
    }

    // ---- teardown: neither CTA leaves (or frees TMEM) while the other may still touch it ----
    tc_fence_before();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
    }
}

// ------------------------------------------------------------------------------------------- host
static bool g_pr_init[64];

cudaError_t launch_ffn_pair(const FfnArgs& a, const SlotTable& tab, const CUtensorMap& map_x, const CUtensorMap& map_h,
                            const CUtensorMap& map_x128, const CUtensorMap& map_h128, const CUtensorMap& map_w, const CUtensorMap& map_h_store, const CUtensorMap& map_y_store,
                            cudaStream_t st, int* n_launch) {
    if (first_call_on_device(g_pr_init)) {
        cudaError_t e = cudaFuncSetAttribute(ffn_pair_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrSmem);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(ffn_pair_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrSmem);
        if (e != cudaSuccess) return e;
    }
    const dim3 grid((unsigned)(a.n_sm & ~1)), block(kPrThreads);
    cudaError_t e = launch_pdl_pairs(ffn_pair_kernel<0>, grid, block, (size_t)kPrSmem, st, a, tab, map_x, map_x128, map_w, map_h_store);
    if (e != cudaSuccess) return e;
    e = launch_pdl_pairs(ffn_pair_kernel<1>, grid, block, (size_t)kPrSmem, st, a, tab, map_h, map_h128, map_w, map_y_store);
    *n_launch = 2;
    return e;
}

}  // namespace saem
