// Grouped SwiGLU expert FFN for LARGE segments (prefill, big decode batches): a real dense
// contraction, so it is tiled for the tensor cores rather than for bytes (Sec. IV-E: one dense
// batched execution per expert over its contiguous rows).
//
//   * Item: 128 or 256 tokens of one expert's segment (one or two MMA M = 128 tiles that share
//     every weight stage; loaded by TMA from x_packed / h) x 256 weight rows (the N operand: for gate/up the 128 gate rows and the 128 up
//     rows of one f-block, which the packed slot layout stores back to back; for the down
//     projection two adjacent 128-row d-blocks) x 64 reduction elements per pipeline stage.
//     tcgen05.mma 128x256x16, fp32 accumulators in TMEM: 256 columns per 128-token tile, a ring
//     of two (512 columns) handed over tile by tile, so the epilogue of one tile overlaps the
//     MMAs into the other.
//   * gate and up land in the same accumulator tile (columns 0..127 and 128..255 of the same
//     token lane), so SiLU(gate)*up is a per-thread operation and h is written once, bf16.
//   * An accumulator lane is a token row, so a thread's results are 64 contiguous bytes of ONE
//     output row and a warp's direct stores would touch 32 different rows per instruction; that
//     store traffic was measured to cost a third of the down projection's time (it also delays the
//     copy warp's loads).  Each epilogue warp therefore stages its 32 rows x 64 bytes in shared
//     memory (64-byte swizzle, conflict-free) and hands them to the TMA as one tile store; only the
//     ragged last rows of a segment are stored directly, row by row.
//   * One persistent CTA per SM; whole tiles are dealt in the order (expert, weight block, token
//     tile), so the CTAs that run at the same time share a weight block and it is fetched from HBM
//     once and re-read from L2.  No tile is split, nothing is reduced across CTAs.
//   * The two launches overlap at their seam.  The gate/up launch deals its items round-robin, and
//     its last, partial round keeps a few SMs busy for one more item (an item alone on an SM is
//     bound by the latency of its K / 64 stages, not by bytes: 25 us on the Mixtral shape) while
//     all the others are done.  The down launch therefore does not wait for the whole gate/up grid
//     (programmatic dependent launch without the wait): its CTAs start on the SMs that grid has
//     left, take their items from a counter in the same order (late starters get less), and wait
//     per expert -- bounded -- for a count of that expert's completed h rows, which the gate/up
//     epilogue warps advance item by item.  Experts complete in ascending order, so only the items
//     of the last expert ever wait.  The counts are put back to zero by their last reader.  (Only
//     where it pays -- see the plan: more than one round of down items, and long segments or a
//     gate/up launch whose last round leaves at least half of the SMs idle; or a single round of
//     down items of which the last expert's are cut into single 128-column blocks, so that the
//     items that wait are not what the launch ends with.  Otherwise the down launch waits for the
//     gate/up grid as a whole.)
//   * 128 or 256 tokens per item is decided per launch on the device: a stage is released only
//     when its MMAs have completed and its refill takes about a microsecond, so with 4 x 48 KB
//     stages of 128-token items the tensor pipe idles about a third of the time; two token tiles
//     per 64 KB stage double the MMA work behind each refill (3 stages), which is faster whenever
//     the launch still has several rounds of such items per SM.
//   * Warp roles and bounded mbarrier waits as in the streaming kernel (ffn_tensor.cu).
#include "tc_common.cuh"

namespace saem {

constexpr int kPfThreads = 320;            // warp 0 copies, warp 1 MMA, warps 2..9 epilogue
constexpr int kPfStageW = 2 * kTileBytes;  // 256 weight rows x 64 k
constexpr int kPfTileX = 128 * 128;        // one 128-token tile x 64 k
constexpr int kPfMaxStages = 4;
constexpr int kPfStageArea = 4 * (kPfStageW + kPfTileX);     // = 3 x (32 KB + 2 x 16 KB) as well
constexpr int kPfStoreBuf = 2048;          // per epilogue warp: 32 rows x 64 bytes on their way out
constexpr int kPfSmem = kPfStageArea + 8 * kPfStoreBuf + 1024;
constexpr int kPfPairHalfRounds = 3;       // two tiles per item only with at least this many such items per TWO CTAs

struct PfPlan {
    int n_active;
    int total_items;
    int tpi;                // tokens per item: 128 or 256
    int seam;               // the down launch overlaps the gate/up launch's last round (both launches take the same decision)
    int half_from;          // down launch: active experts from this one on come as items of ONE 128-column block (see the plan)
    int slot[SAEM_MAX_EXPERTS];
    int eid[SAEM_MAX_EXPERTS];      // expert id of the active expert
    int row0[SAEM_MAX_EXPERTS];
    int rows[SAEM_MAX_EXPERTS];
    int item_base[SAEM_MAX_EXPERTS + 1];
};

struct PfItem {
    int a, wb, mb;
    int row_start, rows_here, n_cols;
    int n_mt;               // 128-token MMA tiles in this item (1 or 2)
};

// item -> (active expert, weight block, token tile); weight block slowest, token tile fastest.  o.wb: gate/up -> the
// f-block; down -> the item's first 128-column d-block (an item is two of them, or one: the last odd one, and every item
// of the experts from plan.half_from on)
__device__ __forceinline__ void pf_decode(const PfPlan& plan, int it, int& cursor, int WB, int last_cols, bool down, PfItem& o) {
    while (cursor + 1 < plan.n_active && plan.item_base[cursor + 1] <= it) ++cursor;
    o.a = cursor;
    const int local = it - plan.item_base[cursor];
    const int tpi = plan.tpi;
    const int m_blocks = (plan.rows[cursor] + tpi - 1) / tpi;
    const int blk = local / m_blocks;
    o.mb = local - blk * m_blocks;
    o.row_start = plan.row0[cursor] + o.mb * tpi;
    const int left = plan.rows[cursor] - o.mb * tpi;
    o.rows_here = left < tpi ? left : tpi;
    if (down && cursor >= plan.half_from) {
        o.wb = blk;
        o.n_cols = 128;
    } else {
        o.wb = down ? 2 * blk : blk;
        o.n_cols = (blk == WB - 1) ? last_cols : 256;
    }
    o.n_mt = o.rows_here > 128 ? 2 : 1;
}

// PHASE 0: h = silu(x Wg^T) * (x Wu^T);  PHASE 1: y = h Wd^T
template <int PHASE>
__global__ void __launch_bounds__(kPfThreads, 1)
ffn_prefill_kernel(FfnArgs a, const __grid_constant__ SlotTable tab, const __grid_constant__ CUtensorMap act_map,
                   const __grid_constant__ CUtensorMap act_map128, const __grid_constant__ CUtensorMap act_map256,
                   const __grid_constant__ CUtensorMap out_map) {
    extern __shared__ uint8_t dyn_smem[];
    __shared__ PfPlan plan;
    __shared__ __align__(8) uint64_t bar_full[kPfMaxStages], bar_empty[kPfMaxStages], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    __shared__ int claimed[16];            // down launch with claimed items: this CTA's items in order (-1: no more, -2: not known yet)
    __shared__ int s_warp_act[kPfThreads / 32], s_warp_t1[kPfThreads / 32], s_warp_t2[kPfThreads / 32];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = PHASE == 0 ? a.d : a.f;
    const int KC = K / kTileK;
    // weight blocks of 256 rows: gate/up -> one f-block (128 gate + 128 up rows); down -> two d-blocks
    const int WB = PHASE == 0 ? a.f / kTileRows : (a.d / kTileRows + 1) / 2;
    const int last_cols = PHASE == 0 ? 256 : ((a.d / kTileRows) & 1 ? 128 : 256);
    const uint32_t smem_base = (smem_u32(dyn_smem) + 1023u) & ~1023u;

    if (tid < 16) claimed[tid] = -2;
    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < kPfMaxStages; ++s) { mbar_init(smem_u32(&bar_full[s]), 1); mbar_init(smem_u32(&bar_empty[s]), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&bar_acc_full[s]), 1); mbar_init(smem_u32(&bar_acc_empty[s]), 8); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // The gate/up launch waits for whatever produced its inputs.  The down launch does not, at this point: it starts on
    // the SMs that the gate/up grid has left (all of that grid's CTAs have passed their own wait by then, so everything
    // older is complete), makes its plan, and then either waits for the whole gate/up grid (a single round of down
    // items, see the plan) or waits per expert for that expert's h rows (counters below), so that the last gate/up
    // items -- a partial round on a few SMs -- overlap the down projection of the other experts.
    if (PHASE == 0) pdl_wait();
    pdl_launch_dependents();
    // a.counters[e]: token rows x f-blocks of expert e whose h is complete, counted once per epilogue warp (8 x f-blocks
    // x rows when all of it is there); a.counters[kMaxCtas + e]: down items of expert e that have seen that.  The last
    // of those puts both back to zero for the next call.
    int* const h_ready = a.counters;
    int* const h_seen = a.counters + kMaxCtas;
    int* const next_item = a.counters + 2 * kMaxCtas;      // down launch: the next unclaimed item

    // ---- plan (one thread per expert, block-wide prefix sums) ----
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
        const int t1 = rows > 0 ? (rows + 127) / 128 : 0, t2 = rows > 0 ? (rows + 255) / 256 : 0;   // 128- / 256-token tiles
        int act_inc = rows > 0 ? 1 : 0, t1_inc = t1, t2_inc = t2;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int na = __shfl_up_sync(0xffffffffu, act_inc, o), n1 = __shfl_up_sync(0xffffffffu, t1_inc, o),
                      n2 = __shfl_up_sync(0xffffffffu, t2_inc, o);
            if (lane >= o) { act_inc += na; t1_inc += n1; t2_inc += n2; }
        }
        if (lane == 31) { s_warp_act[warp] = act_inc; s_warp_t1[warp] = t1_inc; s_warp_t2[warp] = t2_inc; }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        int base_act = 0, base_t1 = 0, base_t2 = 0, tot_act = 0, tot_t1 = 0, tot_t2 = 0;
#pragma unroll
        for (int w = 0; w < kPfThreads / 32; ++w) {
            if (w < warp) { base_act += s_warp_act[w]; base_t1 += s_warp_t1[w]; base_t2 += s_warp_t2[w]; }
            tot_act += s_warp_act[w];
            tot_t1 += s_warp_t1[w];
            tot_t2 += s_warp_t2[w];
        }
        // two token tiles per item when that still leaves several rounds of items per CTA and most
        // of those items really have two tiles (every thread takes the same decision)
        const bool pair = 2ll * tot_t2 * WB >= (long long)kPfPairHalfRounds * gridDim.x && 2 * tot_t1 >= 3 * tot_t2;
        if (rows > 0) {
            const int n = base_act + act_inc - 1;
            plan.slot[n] = tab.slot[e];
            plan.eid[n] = e;
            plan.row0[n] = r0;
            plan.rows[n] = rows;
            plan.item_base[n] = pair ? (base_t2 + t2_inc - t2) * WB : (base_t1 + t1_inc - t1) * WB;
        }
        if (tid == 0) {
            plan.item_base[tot_act] = (pair ? tot_t2 : tot_t1) * WB;
            plan.n_active = tot_act;
            plan.total_items = (pair ? tot_t2 : tot_t1) * WB;
            plan.tpi = pair ? 256 : 128;
            // Do the two launches overlap at their seam?  (Both launches take this decision, from the same numbers.)
            //  * When the segments are long (prefill: the SMs that the gate/up launch's last round leaves idle are idle
            //    tensor pipes), always -- given more than one round of down items.
            //  * When they are short (decode: weight streaming) only if that last round occupies at most half of the SMs:
            //    a fuller round keeps HBM busy by itself, and the overlap's bookkeeping then costs more than the idle SMs
            //    could have fetched (c3 at 32 tokens with 106 of 148 SMs in the last round: 1 % slower with the overlap;
            //    the Qwen3 shape at 16 tokens, 64 of 148: 7 % faster).  The routing decides this step by step.
            //  * A single round of down items (the Mixtral shape at 16 tokens: 896 gate/up items are six rounds and 8
            //    items; 128 down items of 7 MB): the items that wait for the last expert's h are as long as the whole
            //    launch, and overlapping as such gains nothing (measured 1 % slower).  It pays if the LAST expert's down
            //    items -- the only ones that have to wait for the gate/up tail -- are cut in two (one 128-column block
            //    each): they are then no longer what the launch ends with.  Only with one token tile per expert and while
            //    everything still fits one round.
            // (32-bit arithmetic: at most 65535 rows and 128 weight blocks.)
            const int G = (int)gridDim.x;
            const int wb_gu = a.f / kTileRows, wb_down = (a.d / kTileRows + 1) / 2, db = a.d / kTileRows;
            const bool pair_gu = 2 * tot_t2 * wb_gu >= kPfPairHalfRounds * G && 2 * tot_t1 >= 3 * tot_t2;
            const int rest_gu = ((pair_gu ? tot_t2 : tot_t1) * wb_gu) % G;
            const bool small_rest = rest_gu != 0 && 2 * rest_gu <= G;
            const bool long_segments = 2 * tot_t1 >= 3 * tot_act;
            const int items_split = tot_t1 * wb_down + (db - wb_down);
            plan.half_from = 1 << 30;
            if (tot_t1 * wb_down > G) {
                plan.seam = long_segments || small_rest ? 1 : 0;
            } else if (tot_act >= 2 && tot_t1 == tot_act && small_rest && items_split <= G) {
                plan.seam = 1;
                if (PHASE == 1) {
                    plan.half_from = tot_act - 1;
                    plan.total_items = items_split;
                    plan.item_base[tot_act] = items_split;
                }
            } else {
                plan.seam = 0;
            }
        }
        __syncthreads();
    }
    const bool seam = plan.seam != 0;
    if (PHASE == 1 && !seam) pdl_wait();        // (the plan above read only what was complete before the gate/up launch began)
    const uint32_t tmem_base = tmem_base_s;
    const int total_items = plan.total_items;
    const int n_stages = plan.tpi == 128 ? 4 : 3;
    const uint32_t stage_bytes = kPfStageW + (uint32_t)(plan.tpi / 128) * kPfTileX;
    const int G = gridDim.x;
    volatile int* abort_p = &abort_flag;
    // The copy warp publishes each claimed item in `claimed` as soon as it knows it; the other warps read it there before
    // the item's first stage has arrived (bounded: -3 if the CTA has given up).
    auto claimed_item = [&](int n) -> int {
        const volatile int* slot = &claimed[n & 15];
        unsigned long long t0 = 0;
        for (uint32_t i = 0;; ++i) {
            const int v = *slot;
            if (v != -2) return v;
            if ((i & 1023u) == 1023u) {
                if (*abort_p) return -3;
                const unsigned long long now = globaltimer_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > kWaitLimitNs) { *abort_p = 1; atomicExch(a.status, SAEM_ERR_TIMEOUT); return -3; }
            }
        }
    };

    if (warp == 0) {
        // =============================== producer ===============================
        int stage = 0, cursor = 0, ready_a = -1;
        uint32_t phase = 0;
        bool ok = true;
        int issued = 0;
        PfItem it;
        // Gate/up: whole items round-robin.  Down: items are claimed in the same order with one atomic add each, because
        // this launch's CTAs start at different times -- the SMs of the gate/up launch's last round join late and must
        // get less.  The G failing claims at the end put the counter back to zero.
        auto claim = [&](int after) -> int {
            if (!seam) return after + G;            // every CTA starts at the same time: round-robin
            int v = 0;
            if (lane == 0) {
                v = atomicAdd(next_item, 1);
                if (v == total_items + G - 1) *next_item = 0;
            }
            return v;
        };
        int upcoming = PHASE == 0 || !seam ? (int)blockIdx.x : claim(0);
        for (int n = 0; ok; ++n) {
            const int item = __shfl_sync(0xffffffffu, upcoming, 0);
            if (PHASE == 1 && seam && lane == 0) {
                claimed[(n + 1) & 15] = -2;          // (its previous user is fifteen items back: nobody reads it any more)
                claimed[n & 15] = item < total_items ? item : -1;
            }
            if (item >= total_items) break;
            pf_decode(plan, item, cursor, WB, last_cols, PHASE == 1, it);
            const uint8_t* slot = a.slot_region + (size_t)plan.slot[it.a] * a.slot_bytes;
            // gate/up: chunk (f-block, kc) is 32 KB (gate tile, up tile); down: tiles (2 wb, kc), (2 wb + 1, kc)
            const uint8_t* w0 = PHASE == 0 ? slot + (size_t)it.wb * KC * kPfStageW
                                           : slot + (size_t)2 * a.d * a.f * 2 + (size_t)it.wb * KC * kTileBytes;
            const uint8_t* w1 = PHASE == 0 ? w0 + kTileBytes : w0 + (size_t)KC * kTileBytes;
            const size_t w_step = PHASE == 0 ? kPfStageW : kTileBytes;
            const int n_boxes = (it.rows_here + 31) / 32;
            const uint32_t w_bytes = it.n_cols == 256 ? kPfStageW : kTileBytes;
            if (PHASE == 1 && seam) {       // this expert's h must be complete; every item says that it has seen it
                const int e = plan.eid[it.a];
                int good = 1;
                if (lane == 0) {
                    if (it.a != ready_a) good = counter_wait(h_ready + e, 8 * (a.f / kTileRows) * plan.rows[it.a], abort_p, a.status) ? 1 : 0;
                    if (good && atomicAdd(h_seen + e, 1) == plan.item_base[it.a + 1] - plan.item_base[it.a] - 1) {
                        h_ready[e] = 0;
                        h_seen[e] = 0;
                    }
                    fence_proxy_async_all();
                }
                ok = __shfl_sync(0xffffffffu, good, 0) != 0;
                if (!ok) break;
                ready_a = it.a;
            }
            for (int kc = 0; kc < KC; ++kc) {
                ok = mbar_wait(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_p, a.status);
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t full = smem_u32(&bar_full[stage]);
                    const uint32_t ws = smem_base + (uint32_t)stage * stage_bytes;
                    mbar_expect_tx(full, w_bytes + (uint32_t)n_boxes * 4096u);
                    // few, large copies: issuing them is serial work of this one thread on the refill path
                    if (PHASE == 0) {       // the gate tile and the up tile of a chunk are adjacent
                        bulk_g2s(ws, w0 + (size_t)kc * w_step, kPfStageW, full);
                    } else {
                        bulk_g2s(ws, w0 + (size_t)kc * w_step, kTileBytes, full);
                        if (it.n_cols == 256) bulk_g2s(ws + kTileBytes, w1 + (size_t)kc * w_step, kTileBytes, full);
                    }
                    // whole token tiles in one copy (256 or 128 rows), the ragged rest in 32-row boxes
                    int b = 0;
                    if (n_boxes == 8) {
                        tma_2d(ws + kPfStageW, &act_map256, kc * kTileK, it.row_start, full);
                        b = 8;
                    }
                    for (; b + 4 <= n_boxes; b += 4)
                        tma_2d(ws + kPfStageW + (uint32_t)b * 4096u, &act_map128, kc * kTileK, it.row_start + b * 32, full);
                    for (; b < n_boxes; ++b)
                        tma_2d(ws + kPfStageW + (uint32_t)b * 4096u, &act_map, kc * kTileK, it.row_start + b * 32, full);
                }
                ++issued;
                if (++stage == n_stages) { stage = 0; phase ^= 1u; }
            }
            // the next item: claimed only now, with this item's last stages still in flight -- a CTA never holds an item
            // it is not yet working on, so that a launch of fewer items than CTAs gives each CTA at most one
            upcoming = PHASE == 0 ? item + G : claim(item);
        }
        if (!ok && issued > 0) {     // let copies already in flight land before the CTA's memory goes away
            unsigned long long t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 200000ull) {}
        }
    } else if (warp == 1) {
        // =============================== MMA issuer ===============================
        int stage = 0, acc = 0, cursor = 0;
        uint32_t phase = 0, acc_phase[2] = {0u, 0u};
        bool ok = true;
        PfItem it;
        for (int n = 0; ok; ++n) {
            int item = blockIdx.x + n * G;
            const bool dealt = PHASE == 0 || !seam;      // round-robin: the item is known before its first stage arrives
            if (dealt) {
                if (item >= total_items) break;
                pf_decode(plan, item, cursor, WB, last_cols, PHASE == 1, it);
            }
            if (!dealt) {
                item = claimed_item(n);
                if (item < 0) { ok = item == -1; break; }
                pf_decode(plan, item, cursor, WB, last_cols, PHASE == 1, it);
            }
            ok = mbar_wait(smem_u32(&bar_full[stage]), phase, abort_p, a.status);     // the item's first stage
            if (!ok) break;
            const int acc0 = acc, acc1 = acc ^ 1;             // accumulators of the item's first / second tile
            const uint32_t idesc = idesc_bf16(it.n_cols);
            for (int kc = 0; ok && kc < KC; ++kc) {
                if (kc > 0) ok = mbar_wait(smem_u32(&bar_full[stage]), phase, abort_p, a.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t ws = smem_base + (uint32_t)stage * stage_bytes;
                const uint32_t xs = ws + kPfStageW;
                for (int t = 0; t < it.n_mt; ++t) {
                    const int ac = t == 0 ? acc0 : acc1;
                    if (kc == 0) {      // the accumulator must have been drained by the epilogue
                        ok = mbar_wait(smem_u32(&bar_acc_empty[ac]), acc_phase[ac] ^ 1u, abort_p, a.status);
                        if (!ok) break;
                        tc_fence_after();
                    }
                    if (lane == 0) {
                        const uint32_t d_tmem = tmem_base + (uint32_t)(ac * 256);
#pragma unroll
                        for (int k4 = 0; k4 < kTileK / 16; ++k4)
                            tc_mma_bf16(d_tmem, smem_desc_sw128(xs + t * kPfTileX + k4 * 32),
                                        smem_desc_sw128(ws + k4 * 32), idesc, (kc > 0 || k4 > 0) ? 1u : 0u);
                    }
                }
                if (!ok) break;
                if (lane == 0) tc_commit(smem_u32(&bar_empty[stage]));
                __syncwarp();
                if (++stage == n_stages) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            if (lane == 0) {
                tc_commit(smem_u32(&bar_acc_full[acc0]));
                if (it.n_mt == 2) tc_commit(smem_u32(&bar_acc_full[acc1]));
            }
            __syncwarp();
            acc_phase[acc0] ^= 1u;
            if (it.n_mt == 2) acc_phase[acc1] ^= 1u;
            else acc ^= 1;                                    // a one-tile item takes one accumulator of the ring
        }
    } else {
        // =============================== epilogue (warps 2..9) ===============================
        const int q = warp & 3;                 // TMEM lane quarter = token rows 32q .. 32q+31
        const int half = (warp - 2) >> 2;       // which half of the tile's columns
        const int i = q * 32 + lane;            // token row inside the tile
        const uint32_t store_buf = smem_base + (uint32_t)kPfStageArea + (uint32_t)(warp - 2) * kPfStoreBuf;
        int acc = 0, cursor = 0;
        uint32_t acc_phase[2] = {0u, 0u};
        bool ok = true;
        PfItem it;
        for (int n = 0; ok; ++n) {
            int item = blockIdx.x + n * G;
            const bool dealt = PHASE == 0 || !seam;
            if (dealt) {
                if (item >= total_items) break;
                pf_decode(plan, item, cursor, WB, last_cols, PHASE == 1, it);
            }
            if (!dealt) {
                item = claimed_item(n);
                if (item < 0) { ok = item == -1; break; }
                pf_decode(plan, item, cursor, WB, last_cols, PHASE == 1, it);
            }
            ok = mbar_wait(smem_u32(&bar_acc_full[acc]), acc_phase[acc], abort_p, a.status);     // the item's first tile
            if (!ok) break;
            for (int t = 0; ok && t < it.n_mt; ++t) {
                const int ac = t == 0 ? acc : acc ^ 1;
                if (t > 0) ok = mbar_wait(smem_u32(&bar_acc_full[ac]), acc_phase[ac], abort_p, a.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ac * 256);
                // This warp's slice of the tile goes to registers in one batch and the accumulator is
                // handed back at once: the stores below overlap the MMAs of the next tile.
                uint32_t v[128];
                const int c_half = PHASE == 0 ? 64 : it.n_cols / 2;      // output columns of this warp: 64 or 128
                if (PHASE == 0) {     // gate at TMEM columns [64 half, +64), up at 128 + the same
                    tc_ld32_issue(t_row + (uint32_t)(half * 64), v);
                    tc_ld32_issue(t_row + (uint32_t)(half * 64 + 32), v + 32);
                    tc_ld32_issue(t_row + (uint32_t)(128 + half * 64), v + 64);
                    tc_ld32_issue(t_row + (uint32_t)(128 + half * 64 + 32), v + 96);
                } else {
                    tc_ld32_issue(t_row + (uint32_t)(half * c_half), v);
                    tc_ld32_issue(t_row + (uint32_t)(half * c_half + 32), v + 32);
                    if (c_half == 128) {
                        tc_ld32_issue(t_row + (uint32_t)(half * c_half + 64), v + 64);
                        tc_ld32_issue(t_row + (uint32_t)(half * c_half + 96), v + 96);
                    }
                }
                tc_wait_ld();
#pragma unroll
                for (int g16 = 0; g16 < 8; ++g16) tc_reg_fence16(v + 16 * g16);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[ac]));
                acc_phase[ac] ^= 1u;

                const int r = t * 128 + i;
                const bool valid = r < it.rows_here;
                const bool full_box = t * 128 + q * 32 + 32 <= it.rows_here;     // this warp's 32 rows all exist
                const int box_row = it.row_start + t * 128 + q * 32;
                const size_t row = (size_t)(it.row_start + r);
                const uint32_t my_buf = store_buf + (uint32_t)lane * 64u;
                const uint32_t sw = (uint32_t)((lane >> 1) & 3);
                if (PHASE == 0) {
                    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.h) + row * a.f + (size_t)it.wb * kTileRows + half * 64;
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
                                tma_store_2d(&out_map, it.wb * kTileRows + half * 64 + 32 * bx, box_row, store_buf);
                                bulk_commit();
                            }
                        } else if (valid) {
                            uint4* o = reinterpret_cast<uint4*>(dst + 32 * bx);
#pragma unroll
                            for (int c = 0; c < 4; ++c) o[c] = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                        }
                    }
                } else {
                    float* dst = a.y_packed + row * a.d + (size_t)it.wb * 128 + half * c_half;
#pragma unroll
                    for (int bx = 0; bx < 8; ++bx) {          // boxes of 16 y columns
                        if (bx * 16 < c_half) {
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
                                    tma_store_2d(&out_map, it.wb * 128 + half * c_half + 16 * bx, box_row, store_buf);
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
            }
            if (it.n_mt == 1) acc ^= 1;
            if (PHASE == 0 && seam && ok) {         // this warp's share of the item's h is complete and visible device-wide
                if (lane == 0) bulk_wait_all();          // the tile stores (async proxy) are complete
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(h_ready + plan.eid[it.a], it.rows_here);
            }
        }
        if (lane == 0) bulk_wait_all();         // this warp's tile stores have landed
    }

    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
    }
}

// ------------------------------------------------------------------------------------------- host
static bool g_pf_init[64];

cudaError_t ffn_prefill_init() {
    if (!first_call_on_device(g_pf_init)) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(ffn_prefill_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPfSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(ffn_prefill_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPfSmem);
    if (e != cudaSuccess) return e;
    return cudaSuccess;
}

cudaError_t launch_ffn_prefill(const FfnArgs& a, const SlotTable& tab, const CUtensorMap& map_x, const CUtensorMap& map_h,
                               const CUtensorMap& map_x128, const CUtensorMap& map_h128, const CUtensorMap& map_x256,
                               const CUtensorMap& map_h256, const CUtensorMap& map_h_store, const CUtensorMap& map_y_store, cudaStream_t st,
                               int* n_launch) {
    cudaError_t e = ffn_prefill_init();
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)a.n_sm), block(kPfThreads);
    e = launch_pdl(ffn_prefill_kernel<0>, grid, block, (size_t)kPfSmem, st, a, tab, map_x, map_x128, map_x256, map_h_store);
    if (e != cudaSuccess) return e;
    e = launch_pdl(ffn_prefill_kernel<1>, grid, block, (size_t)kPfSmem, st, a, tab, map_h, map_h128, map_h256, map_y_store);
    *n_launch = 2;
    return e;
}

}  // namespace saem
