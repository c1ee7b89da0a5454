// Grouped SwiGLU expert FFN over the repacked segments (Sec. IV-E: one dense batched execution
// per expert over its contiguous rows; Sec. IV-C: weights live in fixed HBM cache slots),
// written for sm_100a as a weight-streaming kernel.  It serves launches whose segments have at
// most 64 rows (decode); larger segments go to the tensor-tiled kernels of ffn_prefill.cu.
//
//   * Operands are swapped: a 128-row tile of the expert's WEIGHTS is the MMA's M operand and the
//     segment's tokens are the narrow N operand (16..64), so decode-sized segments still fill the
//     tensor core's M dimension and every weight byte is read from HBM exactly once per token tile.
//   * Weight tiles are stored in the slot pre-swizzled (see saem_pack_expert_host), so one
//     cp.async.bulk per stage lands a 16/32 KB tile in shared memory ready for tcgen05.mma;
//     activation tiles come through a TMA tensor map with the same 128-byte swizzle.
//   * Persistent CTAs, two per SM (each with half of the shared memory and only the TMEM columns
//     it needs), so that one CTA's set-up, epilogue and split-item reduction overlap the other's
//     streaming.  The flat list of (expert, token tile, weight-row block,
//     k-chunk) units of the ACTIVE experts only is cut into equal contiguous ranges, one per CTA
//     (inactive experts' weights are never touched).  A (expert, token tile, row block) item whose
//     k-range is split across CTAs is finished by whichever contributor arrives last, which adds
//     the partial tiles in ascending CTA order -- deterministic, and no CTA ever waits for another.
//   * Warp roles: warp 0 issues the copies, warp 1 issues tcgen05.mma into TMEM accumulators
//     (double-buffered when they fit), warps 2..9 read TMEM back (tcgen05.ld), apply SiLU*up or
//     store y.  Stages are handed over with mbarriers; every wait is bounded and, when it runs out,
//     sets SAEM_ERR_TIMEOUT in the device status word and makes the CTA drain and return.
//
// Two launches per FFN: gate/up (+SiLU*mul -> h, bf16) and down (-> y_packed, fp32).
#include "tc_common.cuh"

namespace saem {

constexpr int kThreads = 320;                 // warp 0 copies, warp 1 MMA, warps 2..9 epilogue
constexpr int kEpiThreads = 256;
constexpr int kGateUpMaxTile = 128;           // widest token tile of the gate/up phase (two accumulator sets fit TMEM)
constexpr int kMaxStages = 8;
constexpr int kDynSmemMax = 220 * 1024;
constexpr long long kSplitBelowItemsPerCta = 6;   // split items across CTAs only below this many items per CTA
constexpr long long kMinChunksPerCta = 6;        // below this many k-chunks per CTA, use fewer CTAs

// --------------------------------------------------------------------------------------- the plan
struct Plan {
    int n_active;
    int total_items;
    int e[SAEM_MAX_EXPERTS];
    int slot[SAEM_MAX_EXPERTS];
    int row0[SAEM_MAX_EXPERTS];
    int rows[SAEM_MAX_EXPERTS];
    int item_base[SAEM_MAX_EXPERTS + 1];
};

struct Item {
    int a, nb, rb;          // active-expert index, token tile, weight-row block
    int kc_begin, kc_end;   // this CTA's part of the item's k-chunks
    int row_start, rows_here, n_eff;
    long long it;           // global item index
};

struct ItemWalker {
    const Plan* plan;
    long long c, c1;        // next chunk, end of this CTA's range (contiguous mode)
    long long stride;       // > 0: whole items it, it + stride, ... < c1 (c, c1 then count items)
    int KC, RB, n_tile;
    int a_cursor;
    __device__ __forceinline__ ItemWalker(const Plan* p, long long c0_, long long c1_, long long stride_, int KC_,
                                          int RB_, int nt)
        : plan(p), c(c0_), c1(c1_), stride(stride_), KC(KC_), RB(RB_), n_tile(nt), a_cursor(0) {}
    __device__ __forceinline__ bool next(Item& o) {
        if (c >= c1) return false;
        long long it;
        if (stride > 0) {
            it = c;
            o.kc_begin = 0;
            o.kc_end = KC;
            c += stride;
        } else {
            it = c / KC;
            o.kc_begin = (int)(c - it * KC);
            long long end = (it + 1) * KC;
            if (end > c1) end = c1;
            o.kc_end = (int)(end - it * KC);
            c = end;
        }
        o.it = it;
        while (a_cursor + 1 < plan->n_active && plan->item_base[a_cursor + 1] <= it) ++a_cursor;
        o.a = a_cursor;
        // items of one expert: weight-row block slowest, token tile fastest, so that the token
        // tiles that share a weight block are worked on at the same time by neighbouring CTAs
        // (whole-item mode deals items round-robin) and the block is fetched from HBM once
        const int local = (int)(it - plan->item_base[a_cursor]);
        const int n_blocks = (plan->rows[a_cursor] + n_tile - 1) / n_tile;
        o.rb = local / n_blocks;
        o.nb = local - o.rb * n_blocks;
        o.row_start = plan->row0[a_cursor] + o.nb * n_tile;
        int left = plan->rows[a_cursor] - o.nb * n_tile;
        o.rows_here = left < n_tile ? left : n_tile;
        o.n_eff = (o.rows_here + 15) & ~15;
        return true;
    }
};

// ----------------------------------------------------------------------------------------- kernel
// PHASE 0: h = silu(Wg x) * (Wu x)   (activations = x_packed, reduction over d)
// PHASE 1: y = Wd h                  (activations = h,        reduction over f)
template <int PHASE>
__global__ void __launch_bounds__(kThreads, 2)
ffn_tensor_kernel(FfnArgs a, const __grid_constant__ SlotTable tab, const __grid_constant__ CUtensorMap act_map,
                  int n_stages, int box_rows) {
    constexpr int W_BYTES = PHASE == 0 ? 2 * kTileBytes : kTileBytes;
    extern __shared__ uint8_t dyn_smem[];
    __shared__ Plan plan;
    __shared__ __align__(8) uint64_t bar_full[kMaxStages], bar_empty[kMaxStages], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag, last_flag, s_ncontrib;
    __shared__ short s_contrib[256];            // contributors of a split item (at most K/64 <= 256)
    __shared__ int s_warp_act[kThreads / 32], s_warp_items[kThreads / 32];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = PHASE == 0 ? a.d : a.f;
    const int KC = K / kTileK;
    const int RB = (PHASE == 0 ? a.f : a.d) / kTileRows;
    const int n_tile = a.n_tile;
    const int acc_cols = (PHASE == 0 ? 2 : 1) * n_tile;
    const int n_acc = (2 * acc_cols <= 512) ? 2 : 1;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < n_acc * acc_cols) tmem_cols <<= 1;
    const uint32_t x_stage_bytes = (uint32_t)n_tile * 128u;
    const uint32_t stage_bytes = W_BYTES + x_stage_bytes;
    const uint32_t smem_base = (smem_u32(dyn_smem) + 1023u) & ~1023u;

    // ---- set-up that does not depend on earlier kernels: barriers, tensor memory ----
    if (tid == 0) {
        abort_flag = 0;
        last_flag = 0;
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(smem_u32(&bar_full[s]), 1); mbar_init(smem_u32(&bar_empty[s]), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&bar_acc_full[s]), 1); mbar_init(smem_u32(&bar_acc_empty[s]), kEpiThreads / 32); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // TMEM: only the columns this launch needs, so that two CTAs can share an SM
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(tmem_cols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Under programmatic dependent launch this kernel may have started before the preceding kernels
    // of the stream finished.  The gate/up kernel reads what its predecessor (the repack) wrote right
    // away (offsets), so it waits here.  The down kernel's predecessor is the gate/up kernel, which
    // has passed this very wait before it let dependents launch: the repack's outputs are final, so
    // the down kernel may build its plan and even start loading WEIGHTS (which no kernel writes)
    // before it waits for h; see the producer.
    if (PHASE == 0) {
        pdl_wait();
        pdl_launch_dependents();
    }

    // ---- plan: active experts of this launch, in ascending id (one thread per expert) ----
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
        const int my_items = rows > 0 ? ((rows + n_tile - 1) / n_tile) * RB : 0;
        int act_inc = rows > 0 ? 1 : 0, item_inc = my_items;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int na = __shfl_up_sync(0xffffffffu, act_inc, o), ni = __shfl_up_sync(0xffffffffu, item_inc, o);
            if (lane >= o) { act_inc += na; item_inc += ni; }
        }
        if (lane == 31) { s_warp_act[warp] = act_inc; s_warp_items[warp] = item_inc; }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        int base_act = 0, base_items = 0, tot_act = 0, tot_items = 0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) {
            if (w < warp) { base_act += s_warp_act[w]; base_items += s_warp_items[w]; }
            tot_act += s_warp_act[w];
            tot_items += s_warp_items[w];
        }
        if (rows > 0) {
            const int n = base_act + act_inc - 1;
            plan.e[n] = e;
            plan.slot[n] = tab.slot[e];
            plan.row0[n] = r0;
            plan.rows[n] = rows;
            plan.item_base[n] = base_items + item_inc - my_items;
        }
        if (tid == 0) {
            plan.item_base[tot_act] = tot_items;
            plan.n_active = tot_act;
            plan.total_items = tot_items;
        }
        __syncthreads();
    }
    const uint32_t tmem_base = tmem_base_s;

    // Decode-sized work (few items per CTA) is cut at k-chunk granularity so that every SM streams
    // the same number of bytes; with many items per CTA whole items are dealt out instead and no
    // partial tiles are needed.
    const long long total_chunks = (long long)plan.total_items * KC;
    // Tiny launches use fewer CTAs, so that no item is cut into dozens of slivers whose partial
    // tiles would then have to be added up one after the other.
    long long G = gridDim.x;
    if (total_chunks < G * kMinChunksPerCta) G = total_chunks / kMinChunksPerCta > 0 ? total_chunks / kMinChunksPerCta : 1;
    const long long my_cta = blockIdx.x < G ? blockIdx.x : G - 1;     // surplus CTAs get an empty range below
    const bool split_k = (long long)plan.total_items < kSplitBelowItemsPerCta * G;
    long long c0 = split_k ? total_chunks * my_cta / G : my_cta;
    long long c1 = split_k ? total_chunks * (my_cta + 1) / G : (long long)plan.total_items;
    if (blockIdx.x >= G) c1 = c0;
    const long long walk_stride = split_k ? 0 : G;
    volatile int* abort_p = &abort_flag;
    if (PHASE == 1 && warp != 0) {
        pdl_wait();
        pdl_launch_dependents();
    }

    if (warp == 0) {
        // =============================== producer ===============================
        ItemWalker walk(&plan, c0, c1, walk_stride, KC, RB, n_tile);
        Item it;
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        int issued = 0;
        int pre = 0;                 // stages whose weights went out before the dependency wait (down kernel)
        const size_t w_region = PHASE == 0 ? 0 : (size_t)2 * a.d * a.f * 2;
        if (PHASE == 1) {
            // weights of the first stages: they do not depend on the gate/up kernel
            ItemWalker early(&plan, c0, c1, walk_stride, KC, RB, n_tile);
            Item ei;
            while (pre < n_stages && early.next(ei)) {
                const uint8_t* wsrc = a.slot_region + (size_t)plan.slot[ei.a] * a.slot_bytes + w_region +
                                      (size_t)ei.rb * KC * W_BYTES;
                const int nb = (ei.rows_here + box_rows - 1) / box_rows;
                for (int kc = ei.kc_begin; kc < ei.kc_end && pre < n_stages; ++kc, ++pre) {
                    if (lane == 0) {
                        const uint32_t full = smem_u32(&bar_full[pre]);
                        mbar_expect_tx(full, W_BYTES + (uint32_t)(nb * box_rows) * 128u);
                        bulk_g2s(smem_base + (uint32_t)pre * stage_bytes, wsrc + (size_t)kc * W_BYTES, kTileBytes, full);
                    }
                }
            }
            pdl_wait();              // h is complete from here on
            pdl_launch_dependents();
        }
        while (ok && walk.next(it)) {
            const uint8_t* slot = a.slot_region + (size_t)plan.slot[it.a] * a.slot_bytes;
            const uint8_t* wbase = slot + w_region + (size_t)it.rb * KC * W_BYTES;
            const int n_boxes = (it.rows_here + box_rows - 1) / box_rows;
            for (int kc = it.kc_begin; kc < it.kc_end; ++kc) {
                const bool early_w = issued < pre;          // this stage's weights are already on their way
                if (!early_w) {
                    ok = mbar_wait(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_p, a.status);
                    if (!ok) break;
                }
                if (lane == 0) {
                    const uint32_t full = smem_u32(&bar_full[stage]);
                    const uint32_t ws = smem_base + (uint32_t)stage * stage_bytes;
                    if (!early_w) {
                        mbar_expect_tx(full, W_BYTES + (uint32_t)(n_boxes * box_rows) * 128u);
                        const uint8_t* src = wbase + (size_t)kc * W_BYTES;
                        bulk_g2s(ws, src, W_BYTES, full);        // gate/up: the two tiles of a chunk are adjacent
                    }
                    for (int b = 0; b < n_boxes; ++b)
                        tma_2d(ws + W_BYTES + (uint32_t)(b * box_rows) * 128u, &act_map, kc * kTileK,
                               it.row_start + b * box_rows, full);
                }
                ++issued;
                if (++stage == n_stages) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok && issued > 0) {     // let copies already in flight land before the CTA's memory goes away
            unsigned long long t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 200000ull) {}
        }
    } else if (warp == 1) {
        // =============================== MMA issuer ===============================
        ItemWalker walk(&plan, c0, c1, walk_stride, KC, RB, n_tile);
        Item it;
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase[2] = {0u, 0u};
        bool ok = true;
        while (ok && walk.next(it)) {
            ok = mbar_wait(smem_u32(&bar_acc_empty[acc]), acc_phase[acc] ^ 1u, abort_p, a.status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(acc * acc_cols);
            const uint32_t idesc = idesc_bf16(it.n_eff);
            for (int kc = it.kc_begin; kc < it.kc_end; ++kc) {
                ok = mbar_wait(smem_u32(&bar_full[stage]), phase, abort_p, a.status);
                if (!ok) break;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t ws = smem_base + (uint32_t)stage * stage_bytes;
                    const uint32_t xs = ws + W_BYTES;
#pragma unroll
                    for (int k4 = 0; k4 < kTileK / 16; ++k4) {
                        const uint32_t accum = (kc > it.kc_begin || k4 > 0) ? 1u : 0u;
                        const uint64_t bd = smem_desc_sw128(xs + k4 * 32);
                        tc_mma_bf16(d_tmem, smem_desc_sw128(ws + k4 * 32), bd, idesc, accum);
                        if (PHASE == 0)
                            tc_mma_bf16(d_tmem + (uint32_t)n_tile, smem_desc_sw128(ws + kTileBytes + k4 * 32), bd, idesc, accum);
                    }
                    tc_commit(smem_u32(&bar_empty[stage]));
                }
                __syncwarp();
                if (++stage == n_stages) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            if (lane == 0) tc_commit(smem_u32(&bar_acc_full[acc]));
            __syncwarp();
            acc_phase[acc] ^= 1u;
            if (n_acc == 2) acc ^= 1;
        }
    } else {
        // =============================== epilogue (warps 2..9) ===============================
        // Two warps per TMEM lane quarter; each takes half of the item's token columns.
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;
        const int i = q * 32 + lane;            // weight row inside the tile
        const int epi_tid = tid - 64;
        ItemWalker walk(&plan, c0, c1, walk_stride, KC, RB, n_tile);
        Item it;
        int acc = 0;
        uint32_t acc_phase[2] = {0u, 0u};
        bool ok = true;
        const size_t out_ld = PHASE == 0 ? (size_t)a.f : (size_t)a.d;
        while (ok && walk.next(it)) {
            ok = mbar_wait(smem_u32(&bar_acc_full[acc]), acc_phase[acc], abort_p, a.status);
            // The epilogue warps meet at named barriers below; if one of them gave up its wait, all of
            // them must leave together (every warp reaches this vote because the wait is bounded).
            {
                uint32_t all_ok;
                asm volatile(
                    "{\n\t.reg .pred p, q;\n\t"
                    "setp.ne.u32 q, %1, 0;\n\t"
                    "bar.red.and.pred p, 1, 256, q;\n\t"
                    "selp.u32 %0, 1, 0, p;\n\t}"
                    : "=r"(all_ok) : "r"((uint32_t)ok) : "memory");
                ok = all_ok != 0;
            }
            if (!ok) break;
            tc_fence_after();
            const bool whole = it.kc_begin == 0 && it.kc_end == KC;
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * acc_cols);
            // which partial slot this CTA's share of the item goes to: it starts inside the item -> 0, else 1
            const int my_slot = it.kc_begin > 0 ? 0 : 1;
            float* part = a.partials + ((size_t)blockIdx.x * 2 + my_slot) * a.partial_slot_floats;
            const size_t col = (size_t)it.rb * kTileRows + i;
            const int split = ((it.n_eff >> 1) + 15) & ~15;
            const int n_begin = half == 0 ? 0 : split, n_end = half == 0 ? split : it.n_eff;
            for (int n0 = n_begin; n0 < n_end; n0 += 16) {
                float g[16], u[16];
                tc_ld16(t_row + (uint32_t)n0, g);
                if (PHASE == 0) tc_ld16(t_row + (uint32_t)(n_tile + n0), u);
                if (whole) {
#pragma unroll
                    for (int n = 0; n < 16; ++n) {
                        if (n0 + n < it.rows_here) {
                            const size_t row = (size_t)(it.row_start + n0 + n);
                            if (PHASE == 0) {
                                const float hv = __fdividef(g[n], 1.f + __expf(-g[n])) * u[n];
                                reinterpret_cast<__nv_bfloat16*>(a.h)[row * out_ld + col] = __float2bfloat16_rn(hv);
                            } else {
                                a.y_packed[row * out_ld + col] = g[n];
                            }
                        }
                    }
                } else {
#pragma unroll
                    for (int n = 0; n < 16; ++n) {
                        part[(size_t)(n0 + n) * kTileRows + i] = g[n];
                        if (PHASE == 0) part[(size_t)(n_tile + n0 + n) * kTileRows + i] = u[n];
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[acc]));
            acc_phase[acc] ^= 1u;
            if (n_acc == 2) acc ^= 1;

            if (!whole) {
                // The contributors of this item are the CTAs whose (non-empty) ranges meet
                // [it*KC, (it+1)*KC).  CTA b owns chunks [b*total/G, (b+1)*total/G); when there are
                // fewer chunks than CTAs some ranges are empty, so the list is walked, not counted.
                const long long s0 = it.it * KC, s1 = s0 + KC - 1;
                __threadfence();
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (epi_tid == 0) {
                    int n_contrib = 0;
                    for (long long c = s0; c <= s1;) {
                        const int b = (int)(((c + 1) * G - 1) / total_chunks);    // the CTA that owns chunk c
                        s_contrib[n_contrib++] = (short)b;
                        c = ((long long)(b + 1) * total_chunks) / G;              // first chunk of the next CTA
                    }
                    s_ncontrib = n_contrib;
                    int* ctr = a.counters + PHASE * kMaxCtas + s_contrib[0];
                    const int old = atomicAdd(ctr, 1);
                    const int last = old == n_contrib - 1;
                    if (last) *ctr = 0;                       // ready for the next launch
                    last_flag = last;
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (last_flag) {
                    __threadfence();
                    // eight token columns at a time: 8 (16 with the up half) independent L2 loads
                    // in flight per thread and contributor; contributors added in ascending order
                    const int nc = s_ncontrib;
                    const int r_end = n_end < it.rows_here ? n_end : it.rows_here;
                    for (int n0 = n_begin; n0 < r_end; n0 += 8) {
                        float sg[8], su[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) sg[j] = su[j] = 0.f;
                        // contributors several at a time: all their loads are issued before the first
                        // sum needs a value (one L2 round trip per group of contributors, not per one);
                        // the additions still run in ascending contributor order
                        constexpr int CB = PHASE == 0 ? 2 : 4;     // bounded by the register budget
                        for (int c0i = 0; c0i < nc; c0i += CB) {
                            float vg[CB][8], vu[CB][8];
#pragma unroll
                            for (int cc = 0; cc < CB; ++cc) {
                                const int ci = c0i + cc;
                                if (ci < nc) {
                                    const float* p = a.partials +
                                                     ((size_t)s_contrib[ci] * 2 + (ci == 0 ? 1 : 0)) * a.partial_slot_floats +
                                                     (size_t)n0 * kTileRows + i;
#pragma unroll
                                    for (int j = 0; j < 8; ++j) vg[cc][j] = __ldcg(p + (size_t)j * kTileRows);
                                    if (PHASE == 0) {
#pragma unroll
                                        for (int j = 0; j < 8; ++j) vu[cc][j] = __ldcg(p + (size_t)(n_tile + j) * kTileRows);
                                    }
                                }
                            }
#pragma unroll
                            for (int cc = 0; cc < CB; ++cc) {
                                if (c0i + cc < nc) {
#pragma unroll
                                    for (int j = 0; j < 8; ++j) {
                                        sg[j] += vg[cc][j];
                                        if (PHASE == 0) su[j] += vu[cc][j];
                                    }
                                }
                            }
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            if (n0 + j < it.rows_here) {
                                const size_t row = (size_t)(it.row_start + n0 + j);
                                if (PHASE == 0) {
                                    const float hv = __fdividef(sg[j], 1.f + __expf(-sg[j])) * su[j];
                                    reinterpret_cast<__nv_bfloat16*>(a.h)[row * out_ld + col] = __float2bfloat16_rn(hv);
                                } else {
                                    a.y_packed[row * out_ld + col] = sg[j];
                                }
                            }
                        }
                    }
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
            }
        }
    }

    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols));
    }
}

// One CTA waits, with the kernels' bounded wait, on an mbarrier that nothing ever completes: the
// wait must run out after `limit_ns`, set SAEM_ERR_TIMEOUT in the status word and return normally.
__global__ void bounded_wait_selftest_kernel(int* status, unsigned long long limit_ns) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    mbar_wait(smem_u32(&bar), 0u, &abort_flag, status, limit_ns);    // phase 0 never completes
}

cudaError_t launch_bounded_wait_selftest(int* status, unsigned long long limit_ns, cudaStream_t st) {
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(status, limit_ns);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;
static bool g_init_done[64];

cudaError_t ffn_tensor_init() {
    if (!first_call_on_device(g_init_done)) return cudaSuccess;
    cudaError_t e;
    if (!g_encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (!fn || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
        g_encode = (EncodeTiledFn)fn;
    }
    e = cudaFuncSetAttribute(ffn_tensor_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemMax);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(ffn_tensor_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmemMax);
    if (e != cudaSuccess) return e;
    return cudaSuccess;
}

static bool make_act_map(CUtensorMap* m, const void* base, int rows, int K, int box_rows) {
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Store map of the tiled kernels' epilogue: boxes of 32 rows x 64 bytes, 64-byte swizzle.
static bool make_store_map(CUtensorMap* m, void* base, CUtensorMapDataType dt, int elem_bytes, int rows, int cols) {
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * elem_bytes};
    cuuint32_t box[2] = {(cuuint32_t)(64 / elem_bytes), 32u};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(m, dt, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// The slot region as rows of 128 bytes; a box of 128 rows is one packed 16 KB weight tile, copied as it is.
static bool make_weight_map(CUtensorMap* m, const void* base, size_t bytes) {
    cuuint64_t dims[2] = {128, (cuuint64_t)(bytes >> 7)};
    cuuint64_t strides[1] = {128};
    cuuint32_t box[2] = {128, 128};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

cudaError_t launch_ffn_tensor(const FfnArgs& a, const SlotTable& tab, cudaStream_t st, int* n_launch) {
    {
        cudaError_t e = ffn_tensor_init();
        if (e != cudaSuccess) return e;
    }
    const int box_rows = a.n_tile >= 32 ? 32 : 16;
    if (a.n_tile % box_rows) return cudaErrorInvalidValue;     // an activation stage is a whole number of boxes
    const int nt0 = a.n_tile < kGateUpMaxTile ? a.n_tile : kGateUpMaxTile, nt1 = a.n_tile;
    alignas(64) CUtensorMap map_x, map_h;
    if (!make_act_map(&map_x, a.x_packed, a.max_rows, a.d, box_rows)) return cudaErrorInvalidValue;
    if (!make_act_map(&map_h, a.h, a.max_rows, a.f, box_rows)) return cudaErrorInvalidValue;
    // Hand-over to the tiled kernels.  Measured on whole layers (graph-replayed steps): from 9 tokens upwards the
    // tiled kernels give the shorter step on every layer shape of the benchmark (1-8 %), although they pad every
    // segment to 128 tokens -- one CTA per SM, whole items, no reductions across CTAs.  SAEM_FFN_AUTO therefore
    // sends everything beyond the matrix-vector kernels' 8 rows there; SAEM_FFN_TENSOR keeps the streaming kernels
    // up to 64 rows.
    if (a.n_tile > a.stream_max_tile) {
        alignas(64) CUtensorMap map_h_store, map_y_store, map_x128, map_h128, map_x256, map_h256;
        if (box_rows != 32) {      // the tiled kernels load ragged token tiles as 32-row boxes, whatever the launch's tile
            if (!make_act_map(&map_x, a.x_packed, a.max_rows, a.d, 32)) return cudaErrorInvalidValue;
            if (!make_act_map(&map_h, a.h, a.max_rows, a.f, 32)) return cudaErrorInvalidValue;
        }
        if (!make_act_map(&map_x256, a.x_packed, a.max_rows, a.d, 256)) return cudaErrorInvalidValue;
        if (!make_act_map(&map_h256, a.h, a.max_rows, a.f, 256)) return cudaErrorInvalidValue;
        if (!make_act_map(&map_x128, a.x_packed, a.max_rows, a.d, 128)) return cudaErrorInvalidValue;
        if (!make_act_map(&map_h128, a.h, a.max_rows, a.f, 128)) return cudaErrorInvalidValue;
        if (!make_store_map(&map_h_store, a.h, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.max_rows, a.f)) return cudaErrorInvalidValue;
        if (!make_store_map(&map_y_store, a.y_packed, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.max_rows, a.d)) return cudaErrorInvalidValue;
        // CTA pairs pay when the reductions are long (their items use every accumulator column, so
        // an item boundary costs more) and there are rows for several rounds of 256 x 512 items
        const bool pairs_fit = a.d % 256 == 0 && a.n_sm >= 2 && (a.slot_region_bytes >> 7) < (1ull << 31);
        if (pairs_fit && (a.force_pairs || (a.d >= 4096 && a.max_rows >= 1536))) {
            alignas(64) CUtensorMap map_w;
            if (!make_weight_map(&map_w, a.slot_region, a.slot_region_bytes)) return cudaErrorInvalidValue;
            return launch_ffn_pair(a, tab, map_x, map_h, map_x128, map_h128, map_w, map_h_store, map_y_store, st, n_launch);
        }
        return launch_ffn_prefill(a, tab, map_x, map_h, map_x128, map_h128, map_x256, map_h256, map_h_store, map_y_store, st, n_launch);
    }
    // Small token tiles (decode): two CTAs per SM, each with half the shared memory, so that one
    // CTA's prologue, epilogue and split-item reduction overlap the other's streaming.
    const bool two_per_sm = a.n_tile <= 64;
    const int smem_budget = two_per_sm ? 108 * 1024 : kDynSmemMax;
    auto stages_for = [&](int w_bytes, int nt) {
        int sb = w_bytes + nt * 128;
        int s = (smem_budget - 1024) / sb;
        return s > kMaxStages ? kMaxStages : s;
    };
    const int s0 = stages_for(2 * kTileBytes, nt0), s1 = stages_for(kTileBytes, nt1);
    const size_t smem0 = (size_t)s0 * (2 * kTileBytes + nt0 * 128) + 1024;
    const size_t smem1 = (size_t)s1 * (kTileBytes + nt1 * 128) + 1024;
    FfnArgs args0 = a, args1 = a;
    args0.n_tile = nt0;
    args1.n_tile = nt1;
    args0.partial_slot_floats = (size_t)2 * nt0 * kTileRows;
    args1.partial_slot_floats = (size_t)2 * nt1 * kTileRows;
    const dim3 grid((unsigned)(two_per_sm ? 2 * a.n_sm : a.n_sm)), block(kThreads);
    cudaError_t e = launch_pdl(ffn_tensor_kernel<0>, grid, block, smem0, st, args0, tab, map_x, s0, box_rows);
    if (e != cudaSuccess) return e;
    e = launch_pdl(ffn_tensor_kernel<1>, grid, block, smem1, st, args1, tab, map_h, s1, box_rows);
    *n_launch = 2;
    return e;
}

}  // namespace saem
