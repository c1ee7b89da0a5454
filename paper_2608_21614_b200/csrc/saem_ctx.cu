// Host side of libsaem: context, workspace carving, expert-slot table with asynchronous loads
// (Sec. IV-C: fixed-size expert cache region, residency map, DMA + event prefetch), the offline
// weight packer, and the step drivers that chain the four kernels' launchers.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "saem_internal.h"

namespace saem {

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

int validate_config(const saem_config* c) {
    if (!c) return SAEM_ERR_INVALID_ARG;
    if (c->d_model <= 0 || c->d_ff <= 0 || c->d_model % 128 || c->d_ff % 128) return SAEM_ERR_SHAPE;
    if (c->d_model > 16384 || c->d_ff > 16384) return SAEM_ERR_SHAPE;      // a split item has at most 256 k-chunks
    if (c->n_experts < 1 || c->n_experts > SAEM_MAX_EXPERTS) return SAEM_ERR_SHAPE;
    if (c->top_k < 1 || c->top_k > c->n_experts) return SAEM_ERR_SHAPE;
    if (c->max_tokens < 1 || (long long)c->max_tokens * c->top_k > 65535) return SAEM_ERR_SHAPE;
    if (c->n_shared < 0 || c->n_shared > 16 || c->n_experts + c->n_shared > SAEM_MAX_EXPERTS) return SAEM_ERR_SHAPE;
    if (c->n_layers < 1 || c->slots_per_layer < 0 || c->slots_per_layer > c->n_experts + c->n_shared) return SAEM_ERR_SHAPE;
    if (c->temp_slots < 0 || c->temp_slots > 4096) return SAEM_ERR_SHAPE;
    if ((long long)c->n_layers * c->slots_per_layer + c->temp_slots < 1) return SAEM_ERR_SHAPE;
    if (c->out_dtype != SAEM_OUT_F32 && c->out_dtype != SAEM_OUT_BF16) return SAEM_ERR_INVALID_ARG;
    if (c->ffn_path < SAEM_FFN_AUTO || c->ffn_path > SAEM_FFN_DECODE_FUSED) return SAEM_ERR_INVALID_ARG;
    return SAEM_OK;
}

WorkspaceLayout workspace_layout(const saem_config& c) {
    WorkspaceLayout L{};
    const size_t A = 1024;
    size_t P = (size_t)c.max_tokens * c.top_k, T = c.max_tokens, d = c.d_model, f = c.d_ff;
    size_t E = (size_t)c.n_experts + c.n_shared;            // experts with a segment: routed, then shared
    size_t R = P + (size_t)c.n_shared * T;                  // packed rows: pairs, then T rows per shared expert
    // token tiles above 32 rows are loaded as 32-row boxes: keep them a whole number of boxes
    int nt = round_up(c.max_tokens < kMaxNTile ? c.max_tokens : kMaxNTile, 16);
    if (nt > 32) nt = round_up(nt, 32);
    L.n_tile_max = nt;
    L.partial_slot_floats = (size_t)2 * nt * kTileRows;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, A); return o; };
    L.status = take(256);
    L.counters = take(sizeof(int) * (2 * kMaxCtas + 16));
    L.decode_sync = take(sizeof(int) * kDecodeSyncInts);
    L.h = take(R * f * 2);
    {   // split-K partial tiles of the streaming kernels: token tiles of at most 64 rows, two slots per CTA
        size_t small_tile = (size_t)2 * (nt < 64 ? nt : 64) * kTileRows;
        L.partials = take((size_t)kMaxCtas * 2 * small_tile * sizeof(float));
    }
    {   // multi-CTA repack (more than 2048 pairs): at most 64 blocks of 1024 pairs
        const bool big = P > 2048;
        L.repack_hist = take(big ? (size_t)64 * SAEM_MAX_EXPERTS * 4 : 16);
        L.repack_rank = take(big ? (size_t)65536 * 2 : 16);
    }
    L.logits = take(T * (size_t)c.n_experts * 4);
    L.x = take(T * d * 2);
    L.topk_idx = take(P * 4);
    L.topk_w = take(P * 4);
    L.counts = take(E * 4);
    L.offsets = take((E + 1) * 4);
    L.perm = take(P * 4);
    L.inv_perm = take(P * 4);
    L.x_packed = take(R * d * 2);
    L.y_packed = take(R * d * 4);
    L.shared_y = take(T * d * 4);
    L.out = take(T * d * 4);
    L.total = off;
    return L;
}

static int n_tile_for(const saem_ctx* ctx, int max_rows) {
    int m = max_rows < ctx->cfg.max_tokens ? max_rows : ctx->cfg.max_tokens;   // a token picks an expert once
    if (m < 1) m = 1;
    int nt = round_up(m, 16);
    if (nt > 32) nt = round_up(nt, 32);
    if (nt > kMaxNTile) nt = kMaxNTile;
    if (nt > ctx->lay.n_tile_max) nt = ctx->lay.n_tile_max;
    return nt;
}

}  // namespace saem

using namespace saem;

#define CUDA_TRY(expr)                                 \
    do {                                               \
        cudaError_t e_ = (expr);                       \
        if (e_ != cudaSuccess) return SAEM_ERR_CUDA;   \
    } while (0)

extern "C" {

int saem_version(void) { return 100; }

const char* saem_status_string(int s) {
    switch (s) {
        case SAEM_OK: return "ok";
        case SAEM_ERR_INVALID_ARG: return "invalid argument";
        case SAEM_ERR_SHAPE: return "shape outside the supported range";
        case SAEM_ERR_ALIGNMENT: return "pointer alignment";
        case SAEM_ERR_WORKSPACE: return "workspace or slot region too small";
        case SAEM_ERR_NOT_RESIDENT: return "expert not resident";
        case SAEM_ERR_SLOT_BUSY: return "slot busy";
        case SAEM_ERR_TIMEOUT: return "bounded device wait ran out";
        case SAEM_ERR_CUDA: return "CUDA runtime error";
        case SAEM_ERR_UNSUPPORTED: return "unsupported configuration";
    }
    return "unknown status";
}

size_t saem_slot_bytes(const saem_config* c) {
    if (validate_config(c) != SAEM_OK) return 0;
    return (size_t)3 * c->d_model * c->d_ff * 2;
}

size_t saem_slot_region_bytes(const saem_config* c) {
    size_t sb = saem_slot_bytes(c);
    if (!sb) return 0;
    return sb * ((size_t)c->n_layers * c->slots_per_layer + c->temp_slots);
}

size_t saem_workspace_bytes(const saem_config* c) {
    if (validate_config(c) != SAEM_OK) return 0;
    return workspace_layout(*c).total;
}

int saem_create(const saem_config* cfg, void* slot_region, size_t slot_region_bytes, void* ws, size_t ws_bytes,
                saem_ctx** out) {
    if (!out) return SAEM_ERR_INVALID_ARG;
    *out = nullptr;
    int v = validate_config(cfg);
    if (v != SAEM_OK) return v;
    if (!slot_region || !ws) return SAEM_ERR_INVALID_ARG;
    if (((uintptr_t)slot_region | (uintptr_t)ws) & 1023) return SAEM_ERR_ALIGNMENT;
    if (slot_region_bytes < saem_slot_region_bytes(cfg)) return SAEM_ERR_WORKSPACE;
    WorkspaceLayout lay = workspace_layout(*cfg);
    if (ws_bytes < lay.total) return SAEM_ERR_WORKSPACE;

    saem_ctx* c = new (std::nothrow) saem_ctx();
    if (!c) return SAEM_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->lay = lay;
    c->slot_region = (uint8_t*)slot_region;
    c->slot_bytes = saem_slot_bytes(cfg);
    c->ws = (uint8_t*)ws;
    c->n_fixed_slots = cfg->n_layers * cfg->slots_per_layer;
    c->next_temp = 0;
    c->launches = 0;
    c->n_total = cfg->n_experts + cfg->n_shared;
    c->dynamic_residency = cfg->slots_per_layer < c->n_total || cfg->temp_slots > 0;
    int n_slots = c->n_fixed_slots + cfg->temp_slots;
    size_t LE = (size_t)cfg->n_layers * c->n_total;
    c->slot_of = (int32_t*)malloc(sizeof(int32_t) * LE);
    c->temp_of = (int32_t*)malloc(sizeof(int32_t) * LE);
    c->host_of = (const uint8_t**)calloc(LE, sizeof(const uint8_t*));
    c->slot_owner = (int32_t*)malloc(sizeof(int32_t) * n_slots);
    c->ready_ev = (cudaEvent_t*)calloc(n_slots, sizeof(cudaEvent_t));
    c->ev_pending = (uint8_t*)calloc(n_slots, 1);
    c->ev_recorded = (uint8_t*)calloc(n_slots, 1);
    c->read_ev = (cudaEvent_t*)calloc(cfg->n_layers, sizeof(cudaEvent_t));
    c->read_recorded = (uint8_t*)calloc(cfg->n_layers, 1);
    c->temp_last_layer = (int32_t*)malloc(sizeof(int32_t) * (cfg->temp_slots > 0 ? cfg->temp_slots : 1));
    c->last_stream = (cudaStream_t*)calloc(cfg->n_layers, sizeof(cudaStream_t));
    c->ffn_seen = (uint8_t*)calloc(cfg->n_layers, 1);
    c->pinned_status = nullptr;
    for (size_t i = 0; i < LE; ++i) c->slot_of[i] = c->temp_of[i] = -1;
    for (int i = 0; i < n_slots; ++i) c->slot_owner[i] = -1;
    for (int i = 0; i < cfg->temp_slots; ++i) c->temp_last_layer[i] = -1;

    bool ok = cudaGetDevice(&c->device) == cudaSuccess;
    ok = ok && cudaDeviceGetAttribute(&c->n_sm, cudaDevAttrMultiProcessorCount, c->device) == cudaSuccess;
    if (ok && c->n_sm > kMaxSms) c->n_sm = kMaxSms;
    for (int i = 0; ok && i < n_slots; ++i)
        ok = cudaEventCreateWithFlags(&c->ready_ev[i], cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < cfg->n_layers; ++i)
        ok = cudaEventCreateWithFlags(&c->read_ev[i], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaHostAlloc((void**)&c->pinned_status, sizeof(int), cudaHostAllocDefault) == cudaSuccess;
    // the status word, the arrival counters and the decode step's barrier / tickets start at zero; nothing else needs clearing
    ok = ok && cudaMemsetAsync(c->ws + lay.status, 0, lay.h - lay.status, 0) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(0) == cudaSuccess;
    if (ok && cfg->ffn_path != SAEM_FFN_SCALAR) ok = ffn_tensor_init() == cudaSuccess;
    if (!ok) {
        saem_destroy(c);
        return SAEM_ERR_CUDA;
    }
    *out = c;
    return SAEM_OK;
}

void saem_destroy(saem_ctx* c) {
    if (!c) return;
    int n_slots = c->n_fixed_slots + c->cfg.temp_slots;
    if (c->ready_ev)
        for (int i = 0; i < n_slots; ++i)
            if (c->ready_ev[i]) cudaEventDestroy(c->ready_ev[i]);
    if (c->read_ev)
        for (int i = 0; i < c->cfg.n_layers; ++i)
            if (c->read_ev[i]) cudaEventDestroy(c->read_ev[i]);
    if (c->pinned_status) cudaFreeHost(c->pinned_status);
    free(c->slot_of); free(c->temp_of); free(c->host_of); free(c->slot_owner); free(c->ready_ev); free(c->ev_pending);
    free(c->ev_recorded); free(c->read_ev); free(c->read_recorded); free(c->temp_last_layer); free(c->last_stream); free(c->ffn_seen);
    delete c;
}

// ------------------------------------------------------------------------------------ weight packer
// Tile (rb, kc) of a [rows, K] row-major matrix: 128 rows x 64 elements; row r of the tile is
// 128 bytes; its 16-byte chunk c lands at chunk position c ^ (r & 7).
static void pack_matrix(const uint16_t* src, int rows, int K, uint8_t* dst, size_t tile_stride_bytes,
                        size_t first_tile_offset) {
    int RB = rows / kTileRows, KC = K / kTileK;
    for (int rb = 0; rb < RB; ++rb)
        for (int kc = 0; kc < KC; ++kc) {
            uint8_t* tile = dst + first_tile_offset + ((size_t)rb * KC + kc) * tile_stride_bytes;
            for (int r = 0; r < kTileRows; ++r) {
                const uint16_t* s = src + (size_t)(rb * kTileRows + r) * K + (size_t)kc * kTileK;
                for (int ch = 0; ch < 8; ++ch)
                    memcpy(tile + (size_t)r * 128 + (size_t)((ch ^ (r & 7)) * 16), s + ch * 8, 16);
            }
        }
}

int saem_pack_expert_host(const saem_config* cfg, const void* gate, const void* up, const void* down, void* out) {
    int v = validate_config(cfg);
    if (v != SAEM_OK) return v;
    if (!gate || !up || !down || !out) return SAEM_ERR_INVALID_ARG;
    int d = cfg->d_model, f = cfg->d_ff;
    uint8_t* o = (uint8_t*)out;
    // gate/up region: per (f-block, k-chunk) a gate tile followed by the matching up tile
    pack_matrix((const uint16_t*)gate, f, d, o, 2 * kTileBytes, 0);
    pack_matrix((const uint16_t*)up, f, d, o, 2 * kTileBytes, kTileBytes);
    // down region: per (d-block, k-chunk over f) one tile
    pack_matrix((const uint16_t*)down, d, f, o + (size_t)2 * d * f * 2, kTileBytes, 0);
    return SAEM_OK;
}

// ------------------------------------------------------------------------------------------- steps
static bool misaligned(const void* p) { return ((uintptr_t)p & 15) != 0; }

static int check_T(saem_ctx* c, int T) {
    if (!c) return SAEM_ERR_INVALID_ARG;
    if (T < 0 || T > c->cfg.max_tokens) return SAEM_ERR_SHAPE;
    return SAEM_OK;
}

int saem_route(saem_ctx* c, const float* logits, int T, int32_t* idx, float* w, void* stream) {
    int s = check_T(c, T);
    if (s != SAEM_OK) return s;
    if (T == 0) return SAEM_OK;
    if (!logits || !idx || !w) return SAEM_ERR_INVALID_ARG;
    CUDA_TRY(launch_route(logits, T, c->cfg.n_experts, c->cfg.top_k, c->cfg.renorm, idx, w, (cudaStream_t)stream));
    c->launches += 1;
    return SAEM_OK;
}

int saem_route_fused(saem_ctx* c, const void* x, const void* w_router, int T, float* logits_out, int32_t* idx,
                     float* w, void* stream) {
    int s = check_T(c, T);
    if (s != SAEM_OK) return s;
    if (T == 0) return SAEM_OK;
    if (!x || !w_router || !idx || !w) return SAEM_ERR_INVALID_ARG;
    if (misaligned(x) || misaligned(w_router)) return SAEM_ERR_ALIGNMENT;
    CUDA_TRY(launch_route_fused((const uint16_t*)x, (const uint16_t*)w_router, T, c->cfg.n_experts, c->cfg.d_model,
                                c->cfg.top_k, c->cfg.renorm, logits_out, idx, w, (cudaStream_t)stream));
    c->launches += 1;
    return SAEM_OK;
}

int saem_repack(saem_ctx* c, const int32_t* idx, const void* x, int T, int32_t* counts, int32_t* offsets,
                int32_t* perm, int32_t* inv_perm, void* x_packed, void* stream) {
    int s = check_T(c, T);
    if (s != SAEM_OK) return s;
    if (!counts || !offsets) return SAEM_ERR_INVALID_ARG;
    if (T > 0 && (!idx || !x || !perm || !inv_perm || !x_packed)) return SAEM_ERR_INVALID_ARG;
    if (misaligned(x) || misaligned(x_packed)) return SAEM_ERR_ALIGNMENT;
    int nl = 0;
    CUDA_TRY(launch_repack(idx, (const uint16_t*)x, T, c->cfg.n_experts, c->cfg.n_shared, c->cfg.top_k, c->cfg.d_model, counts,
                           offsets, perm, inv_perm, (uint16_t*)x_packed, (int*)(c->ws + c->lay.status),
                           (int32_t*)(c->ws + c->lay.repack_hist), (uint16_t*)(c->ws + c->lay.repack_rank), c->n_sm,
                           (cudaStream_t)stream, &nl));
    c->launches += nl;
    return SAEM_OK;
}

// Slot of every expert of `layer` for one FFN launch (fixed slot, else temporary binding, else -1),
// and `st` ordered after the loads still in flight for those slots.
static int resolve_slots(saem_ctx* c, int layer, const int32_t* subset, int n_subset, cudaStream_t st, SlotTable& tab,
                         bool host_mapped_ok = false) {
    const int ES = c->n_total;
    const int32_t* so = c->slot_of + (size_t)layer * ES;
    const int32_t* to = c->temp_of + (size_t)layer * ES;
    const uint8_t* const* ho = c->host_of + (size_t)layer * ES;
    for (int e = 0; e < SAEM_MAX_EXPERTS; ++e) { tab.slot[e] = -1; tab.in_subset[e] = 0; }
    for (int i = 0; i < kMaxHostMapped; ++i) tab.host[i] = nullptr;
    int n_host = 0;
    bool too_many = false;
    // fixed slot, else temporary binding, else (where the kernels can read it) mapped host memory
    auto resolve = [&](int e) -> int {
        if (so[e] >= 0) return so[e];
        if (to[e] >= 0) return to[e];
        if (ho[e] && host_mapped_ok) {
            if (n_host == kMaxHostMapped) { too_many = true; return -1; }
            tab.host[n_host] = ho[e];
            return -(2 + n_host++);
        }
        return -1;
    };
    if (subset) {
        for (int i = 0; i < n_subset; ++i) {
            int e = subset[i];
            if (e < 0 || e >= ES) return SAEM_ERR_INVALID_ARG;
            if (so[e] < 0 && to[e] < 0 && !(ho[e] && host_mapped_ok)) return SAEM_ERR_NOT_RESIDENT;
        }
        for (int i = 0; i < n_subset; ++i) {
            if (!tab.in_subset[subset[i]]) tab.slot[subset[i]] = resolve(subset[i]);
            tab.in_subset[subset[i]] = 1;
        }
    } else {
        for (int e = 0; e < ES; ++e) { tab.slot[e] = resolve(e); tab.in_subset[e] = 1; }
    }
    if (too_many) return SAEM_ERR_UNSUPPORTED;
    // order this stream after loads still in flight for the slots it may read
    for (int e = 0; e < ES; ++e) {
        int s = tab.slot[e];
        if (s < 0 || !c->ev_pending[s]) continue;
        cudaError_t q = cudaEventQuery(c->ready_ev[s]);
        if (q == cudaSuccess) { c->ev_pending[s] = 0; continue; }
        if (q != cudaErrorNotReady) return SAEM_ERR_CUDA;
        CUDA_TRY(cudaStreamWaitEvent(st, c->ready_ev[s], 0));
    }
    return SAEM_OK;
}

// Book-keeping after an FFN of `layer` has been enqueued on `st`: later loads into the slots it reads
// must wait for it.
static int note_ffn_enqueued(saem_ctx* c, int layer, cudaStream_t st, const SlotTable& tab) {
    c->last_stream[layer] = st;
    c->ffn_seen[layer] = 1;
    if (c->dynamic_residency) {
        CUDA_TRY(cudaEventRecord(c->read_ev[layer], st));
        c->read_recorded[layer] = 1;
        for (int e = 0; e < c->n_total; ++e) {
            int s = tab.slot[e];
            if (s >= c->n_fixed_slots) c->temp_last_layer[s - c->n_fixed_slots] = layer;
        }
    }
    return SAEM_OK;
}

int saem_expert_ffn(saem_ctx* c, int layer, const void* x_packed, const int32_t* offsets, int max_rows,
                    const int32_t* subset, int n_subset, float* y_packed, void* stream) {
    if (!c) return SAEM_ERR_INVALID_ARG;
    const saem_config& g = c->cfg;
    if (layer < 0 || layer >= g.n_layers) return SAEM_ERR_INVALID_ARG;
    if (max_rows < 0 || max_rows > g.max_tokens * (g.top_k + g.n_shared)) return SAEM_ERR_SHAPE;
    if (max_rows == 0) return SAEM_OK;
    if (!x_packed || !y_packed) return SAEM_ERR_INVALID_ARG;
    const int ES = c->n_total;
    if (!offsets && ES != 1) return SAEM_ERR_INVALID_ARG;
    if (misaligned(x_packed) || misaligned(y_packed)) return SAEM_ERR_ALIGNMENT;
    if (subset && n_subset < 0) return SAEM_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;

    const int seg_bound = max_rows < g.max_tokens ? max_rows : g.max_tokens;     // a token picks an expert once
    const bool gemv_path = (g.ffn_path == SAEM_FFN_AUTO || g.ffn_path == SAEM_FFN_DECODE_FUSED) && seg_bound <= 8;
    SlotTable tab;
    {
        int r = resolve_slots(c, layer, subset, n_subset, st, tab, gemv_path);
        if (r != SAEM_OK) return r;
    }

    FfnArgs a;
    a.x_packed = (const uint16_t*)x_packed;
    a.offsets = offsets;
    a.max_rows = max_rows;
    a.E = ES; a.d = g.d_model; a.f = g.d_ff;
    a.slot_region = c->slot_region;
    a.slot_bytes = c->slot_bytes;
    a.slot_region_bytes = c->slot_bytes * (size_t)(c->n_fixed_slots + c->cfg.temp_slots);
    a.h = (uint16_t*)(c->ws + c->lay.h);
    a.y_packed = y_packed;
    a.status = (int*)(c->ws + c->lay.status);
    a.counters = (int*)(c->ws + c->lay.counters);
    a.partials = (float*)(c->ws + c->lay.partials);
    a.partial_slot_floats = c->lay.partial_slot_floats;
    a.n_tile = n_tile_for(c, max_rows);
    {
        // max_rows = T * (top_k + n_shared): at most T * top_k routed experts and the n_shared shared ones have rows
        int t = (max_rows + g.top_k + g.n_shared - 1) / (g.top_k + g.n_shared);
        long long bound = (long long)t * g.top_k + g.n_shared;
        a.max_active = bound < ES ? (int)bound : ES;
    }
    a.n_sm = c->n_sm;
    a.force_pairs = g.ffn_path == SAEM_FFN_TENSOR_PAIRS;
    // AUTO: the tiled kernels take every launch beyond the matrix-vector kernels' 8 rows (measured on whole layers:
    // shorter steps on every shape) -- provided the launch can have enough whole items to occupy the SMs.  The tiled
    // kernels deal whole (expert, 256-row weight block) items, so a launch of one or two experts (a subset, a shared
    // expert in a context of its own) would leave most SMs idle in the down projection; the streaming kernels cut
    // their work at k-chunk granularity and keep every SM busy.  It matters when an item is long (one Mixtral-shaped
    // expert, d_ff 14336, at 16..64 rows: 82-102 us streaming against 127-136 us tiled); with short items the tiled
    // kernels stay ahead even for a single expert (d_ff 1408: 30-32 us against 33-46 us).
    {
        const long long experts_bound = subset ? n_subset : a.max_active;
        const bool enough_items = experts_bound * ((g.d_model + 255) / 256) * 4 >= 3LL * c->n_sm;
        const bool auto_path = g.ffn_path == SAEM_FFN_AUTO || g.ffn_path == SAEM_FFN_DECODE_FUSED;
        a.stream_max_tile = (auto_path && (enough_items || g.d_ff < 4096)) ? 0 : 64;
    }
    int nl = 0;
    if (g.ffn_path == SAEM_FFN_SCALAR) {
        CUDA_TRY(launch_ffn_scalar(a, tab, st, &nl));
    } else if (gemv_path) {
        CUDA_TRY(launch_ffn_gemv(a, tab, st, &nl));
    } else {
        CUDA_TRY(launch_ffn_tensor(a, tab, st, &nl));
    }
    c->launches += nl;
    return note_ffn_enqueued(c, layer, st, tab);
}

int saem_combine(saem_ctx* c, const float* y, const int32_t* inv_perm, const float* w, int T, const float* shared_y,
                 void* out, void* stream) {
    int s = check_T(c, T);
    if (s != SAEM_OK) return s;
    if (T == 0) return SAEM_OK;
    if (!y || !inv_perm || !w || !out) return SAEM_ERR_INVALID_ARG;
    if (misaligned(y) || misaligned(out) || misaligned(shared_y)) return SAEM_ERR_ALIGNMENT;
    CUDA_TRY(launch_combine(y, inv_perm, w, T, c->cfg.top_k, c->cfg.n_shared, c->cfg.d_model, shared_y, out,
                            c->cfg.out_dtype == SAEM_OUT_BF16, (cudaStream_t)stream));
    c->launches += 1;
    return SAEM_OK;
}

void* saem_step_buffer(saem_ctx* c, int which) {
    if (!c) return nullptr;
    const WorkspaceLayout& L = c->lay;
    size_t offs[11] = {L.topk_idx, L.topk_w, L.counts, L.offsets, L.perm, L.inv_perm, L.x_packed, L.y_packed,
                       L.shared_y, L.h, L.counters};
    if (which < 0 || which >= 11) return nullptr;
    return c->ws + offs[which];
}

int saem_moe_step(saem_ctx* c, saem_ctx* sh, int layer, const float* logits, const void* x, int T, void* out,
                  void* stream) {
    int s = check_T(c, T);
    if (s != SAEM_OK) return s;
    if (T == 0) return SAEM_OK;
    if (!logits || !x || !out) return SAEM_ERR_INVALID_ARG;
    const saem_config& g = c->cfg;
    if (sh && (sh->cfg.n_experts != 1 || sh->cfg.top_k != 1 || sh->cfg.d_model != g.d_model ||
               sh->cfg.max_tokens < T || layer >= sh->cfg.n_layers))
        return SAEM_ERR_INVALID_ARG;
    uint8_t* w = c->ws;
    const WorkspaceLayout& L = c->lay;
    int32_t* idx = (int32_t*)(w + L.topk_idx);
    float* tw = (float*)(w + L.topk_w);
    int32_t* offsets = (int32_t*)(w + L.offsets);
    int32_t* inv = (int32_t*)(w + L.inv_perm);
    float* y = (float*)(w + L.y_packed);
    float* shy = (float*)(w + L.shared_y);
    bool host_mapped = false;
    if (layer >= 0 && layer < g.n_layers)
        for (int e = 0; e < c->n_total; ++e) host_mapped = host_mapped || c->host_of[(size_t)layer * c->n_total + e] != nullptr;
    // SAEM_FFN_AUTO takes the one-launch form up to 4 tokens, and up to 8 where it was measured ahead of the five
    // launches: experts of at most 20 MB (a short step, of which the launches' fixed costs are a visible part; the
    // ERNIE shape's 23.6 MB experts tie, the Mixtral shape's 352 MB lose 5 %) and enough (expert, 32 columns) units in
    // the down projection for the even unit-major deal (fewer are dealt whole, some CTAs one more than others).
    bool auto_fused = T <= kDecodeFusedAutoTokens;
    if (!auto_fused && T <= 8) {
        const long long expert_bytes = 3ll * g.d_model * g.d_ff * 2;
        const long long pairs = (long long)T * g.top_k;
        const long long units = ((pairs < g.n_experts ? pairs : g.n_experts) + g.n_shared) * (g.d_model / 32);
        auto_fused = expert_bytes <= 20ll * 1024 * 1024 && units >= 8ll * c->n_sm;
    }
    if (!sh && !host_mapped && decode_fused_supported(T, g.top_k) &&
        (g.ffn_path == SAEM_FFN_DECODE_FUSED || (g.ffn_path == SAEM_FFN_AUTO && auto_fused))) {
        // The smallest decode batches: one launch for the whole step (gate + repack indices + gate/up,
        // grid barrier, down + merge); x_packed is not produced.
        if (layer < 0 || layer >= g.n_layers) return SAEM_ERR_INVALID_ARG;
        if (misaligned(x) || misaligned(out)) return SAEM_ERR_ALIGNMENT;
        cudaStream_t st = (cudaStream_t)stream;
        SlotTable tab;
        if ((s = resolve_slots(c, layer, nullptr, 0, st, tab)) != SAEM_OK) return s;
        DecodeArgs a;
        a.logits = logits; a.x = (const uint16_t*)x;
        a.T = T; a.E = g.n_experts; a.S = g.n_shared; a.k = g.top_k; a.d = g.d_model; a.f = g.d_ff; a.renorm = g.renorm;
        a.slot_region = c->slot_region; a.slot_bytes = c->slot_bytes;
        a.h = (uint16_t*)(w + L.h);
        a.y_packed = y;
        a.sync = (int*)(w + L.decode_sync);
        a.out = out; a.out_bf16 = g.out_dtype == SAEM_OUT_BF16;
        a.topk_idx = idx; a.topk_w = tw; a.counts = (int32_t*)(w + L.counts); a.offsets = offsets;
        a.perm = (int32_t*)(w + L.perm); a.inv_perm = inv;
        a.status = (int*)(w + L.status);
        int nl = 0;
        CUDA_TRY(launch_decode_fused(a, tab, c->n_sm, st, &nl));
        c->launches += nl;
        return note_ffn_enqueued(c, layer, st, tab);
    }
    if ((s = saem_route(c, logits, T, idx, tw, stream)) != SAEM_OK) return s;
    if ((s = saem_repack(c, idx, x, T, (int32_t*)(w + L.counts), offsets, (int32_t*)(w + L.perm), inv,
                         w + L.x_packed, stream)) != SAEM_OK) return s;
    if ((s = saem_expert_ffn(c, layer, w + L.x_packed, offsets, T * (g.top_k + g.n_shared), nullptr, 0, y, stream)) != SAEM_OK)
        return s;
    if (sh && (s = saem_expert_ffn(sh, layer, x, nullptr, T, nullptr, 0, shy, stream)) != SAEM_OK) return s;
    return saem_combine(c, y, inv, tw, T, sh ? shy : nullptr, out, stream);
}

static int step_from_host(saem_ctx* c, saem_ctx* sh, int layer, const float* logits_h, const void* x_h, int T, void* out_h,
                          void* stream, bool synchronise) {
    int s = check_T(c, T);
    if (s != SAEM_OK) return s;
    if (T == 0) return SAEM_OK;
    if (!logits_h || !x_h || !out_h) return SAEM_ERR_INVALID_ARG;
    const saem_config& g = c->cfg;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* w = c->ws;
    const WorkspaceLayout& L = c->lay;
    size_t out_bytes = (size_t)T * g.d_model * (g.out_dtype == SAEM_OUT_BF16 ? 2 : 4);
    CUDA_TRY(cudaMemcpyAsync(w + L.logits, logits_h, (size_t)T * g.n_experts * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(w + L.x, x_h, (size_t)T * g.d_model * 2, cudaMemcpyHostToDevice, st));
    s = saem_moe_step(c, sh, layer, (const float*)(w + L.logits), w + L.x, T, w + L.out, stream);
    if (s != SAEM_OK) return s;
    CUDA_TRY(cudaMemcpyAsync(out_h, w + L.out, out_bytes, cudaMemcpyDeviceToHost, st));
    if (synchronise) CUDA_TRY(cudaStreamSynchronize(st));
    return SAEM_OK;
}

int saem_moe_step_host(saem_ctx* c, saem_ctx* sh, int layer, const float* logits_h, const void* x_h, int T, void* out_h,
                       void* stream) {
    return step_from_host(c, sh, layer, logits_h, x_h, T, out_h, stream, true);
}

int saem_moe_step_host_async(saem_ctx* c, saem_ctx* sh, int layer, const float* logits_h, const void* x_h, int T,
                             void* out_h, void* stream) {
    return step_from_host(c, sh, layer, logits_h, x_h, T, out_h, stream, false);
}

// ------------------------------------------------------------------------------------------- cache
static int check_le(saem_ctx* c, int layer, int expert) {
    if (!c) return SAEM_ERR_INVALID_ARG;
    if (layer < 0 || layer >= c->cfg.n_layers || expert < 0 || expert >= c->n_total) return SAEM_ERR_INVALID_ARG;
    return SAEM_OK;
}

int saem_cache_load(saem_ctx* c, int layer, int expert, int slot, const void* pinned, void* copy_stream) {
    int s = check_le(c, layer, expert);
    if (s != SAEM_OK) return s;
    if (!pinned) return SAEM_ERR_INVALID_ARG;
    const saem_config& g = c->cfg;
    size_t le = (size_t)layer * c->n_total + expert;
    cudaStream_t cs = (cudaStream_t)copy_stream;
    // Work out the slot first, enqueue the wait / copy / event, and only then change the host tables:
    // if a CUDA call fails nothing is marked resident that was never copied.
    int gslot, temp_index = -1;
    int wait_layer = -1;
    if (slot == SAEM_TEMP) {
        if (g.temp_slots < 1) return SAEM_ERR_INVALID_ARG;
        if (c->slot_of[le] >= 0) return SAEM_ERR_INVALID_ARG;
        temp_index = c->next_temp;
        gslot = c->n_fixed_slots + temp_index;
        wait_layer = c->temp_last_layer[temp_index];
    } else {
        if (slot < 0 || slot >= g.slots_per_layer) return SAEM_ERR_INVALID_ARG;
        if (c->slot_of[le] >= 0) return SAEM_ERR_INVALID_ARG;
        gslot = layer * g.slots_per_layer + slot;
        if (c->slot_owner[gslot] >= 0) return SAEM_ERR_SLOT_BUSY;
        wait_layer = layer;
    }
    // the copy must not overtake an enqueued FFN that still reads the slot's previous content
    if (wait_layer >= 0 && !c->read_recorded[wait_layer] && c->ffn_seen[wait_layer]) {
        // fully resident configurations record no event per FFN: mark the tail of that layer's
        // compute stream now (everything enqueued so far, hence every FFN that reads the slot)
        if (cudaEventRecord(c->read_ev[wait_layer], c->last_stream[wait_layer]) != cudaSuccess) return SAEM_ERR_CUDA;
        if (cudaStreamWaitEvent(cs, c->read_ev[wait_layer], 0) != cudaSuccess) return SAEM_ERR_CUDA;
    } else if (wait_layer >= 0 && c->read_recorded[wait_layer]) {
        if (cudaStreamWaitEvent(cs, c->read_ev[wait_layer], 0) != cudaSuccess) return SAEM_ERR_CUDA;
    }
    if (cudaMemcpyAsync(c->slot_region + (size_t)gslot * c->slot_bytes, pinned, c->slot_bytes, cudaMemcpyHostToDevice,
                        cs) != cudaSuccess)
        return SAEM_ERR_CUDA;
    if (cudaEventRecord(c->ready_ev[gslot], cs) != cudaSuccess) {
        // the copy is enqueued but cannot be waited for: whatever the slot held is no longer valid
        if (c->slot_owner[gslot] >= 0) { c->temp_of[c->slot_owner[gslot]] = -1; c->slot_owner[gslot] = -1; }
        return SAEM_ERR_CUDA;
    }
    if (slot == SAEM_TEMP) {
        c->next_temp = (temp_index + 1) % g.temp_slots;
        if (c->slot_owner[gslot] >= 0) c->temp_of[c->slot_owner[gslot]] = -1;   // drop the old binding
        if (c->temp_of[le] >= 0) c->slot_owner[c->temp_of[le]] = -1;             // expert re-bound: free its old temp slot
        c->temp_of[le] = gslot;
    } else {
        c->slot_of[le] = gslot;
    }
    c->slot_owner[gslot] = (int32_t)le;
    c->ev_pending[gslot] = 1;
    c->ev_recorded[gslot] = 1;
    return SAEM_OK;
}

int saem_cache_map_host(saem_ctx* c, int layer, int expert, const void* pinned) {
    int s = check_le(c, layer, expert);
    if (s != SAEM_OK) return s;
    if (!pinned || ((uintptr_t)pinned & 15)) return pinned ? SAEM_ERR_ALIGNMENT : SAEM_ERR_INVALID_ARG;
    size_t le = (size_t)layer * c->n_total + expert;
    if (c->slot_of[le] >= 0 || c->temp_of[le] >= 0) return SAEM_ERR_INVALID_ARG;     // it has a slot: evict first
    void* dev = nullptr;
    if (cudaHostGetDevicePointer(&dev, const_cast<void*>(pinned), 0) != cudaSuccess || !dev) {
        (void)cudaGetLastError();
        return SAEM_ERR_INVALID_ARG;                                                  // not mapped pinned memory
    }
    c->host_of[le] = (const uint8_t*)dev;
    return SAEM_OK;
}

int saem_cache_evict(saem_ctx* c, int layer, int expert) {
    int s = check_le(c, layer, expert);
    if (s != SAEM_OK) return s;
    size_t le = (size_t)layer * c->n_total + expert;
    if (c->host_of[le]) {
        c->host_of[le] = nullptr;
        if (c->slot_of[le] < 0 && c->temp_of[le] < 0) return SAEM_OK;
    }
    if (c->slot_of[le] >= 0) {
        c->slot_owner[c->slot_of[le]] = -1;
        c->slot_of[le] = -1;
        return SAEM_OK;
    }
    if (c->temp_of[le] >= 0) {
        c->slot_owner[c->temp_of[le]] = -1;
        c->temp_of[le] = -1;
        return SAEM_OK;
    }
    return SAEM_ERR_NOT_RESIDENT;
}

int saem_cache_query(saem_ctx* c, int layer, int expert, int* slot, int* ready) {
    int s = check_le(c, layer, expert);
    if (s != SAEM_OK) return s;
    size_t le = (size_t)layer * c->n_total + expert;
    int gs = c->slot_of[le] >= 0 ? c->slot_of[le] : c->temp_of[le];
    if (gs < 0 && c->host_of[le]) {                  // bound to mapped host memory: nothing to wait for
        if (slot) *slot = SAEM_HOST_MAPPED;
        if (ready) *ready = 1;
        return SAEM_OK;
    }
    if (slot) *slot = gs;
    if (ready) {
        *ready = 0;
        if (gs >= 0 && c->ev_recorded[gs]) {
            cudaError_t q = cudaEventQuery(c->ready_ev[gs]);
            if (q == cudaSuccess) { *ready = 1; c->ev_pending[gs] = 0; }
            else if (q != cudaErrorNotReady) return SAEM_ERR_CUDA;
        }
    }
    return SAEM_OK;
}

int saem_cache_wait(saem_ctx* c, int layer, int expert, void* consumer) {
    int s = check_le(c, layer, expert);
    if (s != SAEM_OK) return s;
    size_t le = (size_t)layer * c->n_total + expert;
    int gs = c->slot_of[le] >= 0 ? c->slot_of[le] : c->temp_of[le];
    if (gs < 0 || !c->ev_recorded[gs]) return SAEM_ERR_NOT_RESIDENT;
    CUDA_TRY(cudaStreamWaitEvent((cudaStream_t)consumer, c->ready_ev[gs], 0));
    return SAEM_OK;
}

int saem_last_device_status(saem_ctx* c, int* code) {
    if (!c || !code) return SAEM_ERR_INVALID_ARG;
    CUDA_TRY(cudaDeviceSynchronize());
    CUDA_TRY(cudaMemcpy(c->pinned_status, c->ws + c->lay.status, sizeof(int), cudaMemcpyDeviceToHost));
    *code = *c->pinned_status;
    CUDA_TRY(cudaMemset(c->ws + c->lay.status, 0, sizeof(int)));
    // a CTA that gave up a bounded wait skipped its arrival on a split item's counter: start the next
    // launch from clean counters (nothing is in flight after the synchronisation above)
    if (*code == SAEM_ERR_TIMEOUT) CUDA_TRY(cudaMemset(c->ws + c->lay.counters, 0, c->lay.h - c->lay.counters));
    return SAEM_OK;
}

long long saem_launch_count(saem_ctx* c) { return c ? c->launches : 0; }

int saem_selftest_bounded_wait(saem_ctx* c, int limit_us, void* stream) {
    if (!c || limit_us < 1 || limit_us > 1000000) return SAEM_ERR_INVALID_ARG;
    CUDA_TRY(launch_bounded_wait_selftest((int*)(c->ws + c->lay.status), (unsigned long long)limit_us * 1000ull,
                                          (cudaStream_t)stream));
    c->launches += 1;
    return SAEM_OK;
}

}  // extern "C"
