// Internal declarations shared by the translation units of libsaem (host context + kernels).
#ifndef SAEM_INTERNAL_H_
#define SAEM_INTERNAL_H_

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "saem.h"

namespace saem {

constexpr int kTileRows = 128;              // weight rows per tile (the MMA M)
constexpr int kTileK = 64;                  // reduction elements per tile (128 bytes of bf16)
constexpr int kTileBytes = kTileRows * kTileK * 2;   // 16 KB
constexpr int kMaxCtas = 320;               // upper bound of the persistent grid (two CTAs per SM on 148 SMs)
constexpr int kMaxSms = 160;
constexpr int kMaxNTile = 256;              // widest token tile (the MMA N)

// Slot index per expert for one FFN launch; travels as a kernel parameter so that the residency
// table never needs a device mirror.  -1: the expert has no slot or is outside the subset.
// An expert bound to mapped pinned host memory (saem_cache_map_host) has slot -(2 + i) and its weights at
// host[i]; only the matrix-vector kernels read such experts, every other kernel sees them as absent.
constexpr int kMaxHostMapped = 8;
struct SlotTable {
    int32_t slot[SAEM_MAX_EXPERTS];
    uint8_t in_subset[SAEM_MAX_EXPERTS];    // 0: skip silently (not asked for)
    const uint8_t* host[kMaxHostMapped];
};

struct WorkspaceLayout {
    size_t status;        // int32 status word (+ padding)
    size_t counters;      // int32[2 * kMaxCtas + 16] split-K arrival counters (gate/up, down) of the streaming kernels; the tiled
                          // kernels keep per-expert "h complete" / "seen" counts and the down launch's item counter there
    size_t decode_sync;   // int32[kDecodeSyncInts] grid barrier and (column group, token) tickets of the one-launch decode step
    size_t h;             // bf16 [max_rows, d_ff]
    size_t partials;      // fp32 [CTAs][2][2][n_tile][128]: 2 CTAs/SM for n_tile <= 64, else 1 CTA/SM
    size_t repack_hist;   // int32 [64][SAEM_MAX_EXPERTS] per-block histograms of the multi-CTA repack
    size_t repack_rank;   // uint16 [65536] rank of a pair inside its block and expert
    size_t logits, x, topk_idx, topk_w, counts, offsets, perm, inv_perm, x_packed, y_packed, shared_y, out;
    size_t total;
    int n_tile_max;
    size_t partial_slot_floats;   // floats of one partial slot (2 accumulators)
};

WorkspaceLayout workspace_layout(const saem_config& c);
int validate_config(const saem_config* c);
inline int round_up(int a, int b) { return (a + b - 1) / b * b; }

// Launch with programmatic stream serialization: the kernel may start while the previous kernel of
// the stream is still draining; every kernel launched this way executes `griddepcontrol.wait`
// (pdl_wait) before it reads or writes anything a predecessor may touch.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
// The same for a kernel that runs as clusters of two CTAs (grid.x must be even).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_pairs(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args... args) {
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
// Function attributes (large dynamic shared memory) are per device: returns true the first time it is
// called for the current device with this flag array.
inline bool first_call_on_device(bool (&done)[64]) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;
    if (done[dev]) return false;
    done[dev] = true;
    return true;
}
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

// ---- kernel launchers (each returns a cudaError_t from the launch) ----
cudaError_t launch_route(const float* logits, int T, int E, int k, int renorm, int32_t* idx, float* w,
                         cudaStream_t st);
cudaError_t launch_route_fused(const uint16_t* x, const uint16_t* w_router, int T, int E, int d, int k, int renorm,
                               float* logits_out, int32_t* idx, float* w, cudaStream_t st);
// Returns the number of kernels launched (1 or 3) in *n_launch.  hist [ceil(P / 1024)][E] and rank16 [P]: workspace
// of the multi-CTA index phase (more than 2048 pairs).
cudaError_t launch_repack(const int32_t* idx, const uint16_t* x, int T, int E, int S, int k, int d, int32_t* counts,
                          int32_t* offsets, int32_t* perm, int32_t* inv_perm, uint16_t* x_packed, int* status,
                          int32_t* hist, uint16_t* rank16, int n_sm, cudaStream_t st, int* n_launch);
cudaError_t launch_combine(const float* y, const int32_t* inv_perm, const float* w, int T, int k, int S, int d,
                           const float* shared_y, void* out, int out_bf16, cudaStream_t st);

struct FfnArgs {
    const uint16_t* x_packed;   // [max_rows, d]
    const int32_t* offsets;     // [E+1] or nullptr (E == 1: one segment [0, max_rows))
    int max_rows;
    int E, d, f;
    const uint8_t* slot_region;
    size_t slot_bytes;
    size_t slot_region_bytes;   // whole region (every slot)
    uint16_t* h;                // [max_rows, f] bf16 workspace
    float* y_packed;            // [max_rows, d]
    int* status;
    int* counters;              // [2 * kMaxCtas + 16]
    float* partials;
    size_t partial_slot_floats;
    int n_tile;                 // token tile for this launch (multiple of 16, <= 256)
    int max_active;             // upper bound of experts with rows: min(E, T * top_k + n_shared)
    int n_sm;
    int force_pairs;            // tiled kernels: CTA pairs whenever the shape allows
    int stream_max_tile;        // widest token tile the streaming kernels take (0: none, or 64); wider launches go to the tiled kernels
};
cudaError_t launch_ffn_scalar(const FfnArgs& a, const SlotTable& tab, cudaStream_t st, int* n_launch);
cudaError_t launch_ffn_tensor(const FfnArgs& a, const SlotTable& tab, cudaStream_t st, int* n_launch);
// Segments of at most 8 rows (decode batches 1..8): row-split matrix-vector kernels.
cudaError_t launch_ffn_gemv(const FfnArgs& a, const SlotTable& tab, cudaStream_t st, int* n_launch);
// The whole step for batches of at most 8 tokens (top_k at most 8) in one launch (two where a
// cooperative launch is not available): gate + repack indices + gate/up projection, grid barrier,
// down projection + merge (decode_fused.cu).
struct DecodeArgs {
    const float* logits;        // [T, E]
    const uint16_t* x;          // [T, d]
    int T, E, S, k, d, f, renorm;
    const uint8_t* slot_region;
    size_t slot_bytes;
    uint16_t* h;                // [T * (k + S), f] bf16 workspace
    float* y_packed;            // [T * (k + S), d] fp32 workspace
    int* sync;                  // [0..1] 64-bit count of barrier arrivals (only grows), [64 + j] ticket of output columns 32j..32j+31
    void* out;                  // [T, d]
    int out_bf16;
    int32_t* topk_idx;          // index outputs of the step, written by one CTA
    float* topk_w;
    int32_t* counts;
    int32_t* offsets;
    int32_t* perm;
    int32_t* inv_perm;
    int* status;
};
bool decode_fused_supported(int T, int k);
// SAEM_FFN_AUTO takes the one-launch step up to this many tokens (measured: 7-11 % faster than the five-launch
// step at 1..4 tokens on every layer shape tried, level with it or 1-2 % behind at 8)
constexpr int kDecodeFusedAutoTokens = 4;
cudaError_t launch_decode_fused(const DecodeArgs& a, const SlotTable& tab, int n_sm, cudaStream_t st, int* n_launch);
constexpr int kDecodeSyncInts = 64 + 4096;   // d_model <= 16384: at most 512 groups of 32 columns, a ticket per group and token (<= 8)
// One-time per process: resolves the driver entry point for tensor-map encoding and opts the
// kernels into large dynamic shared memory.  Returns cudaSuccess or the failing error.
cudaError_t ffn_tensor_init();
// Exercises the kernels' bounded mbarrier wait: a 1-CTA kernel whose wait can only run out.
cudaError_t launch_bounded_wait_selftest(int* status, unsigned long long limit_ns, cudaStream_t st);

}  // namespace saem

struct saem_ctx {
    saem_config cfg;
    int device;
    int n_sm;
    uint8_t* slot_region;
    size_t slot_bytes;
    uint8_t* ws;
    saem::WorkspaceLayout lay;
    int n_fixed_slots;
    int n_total;             // routed + shared experts per layer
    // residency: fixed slot per (layer, expert), -1 none; temp binding per (layer, expert), -1 none
    int32_t* slot_of;        // [L*E] global slot index
    int32_t* temp_of;        // [L*E] global slot index of a temporary binding
    const uint8_t** host_of; // [L*E] device-visible address of a packed expert in mapped pinned host memory, or null
    int32_t* slot_owner;     // [n_slots] layer*E + expert, -1 empty
    cudaEvent_t* ready_ev;   // [n_slots] recorded on the copy stream after a load
    uint8_t* ev_pending;     // [n_slots] 1: a load was enqueued and no consumer has been ordered after it yet
    uint8_t* ev_recorded;    // [n_slots]
    cudaEvent_t* read_ev;    // [L] recorded on the compute stream after each FFN of that layer
    uint8_t* read_recorded;  // [L]
    int32_t* temp_last_layer;  // [temp_slots] layer whose FFN may still be reading the slot, -1 none
    cudaStream_t* last_stream; // [L] stream of the layer's most recent FFN
    uint8_t* ffn_seen;         // [L] 1 once an FFN of the layer has been enqueued
    int next_temp;
    bool dynamic_residency;  // fewer fixed slots than experts, or temporary slots exist: events are kept
    long long launches;
    int* pinned_status;      // pinned host int for status read-back
};

#endif  // SAEM_INTERNAL_H_
