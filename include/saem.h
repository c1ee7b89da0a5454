/*
 * saem.h -- C ABI of the B200 (sm_100a) MoE expert-step library.
 *
 * One MoE layer step of a stage-aware MoE decoding runtime:
 *
 *   saem_route      top-k gating                         (Background, "Mixture-of-Experts Inference")
 *   saem_repack     expert-aligned token repacking       (Sec. IV-E)
 *   saem_expert_ffn grouped SwiGLU expert FFN over the   (Sec. IV-E "single batched launch per expert",
 *                   repacked segments, weights read from  Sec. IV-C fixed-size expert cache region)
 *                   an HBM expert-slot cache
 *   saem_combine    weighted merge back to token order   (Sec. IV-D, merge of expert outputs)
 *   saem_cache_*    expert-slot table: asynchronous       (Sec. IV-C "Latency-Hiding Prefetch and Overlap",
 *                   host->HBM loads with events, evict     residency map + fixed per-layer slot layout)
 *
 * General conventions
 *   - Plain C.  Streams are passed as `void*` holding a cudaStream_t (NULL = the legacy default stream).
 *   - "dev" pointers are CUDA device pointers, "host" pointers ordinary host memory, "pinned" host
 *     memory registered with CUDA (cudaHostAlloc / cudaHostRegister).  All device buffers are owned
 *     by the caller, must be 16-byte aligned (slot region and workspace: 1024-byte aligned) and
 *     must stay valid until the work enqueued on them has finished.
 *   - The library allocates no device memory.  It owns only host tables and CUDA events.
 *   - bf16 tensors are raw 16-bit patterns; every matrix is row-major; pair id p = t*top_k + j.
 *   - Every function returns a saem_status.  Errors a host can see (bad argument, shape, alignment,
 *     residency) are returned before anything is enqueued.  Conditions only the device can see
 *     (a routed expert that is not resident when no subset was given, an index out of range, a
 *     bounded wait that ran out) set a sticky device status word, read by
 *     saem_last_device_status(); kernels never trap and never wait without a bound.
 *   - The four step calls never synchronise and never read device results on the host.
 *   - A context is not thread-safe: calls on one context must come from one thread at a time.
 *   - Calls on one context must also be ordered on the GPU (one stream, or events between streams):
 *     the hidden activations, the partial tiles and arrival counters of split reductions and the
 *     buffers of saem_moe_step live in the context's workspace, so two saem_expert_ffn or
 *     saem_moe_step calls of one context whose kernels overlap corrupt each other.  Use one context
 *     per concurrent stream.
 */
#ifndef SAEM_H_
#define SAEM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct saem_ctx saem_ctx;   /* opaque: host tables, events, workspace carving */

typedef enum saem_status {
    SAEM_OK = 0,
    SAEM_ERR_INVALID_ARG = 1,
    SAEM_ERR_SHAPE = 2,
    SAEM_ERR_ALIGNMENT = 3,
    SAEM_ERR_WORKSPACE = 4,
    SAEM_ERR_NOT_RESIDENT = 5,
    SAEM_ERR_SLOT_BUSY = 6,
    SAEM_ERR_TIMEOUT = 7,
    SAEM_ERR_CUDA = 8,
    SAEM_ERR_UNSUPPORTED = 9
} saem_status;

enum { SAEM_MAX_EXPERTS = 128 };         /* routed experts per layer */
enum { SAEM_TEMP = -2 };                 /* slot argument of saem_cache_load: take a temporary slot */
enum { SAEM_HOST_MAPPED = -3 };          /* slot reported by saem_cache_query for an expert bound by saem_cache_map_host */
enum { SAEM_OUT_F32 = 0, SAEM_OUT_BF16 = 1 };
enum { SAEM_FFN_AUTO = 0, SAEM_FFN_SCALAR = 1, SAEM_FFN_TENSOR = 2, SAEM_FFN_TENSOR_PAIRS = 3, SAEM_FFN_DECODE_FUSED = 4 };

/*
 * Shape of one context.  d_model and d_ff must be multiples of 128, at most 16384; 1 <= top_k <= n_experts <=
 * SAEM_MAX_EXPERTS; max_tokens * top_k <= 65535.  The slot region holds n_layers * slots_per_layer
 * fixed slots (slot s of layer l is global slot l * slots_per_layer + s) followed by temp_slots
 * temporary slots shared by all layers (Sec. VI ablation: on-demand loads through a reserved
 * temporary slot).  renorm: 1 = softmax over the k selected logits (weights sum to 1), 0 = the
 * selected experts' probabilities under the softmax over all experts.  out_dtype: SAEM_OUT_*.
 * ffn_path: SAEM_FFN_AUTO picks per call -- matrix-vector kernels when no segment can exceed 8
 * rows, the tcgen05 tiled kernels beyond (measured hand-over point; a launch of one or two experts with
 * d_ff >= 4096 keeps the weight-streaming kernels up to 64 rows); SAEM_FFN_TENSOR always uses the
 * tcgen05 kernels: the weight-streaming ones (weights as the MMA's M operand, reductions split across
 * CTAs) up to 64 rows, the tiled ones beyond; SAEM_FFN_SCALAR forces the plain scalar
 * kernels (kept for triage).  The tiled kernels exist in two forms: one CTA per tile, and CTA pairs
 * (tcgen05 cta_group::2: 256 tokens x 512 weight rows per pair of SMs), which AUTO and TENSOR take
 * for long reductions and many rows (d_model >= 4096, d_model % 256 == 0, at least 1536 packed
 * rows in the call); SAEM_FFN_TENSOR_PAIRS is SAEM_FFN_TENSOR with the pair form whenever
 * d_model % 256 == 0 (for tests and measurements).  SAEM_FFN_DECODE_FUSED is SAEM_FFN_AUTO, except that
 * saem_moe_step takes its one-launch form (see there) for every batch it supports (up to 8 tokens, top_k
 * up to 8); AUTO takes it up to 4 tokens, and up to 8 on layers whose experts are at most 20 MB
 * (3 * d_model * d_ff * 2 bytes) and numerous enough (see saem_moe_step).
 * n_shared (0..16, n_experts + n_shared <= SAEM_MAX_EXPERTS): always-on shared experts of the same
 * width d_ff that run INSIDE the layer's grouped launch.  They are experts n_experts ..
 * n_experts + n_shared - 1 of every layer for the cache calls (outside the routed cache-ratio
 * budget: give them slots); saem_repack appends one segment of all T tokens per shared expert
 * after the T*top_k pair rows (counts, offsets get n_shared more entries; x_packed, y_packed
 * hold T*(top_k + n_shared) rows); saem_combine adds their outputs with weight 1.  A shared
 * expert of width m*d_ff is m such experts (the down projection sums over the hidden units).
 * Shared experts of another width use a second context instead (see saem_moe_step).
 */
typedef struct saem_config {
    int32_t d_model;
    int32_t d_ff;
    int32_t n_experts;
    int32_t top_k;
    int32_t max_tokens;
    int32_t n_layers;
    int32_t slots_per_layer;
    int32_t temp_slots;
    int32_t renorm;
    int32_t out_dtype;
    int32_t ffn_path;
    int32_t n_shared;
} saem_config;

/* Library version (major*10000 + minor*100 + patch) and a static string for a status code. */
int saem_version(void);
const char* saem_status_string(int status);

/* Bytes of one packed expert (= one slot): 3 * d_model * d_ff * 2.  0 on an invalid config. */
size_t saem_slot_bytes(const saem_config* cfg);
/* Bytes the slot region must have: (n_layers * slots_per_layer + temp_slots) * saem_slot_bytes. */
size_t saem_slot_region_bytes(const saem_config* cfg);
/* Bytes of device workspace a context needs (hidden activations h[max_tokens*top_k, d_ff] in
 * bf16, split-K partial tiles and counters, the device status word, and the buffers of
 * saem_moe_step).  Allocated once by the caller and reused by every layer (Sec. IV-E). */
size_t saem_workspace_bytes(const saem_config* cfg);

/*
 * Create a context over caller-owned device memory.  Both regions must be 1024-byte aligned and at
 * least as large as the two size queries say.  The workspace is cleared by an asynchronous memset
 * on the legacy default stream followed by a synchronisation; all slots start empty.  The current
 * CUDA device at the time of the call is the context's device.
 * Errors: INVALID_ARG (null), SHAPE (config limits), ALIGNMENT, WORKSPACE (too small), CUDA.
 */
int saem_create(const saem_config* cfg, void* dev_slot_region, size_t slot_region_bytes,
                void* dev_workspace, size_t workspace_bytes, saem_ctx** out);
void saem_destroy(saem_ctx* ctx);

/*
 * One-time, offline: rewrite one expert from the canonical layout (gate[d_ff, d_model],
 * up[d_ff, d_model], down[d_model, d_ff], row-major bf16, host memory) into the slot layout
 * (host memory, saem_slot_bytes): tiles of 128 weight rows x 64 reduction elements, each tile
 * 16 KB with its 16-byte chunks XOR-swizzled by (row mod 8) so that a tile can be bulk-copied
 * into shared memory and fed to the tensor cores as is; gate and up tiles of the same position
 * are adjacent.  A slot's content is opaque to the caller.
 */
int saem_pack_expert_host(const saem_config* cfg, const void* gate, const void* up, const void* down,
                          void* packed_out);

/*
 * Top-k gating.  logits[T, n_experts] fp32 (dev) -> topk_idx[T, top_k] int32, topk_w[T, top_k] fp32
 * (dev).  Slot j of a token holds its j-th largest logit: k rounds of arg-max comparing (value
 * descending, expert id ascending); NaN counts as -inf; +0 == -0.  Weights per config.renorm,
 * computed in fp32 with the row maximum subtracted.  A row whose best logit is -inf gets 1/k
 * everywhere; +inf logits share the weight equally.  Errors: SHAPE if T < 0 or T > max_tokens.
 * T == 0 is a no-op.
 */
int saem_route(saem_ctx* ctx, const float* logits, int T, int32_t* topk_idx, float* topk_w, void* stream);

/*
 * Gating with the router projection fused in: logits[t, e] = <x[t, :], w_router[e, :]> (x[T, d_model]
 * and w_router[n_experts, d_model] bf16, dev, 16-byte aligned; fp32 accumulation), followed by the
 * selection and weights of saem_route in the same kernel.  logits_out[T, n_experts] fp32 (dev) may
 * be NULL.  The paper only says that a routing mechanism selects the top-k experts (Background,
 * "Mixture-of-Experts Inference"); a linear router without bias is the reading taken.  Because the
 * logits are rounded sums, two experts whose exact logits differ by less than the accumulation
 * error (about 1e-5 relative) may swap ranks against an exact evaluation.
 */
int saem_route_fused(saem_ctx* ctx, const void* x, const void* w_router, int T, float* logits_out,
                     int32_t* topk_idx, float* topk_w, void* stream);

/*
 * Expert-aligned token repacking.  topk_idx[T, top_k] (dev) and x[T, d_model] bf16 (dev) ->
 * counts[n_experts], offsets[n_experts + 1] (exclusive scan, offsets[E] = T*top_k), perm[T*top_k]
 * (pair stored at packed row r), inv_perm[T*top_k] (packed row of pair p), x_packed[T*top_k,
 * d_model] bf16 = x[perm[r] / top_k].  Segments are in ascending expert id and keep ascending pair
 * id inside (a stable counting sort), so the permutation is unique.  An index outside
 * [0, n_experts) sets the device status word (INVALID_ARG) and the pair is dropped from every output:
 * its inv_perm entry is -1, the segments hold the valid pairs only, and the perm entries behind the
 * last segment are -1.
 * With config.n_shared = S > 0 the outputs grow: counts[n_experts + S], offsets[n_experts + S + 1],
 * x_packed[T*(top_k + S), d_model]; shared expert s owns rows [T*top_k + s*T, T*top_k + (s+1)*T),
 * a copy of x, and offsets[n_experts] is T*top_k.
 */
int saem_repack(saem_ctx* ctx, const int32_t* topk_idx, const void* x, int T, int32_t* counts,
                int32_t* offsets, int32_t* perm, int32_t* inv_perm, void* x_packed, void* stream);

/*
 * Grouped SwiGLU expert FFN.  For every expert e with rows r in [offsets[e], offsets[e+1]) of
 * x_packed (dev, bf16): y_packed[r] = Wd_e * ( silu(Wg_e * x_r) .* (Wu_e * x_r) ), fp32
 * accumulation, hidden activations rounded to bf16 in the context's workspace, y_packed[max_rows,
 * d_model] fp32 (dev).  Weights come from the slots that `layer`'s residency map (or a temporary
 * slot) gives.  offsets (dev, n_experts + n_shared + 1 entries) is read on the device only;
 * max_rows bounds its last entry and must not exceed max_tokens * (top_k + n_shared).  offsets may be NULL only when n_experts == 1: the single
 * segment is then rows [0, max_rows) (used for always-on shared experts, whose input is x itself).
 *   expert_subset (host, may be NULL): run only these experts (rows of the others are left
 *   untouched).  With a subset, an expert that has no slot returns NOT_RESIDENT before any
 *   enqueue.  Without one, experts without a slot are skipped on the device; if such an expert has
 *   rows, the device status word becomes NOT_RESIDENT and its rows are left untouched.
 * If a needed slot's load is still in flight on another stream, `stream` is made to wait for its
 * completion event first.
 */
int saem_expert_ffn(saem_ctx* ctx, int layer, const void* x_packed, const int32_t* offsets, int max_rows,
                    const int32_t* expert_subset, int n_subset, float* y_packed, void* stream);

/*
 * Weighted merge: out[t] = sum_{j = 0..top_k-1, in that order} topk_w[t, j] *
 * y_packed[inv_perm[t*top_k + j]] (+ the rows y_packed[T*top_k + s*T + t] of the config.n_shared
 * in-layer shared experts, weight 1) (+ shared_y[t] if not NULL, fp32 [T, d_model], added last).
 * Gather-based, no atomics: two runs give identical bits.  out[T, d_model] fp32 or bf16 per
 * config.out_dtype.
 */
int saem_combine(saem_ctx* ctx, const float* y_packed, const int32_t* inv_perm, const float* topk_w, int T,
                 const float* shared_y, void* out, void* stream);

/*
 * The whole layer step on device buffers: route -> repack -> expert FFN -> [shared expert FFN via
 * shared_ctx over x itself] -> combine, enqueued on `stream`, intermediates in ctx's workspace.
 * shared_ctx (may be NULL) is a context with n_experts = top_k = 1 whose layer `layer` slot 0
 * holds an always-on shared expert whose width is not a multiple of d_ff (otherwise use
 * config.n_shared and pass NULL).
 * logits[T, E] fp32, x[T, d] bf16, out[T, d] (all dev).
 * Smallest decode batches (ffn_path DECODE_FUSED: T <= 8; AUTO: T <= 4, and T <= 8 when an expert is at most 20 MB and
 * (min(n_experts, T * top_k) + n_shared) * d_model / 32 >= 8 * the device's SM count; top_k <= 8; no shared_ctx): the whole step runs as ONE
 * kernel launch -- gate, repack indices and gate/up projection, a grid-wide barrier, down projection and
 * merge -- launched cooperatively (two launches where the device refuses that).  topk_idx, topk_w, counts,
 * offsets, perm, inv_perm, h and y_packed are still left in the workspace; x_packed is not produced.  A
 * routed expert without a slot sets NOT_RESIDENT in the device status word and contributes nothing.  The
 * first such call on a device should come before any stream capture (it probes what the driver accepts).
 */
int saem_moe_step(saem_ctx* ctx, saem_ctx* shared_ctx, int layer, const float* logits, const void* x, int T,
                  void* out, void* stream);

/*
 * The same step from HOST buffers (pinned memory recommended): copies logits and x to the device,
 * runs saem_moe_step, copies out back and synchronises `stream`.  Expert weights stay in the HBM
 * slots.  logits_host[T, E] fp32, x_host[T, d] bf16, out_host[T, d] per out_dtype.
 */
int saem_moe_step_host(saem_ctx* ctx, saem_ctx* shared_ctx, int layer, const float* logits_host,
                       const void* x_host, int T, void* out_host, void* stream);

/*
 * saem_moe_step_host without the final synchronisation: the two copies in, the kernels and the copy out
 * are enqueued on `stream` and the call returns.  out_host is valid, and logits_host / x_host may be
 * reused, once `stream` has passed that point (an event or a synchronisation of the caller's).  Steps
 * enqueued one after the other run in order; the host's launch work of one overlaps the device's work on
 * the one before.  Pinned host memory is required for the copies to be asynchronous.
 */
int saem_moe_step_host_async(saem_ctx* ctx, saem_ctx* shared_ctx, int layer, const float* logits_host,
                       const void* x_host, int T, void* out_host, void* stream);

/* Device pointers of the intermediates of the last saem_moe_step (inside the workspace), for
 * inspection by tests: 0 topk_idx, 1 topk_w, 2 counts, 3 offsets, 4 perm, 5 inv_perm, 6 x_packed,
 * 7 y_packed, 8 shared_y, 9 h (hidden activations), 10 the 656 int32 counters through which the FFN
 * kernels' CTAs meet (arrivals at items whose reduction is split across CTAs; per expert, the hidden
 * activations completed by the gate/up launch and seen by the down launch, the down launch's item
 * counter): all zero between calls.  NULL for an unknown id.  The one-launch form of
 * the step (see saem_moe_step) does not produce x_packed. */
void* saem_step_buffer(saem_ctx* ctx, int which);

/*
 * Expert cache.  saem_cache_load copies one packed expert (pinned host, saem_slot_bytes) into a
 * slot with cudaMemcpyAsync on copy_stream and records a completion event; the residency map
 * changes at once on the host.  slot: 0..slots_per_layer-1 of `layer`, which must be empty
 * (SLOT_BUSY otherwise: evict first), or SAEM_TEMP: take the next temporary slot round-robin,
 * dropping whatever it held; a temporary binding serves saem_expert_ffn but is not part of the
 * residency map.  The copy is ordered after the last FFN that read the slot.  Loading an expert
 * that already has a fixed slot returns INVALID_ARG.
 * saem_cache_evict frees the expert's slot (fixed or temporary) on the host table; NOT_RESIDENT
 * if it has none.  No device work is enqueued.
 * saem_cache_query: *slot = global slot index, -1 if none; *ready = 1 once the load has completed.
 * saem_cache_wait: makes consumer_stream wait for the expert's load event (NOT_RESIDENT if none).
 */
int saem_cache_load(saem_ctx* ctx, int layer, int expert, int slot, const void* pinned_packed_expert,
                    void* copy_stream);
int saem_cache_evict(saem_ctx* ctx, int layer, int expert);
/*
 * Binds an expert that has no slot to a packed expert in MAPPED PINNED HOST memory (cudaHostAlloc /
 * cudaHostRegister; saem_slot_bytes, 16-byte aligned), to be read in place over the host link by the
 * matrix-vector kernels of saem_expert_ffn (calls whose segments have at most 8 rows, ffn_path AUTO): the
 * GPU-side analogue of executing a missed expert where its weights are (Sec. IV-D in-situ execution; the
 * Sec. VI ablation's on-demand transfer through a temporary slot is the other way).  No copy, no slot, no
 * event: the memory must stay valid and unchanged until the FFNs that use it have finished.  Every other
 * kernel treats such an expert as absent, and saem_moe_step takes its five-launch form for a layer that
 * has one.  At most 8 host-mapped experts per FFN call (UNSUPPORTED beyond).  saem_cache_evict removes
 * the binding; a slot loaded later takes precedence.  Errors: INVALID_ARG (has a slot; not mapped pinned
 * memory), ALIGNMENT.
 */
int saem_cache_map_host(saem_ctx* ctx, int layer, int expert, const void* pinned_packed_expert);
int saem_cache_query(saem_ctx* ctx, int layer, int expert, int* slot, int* ready);
int saem_cache_wait(saem_ctx* ctx, int layer, int expert, void* consumer_stream);

/*
 * (No counterpart in the paper: an addition for callers that cannot allocate device memory.)
 *
 * saem_expert_ffn_static is saem_expert_ffn for code that must not, or cannot, call cudaMalloc: a
 * plugin inside an application that owns the whole memory pool, a latency-critical loop where an
 * allocation may block, a process whose pool is already exhausted.  It needs no saem_ctx and no
 * workspace: the hidden activations h[max_rows, d_ff] (bf16) live in a fixed array inside the
 * library, SAEM_STATIC_SCRATCH_ELEMS elements (2 MiB) that every GPU which loads the library
 * holds until the process exits.  The function calls no allocating routine of any kind.
 *
 *   x_packed[max_rows, d_model] bf16, offsets[n_experts + 1] int32, y_packed[max_rows, d_model] fp32:
 *   device, caller-owned, 16-byte aligned, with the meaning they have in saem_expert_ffn.
 *   packed_experts: device, n_experts packed experts (saem_pack_expert_host layout) back to back,
 *   expert e at byte offset e * 3 * d_model * d_ff * 2 -- for instance the slots of one layer of a
 *   fully resident slot region.  Plain scalar kernels; results agree with saem_expert_ffn within
 *   its tolerance.
 *
 * Limits and errors: max_rows * d_ff > SAEM_STATIC_SCRATCH_ELEMS returns SAEM_ERR_WORKSPACE and
 * enqueues nothing; shapes and alignment as for saem_expert_ffn (SAEM_ERR_SHAPE, _ALIGNMENT,
 * _INVALID_ARG).  The first call on a device looks the array's device address up (a short
 * host-side set-up with that device current); make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps the previous call's contents: every
 * element a call reads it has written itself first, so nothing needs clearing, but two calls
 * whose kernels may overlap on the GPU (different streams, no ordering between them) race on it
 * -- order them on one stream or with events.
 */
enum { SAEM_STATIC_SCRATCH_ELEMS = 1 << 20 };
int saem_expert_ffn_static(const void* x_packed, const int32_t* offsets, int n_experts, int max_rows,
                           int d_model, int d_ff, const void* packed_experts, float* y_packed, void* stream);

/* Reads and clears the sticky device status word (synchronises the device).  When the word is
 * SAEM_ERR_TIMEOUT the arrival counters of split reductions are cleared as well (a CTA that gave up
 * its wait did not arrive), so that the context can be used again; the outputs of the call that
 * timed out are undefined. */
int saem_last_device_status(saem_ctx* ctx, int* code);

/* Number of kernels this library has launched through `ctx` since creation (host counter). */
long long saem_launch_count(saem_ctx* ctx);

/*
 * Self-test of the failure path of the kernels' device-side waits (no counterpart in the paper).
 * Every wait inside the FFN kernels is bounded; this enqueues a one-CTA kernel that waits, with the
 * same helper, on a barrier nothing will ever complete, with a limit of limit_us microseconds
 * (1..1 000 000).  The kernel must return by itself and leave SAEM_ERR_TIMEOUT in the device status
 * word (read it with saem_last_device_status); the context stays usable.  Nothing traps or hangs.
 */
int saem_selftest_bounded_wait(saem_ctx* ctx, int limit_us, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SAEM_H_ */
