/*
 * expertweave.h - C ABI of the B200 (sm_100a) adapter-aware MoE layer forward of ExpertWeave.
 *
 * The library serves many ESFT adapters over one shared MoE base model.  All expert weights of a
 * layer live in ONE slot-indexed pool per stacked linear (the "virtual weight tensor" of Section 4.1:
 * first dimension M + N*E_max, base experts first, then E_max reserved slots per adapter), whose
 * virtual address range is contiguous while physical pages are mapped only under live experts
 * (Section 4.2).  A forward call takes a mixed batch of tokens, each tagged with an adapter id
 * (-1 = base model, Section 4.3), routes them with the base router, rewrites the routed expert ids
 * through the per-layer ESFT expert map Pi (batched rerouting, Section 4.1/4.3), and runs the usual
 * dispatch -> grouped expert FFN -> weighted combine (Section 2.1) over the pool.
 *
 * Conventions
 *   - Every function returns ew_status_t.  Nothing throws, aborts or traps the device.
 *   - "host" / "device" in a parameter comment says where the pointer must live.
 *   - bf16 tensors are passed as void* to raw 16-bit patterns, row-major, innermost dimension
 *     contiguous.  int32 and float are the C types.
 *   - One pool may be used by one host thread at a time.  Forward calls on one pool share one
 *     workspace; the pool orders them itself (a call on another stream than the previous one first
 *     makes its stream wait for that forward, on the device).
 *   - Every entry point makes the pool's device current while it runs and restores the caller's
 *     current device before it returns.
 *   - H must be a multiple of 64 and I a multiple of 8; M <= 256; top_k <= 32 and <= M.
 */
#ifndef EXPERTWEAVE_H_
#define EXPERTWEAVE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ew_pool ew_pool_t; /* opaque; created and destroyed by the library */

typedef enum {
    EW_OK = 0,
    EW_ERR_INVALID_ARG = 1,      /* null pointer, size out of range, bad configuration             */
    EW_ERR_OOM = 2,              /* device memory or the page budget is exhausted                  */
    EW_ERR_SLOT_IN_USE = 3,      /* ew_load_adapter on an adapter id that is already loaded        */
    EW_ERR_NOT_LOADED = 4,       /* ew_unload_adapter on an id that is not loaded; forward before ew_load_base */
    EW_ERR_TOO_MANY_EXPERTS = 5, /* an adapter tunes more than E_max experts in some layer         */
    EW_ERR_CUDA = 6,             /* a CUDA call failed; ew_last_error_string() has the detail      */
    EW_ERR_TIMEOUT = 7,          /* a bounded device-side wait expired (reported by ew_last_device_error) */
    EW_ERR_BAD_ADAPTER_ID_IN_BATCH = 8, /* some token carried an id outside [-1,N) or of an unloaded adapter */
    EW_ERR_NO_DEVICE = 9         /* the call needs a GPU and the pool is an accounting-only pool   */
} ew_status_t;

/* Pool configuration (Section 3.1: N = adapters servable in one batch, E_max = slots per adapter). */
typedef struct {
    int32_t device;        /* CUDA device ordinal; -1 = accounting-only pool: the page bookkeeping of
                              Section 4.2 runs, no device memory is touched, forward calls fail with
                              EW_ERR_NO_DEVICE (for capacity planning and host-side tests)          */
    int32_t num_layers;    /* L  MoE layers held by this pool                                      */
    int32_t hidden;        /* H                                                                    */
    int32_t inter;         /* I  expert intermediate size (SwiGLU: gate and up are [I,H], down [H,I]) */
    int32_t num_experts;   /* M  routed experts of the base model                                  */
    int32_t num_shared;    /* S  shared experts (always active, weight 1, never rerouted)          */
    int32_t top_k;         /* k                                                                    */
    int32_t max_adapters;  /* N                                                                    */
    int32_t e_max;         /* E_max                                                                */
    int32_t max_tokens;    /* largest n_tokens a forward call may pass (sizes the workspace)       */
    int32_t renormalize;   /* 0: combine weights are the selected softmax probabilities; 1: divided by their sum */
    float routed_scale;    /* multiplies the k combine weights (1.0 for the DeepSeek-V2-Lite shape) */
    int32_t pool_mode;     /* 0: pages mapped on demand under live experts (Section 4.2)
                              1: "padding" baseline of Section 3.1: the whole tensor is backed at creation */
    int32_t ep_size;       /* expert parallelism (Section 5.1: "EP for MoE layers"): number of ranks the experts are
                              partitioned over; 0 or 1 = none.  See ew_moe_forward_partial.                  */
    uint64_t page_bytes;   /* physical page size; 0 = the driver's minimum granularity (2 MiB on B200);
                              otherwise a multiple of it                                            */
    uint64_t prealloc_pages; /* pages created up front and kept in the pool's free list            */
    uint64_t max_pages;    /* 0 = unlimited; else creating more pages than this fails with EW_ERR_OOM */
    int32_t ep_rank;       /* this pool's rank in [0, ep_size)                                              */
    int32_t reserved0;
} ew_config_t;

/* Memory accounting (Section 4.2; Section 3.1's F_mem is padding_bytes / live_expert_bytes). */
typedef struct {
    uint64_t page_bytes;
    uint64_t va_reserved_bytes;   /* sum of the virtual ranges of all virtual weight tensors        */
    uint64_t pages_mapped;        /* pages currently mapped under some live expert                  */
    uint64_t pages_free;          /* created, unmapped, waiting in the pool's free list             */
    uint64_t pages_created_total; /* pages ever created (reuse keeps this flat under churn)         */
    uint64_t physical_bytes;      /* (pages_mapped + pages_free) * page_bytes                       */
    uint64_t live_expert_bytes;   /* bytes of the experts that are loaded (base + adapters + shared) */
    uint64_t padding_bytes;       /* what a fully backed [M + N*E_max (+S)] tensor would take       */
    uint64_t live_experts;        /* routed base + adapter experts currently loaded, over all layers */
    uint64_t adapters_loaded;
    uint64_t workspace_bytes;
    uint64_t last_forward_kernels; /* kernels the most recent forward launched: 4 (decode-sized batch: router, GEMM-1,
                                      GEMM-2, combine; the GEMM kernels derive their work items themselves), 5 (the
                                      same with the planning kernel) or 7 (prefill-sized batch: planning kernel and
                                      two kernels per GEMM); 0 before the first forward                        */
} ew_stats_t;

/* Create a pool: reserves, per layer and per stacked linear (gate|up fused as one tensor, down as
 * another), a contiguous virtual range for M + N*E_max slots (+S trailing slots that hold the shared
 * experts and are never addressed by the expert map); no physical page is mapped under it at this
 * point (Section 4.2: reservation and mapping are separate steps).  Allocates the
 * expert maps (identity rows), router storage and the forward workspace for cfg->max_tokens.
 * Errors: EW_ERR_INVALID_ARG (bad sizes), EW_ERR_OOM, EW_ERR_CUDA.  *out is set only on EW_OK. */
ew_status_t ew_pool_create(const ew_config_t *cfg, ew_pool_t **out);

/* Unmaps and releases everything.  Blocks until forwards issued earlier have finished. */
ew_status_t ew_pool_destroy(ew_pool_t *pool);

/* Load the base model's weights of one layer: the range [0, M) of the pool plus the shared experts
 * (Section 4.2 treats the base model as one more range of consecutive experts, loaded once at start-up
 * through the same map-and-copy path that adapters take later).  All pointers are HOST bf16:
 *   router_w [M,H]; w_gate, w_up [M,I,H]; w_down [M,H,I]; sh_gate, sh_up [S,I,H]; sh_down [S,H,I]
 * (the sh_* pointers may be null when S = 0).  Data is copied before the call returns; the caller
 * keeps ownership.  Calling it again for the same layer overwrites the weights in place. */
ew_status_t ew_load_base(ew_pool_t *pool, int32_t layer, const void *router_w, const void *w_gate,
                         const void *w_up, const void *w_down, const void *sh_gate, const void *sh_up,
                         const void *sh_down);

/* Load ESFT adapter `adapter_id` in [0,N) (Sections 4.1-4.2).
 *   counts      host int32 [L]: e_i^(l), experts the adapter re-tunes in layer l (0 allowed)
 *   expert_ids  host int32 [sum counts]: per layer, strictly ascending base expert ids in [0,M);
 *               the r-th id of a layer gets delta = r, i.e. slot M + adapter_id*E_max + r
 *   w_gate,w_up bf16 [sum counts, I, H];  w_down bf16 [sum counts, H, I], same order.  The weight
 *               pointers may be host memory (page-locked memory copies at the host link's speed) or
 *               device memory (an adapter kept resident outside the pool): the copy follows unified
 *               addressing.  The same holds for the weight pointers of ew_load_base.
 * For each layer the byte range of slots [Delta_i, Delta_i + e) is backed by pages taken from the
 * pool's free list (or created); a page shared with a neighbouring adapter is mapped once and
 * reference-counted (sub-page allocation).  Weights are copied, then row adapter_id of every layer's
 * expert map is published.  All-or-nothing: on any error every page mapped by this call is unmapped
 * again and the maps are untouched.
 * Errors: EW_ERR_INVALID_ARG, EW_ERR_SLOT_IN_USE, EW_ERR_TOO_MANY_EXPERTS, EW_ERR_OOM, EW_ERR_CUDA. */
ew_status_t ew_load_adapter(ew_pool_t *pool, int32_t adapter_id, const int32_t *counts,
                            const int32_t *expert_ids, const void *w_gate, const void *w_up,
                            const void *w_down);

/* Evict an adapter: the call waits for every forward issued before it (they complete as issued, with
 * the adapter still in place), then its expert-map rows return to identity and pages whose reference
 * count drops to zero are unmapped and returned to the pool's free list for reuse (Section 4.2).
 * Errors: EW_ERR_INVALID_ARG, EW_ERR_NOT_LOADED. */
ew_status_t ew_unload_adapter(ew_pool_t *pool, int32_t adapter_id);

/* Release the free list's pages back to the driver (Section 4.2: pages that are not reused are reclaimed). */
ew_status_t ew_pool_trim(ew_pool_t *pool);

/* The adapter-aware MoE layer forward (Sections 2.1, 4.1, 4.3), asynchronous on `cuda_stream`:
 *   softmax router + top-k over the M base experts (ties to the lower index)
 *   -> batched rerouting  slot = adapter_ids[t] < 0 ? id : Pi[layer][adapter_ids[t]][id]
 *   -> per-slot token counts, permutation into slot-contiguous rows (as index tables: no copy of x is made)
 *   -> grouped SwiGLU FFN over the live slots and the shared experts (fp32 accumulation)
 *   -> out[t] = sum_j w[t,j] * FFN_slot(t,j)(x[t]) + sum_shared FFN(x[t]), rounded once to bf16.
 *   x            device bf16 [n_tokens, H], 16-byte aligned
 *   adapter_ids  device int32 [n_tokens]; values outside [-1,N) or naming an adapter that is not
 *                loaded are treated as -1 and raise EW_ERR_BAD_ADAPTER_ID_IN_BATCH in the device
 *                error word (ew_last_device_error)
 *   out          device bf16 [n_tokens, H]
 *   cuda_stream  a cudaStream_t (null = the legacy default stream)
 * No host synchronisation; token counts never leave the device.  n_tokens = 0 is a no-op.
 * A pool owns one workspace, so its forwards run one after another: a call on another stream than the
 * previous one first makes its stream wait for that forward (device-side; the host does not block).
 * Host calls on one pool are not thread-safe: serialise them, or give each thread its own pool.
 * The call may be captured into a CUDA graph after one uncaptured warm-up call with the same n_tokens;
 * ew_unload_adapter and ew_load_base wait for forwards issued directly, not for replays of such a graph:
 * synchronise those yourself before evicting.
 * Errors: EW_ERR_INVALID_ARG (null, layer out of range, n_tokens > max_tokens), EW_ERR_NOT_LOADED,
 * EW_ERR_NO_DEVICE, EW_ERR_CUDA (launch failure). */
ew_status_t ew_moe_forward(ew_pool_t *pool, int32_t layer, const void *x, const int32_t *adapter_ids,
                           int32_t n_tokens, void *out, void *cuda_stream);

/* Same forward, also copying intermediate results to optional DEVICE buffers (null = skip):
 *   topk_ids [n_tokens,k] int32 base expert ids, in (probability descending, index ascending) order
 *   topk_w   [n_tokens,k] float combine weights, same order
 *   slot_ids [n_tokens,k] int32 after rerouting
 *   counts   [M + N*E_max] int32 tokens per slot
 *   inv      [n_tokens,k] int32 row of pair (t,j) in the slot-contiguous order
 *   offsets  [M + N*E_max + 1] int32 exclusive scan of counts                                      */
ew_status_t ew_moe_forward_debug(ew_pool_t *pool, int32_t layer, const void *x, const int32_t *adapter_ids,
                                 int32_t n_tokens, void *out, void *cuda_stream, int32_t *topk_ids,
                                 float *topk_w, int32_t *slot_ids, int32_t *counts, int32_t *inv,
                                 int32_t *offsets);

/* Expert parallelism (Section 5.1: tensor parallelism for self-attention, expert parallelism for the MoE layers;
 * Section 5.2 runs TP = EP = 8 and 2).  The paper does not say how tokens reach experts on other devices; under tensor-
 * parallel attention every rank holds the hidden states of all tokens, so this build needs no token exchange:
 * a pool created with ep_size = R > 1 and ep_rank = r holds the base experts
 *     [r * ceil(M/R), min(M, (r+1) * ceil(M/R)))
 * with every adapter's re-tuned copies of them (a pair's device is decided by its base expert id alone, so a
 * rerouted pair never leaves the rank of its base expert), and the shared experts [r * ceil(S/R), ...) likewise;
 * ew_load_base / ew_load_adapter take the same full arguments on every rank and map and copy only that share, the
 * other slots of the virtual tensors stay unbacked (Section 4.2's on-demand pages), and the expert map is the same
 * on all ranks.  ew_moe_forward_partial runs the layer on ALL n_tokens tokens: the router (redundantly on every
 * rank), then the grouped FFN over the pairs whose expert lives here, and writes the rank's partial sums
 *     partial[t] = sum over local pairs j of w[t,j] * FFN_slot(t,j)(x[t]) + sum over local shared experts FFN(x[t])
 * unrounded: DEVICE fp32 [n_tokens, H], 16-byte aligned.  The caller adds the R partials (an all-reduce; the Python
 * package does it with torch.distributed) and calls ew_ep_finish on the sum for the layer's single rounding to bf16
 * (summed: DEVICE fp32 [n_tokens, H]; out: DEVICE bf16 [n_tokens, H]; they may not overlap).
 * On such a pool ew_moe_forward, ew_moe_forward_debug and ew_moe_forward_host fail with EW_ERR_INVALID_ARG.
 * With ep_size <= 1 ew_moe_forward_partial is the whole layer, unrounded.  Other arguments, ordering and errors as
 * for ew_moe_forward. */
ew_status_t ew_moe_forward_partial(ew_pool_t *pool, int32_t layer, const void *x, const int32_t *adapter_ids,
                                   int32_t n_tokens, float *partial, void *cuda_stream);
ew_status_t ew_ep_finish(ew_pool_t *pool, const float *summed, int32_t n_tokens, void *out, void *cuda_stream);

/* The same exchange done by the kernel that produces the data (Section 5.1's deployment; the fused form of the step
 * above).  ew_moe_forward_scatter runs the partial forward and its last kernel stores the rank's partial sums straight
 * into every rank's gather buffer: gather_bufs is a DEVICE array of ep_size pointers, gather_bufs[r'] = rank r''s
 * buffer, fp32 [ep_size, n_tokens, H], 16-byte aligned, of which this call fills block ep_rank.  The buffers of the
 * other ranks must be device memory this GPU can store to (peer access, an imported allocation, symmetric memory);
 * plain stores only, nothing is loaded from a peer.  When the scatter calls of ALL ranks for this step have completed
 * (a barrier between the ranks that the caller provides, ordered on the stream), ew_ep_finish_gathered adds the
 * ep_size blocks of this rank's own buffer in rank order and rounds once: the same bits on every rank and in every
 * run, whatever the interconnect did.  It serves an all-gather of the ew_moe_forward_partial results just as well.
 * gathered: DEVICE fp32 [ep_size, n_tokens, H]; out: DEVICE bf16 [n_tokens, H].  Errors as for ew_moe_forward. */
ew_status_t ew_moe_forward_scatter(ew_pool_t *pool, int32_t layer, const void *x, const int32_t *adapter_ids,
                                   int32_t n_tokens, float *const *gather_bufs, void *cuda_stream);
ew_status_t ew_ep_finish_gathered(ew_pool_t *pool, const float *gathered, int32_t n_tokens, void *out, void *cuda_stream);

/* Same forward with HOST buffers, pipelined across calls: x and adapter_ids are uploaded to device staging
 * owned by the pool, the forward runs on them and the result is downloaded to out_host.  Upload, kernels and
 * download run on three streams of the pool with double-buffered staging, so that, with page-locked host
 * buffers, the upload of the next call and the download of the previous one overlap the kernels of the current
 * one (pageable buffers make the copies synchronous).  `cuda_stream` is made to wait for the download: the
 * caller synchronises that stream (or an event recorded on it) before reading out_host or reusing x_host.
 * The host buffers must be ready when the call is made (work queued earlier on `cuda_stream` is not waited for).
 * x_host, out_host: host bf16 [n_tokens, H]; adapter_ids_host: host int32 [n_tokens]. */
ew_status_t ew_moe_forward_host(ew_pool_t *pool, int32_t layer, const void *x_host,
                                const int32_t *adapter_ids_host, int32_t n_tokens, void *out_host,
                                void *cuda_stream);

/* Per-kernel timing.  While enabled, every forward records CUDA events on its stream around its
 * kernels (no host synchronisation).  ew_profile_read waits for the recorded forwards, adds up the
 * elapsed milliseconds per kernel into ms[5] = {route (incl. zeroing the counts), permute+plan,
 * GEMM-1+SwiGLU, GEMM-2, combine}, writes how many forwards were measured, and clears the record.
 * A decode-sized forward has no planning kernel (ew_stats_t.last_forward_kernels = 4): its ms[1] is the
 * cost of the two event records alone, and the GEMM kernels' times include the derivation of their work items.
 * At most 4096 forwards are recorded between two reads. */
ew_status_t ew_profile_enable(ew_pool_t *pool, int32_t on);
ew_status_t ew_profile_read(ew_pool_t *pool, double *ms, int32_t *n_forwards);

/* The batched rerouting operator on its own (Section 4.3): given the router's top-k ids, write
 * slot_ids[t,j] = adapter_ids[t] < 0 ? topk_ids[t,j] : Pi[layer][adapter_ids[t]][topk_ids[t,j]] and,
 * if counts is not null, the number of pairs per slot (counts is overwritten, not accumulated).
 * All pointers DEVICE: topk_ids, slot_ids [n_tokens,k] int32 (may alias), adapter_ids [n_tokens],
 * counts [M + N*E_max].  n_tokens is not limited by max_tokens.  Ids outside [0,M) are passed
 * through unchanged and flagged in the device error word; adapter ids outside [-1,N) or of an adapter that
 * is not loaded behave as -1 and are flagged.  With 16-byte-aligned buffers a call is one kernel launch
 * (the kernel zeroes the counters itself, through two handshake words in the pool's workspace); calls on
 * different streams are therefore ordered by the pool like forwards.  Asynchronous on cuda_stream. */
ew_status_t ew_reroute(ew_pool_t *pool, int32_t layer, const int32_t *topk_ids, const int32_t *adapter_ids,
                       int32_t n_tokens, int32_t *slot_ids, int32_t *counts, void *cuda_stream);

/* Ablation of the operator above (Section 5.3, Figure 7, the "SingleOp" variant): the same rewrite as one kernel per
 * elementary tensor operation - broadcast the adapter ids to [n_tokens,k], compute offsets into the flattened map,
 * gather - with both intermediates materialised, plus a histogram kernel when counts is not null.  Results are
 * identical to ew_reroute's; only the cost differs.  scratch: DEVICE int32 [2 * n_tokens * k], caller-owned.
 * All other arguments as for ew_reroute (slot_ids may alias topk_ids). */
ew_status_t ew_reroute_unfused(ew_pool_t *pool, int32_t layer, const int32_t *topk_ids, const int32_t *adapter_ids,
                               int32_t n_tokens, int32_t *slot_ids, int32_t *counts, int32_t *scratch,
                               void *cuda_stream);

/* Gate function and rerouting from given logits, in one kernel (Sections 2.1 and 4.3; the operator of
 * ew_reroute fused with the softmax + top-k that precedes it): for every token softmax over its M logits, the
 * top_k largest probabilities (ties to the lower index) as topk_ids / topk_w (renormalised and scaled as the
 * pool's config says), slot_ids[t,j] = adapter_ids[t] < 0 ? id : Pi[layer][adapter_ids[t]][id], and the
 * number of pairs per slot in counts (overwritten).  All pointers DEVICE: logits fp32 [n_tokens, M],
 * row-major, 16-byte aligned; adapter_ids [n_tokens]; topk_ids, slot_ids [n_tokens, top_k] int32; topk_w
 * [n_tokens, top_k] fp32; counts [M + N*E_max] int32.  n_tokens is not limited by max_tokens; M must be a
 * multiple of 4.  Bad adapter ids behave as -1 and raise the device error word.  Asynchronous on cuda_stream.
 * Errors: EW_ERR_INVALID_ARG, EW_ERR_NOT_LOADED, EW_ERR_NO_DEVICE, EW_ERR_CUDA. */
ew_status_t ew_route_logits(ew_pool_t *pool, int32_t layer, const float *logits, const int32_t *adapter_ids,
                            int32_t n_tokens, int32_t *topk_ids, float *topk_w, int32_t *slot_ids, int32_t *counts,
                            void *cuda_stream);

/* Routing without any allocation (the paper has no counterpart: this entry point exists for callers
 * of this library that cannot allocate device memory when they need a routing decision - an engine
 * whose KV cache has taken all free HBM, code running where the CUDA allocator must not be entered,
 * or a second batch to route while a forward on this pool, which owns a single workspace, is still in
 * flight).  It runs the same fused router kernel as ew_moe_forward (logits, softmax, top-k, batched
 * rerouting, per-slot counts) for x [n_tokens,H] and writes into buffers the CALLER provides:
 *   topk_ids, slot_ids [n_tokens,k] int32; topk_w [n_tokens,k] float; counts [M + N*E_max] int32
 *   (overwritten); device_status (optional, device int32): 0, or bits as in ew_last_device_error's
 *   word (bit 0 bad adapter id, bit 1 expired wait); written for n_tokens = 0 as well.
 * All pointers DEVICE.  The kernel's scratch lives in one fixed array inside the library (about 256 KiB
 * per GPU, held from the moment the library's code is loaded on that GPU until the process exits); therefore
 *   - n_tokens * top_k must not exceed 65536, otherwise EW_ERR_INVALID_ARG and nothing is launched;
 *   - the call performs no cudaMalloc / cudaFree and enters no allocating library routine.  Everything
 *     that may load code or reserve memory on first use - the array's device address
 *     (cudaGetSymbolAddress), the router kernels' attributes - is resolved by ew_pool_create, once per
 *     device, so the first routing call already finds it done;
 *   - all calls share the array, which still holds the previous call's contents (the words that must
 *     start at zero are cleared on the stream at the start of each call): two calls that overlap on
 *     the GPU (different streams, no ordering) race on it.  Order them.
 * The pool's weights and expert maps are read, its workspace is not touched.  ew_unload_adapter and
 * ew_load_base wait for the latest call of this entry point (an event created with the pool is recorded
 * after it) as they wait for forwards; calls made during stream capture are not tracked.
 * Errors: EW_ERR_INVALID_ARG, EW_ERR_NOT_LOADED, EW_ERR_NO_DEVICE, EW_ERR_CUDA. */
ew_status_t ew_route_noalloc(ew_pool_t *pool, int32_t layer, const void *x, const int32_t *adapter_ids,
                             int32_t n_tokens, int32_t *topk_ids, float *topk_w, int32_t *slot_ids,
                             int32_t *counts, int32_t *device_status, void *cuda_stream);

/* Copy one layer's expert map Pi^(l) [N,M] to HOST memory (the host-side master copy). */
ew_status_t ew_get_expert_map(ew_pool_t *pool, int32_t layer, int32_t *host_out);

ew_status_t ew_pool_stats(ew_pool_t *pool, ew_stats_t *out);

/* Read and clear the device error word (synchronises with the pool's last forward).  *code receives
 * an ew_status_t: EW_OK, EW_ERR_BAD_ADAPTER_ID_IN_BATCH, EW_ERR_TIMEOUT or EW_ERR_INVALID_ARG. */
ew_status_t ew_last_device_error(ew_pool_t *pool, int32_t *code);

/* Self-test of the bounded device-side waits (the tensor-core kernels wait on shared-memory barriers with a
 * time limit instead of spinning forever).  Launches a one-CTA kernel that waits, with a limit of about a
 * millisecond, on a barrier nothing arrives at; synchronises the stream; returns EW_OK if the wait expired and
 * the kernel ran to its end.  Afterwards ew_last_device_error reports EW_ERR_TIMEOUT once.  No memory is
 * touched outside the pool's error word. */
ew_status_t ew_selftest_bounded_wait(ew_pool_t *pool, void *cuda_stream);

/* Device address of slot `slot` of a layer's fused gate|up tensor (which = 0) or down tensor
 * (which = 1); slots M + N*E_max .. +S-1 are the shared experts.  For tests and tools: reading an
 * unmapped slot faults, so callers must only touch slots of loaded experts. */
ew_status_t ew_slot_address(ew_pool_t *pool, int32_t layer, int32_t which, int32_t slot, void **device_ptr);

const char *ew_status_str(ew_status_t s);
const char *ew_last_error_string(void); /* detail of the last EW_ERR_CUDA on this thread */

#ifdef __cplusplus
}
#endif
#endif /* EXPERTWEAVE_H_ */
