// Internal state of a pool and the launch interface between the host API and the kernels.
#pragma once
#include <cuda.h>
#include <cuda_runtime_api.h>

#include <cstdint>
#include <string>
#include <vector>

#include "../../include/expertweave.h"
#include "ew_vmm.h"

namespace ew {

// One work item of the grouped GEMMs, built on the device from the per-slot counts.  Thin item: a 128-row tile
// of one slot's weight matrix times up to NT token rows of that slot.  Fat item (CTA-pair kernel): 256 weight rows
// (GEMM-1: gate tile + up tile of 128 output features; GEMM-2: 256 output features) times 129..256 token rows.
struct alignas(16) GemmItem {
    int32_t slot;       // first-dimension index into the virtual weight tensor (>= P: shared expert)
    int32_t tile;       // tile of the weight matrix (thin: 128 rows; fat: see above)
    int32_t in_row;     // first activation row (x rows for shared experts, slot-contiguous rows otherwise)
    int32_t out_row;    // first output row
    int32_t rows;       // token rows in this item
    int32_t from_x;     // 1: activation rows come straight from the caller's x (shared experts)
    int32_t chain;      // experts chained along K in this item (GEMM-2 of the shared experts: S; otherwise 1): the
                        // item's K loop runs over slots slot .. slot + chain - 1, whose activation blocks start
    int32_t chain_rows; // chain_rows rows apart, and accumulates them into one output block
};

struct Workspace {
    int32_t *topk_ids = nullptr;   // [Bmax, k]
    float *topk_w = nullptr;       // [Bmax, k]
    int32_t *slot_ids = nullptr;   // [Bmax, k]
    int32_t *rank = nullptr;       // [Bmax, k] position of the pair inside its slot's chunk
    int32_t *inv = nullptr;        // [Bmax, k] row of the pair in slot-contiguous order
    int32_t *counts = nullptr;     // [P]
    int32_t *offsets = nullptr;    // [P + 1]
    int32_t *n_items = nullptr;    // [4]  thin items of GEMM-1, GEMM-2; fat items of GEMM-1, GEMM-2
    GemmItem *items1 = nullptr, *items2 = nullptr;   // thin items
    GemmItem *fat1 = nullptr, *fat2 = nullptr;       // fat items (prefill-sized batches)
    int32_t *src_tok = nullptr;    // [Bmax*k] token of each slot-contiguous row: GEMM-1 fetches those rows of x itself
    int32_t *slot_tok = nullptr;   // [P, B] self-planned forwards: the tokens of each slot in rank order, written by the router kernel
    void *act = nullptr;           // [S*Bmax + Bmax*k, I] bf16 SwiGLU output
    float *y = nullptr;            // [S*Bmax + Bmax*k, H] fp32 expert outputs
    int32_t *err = nullptr;        // device error word
    int32_t *loaded = nullptr;     // [N] 1 = adapter loaded
    size_t bytes = 0;
};

struct LayerState {
    VirtualTensor w13;             // [P + S, 2, I, H] bf16: per slot the gate block then the up block
    VirtualTensor w2;              // [P + S, H, I] bf16
    void *router_w = nullptr;      // device [M, H] bf16
    int32_t *pi_dev = nullptr;     // device [N, M]
    std::vector<int32_t> pi_host;  // master copy
    bool base_loaded = false;
    bool base_mapped = false;      // the pages under the base and shared experts are mapped (a failed first load is retried without remapping)
    CUtensorMap map_w13, map_w2;   // TMA descriptors over the two virtual tensors
    CUtensorMap map_router[3];     // and over the router rows [M, H], with boxes of 1, 2 and 4 K-atoms
};

}  // namespace ew

struct ew_pool {
    ew_config_t cfg;
    int P = 0;                      // M + N * E_max
    // expert parallelism: this rank holds the base experts [own_lo, own_hi) with every adapter's copies of them, and
    // the shared experts [sh_lo, sh_hi); without it, all of them
    int own_lo = 0, own_hi = 0, sh_lo = 0, sh_hi = 0;
    std::vector<std::vector<std::pair<int32_t, int32_t>>> adapter_owned;   // [N][L] positions [first, last) of an adapter's tuned experts held here
    int token_tile = 32;            // NT: token rows per thin work item (32, 64 or 128)
    bool fat = false;               // prefill-sized batch: blocks of more than 128 rows run on the CTA-pair kernel
    int last_forward_kernels = 0;   // kernels launched by the most recent forward (reported by ew_pool_stats)
    bool self_plan = false;         // decode-sized batch: no planning kernel, the GEMM kernels derive their items from the counts
    ew::PageBackend *be = nullptr;
    ew::PagePool pages;
    std::vector<ew::LayerState> layers;
    std::vector<std::vector<int32_t>> adapter_counts;   // [N][L]; empty = not loaded
    ew::Workspace ws;
    CUtensorMap map_act, map_act_big;   // TMA descriptors over the SwiGLU output (boxes of 64 x 32 and 64 x 128 rows)
    cudaStream_t copy_stream = nullptr;
    std::vector<std::pair<cudaStream_t, cudaEvent_t>> fwd_events;   // last forward per caller stream
    int sm_count = 148;
    bool counts_clean = true;      // the slot counters are zero (the combine kernel of a finished forward re-zeroes them)
    cudaEvent_t route_event = nullptr;   // last ew_route_noalloc call (created with the pool: that call creates nothing)
    bool route_event_used = false;
    bool profiling = false;
    bool profiling_this_forward = false;    // the forward being launched records events between its kernels
    std::vector<cudaEvent_t> prof_events;   // 6 per recorded forward
    size_t prof_used = 0;                   // events in use
    // ew_moe_forward_host: double-buffered device staging and three internal streams, so that the upload of call
    // n+1 and the download of call n-1 overlap the kernels of call n
    void *stage_x[2] = {nullptr, nullptr}, *stage_out[2] = {nullptr, nullptr};
    int32_t *stage_aid[2] = {nullptr, nullptr};
    cudaStream_t host_h2d = nullptr, host_comp = nullptr, host_d2h = nullptr;
    cudaEvent_t host_h2d_done[2] = {nullptr, nullptr}, host_comp_done[2] = {nullptr, nullptr}, host_d2h_done[2] = {nullptr, nullptr};
    uint64_t host_calls = 0;
    uint64_t live_expert_bytes = 0, live_experts = 0;
    CUresult (*encode_tiled)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                             const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill) = nullptr;
};

namespace ew {

void set_last_error(const std::string &s);

// Makes the pool's device current for the duration of an entry point and puts the caller's device back on exit.
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    cudaError_t enter(int device) {
        cudaError_t e = cudaGetDevice(&prev);
        if (e != cudaSuccess || prev == device) return e;
        e = cudaSetDevice(device);
        switched = e == cudaSuccess;
        return e;
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

// EW_DISABLE_PDL=1 in the environment turns the launch overlap off (plain stream order), for debugging.
bool pdl_enabled();
// EW_DISABLE_FAT=1 keeps every block of token rows on the weight-streaming kernel (128-row blocks at prefill).
bool fat_enabled();
// EW_DISABLE_SELFPLAN=1 runs the planning kernel for every batch size.
bool self_plan_enabled();

// Launch with programmatic stream serialization (the kernel calls pdl_wait() before it reads its
// predecessor's output).
template <class... KArgs, class... Args>
int launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return (int)cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// bf16 2-D/3-D tiled descriptor with 128-byte swizzle; dims/box innermost first.
int make_tensor_map(ew_pool *p, CUtensorMap *out, const void *base, int rank, const uint64_t *dims,
                    const uint32_t *box);

// bf16 [rows, H] matrix (H a multiple of 64) seen as (64 elements, rows, H/64 K-atoms): one box of
// 64 x box_rows x atoms lands in shared memory as `atoms` consecutive 128-byte-swizzled tiles.
int make_atom_map(ew_pool *p, CUtensorMap *out, const void *base, int H, int rows, int box_rows, int atoms);

// Kernel launchers (all asynchronous on `st`; return cudaError_t as int).
int launch_route(ew_pool *p, int layer, const void *x, const int32_t *aid, int B, cudaStream_t st);
int launch_permute(ew_pool *p, int B, cudaStream_t st);
int launch_gemm1(ew_pool *p, int layer, const CUtensorMap &map_x, const CUtensorMap &map_x_big, const void *x, int B,
                 cudaStream_t st);
int pick_token_tile(const ew_pool *p, int B);
int launch_gemm2(ew_pool *p, int layer, int B, cudaStream_t st);
// out_mode 0: bf16 result; 1: fp32 partial sums (expert parallelism); 2: fp32 partial sums stored into every rank's
// gather buffer (`out` = device array of ep_size pointers)
int launch_combine(ew_pool *p, int B, void *out, int out_mode, cudaStream_t st);
int launch_round_bf16(const float *in, int n_parts, void *out, size_t n, cudaStream_t st);   // out = bf16(in[0] + ... + in[n_parts - 1])
int launch_reroute(ew_pool *p, int layer, const int32_t *ids, const int32_t *aid, int B, int32_t *slots,
                   int32_t *counts, cudaStream_t st);
int launch_route_logits(ew_pool *p, int layer, const float *logits, const int32_t *aid, int B, int32_t *topk_ids,
                        float *topk_w, int32_t *slot_ids, int32_t *counts, cudaStream_t st);
bool self_plan_fits(const ew_pool *p, int B, int NT);   // a forward of B tokens with NT-row items can skip the planning kernel
int gemm_setup(ew_pool *p);   // once per pool: opt in to the shared memory the GEMM kernels need
int router_setup(ew_pool *p); // once per pool: the router kernels' attributes and the fixed scratch array's device address

}  // namespace ew
