// Host side of the C ABI: pool creation, base / adapter loading and eviction, the forward call.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "ew_internal.h"

namespace ew {
static thread_local std::string g_last_error;
void set_last_error(const std::string &s) { g_last_error = s; }
bool fat_enabled() {
    static const bool on = [] { const char *e = getenv("EW_DISABLE_FAT"); return !(e && e[0] == '1'); }();
    return on;
}
bool self_plan_enabled() {
    static const bool on = [] { const char *e = getenv("EW_DISABLE_SELFPLAN"); return !(e && e[0] == '1'); }();
    return on;
}
bool pdl_enabled() {
    static const bool on = [] { const char *e = getenv("EW_DISABLE_PDL"); return !(e && e[0] == '1'); }();
    return on;
}
}  // namespace ew

using namespace ew;

#define CU_TRY(expr)                                                                         \
    do {                                                                                     \
        cudaError_t e__ = (expr);                                                            \
        if (e__ != cudaSuccess) {                                                            \
            set_last_error(std::string(#expr) + ": " + cudaGetErrorString(e__));             \
            return e__ == cudaErrorMemoryAllocation ? EW_ERR_OOM : EW_ERR_CUDA;              \
        }                                                                                    \
    } while (0)

static ew_status_t be_status(ew_pool *p, int rc) {
    if (rc == 0) return EW_OK;
    set_last_error(p->be->last_error);
    return rc == 2 ? EW_ERR_OOM : EW_ERR_CUDA;
}

extern "C" const char *ew_status_str(ew_status_t s) {
    switch (s) {
        case EW_OK: return "EW_OK";
        case EW_ERR_INVALID_ARG: return "EW_ERR_INVALID_ARG";
        case EW_ERR_OOM: return "EW_ERR_OOM";
        case EW_ERR_SLOT_IN_USE: return "EW_ERR_SLOT_IN_USE";
        case EW_ERR_NOT_LOADED: return "EW_ERR_NOT_LOADED";
        case EW_ERR_TOO_MANY_EXPERTS: return "EW_ERR_TOO_MANY_EXPERTS";
        case EW_ERR_CUDA: return "EW_ERR_CUDA";
        case EW_ERR_TIMEOUT: return "EW_ERR_TIMEOUT";
        case EW_ERR_BAD_ADAPTER_ID_IN_BATCH: return "EW_ERR_BAD_ADAPTER_ID_IN_BATCH";
        case EW_ERR_NO_DEVICE: return "EW_ERR_NO_DEVICE";
    }
    return "EW_ERR_?";
}

extern "C" const char *ew_last_error_string(void) { return g_last_error.c_str(); }

int ew::make_tensor_map(ew_pool *p, CUtensorMap *out, const void *base, int rank, const uint64_t *dims,
                        const uint32_t *box) {
    cuuint64_t gdim[5], gstride[5];
    cuuint32_t bx[5], estr[5];
    uint64_t stride = 2;
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bx[i] = box[i];
        estr[i] = 1;
        stride *= dims[i];
        if (i + 1 < rank) gstride[i] = stride;   // byte stride of dimension i+1
    }
    CUresult r = p->encode_tiled(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), gdim,
                                 gstride, bx, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_error("cuTensorMapEncodeTiled failed with code " + std::to_string((int)r));
        return 1;
    }
    return 0;
}

int ew::make_atom_map(ew_pool *p, CUtensorMap *out, const void *base, int H, int rows, int box_rows, int atoms) {
    cuuint64_t gdim[3] = {64, (cuuint64_t)rows, (cuuint64_t)(H / 64)};
    cuuint64_t gstride[2] = {(cuuint64_t)H * 2, 128};
    cuuint32_t bx[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)atoms}, estr[3] = {1, 1, 1};
    CUresult r = p->encode_tiled(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), gdim, gstride, bx, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_error("cuTensorMapEncodeTiled (atom map) failed with code " + std::to_string((int)r));
        return 1;
    }
    return 0;
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static ew_status_t alloc_workspace(ew_pool *p) {
    const ew_config_t &c = p->cfg;
    size_t Bm = (size_t)c.max_tokens, k = c.top_k, P = p->P, S = c.num_shared, H = c.hidden, I = c.inter;
    // blocks of token rows: at most one ragged block per group plus the full blocks (32 rows at the least); a fat
    // block has more than 128 rows
    size_t rb = P + S * ((Bm + 31) / 32) + (Bm * k + 31) / 32 + 1;
    size_t rbf = (P + S) + (S * Bm + Bm * k) / 128 + 1;
    size_t r1 = (I + 127) / 128, r2 = (H + 127) / 128, rf2 = (H + 255) / 256;
    size_t rows = S * Bm + Bm * k + 32;     // +32: a token tile may start at the last row
    // self-planned forwards (batches below the prefill threshold of pick_token_tile): [P][B] tokens per slot
    size_t Bs = std::min(Bm, (size_t)128 * c.num_experts / k + 1);
    struct Seg { void **ptr; size_t bytes; };
    Workspace &w = p->ws;
    Seg segs[] = {
        {(void **)&w.topk_ids, Bm * k * 4}, {(void **)&w.topk_w, Bm * k * 4}, {(void **)&w.slot_ids, Bm * k * 4},
        {(void **)&w.rank, Bm * k * 4}, {(void **)&w.inv, Bm * k * 4}, {(void **)&w.counts, P * 4},
        {(void **)&w.offsets, (P + 1) * 4}, {(void **)&w.n_items, 16}, {(void **)&w.items1, rb * r1 * sizeof(GemmItem)},
        {(void **)&w.items2, rb * r2 * sizeof(GemmItem)}, {(void **)&w.fat1, rbf * r1 * sizeof(GemmItem)},
        {(void **)&w.fat2, rbf * rf2 * sizeof(GemmItem)}, {(void **)&w.src_tok, (Bm * k + 32) * 4},
        {(void **)&w.slot_tok, (P * Bs + 32) * 4},
        {(void **)&w.act, rows * I * 2}, {(void **)&w.y, rows * H * 4}, {(void **)&w.err, 256},
        {(void **)&w.loaded, (size_t)c.max_adapters * 4 + 16},
        {&p->stage_x[0], Bm * H * 2}, {&p->stage_out[0], Bm * H * 2}, {(void **)&p->stage_aid[0], Bm * 4},
        {&p->stage_x[1], Bm * H * 2}, {&p->stage_out[1], Bm * H * 2}, {(void **)&p->stage_aid[1], Bm * 4},
    };
    size_t total = 0;
    for (auto &s : segs) total += align_up(s.bytes, 1024);
    char *base = nullptr;
    CU_TRY(cudaMalloc(&base, total));
    CU_TRY(cudaMemset(base, 0, total));
    size_t off = 0;
    for (auto &s : segs) {
        *s.ptr = base + off;
        off += align_up(s.bytes, 1024);
    }
    w.bytes = total;
    // TMA descriptors over the SwiGLU output (boxes of 64 k-elements x 32 rows and x 128 rows)
    uint64_t d_act[2] = {I, rows};
    uint32_t box[2] = {64, 32}, bbox[2] = {64, 128};
    if (make_tensor_map(p, &p->map_act, w.act, 2, d_act, box) || make_tensor_map(p, &p->map_act_big, w.act, 2, d_act, bbox))
        return EW_ERR_CUDA;
    return EW_OK;
}

static void destroy_pool(ew_pool *p) {
    if (!p) return;
    bool gpu = p->cfg.device >= 0;
    DeviceGuard guard;
    if (gpu) {
        guard.enter(p->cfg.device);
        cudaDeviceSynchronize();
    }
    for (auto &L : p->layers) {
        L.w13.destroy();
        L.w2.destroy();
        if (gpu && L.router_w) cudaFree(L.router_w);
        if (gpu && L.pi_dev) cudaFree(L.pi_dev);
    }
    p->pages.trim();
    if (gpu) {
        if (p->ws.topk_ids) cudaFree(p->ws.topk_ids);   // the workspace is one allocation; topk_ids is its base
        for (auto &e : p->fwd_events) cudaEventDestroy(e.second);
        for (auto &e : p->prof_events) cudaEventDestroy(e);
        if (p->route_event) cudaEventDestroy(p->route_event);
        for (int i = 0; i < 2; ++i) {
            if (p->host_h2d_done[i]) cudaEventDestroy(p->host_h2d_done[i]);
            if (p->host_comp_done[i]) cudaEventDestroy(p->host_comp_done[i]);
            if (p->host_d2h_done[i]) cudaEventDestroy(p->host_d2h_done[i]);
        }
        if (p->host_h2d) cudaStreamDestroy(p->host_h2d);
        if (p->host_comp) cudaStreamDestroy(p->host_comp);
        if (p->host_d2h) cudaStreamDestroy(p->host_d2h);
        if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
    }
    delete p->be;
    delete p;
}

extern "C" ew_status_t ew_pool_create(const ew_config_t *cfg, ew_pool_t **out) {
    if (!cfg || !out) return EW_ERR_INVALID_ARG;
    const ew_config_t &c = *cfg;
    if (c.num_layers < 1 || c.hidden < 64 || c.inter < 8 || c.hidden % 64 || c.inter % 8 || c.num_experts < 1 ||
        c.num_experts > 256 || c.num_shared < 0 || c.top_k < 1 || c.top_k > 32 || c.top_k > c.num_experts ||
        c.max_adapters < 0 || c.e_max < 0 || c.max_tokens < 1 || (c.pool_mode != 0 && c.pool_mode != 1) ||
        (c.max_adapters > 0 && c.e_max < 1) || c.ep_size < 0 || c.ep_size > c.num_experts ||
        (c.ep_size > 1 ? (c.ep_rank < 0 || c.ep_rank >= c.ep_size) : c.ep_rank != 0)) {
        set_last_error("ew_pool_create: configuration out of range");
        return EW_ERR_INVALID_ARG;
    }
    ew_pool *p = new (std::nothrow) ew_pool();
    if (!p) return EW_ERR_OOM;
    p->cfg = c;
    p->P = c.num_experts + c.max_adapters * c.e_max;
    {   // expert parallelism: contiguous blocks of base experts (and of shared experts) per rank
        const int R = c.ep_size > 1 ? c.ep_size : 1, r = c.ep_rank;
        const int per = (c.num_experts + R - 1) / R, per_s = (c.num_shared + R - 1) / R;
        p->own_lo = std::min(c.num_experts, r * per);
        p->own_hi = std::min(c.num_experts, p->own_lo + per);
        p->sh_lo = std::min(c.num_shared, r * per_s);
        p->sh_hi = std::min(c.num_shared, p->sh_lo + per_s);
    }
    bool gpu = c.device >= 0;
    ew_status_t st = EW_OK;
    std::string err;
    DeviceGuard guard;
    if (gpu) {
        cudaError_t e = guard.enter(c.device);
        if (e != cudaSuccess) {
            set_last_error(std::string("cudaSetDevice: ") + cudaGetErrorString(e));
            delete p;
            return EW_ERR_CUDA;
        }
        cudaFree(0);
        p->be = make_cuda_backend(c.device, &err);
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (p->be && cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess && fn)
            p->encode_tiled = reinterpret_cast<decltype(p->encode_tiled)>(fn);
        if (!p->be || !p->encode_tiled) {
            set_last_error(err.empty() ? "cuTensorMapEncodeTiled not available" : err);
            delete p->be;
            delete p;
            return EW_ERR_CUDA;
        }
        cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, c.device);
    } else {
        p->be = make_mock_backend();
    }
    size_t gran = 0;
    if ((st = be_status(p, p->be->granularity(&gran))) != EW_OK) { destroy_pool(p); return st; }
    size_t page = c.page_bytes ? (size_t)c.page_bytes : gran;
    if (page % gran) {
        set_last_error("page_bytes must be a multiple of the allocation granularity");
        destroy_pool(p);
        return EW_ERR_INVALID_ARG;
    }
    p->pages.be = p->be;
    p->pages.page_bytes = page;
    p->pages.max_pages = c.max_pages;
    p->adapter_counts.assign(c.max_adapters, {});
    p->adapter_owned.assign(c.max_adapters, {});
    size_t H = c.hidden, I = c.inter, slots = (size_t)p->P + c.num_shared;
    p->layers.resize(c.num_layers);
    for (auto &L : p->layers) {
        if ((st = be_status(p, L.w13.init(p->be, &p->pages, 2 * I * H * 2, slots))) != EW_OK) break;
        if ((st = be_status(p, L.w2.init(p->be, &p->pages, H * I * 2, slots))) != EW_OK) break;
        L.pi_host.resize((size_t)c.max_adapters * c.num_experts);
        for (int i = 0; i < c.max_adapters; ++i)
            for (int j = 0; j < c.num_experts; ++j) L.pi_host[(size_t)i * c.num_experts + j] = j;
    }
    if (st == EW_OK) st = be_status(p, p->pages.prealloc(c.prealloc_pages));
    if (st == EW_OK && c.pool_mode == 1)   // padding baseline: back the whole tensor now
        for (auto &L : p->layers) {
            if ((st = be_status(p, L.w13.map_slots(0, slots))) != EW_OK) break;
            if ((st = be_status(p, L.w2.map_slots(0, slots))) != EW_OK) break;
        }
    if (st == EW_OK && gpu) {
        auto body = [&]() -> ew_status_t {
            CU_TRY(cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking));
            for (auto &L : p->layers) {
                CU_TRY(cudaMalloc(&L.router_w, (size_t)c.num_experts * H * 2));
                size_t pib = std::max<size_t>(L.pi_host.size() * 4, 16);
                CU_TRY(cudaMalloc(&L.pi_dev, pib));
                if (!L.pi_host.empty())
                    CU_TRY(cudaMemcpy(L.pi_dev, L.pi_host.data(), L.pi_host.size() * 4, cudaMemcpyHostToDevice));
                // gate|up tensor seen as [2*(P+S), I, H]; down tensor as [P+S, H, I]; box = 64 x 128 x 1
                uint64_t d13[3] = {H, I, 2 * slots}, d2[3] = {I, H, slots};
                uint32_t box[3] = {64, 128, 1};
                if (make_tensor_map(p, &L.map_w13, (void *)L.w13.base, 3, d13, box) ||
                    make_tensor_map(p, &L.map_w2, (void *)L.w2.base, 3, d2, box) ||
                    make_atom_map(p, &L.map_router[0], L.router_w, c.hidden, c.num_experts, (c.num_experts + 15) / 16 * 16, 1) ||
                    make_atom_map(p, &L.map_router[1], L.router_w, c.hidden, c.num_experts, (c.num_experts + 15) / 16 * 16, 2) ||
                    make_atom_map(p, &L.map_router[2], L.router_w, c.hidden, c.num_experts, (c.num_experts + 15) / 16 * 16, 4))
                    return EW_ERR_CUDA;
            }
            ew_status_t s = alloc_workspace(p);
            if (s != EW_OK) return s;
            if (gemm_setup(p) || router_setup(p)) return EW_ERR_CUDA;
            CU_TRY(cudaEventCreateWithFlags(&p->route_event, cudaEventDisableTiming));
            return EW_OK;
        };
        st = body();
    }
    if (st != EW_OK) {
        std::string keep = g_last_error;
        destroy_pool(p);
        set_last_error(keep);
        return st;
    }
    *out = p;
    return EW_OK;
}

extern "C" ew_status_t ew_pool_destroy(ew_pool_t *pool) {
    if (!pool) return EW_ERR_INVALID_ARG;
    destroy_pool(pool);
    return EW_OK;
}

extern "C" ew_status_t ew_pool_trim(ew_pool_t *p) {
    if (!p) return EW_ERR_INVALID_ARG;
    return be_status(p, p->pages.trim());
}

// Copy e experts' gate and up blocks into slots [first, first+e) of the fused tensor, and the down
// blocks into the down tensor.  Source layout: [e, I, H], [e, I, H], [e, H, I].
// Weight sources may be host (pageable or page-locked) or device memory: the copy kind is left to unified addressing.
static ew_status_t copy_gate_up(ew_pool *p, LayerState &L, size_t first, size_t e, const void *g, const void *u) {
    if (e == 0 || p->cfg.device < 0) return EW_OK;
    size_t blk = (size_t)p->cfg.inter * p->cfg.hidden * 2;
    char *dst13 = (char *)L.w13.slot_addr(first);
    CU_TRY(cudaMemcpy2DAsync(dst13, 2 * blk, g, blk, blk, e, cudaMemcpyDefault, p->copy_stream));
    CU_TRY(cudaMemcpy2DAsync(dst13 + blk, 2 * blk, u, blk, blk, e, cudaMemcpyDefault, p->copy_stream));
    return EW_OK;
}
static ew_status_t copy_down(ew_pool *p, LayerState &L, size_t first, size_t e, const void *d) {
    if (e == 0 || p->cfg.device < 0) return EW_OK;
    size_t blk = (size_t)p->cfg.inter * p->cfg.hidden * 2;
    CU_TRY(cudaMemcpyAsync((void *)L.w2.slot_addr(first), d, blk * e, cudaMemcpyDefault, p->copy_stream));
    return EW_OK;
}
static ew_status_t copy_experts(ew_pool *p, LayerState &L, size_t first, size_t e, const void *g, const void *u,
                                const void *d) {
    ew_status_t st = copy_gate_up(p, L, first, e, g, u);
    return st == EW_OK ? copy_down(p, L, first, e, d) : st;
}

extern "C" ew_status_t ew_load_base(ew_pool_t *p, int32_t layer, const void *router_w, const void *w_gate,
                                    const void *w_up, const void *w_down, const void *sh_gate, const void *sh_up,
                                    const void *sh_down) {
    if (!p || layer < 0 || layer >= p->cfg.num_layers) return EW_ERR_INVALID_ARG;
    const ew_config_t &c = p->cfg;
    bool gpu = c.device >= 0;
    if (gpu && (!router_w || !w_gate || !w_up || !w_down || (c.num_shared > 0 && (!sh_gate || !sh_up || !sh_down))))
        return EW_ERR_INVALID_ARG;
    DeviceGuard guard;
    if (gpu) CU_TRY(guard.enter(c.device));
    LayerState &L = p->layers[layer];
    size_t M = c.num_experts, P = p->P;
    // the experts this rank holds (all of them without expert parallelism): base [m0, m0 + Mo), shared [s0, s0 + So)
    const size_t m0 = p->own_lo, Mo = p->own_hi - p->own_lo, s0 = p->sh_lo, So = p->sh_hi - p->sh_lo;
    if (!L.base_mapped && c.pool_mode == 0) {
        ew_status_t st;
        if ((st = be_status(p, L.w13.map_slots(m0, Mo))) != EW_OK) return st;
        if ((st = be_status(p, L.w2.map_slots(m0, Mo))) != EW_OK) { L.w13.unmap_slots(m0, Mo); return st; }
        if ((st = be_status(p, L.w13.map_slots(P + s0, So))) != EW_OK) { L.w13.unmap_slots(m0, Mo); L.w2.unmap_slots(m0, Mo); return st; }
        if ((st = be_status(p, L.w2.map_slots(P + s0, So))) != EW_OK) {
            L.w13.unmap_slots(m0, Mo); L.w2.unmap_slots(m0, Mo); L.w13.unmap_slots(P + s0, So);
            return st;
        }
    }
    L.base_mapped = true;
    if (gpu) {
        // forwards in flight may still read the old weights of this layer
        for (auto &e : p->fwd_events) CU_TRY(cudaEventSynchronize(e.second));
        if (p->route_event_used) CU_TRY(cudaEventSynchronize(p->route_event));
        const size_t blk = (size_t)c.inter * c.hidden * 2;
        auto at = [blk](const void *base, size_t i) { return (const void *)((const char *)base + i * blk); };
        CU_TRY(cudaMemcpyAsync(L.router_w, router_w, M * c.hidden * 2, cudaMemcpyDefault, p->copy_stream));
        ew_status_t st = copy_experts(p, L, m0, Mo, at(w_gate, m0), at(w_up, m0), at(w_down, m0));
        if (st == EW_OK && So) st = copy_experts(p, L, P + s0, So, at(sh_gate, s0), at(sh_up, s0), at(sh_down, s0));
        if (st != EW_OK) return st;
        CU_TRY(cudaStreamSynchronize(p->copy_stream));
    }
    if (!L.base_loaded) {                               // counted once, when the first load of the layer has succeeded
        p->live_experts += Mo;
        p->live_expert_bytes += (Mo + So) * 3 * (size_t)c.inter * c.hidden * 2;
    }
    L.base_loaded = true;
    return EW_OK;
}

extern "C" ew_status_t ew_load_adapter(ew_pool_t *p, int32_t a, const int32_t *counts, const int32_t *expert_ids,
                                       const void *w_gate, const void *w_up, const void *w_down) {
    if (!p || !counts || a < 0 || a >= p->cfg.max_adapters) return EW_ERR_INVALID_ARG;
    const ew_config_t &c = p->cfg;
    bool gpu = c.device >= 0;
    int L = c.num_layers, M = c.num_experts;
    if (!p->adapter_counts[a].empty()) return EW_ERR_SLOT_IN_USE;
    size_t total = 0;
    for (int l = 0; l < L; ++l) {
        if (counts[l] < 0) return EW_ERR_INVALID_ARG;
        if (counts[l] > c.e_max) return EW_ERR_TOO_MANY_EXPERTS;
        total += counts[l];
    }
    if (total && (!expert_ids || (gpu && (!w_gate || !w_up || !w_down)))) return EW_ERR_INVALID_ARG;
    for (size_t l = 0, q = 0; l < (size_t)L; ++l)
        for (int r = 0; r < counts[l]; ++r, ++q) {
            int j = expert_ids[q];
            if (j < 0 || j >= M || (r > 0 && expert_ids[q - 1] >= j)) {
                set_last_error("ew_load_adapter: expert ids must be strictly ascending in [0,M) per layer");
                return EW_ERR_INVALID_ARG;
            }
        }
    DeviceGuard guard;
    if (gpu) CU_TRY(guard.enter(c.device));
    size_t delta = (size_t)M + (size_t)a * c.e_max;     // Delta_i = M + i * E_max
    // Expert parallelism: of each layer's tuned experts (ascending base ids) this rank holds those whose base expert
    // it holds, a contiguous run [first, last) of positions; the others' slots stay unmapped here.
    std::vector<std::pair<int32_t, int32_t>> own(L);
    size_t owned_total = 0;
    for (size_t l = 0, q0 = 0; l < (size_t)L; q0 += counts[l], ++l) {
        int lo = 0, hi = 0;
        for (int r = 0; r < counts[l]; ++r) {
            if (expert_ids[q0 + r] < p->own_lo) ++lo;
            if (expert_ids[q0 + r] < p->own_hi) ++hi;
        }
        own[l] = {lo, hi};
        owned_total += hi - lo;
    }
    ew_status_t st = EW_OK;
    // Layer by layer, tensor by tensor: map the slots' pages (driver calls on this thread, ~0.1 ms per page), then
    // queue the copy into them, so that the copies run while the next pages are being mapped.
    int done13 = 0, done2 = 0;                          // layers whose gate/up and down slots are mapped (for rollback)
    const bool vmm = c.pool_mode == 0;
    size_t blk = (size_t)c.inter * c.hidden * 2;
    size_t q = 0;
    for (int l = 0; l < L && st == EW_OK; ++l) {
        LayerState &Ls = p->layers[l];
        const size_t first = delta + own[l].first, n = own[l].second - own[l].first, src = q + own[l].first;
        if (vmm && (st = be_status(p, Ls.w13.map_slots(first, n))) == EW_OK) ++done13;
        if (st == EW_OK && gpu)
            st = copy_gate_up(p, Ls, first, n, (const char *)w_gate + src * blk, (const char *)w_up + src * blk);
        if (st == EW_OK && vmm && (st = be_status(p, Ls.w2.map_slots(first, n))) == EW_OK) ++done2;
        if (st == EW_OK && gpu) st = copy_down(p, Ls, first, n, (const char *)w_down + src * blk);
        q += counts[l];
    }
    if (gpu && cudaStreamSynchronize(p->copy_stream) != cudaSuccess && st == EW_OK) {   // also before any rollback
        set_last_error("ew_load_adapter: weight copy failed");
        st = EW_ERR_CUDA;
    }
    if (st != EW_OK) {
        for (int l = 0; l < done13; ++l) p->layers[l].w13.unmap_slots(delta + own[l].first, own[l].second - own[l].first);
        for (int l = 0; l < done2; ++l) p->layers[l].w2.unmap_slots(delta + own[l].first, own[l].second - own[l].first);
        return st;
    }
    // publish: Pi[l][a][j] = Delta + rank of j, only after the weights are in place
    for (size_t l = 0, q = 0; l < (size_t)L; ++l) {
        LayerState &Ls = p->layers[l];
        int32_t *row = Ls.pi_host.data() + (size_t)a * M;
        for (int r = 0; r < counts[l]; ++r, ++q) row[expert_ids[q]] = (int32_t)(delta + r);
        if (gpu) CU_TRY(cudaMemcpyAsync(Ls.pi_dev + (size_t)a * M, row, (size_t)M * 4, cudaMemcpyHostToDevice, p->copy_stream));
    }
    if (gpu) {
        int32_t one = 1;
        CU_TRY(cudaMemcpyAsync(p->ws.loaded + a, &one, 4, cudaMemcpyHostToDevice, p->copy_stream));
        CU_TRY(cudaStreamSynchronize(p->copy_stream));
    }
    p->adapter_counts[a].assign(counts, counts + L);
    p->adapter_owned[a] = own;
    p->live_experts += owned_total;
    p->live_expert_bytes += owned_total * 3 * blk;
    return EW_OK;
}

extern "C" ew_status_t ew_unload_adapter(ew_pool_t *p, int32_t a) {
    if (!p || a < 0 || a >= p->cfg.max_adapters) return EW_ERR_INVALID_ARG;
    if (p->adapter_counts[a].empty()) return EW_ERR_NOT_LOADED;
    const ew_config_t &c = p->cfg;
    bool gpu = c.device >= 0;
    int L = c.num_layers, M = c.num_experts;
    DeviceGuard guard;
    if (gpu) CU_TRY(guard.enter(c.device));
    // 1. forwards (and allocation-free routing calls) issued earlier may still read the adapter's slots and its
    //    map rows: let them finish as issued
    if (gpu) {
        for (auto &e : p->fwd_events) CU_TRY(cudaEventSynchronize(e.second));
        if (p->route_event_used) CU_TRY(cudaEventSynchronize(p->route_event));
    }
    // 2. rows back to identity, so that later forwards no longer reach the adapter's slots
    for (int l = 0; l < L; ++l) {
        LayerState &Ls = p->layers[l];
        int32_t *row = Ls.pi_host.data() + (size_t)a * M;
        for (int j = 0; j < M; ++j) row[j] = j;
        if (gpu) CU_TRY(cudaMemcpyAsync(Ls.pi_dev + (size_t)a * M, row, (size_t)M * 4, cudaMemcpyHostToDevice, p->copy_stream));
    }
    if (gpu) {
        int32_t zero = 0;
        CU_TRY(cudaMemcpyAsync(p->ws.loaded + a, &zero, 4, cudaMemcpyHostToDevice, p->copy_stream));
        CU_TRY(cudaStreamSynchronize(p->copy_stream));
    }
    // 3. drop the reference counts; pages reaching zero go back to the pool
    size_t delta = (size_t)M + (size_t)a * c.e_max, total = 0;
    for (int l = 0; l < L; ++l) {
        const auto &o = p->adapter_owned[a][l];
        const int e = o.second - o.first;
        total += e;
        if (c.pool_mode == 0) {
            p->layers[l].w13.unmap_slots(delta + o.first, e);
            p->layers[l].w2.unmap_slots(delta + o.first, e);
        }
    }
    p->adapter_counts[a].clear();
    p->adapter_owned[a].clear();
    p->live_experts -= total;
    p->live_expert_bytes -= total * 3 * (size_t)c.inter * c.hidden * 2;
    return EW_OK;
}

extern "C" ew_status_t ew_get_expert_map(ew_pool_t *p, int32_t layer, int32_t *host_out) {
    if (!p || !host_out || layer < 0 || layer >= p->cfg.num_layers) return EW_ERR_INVALID_ARG;
    const auto &pi = p->layers[layer].pi_host;
    if (!pi.empty()) memcpy(host_out, pi.data(), pi.size() * 4);
    return EW_OK;
}

extern "C" ew_status_t ew_pool_stats(ew_pool_t *p, ew_stats_t *out) {
    if (!p || !out) return EW_ERR_INVALID_ARG;
    memset(out, 0, sizeof(*out));
    const ew_config_t &c = p->cfg;
    out->page_bytes = p->pages.page_bytes;
    for (auto &L : p->layers) {
        out->va_reserved_bytes += L.w13.va_bytes + L.w2.va_bytes;
        out->pages_mapped += L.w13.pages_mapped + L.w2.pages_mapped;
    }
    out->pages_free = p->pages.free_list.size();
    out->pages_created_total = p->pages.created_total;
    out->physical_bytes = (out->pages_mapped + out->pages_free) * out->page_bytes;
    out->live_expert_bytes = p->live_expert_bytes;
    out->padding_bytes = (uint64_t)c.num_layers * ((uint64_t)p->P + c.num_shared) * 3 * c.inter * c.hidden * 2;
    out->live_experts = p->live_experts;
    for (auto &a : p->adapter_counts) out->adapters_loaded += !a.empty();
    out->workspace_bytes = p->ws.bytes;
    out->last_forward_kernels = p->last_forward_kernels;
    return EW_OK;
}

extern "C" ew_status_t ew_slot_address(ew_pool_t *p, int32_t layer, int32_t which, int32_t slot, void **ptr) {
    if (!p || !ptr || layer < 0 || layer >= p->cfg.num_layers || slot < 0 || slot >= p->P + p->cfg.num_shared ||
        (which != 0 && which != 1))
        return EW_ERR_INVALID_ARG;
    LayerState &L = p->layers[layer];
    *ptr = (void *)(which == 0 ? L.w13.slot_addr(slot) : L.w2.slot_addr(slot));
    return EW_OK;
}

extern "C" ew_status_t ew_last_device_error(ew_pool_t *p, int32_t *code) {
    if (!p || !code) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    DeviceGuard guard;
    CU_TRY(guard.enter(p->cfg.device));
    for (auto &e : p->fwd_events) CU_TRY(cudaEventSynchronize(e.second));
    int32_t v = 0;
    CU_TRY(cudaMemcpy(&v, p->ws.err, 4, cudaMemcpyDeviceToHost));
    CU_TRY(cudaMemset(p->ws.err, 0, 4));
    // a kernel that gave up on a wait may have left the forward unfinished: the combine kernel, which leaves the slot
    // counters at zero for the next forward, may not have run
    if (v & 2) {
        p->counts_clean = false;
        CU_TRY(cudaMemset(p->ws.err + 8, 0, 8));        // and the rerouting operator's zeroing handshake may be half done
    }
    // the word is a bit set: 1 = bad adapter id, 2 = a bounded wait expired, 4 = expert id out of range
    *code = (v & 2) ? EW_ERR_TIMEOUT : (v & 1) ? EW_ERR_BAD_ADAPTER_ID_IN_BATCH : (v & 4) ? EW_ERR_INVALID_ARG : EW_OK;
    return EW_OK;
}

// The pool has one workspace: a forward issued on one stream must not overlap a forward that was issued earlier on
// another.  Makes `st` wait for the last forward of every other stream (a no-op when those have finished).
static ew_status_t order_after_other_streams(ew_pool *p, cudaStream_t st) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap != cudaStreamCaptureStatusNone) return EW_OK;
    for (auto &e : p->fwd_events)
        if (e.first != st) CU_TRY(cudaStreamWaitEvent(st, e.second, 0));
    return EW_OK;
}

static ew_status_t note_forward(ew_pool *p, cudaStream_t st) {
    // A forward that is being captured into a CUDA graph is not running yet: there is nothing to record.  The
    // caller who replays such a graph orders its replays against ew_unload_adapter / ew_load_base itself.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap != cudaStreamCaptureStatusNone) return EW_OK;
    for (auto &e : p->fwd_events)
        if (e.first == st) {
            CU_TRY(cudaEventRecord(e.second, st));
            return EW_OK;
        }
    // a caller that keeps creating streams would grow the list without bound: entries whose forward has completed
    // carry no ordering information any more
    if (p->fwd_events.size() >= 32) {
        size_t kept = 0;
        for (auto &e : p->fwd_events) {
            if (cudaEventQuery(e.second) == cudaSuccess) cudaEventDestroy(e.second);
            else p->fwd_events[kept++] = e;
        }
        p->fwd_events.resize(kept);
        (void)cudaGetLastError();                       // cudaErrorNotReady from the queries is not an error
    }
    cudaEvent_t ev;
    CU_TRY(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    CU_TRY(cudaEventRecord(ev, st));
    p->fwd_events.push_back({st, ev});
    return EW_OK;
}

#define LAUNCH_TRY(call)                                                                       \
    do {                                                                                       \
        int e__ = (call);                                                                      \
        if (e__ != 0) {                                                                        \
            set_last_error(std::string(#call) + ": " + cudaGetErrorString((cudaError_t)e__));  \
            return EW_ERR_CUDA;                                                                \
        }                                                                                      \
    } while (0)

// The forward.  out_mode 0: `out` receives the rounded bf16 result; 1: this rank's fp32 partial sums; 2: `out` is a device
// array of ep_size gather buffers, each of which receives the partial sums in block ep_rank.
static ew_status_t forward_impl(ew_pool_t *p, int32_t layer, const void *x, const int32_t *aid, int32_t B, void *out,
                                int out_mode, void *cuda_stream, int32_t *topk_ids, float *topk_w, int32_t *slot_ids,
                                int32_t *counts, int32_t *inv, int32_t *offsets) {
    if (!p || layer < 0 || layer >= p->cfg.num_layers || B < 0 || B > p->cfg.max_tokens) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    if (out_mode == 0 && p->cfg.ep_size > 1) {
        set_last_error("this pool holds one rank's share of the experts: call ew_moe_forward_partial, add the ranks' partial sums, then ew_ep_finish");
        return EW_ERR_INVALID_ARG;
    }
    if (B == 0) return EW_OK;
    if (!x || !aid || !out || ((uintptr_t)x & 15) || ((uintptr_t)out & 15)) return EW_ERR_INVALID_ARG;
    if (!p->layers[layer].base_loaded) return EW_ERR_NOT_LOADED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const ew_config_t &c = p->cfg;
    DeviceGuard guard;
    CU_TRY(guard.enter(c.device));
    // the caller's x becomes the activation operand of the shared experts: describe it for TMA
    CUtensorMap map_x;
    uint64_t dx[2] = {(uint64_t)c.hidden, (uint64_t)B};
    uint32_t box[2] = {64, 32};
    if (make_tensor_map(p, &map_x, x, 2, dx, box)) return EW_ERR_CUDA;
    CUtensorMap map_x_big = map_x;
    // Token rows per thin work item, and whether the batch is large enough for fat items (blocks of more than 128
    // rows on the CTA-pair kernel).  A permuted copy of x (k rows per token) is never written: the permute kernel
    // only records which token each slot-contiguous row is, and GEMM-1 gathers those rows of x (which stay in L2).
    const int tile = pick_token_tile(p, B);
    p->fat = tile == 256 && fat_enabled();
    p->token_tile = tile == 256 ? 128 : tile;
    // decode-sized batches run without the planning kernel when every GEMM CTA can hold its own items
    p->self_plan = !p->fat && tile != 256 && self_plan_enabled() && self_plan_fits(p, B, p->token_tile);
    if (p->token_tile >= 128) {
        uint32_t bbox[2] = {64, 128};
        if (make_tensor_map(p, &map_x_big, x, 2, dx, bbox)) return EW_ERR_CUDA;
    }
    size_t nk = (size_t)B * c.top_k;
    cudaEvent_t *pe = nullptr;
    if (p->profiling && p->prof_used + 6 <= 6 * 4096) {
        while (p->prof_events.size() < p->prof_used + 6) {
            cudaEvent_t ev;
            CU_TRY(cudaEventCreate(&ev));
            p->prof_events.push_back(ev);
        }
        pe = p->prof_events.data() + p->prof_used;
        p->prof_used += 6;
    }
    p->profiling_this_forward = pe != nullptr;
#define PROF_MARK(i) do { if (pe) CU_TRY(cudaEventRecord(pe[i], st)); } while (0)
    {
        ew_status_t ordered = order_after_other_streams(p, st);
        if (ordered != EW_OK) return ordered;
    }
    PROF_MARK(0);
    if (!p->counts_clean) CU_TRY(cudaMemsetAsync(p->ws.counts, 0, (size_t)p->P * 4, st));   // an earlier forward failed midway
    p->counts_clean = false;
    LAUNCH_TRY(launch_route(p, layer, x, aid, B, st));
    PROF_MARK(1);
    if (!p->self_plan) LAUNCH_TRY(launch_permute(p, B, st));
    PROF_MARK(2);
    if (topk_ids) CU_TRY(cudaMemcpyAsync(topk_ids, p->ws.topk_ids, nk * 4, cudaMemcpyDeviceToDevice, st));
    if (topk_w) CU_TRY(cudaMemcpyAsync(topk_w, p->ws.topk_w, nk * 4, cudaMemcpyDeviceToDevice, st));
    if (slot_ids) CU_TRY(cudaMemcpyAsync(slot_ids, p->ws.slot_ids, nk * 4, cudaMemcpyDeviceToDevice, st));
    if (counts) CU_TRY(cudaMemcpyAsync(counts, p->ws.counts, (size_t)p->P * 4, cudaMemcpyDeviceToDevice, st));
    // the pair -> row table and the offsets come from the planning kernel, or (self-planned forwards) from GEMM-1's CTAs
    if (p->self_plan) LAUNCH_TRY(launch_gemm1(p, layer, map_x, map_x_big, x, B, st));
    if (inv) CU_TRY(cudaMemcpyAsync(inv, p->ws.inv, nk * 4, cudaMemcpyDeviceToDevice, st));
    if (offsets) CU_TRY(cudaMemcpyAsync(offsets, p->ws.offsets, ((size_t)p->P + 1) * 4, cudaMemcpyDeviceToDevice, st));
    if (!p->self_plan) LAUNCH_TRY(launch_gemm1(p, layer, map_x, map_x_big, x, B, st));
    PROF_MARK(3);
    LAUNCH_TRY(launch_gemm2(p, layer, B, st));
    PROF_MARK(4);
    LAUNCH_TRY(launch_combine(p, B, out, out_mode, st));
    p->counts_clean = true;                             // the combine kernel zeroes the counters when it is done with them
    p->last_forward_kernels = p->self_plan ? 4 : p->fat ? 7 : 5;
    PROF_MARK(5);
#undef PROF_MARK
    return note_forward(p, st);
}

extern "C" ew_status_t ew_moe_forward_debug(ew_pool_t *p, int32_t layer, const void *x, const int32_t *aid,
                                            int32_t B, void *out, void *cuda_stream, int32_t *topk_ids,
                                            float *topk_w, int32_t *slot_ids, int32_t *counts, int32_t *inv,
                                            int32_t *offsets) {
    return forward_impl(p, layer, x, aid, B, out, 0, cuda_stream, topk_ids, topk_w, slot_ids, counts, inv, offsets);
}

extern "C" ew_status_t ew_moe_forward(ew_pool_t *p, int32_t layer, const void *x, const int32_t *aid, int32_t B,
                                      void *out, void *cuda_stream) {
    return forward_impl(p, layer, x, aid, B, out, 0, cuda_stream, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr);
}

extern "C" ew_status_t ew_moe_forward_partial(ew_pool_t *p, int32_t layer, const void *x, const int32_t *aid, int32_t B,
                                              float *partial, void *cuda_stream) {
    return forward_impl(p, layer, x, aid, B, partial, 1, cuda_stream, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr);
}

extern "C" ew_status_t ew_moe_forward_scatter(ew_pool_t *p, int32_t layer, const void *x, const int32_t *aid, int32_t B,
                                              float *const *gather_bufs, void *cuda_stream) {
    return forward_impl(p, layer, x, aid, B, (void *)gather_bufs, 2, cuda_stream, nullptr, nullptr, nullptr, nullptr, nullptr,
                        nullptr);
}

extern "C" ew_status_t ew_ep_finish_gathered(ew_pool_t *p, const float *gathered, int32_t B, void *out, void *cuda_stream) {
    if (!p || B < 0) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    if (B == 0) return EW_OK;
    if (!gathered || !out || ((uintptr_t)gathered & 15) || ((uintptr_t)out & 7)) return EW_ERR_INVALID_ARG;
    DeviceGuard guard;
    CU_TRY(guard.enter(p->cfg.device));
    LAUNCH_TRY(launch_round_bf16(gathered, p->cfg.ep_size > 1 ? p->cfg.ep_size : 1, out, (size_t)B * p->cfg.hidden,
                                 (cudaStream_t)cuda_stream));
    return EW_OK;
}

extern "C" ew_status_t ew_ep_finish(ew_pool_t *p, const float *summed, int32_t B, void *out, void *cuda_stream) {
    if (!p || B < 0) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    if (B == 0) return EW_OK;
    if (!summed || !out || ((uintptr_t)summed & 15) || ((uintptr_t)out & 7)) return EW_ERR_INVALID_ARG;
    DeviceGuard guard;
    CU_TRY(guard.enter(p->cfg.device));
    LAUNCH_TRY(launch_round_bf16(summed, 1, out, (size_t)B * p->cfg.hidden, (cudaStream_t)cuda_stream));
    return EW_OK;
}

extern "C" ew_status_t ew_reroute(ew_pool_t *p, int32_t layer, const int32_t *topk_ids, const int32_t *aid,
                                  int32_t B, int32_t *slot_ids, int32_t *counts, void *cuda_stream) {
    if (!p || layer < 0 || layer >= p->cfg.num_layers || B < 0) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    DeviceGuard guard;
    CU_TRY(guard.enter(p->cfg.device));
    if (B == 0) {
        if (counts) CU_TRY(cudaMemsetAsync(counts, 0, (size_t)p->P * 4, st));
        return EW_OK;
    }
    if (!topk_ids || !aid || !slot_ids || ((uintptr_t)topk_ids & 3) || ((uintptr_t)slot_ids & 3)) return EW_ERR_INVALID_ARG;
    // the aligned kernel zeroes the counters itself (one launch per call) through two words of the pool's workspace:
    // calls on different streams are ordered like forwards
    const bool aligned = (((uintptr_t)topk_ids | (uintptr_t)slot_ids | (uintptr_t)aid) & 15) == 0;
    if (aligned) {
        ew_status_t ordered = order_after_other_streams(p, st);
        if (ordered != EW_OK) return ordered;
    } else if (counts) {
        CU_TRY(cudaMemsetAsync(counts, 0, (size_t)p->P * 4, st));
    }
    LAUNCH_TRY(launch_reroute(p, layer, topk_ids, aid, B, slot_ids, counts, st));
    return note_forward(p, st);
}

extern "C" ew_status_t ew_route_logits(ew_pool_t *p, int32_t layer, const float *logits, const int32_t *aid, int32_t B,
                                       int32_t *topk_ids, float *topk_w, int32_t *slot_ids, int32_t *counts,
                                       void *cuda_stream) {
    if (!p || layer < 0 || layer >= p->cfg.num_layers || B < 0 || !counts) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    if (!p->layers[layer].base_loaded) return EW_ERR_NOT_LOADED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    DeviceGuard guard;
    CU_TRY(guard.enter(p->cfg.device));
    CU_TRY(cudaMemsetAsync(counts, 0, (size_t)p->P * 4, st));
    if (B == 0) return EW_OK;
    if (!logits || !aid || !topk_ids || !topk_w || !slot_ids || ((uintptr_t)logits & 15) || (p->cfg.num_experts & 3)) {
        set_last_error("ew_route_logits: null argument, logits not 16-byte aligned, or M not a multiple of 4");
        return EW_ERR_INVALID_ARG;
    }
    LAUNCH_TRY(launch_route_logits(p, layer, logits, aid, B, topk_ids, topk_w, slot_ids, counts, st));
    return note_forward(p, st);
}

extern "C" ew_status_t ew_moe_forward_host(ew_pool_t *p, int32_t layer, const void *x_host, const int32_t *aid_host,
                                           int32_t B, void *out_host, void *cuda_stream) {
    if (!p || layer < 0 || layer >= p->cfg.num_layers || B < 0 || B > p->cfg.max_tokens) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    if (B == 0) return EW_OK;
    if (!x_host || !aid_host || !out_host) return EW_ERR_INVALID_ARG;
    cudaStream_t user = (cudaStream_t)cuda_stream;
    DeviceGuard guard;
    CU_TRY(guard.enter(p->cfg.device));
    if (!p->host_h2d) {                                   // first use: the pipeline's streams and events
        CU_TRY(cudaStreamCreateWithFlags(&p->host_h2d, cudaStreamNonBlocking));
        CU_TRY(cudaStreamCreateWithFlags(&p->host_comp, cudaStreamNonBlocking));
        CU_TRY(cudaStreamCreateWithFlags(&p->host_d2h, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            CU_TRY(cudaEventCreateWithFlags(&p->host_h2d_done[i], cudaEventDisableTiming));
            CU_TRY(cudaEventCreateWithFlags(&p->host_comp_done[i], cudaEventDisableTiming));
            CU_TRY(cudaEventCreateWithFlags(&p->host_d2h_done[i], cudaEventDisableTiming));
        }
    }
    const int slot = (int)(p->host_calls & 1);
    const bool reuse = p->host_calls >= 2;                // the slot was used two calls ago
    const size_t xb = (size_t)B * p->cfg.hidden * 2;
    // upload: may start as soon as the kernels of the call that last used this slot have read it
    if (reuse) CU_TRY(cudaStreamWaitEvent(p->host_h2d, p->host_comp_done[slot], 0));
    CU_TRY(cudaMemcpyAsync(p->stage_x[slot], x_host, xb, cudaMemcpyHostToDevice, p->host_h2d));
    CU_TRY(cudaMemcpyAsync(p->stage_aid[slot], aid_host, (size_t)B * 4, cudaMemcpyHostToDevice, p->host_h2d));
    CU_TRY(cudaEventRecord(p->host_h2d_done[slot], p->host_h2d));
    // kernels: after the upload, after the download that last read this slot's output, and after forwards the
    // caller issued directly on other streams (they share the workspace)
    CU_TRY(cudaStreamWaitEvent(p->host_comp, p->host_h2d_done[slot], 0));
    if (reuse) CU_TRY(cudaStreamWaitEvent(p->host_comp, p->host_d2h_done[slot], 0));
    for (auto &e : p->fwd_events)
        if (e.first != p->host_comp) CU_TRY(cudaStreamWaitEvent(p->host_comp, e.second, 0));
    ew_status_t s = ew_moe_forward(p, layer, p->stage_x[slot], p->stage_aid[slot], B, p->stage_out[slot], p->host_comp);
    if (s != EW_OK) return s;
    CU_TRY(cudaEventRecord(p->host_comp_done[slot], p->host_comp));
    // download, then join the caller's stream: synchronising it covers the whole call
    CU_TRY(cudaStreamWaitEvent(p->host_d2h, p->host_comp_done[slot], 0));
    CU_TRY(cudaMemcpyAsync(out_host, p->stage_out[slot], xb, cudaMemcpyDeviceToHost, p->host_d2h));
    CU_TRY(cudaEventRecord(p->host_d2h_done[slot], p->host_d2h));
    CU_TRY(cudaStreamWaitEvent(user, p->host_d2h_done[slot], 0));
    ++p->host_calls;
    return EW_OK;
}

extern "C" ew_status_t ew_profile_enable(ew_pool_t *p, int32_t on) {
    if (!p) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    p->profiling = on != 0;
    return EW_OK;
}

extern "C" ew_status_t ew_profile_read(ew_pool_t *p, double *ms, int32_t *n_forwards) {
    if (!p || !ms || !n_forwards) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    DeviceGuard guard;
    CU_TRY(guard.enter(p->cfg.device));
    for (int i = 0; i < 5; ++i) ms[i] = 0.0;
    size_t n = p->prof_used / 6;
    for (size_t f = 0; f < n; ++f) {
        cudaEvent_t *e = p->prof_events.data() + 6 * f;
        CU_TRY(cudaEventSynchronize(e[5]));
        for (int i = 0; i < 5; ++i) {
            float t = 0.f;
            CU_TRY(cudaEventElapsedTime(&t, e[i], e[i + 1]));
            ms[i] += t;
        }
    }
    *n_forwards = (int32_t)n;
    p->prof_used = 0;
    return EW_OK;
}
