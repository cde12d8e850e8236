// Ablation: the batched rerouting step built from one kernel per elementary tensor operation, the way a
// framework's stock operators would run it (the "SingleOp" variant of Section 5.3, Figure 7: broadcast the
// adapter ids, compute offsets into the expert map, gather), against which the fused operator (ew_reroute) and
// the routing fused into the router kernel are measured.  Three kernels with two materialised [n_tokens, k]
// intermediates, plus a histogram kernel when per-slot counts are asked for.  Same results as ew_reroute, bit for bit.
#include <string>

#include "ew_internal.h"

namespace ew {
namespace {

// 1. broadcast: aid_b[t, j] = adapter_ids[t]  (ids outside [-1, N) or of an unloaded adapter become -1, flagged)
__global__ void __launch_bounds__(256) broadcast_aid_kernel(const int32_t *__restrict__ aid, const int32_t *__restrict__ loaded,
                                                            long long n_pairs, int k, int N, int32_t *__restrict__ aid_b, int *err) {
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < n_pairs; q += (long long)gridDim.x * blockDim.x) {
        int a = aid[q / k];
        if (a < -1 || a >= N || (a >= 0 && !loaded[a])) { atomicOr(err, 1); a = -1; }
        aid_b[q] = a;
    }
}

// 2. offsets into the flattened map: off[t, j] = aid_b < 0 ? -1 : aid_b * M + id   (ids outside [0, M): -1, flagged)
__global__ void __launch_bounds__(256) map_offset_kernel(const int32_t *__restrict__ ids, const int32_t *__restrict__ aid_b,
                                                         long long n_pairs, int M, int32_t *__restrict__ off, int *err) {
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < n_pairs; q += (long long)gridDim.x * blockDim.x) {
        const int e = ids[q], a = aid_b[q];
        if ((unsigned)e >= (unsigned)M) { atomicOr(err, 4); off[q] = -1; continue; }
        off[q] = a < 0 ? -1 : a * M + e;
    }
}

// 3. gather: slots[t, j] = off < 0 ? id : Pi_flat[off]     (ids and slots may be the same buffer)
__global__ void __launch_bounds__(256) gather_map_kernel(const int32_t *ids, const int32_t *__restrict__ off,
                                                         const int32_t *__restrict__ pi, long long n_pairs, int32_t *slots) {
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < n_pairs; q += (long long)gridDim.x * blockDim.x) {
        const int o = off[q];
        slots[q] = o < 0 ? ids[q] : pi[o];
    }
}

// 4. per-slot counts (only when asked for)
__global__ void __launch_bounds__(256) slot_histogram_kernel(const int32_t *__restrict__ slots, long long n_pairs, int P,
                                                             int32_t *__restrict__ counts) {
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < n_pairs; q += (long long)gridDim.x * blockDim.x) {
        const int s = slots[q];
        if ((unsigned)s < (unsigned)P) atomicAdd(counts + s, 1);
    }
}

}  // namespace
}  // namespace ew

extern "C" ew_status_t ew_reroute_unfused(ew_pool_t *p, int32_t layer, const int32_t *topk_ids, const int32_t *adapter_ids,
                                          int32_t n_tokens, int32_t *slot_ids, int32_t *counts, int32_t *scratch,
                                          void *cuda_stream) {
    using namespace ew;
    if (!p || layer < 0 || layer >= p->cfg.num_layers || n_tokens < 0) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    DeviceGuard guard;
    cudaError_t e = guard.enter(p->cfg.device);
    if (e == cudaSuccess && counts) e = cudaMemsetAsync(counts, 0, (size_t)p->P * 4, st);
    if (e == cudaSuccess && n_tokens > 0) {
        if (!topk_ids || !adapter_ids || !slot_ids || !scratch) return EW_ERR_INVALID_ARG;
        const ew_config_t &c = p->cfg;
        const long long pairs = (long long)n_tokens * c.top_k;
        long long blocks = (pairs + 255) / 256;
        if (blocks > (long long)p->sm_count * 8) blocks = (long long)p->sm_count * 8;
        int32_t *aid_b = scratch, *off = scratch + pairs;
        broadcast_aid_kernel<<<(int)blocks, 256, 0, st>>>(adapter_ids, p->ws.loaded, pairs, c.top_k, c.max_adapters, aid_b, p->ws.err);
        map_offset_kernel<<<(int)blocks, 256, 0, st>>>(topk_ids, aid_b, pairs, c.num_experts, off, p->ws.err);
        gather_map_kernel<<<(int)blocks, 256, 0, st>>>(topk_ids, off, p->layers[layer].pi_dev, pairs, slot_ids);
        if (counts) slot_histogram_kernel<<<(int)blocks, 256, 0, st>>>(slot_ids, pairs, p->P, counts);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) {
        set_last_error(std::string("ew_reroute_unfused: ") + cudaGetErrorString(e));
        return EW_ERR_CUDA;
    }
    return EW_OK;
}
