// Routing-side kernels of the adapter-aware MoE layer:
//   reroute_kernel   the batched rerouting operator alone (Section 4.3) + histogram
//   permute_kernel   exclusive scan of the counts, the slot-contiguous order of the (token, expert) pairs as a
//                    row -> token table (GEMM-1 gathers the rows of x itself), and the work-item lists of the
//                    grouped GEMMs
//   combine_kernel   weighted un-permute and sum, one rounding to bf16 (Section 2.1)
#include <cuda_bf16.h>

#include "ew_internal.h"
#include "ew_plan.cuh"
#include "ew_tc.cuh"

namespace ew {
namespace {

// ------------------------------------------------------------------------------------------------
// Batched rerouting alone: slot = aid < 0 ? id : Pi[aid][id] (bad adapter ids behave as -1 and raise
// bit 0 of the error word).  A persistent CTA moves tiles of 256 tokens (256*k ids plus their 256
// adapter ids) through a four-stage shared-memory ring with bulk asynchronous copies in both
// directions (cp.async.bulk global->shared completing on an mbarrier, shared->global as bulk groups),
// so the data path costs a handful of instructions per tile and many tiles are in flight per SM; the
// threads only rewrite the ids in place, four at a time (the token of an id is a multiply-shift on
// its index inside the tile, exact for i < 8192 and k <= 32).  Expert map and loaded flags sit in
// shared memory; the per-CTA shared-memory histogram is flushed with one atomic per non-empty slot.
// Buffers that are not 16-byte aligned take reroute_kernel_unaligned (one thread per pair).
// ------------------------------------------------------------------------------------------------
constexpr int kRerouteTok = 256;
constexpr int kRerouteStages = 4;

__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void *gmem_src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_dst), "l"(gmem_src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void *gmem_dst, uint32_t smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gmem_dst), "r"(smem_src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }

// (ids and slots may be the same buffer - the rewrite in place the ABI allows - so neither is __restrict__)
//
// The per-slot counts are overwritten, not accumulated, and the call is one launch: CTA 0 zeroes the caller's
// counters and raises a flag in the pool's workspace; every CTA waits for that flag (bounded) before it adds its
// histogram; the CTA that finishes last lowers the flag again for the next call.  All CTAs of the grid are resident
// at once (one wave), so the wait cannot starve CTA 0.
__global__ void __launch_bounds__(256) reroute_kernel(const int32_t *ids, const int32_t *__restrict__ aid,
                                                      const int32_t *__restrict__ pi, const int32_t *__restrict__ loaded,
                                                      int n_tokens, int k, int M, int N, int P,
                                                      int32_t *slots, int32_t *__restrict__ counts, int *err, int *sync) {
    extern __shared__ __align__(128) int32_t smem_i[];
    const int tile_ints_max = kRerouteTok * k;
    const int stage_ints = kRerouteTok + tile_ints_max;            // a stage = 256 adapter ids, then 256*k ids (both 16-byte multiples)
    int32_t *stages = smem_i;
    int32_t *pi_s = stages + kRerouteStages * stage_ints, *hist = pi_s + N * M, *loaded_s = hist + P;
    uint64_t *bars = reinterpret_cast<uint64_t *>(((uintptr_t)(loaded_s + N) + 7) & ~(uintptr_t)7);
    __shared__ int abort_flag;
    for (int i = threadIdx.x; i < N * M; i += blockDim.x) pi_s[i] = pi[i];
    for (int i = threadIdx.x; i < N; i += blockDim.x) loaded_s[i] = loaded[i];
    if (counts) {
        for (int i = threadIdx.x; i < P; i += blockDim.x) hist[i] = 0;
        if (blockIdx.x == 0)
            for (int i = threadIdx.x; i < P; i += blockDim.x) counts[i] = 0;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < kRerouteStages; ++s) tc::mbar_init(tc::smem_u32(bars + s), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (counts && blockIdx.x == 0 && threadIdx.x == 0) {        // the counters are zero: publish
        __threadfence();
        atomicExch(sync, 1);
    }
    const unsigned div_magic = ((1u << 20) + k - 1) / k;
    const int n_tiles = (n_tokens + kRerouteTok - 1) / kRerouteTok;
    int flags = 0;
    // thread 0 starts the two bulk loads of tile tl into stage s; a tail shorter than 16 bytes is fetched with plain loads
    auto fetch = [&](int tl, int s) {
        const int n_tok = min(kRerouteTok, n_tokens - tl * kRerouteTok), n_int = n_tok * k;
        const uint32_t ab = (uint32_t)(n_tok & ~3) * 4, ib = (uint32_t)(n_int & ~3) * 4;
        const uint32_t bar = tc::smem_u32(bars + s);
        int32_t *st = stages + s * stage_ints;
        const int32_t *asrc = aid + (size_t)tl * kRerouteTok, *isrc = ids + (size_t)tl * tile_ints_max;
        for (int i = n_tok & ~3; i < n_tok; ++i) st[i] = asrc[i];              // before the arrive, which releases them
        for (int i = n_int & ~3; i < n_int; ++i) st[kRerouteTok + i] = isrc[i];
        tc::mbar_expect_tx(bar, ab + ib);
        if (ab) bulk_load(tc::smem_u32(st), asrc, ab, bar);
        if (ib) bulk_load(tc::smem_u32(st + kRerouteTok), isrc, ib, bar);
    };
    auto checked = [&](int a) -> int {                 // adapter ids outside [-1,N) or of unloaded adapters act as -1
        if (a < -1 || a >= N || (a >= 0 && !loaded_s[a])) { flags |= 1; a = -1; }
        return a;
    };
    auto map_one = [&](int e, int a) -> int {
        if ((unsigned)e >= (unsigned)M) { flags |= 4; return e; }
        const int sl = a < 0 ? e : pi_s[a * M + e];
        if (counts) atomicAdd(hist + sl, 1);
        return sl;
    };
    if (threadIdx.x == 0)
        for (int s = 0; s < kRerouteStages; ++s)
            if (blockIdx.x + s * (int)gridDim.x < n_tiles) fetch(blockIdx.x + s * gridDim.x, s);
    int it = 0;
    for (int tl = blockIdx.x; tl < n_tiles; tl += gridDim.x, ++it) {
        const int s = it % kRerouteStages;
        const uint32_t parity = (it / kRerouteStages) & 1;
        const int n_tok = min(kRerouteTok, n_tokens - tl * kRerouteTok), n_int = n_tok * k, n_vec = n_int >> 2;
        int32_t *aid_s = stages + s * stage_ints, *tile = aid_s + kRerouteTok;
        // one warp polls the barrier, the others sleep in the CTA barrier instead of spending issue slots on polling
        if (threadIdx.x < 32) tc::mbar_wait(tc::smem_u32(bars + s), parity, &abort_flag, err);
        __syncthreads();
        if (abort_flag) break;
        for (int v = threadIdx.x; v < n_vec; v += 256) {
            int4 r = reinterpret_cast<int4 *>(tile)[v];
            const int i0 = v << 2;
            int tok = (int)(((unsigned)i0 * div_magic) >> 20);
            int rem = i0 - tok * k;                    // position of the vector's first id inside its token's row
            int a = checked(aid_s[tok]);
            int *e = reinterpret_cast<int *>(&r);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (rem == k) { rem = 0; a = checked(aid_s[++tok]); }
                e[j] = map_one(e[j], a);
                ++rem;
            }
            reinterpret_cast<int4 *>(tile)[v] = r;
        }
        for (int i = (n_vec << 2) + threadIdx.x; i < n_int; i += 256)       // last tile when its length is not a multiple of 4
            tile[i] = map_one(tile[i], checked(aid_s[((unsigned)i * div_magic) >> 20]));
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");          // generic-proxy writes -> visible to the bulk store
        __syncthreads();
        if (threadIdx.x == 0) {
            int32_t *dst = slots + (size_t)tl * tile_ints_max;
            const uint32_t ib = (uint32_t)(n_int & ~3) * 4;
            if (ib) bulk_store(dst, tc::smem_u32(tile), ib);
            bulk_commit();
            for (int i = n_int & ~3; i < n_int; ++i) dst[i] = tile[i];
            // the stage used one tile ago has been read out by its store by now: refill it
            if (it >= 1) {
                bulk_wait_read<1>();
                const int nxt = tl + (kRerouteStages - 1) * (int)gridDim.x;
                if (nxt < n_tiles) fetch(nxt, (it - 1) % kRerouteStages);
            }
        }
    }
    if (threadIdx.x == 0) bulk_wait_read<0>();
    if (flags) atomicOr(err, flags);
    if (counts) {
        if (threadIdx.x == 0) {                                  // wait (bounded) until CTA 0 has zeroed the counters
            long long t0 = clock64();
            while (atomicAdd(sync, 0) == 0) {
                if (clock64() - t0 > tc::kWaitLimitCycles) { atomicOr(err, 2); abort_flag = 1; break; }
                __nanosleep(64);
            }
            __threadfence();
        }
        __syncthreads();
        if (!abort_flag)
            for (int i = threadIdx.x; i < P; i += blockDim.x)
                if (hist[i]) atomicAdd(counts + i, hist[i]);
        __syncthreads();
        if (threadIdx.x == 0) {                                  // last CTA out lowers the flag for the next call
            __threadfence();
            if (atomicAdd(sync + 1, 1) == (int)gridDim.x - 1) {
                atomicExch(sync + 1, 0);
                atomicExch(sync, 0);
            }
        }
    }
}

// any alignment: one thread per (token, expert) pair
__global__ void __launch_bounds__(256) reroute_kernel_unaligned(const int32_t *ids, const int32_t *__restrict__ aid,
                                                                const int32_t *__restrict__ pi, const int32_t *__restrict__ loaded,
                                                                long long n_pairs, int k, int M, int N,
                                                                int32_t *slots, int32_t *__restrict__ counts, int *err) {
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < n_pairs; q += (long long)gridDim.x * blockDim.x) {
        int a = aid[q / k];
        if (a < -1 || a >= N || (a >= 0 && !loaded[a])) { atomicOr(err, 1); a = -1; }
        const int e = ids[q];
        if ((unsigned)e >= (unsigned)M) { atomicOr(err, 4); slots[q] = e; continue; }
        const int sl = a < 0 ? e : pi[a * M + e];
        slots[q] = sl;
        if (counts) atomicAdd(counts + sl, 1);
    }
}

// ------------------------------------------------------------------------------------------------
// Gate + rerouting from given logits (the stand-alone operator fused with the gate function it follows,
// Sections 2.1 and 4.3): softmax over the M logits of each token, k largest probabilities (lower index on ties),
// slot = Pi[aid][id], per-slot counts.  A CTA owns 128 tokens; the threads copy their logits [128, M] fp32 into
// shared memory with coalesced 16-byte loads, rows M + 1 words apart so that the per-token reads that follow spread
// over the banks.  Four neighbouring lanes of a warp share a token, lane g of the four owning the experts
// [EPT*g, EPT*g + EPT) in registers (EPT = 64: this kernel serves M > 64; smaller M takes the sorted kernel below).  Softmax by partial max and partial sum,
// exchanged with two butterfly shuffles; then k rounds in which every lane offers its best remaining candidate and
// the four settle the token's best the same way - no block-wide barrier after the tile has landed.  Counts go
// through a shared-memory histogram, one atomic per non-empty slot and CTA.
// ------------------------------------------------------------------------------------------------
constexpr int kLogitTok = 128;

template <int EPT>
__global__ void __launch_bounds__(4 * kLogitTok) route_logits_kernel(const float4 *__restrict__ logits, const int32_t *__restrict__ aid,
                                                                     const int32_t *__restrict__ pi, const int32_t *__restrict__ loaded,
                                                                     int B, int M, int k, int N, int P, int renormalize, float scale,
                                                                     int32_t *topk_ids, float *topk_w, int32_t *slot_ids,
                                                                     int32_t *counts, int *err) {
    extern __shared__ __align__(16) uint8_t rl_smem[];
    const int ld = M + 1;                                                   // row stride of the tile, in words
    float *tile = reinterpret_cast<float *>(rl_smem);                       // [128][M + 1]
    int32_t *hist_s = reinterpret_cast<int32_t *>(tile + (size_t)kLogitTok * ld);   // [P]
    int32_t *pi_s = hist_s + P;                                             // [N][M]

    const int tid = threadIdx.x, lane = tid & 31;
    const int tl = (tid >> 5) * 8 + (lane >> 2), g = lane & 3;              // token inside the tile, expert group
    const int tok0 = blockIdx.x * kLogitTok;
    const int rows = min(kLogitTok, B - tok0);
    const int t = tok0 + tl;
    {
        const int mv = M >> 2;                                               // float4 per row
        const float4 *src = logits + (size_t)tok0 * mv;
        // (row, column) of this thread's float4 and of the one blockDim further: one division here, additions below
        int row = tid / mv, col = tid - row * mv;
        const int drow = (int)blockDim.x / mv, dcol = (int)blockDim.x - drow * mv;
        for (int v0 = tid; v0 < rows * mv; v0 += 4 * (int)blockDim.x) {      // four loads in flight per thread
            float4 r[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (v0 + u * (int)blockDim.x < rows * mv) r[u] = src[v0 + u * blockDim.x];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (v0 + u * (int)blockDim.x < rows * mv) {
                    float *d = tile + (size_t)row * ld + 4 * col;
                    d[0] = r[u].x; d[1] = r[u].y; d[2] = r[u].z; d[3] = r[u].w;
                }
                row += drow;
                col += dcol;
                if (col >= mv) { col -= mv; ++row; }
            }
        }
    }
    for (int i = tid; i < P; i += blockDim.x) hist_s[i] = 0;
    for (int i = tid; i < N * M; i += blockDim.x) pi_s[i] = pi[i];
    __syncthreads();

    constexpr unsigned kFull = 0xffffffffu;
    const bool live = tl < rows;
    float p[EPT];                                                            // register i: expert EPT*g + i
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
        const int j = EPT * g + i;
        p[i] = (live && j < M) ? tile[(size_t)tl * ld + j] : -INFINITY;
        mx = fmaxf(mx, p[i]);
    }
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 2));
    if (!live) mx = 0.f;
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < EPT; ++i) {                                          // exp(-inf) = 0 for the absent experts
        p[i] = expf(p[i] - mx);
        sum += p[i];
    }
    sum += __shfl_xor_sync(kFull, sum, 1);                                   // (s0 + s1) + (s2 + s3) on all four lanes
    sum += __shfl_xor_sync(kFull, sum, 2);
    const float inv_sum = live ? 1.f / sum : 0.f;
#pragma unroll
    for (int i = 0; i < EPT; ++i) p[i] = EPT * g + i < M ? p[i] * inv_sum : -1.f;
    int a = -1;
    if (live) {
        a = aid[t];
        if (a < -1 || a >= N || (a >= 0 && !loaded[a])) {
            atomicOr(err, 1);
            a = -1;
        }
    }
    float wsum = 0.f;
    float my_w[8];                                                           // weights of the pairs this lane writes (r = g, g+4, ...)
    for (int r = 0; r < k; ++r) {
        // arg-max as a tree over neighbouring ranges (short dependency chains); the right half wins only if
        // strictly greater, so the lower index keeps a tie
        float tv[EPT / 2];
        int ti[EPT / 2];
#pragma unroll
        for (int i = 0; i < EPT / 2; ++i) {
            const bool gt = p[2 * i + 1] > p[2 * i];
            tv[i] = gt ? p[2 * i + 1] : p[2 * i];
            ti[i] = gt ? 2 * i + 1 : 2 * i;
        }
#pragma unroll
        for (int w = EPT / 4; w >= 1; w >>= 1) {
#pragma unroll
            for (int i = 0; i < w; ++i) {
                const bool gt = tv[2 * i + 1] > tv[2 * i];
                tv[i] = gt ? tv[2 * i + 1] : tv[2 * i];
                ti[i] = gt ? ti[2 * i + 1] : ti[2 * i];
            }
        }
        const float bv = tv[0];
        const int bi = ti[0];
        float wv = bv;
        int wi = EPT * g + bi;
#pragma unroll
        for (int o = 1; o <= 2; o <<= 1) {                                   // the four lanes agree on the token's best
            const float ov = __shfl_xor_sync(kFull, wv, o);
            const int oi = __shfl_xor_sync(kFull, wi, o);
            const bool better = ov > wv || (ov == wv && oi < wi);
            wv = better ? ov : wv;
            wi = better ? oi : wi;
        }
        if (wi == EPT * g + bi) {                                            // mine: taken (probabilities are >= 0)
#pragma unroll
            for (int i = 0; i < EPT; ++i) p[i] = (i == bi) ? -1.f : p[i];
        }
        wsum += wv;
        if ((r & 3) == g && live) {                                          // the four lanes share the output work
            const int slot = a < 0 ? wi : pi_s[a * M + wi];
            const size_t o = (size_t)t * k + r;
            topk_ids[o] = wi;
            slot_ids[o] = slot;
            atomicAdd(hist_s + slot, 1);
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (u == (r >> 2)) my_w[u] = wv;
        }
    }
    if (live) {
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (g + 4 * u < k) {
                float w = my_w[u];
                if (renormalize) w = w / wsum;
                topk_w[(size_t)t * k + g + 4 * u] = (renormalize || scale != 1.f) ? w * scale : w;
            }
    }
    __syncthreads();
    for (int i = tid; i < P; i += blockDim.x)
        if (hist_s[i]) atomicAdd(counts + i, hist_s[i]);
}

// ------------------------------------------------------------------------------------------------
// The same operator for M <= 64 with about a third of the warp instructions per token (the kernel above spends most
// of its issue slots on k arg-max-with-removal passes over register arrays).  Four lanes share a token, lane g owning
// the sixteen experts [16g, 16g + 16): it loads them straight from global memory, exponentiates, and sorts its sixteen
// probabilities ONCE with a 63-comparator network of max/min pairs (values only).  A selection round is then a
// butterfly max over the four lanes' current heads, a ballot to find the lowest lane that holds the maximum (lower
// lane = lower expert index: the tie rule between lanes) and a pop of that lane's head; the lane notes the round in a
// bit mask.  After the k rounds a lane's wins are the first entries of its sorted list, in round order; only then
// does it look their indices up among its sixteen originals (lowest index not taken yet: the tie rule inside a lane)
// and write ids, weights and slots.  A warp serves eight tokens at a time, a CTA 256 tokens in four passes, so the
// expert map and the histogram are staged once per 256 tokens.  DEEP: k > 8, a lane may win up to sixteen rounds.
// ------------------------------------------------------------------------------------------------
constexpr int kLogitTok4 = 256;      // tokens per CTA: 64 groups of four lanes, four passes

template <bool DEEP>
__global__ void __launch_bounds__(256) route_logits4_kernel(const float4 *__restrict__ logits, const int32_t *__restrict__ aid,
                                                            const int32_t *__restrict__ pi, const int32_t *__restrict__ loaded,
                                                            int B, int M, int k, int N, int P, int renormalize, float scale,
                                                            int32_t *topk_ids, float *topk_w, int32_t *slot_ids,
                                                            int32_t *counts, int *err) {
    extern __shared__ __align__(16) int32_t rl4_smem[];
    int32_t *hist_s = rl4_smem;              // [P]
    int32_t *pi_s = hist_s + P;              // [N][M]
    constexpr unsigned kFull = 0xffffffffu;
    constexpr int kDepth = DEEP ? 16 : 8;    // entries of the sorted list that can still be popped
    const int tid = threadIdx.x, lane = tid & 31, g = lane & 3;
    const unsigned group_shift = lane & 28;  // first lane of this token's four within the warp
    const int mv = M >> 2;

    for (int i = tid; i < P; i += blockDim.x) hist_s[i] = 0;
    for (int i = tid; i < N * M; i += blockDim.x) pi_s[i] = pi[i];
    __syncthreads();

#pragma unroll 1
    for (int ps = 0; ps < kLogitTok4 / 64; ++ps) {
        const int t = blockIdx.x * kLogitTok4 + ps * 64 + (tid >> 2);
        if (blockIdx.x * kLogitTok4 + ps * 64 >= B) break;            // nothing left for the whole CTA
        const bool live = t < B;
        float e[16];
        {
            const float4 *row = logits + (size_t)t * mv;
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                float4 r = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
                if (live && 4 * g + h < mv) r = __ldg(row + 4 * g + h);
                e[4 * h] = r.x; e[4 * h + 1] = r.y; e[4 * h + 2] = r.z; e[4 * h + 3] = r.w;
            }
        }
        int a = live ? __ldg(aid + t) : -1;
        if (a < -1 || a >= N || (a >= 0 && !loaded[a])) {
            if (g == 0) atomicOr(err, 1);
            a = -1;
        }
        float mx = e[0];
#pragma unroll
        for (int i = 1; i < 16; ++i) mx = fmaxf(mx, e[i]);
        mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 2));
        if (!live) mx = 0.f;
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < 16; ++i) {                    // exp(-inf) = 0 for the absent experts
            e[i] = __expf(e[i] - mx);                     // ex2.approx: relative error about 5e-7 for the arguments that matter
            sum += e[i];
        }
        sum += __shfl_xor_sync(kFull, sum, 1);
        sum += __shfl_xor_sync(kFull, sum, 2);
        const float inv_sum = 1.f / sum;
#pragma unroll
        for (int i = 0; i < 16; ++i) e[i] = 16 * g + i < M ? e[i] * inv_sum : -1.f;   // absent experts below every real one

        float s0[16];                                    // the lane's probabilities sorted descending
#pragma unroll
        for (int i = 0; i < 16; ++i) s0[i] = e[i];
#define EW_CE(x, y) { const float hi_ = fmaxf(s0[x], s0[y]), lo_ = fminf(s0[x], s0[y]); s0[x] = hi_; s0[y] = lo_; }
        EW_CE(0, 1) EW_CE(2, 3) EW_CE(0, 2) EW_CE(1, 3) EW_CE(1, 2) EW_CE(4, 5) EW_CE(6, 7) EW_CE(4, 6) EW_CE(5, 7)
        EW_CE(5, 6) EW_CE(0, 4) EW_CE(2, 6) EW_CE(2, 4) EW_CE(1, 5) EW_CE(3, 7) EW_CE(3, 5) EW_CE(1, 2) EW_CE(3, 4)
        EW_CE(5, 6) EW_CE(8, 9) EW_CE(10, 11) EW_CE(8, 10) EW_CE(9, 11) EW_CE(9, 10) EW_CE(12, 13) EW_CE(14, 15)
        EW_CE(12, 14) EW_CE(13, 15) EW_CE(13, 14) EW_CE(8, 12) EW_CE(10, 14) EW_CE(10, 12) EW_CE(9, 13) EW_CE(11, 15)
        EW_CE(11, 13) EW_CE(9, 10) EW_CE(11, 12) EW_CE(13, 14) EW_CE(0, 8) EW_CE(4, 12) EW_CE(4, 8) EW_CE(2, 10)
        EW_CE(6, 14) EW_CE(6, 10) EW_CE(2, 4) EW_CE(6, 8) EW_CE(10, 12) EW_CE(1, 9) EW_CE(5, 13) EW_CE(5, 9)
        EW_CE(3, 11) EW_CE(7, 15) EW_CE(7, 11) EW_CE(3, 5) EW_CE(7, 9) EW_CE(11, 13) EW_CE(1, 2) EW_CE(3, 4)
        EW_CE(5, 6) EW_CE(7, 8) EW_CE(9, 10) EW_CE(11, 12) EW_CE(13, 14)
#undef EW_CE
        float s[kDepth];                                 // the part of it that is popped during the rounds
#pragma unroll
        for (int i = 0; i < kDepth; ++i) s[i] = s0[i];

        unsigned won = 0;                                // bit r: this lane's head won round r
        float wsum = 0.f;
        for (int r = 0; r < k; ++r) {
            float wv = s[0];
            wv = fmaxf(wv, __shfl_xor_sync(kFull, wv, 1));
            wv = fmaxf(wv, __shfl_xor_sync(kFull, wv, 2));
            const unsigned holders = (__ballot_sync(kFull, s[0] == wv) >> group_shift) & 0xfu;
            wsum += wv;
            if (g == __ffs(holders) - 1) {               // the lowest lane that holds it pops its head
                won |= 1u << r;
#pragma unroll
                for (int i = 0; i < kDepth - 1; ++i) s[i] = s[i + 1];
                s[kDepth - 1] = -2.f;
            }
        }
        // this lane's wins, in round order, are s0[0], s0[1], ...
        unsigned taken = 0;
        const float wnorm = renormalize ? scale / wsum : scale;
#pragma unroll
        for (int j = 0; j < kDepth; ++j) {
            if (__any_sync(kFull, won != 0)) {
                if (won) {
                    const int r = __ffs(won) - 1;
                    won &= won - 1;
                    const float wv = s0[j];
                    unsigned eq = 0;
#pragma unroll
                    for (int i = 0; i < 16; ++i) eq |= (e[i] == wv) ? (1u << i) : 0u;
                    const int idx = __ffs(eq & ~taken) - 1;   // lowest index with that value not taken yet
                    taken |= 1u << idx;
                    if (live) {
                        const int id = 16 * g + idx;
                        const int slot = a < 0 ? id : pi_s[a * M + id];
                        const size_t o = (size_t)t * k + r;
                        topk_ids[o] = id;
                        slot_ids[o] = slot;
                        topk_w[o] = (renormalize || scale != 1.f) ? wv * wnorm : wv;
                        atomicAdd(hist_s + slot, 1);
                    }
                }
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < P; i += blockDim.x)
        if (hist_s[i]) atomicAdd(counts + i, hist_s[i]);
}

// ------------------------------------------------------------------------------------------------
// Scan + permute + plan.  Every CTA recomputes the exclusive scan of the (small) count array in
// shared memory; the first kPlanners CTAs publish the offsets and write the GEMM work items (the item
// loop is a chain of dependent integer arithmetic, so it is spread over several CTAs), the other CTAs record for
// each (token, expert) pair its slot-contiguous row (inv) and for each row its token (src_tok), one thread per
// pair.  No copy of x is made: GEMM-1 gathers its token rows through src_tok.
// ------------------------------------------------------------------------------------------------
constexpr int kPlanners = 8;

__global__ void __launch_bounds__(256) permute_kernel(const int32_t *slot_ids, const int32_t *rank, const int32_t *counts,
                                                      plan::Params A, int32_t *inv, int32_t *src_tok) {
    extern __shared__ int32_t sm[];
    __shared__ int32_t warp_sums[8];
    tc::pdl_launch_dependents();
    // counts, slot ids and ranks come from the router kernel: none of the kernel's pointer parameters is
    // __restrict__, so that no load can be hoisted above this wait
    tc::pdl_wait();
    const int32_t *cnt_s = plan::stage_and_scan(sm, counts, A.P, A.S, warp_sums, 256);
    const int32_t *off = sm;                 // [P + 1]
    const int warp = threadIdx.x >> 5;
    const long long n_pairs = (long long)A.B * A.k;
    if (blockIdx.x >= kPlanners) {           // the first CTAs (dispatched first) are the planners
        // one thread per (token, j) pair records the pair's row and the row's token
        const long long q = (long long)(blockIdx.x - kPlanners) * 256 + threadIdx.x;
        if (q < n_pairs) {
            const int rk = rank[q];
            const int dest = rk < 0 ? -1 : off[slot_ids[q]] + rk;    // position -1: the pair belongs to another rank (expert parallelism)
            if (dest < 0) {
                inv[q] = -1;
            } else if (dest < n_pairs) {     // always, unless the routing kernel gave up midway (error word set)
                inv[q] = dest;
                src_tok[dest] = (int32_t)(q / A.k);
            }
        }
        return;
    }
    // ---- planner CTAs: each has repeated the (cheap) scan and writes the items of every kPlanners-th group
    plan::write_items(sm, cnt_s, A, warp_sums, 256, warp + 8 * blockIdx.x, 8 * kPlanners, blockIdx.x == 0);
}

// ------------------------------------------------------------------------------------------------
// out[t] = sum_j w[t,j] * Y[Yb + inv[t,j]] + Y[t], fp32, j in router order, one rounding.  Rows [0, B) of Y hold the
// sum of the shared experts' outputs (GEMM-2 chains them along K); the routed rows start at Yb = B (0 without shared
// experts).
// ------------------------------------------------------------------------------------------------
// OUT = 0: rounded bf16 result.  1: this rank's fp32 partial sums (expert parallelism, added by an all-reduce).
// 2: the same partial sums stored straight into every rank's gather buffer - `out` is a device array of ep_size
// pointers, buffer r' = rank r''s [ep_size][B][H] fp32 area, of which this rank fills block ep_rank: the exchange step
// of the layer done by the kernel that produces the data, with plain (peer) stores.
template <int OUT>
__global__ void __launch_bounds__(256) combine_kernel(const float4 *y, const int32_t *inv,
                                                      const float *w, int B, int k, int H, int S,
                                                      void *out, int32_t *counts, int P, int ep_size, int ep_rank) {
    __shared__ int32_t rows[32];
    __shared__ float wts[32];
    const int t = blockIdx.x;
    tc::pdl_launch_dependents();
    tc::pdl_wait();                                     // expert outputs come from GEMM-2
    if (t == 0)                                         // the slot counters are spent: leave them zero for the next forward
        for (int i = threadIdx.x; i < P; i += blockDim.x) counts[i] = 0;
    const int y_base = S > 0 ? B : 0;
    if (threadIdx.x < k) {
        const int r = inv[(size_t)t * k + threadIdx.x];
        rows[threadIdx.x] = r < 0 ? -1 : y_base + r;    // -1: the pair's expert lives on another rank (expert parallelism)
        wts[threadIdx.x] = w[(size_t)t * k + threadIdx.x];
    }
    __syncthreads();
    const int hv = H >> 2;
    for (int v = threadIdx.x; v < hv; v += blockDim.x) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j = 0; j < k; ++j) {
            if (rows[j] < 0) continue;
            const float4 a = y[(size_t)rows[j] * hv + v];
            const float wj = wts[j];
            acc.x = fmaf(wj, a.x, acc.x); acc.y = fmaf(wj, a.y, acc.y);
            acc.z = fmaf(wj, a.z, acc.z); acc.w = fmaf(wj, a.w, acc.w);
        }
        if (S > 0) {
            const float4 a = y[(size_t)t * hv + v];
            acc.x += a.x; acc.y += a.y; acc.z += a.z; acc.w += a.w;
        }
        if (OUT == 2) {
            float4 *const *dst = reinterpret_cast<float4 *const *>(out);
            const size_t o = ((size_t)ep_rank * B + t) * hv + v;
            for (int r = 0; r < ep_size; ++r) dst[r][o] = acc;
        } else if (OUT == 1) {                          // this rank's partial sum, rounded after the sum over ranks
            reinterpret_cast<float4 *>(out)[(size_t)t * hv + v] = acc;
        } else {
            const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
            uint2 o;
            o.x = *reinterpret_cast<const uint32_t *>(&lo);
            o.y = *reinterpret_cast<const uint32_t *>(&hi);
            reinterpret_cast<uint2 *>(out)[(size_t)t * hv + v] = o;
        }
    }
}

// out[i] = bf16(in[0][i] + in[1][i] + ... + in[R-1][i]), added in that order (R = 1: the single rounding of a sum
// that an all-reduce has already formed; R > 1: the gathered partial sums of all ranks, the same bits on every rank
// and in every run)
__global__ void __launch_bounds__(256) round_bf16_kernel(const float4 *in, uint2 *out, size_t n4, int R) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        float4 a = in[i];
        for (int r = 1; r < R; ++r) {
            const float4 b = in[(size_t)r * n4 + i];
            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        }
        const __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
        uint2 o;
        o.x = *reinterpret_cast<const uint32_t *>(&lo);
        o.y = *reinterpret_cast<const uint32_t *>(&hi);
        out[i] = o;
    }
}

}  // namespace

// Token rows per GEMM work item: the smallest tile that holds ~1.5x the mean rows per routed expert.  256 means
// "prefill-sized": blocks of more than 128 rows become fat items of the CTA-pair kernel.
int pick_token_tile(const ew_pool *p, int B) {
    const double mean = (double)B * p->cfg.top_k / p->cfg.num_experts;
    const double want = mean * 1.5;
    return want <= 32 ? 32 : want <= 64 ? 64 : want <= 192 ? 128 : 256;
}

int launch_permute(ew_pool *p, int B, cudaStream_t st) {
    const ew_config_t &c = p->cfg;
    plan::Params A;
    A.B = B; A.k = c.top_k; A.P = p->P; A.S = p->sh_hi - p->sh_lo; A.sh0 = p->sh_lo;
    A.NT = p->token_tile; A.fat = p->fat ? 1 : 0;
    A.R1 = (c.inter + 127) / 128; A.R2 = (c.hidden + 127) / 128;
    A.RF1 = (c.inter + 127) / 128; A.RF2 = (c.hidden + 255) / 256;
    A.offsets = p->ws.offsets; A.items1 = p->ws.items1; A.items2 = p->ws.items2; A.fat1 = p->ws.fat1; A.fat2 = p->ws.fat2;
    A.n_items = p->ws.n_items;
    const long long pairs = (long long)B * c.top_k;
    const int grid = (int)((pairs + 255) / 256) + kPlanners;
    const size_t smem = plan::smem_words(p->P, A.S) * 4;
    return launch_pdl(permute_kernel, dim3(grid), dim3(256), smem, st, (const int32_t *)p->ws.slot_ids, (const int32_t *)p->ws.rank,
                      (const int32_t *)p->ws.counts, A, p->ws.inv, p->ws.src_tok);
}

int launch_combine(ew_pool *p, int B, void *out, int out_mode, cudaStream_t st) {
    const ew_config_t &c = p->cfg;
    const int S = p->sh_hi - p->sh_lo;                  // the shared experts this rank computes
    const int R = c.ep_size > 1 ? c.ep_size : 1;
    auto go = [&](auto kernel) {
        return launch_pdl(kernel, dim3(B), dim3(256), 0, st, (const float4 *)p->ws.y, p->ws.inv, p->ws.topk_w, B, c.top_k,
                          c.hidden, S, out, p->ws.counts, p->P, R, c.ep_rank);
    };
    return out_mode == 2 ? go(combine_kernel<2>) : out_mode == 1 ? go(combine_kernel<1>) : go(combine_kernel<0>);
}

int launch_round_bf16(const float *in, int n_parts, void *out, size_t n, cudaStream_t st) {
    const size_t n4 = n / 4;
    const int grid = (int)std::min<size_t>((n4 + 255) / 256, 148 * 8);
    round_bf16_kernel<<<grid, 256, 0, st>>>((const float4 *)in, (uint2 *)out, n4, n_parts);
    return (int)cudaGetLastError();
}

int launch_route_logits(ew_pool *p, int layer, const float *logits, const int32_t *aid, int B, int32_t *topk_ids,
                        float *topk_w, int32_t *slot_ids, int32_t *counts, cudaStream_t st) {
    const ew_config_t &c = p->cfg;
    const int M = c.num_experts, N = c.max_adapters;
    const size_t smem = ((size_t)kLogitTok * (M + 1) + p->P + (size_t)N * M) * 4;      // the M > 64 kernel: tile + histogram + map
    const int grid = (B + kLogitTok - 1) / kLogitTok;
    const int32_t *pi = p->layers[layer].pi_dev;
    cudaError_t e;
    const size_t smem4 = ((size_t)p->P + (size_t)N * M) * 4;
    if (M <= 64) {
        if (smem4 > 200 * 1024) return (int)cudaErrorInvalidConfiguration;   // expert map + histogram beyond shared memory
        const int grid4 = (B + kLogitTok4 - 1) / kLogitTok4;
        if (c.top_k > 8) {
            e = cudaFuncSetAttribute(route_logits4_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem4);
            if (e != cudaSuccess) return (int)e;
            route_logits4_kernel<true><<<grid4, 256, smem4, st>>>((const float4 *)logits, aid, pi, p->ws.loaded, B, M, c.top_k, N, p->P,
                                                                  c.renormalize, c.routed_scale, topk_ids, topk_w, slot_ids, counts, p->ws.err);
        } else {
            e = cudaFuncSetAttribute(route_logits4_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem4);
            if (e != cudaSuccess) return (int)e;
            route_logits4_kernel<false><<<grid4, 256, smem4, st>>>((const float4 *)logits, aid, pi, p->ws.loaded, B, M, c.top_k, N, p->P,
                                                                   c.renormalize, c.routed_scale, topk_ids, topk_w, slot_ids, counts, p->ws.err);
        }
    } else {
        if (smem > 227 * 1024) return (int)cudaErrorInvalidConfiguration;
        e = cudaFuncSetAttribute(route_logits_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return (int)e;
        route_logits_kernel<64><<<grid, 4 * kLogitTok, smem, st>>>((const float4 *)logits, aid, pi, p->ws.loaded, B, M, c.top_k, N, p->P, c.renormalize,
                                                                   c.routed_scale, topk_ids, topk_w, slot_ids, counts, p->ws.err);
    }
    return (int)cudaGetLastError();
}

int launch_reroute(ew_pool *p, int layer, const int32_t *ids, const int32_t *aid, int B, int32_t *slots,
                   int32_t *counts, cudaStream_t st) {
    const ew_config_t &c = p->cfg;
    const int32_t *pi = p->layers[layer].pi_dev;
    if ((((uintptr_t)ids | (uintptr_t)slots | (uintptr_t)aid) & 15) != 0) {
        const long long pairs = (long long)B * c.top_k;
        long long blocks = (pairs + 255) / 256;
        if (blocks > (long long)p->sm_count * 8) blocks = (long long)p->sm_count * 8;
        reroute_kernel_unaligned<<<(int)blocks, 256, 0, st>>>(ids, aid, pi, p->ws.loaded, pairs, c.top_k, c.num_experts,
                                                              c.max_adapters, slots, counts, p->ws.err);
        return (int)cudaGetLastError();
    }
    long long blocks = ((long long)B + kRerouteTok - 1) / kRerouteTok;
    const size_t smem = ((size_t)kRerouteStages * kRerouteTok * (c.top_k + 1) + (size_t)c.max_adapters * c.num_experts + p->P +
                         c.max_adapters) * 4 + 8 * kRerouteStages + 32;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(reroute_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return (int)e;
    }
    // exactly one wave: every CTA is resident and walks its share of the tiles
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, reroute_kernel, 256, smem) != cudaSuccess || per_sm < 1) per_sm = 1;
    const long long cap = (long long)p->sm_count * per_sm;
    if (blocks > cap) blocks = cap;
    reroute_kernel<<<(int)blocks, 256, smem, st>>>(ids, aid, pi, p->ws.loaded, B, c.top_k, c.num_experts, c.max_adapters,
                                                   p->P, slots, counts, p->ws.err, p->ws.err + 8);
    return (int)cudaGetLastError();
}

}  // namespace ew
