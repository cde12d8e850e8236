// Fused router kernel: logits on the tensor cores, then softmax + top-k + batched rerouting +
// per-slot histogram in the epilogue (Sections 2.1 and 4.3).
//
// One CTA owns `tok_tile` (32, 64 or 128) tokens.  The logits tile D[128, M] = X[128, H] * Wr[M, H]^T is
// one tcgen05 accumulator (M <= 256 fp32 columns of TMEM); X and the router rows stream through a TMA
// ring.  The kernel is latency-bound, so each TMA instruction fetches up to four 64-element K-atoms at once
// (3-D descriptors ordered element, row, atom: shared memory receives one swizzled tile per atom).  Only the first
// `tok_tile` rows of the 128-row MMA tile are loaded; the other rows hold whatever shared memory held
// and feed accumulator lanes nobody reads.  TMEM lane i belongs to token i.  With 32-token tiles (small
// batches) one warp spills the logits to shared memory and four adjacent lanes share each token's softmax and
// top-k (quad_epilogue); with larger tiles every epilogue
// thread owns one token: it reads its M logits from TMEM, forms the softmax probabilities in fp32, takes
// k arg-max rounds (probability descending, lower index on ties), looks each chosen expert up in the
// layer's expert map Pi (staged in shared memory) under the token's adapter id, and bumps the slot's
// counter; the atomic's return value is the pair's position inside the slot's chunk.
//
// Small batches (32-token tiles that leave most SMs idle) split K over a cluster: the 4 or 8 CTAs of a cluster own one
// token tile and a quarter or an eighth of the K range each, so the chain of dependent load rounds is one or two stages
// long instead of eight; every CTA sends its partial logits to the cluster's first CTA through distributed shared
// memory, and that CTA adds them in rank order (the sum does not depend on timing) and runs the epilogue.
#include <cstdlib>
#include <mutex>
#include <string>

#include "ew_internal.h"
#include "ew_tc.cuh"

namespace ew {
namespace {
using namespace tc;

constexpr int kThreads = 192;
constexpr int kThreadsBig = 320;     // large tiles: eight epilogue warps, so that 64 tokens are selected in one pass
constexpr int kTileRows = 128;
constexpr int kMaxStages = 16;
constexpr int kMaxAtoms = 4;         // 64-element K-atoms per TMA box and pipeline stage: 4, 2 or 1
constexpr int kMaxPiSmem = 16 * 1024;

__device__ __forceinline__ int checked_aid(int a, int N, const int32_t *loaded, int *err) {
    if (a < -1 || a >= N || (a >= 0 && !loaded[a])) {
        atomicOr(err, 1);
        return -1;
    }
    return a;
}

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
// store into the same shared-memory offset of the cluster's CTA 0
__device__ __forceinline__ void st_leader_f32(const float *local_ptr, float v) {
    asm volatile(
        "{\n\t.reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %0, 0;\n\t"
        "st.shared::cluster.f32 [ra], %1;\n\t}"
        ::"r"(smem_u32(local_ptr)), "f"(v) : "memory");
}

struct RouterArgs {
    const int32_t *aid, *pi, *loaded;
    int B, H, M, k, N, renormalize;
    float scale;
    int stages, tmem_cols, pi_in_smem, tok_tile, atoms;
    int hold_dependents = 0;   // do not release the next kernel in the stream before this one has finished
    int big_quad;          // 64- and 128-token tiles: four lanes per token and a histogram per CTA (needs room in the drained ring)
    int P;                 // slots of the pool (size of the counters)
    int ksplit;            // CTAs per cluster that share one token tile, each with 1/ksplit of K (1: no cluster)
    int part_off;          // byte offset of the partial-logit buffer [ksplit][n_mma][32] floats in shared memory
    int32_t *topk_ids;
    float *topk_w;
    int32_t *slot_ids, *rank, *counts;
    int *err;
    int own_lo = 0, own_hi = 1 << 30;   // expert parallelism: pairs whose base expert lies outside [own_lo, own_hi) belong to another rank:
                                        // ids, weights and slot ids are written as usual, but they are not counted and get position -1
    int32_t *slot_tok = nullptr;   // [P][B] or null.  Forwards without a planning kernel: the token of the pair at position r of slot s
};

// write one selected pair: reroute through Pi, outputs (the histogram follows in emit_ranks)
__device__ __forceinline__ void emit_pair(const RouterArgs &A, const int32_t *pi_s, int t, int r, int a, int id, float w,
                                          int (&sl)[8], uint32_t &local_mask) {
    if (id >= A.own_lo && id < A.own_hi) local_mask |= 1u << r;
    const int slot = a < 0 ? id : (A.pi_in_smem ? pi_s[a * A.M + id] : __ldg(A.pi + a * A.M + id));
    const size_t o = (size_t)t * A.k + r;
    A.topk_ids[o] = id;
    A.topk_w[o] = w;
    A.slot_ids[o] = slot;
#pragma unroll
    for (int u = 0; u < 8; ++u)
        if (u == r) sl[u] = slot;       // the first eight slots stay in registers for emit_ranks
}

// per-slot histogram: one atomic per pair, eight in flight per thread; the value returned is the
// pair's position inside its slot's chunk
__device__ __forceinline__ void emit_ranks(const RouterArgs &A, int t, const int (&sl)[8], uint32_t local_mask) {
    for (int r0 = 0; r0 < A.k; r0 += 8) {
        int got[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (r0 + u < A.k)
                got[u] = ((local_mask >> (r0 + u)) & 1u) ? atomicAdd(A.counts + (r0 == 0 ? sl[u] : A.slot_ids[(size_t)t * A.k + r0 + u]), 1) : -1;
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (r0 + u < A.k) {
                A.rank[(size_t)t * A.k + r0 + u] = got[u];
                if (A.slot_tok && got[u] >= 0 && got[u] < A.B)
                    A.slot_tok[(size_t)(r0 == 0 ? sl[u] : A.slot_ids[(size_t)t * A.k + r0 + u]) * A.B + got[u]] = t;
            }
    }
}

// Softmax, top-k, rerouting and histogram of one 32-token tile whose logits lie in shared memory (expert-major,
// lg_s[j * 32 + token]), by the four epilogue warps: four adjacent lanes share a token, lane q of them owning the
// experts [q E, q E + E).  Each lane sorts its probabilities once (a 63-comparator network of max/min pairs, values
// only); the k rounds then look at the four lanes' heads alone - two shuffles for the maximum, a ballot for the
// lowest lane that holds it (lower expert index on ties), a pop; the expert index of a value is looked up afterwards,
// only for the values the lane contributed (lowest index with that value not taken yet, so ties inside a lane also go
// to the lower index).  No shared-memory exchange and no barrier between the rounds.  KD: how many of a lane's sorted
// values can be popped (8 for k <= 8, else 16).
//
// lg_s[j * stride + token]; this call handles the tile's tokens tl_base .. tl_base + 31.  hist_s null: the pairs are
// counted in the global counters right away (the value returned is the pair's position in its slot).  Otherwise (large
// batches, where thousands of pairs per slot would queue up at one counter) they are counted in the CTA's own
// histogram, the position inside the CTA is stored, and the caller adds the CTA's base per slot afterwards.
template <int KD>
__device__ __forceinline__ void quad_epilogue(const RouterArgs &A, const float *lg_s, int stride, int tl_base, const int32_t *pi_s,
                                              int tok0, int E, int a, int32_t *hist_s) {
    constexpr unsigned kFull = 0xffffffffu;
    const int tid2 = (int)threadIdx.x - 64;                          // 0..127 over the four epilogue warps
    const int tl = tl_base + (tid2 >> 2), q = tid2 & 3;              // token inside the tile, quarter of the experts
    const int t = tok0 + tl, M = A.M, k = A.k;
    const unsigned group_shift = threadIdx.x & 28;                   // first lane of this token's four within the warp
    const bool live = t < A.B;
    float e[16];
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int j = q * E + i;
        e[i] = (i < E && j < M) ? lg_s[j * stride + tl] : -INFINITY;
        mx = fmaxf(mx, e[i]);
    }
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 2));
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) {                                   // exp(-inf) = 0 for the absent experts
        e[i] = expf(e[i] - mx);
        sum += e[i];
    }
    sum += __shfl_xor_sync(kFull, sum, 1);
    sum += __shfl_xor_sync(kFull, sum, 2);
    const float inv_sum = 1.f / sum;
#pragma unroll
    for (int i = 0; i < 16; ++i) e[i] = (i < E && q * E + i < M) ? e[i] * inv_sum : -1.f;   // absent experts below every real one

    float s0[16];                                                    // the lane's probabilities sorted descending
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
    float s[KD];                                                     // the part of it that is popped during the rounds
#pragma unroll
    for (int i = 0; i < KD; ++i) s[i] = s0[i];
    unsigned won = 0;                                                // bit r: this lane's head won round r
    float wsum = 0.f;
    for (int r = 0; r < k; ++r) {
        float wv = s[0];
        wv = fmaxf(wv, __shfl_xor_sync(kFull, wv, 1));
        wv = fmaxf(wv, __shfl_xor_sync(kFull, wv, 2));
        const unsigned holders = (__ballot_sync(kFull, s[0] == wv) >> group_shift) & 0xfu;
        wsum += wv;
        if (q == __ffs(holders) - 1) {                               // the lowest lane that holds it pops its head
            won |= 1u << r;
#pragma unroll
            for (int i = 0; i < KD - 1; ++i) s[i] = s[i + 1];
            s[KD - 1] = -2.f;
        }
    }
    // this lane's wins, in round order, are s0[0], s0[1], ...: outputs first, all histogram atomics in flight together
    // (the value returned is the pair's position inside its slot's chunk), then the positions
    unsigned taken = 0;
    int p_slot[KD], p_r[KD], got[KD];                                // pending pairs: slot (-1: another rank's, -2: none), round
#pragma unroll
    for (int j = 0; j < KD; ++j) {
        p_slot[j] = -2;
        p_r[j] = 0;
        if (won && live) {
            const int r = __ffs(won) - 1;
            won &= won - 1;
            const float wv = s0[j];
            unsigned eq = 0;
#pragma unroll
            for (int i = 0; i < 16; ++i) eq |= (e[i] == wv) ? (1u << i) : 0u;
            const int idx = __ffs(eq & ~taken) - 1;                  // lowest index with that value not taken yet
            taken |= 1u << idx;
            const int id = q * E + idx;
            const int slot = a < 0 ? id : (A.pi_in_smem ? pi_s[a * M + id] : __ldg(A.pi + a * M + id));
            const size_t o = (size_t)t * k + r;
            float w = wv;
            if (A.renormalize) w = w / wsum;
            A.topk_ids[o] = id;
            A.slot_ids[o] = slot;
            A.topk_w[o] = (A.renormalize || A.scale != 1.f) ? w * A.scale : w;
            p_slot[j] = (id >= A.own_lo && id < A.own_hi) ? slot : -1;      // expert parallelism: another rank's pair is not counted
            p_r[j] = r;
        }
    }
#pragma unroll
    for (int j = 0; j < KD; ++j) got[j] = p_slot[j] >= 0 ? atomicAdd((hist_s ? hist_s : A.counts) + p_slot[j], 1) : -1;
#pragma unroll
    for (int j = 0; j < KD; ++j)
        if (p_slot[j] >= -1) {
            A.rank[(size_t)t * k + p_r[j]] = got[j];
            if (!hist_s && A.slot_tok && got[j] >= 0 && got[j] < A.B) A.slot_tok[(size_t)p_slot[j] * A.B + got[j]] = t;
        }
}

// REG = true: M <= 64, the token's probabilities stay in registers
template <bool REG>
__global__ void __launch_bounds__(kThreadsBig, 1)
router_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_r, const RouterArgs A) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
    const int M = A.M, stages = A.stages, tok_tile = A.tok_tile, kAtoms = A.atoms;
    const int n_mma = ((M + 15) >> 4) << 4;                          // router rows arrive as one box of n_mma rows
    const int x_atom = tok_tile * kBlockK * 2;                       // bytes of one K-atom of the token tile (multiple of 4 KiB)
    const int r_atom = (n_mma * kBlockK * 2 + 1023) & ~1023;         // and of the router tile
    const int x_bytes = kAtoms * x_atom;
    const int stage_bytes = x_bytes + kAtoms * r_atom;
    // ring, then 16 KiB of slack (the MMA reads a full 128-row A tile from every stage), then barriers
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + stages * stage_bytes + kTileRows * kBlockK * 2);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * kMaxStages, bar_done = bar_empty + 8 * kMaxStages;
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(bars + 2 * kMaxStages + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);
    int32_t *pi_s = reinterpret_cast<int32_t *>(tmem_holder + 2);
    float *pbuf = reinterpret_cast<float *>(smem_al);                // [M][128]; aliases the ring once it has drained

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // K split over a cluster: CTA `krank` of the `cs` CTAs that share token tile `blockIdx.x / cs` owns the K-atoms
    // [atom0, atom0 + num_atoms)
    const int cs = A.ksplit;
    const int krank = cs > 1 ? (int)cluster_ctarank() : 0;
    const int atoms_all = A.H / kBlockK, atoms_per = (atoms_all + cs - 1) / cs;
    const int atom0 = krank * atoms_per;
    const int num_atoms = max(0, min(atoms_per, atoms_all - atom0));
    const int num_kb = (num_atoms + kAtoms - 1) / kAtoms;
    const int tok0 = (cs > 1 ? (int)blockIdx.x / cs : (int)blockIdx.x) * tok_tile;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_done, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_map(&map_x);
        prefetch_map(&map_r);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"((uint32_t)A.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (A.pi_in_smem)
        for (int i = threadIdx.x; i < A.N * M; i += blockDim.x) pi_s[i] = A.pi[i];
    if (!A.hold_dependents) pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    pdl_wait();                                         // x and the slot counters belong to earlier work in the stream

    if (warp == 0) {
        if (lane == 0) {                                             // TMA producer
            uint32_t stage = 0, phase = 0;
            for (int kb = 0; kb < num_kb; ++kb) {
                if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, abort_flag, A.err)) break;
                const uint32_t sa = smem_base + stage * stage_bytes, full = bar_full + 8 * stage;
                mbar_expect_tx(full, kAtoms * (tok_tile + n_mma) * kBlockK * 2);
                tma_load_3d(sa, &map_x, 0, tok0, atom0 + kb * kAtoms, full);
                tma_load_3d(sa + x_bytes, &map_r, 0, 0, atom0 + kb * kAtoms, full);
                if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1; }
            }
        }
        if (cs > 1) cluster_arrive();                                // every thread of the cluster arrives exactly once
    } else if (warp == 1) {
        if (lane == 0) {                                             // MMA issuer
            uint32_t stage = 0, phase = 0;
            const uint32_t idesc = instr_desc(n_mma);
            bool ok = true;
            for (int kb = 0; kb < num_kb && ok; ++kb) {
                if (!(ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, A.err))) break;
                tc_fence_after();
                const uint32_t sa = smem_base + stage * stage_bytes;
                const int atoms = min(kAtoms, num_atoms - kb * kAtoms);      // atoms past H arrive zero-filled: skip them
                for (int at = 0; at < atoms; ++at) {
                    const uint64_t a = smem_desc_sw128(sa + at * x_atom), b = smem_desc_sw128(sa + x_bytes + at * r_atom);
#pragma unroll
                    for (int ki = 0; ki < kBlockK / 16; ++ki)
                        tc_mma(tmem_base, a + 2 * ki, b + 2 * ki, idesc, (kb | at | ki) ? 1u : 0u);
                }
                tc_commit(bar_empty + 8 * stage);
                if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1; }
            }
            if (ok) tc_commit(bar_done);
        }
        if (cs > 1) cluster_arrive();
    } else if (REG && tok_tile == 32) {
        // epilogue for 32-token tiles (small batches, where this kernel's latency is exposed): the logits sit in
        // TMEM lanes 0..31 only, which one warp can read; that warp spills them to shared memory and then all four
        // epilogue warps work on them, four threads per token, each owning a quarter of the experts (quad_epilogue).
        const int g = warp & 3;                                      // g == 0: the warp that reads TMEM
        const int E = n_mma >> 2;                                    // experts per quarter (4, 8, 12 or 16)
        const int k = A.k;
        auto quad_sync = [] { asm volatile("bar.sync 1, 128;" ::: "memory"); };   // the four epilogue warps
        // the adapter id of this thread's token (quad_epilogue's mapping), fetched while the logits are still being computed
        const int t_mine = tok0 + (((int)threadIdx.x - 64) >> 2);
        const int a_mine = (krank == 0 && t_mine < A.B) ? checked_aid(A.aid[t_mine], A.N, A.loaded, A.err) : -1;
        mbar_wait(bar_done, 0, abort_flag, A.err);
        quad_sync();                                                 // every epilogue thread is past its (bounded) wait
        float *lg_s = reinterpret_cast<float *>(smem_al);            // [n_mma][32] logits, expert-major (the ring has drained)
        float *part_s = reinterpret_cast<float *>(smem_al + A.part_off);   // K split: [cs][n_mma][32] partial logits (CTA 0's is used)
        if (!*abort_flag && g == 0) {
            tc_fence_after();
            uint32_t v0[32], v1[32];
            if (n_mma >= 32) tc_ld32(tmem_base, v0); else tc_ld16(tmem_base, v0);
            if (n_mma > 32) { if (n_mma - 32 >= 32) tc_ld32(tmem_base + 32, v1); else tc_ld16(tmem_base + 32, v1); }
            tc_wait_ld();
            if (cs == 1) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    if (j < n_mma) lg_s[j * 32 + lane] = __uint_as_float(v0[j]);
                    if (32 + j < n_mma) lg_s[(32 + j) * 32 + lane] = __uint_as_float(v1[j]);
                }
            } else {                                                 // this CTA's share of K: to the cluster's first CTA
                float *mine = part_s + krank * (n_mma * 32);
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    if (j < n_mma) st_leader_f32(mine + j * 32 + lane, num_atoms ? __uint_as_float(v0[j]) : 0.f);
                    if (32 + j < n_mma) st_leader_f32(mine + (32 + j) * 32 + lane, num_atoms ? __uint_as_float(v1[j]) : 0.f);
                }
            }
        }
        if (cs > 1) {
            cluster_arrive();
            if (krank == 0) {
                cluster_wait();                                      // all partial logits have landed here
                const int tid2 = (int)threadIdx.x - 64;              // 0..127 over the four epilogue warps
                for (int i = tid2; i < n_mma * 32; i += 128) {
                    float acc = part_s[i];
                    for (int r = 1; r < cs; ++r) acc += part_s[r * (n_mma * 32) + i];    // rank order: independent of timing
                    lg_s[i] = acc;
                }
            }
        }
        quad_sync();
        if (!*abort_flag && krank == 0) {
            if (k <= 8) quad_epilogue<8>(A, lg_s, 32, 0, pi_s, tok0, E, a_mine, nullptr);
            else quad_epilogue<16>(A, lg_s, 32, 0, pi_s, tok0, E, a_mine, nullptr);
        }
    } else if (REG && A.big_quad) {
        // epilogue for 64- and 128-token tiles (large batches): the warps that own TMEM lanes with tokens spill the
        // logits to shared memory (the ring has drained), then eight warps go through the tile 64 tokens at a time
        // with four lanes per token (quad_epilogue; one warp works through its eight tokens' selection in ~9 us of
        // dependent instructions, so the passes are spread over warps rather than run one after the other).  The pairs are counted in a histogram of the CTA; afterwards one
        // atomic per live slot fetches the CTA's base in the global counter, and a sweep over the tile's pairs turns the
        // positions inside the CTA into positions inside the slot.  (Counting every pair in the global counters
        // directly took 10-17 us of an 8192-token batch: some 700 returning atomics queue up per base expert.)
        const int lgp = warp & 3;
        const int E = n_mma >> 2;
        const int k = A.k;
        const int tid2 = (int)threadIdx.x - 64;
        auto quad_sync = [] { asm volatile("bar.sync 1, 256;" ::: "memory"); };   // the eight epilogue warps (320 threads per CTA in this mode)
        constexpr int kEpi = kThreadsBig - 64;
        float *lg_s = reinterpret_cast<float *>(smem_al);            // [n_mma][tok_tile] logits, expert-major
        int32_t *hist_s = reinterpret_cast<int32_t *>(lg_s + 64 * tok_tile);      // [P] pairs of this CTA per slot, then the CTA's base
        int32_t *aid_s = hist_s + A.P;                               // [tok_tile] checked adapter ids
        const int P = A.P;
        // adapter ids of the tile's tokens, fetched while the logits are still being computed (kept in registers until
        // the ring has drained)
        const int a_reg = (tid2 < tok_tile && tok0 + tid2 < A.B) ? checked_aid(A.aid[tok0 + tid2], A.N, A.loaded, A.err) : -1;
        mbar_wait(bar_done, 0, abort_flag, A.err);
        quad_sync();                                                 // every epilogue thread is past its (bounded) wait
        const bool go = !*abort_flag;
        if (go) {
            for (int i = tid2; i < P; i += kEpi) hist_s[i] = 0;
            if (tid2 < tok_tile) aid_s[tid2] = a_reg;
            if (warp < 6 && lgp * 32 < tok_tile) {                  // warps 2..5 own the four TMEM lane groups
                tc_fence_after();
                const uint32_t t0 = tmem_base + ((uint32_t)(lgp * 32) << 16);
                uint32_t v0[32], v1[32];
                if (n_mma >= 32) tc_ld32(t0, v0); else tc_ld16(t0, v0);
                if (n_mma > 32) { if (n_mma - 32 >= 32) tc_ld32(t0 + 32, v1); else tc_ld16(t0 + 32, v1); }
                tc_wait_ld();
                float *col = lg_s + lgp * 32 + lane;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    if (j < n_mma) col[j * tok_tile] = __uint_as_float(v0[j]);
                    if (32 + j < n_mma) col[(32 + j) * tok_tile] = __uint_as_float(v1[j]);
                }
            }
        }
        quad_sync();
        if (go) {
#pragma unroll 1
            for (int tb = 0; tb < tok_tile; tb += 64) {           // 256 threads: 64 tokens per pass
                const int a = aid_s[tb + (tid2 >> 2)];
                if (k <= 8) quad_epilogue<8>(A, lg_s, tok_tile, tb, pi_s, tok0, E, a, hist_s);
                else quad_epilogue<16>(A, lg_s, tok_tile, tb, pi_s, tok0, E, a, hist_s);
            }
        }
        quad_sync();
        if (go)
            for (int i = tid2; i < P; i += kEpi) {
                const int c = hist_s[i];
                if (c) hist_s[i] = atomicAdd(A.counts + i, c);        // the CTA's first position in slot i
            }
        quad_sync();
        if (go) {
            const int n_q = min(tok_tile, A.B - tok0) * k;
            for (int qq = tid2; qq < n_q; qq += kEpi) {
                const size_t o = (size_t)tok0 * k + qq;
                int r = *reinterpret_cast<volatile int32_t *>(A.rank + o);
                if (r >= 0) {                                         // (-1: another rank's pair, expert parallelism)
                    const int slot = *reinterpret_cast<volatile int32_t *>(A.slot_ids + o);
                    r += hist_s[slot];
                    A.rank[o] = r;
                    if (A.slot_tok && r < A.B) A.slot_tok[(size_t)slot * A.B + r] = tok0 + qq / k;
                }
            }
        }
    } else {
        // epilogue: thread <-> token
        const int lg = warp & 3;
        const int tl = lg * 32 + lane;                               // token inside the tile = TMEM lane
        const int t = tok0 + tl;
        const int k = A.k;
        if (lg * 32 < tok_tile && mbar_wait(bar_done, 0, abort_flag, A.err)) {
            tc_fence_after();
            const uint32_t t0 = tmem_base + ((uint32_t)(lg * 32) << 16);
            if (REG) {
                uint32_t v0[32], v1[32];
                if (n_mma >= 32) tc_ld32(t0, v0); else tc_ld16(t0, v0);
                if (n_mma > 32) { if (n_mma - 32 >= 32) tc_ld32(t0 + 32, v1); else tc_ld16(t0 + 32, v1); }
                tc_wait_ld();
                float p[64];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    p[j] = j < M ? __uint_as_float(v0[j]) : -INFINITY;
                    p[32 + j] = 32 + j < M ? __uint_as_float(v1[j]) : -INFINITY;
                }
                float mx = p[0];
#pragma unroll
                for (int j = 1; j < 64; ++j) mx = fmaxf(mx, p[j]);
                float sum = 0.f;
#pragma unroll
                for (int j = 0; j < 64; ++j) {                       // exp(-inf) = 0 for the absent experts
                    p[j] = expf(p[j] - mx);
                    sum += p[j];
                }
                const float inv_sum = 1.f / sum;
#pragma unroll
                for (int j = 0; j < 64; ++j) p[j] = j < M ? p[j] * inv_sum : -1.f;
                if (t < A.B) {
                    const int a = checked_aid(A.aid[t], A.N, A.loaded, A.err);
                    float wsum = 0.f;
                    int sl[8];
                    uint32_t local_mask = 0;
                    for (int r = 0; r < k; ++r) {
                        float bv = -1.f;
                        int bi = 0;
#pragma unroll
                        for (int j = 0; j < 64; ++j) {               // branch-free selects; strict >: the lower index keeps a tie
                            const bool gt = p[j] > bv;
                            bv = gt ? p[j] : bv;
                            bi = gt ? j : bi;
                        }
#pragma unroll
                        for (int j = 0; j < 64; ++j) p[j] = (j == bi) ? -1.f : p[j];   // taken (probabilities are >= 0)
                        wsum += bv;
                        emit_pair(A, pi_s, t, r, a, bi, bv, sl, local_mask);
                    }
                    emit_ranks(A, t, sl, local_mask);
                    if (A.renormalize || A.scale != 1.f)
                        for (int r = 0; r < k; ++r) {
                            const size_t o = (size_t)t * k + r;
                            float w = A.topk_w[o];
                            if (A.renormalize) w = w / wsum;
                            A.topk_w[o] = w * A.scale;
                        }
                }
            } else {
                uint32_t v[32];
                float mx = -INFINITY;
                for (int c0 = 0; c0 < n_mma; c0 += 32) {             // pass 1: max logit
                    if (n_mma - c0 >= 32) tc_ld32(t0 + c0, v); else tc_ld16(t0 + c0, v);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (c0 + j < M) mx = fmaxf(mx, __uint_as_float(v[j]));
                }
                float sum = 0.f;
                for (int c0 = 0; c0 < n_mma; c0 += 32) {             // pass 2: exponentials and their sum (j ascending)
                    if (n_mma - c0 >= 32) tc_ld32(t0 + c0, v); else tc_ld16(t0 + c0, v);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (c0 + j < M) {
                            const float e = expf(__uint_as_float(v[j]) - mx);
                            pbuf[(c0 + j) * kTileRows + tl] = e;
                            sum += e;
                        }
                }
                for (int j = 0; j < M; ++j) pbuf[j * kTileRows + tl] = pbuf[j * kTileRows + tl] / sum;
                if (t < A.B) {
                    const int a = checked_aid(A.aid[t], A.N, A.loaded, A.err);
                    float wsum = 0.f;
                    int sl[8];
                    uint32_t local_mask = 0;
                    for (int r = 0; r < k; ++r) {
                        float bv = -1.f;
                        int bi = 0;
                        for (int j = 0; j < M; ++j) {
                            const float pj = pbuf[j * kTileRows + tl];
                            const bool gt = pj > bv;
                            bv = gt ? pj : bv;
                            bi = gt ? j : bi;
                        }
                        pbuf[bi * kTileRows + tl] = -1.f;
                        wsum += bv;
                        emit_pair(A, pi_s, t, r, a, bi, bv, sl, local_mask);
                    }
                    emit_ranks(A, t, sl, local_mask);
                    if (A.renormalize || A.scale != 1.f)
                        for (int r = 0; r < k; ++r) {
                            const size_t o = (size_t)t * k + r;
                            float w = A.topk_w[o];
                            if (A.renormalize) w = w / wsum;
                            A.topk_w[o] = w * A.scale;
                        }
                }
            }
        }
    }

    if (*abort_flag) {
        long long c0 = clock64();
        while (clock64() - c0 < 2000000ll) {}
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)A.tmem_cols)
                     : "memory");
}


// Launch geometry of the router kernel for a batch of B tokens: tokens per CTA, K-atoms per stage, ring depth.
struct RouterGeometry {
    int tok_tile, atoms, stages, pi_in_smem, tmem_cols, grid, ksplit, part_off, big_quad;
    bool reg;
    size_t smem;
};

static bool ksplit_enabled() {       // EW_DISABLE_KSPLIT=1: every CTA runs the whole K range (debugging and A/B runs)
    static const bool on = [] { const char *e = getenv("EW_DISABLE_KSPLIT"); return !(e && e[0] == '1'); }();
    return on;
}

static bool router_geometry(const ew_pool *p, int B, RouterGeometry *g) {
    const ew_config_t &c = p->cfg;
    const int M = c.num_experts, n_mma = (M + 15) / 16 * 16;
    // tokens per CTA: small batches are spread over more SMs (each CTA streams the whole router matrix)
    g->tok_tile = B <= 32 * p->sm_count ? 32 : B <= 64 * p->sm_count ? 64 : 128;
    const size_t pi_bytes = (size_t)c.max_adapters * M * 4;
    g->pi_in_smem = pi_bytes <= (size_t)kMaxPiSmem;
    g->reg = M <= 64;
    const int tiles = (B + g->tok_tile - 1) / g->tok_tile, atoms_all = c.hidden / kBlockK;
    // K split over a cluster where the tiles alone would leave most SMs idle
    g->ksplit = 1;
    if (g->reg && g->tok_tile == 32 && ksplit_enabled()) {
        if (tiles * 8 <= p->sm_count && atoms_all >= 8) g->ksplit = 8;
        else if (tiles * 4 <= p->sm_count && atoms_all >= 4) g->ksplit = 4;
    }
    const size_t part_bytes = g->ksplit > 1 ? (size_t)g->ksplit * n_mma * 32 * 4 : 0;
    const size_t fixed = kTileRows * kBlockK * 2 + 8 * (2 * kMaxStages + 1) + 8 + (g->pi_in_smem ? pi_bytes : 0);   // slack, barriers, map
    const size_t tail = 1024 /*alignment*/ + fixed + 16 + part_bytes + 64;
    const size_t pbuf_bytes = g->reg ? 0 : (size_t)M * kTileRows * 4;
    for (int atoms = kMaxAtoms; atoms >= 1; atoms >>= 1) {      // as many K-atoms per stage as leave a ring of >= 3 (else 2) stages
        const int stage_bytes = atoms * (g->tok_tile * kBlockK * 2 + ((n_mma * kBlockK * 2 + 1023) & ~1023));
        int stages = (int)((227 * 1024 - tail) / stage_bytes);
        if (stages > kMaxStages) stages = kMaxStages;
        if (g->ksplit > 1) {                                        // a CTA only has atoms_all / ksplit atoms to load
            const int need = ((atoms_all + g->ksplit - 1) / g->ksplit + atoms - 1) / atoms;
            if (stages > (need < 2 ? 2 : need)) stages = need < 2 ? 2 : need;
        }
        const bool fits = (size_t)stages * stage_bytes + kTileRows * kBlockK * 2 >= pbuf_bytes &&
                          (size_t)stages * stage_bytes >= (size_t)(64 * 32 + 3 * 2 * 4 * 32) * 4;   // the epilogue's scratch aliases the ring
        if ((stages >= 3 || ((atoms == 1 || g->ksplit > 1) && stages >= 2)) && fits) {
            g->atoms = atoms;
            g->stages = stages;
            g->part_off = (int)(((size_t)stages * stage_bytes + fixed + 15) & ~(size_t)15);
            // the large-tile epilogue keeps logits, a histogram over the slots and the tile's adapter ids in the drained ring
            g->big_quad = g->reg && g->tok_tile >= 64 &&
                          (size_t)stages * stage_bytes >= ((size_t)64 * g->tok_tile + p->P + g->tok_tile) * 4;
            g->smem = (size_t)stages * stage_bytes + tail;
            g->tmem_cols = n_mma <= 32 ? 32 : n_mma <= 64 ? 64 : n_mma <= 128 ? 128 : 256;
            g->grid = tiles * g->ksplit;
            return true;
        }
    }
    return false;
}

static int router_launch(ew_pool *p, int layer, const void *x, const RouterGeometry &g, RouterArgs &A, bool pdl, cudaStream_t st) {
    const ew_config_t &c = p->cfg;
    const LayerState &L = p->layers[layer];
    CUtensorMap map_x;
    if (make_atom_map(p, &map_x, x, c.hidden, A.B, g.tok_tile, g.atoms)) return (int)cudaErrorInvalidValue;
    const CUtensorMap &map_r = L.map_router[g.atoms == 4 ? 2 : g.atoms == 2 ? 1 : 0];
    A.pi = L.pi_dev; A.loaded = p->ws.loaded;
    A.H = c.hidden; A.M = c.num_experts; A.k = c.top_k; A.N = c.max_adapters; A.renormalize = c.renormalize;
    A.scale = c.routed_scale;
    A.stages = g.stages; A.tmem_cols = g.tmem_cols; A.pi_in_smem = g.pi_in_smem; A.tok_tile = g.tok_tile; A.atoms = g.atoms;
    A.ksplit = g.ksplit; A.part_off = g.part_off; A.big_quad = g.big_quad; A.P = p->P;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g.grid);
    cfg.blockDim = dim3(g.big_quad ? kThreadsBig : kThreads);
    cfg.dynamicSmemBytes = g.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (g.ksplit > 1) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = g.ksplit;
        attr[n_attr].val.clusterDim.y = 1;
        attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    if (pdl && pdl_enabled()) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    if (g.reg) return (int)cudaLaunchKernelEx(&cfg, router_kernel<true>, map_x, map_r, A);
    return (int)cudaLaunchKernelEx(&cfg, router_kernel<false>, map_x, map_r, A);
}

}  // namespace

int launch_route(ew_pool *p, int layer, const void *x, const int32_t *aid, int B, cudaStream_t st) {
    RouterGeometry g;
    if (!router_geometry(p, B, &g)) return (int)cudaErrorInvalidConfiguration;
    RouterArgs A;
    A.aid = aid; A.B = B;
    A.topk_ids = p->ws.topk_ids; A.topk_w = p->ws.topk_w; A.slot_ids = p->ws.slot_ids; A.rank = p->ws.rank;
    A.counts = p->ws.counts; A.err = p->ws.err;
    A.slot_tok = p->self_plan ? p->ws.slot_tok : nullptr;
    A.own_lo = p->own_lo; A.own_hi = p->own_hi;
    // followed by the planning kernel: not released early (its CTAs, resident beside this kernel's and waiting, cost the
    // decode layer 3 us and the prefill layer 4 us); followed by GEMM-1 (self-planned forwards): released at once,
    // GEMM-1 sets itself up and rehearses its item derivation meanwhile on the SMs this kernel leaves free
    A.hold_dependents = p->self_plan ? 0 : 1;
    return router_launch(p, layer, x, g, A, true, st);
}

}  // namespace ew

// ================================================================================================
// Allocation-free routing.
//
// Some callers may not allocate device memory at the moment they need a routing decision: a serving
// engine that has handed every free byte of HBM to its KV cache (any cudaMalloc then fails or
// fragments), or code that runs where the CUDA allocator must not be entered at all.  The pool's own
// forward never allocates either, but it owns exactly one workspace, so a second batch cannot be routed
// while a forward is in flight without a second workspace, i.e. an allocation.  ew_route_noalloc runs
// the fused router kernel with the caller's output buffers and keeps the kernel's scratch (the
// device status word and the per-pair positions inside each slot) in the fixed array below, which every
// GPU that loads this library holds until the process exits.
// ================================================================================================
namespace ew {
namespace {
constexpr int kNoAllocMaxPairs = 65536;                 // n_tokens * top_k accepted by ew_route_noalloc
constexpr int kNoAllocHeader = 256;                     // bytes before the per-pair array; word 0 = status
}  // namespace
}  // namespace ew

static __device__ __align__(256) unsigned char g_route_noalloc_scratch[ew::kNoAllocHeader + ew::kNoAllocMaxPairs * 4];

namespace ew {
namespace {
std::mutex g_noalloc_mu;
unsigned char *g_noalloc_ptr[64] = {};                  // device address of the array, per device ordinal

// The array's name is only a host-side handle: resolve its device address once per device, with that
// device current, and hand the address to the kernel.
int noalloc_scratch(int device, unsigned char **out) {
    if (device < 0 || device >= 64) return (int)cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_noalloc_mu);
    if (!g_noalloc_ptr[device]) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_route_noalloc_scratch);
        if (e != cudaSuccess) return (int)e;
        g_noalloc_ptr[device] = static_cast<unsigned char *>(ptr);
    }
    *out = g_noalloc_ptr[device];
    return 0;
}
}  // namespace

// Once per pool, with the pool's device current (ew_pool_create): everything about the router kernels that may load
// code or reserve memory on first use happens here, where the pool allocates anyway - the opt-in to large dynamic
// shared memory, a query that forces both instantiations to be loaded, and the device address of the fixed scratch
// array.  ew_route_noalloc then only looks the address up.
int router_setup(ew_pool *p) {
    cudaError_t e = cudaFuncSetAttribute(router_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(router_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    cudaFuncAttributes fa;
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, router_kernel<true>);
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, router_kernel<false>);
    unsigned char *scratch = nullptr;
    int rc = e == cudaSuccess ? noalloc_scratch(p->cfg.device, &scratch) : (int)e;
    if (rc) set_last_error(std::string("router set-up: ") + cudaGetErrorString((cudaError_t)rc));
    return rc;
}
}  // namespace ew

extern "C" ew_status_t ew_route_noalloc(ew_pool_t *p, int32_t layer, const void *x, const int32_t *adapter_ids,
                                        int32_t n_tokens, int32_t *topk_ids, float *topk_w, int32_t *slot_ids,
                                        int32_t *counts, int32_t *device_status, void *cuda_stream) {
    using namespace ew;
    if (!p || layer < 0 || layer >= p->cfg.num_layers || n_tokens < 0) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    const ew_config_t &c = p->cfg;
    if ((long long)n_tokens * c.top_k > kNoAllocMaxPairs) {
        set_last_error("ew_route_noalloc: n_tokens * top_k exceeds the fixed scratch array (65536 pairs)");
        return EW_ERR_INVALID_ARG;
    }
    if (!counts) return EW_ERR_INVALID_ARG;
    if (!p->layers[layer].base_loaded) return EW_ERR_NOT_LOADED;
    if (n_tokens > 0 && (!x || !adapter_ids || !topk_ids || !topk_w || !slot_ids || ((uintptr_t)x & 15))) return EW_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    DeviceGuard guard;
    cudaError_t e = guard.enter(c.device);
    unsigned char *scratch = nullptr;
    int rc = e == cudaSuccess ? noalloc_scratch(c.device, &scratch) : (int)e;      // resolved when the pool was created
    // the array keeps the previous call's contents: the status word and the counters must start at zero
    if (!rc) rc = (int)cudaMemsetAsync(scratch, 0, kNoAllocHeader, st);
    if (!rc) rc = (int)cudaMemsetAsync(counts, 0, (size_t)p->P * 4, st);
    if (!rc && n_tokens > 0) {
        RouterGeometry g;
        if (!router_geometry(p, n_tokens, &g)) return EW_ERR_INVALID_ARG;
        RouterArgs A;
        A.aid = adapter_ids; A.B = n_tokens;
        A.topk_ids = topk_ids; A.topk_w = topk_w; A.slot_ids = slot_ids; A.counts = counts;
        A.rank = reinterpret_cast<int32_t *>(scratch + kNoAllocHeader);      // scratch: position of each pair in its slot
        A.err = reinterpret_cast<int *>(scratch);                            // scratch: device status word
        rc = router_launch(p, layer, x, g, A, false, st);
    }
    if (!rc && device_status) rc = (int)cudaMemcpyAsync(device_status, scratch, 4, cudaMemcpyDeviceToDevice, st);
    // eviction and base reloads wait for this call through an event that was created with the pool
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (!rc && cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone) {
        rc = (int)cudaEventRecord(p->route_event, st);
        p->route_event_used = true;
    }
    if (rc) {
        set_last_error(std::string("ew_route_noalloc: ") + cudaGetErrorString((cudaError_t)rc));
        return EW_ERR_CUDA;
    }
    return EW_OK;
}

// ================================================================================================
// Self-test of the bounded wait: a one-CTA kernel waits on an mbarrier that nothing ever arrives at,
// with the same wait routine the tensor-core kernels use and a limit of about a millisecond.  The wait
// must expire, raise bit 1 of the device error word and let the kernel return normally.
// ================================================================================================
namespace ew {
namespace {
__global__ void wait_selftest_kernel(int *err, int *reached_end) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool ok = true;
    if (threadIdx.x == 0) ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, err, 2000000ll);
    __syncthreads();
    if (threadIdx.x == 0) *reached_end = ok ? 2 : 1;     // 1: the wait gave up and the kernel went on to its end
}
}  // namespace
}  // namespace ew

extern "C" ew_status_t ew_selftest_bounded_wait(ew_pool_t *p, void *cuda_stream) {
    using namespace ew;
    if (!p) return EW_ERR_INVALID_ARG;
    if (p->cfg.device < 0) return EW_ERR_NO_DEVICE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    DeviceGuard guard;
    int *flag = p->ws.err + 1;                            // second word of the error segment
    cudaError_t e = guard.enter(p->cfg.device);
    if (e == cudaSuccess) e = cudaMemsetAsync(flag, 0, 4, st);
    if (e == cudaSuccess) {
        wait_selftest_kernel<<<1, 32, 0, st>>>(p->ws.err, flag);
        e = cudaGetLastError();
    }
    int reached = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&reached, flag, 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) {
        set_last_error(std::string("ew_selftest_bounded_wait: ") + cudaGetErrorString(e));
        return EW_ERR_CUDA;
    }
    return reached == 1 ? EW_OK : EW_ERR_INVALID_ARG;
}
