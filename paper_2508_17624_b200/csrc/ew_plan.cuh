// Dispatch planning (device functions used by the permute kernel): the exclusive scan of the
// per-slot token counts (Section 2.1 dispatch), the slot-contiguous order of the (token, expert) pairs as two
// tables (inv: pair -> row, src_tok: row -> token), and the work-item lists of the two grouped GEMMs.
//
// All functions are block-wide: every thread of the CTA calls them with the same arguments; `nthreads` =
// blockDim.x must be a multiple of 32 and at most 256.
#pragma once
#include "ew_internal.h"

namespace ew {
namespace plan {

// Shared-memory words the planner needs for P slots and S shared experts.
__host__ __device__ constexpr size_t smem_words(int P, int S) { return (size_t)(P + 1) + 4 * (size_t)(P + S + 1) + (size_t)P; }

// out[0..n] = exclusive scan of in[0..n-1] (out[n] = total).
__device__ inline void block_exclusive_scan(const int32_t *in, int32_t *out, int n, int32_t *warp_sums, int nthreads) {
    const int per = (n + nthreads - 1) / nthreads;
    const int lo = min((int)threadIdx.x * per, n), hi = min(lo + per, n);
    int32_t s = 0;
    for (int i = lo; i < hi; ++i) s += in[i];
    int32_t incl = s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int32_t base = 0;
    for (int w = 0; w < warp; ++w) base += warp_sums[w];
    int32_t run = base + incl - s;
    for (int i = lo; i < hi; ++i) { out[i] = run; run += in[i]; }
    if ((int)threadIdx.x == nthreads - 1) out[n] = run;     // the last thread's range ends at n
    __syncthreads();
}

struct Params {
    int B, k, P, S;
    int NT1, NT2;        // token rows per work item of GEMM-1 / GEMM-2
    int R1, R2;          // weight tiles per group of GEMM-1 / GEMM-2
    int32_t *offsets;    // [P + 1] out
    GemmItem *items1, *items2;
    int32_t *n_items;    // [2] out
};

// Stages the counts and scans them: sm[0..P] = offsets, and cnt_s (returned) = the counts.  `counts` is read
// with L1 bypassed (other CTAs' atomics produced it).
__device__ inline int32_t *stage_and_scan(int32_t *sm, const int32_t *counts, int P, int S, int32_t *warp_sums, int nthreads) {
    int32_t *cnt_s = sm + (P + 1) + 4 * (P + S + 1);
    for (int i = threadIdx.x; i < P; i += nthreads) cnt_s[i] = __ldcg(counts + i);
    __syncthreads();
    block_exclusive_scan(cnt_s, sm, P, warp_sums, nthreads);
    return cnt_s;
}

// Writes the work items of the groups g = first_group, first_group + group_stride, ... (one warp per group, lanes
// over the group's items); planner 0 also publishes the offsets and the item counts.  `sm` as left by
// stage_and_scan.
//
// groups: g < S shared expert g (rows = B); g >= S slot g - S (rows = counts).  Two classes: "thin" groups (at
// most kThinRows rows: their items are weight streams) and "fat" ones (tensor-core bound at prefill).  The two
// item sequences are merged evenly, so that at any moment the CTAs hold a mix of both and the weight stream of the
// thin items overlaps the arithmetic of the fat ones.  Per group the items are ordered (weight tile, token block)
// so that CTAs working at the same time share a weight tile through L2.
__device__ inline void write_items(int32_t *sm, const int32_t *cnt_s, const Params &A, int32_t *warp_sums, int nthreads,
                                   int first_warp, int warp_stride, bool publish) {
    constexpr int kThinRows = 64;
    const int P = A.P, S = A.S, B = A.B;
    const int G = P + S;
    const int32_t *off = sm;
    int32_t *blk = sm + P + 1;              // [G + 1] scan of the fat groups' token blocks
    int32_t *nblk = blk + G + 1;            // [G] token blocks of fat groups (0 for thin ones)
    int32_t *blk_t = nblk + G;              // [G + 1] scan of the thin groups' token blocks
    int32_t *nblk_t = blk_t + G + 1;        // [G]
    const int lane = threadIdx.x & 31;
    if (publish)
        for (int i = threadIdx.x; i <= P; i += nthreads) A.offsets[i] = off[i];
    // GEMM-1 and GEMM-2 may use different token tiles (NT1, NT2): each pass has its own block counts and scans
    for (int pass = 0; pass < 2; ++pass) {
        const int NT = pass ? A.NT2 : A.NT1;
        const int R = pass ? A.R2 : A.R1;
        if (pass == 0 || A.NT2 != A.NT1) {                // same tile in both GEMMs (decode): one set of scans serves both
            __syncthreads();                              // the previous pass has finished reading the scan arrays
            for (int g = threadIdx.x; g < G; g += nthreads) {
                const int rows = g < S ? B : cnt_s[g - S];
                const int nb = (rows + NT - 1) / NT;
                const bool thin = rows <= kThinRows;
                nblk[g] = thin ? 0 : nb;
                nblk_t[g] = thin ? nb : 0;
            }
            __syncthreads();
            block_exclusive_scan(nblk, blk, G, warp_sums, nthreads);
            block_exclusive_scan(nblk_t, blk_t, G, warp_sums, nthreads);
        }
        const int fat_blocks = blk[G], thin_blocks = blk_t[G];
        if (publish && threadIdx.x == 0) A.n_items[pass] = (fat_blocks + thin_blocks) * R;
        const long long n_fat = (long long)fat_blocks * R, n_thin = (long long)thin_blocks * R;
        const bool small = (n_fat + 1) * (n_thin + 1) < (1ll << 31);
        GemmItem *dst = pass ? A.items2 : A.items1;
        for (int g = first_warp; g < G; g += warp_stride) {
            const bool thin = nblk_t[g] > 0;
            const int nb = thin ? nblk_t[g] : nblk[g];
            if (nb == 0) continue;
            const bool shared = g < S;
            const int rows = shared ? B : cnt_s[g - S];
            const int slot = shared ? P + g : g - S;
            const int in0 = shared ? 0 : off[g - S];
            const int out0 = shared ? g * B : S * B + off[g - S];
            const long long first = (long long)(thin ? blk_t[g] : blk[g]) * R;    // index inside the group's own class
            for (int i = lane; i < nb * R; i += 32) {
                const int tile = i / nb, c = i % nb;
                const int in_row = (pass ? out0 : in0) + c * NT;     // GEMM-2 reads what GEMM-1 wrote
                const int out_row = out0 + c * NT;
                const int item_rows = min(NT, rows - c * NT);
                const int from_x = (!pass && shared) ? 1 : 0;
                // merged position: thin item q has floor(q*n_fat/n_thin) fat items before it, and fat item q
                // the thin items that rule puts before it
                const long long q = first + i;
                long long pos;
                if (small) {                                  // every product fits 32 bits: cheap divisions
                    const unsigned qu = (unsigned)q, nf = (unsigned)n_fat, nt = (unsigned)n_thin;
                    if (thin) pos = nf ? qu + qu * nf / nt : qu;
                    else pos = nt ? qu + min(nt, ((qu + 1) * nt + nf - 1) / nf) : qu;
                } else {
                    if (thin) pos = n_fat ? q + q * n_fat / n_thin : q;
                    else pos = n_thin ? q + min(n_thin, ((q + 1) * n_thin + n_fat - 1) / n_fat) : q;
                }
                int4 *d4 = reinterpret_cast<int4 *>(dst + pos);      // one item = two 16-byte stores
                d4[0] = make_int4(slot, tile, in_row, out_row);
                d4[1] = make_int4(item_rows, from_x, 0, 0);
            }
        }
    }
}

}  // namespace plan
}  // namespace ew
