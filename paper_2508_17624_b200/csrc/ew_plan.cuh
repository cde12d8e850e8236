// Dispatch planning (device functions used by the permute kernel): the exclusive scan of the
// per-slot token counts (Section 2.1 dispatch), the slot-contiguous order of the (token, expert) pairs as two
// tables (inv: pair -> row, src_tok: row -> token), and the work-item lists of the grouped GEMM kernels.
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
    int NT;              // token rows per "thin" work item (swap-AB kernel: weight tile x up to NT token rows)
    int fat;             // 1: blocks of more than kFatMin rows go to the CTA-pair kernel (256 token rows x 256 weight rows)
    int R1, R2;          // weight tiles per group of the thin GEMM-1 / GEMM-2 items (128 rows each)
    int RF1, RF2;        // and of the fat items (GEMM-1: 128 gate + 128 up rows; GEMM-2: 256 rows)
    int32_t *offsets;    // [P + 1] out
    GemmItem *items1, *items2, *fat1, *fat2;
    int32_t *n_items;    // [4] out: thin GEMM-1, thin GEMM-2, fat GEMM-1, fat GEMM-2
};

constexpr int kFatRows = 256;    // token rows of a fat item
constexpr int kFatMin = 128;     // a block of at most this many rows is a thin item

// Stages the counts and scans them: sm[0..P] = offsets, and cnt_s (returned) = the counts.  `counts` is read
// with L1 bypassed (other CTAs' atomics produced it).
__device__ inline int32_t *stage_and_scan(int32_t *sm, const int32_t *counts, int P, int S, int32_t *warp_sums, int nthreads) {
    int32_t *cnt_s = sm + (P + 1) + 4 * (P + S + 1);
    for (int i = threadIdx.x; i < P; i += nthreads) cnt_s[i] = __ldcg(counts + i);
    __syncthreads();
    block_exclusive_scan(cnt_s, sm, P, warp_sums, nthreads);
    return cnt_s;
}

// Writes the work items of the groups g = first_warp, first_warp + warp_stride, ... (one warp per group, lanes
// over the group's items); the publishing planner also writes the offsets and the item counts.  `sm` as left by
// stage_and_scan.
//
// groups: g < S shared expert g (rows = B); g >= S slot g - S (rows = counts).  A group's rows are cut into
// blocks.  Decode-sized batches (fat = 0): blocks of NT rows, all "thin" items = one 128-row weight tile times
// the block (the weight-streaming kernel).  Prefill-sized batches (fat = 1): full blocks of 256 rows, and a
// remainder of more than 128 rows, are "fat" items for the CTA-pair kernel; a remainder of at most 128 rows
// (every adapter slot with few tokens is just that) is a thin item.  Per group the items are ordered (weight
// tile, token block) so that CTAs working at the same time share a weight tile through L2.
__device__ inline void write_items(int32_t *sm, const int32_t *cnt_s, const Params &A, int32_t *warp_sums, int nthreads,
                                   int first_warp, int warp_stride, bool publish) {
    const int P = A.P, S = A.S, B = A.B;
    const int G = P + S;
    const int32_t *off = sm;
    int32_t *blk = sm + P + 1;              // [G + 1] scan of the groups' fat blocks
    int32_t *nblk = blk + G + 1;            // [G] fat blocks
    int32_t *blk_t = nblk + G;              // [G + 1] scan of the groups' thin blocks
    int32_t *nblk_t = blk_t + G + 1;        // [G]
    const int lane = threadIdx.x & 31;
    if (publish)
        for (int i = threadIdx.x; i <= P; i += nthreads) A.offsets[i] = off[i];
    for (int g = threadIdx.x; g < G; g += nthreads) {
        const int rows = g < S ? B : cnt_s[g - S];
        if (A.fat) {
            const int rem = rows % kFatRows;
            nblk[g] = rows / kFatRows + (rem > kFatMin ? 1 : 0);
            nblk_t[g] = (rem > 0 && rem <= kFatMin) ? 1 : 0;
        } else {
            nblk[g] = 0;
            nblk_t[g] = (rows + A.NT - 1) / A.NT;
        }
    }
    __syncthreads();
    block_exclusive_scan(nblk, blk, G, warp_sums, nthreads);
    block_exclusive_scan(nblk_t, blk_t, G, warp_sums, nthreads);
    // GEMM-2 runs the S shared experts as ONE group chained along K (out[t] = sum_s Wdown_s . act_s[t] is a single
    // product over the concatenated K), so that one fp32 row per token is written and read back instead of S: the
    // shared groups 1 .. S-1 (same row count as group 0, hence the same blocks) emit no GEMM-2 items.
    const int skip_t = S > 1 ? (S - 1) * nblk_t[0] : 0, skip_f = S > 1 ? (S - 1) * nblk[0] : 0;
    const int y_base = S > 0 ? B : 0;                      // rows of Y: [0, B) the shared sum, then the routed rows
    if (publish && threadIdx.x == 0) {
        A.n_items[0] = blk_t[G] * A.R1;
        A.n_items[1] = (blk_t[G] - skip_t) * A.R2;
        A.n_items[2] = blk[G] * A.RF1;
        A.n_items[3] = (blk[G] - skip_f) * A.RF2;
    }
    for (int g = first_warp; g < G; g += warp_stride) {
        const bool shared = g < S;
        const int rows = shared ? B : cnt_s[g - S];
        if (rows == 0) continue;
        const int slot = shared ? P + g : g - S;
        const int in0 = shared ? 0 : off[g - S];                  // GEMM-1 reads x rows (shared) or slot-contiguous rows
        const int act0 = shared ? g * B : S * B + off[g - S];     // rows of act: GEMM-1 writes them, GEMM-2 reads them
        const int y0 = shared ? 0 : y_base + off[g - S];          // rows of Y
        for (int pass = 0; pass < 2; ++pass) {
            if (pass && shared && g > 0) continue;                // chained into group 0's items
            const int from_x = (!pass && shared) ? 1 : 0;
            const int in_base = pass ? act0 : in0, out_base = pass ? y0 : act0;
            const int chain = (pass && shared) ? S : 1;
            // thin items
            const int nt = nblk_t[g], Rt = pass ? A.R2 : A.R1;
            GemmItem *dst = (pass ? A.items2 : A.items1) + (size_t)(blk_t[g] - ((pass && !shared) ? skip_t : 0)) * Rt;
            const int thin0 = A.fat ? (rows / kFatRows) * kFatRows : 0;      // first row of the (only) thin block
            for (int i = lane; i < nt * Rt; i += 32) {
                const int tile = i / nt, c = i % nt;
                const int r0 = thin0 + c * A.NT;
                const int item_rows = A.fat ? rows - thin0 : min(A.NT, rows - r0);
                int4 *d4 = reinterpret_cast<int4 *>(dst + i);        // one item = two 16-byte stores
                d4[0] = make_int4(slot, tile, in_base + r0, out_base + r0);
                d4[1] = make_int4(item_rows, from_x, chain, B);
            }
            // fat items
            const int nf = nblk[g], Rf = pass ? A.RF2 : A.RF1;
            GemmItem *dstf = (pass ? A.fat2 : A.fat1) + (size_t)(blk[g] - ((pass && !shared) ? skip_f : 0)) * Rf;
            for (int i = lane; i < nf * Rf; i += 32) {
                const int tile = i / nf, c = i % nf;
                const int r0 = c * kFatRows;
                int4 *d4 = reinterpret_cast<int4 *>(dstf + i);
                d4[0] = make_int4(slot, tile, in_base + r0, out_base + r0);
                d4[1] = make_int4(min(kFatRows, rows - r0), from_x, chain, B);
            }
        }
    }
}

}  // namespace plan
}  // namespace ew
