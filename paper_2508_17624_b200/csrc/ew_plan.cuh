// Dispatch planning (device functions used by the permute kernel): the exclusive scan of the
// per-slot token counts (Section 2.1 dispatch), the slot-contiguous order of the (token, expert) pairs as two
// tables (inv: pair -> row, src_tok: row -> token), and the work-item lists of the grouped GEMM kernels.
//
// All functions are block-wide: every thread of the CTA calls them with the same arguments; `nthreads` =
// blockDim.x must be a multiple of 32 and at most 256 (derive_items: any multiple of 32).
//
// Decode-sized batches skip the planning kernel altogether ("self-planned" forwards): the router records each
// slot's tokens in a slot-major table, and every CTA of the GEMM kernels repeats the scan of the counts and derives
// its own items of the list that write_items would have written (derive_items).
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
    int B, k, P;
    int S, sh0;          // shared experts computed here: slots P + sh0 .. P + sh0 + S - 1 (all of them without expert parallelism)
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
        const int slot = shared ? P + A.sh0 + g : g - S;
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

// ---------------------------------------------------------------------------------------------------------------
// Self-planned forwards (decode-sized batches: thin items only).
struct SelfPlan {
    const int32_t *counts;       // [P] per-slot pair counts of the router kernel; null: walk the planner's item list
    int B, k, P;
    int S, sh0;                  // shared experts computed here: slots P + sh0 .. P + sh0 + S - 1
    int nt_shift;                // token rows per item NT = 1 << nt_shift (32, 64 or 128)
    int R;                       // weight tiles per group of this GEMM
    int pass;                    // 0: GEMM-1 (+ SwiGLU), 1: GEMM-2
    int rehearse;                // GEMM-1: run the planning code once before the wait for the router kernel (see derive_items)
    int hold_dependents;         // the kernel does not release its dependent kernel early (set when that is the combine kernel)
    int release_after_wait;      // the kernel releases its dependent only after its own wait (set when that is the CTA-pair kernel of the same GEMM)
    // GEMM-1 only: its CTAs also publish what the combine step (and the debugging outputs) need
    const int32_t *slot_ids, *rank;      // [B*k] from the router kernel
    int32_t *offsets, *inv;              // out: [P + 1] exclusive scan of the counts, [B*k] pair -> slot-contiguous row
};

constexpr int kSelfMaxGroups = 1024;     // P + S of a self-planned forward: one warp scans them

// One derived item, packed: x = slot | tile << 16, y = first input row, z = first output row,
// w = rows | from_x << 8 | chain << 16.
__device__ inline GemmItem unpack_item(const int4 v, int chain_rows) {
    GemmItem it;
    it.slot = v.x & 0xffff; it.tile = (int)((uint32_t)v.x >> 16);
    it.in_row = v.y; it.out_row = v.z;
    it.rows = v.w & 0xff; it.from_x = (v.w >> 8) & 1; it.chain = (int)((uint32_t)v.w >> 16);
    it.chain_rows = chain_rows;
    return it;
}

// Shared-memory words derive_items needs as scratch (may alias memory that is only used after the call):
// offsets [P + 1], block scan [G + 1], clamped counts [P].
__host__ __device__ constexpr size_t self_plan_words(int P, int S) { return (size_t)(P + 1) + (size_t)(P + S + 1) + (size_t)P; }

// Items blockIdx.x, blockIdx.x + gridDim.x, ... of the thin list of pass A.pass, in list order, packed into
// mine[0 .. n) (n is returned; the host has checked that n <= cap for every possible routing).  The list is the one
// write_items builds with fat = 0: groups in order (shared experts, then slots), per group (weight tile, token block);
// in GEMM-2 the shared experts form one group chained along K.  One difference: a routed GEMM-1 item's in_row indexes
// the router's slot-major token table ([P][B]: slot * B + first row of the block) instead of the row -> token table of
// the planning kernel.  With A.inv set (GEMM-1) the CTAs also write offsets and inv.
//
// The code runs once per CTA and launch, in GEMM-1 on the critical path between the router kernel's end and the first
// weight load, so it is written for latency and kept small (its instructions are cold, see below): all threads stage
// the counters in shared memory; warp `scan_warp` scans counts and token blocks with shuffles; then one thread per item
// finds its group by binary search while the other threads write inv.  Three barriers in all.
//
// `dry`: a rehearsal that writes nothing to global memory and tolerates any values in the counters.  The instructions
// are cold when a CTA gets here (every forward streams the live weights through L2 and evicts them; cold, an earlier
// form of this function took 3.5 us in GEMM-1 and 6.8 us in GEMM-2 of the decode layer against ~1 us to read a
// prepared list), so GEMM-1 rehearses it while it waits for the router kernel.
// (The rehearsal and the real call must execute the same instructions: the caller makes both from one call site in a
// loop that is not unrolled.  The function is inlined there so that the kernel's parameters stay in constant memory;
// as a separate function it received them through the stack, which cost several dependent L2 round trips.)
__device__ __forceinline__ int derive_items(int32_t *sm, const SelfPlan &A, int nthreads, int scan_warp, int4 *mine, int cap,
                                                bool dry) {
    const int P = A.P, S = A.S, B = A.B, G = P + S;
    int32_t *off = sm;                       // [P + 1] exclusive scan of the counts
    int32_t *eblk = sm + P + 1;              // [G + 1] exclusive scan of the groups' token blocks in this pass
    int32_t *cnt_s = eblk + G + 1;           // [P] the counts (clamped to [0, B]: a rehearsal may see anything)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long n_pairs = (long long)B * A.k;
    // this thread's first pair (GEMM-1): the loads go out together with the loads of the counts
    const long long q0 = (long long)blockIdx.x * nthreads + threadIdx.x;
    int my_slot = 0, my_rank = 0;
    if (A.inv && q0 < n_pairs) { my_slot = __ldcg(A.slot_ids + q0); my_rank = __ldcg(A.rank + q0); }
    // all threads: the counts, clamped to [0, B] (a rehearsal may see anything), into shared memory
    for (int i = threadIdx.x; i < P; i += nthreads) cnt_s[i] = min(max(__ldcg(A.counts + i), 0), B);
    __syncthreads();
    if (warp == scan_warp) {
        const int per = (G + 31) >> 5, g0 = lane * per, g1 = min(g0 + per, G);       // lane owns groups [g0, g1)
        const int round_up = (1 << A.nt_shift) - 1;
        int csum = 0, bsum = 0;
#pragma unroll 4
        for (int g = g0; g < g1; ++g) {
            const int rows = g < S ? B : cnt_s[g - S];
            if (g >= S) csum += rows;
            // GEMM-2: the shared experts 1 .. S-1 ride in group 0's items
            if (!(A.pass && g > 0 && g < S)) bsum += (rows + round_up) >> A.nt_shift;
        }
        int cinc = csum, binc = bsum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int c = __shfl_up_sync(0xffffffffu, cinc, o), b = __shfl_up_sync(0xffffffffu, binc, o);
            if (lane >= o) { cinc += c; binc += b; }
        }
        int crun = cinc - csum, brun = binc - bsum;
#pragma unroll 4
        for (int g = g0; g < g1; ++g) {
            const int rows = g < S ? B : cnt_s[g - S];
            eblk[g] = brun;
            if (!(A.pass && g > 0 && g < S)) brun += (rows + round_up) >> A.nt_shift;
            if (g >= S) { off[g - S] = crun; crun += rows; }
        }
        if (lane == 31) { off[P] = cinc; eblk[G] = binc; }
    }
    __syncthreads();
    const int total = eblk[G] * A.R;
    const int y_base = S > 0 ? B : 0;
    int n_mine = total > (int)blockIdx.x ? (total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    n_mine = min(n_mine, cap);
    // one thread per item, taken from the top of the CTA so that they are not the threads that write inv first
    const int j = nthreads - 1 - (int)threadIdx.x;
    for (int jj = j; jj < n_mine; jj += nthreads) {
        const int i = (int)blockIdx.x + jj * (int)gridDim.x;
        const int b = i / A.R;                                   // block coordinate: eblk[g] <= b < eblk[g + 1]
        int lo = 0, hi = G;                                      // invariant: eblk[lo] <= b < eblk[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (eblk[mid] <= b) lo = mid; else hi = mid;
        }
        const int g = lo;
        const bool shared = g < S;
        const int rows = shared ? B : cnt_s[g - S];
        const int nt = max(eblk[g + 1] - eblk[g], 1);
        const int local = i - eblk[g] * A.R;
        int tile = local, c = 0;
        if (nt > 1) { tile = local / nt; c = local - tile * nt; }
        const int r0 = c << A.nt_shift;
        const int slot = shared ? P + A.sh0 + g : g - S;
        const int act0 = shared ? g * B : S * B + off[shared ? 0 : g - S];
        const int in0 = shared ? 0 : (g - S) * B;                // routed rows: index into the slot-major token table
        const int y0 = shared ? 0 : y_base + off[shared ? 0 : g - S];
        const int in_base = A.pass ? act0 : in0, out_base = A.pass ? y0 : act0;
        const int from_x = (!A.pass && shared) ? 1 : 0, chain = (A.pass && shared) ? S : 1;
        mine[jj] = make_int4(slot | (tile << 16), in_base + r0, out_base + r0,
                             min(1 << A.nt_shift, rows - r0) | (from_x << 8) | (chain << 16));
    }
    if (A.inv) {
        if (blockIdx.x == 0 && !dry)
            for (int i = threadIdx.x; i <= P; i += nthreads) A.offsets[i] = off[i];
        for (long long q = q0; q < n_pairs; q += (long long)gridDim.x * nthreads) {
            if (q != q0) { my_slot = __ldcg(A.slot_ids + q); my_rank = __ldcg(A.rank + q); }
            // position -1: the pair belongs to another rank (expert parallelism)
            const int dest = my_rank < 0 ? -1 : off[min(max(my_slot, 0), P - 1)] + my_rank;
            if (dest < n_pairs && !dry) A.inv[q] = dest;         // always, unless the routing kernel gave up midway
        }
    }
    __syncthreads();
    return n_mine;
}

}  // namespace plan
}  // namespace ew
