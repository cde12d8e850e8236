// Grouped expert GEMMs on the 5th-generation tensor cores (tcgen05 + TMEM, operands by TMA).
//
// The grouped matrix multiplication of Section 2.1 ("GMM on the permuted tokens and the stacked
// expert weight tensor"), run unmodified over the virtual weight tensor of Section 4.1: the kernel
// only ever sees a slot index.  Empty slots produce no work item, so unmapped (padding) slots of the
// tensor are never touched.
//
// Orientation ("swap-AB"): the 128-row MMA dimension is a tile of the WEIGHT matrix, the MMA N
// dimension (16..256) is the token rows of one slot.  At decode a slot has a handful of rows, so the
// tensor-core tile is filled by weight rows and the kernel is a pure weight stream; at prefill N
// grows to 256 and the same instruction shape runs at full rate.
//
//   GEMM-1 (GLU = true):  act[row, i] = silu(Wgate[slot][i,:] . x_row) * (Wup[slot][i,:] . x_row)   -> bf16
//                         two accumulators (gate, up) share the token operand; SwiGLU in the epilogue
//   GEMM-2 (GLU = false): y[row, o]   = Wdown[slot][o,:] . act_row                                  -> fp32
//
// One persistent CTA per SM walks the device-built item list.  Warp 0 lane 0 issues TMA loads into a
// ring of shared-memory stages, warp 1 lane 0 issues tcgen05.mma, warps 2..5 drain TMEM.  In gather
// mode (GEMM-1) four more warps fetch the token operand: eight threads copy one 128-byte piece of a
// row of x, found through the row -> token table of the permute step, into the 128-byte-swizzled
// stage with 16-byte cp.async, so no permuted copy of x exists in memory (Section 2.1's "permute"
// folded into the GEMM's operand load).  Every barrier wait is bounded in time: on expiry the CTA raises bit 1 of the device error word, stops
// issuing work, lets its copies in flight land, frees its TMEM and returns.
#include <cuda_bf16.h>

#include "ew_internal.h"
#include "ew_tc.cuh"

namespace ew {
namespace {
using namespace tc;

constexpr int kThreads = 192;
constexpr int kGatherThreads = 128;  // gather mode: one more warpgroup, one thread per token row of the block
constexpr int kTileRows = 128;      // weight rows per tile = MMA M
constexpr int kATileBytes = kTileRows * kBlockK * 2;   // 16 KiB
constexpr int kSmemBudget = 227 * 1024 - 2048;

template <int NT, bool GLU>
struct Cfg {
    static constexpr int kStageBytes = (GLU ? 2 : 1) * kATileBytes + NT * kBlockK * 2;
    static constexpr int kStagesRaw = kSmemBudget / kStageBytes;
    static constexpr int kStages = kStagesRaw > 8 ? 8 : kStagesRaw;
    static constexpr int kAccCols = (GLU ? 2 : 1) * NT;                  // TMEM columns per accumulator set
    static constexpr int kAccStages = (2 * kAccCols <= 512) ? 2 : 1;
    static constexpr int kTmemColsRaw = kAccCols * kAccStages;
    static constexpr int kTmemCols = kTmemColsRaw <= 32 ? 32 : kTmemColsRaw <= 64 ? 64 : kTmemColsRaw <= 128 ? 128
                                     : kTmemColsRaw <= 256 ? 256 : 512;
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// ------------------------------------------------------------------------------------------- kernel
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// arrives on the barrier (whose expected count already includes this arrival) once all cp.async copies issued by
// this thread so far have landed
__device__ __forceinline__ void cp_async_arrive_noinc(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// orders shared-memory writes made through the generic proxy (observed through a barrier) before the tensor
// core's reads of shared memory
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <int NT, bool GLU, bool GATHER = false>
__global__ void __launch_bounds__(GATHER ? kThreads + kGatherThreads : kThreads, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_a,
                    const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_a_big,
                    const __grid_constant__ CUtensorMap map_x_big, const GemmItem *items,
                    const int32_t *n_items_ptr, int K, int out_rows_per_slot, void *out,
                    int *err, const uint8_t *x_rows, const int32_t *src_tok) {
    static_assert(!GATHER || (GLU && NT <= kGatherThreads), "gather mode: GEMM-1, eight gather threads per token row");
    using C = Cfg<NT, GLU>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + C::kStages * C::kStageBytes);
    // barrier layout: full[kStages], empty[kStages], tmem_full[2], tmem_empty[2], then tmem base and abort flag
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * C::kStages;
    const uint32_t bar_tfull = bar_empty + 8 * C::kStages, bar_tempty = bar_tfull + 16;
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(bars + 2 * C::kStages + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (K + kBlockK - 1) / kBlockK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(bar_full + 8 * s, GATHER ? 1 + kGatherThreads : 1);        // the TMA thread, and each gather thread
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);
            mbar_init(bar_tempty + 8 * a, 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_map(&map_w);
        if (!GATHER) prefetch_map(&map_a);
        if (GLU) prefetch_map(&map_x);
    }
    if (warp == 1) {   // TMEM allocation is a whole-warp operation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"((uint32_t)C::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    // The item list and the activations come from the previous kernels: nothing of them may be read before this
    // wait.  (The pointers are deliberately not __restrict__/const-qualified read-only data: the compiler may
    // hoist such loads above the wait.)
    pdl_wait();
    const int n_items = *reinterpret_cast<const volatile int32_t *>(n_items_ptr);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < n_items && ok; w += gridDim.x) {
                const GemmItem it = items[w];
                const int nchunk = (it.rows + kChunkRows - 1) / kChunkRows;
                // thin items fetch their rows in 32-row boxes; fat ones (prefill) with one NT-row box per stage
                const bool big = NT >= 128 && it.rows > 2 * kChunkRows;
                const CUtensorMap *amap = (GLU && it.from_x) ? (big ? &map_x_big : &map_x) : (big ? &map_a_big : &map_a);
                // gather mode: only the shared experts' rows (contiguous in x) still come by TMA
                const bool tma_tokens = !GATHER || it.from_x;
                const uint32_t b_bytes = !tma_tokens ? 0 : big ? NT * kBlockK * 2 : nchunk * kChunkBytes;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!(ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1, abort_flag, err))) break;
                    const uint32_t sa = smem_base + stage * C::kStageBytes;
                    const uint32_t full = bar_full + 8 * stage;
                    mbar_expect_tx(full, (GLU ? 2 : 1) * kATileBytes + b_bytes);
                    if (GLU) {
                        tma_load_3d(sa, &map_w, kb * kBlockK, it.tile * kTileRows, it.slot * 2, full);
                        tma_load_3d(sa + kATileBytes, &map_w, kb * kBlockK, it.tile * kTileRows, it.slot * 2 + 1, full);
                    } else {
                        tma_load_3d(sa, &map_w, kb * kBlockK, it.tile * kTileRows, it.slot, full);
                    }
                    const uint32_t sb = sa + (GLU ? 2 : 1) * kATileBytes;
                    if (!tma_tokens) {
                        // the token operand of this stage is written by the gather warps
                    } else if (big) {
                        tma_load_2d(sb, amap, kb * kBlockK, it.in_row, full);
                    } else {
                        for (int c = 0; c < nchunk; ++c)
                            tma_load_2d(sb + c * kChunkBytes, amap, kb * kBlockK, it.in_row + c * kChunkRows, full);
                    }
                    if (++stage == C::kStages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < n_items && ok; w += gridDim.x) {
                const GemmItem it = items[w];
                const int n = ((it.rows + 15) >> 4) << 4;
                const uint32_t idesc = instr_desc(n);
                if (!(ok = mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1, abort_flag, err))) break;
                tc_fence_after();
                const uint32_t d0 = tmem_base + acc * C::kAccCols;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!(ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, err))) break;
                    if (GATHER) fence_proxy_async_smem();           // the token rows were written by cp.async, not by TMA
                    tc_fence_after();
                    const uint32_t sa = smem_base + stage * C::kStageBytes;
                    const uint64_t a0 = smem_desc_sw128(sa);
                    const uint64_t a1 = smem_desc_sw128(sa + kATileBytes);
                    const uint64_t b = smem_desc_sw128(sa + (GLU ? 2 : 1) * kATileBytes);
#pragma unroll
                    for (int ki = 0; ki < kBlockK / 16; ++ki) {     // 16 bf16 = 32 bytes = 2 descriptor units per step
                        const uint32_t accum = (kb | ki) ? 1u : 0u;
                        tc_mma(d0, a0 + 2 * ki, b + 2 * ki, idesc, accum);
                        if (GLU) tc_mma(d0 + NT, a1 + 2 * ki, b + 2 * ki, idesc, accum);
                    }
                    tc_commit(bar_empty + 8 * stage);   // frees the stage once these MMAs have read it
                    if (++stage == C::kStages) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                tc_commit(bar_tfull + 8 * acc);         // accumulator complete
                if (++acc == C::kAccStages) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else if (GATHER && warp >= kThreads / 32) {
        // ------------------------------------------------------------------ token gather (warps 6..9)
        // Eight consecutive threads copy one 128-byte row segment (one k-block of one token row of x) as eight
        // 16-byte chunks, so a warp instruction reads four whole 128-byte lines; thread t serves chunk t mod 8 of
        // rows t/8 + 16 i (i = 0..7).  Chunk c of row r lands where the 128-byte swizzle puts it: at chunk position
        // c ^ (r mod 8) inside the row.  Each thread's arrival on the stage's barrier fires when its copies have landed
        // (cp.async.mbarrier.arrive.noinc), so the threads never block on their own copies; the MMA thread fences
        // the generic-proxy writes against the tensor core's reads after its wait.
        const int t = (int)threadIdx.x - kThreads;
        const int chunk = t & 7, r0 = t >> 3;
        constexpr int kRowsPerThread = NT / (kGatherThreads / 8);
        uint32_t dst_off[kRowsPerThread];
#pragma unroll
        for (int i = 0; i < kRowsPerThread; ++i) {
            const int r = r0 + i * (kGatherThreads / 8);
            dst_off[i] = (uint32_t)((GLU ? 2 : 1) * kATileBytes + r * 128 + ((chunk ^ (r & 7)) << 4));
        }
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        for (int w = blockIdx.x; w < n_items && ok; w += gridDim.x) {
            const GemmItem it = items[w];
            const int n = ((it.rows + 15) >> 4) << 4;
            const uint8_t *src[kRowsPerThread];                  // rows beyond n are not read by the MMA: not fetched
#pragma unroll
            for (int i = 0; i < kRowsPerThread; ++i) {
                const int r = r0 + i * (kGatherThreads / 8);
                const int rr = min(r, it.rows - 1);               // rows it.rows..n-1 repeat the last row; never stored
                const int tok = it.from_x ? 0 : src_tok[it.in_row + rr];   // shared experts: the TMA thread loads x rows
                src[i] = x_rows + (size_t)tok * K * 2 + chunk * 16;
            }
            for (int kb = 0; kb < num_kb; ++kb) {
                if (!(ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1, abort_flag, err))) break;
                const uint32_t d = smem_base + stage * C::kStageBytes;
#pragma unroll
                for (int i = 0; i < kRowsPerThread; ++i)
                    if (!it.from_x && r0 + i * (kGatherThreads / 8) < n)
                        cp_async16(d + dst_off[i], src[i] + (size_t)kb * (kBlockK * 2));
                cp_async_arrive_noinc(bar_full + 8 * stage);      // fires when this thread's copies have landed
                if (++stage == C::kStages) { stage = 0; phase ^= 1; }
            }
        }
        cp_async_wait_all();                                      // nothing of this thread stays in flight at exit
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int lg = warp & 3;                        // TMEM lane group this warp may read
        const int row = lg * 32 + lane;                 // row inside the 128-row weight tile
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int w = blockIdx.x; w < n_items && ok; w += gridDim.x) {
            const GemmItem it = items[w];
            if (!(ok = mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag, err))) break;
            tc_fence_after();
            const uint32_t t0 = tmem_base + ((uint32_t)(lg * 32) << 16) + acc * C::kAccCols;
            const int orow = it.tile * kTileRows + row;            // output feature index
            const bool row_ok = orow < out_rows_per_slot;
            const int n = ((it.rows + 15) >> 4) << 4;
            for (int c0 = 0; c0 < n; c0 += 32) {
                uint32_t g[32], u[32];
                if (n - c0 >= 32) {
                    tc_ld32(t0 + c0, g);
                    if (GLU) tc_ld32(t0 + NT + c0, u);
                } else {
                    tc_ld16(t0 + c0, g);
                    if (GLU) tc_ld16(t0 + NT + c0, u);
                }
                tc_wait_ld();
                const int lim = min(32, it.rows - c0);
                if (row_ok) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (j < lim) {
                            const size_t o = (size_t)(it.out_row + c0 + j) * out_rows_per_slot + orow;
                            if (GLU) {
                                const float gv = __uint_as_float(g[j]), uv = __uint_as_float(u[j]);
                                const float a = __fdividef(gv, 1.f + __expf(-gv)) * uv;      // silu(g) * u; the result is rounded to bf16
                                reinterpret_cast<__nv_bfloat16 *>(out)[o] = __float2bfloat16_rn(a);
                            } else {
                                reinterpret_cast<float *>(out)[o] = __uint_as_float(g[j]);
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
            if (++acc == C::kAccStages) { acc = 0; acc_phase ^= 1; }
        }
    }

    // ---------------------------------------------------------------------- teardown
    if (*abort_flag) {                                  // let copies in flight land before the CTA's memory is reused
        long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) {}
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols)
                     : "memory");
    }
}

// ------------------------------------------------------------------------------------------- CTA-pair kernel
// Prefill variant (used for GEMM-2, whose accumulator can be double-buffered and whose tile count is even for
// the shapes at hand; for GEMM-1 it measured slower than the one-CTA kernel): the two CTAs of a cluster share one work item = 256 weight rows (two adjacent 128-row tiles,
// one per CTA) x up to 256 token rows.  tcgen05.mma.cta_group::2 (M = 256) is issued by CTA 0; each CTA stages its
// own weight tile(s) and HALF of the token rows, so the token operand crosses L2->SM once per pair instead of once
// per CTA.  Barrier protocol: TMA loads of both CTAs complete on CTA 0's "full" barrier; CTA 0's MMA thread
// releases a stage in both CTAs, and hands the accumulator to both CTAs' epilogues, with multicast commits; the
// epilogue warps of both CTAs arrive on CTA 0's "accumulator free" barrier.  All waits are bounded as above; both
// CTAs meet at a cluster barrier before and after the work loop.
constexpr int kPairTok = 256;       // token rows per item
constexpr int kPairHalf = 128;      // rows of the token box each CTA loads

template <bool GLU>
struct PairCfg {
    static constexpr int kABytes = (GLU ? 2 : 1) * kATileBytes;
    static constexpr int kStageBytes = kABytes + kPairHalf * kBlockK * 2;          // 48 KiB / 32 KiB
    static constexpr int kStages = kSmemBudget / kStageBytes > 8 ? 8 : kSmemBudget / kStageBytes;
    static constexpr int kAccCols = (GLU ? 2 : 1) * kPairTok;
    static constexpr int kAccStages = GLU ? 1 : 2;
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 256;
};

template <bool GLU>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
grouped_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_a,
                         const __grid_constant__ CUtensorMap map_x, const GemmItem *items, const int32_t *n_items_ptr,
                         int K, int out_rows_per_slot, void *out, int *err) {
    using C = PairCfg<GLU>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_al + C::kStages * C::kStageBytes);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * C::kStages;
    const uint32_t bar_tfull = bar_empty + 8 * C::kStages, bar_tempty = bar_tfull + 16;
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(bars + 2 * C::kStages + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int num_kb = (K + kBlockK - 1) / kBlockK;
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);           // CTA 0's is the one in use: its producer's expect_tx arrival
            mbar_init(bar_empty + 8 * s, 1);          // one multicast commit per phase
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);
            mbar_init(bar_tempty + 8 * a, 8);         // CTA 0's: four epilogue warps of each CTA
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_map(&map_w);
        prefetch_map(&map_a);
        if (GLU) prefetch_map(&map_x);
    }
    if (warp == 1) {   // both CTAs allocate, with the same destination offset
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                               // the peer's barriers and TMEM are ready too
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    pdl_wait();
    const int n_items = *reinterpret_cast<const volatile int32_t *>(n_items_ptr);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (each CTA: its own half)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int w = pair_id; w < n_items && ok; w += n_pairs) {
                const GemmItem it = items[w];
                const int n = ((it.rows + 15) >> 4) << 4;
                const int brow = it.in_row + (int)rank * (n >> 1);         // this CTA stages rows [rank*n/2, +n/2) of the block
                const int wrow = (it.tile * 2 + (int)rank) * kTileRows;    // and weight tile 2*pair + rank
                const CUtensorMap *amap = (GLU && it.from_x) ? &map_x : &map_a;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!(ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1, abort_flag, err))) break;
                    const uint32_t sa = smem_base + stage * C::kStageBytes;
                    const uint32_t full = leader_addr(bar_full + 8 * stage);
                    if (rank == 0) mbar_expect_tx(bar_full + 8 * stage, 2 * C::kStageBytes);
                    if (GLU) {
                        tma2_load_3d(sa, &map_w, kb * kBlockK, wrow, it.slot * 2, full);
                        tma2_load_3d(sa + kATileBytes, &map_w, kb * kBlockK, wrow, it.slot * 2 + 1, full);
                    } else {
                        tma2_load_3d(sa, &map_w, kb * kBlockK, wrow, it.slot, full);
                    }
                    tma2_load_2d(sa + C::kABytes, amap, kb * kBlockK, brow, full);
                    if (++stage == C::kStages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (CTA 0 only)
        if (lane == 0 && rank == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int w = pair_id; w < n_items && ok; w += n_pairs) {
                const GemmItem it = items[w];
                const int n = ((it.rows + 15) >> 4) << 4;
                const uint32_t idesc = instr_desc_m256(n);
                if (!(ok = mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1, abort_flag, err))) break;
                tc_fence_after();
                const uint32_t d0 = tmem_base + acc * C::kAccCols;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!(ok = mbar_wait(bar_full + 8 * stage, phase, abort_flag, err))) break;
                    tc_fence_after();
                    const uint32_t sa = smem_base + stage * C::kStageBytes;
                    const uint64_t a0 = smem_desc_sw128(sa);
                    const uint64_t a1 = smem_desc_sw128(sa + kATileBytes);
                    const uint64_t b = smem_desc_sw128(sa + C::kABytes);
#pragma unroll
                    for (int ki = 0; ki < kBlockK / 16; ++ki) {
                        const uint32_t accum = (kb | ki) ? 1u : 0u;
                        tc2_mma(d0, a0 + 2 * ki, b + 2 * ki, idesc, accum);
                        if (GLU) tc2_mma(d0 + kPairTok, a1 + 2 * ki, b + 2 * ki, idesc, accum);
                    }
                    tc2_commit_both(bar_empty + 8 * stage);
                    if (++stage == C::kStages) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                tc2_commit_both(bar_tfull + 8 * acc);
                if (++acc == C::kAccStages) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs, own 128 rows)
        const int lg = warp & 3;
        const int row = lg * 32 + lane;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int w = pair_id; w < n_items && ok; w += n_pairs) {
            const GemmItem it = items[w];
            if (!(ok = mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag, err))) break;
            tc_fence_after();
            const uint32_t t0 = tmem_base + ((uint32_t)(lg * 32) << 16) + acc * C::kAccCols;
            const int orow = (it.tile * 2 + (int)rank) * kTileRows + row;
            const bool row_ok = orow < out_rows_per_slot;
            const int n = ((it.rows + 15) >> 4) << 4;
            for (int c0 = 0; c0 < n; c0 += 32) {
                uint32_t g[32], u[32];
                if (n - c0 >= 32) {
                    tc_ld32(t0 + c0, g);
                    if (GLU) tc_ld32(t0 + kPairTok + c0, u);
                } else {
                    tc_ld16(t0 + c0, g);
                    if (GLU) tc_ld16(t0 + kPairTok + c0, u);
                }
                tc_wait_ld();
                const int lim = min(32, it.rows - c0);
                if (row_ok) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (j < lim) {
                            const size_t o = (size_t)(it.out_row + c0 + j) * out_rows_per_slot + orow;
                            if (GLU) {
                                const float gv = __uint_as_float(g[j]), uv = __uint_as_float(u[j]);
                                const float a = __fdividef(gv, 1.f + __expf(-gv)) * uv;
                                reinterpret_cast<__nv_bfloat16 *>(out)[o] = __float2bfloat16_rn(a);
                            } else {
                                reinterpret_cast<float *>(out)[o] = __uint_as_float(g[j]);
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_leader(bar_tempty + 8 * acc);
            if (++acc == C::kAccStages) { acc = 0; acc_phase ^= 1; }
        }
    }

    // ---------------------------------------------------------------------- teardown
    if (*abort_flag) {
        long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) {}
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                               // neither CTA leaves while the other may still touch it
    tc_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

template <bool GLU>
int launch_pair(ew_pool *p, const CUtensorMap &mw, const CUtensorMap &ma, const CUtensorMap &mx, const GemmItem *items,
                const int32_t *n_items, int K, int out_rows, void *out, cudaStream_t st) {
    using C = PairCfg<GLU>;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p->sm_count & ~1);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled(GLU ? 2 : 3) ? 2 : 1;
    return (int)cudaLaunchKernelEx(&cfg, grouped_gemm_pair_kernel<GLU>, mw, ma, mx, items, n_items, K, out_rows, out, p->ws.err);
}

template <int NT, bool GLU, bool GATHER = false>
int launch_one(ew_pool *p, const CUtensorMap &mw, const CUtensorMap &ma, const CUtensorMap &mx, const CUtensorMap &mab,
               const CUtensorMap &mxb, const GemmItem *items, const int32_t *n_items, int K, int out_rows, void *out,
               cudaStream_t st, const void *x_rows = nullptr) {
    using C = Cfg<NT, GLU>;
    return launch_pdl(GLU ? 2 : 3, grouped_gemm_kernel<NT, GLU, GATHER>, dim3(p->sm_count),
                      dim3(GATHER ? kThreads + kGatherThreads : kThreads), C::kSmemBytes, st, mw, ma, mx, mab, mxb, items, n_items,
                      K, out_rows, out, p->ws.err, (const uint8_t *)x_rows, (const int32_t *)p->ws.src_tok);
}

template <int NT, bool GLU, bool GATHER = false>
int setup_one() {
    return (int)cudaFuncSetAttribute(grouped_gemm_kernel<NT, GLU, GATHER>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     Cfg<NT, GLU>::kSmemBytes);
}

}  // namespace

int gemm_setup(ew_pool *) {
    int rc = 0;
    rc |= setup_one<32, true>() | setup_one<64, true>() | setup_one<128, true>() | setup_one<256, true>();
    rc |= setup_one<128, true, true>() | setup_one<64, true, true>() | setup_one<32, true, true>();
    rc |= setup_one<32, false>() | setup_one<64, false>() | setup_one<128, false>() | setup_one<256, false>();
    rc |= (int)cudaFuncSetAttribute(grouped_gemm_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairCfg<true>::kSmemBytes);
    rc |= (int)cudaFuncSetAttribute(grouped_gemm_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairCfg<false>::kSmemBytes);
    if (rc) set_last_error("cudaFuncSetAttribute(max dynamic shared memory) failed for a grouped GEMM kernel");
    return rc;
}

int launch_gemm1(ew_pool *p, int layer, const CUtensorMap &map_x, const CUtensorMap &map_x_big, const void *x, int,
                 cudaStream_t st) {
    const LayerState &L = p->layers[layer];
    const int K = p->cfg.hidden, I = p->cfg.inter;
    const Workspace &w = p->ws;
    if (p->gather && p->token_tile == 128)
        return launch_one<128, true, true>(p, L.map_w13, p->map_xp, map_x, p->map_xp_big[0], map_x_big, w.items1, w.n_items, K, I,
                                           w.act, st, x);
    if (p->gather && p->token_tile == 64)
        return launch_one<64, true, true>(p, L.map_w13, p->map_xp, map_x, p->map_xp, map_x, w.items1, w.n_items, K, I, w.act, st, x);
    if (p->gather && p->token_tile == 32)
        return launch_one<32, true, true>(p, L.map_w13, p->map_xp, map_x, p->map_xp, map_x, w.items1, w.n_items, K, I, w.act, st, x);
    switch (p->token_tile) {
        case 32: return launch_one<32, true>(p, L.map_w13, p->map_xp, map_x, p->map_xp, map_x, w.items1, w.n_items, K, I, w.act, st);
        case 64: return launch_one<64, true>(p, L.map_w13, p->map_xp, map_x, p->map_xp, map_x, w.items1, w.n_items, K, I, w.act, st);
        case 128: return launch_one<128, true>(p, L.map_w13, p->map_xp, map_x, p->map_xp_big[0], map_x_big, w.items1, w.n_items, K, I, w.act, st);
        default:
            return launch_one<256, true>(p, L.map_w13, p->map_xp, map_x, p->map_xp_big[1], map_x_big, w.items1, w.n_items, K, I, w.act, st);
    }
}

int launch_gemm2(ew_pool *p, int layer, int, cudaStream_t st) {
    const LayerState &L = p->layers[layer];
    const int K = p->cfg.inter, H = p->cfg.hidden;
    const Workspace &w = p->ws;
    const CUtensorMap &a = p->map_act;
    switch (p->token_tile2) {
        case 32: return launch_one<32, false>(p, L.map_w2, a, a, a, a, w.items2, w.n_items + 1, K, H, w.y, st);
        case 64: return launch_one<64, false>(p, L.map_w2, a, a, a, a, w.items2, w.n_items + 1, K, H, w.y, st);
        case 128: return launch_one<128, false>(p, L.map_w2, a, a, p->map_act_big[0], a, w.items2, w.n_items + 1, K, H, w.y, st);
        default:
            if (p->use_pairs) return launch_pair<false>(p, L.map_w2, p->map_act_big[0], a, w.items2, w.n_items + 1, K, H, w.y, st);
            return launch_one<256, false>(p, L.map_w2, a, a, p->map_act_big[1], a, w.items2, w.n_items + 1, K, H, w.y, st);
    }
}

}  // namespace ew
