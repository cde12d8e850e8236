// Grouped expert GEMMs on the 5th-generation tensor cores (tcgen05 + TMEM, operands by TMA).
//
// The grouped matrix multiplication of Section 2.1 ("GMM on the permuted tokens and the stacked
// expert weight tensor"), run unmodified over the virtual weight tensor of Section 4.1: the kernels
// only ever see a slot index.  Empty slots produce no work item, so unmapped (padding) slots of the
// tensor are never touched.
//
//   GEMM-1 (GLU = true):  act[row, i] = silu(Wgate[slot][i,:] . x_row) * (Wup[slot][i,:] . x_row)   -> bf16
//   GEMM-2 (GLU = false): y[row, o]   = Wdown[slot][o,:] . act_row                                  -> fp32
//
// Two kernels, picked per block of token rows by the planner:
//
// grouped_gemm_kernel ("thin" items, up to 128 token rows; every item of a decode-sized batch).  Orientation
//   "swap-AB": the 128-row MMA dimension is a tile of the WEIGHT matrix, the MMA N dimension (16..128) is the
//   token rows of the block.  A slot with a handful of rows still fills the tensor-core tile with weight rows,
//   and the kernel is a pure weight stream.  Gate and up tiles share the token operand and accumulate into two
//   TMEM regions, SwiGLU is a per-lane epilogue.  One persistent CTA per SM walks the device-built item list.
//   Warp 0 lane 0 issues TMA loads into a ring of shared-memory stages, warp 1 lane 0 issues tcgen05.mma,
//   warps 2..5 drain TMEM.  In GEMM-1 four more warps fetch the token operand: eight threads copy one 128-byte
//   piece of a row of x, found through the row -> token table of the permute step, into the 128-byte-swizzled
//   stage with 16-byte cp.async, so no permuted copy of x exists in memory (Section 2.1's "permute" folded into
//   the GEMM's operand load).
//
// fat_gemm_kernel ("fat" items, 129..256 token rows; prefill-sized batches).  Standard orientation on a CTA pair
//   (tcgen05.mma.cta_group::2): the 256-row MMA dimension is the token block, 128 rows per CTA; the MMA N
//   dimension is 256 weight rows, 128 staged by each CTA - in GEMM-1 CTA 0 stages a 128-row gate tile and CTA 1
//   the matching up tile, so a token's gate and up values sit in columns j and 128 + j of its own TMEM lane and
//   SwiGLU stays a per-lane epilogue; in GEMM-2 the two CTAs stage adjacent 128-row tiles of Wdown.  Every weight
//   tile is read once per 256 tokens, each thread of the epilogue owns one token row and writes it with 16-byte
//   stores, and two 256-column accumulator sets let the epilogue of one item overlap the MMAs of the next.
//
// Every barrier wait is bounded in time: on expiry the CTA raises bit 1 of the device error word, stops
// issuing work, lets its copies in flight land, frees its TMEM and returns.
#include <cuda_bf16.h>

#include <cstdlib>

#include "ew_internal.h"
#include "ew_plan.cuh"
#include "ew_tc.cuh"

namespace ew {
namespace {
using namespace tc;

constexpr int kThreads = 192;
constexpr int kGatherThreads = 128;  // GEMM-1: one more warpgroup that gathers the token rows
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
    static constexpr int kRingBytes = kStages * kStageBytes;
    // self-planned forwards: the CTA's own items, 16 bytes each, behind the barriers (as many as the CTA's shared memory leaves)
    static constexpr int kSelfCapRaw = (227 * 1024 - kRingBytes - 1024 - 256) / 16;
    static constexpr int kSelfCap = kSelfCapRaw > 256 ? 256 : kSelfCapRaw;
    static constexpr int kSmemBytes = kRingBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kSelfCap * 16;
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

template <int NT, bool GLU>
__global__ void __launch_bounds__(GLU ? kThreads + kGatherThreads : kThreads, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_a,
                    const __grid_constant__ CUtensorMap map_a_big, const GemmItem *items,
                    const int32_t *n_items_ptr, int K, int out_rows_per_slot, void *out,
                    int *err, const uint8_t *x_rows, const int32_t *src_tok, int n_x_rows, const plan::SelfPlan sp) {
    // GEMM-1 gathers its token rows from x (shared experts: TMA boxes of x through map_a / map_a_big);
    // GEMM-2 reads the activation rows GEMM-1 wrote through map_a / map_a_big
    constexpr bool GATHER = GLU;
    static_assert(NT <= kGatherThreads, "eight gather threads per token row");
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
    int4 *self_items = reinterpret_cast<int4 *>(smem_al + C::kRingBytes + 256);     // [kSelfCap]

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
        prefetch_map(&map_a);
    }
    if (warp == 1) {   // TMEM allocation is a whole-warp operation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"((uint32_t)C::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Self-planned forwards (no planning kernel ran): this CTA's items are derived from the router's counts, with the
    // ring - not yet in use - as scratch.  GEMM-1 does that after its wait for the router kernel (and rehearses it
    // before, see derive_items) and only then releases GEMM-2; GEMM-2 therefore starts with the counts final and plans
    // while it waits for GEMM-1's last CTAs.
    const bool self = sp.counts != nullptr;
    constexpr int kScanWarp = 2;
    int n_mine = 0;
    // GEMM-1 of a self-planned forward releases GEMM-2 after its own wait (below).  GEMM-2 of such a forward does not
    // release the combine kernel early at all (it is launched when GEMM-2 has finished): with the combine kernel's
    // CTAs resident beside GEMM-2's, the decode layer measured 0.2876 instead of 0.2815 ms.
    if (!self && !sp.hold_dependents && !sp.release_after_wait) pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    // The item list and the activations come from the previous kernels: nothing of them may be read before this
    // wait.  (The pointers are deliberately not __restrict__/const-qualified read-only data: the compiler may
    // hoist such loads above the wait.)
    if (self) {
        // one call site, executed twice by GEMM-1 (rehearsal before the wait, then for real) and once by GEMM-2
        // (for real, before the wait)
#pragma unroll 1
        for (int rep = (GLU && sp.rehearse) ? 0 : 1; rep < 2; ++rep) {
            if (GLU && rep == 1) {
                pdl_wait();
                pdl_launch_dependents();
            }
            n_mine = plan::derive_items(reinterpret_cast<int32_t *>(smem_al), sp, (int)blockDim.x, kScanWarp, self_items, C::kSelfCap,
                                        GLU && rep == 0);
        }
        if (!GLU) {
            pdl_wait();
        }
    } else {
        // every gridDim.x-th item of the planning kernel's list
        pdl_wait();
        if (sp.release_after_wait) pdl_launch_dependents();     // the CTA-pair kernel of this GEMM may start without a wait of its own
        const int n_items = *reinterpret_cast<const volatile int32_t *>(n_items_ptr);
        n_mine = n_items > (int)blockIdx.x ? (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    }
    // this CTA's j-th item
    auto item_at = [&](int j) -> GemmItem {
        if (self) return plan::unpack_item(self_items[j], sp.B);
        return items[blockIdx.x + (size_t)j * gridDim.x];
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int w = 0; w < n_mine && ok; ++w) {
                const GemmItem it = item_at(w);
                const int nchunk = (it.rows + kChunkRows - 1) / kChunkRows;
                // thin items fetch their rows in 32-row boxes; fat ones (prefill) with one NT-row box per stage
                const bool big = NT >= 128 && it.rows > 2 * kChunkRows;
                const CUtensorMap *amap = big ? &map_a_big : &map_a;
                // GEMM-1: only the shared experts' rows (contiguous in x) come by TMA
                const bool tma_tokens = !GATHER || it.from_x;
                const uint32_t b_bytes = !tma_tokens ? 0 : big ? NT * kBlockK * 2 : nchunk * kChunkBytes;
                // GEMM-2 of the shared experts: the K loop runs over it.chain experts (slot, slot + 1, ...) whose
                // activation blocks lie it.chain_rows rows apart
                const int n_stage = (GLU ? 1 : it.chain) * num_kb;
                for (int st = 0, kb = 0, ch = 0; st < n_stage; ++st) {
                    if (!(ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1, abort_flag, err))) break;
                    const uint32_t sa = smem_base + stage * C::kStageBytes;
                    const uint32_t full = bar_full + 8 * stage;
                    const int in_row = it.in_row + ch * it.chain_rows;
                    mbar_expect_tx(full, (GLU ? 2 : 1) * kATileBytes + b_bytes);
                    if (GLU) {
                        tma_load_3d(sa, &map_w, kb * kBlockK, it.tile * kTileRows, it.slot * 2, full);
                        tma_load_3d(sa + kATileBytes, &map_w, kb * kBlockK, it.tile * kTileRows, it.slot * 2 + 1, full);
                    } else {
                        tma_load_3d(sa, &map_w, kb * kBlockK, it.tile * kTileRows, it.slot + ch, full);
                    }
                    const uint32_t sb = sa + (GLU ? 2 : 1) * kATileBytes;
                    if (!tma_tokens) {
                        // the token operand of this stage is written by the gather warps
                    } else if (big) {
                        tma_load_2d(sb, amap, kb * kBlockK, in_row, full);
                    } else {
                        for (int c = 0; c < nchunk; ++c)
                            tma_load_2d(sb + c * kChunkBytes, amap, kb * kBlockK, in_row + c * kChunkRows, full);
                    }
                    if (++stage == C::kStages) { stage = 0; phase ^= 1; }
                    if (++kb == num_kb) { kb = 0; ++ch; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int w = 0; w < n_mine && ok; ++w) {
                const GemmItem it = item_at(w);
                const int n = ((it.rows + 15) >> 4) << 4;
                const uint32_t idesc = instr_desc(n);
                if (!(ok = mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1, abort_flag, err))) break;
                tc_fence_after();
                const uint32_t d0 = tmem_base + acc * C::kAccCols;
                const int n_stage = (GLU ? 1 : it.chain) * num_kb;
                for (int kb = 0; kb < n_stage; ++kb) {
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
        for (int w = 0; w < n_mine && ok; ++w) {
            const GemmItem it = item_at(w);
            const int n = ((it.rows + 15) >> 4) << 4;
            const uint8_t *src[kRowsPerThread];                  // rows beyond n are not read by the MMA: not fetched
#pragma unroll
            for (int i = 0; i < kRowsPerThread; ++i) {
                const int r = r0 + i * (kGatherThreads / 8);
                const int rr = min(r, it.rows - 1);               // rows it.rows..n-1 repeat the last row; never stored
                int tok = it.from_x ? 0 : src_tok[it.in_row + rr];         // shared experts: the TMA thread loads x rows
                // a routing kernel that gave up on a wait leaves rows of the table from an earlier, larger batch
                tok = min(max(tok, 0), n_x_rows - 1);
                src[i] = x_rows + (size_t)tok * K * 2 + chunk * 16;
            }
            for (int kb = 0; kb < num_kb; ++kb) {
                if (!(ok = mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1, abort_flag, err))) break;
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
        for (int w = 0; w < n_mine && ok; ++w) {
            const GemmItem it = item_at(w);
            if (!(ok = mbar_wait_warp(bar_tfull + 8 * acc, acc_phase, abort_flag, err))) break;
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
// Fat items: 129..256 token rows x 256 weight rows on a cluster of two CTAs (tcgen05.mma.cta_group::2, M = 256,
// N = 256), issued by CTA 0.  Operand A (M side) = the token block, rows [128 r, 128 r + 128) staged by CTA r;
// operand B (N side) = weight rows, columns [128 r, 128 r + 128) of the accumulator staged by CTA r: the gate tile
// (r = 0) and the up tile (r = 1) of the same 128 output features in GEMM-1, two adjacent 128-row tiles of Wdown in
// GEMM-2.  Each CTA's TMEM holds its own 128 token rows x all 256 columns, twice (two accumulator sets).
//
// Barrier protocol.  full[s] (CTA 0's is the one in use): TMA bytes of both CTAs complete there.  In GEMM-1 the
// gather threads of a CTA arrive on that CTA's own gath[s] as their cp.async copies land (cp.async can only signal
// a barrier of its own CTA); a relay thread per CTA waits for gath[s], issues the proxy fence that orders those
// generic-proxy writes before the tensor core's reads, and arrives on full[s].  (The fence is kept off the MMA
// thread on purpose: there it made the thread wait for its own MMAs in flight at every stage.)
// CTA 0's MMA thread releases a stage in both CTAs, and hands an accumulator set to both CTAs' epilogues, with
// multicast commits; the epilogue warps of both CTAs arrive on CTA 0's "accumulator free" barrier.  All waits are
// bounded; both CTAs meet at a cluster barrier before and after the work loop.
constexpr int kFatHalf = 128;
constexpr int kFatN = 256;          // accumulator columns per set

// GEMM-1 (GLU) stages its bf16 output rows through shared memory (see the epilogue); GEMM-2 writes its fp32 rows
// straight from registers with 32-byte stores and spends that shared memory on a seventh stage instead (its time fell
// with every stage added: 511 / 491 / 476 us at 4 / 5 / 6 stages of the prefill layer, while GEMM-1 did not react).
template <bool GLU>
struct FatCfg {
    static constexpr int kStageBytes = 2 * kATileBytes;                         // 16 KiB of token rows + 16 KiB of weight rows
    static constexpr int kOutRowBytes = 128 + 16;                               // epilogue staging: 128 bytes of a row, padded against bank conflicts
    static constexpr int kOutBytes = GLU ? 4 * 32 * kOutRowBytes : 0;           // 32 rows per epilogue warp
    static constexpr int kStages = (kSmemBudget - kOutBytes) / kStageBytes > 8 ? 8 : (kSmemBudget - kOutBytes) / kStageBytes;   // 6 / 7
    static constexpr int kSmemBytes = kStages * kStageBytes + kOutBytes + 1024 + 512;
};
constexpr int kFatThreadsGlu = kThreads + kGatherThreads + 32;                  // GEMM-1: gather warps and a relay warp

__device__ __forceinline__ bool mbar_try_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait on a barrier that receives arrivals from the peer CTA (acquire at cluster scope)
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *err) {
    if (mbar_try_cluster(bar, parity)) return true;
    long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_cluster(bar, parity)) return true;
        if ((it & 63u) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitLimitCycles) {
                *abort_flag = 1;
                atomicOr(err, 2);
                return false;
            }
        }
    }
}

template <bool GLU>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GLU ? kFatThreadsGlu : kThreads, 1)
fat_gemm_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_a,
                const GemmItem *items, const int32_t *n_items_ptr, int K, int out_cols, void *out, int *err,
                const uint8_t *x_rows, const int32_t *src_tok, int n_x_rows, int early_start) {
    using C = FatCfg<GLU>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
    uint8_t *out_stage = smem_al + C::kStages * C::kStageBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(out_stage + C::kOutBytes);
    // barrier layout: full[kStages], empty[kStages], gath[kStages], tmem_full[2], tmem_empty[2], tmem base, abort flag
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * C::kStages, bar_gath = bar_empty + 8 * C::kStages;
    const uint32_t bar_tfull = bar_gath + 8 * C::kStages, bar_tempty = bar_tfull + 16;
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(bars + 3 * C::kStages + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int num_kb = (K + kBlockK - 1) / kBlockK;
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            // CTA 0's full barrier: its producer's expect_tx arrival; in GEMM-1 also the relay thread of each CTA
            mbar_init(bar_full + 8 * s, GLU ? 3 : 1);
            mbar_init(bar_empty + 8 * s, 1);              // one multicast commit per phase
            mbar_init(bar_gath + 8 * s, kGatherThreads);  // this CTA's gather threads (GEMM-1)
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);
            mbar_init(bar_tempty + 8 * a, 8);             // CTA 0's: four epilogue warps of each CTA
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_map(&map_w);
        prefetch_map(&map_a);
    }
    if (warp == 1) {   // both CTAs allocate, with the same destination offset
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    if (GLU) pdl_launch_dependents();                 // (variant: GEMM-2's pair kernel does not release the combine kernel early)
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                               // the peer's barriers and TMEM are ready too
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    // The item list and the activations come from earlier kernels.  early_start: the weight-streaming kernel of the same
    // GEMM, this kernel's predecessor, released it only after its own wait (so everything before THAT kernel is
    // complete, which is all this kernel reads) and still works on its last items: this kernel starts on the SMs it has
    // left instead of idling through its tail, and waits for it at the end, so that whoever comes next can rely on both.
    if (!early_start) pdl_wait();
    const int n_items = *reinterpret_cast<const volatile int32_t *>(n_items_ptr);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (each CTA: its own halves)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int w = pair_id; w < n_items && ok; w += n_pairs) {
                const GemmItem it = items[w];
                const int arow = it.in_row + (int)rank * kFatHalf;          // this CTA's 128 token rows
                const bool tma_tokens = !GLU || it.from_x;                  // GEMM-1: only the shared experts' rows of x
                // GEMM-1: CTA 0 stages the gate tile, CTA 1 the up tile; GEMM-2: adjacent tiles of Wdown
                const int wrow = GLU ? it.tile * kTileRows : (it.tile * 2 + (int)rank) * kTileRows;
                const int wz = GLU ? it.slot * 2 + (int)rank : it.slot;
                const uint32_t bytes = (uint32_t)(2 * kATileBytes + (tma_tokens ? 2 * kATileBytes : 0));   // of both CTAs
                const int n_stage = (GLU ? 1 : it.chain) * num_kb;           // GEMM-2 of the shared experts: chained along K
                for (int st = 0, kb = 0, ch = 0; st < n_stage; ++st) {
                    if (!(ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1, abort_flag, err))) break;
                    const uint32_t sa = smem_base + stage * C::kStageBytes;
                    const uint32_t full = leader_addr(bar_full + 8 * stage);
                    if (rank == 0) mbar_expect_tx(bar_full + 8 * stage, bytes);
                    tma2_load_3d(sa + kATileBytes, &map_w, kb * kBlockK, wrow, wz + (GLU ? 0 : ch), full);
                    if (tma_tokens) tma2_load_2d(sa, &map_a, kb * kBlockK, arow + ch * it.chain_rows, full);
                    if (++stage == C::kStages) { stage = 0; phase ^= 1; }
                    if (++kb == num_kb) { kb = 0; ++ch; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // -------------------------------------------------------------- MMA issuer (CTA 0)
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            const uint32_t idesc = instr_desc_m256(kFatN);
            bool ok = true;
            for (int w = pair_id; w < n_items && ok; w += n_pairs) {
                const int n_stage = (GLU ? 1 : items[w].chain) * num_kb;
                if (!(ok = mbar_wait_cluster(bar_tempty + 8 * acc, acc_phase ^ 1, abort_flag, err))) break;
                tc_fence_after();
                const uint32_t d0 = tmem_base + acc * kFatN;
                for (int kb = 0; kb < n_stage; ++kb) {
                    if (!(ok = mbar_wait_cluster(bar_full + 8 * stage, phase, abort_flag, err))) break;
                    tc_fence_after();
                    const uint32_t sa = smem_base + stage * C::kStageBytes;
                    const uint64_t a = smem_desc_sw128(sa), b = smem_desc_sw128(sa + kATileBytes);
#pragma unroll
                    for (int ki = 0; ki < kBlockK / 16; ++ki) tc2_mma(d0, a + 2 * ki, b + 2 * ki, idesc, (kb | ki) ? 1u : 0u);
                    tc2_commit_both(bar_empty + 8 * stage);
                    if (++stage == C::kStages) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                tc2_commit_both(bar_tfull + 8 * acc);
                if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else if (GLU && warp == (kThreads + kGatherThreads) / 32) {
        // ------------------------------------------------------------------ relay (warp 10 of both CTAs)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int w = pair_id; w < n_items && ok; w += n_pairs) {
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!(ok = mbar_wait(bar_gath + 8 * stage, phase, abort_flag, err))) break;
                    fence_proxy_async_smem();                       // generic-proxy writes -> the tensor core's reads
                    mbar_arrive_leader(bar_full + 8 * stage);
                    if (++stage == C::kStages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (GLU && warp >= kThreads / 32) {
        // ------------------------------------------------------------------ token gather (warps 6..9 of both CTAs)
        // Eight consecutive threads copy one 128-byte row segment (one k-block of one token row of x) as eight
        // 16-byte chunks; thread t serves chunk t mod 8 of rows t/8 + 16 i (i = 0..7) of this CTA's half of the
        // block.  Chunk c of row r lands at chunk position c ^ (r mod 8) of the row (128-byte swizzle).
        const int t = (int)threadIdx.x - kThreads;
        const int chunk = t & 7, r0 = t >> 3;
        constexpr int kRowsPerThread = kFatHalf / (kGatherThreads / 8);    // 8
        uint32_t dst_off[kRowsPerThread];
#pragma unroll
        for (int i = 0; i < kRowsPerThread; ++i) {
            const int r = r0 + i * (kGatherThreads / 8);
            dst_off[i] = (uint32_t)(r * 128 + ((chunk ^ (r & 7)) << 4));
        }
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        for (int w = pair_id; w < n_items && ok; w += n_pairs) {
            const GemmItem it = items[w];
            const uint8_t *src[kRowsPerThread];
            bool live[kRowsPerThread];                               // rows past the item's last one are not fetched (nor stored later)
#pragma unroll
            for (int i = 0; i < kRowsPerThread; ++i) {
                const int rr = (int)rank * kFatHalf + r0 + i * (kGatherThreads / 8);
                live[i] = !it.from_x && rr < it.rows;
                int tok = live[i] ? src_tok[it.in_row + rr] : 0;
                tok = min(max(tok, 0), n_x_rows - 1);                // stale table rows after an aborted routing kernel
                src[i] = x_rows + (size_t)tok * K * 2 + chunk * 16;
            }
            for (int kb = 0; kb < num_kb; ++kb) {
                if (!(ok = mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1, abort_flag, err))) break;
                const uint32_t d = smem_base + stage * C::kStageBytes;
#pragma unroll
                for (int i = 0; i < kRowsPerThread; ++i)
                    if (live[i]) cp_async16(d + dst_off[i], src[i] + (size_t)kb * (kBlockK * 2));
                cp_async_arrive_noinc(bar_gath + 8 * stage);         // fires when this thread's copies have landed
                if (++stage == C::kStages) { stage = 0; phase ^= 1; }
            }
        }
        cp_async_wait_all();
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5 of both CTAs)
        // thread <-> token row: TMEM lane lg*32 + lane of this CTA = row rank*128 + lg*32 + lane of the item.  A thread
        // holds 32 consecutive output columns of its row; written straight to memory that would be 32 different lines
        // per store instruction, so each warp passes 128 bytes of its 32 rows through shared memory and stores them
        // with eight lanes per row (four whole 128-byte pieces per instruction).
        const int lg = warp & 3;
        uint8_t *stg = out_stage + lg * 32 * C::kOutRowBytes;                // (GEMM-1 only; GEMM-2 has no staging area)
        uint8_t *stg_w = stg + lane * C::kOutRowBytes;                       // this thread's row of the staging tile
        const uint8_t *stg_r = stg + (lane >> 3) * C::kOutRowBytes + (lane & 7) * 16;   // row lane/8 (+4 per step), 16-byte piece lane%8
        constexpr int kElem = GLU ? 2 : 4;                                   // bytes per output element
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int w = pair_id; w < n_items && ok; w += n_pairs) {
            const GemmItem it = items[w];
            if (!(ok = mbar_wait_warp(bar_tfull + 8 * acc, acc_phase, abort_flag, err))) break;
            tc_fence_after();
            const uint32_t t0 = tmem_base + ((uint32_t)(lg * 32) << 16) + acc * kFatN;
            const int row0 = (int)rank * kFatHalf + lg * 32;                 // first row of this warp inside the item
            const int rows_here = min(32, it.rows - row0);                   // <= 0: nothing of this warp's rows exists
            if (rows_here > 0) {
                const int f0 = it.tile * (GLU ? kTileRows : kFatN);          // first output feature of this item
                const int n_feat = min(GLU ? kTileRows : kFatN, out_cols - f0);
                uint8_t *gbase = reinterpret_cast<uint8_t *>(out) + ((size_t)(it.out_row + row0) * out_cols + f0) * kElem;
                const size_t row_bytes = (size_t)out_cols * kElem;
                constexpr int kPieceElems = 128 / kElem;                     // output elements per 128-byte piece: 64 bf16 / 32 fp32
#pragma unroll 1
                for (int e0 = 0; e0 < n_feat; e0 += kPieceElems) {
                    if (GLU) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            uint32_t g[32], u[32];
                            tc_ld32(t0 + e0 + 32 * h, g);
                            tc_ld32(t0 + kTileRows + e0 + 32 * h, u);
                            tc_wait_ld();
                            uint32_t pk[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float g0 = __uint_as_float(g[2 * j]), g1 = __uint_as_float(g[2 * j + 1]);
                                const float a0 = __fdividef(g0, 1.f + __expf(-g0)) * __uint_as_float(u[2 * j]);
                                const float a1 = __fdividef(g1, 1.f + __expf(-g1)) * __uint_as_float(u[2 * j + 1]);
                                const __nv_bfloat162 v = __floats2bfloat162_rn(a0, a1);   // silu(g) * u, rounded to bf16
                                pk[j] = *reinterpret_cast<const uint32_t *>(&v);
                            }
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                *reinterpret_cast<uint4 *>(stg_w + 64 * h + 16 * q) = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
                        }
                    } else {
                        // GEMM-2: the thread's 32 fp32 columns (128 bytes of its row) go out as four 32-byte stores, whole
                        // sectors each; no staging
                        uint32_t v[32];
                        tc_ld32(t0 + e0, v);
                        tc_wait_ld();
                        if (lane < rows_here) {
                            uint8_t *gp = gbase + (size_t)lane * row_bytes + (size_t)e0 * kElem;
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(gp + 32 * q), "r"(v[8 * q]),
                                             "r"(v[8 * q + 1]), "r"(v[8 * q + 2]), "r"(v[8 * q + 3]), "r"(v[8 * q + 4]), "r"(v[8 * q + 5]),
                                             "r"(v[8 * q + 6]), "r"(v[8 * q + 7])
                                             : "memory");
                        }
                        continue;
                    }
                    __syncwarp();
                    // eight lanes per row: lane l writes bytes [16 (l%8), +16) of row l/8 + 4 i
                    const int piece_elems_ok = n_feat - e0;                  // elements of this piece that exist (a multiple of 8)
                    const bool col_ok = (lane & 7) * (16 / kElem) < piece_elems_ok;
                    uint8_t *gp = gbase + (size_t)(lane >> 3) * row_bytes + (size_t)e0 * kElem + (lane & 7) * 16;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint4 val = *reinterpret_cast<const uint4 *>(stg_r + 4 * i * C::kOutRowBytes);
                        if (col_ok && (lane >> 3) + 4 * i < rows_here) *reinterpret_cast<uint4 *>(gp + (size_t)(4 * i) * row_bytes) = val;
                    }
                    __syncwarp();
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_leader(bar_tempty + 8 * acc);
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
    }

    // ---------------------------------------------------------------------- teardown
    if (*abort_flag) {
        long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) {}
    }
    if (early_start) pdl_wait();                      // this grid is complete only when its predecessor is
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                               // neither CTA leaves while the other may still touch it
    tc_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

// EW_DISABLE_TAIL_OVERLAP=1: the CTA-pair kernel waits for the weight-streaming kernel of its GEMM before it starts.
bool tail_overlap_enabled() {
    static const bool on = [] { const char *e = getenv("EW_DISABLE_TAIL_OVERLAP"); return !(e && e[0] == '1'); }();
    return on;
}

template <bool GLU>
int launch_fat(ew_pool *p, const CUtensorMap &mw, const CUtensorMap &ma, const GemmItem *items, const int32_t *n_items, int K,
               int out_cols, void *out, cudaStream_t st, const void *x_rows, int n_x_rows) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p->sm_count & ~1);
    cfg.blockDim = dim3(GLU ? kFatThreadsGlu : kThreads);
    cfg.dynamicSmemBytes = FatCfg<GLU>::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
    // (with the launch overlap switched off the kernels run one after the other anyway)
    return (int)cudaLaunchKernelEx(&cfg, fat_gemm_kernel<GLU>, mw, ma, items, n_items, K, out_cols, out, p->ws.err,
                                   (const uint8_t *)x_rows, (const int32_t *)p->ws.src_tok, n_x_rows, tail_overlap_enabled() ? 1 : 0);
}

template <int NT, bool GLU>
int launch_one(ew_pool *p, const CUtensorMap &mw, const CUtensorMap &ma, const CUtensorMap &mab, const GemmItem *items,
               const int32_t *n_items, int K, int out_rows, void *out, cudaStream_t st, const void *x_rows, int n_x_rows,
               const plan::SelfPlan &sp) {
    using C = Cfg<NT, GLU>;
    // self-planned forwards read the router's slot-major token table instead of the planning kernel's row -> token table
    const int32_t *tok_table = sp.counts ? p->ws.slot_tok : p->ws.src_tok;
    return launch_pdl(grouped_gemm_kernel<NT, GLU>, dim3(p->sm_count), dim3(GLU ? kThreads + kGatherThreads : kThreads),
                      C::kSmemBytes, st, mw, ma, mab, items, n_items, K, out_rows, out, p->ws.err, (const uint8_t *)x_rows,
                      tok_table, n_x_rows, sp);
}

template <int NT, bool GLU>
void self_limits(int *cap, size_t *scratch_bytes) {
    *cap = Cfg<NT, GLU>::kSelfCap;
    *scratch_bytes = Cfg<NT, GLU>::kRingBytes;
}

plan::SelfPlan self_plan_args(const ew_pool *p, int B, int pass) {
    plan::SelfPlan sp = {};
    sp.hold_dependents = (pass == 1 && !p->fat) ? 1 : 0;      // GEMM-2's weight-streaming kernel followed by the combine kernel
    sp.release_after_wait = (p->fat && tail_overlap_enabled()) ? 1 : 0;   // followed by the CTA-pair kernel of the same GEMM
    if (!p->self_plan) return sp;
    const ew_config_t &c = p->cfg;
    sp.counts = p->ws.counts;
    sp.B = B; sp.k = c.top_k; sp.P = p->P; sp.S = p->sh_hi - p->sh_lo; sp.sh0 = p->sh_lo;
    sp.nt_shift = p->token_tile == 32 ? 5 : p->token_tile == 64 ? 6 : 7;
    sp.R = ((pass ? c.hidden : c.inter) + 127) / 128;
    sp.pass = pass;
    // per-kernel profiling puts events between the kernels: nothing runs beside the router kernel then, and a
    // rehearsal would only be added to GEMM-1's measured time
    sp.rehearse = p->profiling_this_forward ? 0 : 1;
    if (!pass) { sp.slot_ids = p->ws.slot_ids; sp.rank = p->ws.rank; sp.offsets = p->ws.offsets; sp.inv = p->ws.inv; }
    return sp;
}

template <int NT, bool GLU>
int setup_one() {
    return (int)cudaFuncSetAttribute(grouped_gemm_kernel<NT, GLU>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     Cfg<NT, GLU>::kSmemBytes);
}

}  // namespace

// Whether a forward of B tokens with NT-row items can run without the planning kernel: every CTA of the GEMM kernels
// must be able to hold its own items (whatever the routing turns out to be) and the planning scratch in shared memory.
bool self_plan_fits(const ew_pool *p, int B, int NT) {
    const ew_config_t &c = p->cfg;
    int cap1, cap2;
    size_t scr1, scr2;
    switch (NT) {
        case 32: self_limits<32, true>(&cap1, &scr1); self_limits<32, false>(&cap2, &scr2); break;
        case 64: self_limits<64, true>(&cap1, &scr1); self_limits<64, false>(&cap2, &scr2); break;
        default: self_limits<128, true>(&cap1, &scr1); self_limits<128, false>(&cap2, &scr2); break;
    }
    const size_t need = plan::self_plan_words(p->P, c.num_shared) * 4;      // (fewer shared experts with expert parallelism)
    if (need > scr1 || need > scr2 || p->P + c.num_shared > plan::kSelfMaxGroups) return false;
    // token blocks of any routing: at most floor(B k / NT) full ones plus one ragged block per live slot, plus the shared experts'
    const long long pairs = (long long)B * c.top_k;
    const long long blocks = pairs / NT + (pairs < p->P ? pairs : p->P) + (long long)c.num_shared * ((B + NT - 1) / NT);
    const long long R1 = (c.inter + 127) / 128, R2 = (c.hidden + 127) / 128;
    const long long per1 = (blocks * R1 + p->sm_count - 1) / p->sm_count, per2 = (blocks * R2 + p->sm_count - 1) / p->sm_count;
    return per1 <= cap1 && per2 <= cap2 && R1 < 65536 && R2 < 65536;
}

int gemm_setup(ew_pool *) {
    int rc = 0;
    rc |= setup_one<32, true>() | setup_one<64, true>() | setup_one<128, true>();
    rc |= setup_one<32, false>() | setup_one<64, false>() | setup_one<128, false>();
    rc |= (int)cudaFuncSetAttribute(fat_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FatCfg<true>::kSmemBytes);
    rc |= (int)cudaFuncSetAttribute(fat_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FatCfg<false>::kSmemBytes);
    if (rc) set_last_error("cudaFuncSetAttribute(max dynamic shared memory) failed for a grouped GEMM kernel");
    return rc;
}

// GEMM-1 + SwiGLU: the thin items on the weight-streaming kernel, then (prefill-sized batches) the fat items on the
// CTA-pair kernel.  map_x / map_x_big: the caller's x with 32-row and 128-row boxes (shared experts' token operand).
int launch_gemm1(ew_pool *p, int layer, const CUtensorMap &map_x, const CUtensorMap &map_x_big, const void *x, int B,
                 cudaStream_t st) {
    const LayerState &L = p->layers[layer];
    const int K = p->cfg.hidden, I = p->cfg.inter;
    const Workspace &w = p->ws;
    const plan::SelfPlan sp = self_plan_args(p, B, 0);
    int rc;
    switch (p->token_tile) {
        case 32: rc = launch_one<32, true>(p, L.map_w13, map_x, map_x, w.items1, w.n_items, K, I, w.act, st, x, B, sp); break;
        case 64: rc = launch_one<64, true>(p, L.map_w13, map_x, map_x, w.items1, w.n_items, K, I, w.act, st, x, B, sp); break;
        default: rc = launch_one<128, true>(p, L.map_w13, map_x, map_x_big, w.items1, w.n_items, K, I, w.act, st, x, B, sp); break;
    }
    if (rc || !p->fat) return rc;
    return launch_fat<true>(p, L.map_w13, map_x_big, w.fat1, w.n_items + 2, K, I, w.act, st, x, B);
}

int launch_gemm2(ew_pool *p, int layer, int B, cudaStream_t st) {
    const LayerState &L = p->layers[layer];
    const int K = p->cfg.inter, H = p->cfg.hidden;
    const Workspace &w = p->ws;
    const CUtensorMap &a = p->map_act, &ab = p->map_act_big;
    const plan::SelfPlan sp = self_plan_args(p, B, 1);
    int rc;
    switch (p->token_tile) {
        case 32: rc = launch_one<32, false>(p, L.map_w2, a, a, w.items2, w.n_items + 1, K, H, w.y, st, nullptr, 0, sp); break;
        case 64: rc = launch_one<64, false>(p, L.map_w2, a, a, w.items2, w.n_items + 1, K, H, w.y, st, nullptr, 0, sp); break;
        default: rc = launch_one<128, false>(p, L.map_w2, a, ab, w.items2, w.n_items + 1, K, H, w.y, st, nullptr, 0, sp); break;
    }
    if (rc || !p->fat) return rc;
    return launch_fat<false>(p, L.map_w2, ab, w.fat2, w.n_items + 3, K, H, w.y, st, nullptr, 0);
}

}  // namespace ew
