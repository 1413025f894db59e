// Family (c): BSR-16 on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM,
// operands brought to shared memory by TMA).
//
// A block-row I of A is a list of dense 16x16 blocks (I, J).  Its 16 output rows are
//     C[16I..16I+15, n0..n0+255] = sum_J  Ablk(I,J) * B[16J..16J+15, n0..n0+255]
// One tcgen05.mma per block and 256-column slab of B (two k steps of two for fp32):
//     M        MMA operand "A" = the block, K-major, unswizzled 8-row cores.  Only its first 16
//              (fp32: 32, see below) rows exist: the tensor core reads the remaining rows of the
//              M = 64 (bf16) or 128 (fp32) shape from whatever follows the block image in shared
//              memory and leaves their products in accumulator rows that nobody reads.  Measured:
//              the tensor core spends 128 x N x K multiply-adds of time on either shape, about 127
//              cycles per bf16 instruction here, and the pipe still has time to spare.
//     N = 256  MMA operand "B" = a 16 x 256 slab of B, MN-major, 128-byte swizzle: exactly the
//              image a TMA box load leaves in shared memory.
//     K = 16 (bf16, kind::f16) or 8 (fp32 as tf32, kind::tf32).
// The accumulator sits in TMEM with the row of C on the lane axis (lanes 0..15) and the dense
// column on the column axis.  One instruction per block matters because the kernel is bound by
// the latency of the single thread that issues them, not by the tensor pipe or by memory.
//
// fp32 values cannot go through one tf32 pass (10 mantissa bits: 2^-11 operand rounding, far
// outside the 1e-5 tolerance).  Both operands are split x = hi + lo with hi = x with its low 13
// mantissa bits cleared (exact in tf32) and lo = x - hi (exact in fp32).  The blocks are split
// at plan time and stored hi block over lo block (32 rows), so that one instruction multiplies
// both with a slab operand: with the slab's hi and lo images that is two instructions per k
// step, accumulator rows 0..15 collect hi*hi + hi*lo, rows 16..31 lo*hi + lo*lo, and the epilogue
// adds the two halves.  M = 128 keeps row r in TMEM lane r (M = 64 would put rows 16..31 into the
// next lane quarter, which the epilogue warp cannot read).  The slab of B is split in shared
// memory by converter warps.
//
// Persistent CTAs, one per SM (two 256-column accumulators fill TMEM).  Warps 0 and 4: epilogue
// (TMEM lanes 0..31 are only visible to warps 0 mod 4; each takes 128 columns).  Warp 1: TMA
// producer.  Warp 2: TMEM owner + MMA issuer.  Warps 3, 5..11 (fp32 only): converters.  A ring
// slot ("stage") holds up to `sb` blocks that share one barrier round trip.  Every wait is
// bounded: on expiry the CTA records an error word, drains, frees its TMEM and returns.
#pragma once

#include <cuda.h>

#include "sd_common.cuh"
#include "sd_launch.cuh"

namespace sd {

constexpr int kTcMaxStages = 24;             // most ring slots a CTA may use
constexpr int kTcSlabCols = 256;             // dense columns per work item (one N = 256 instruction)
constexpr int kTcTmemCols = 512;             // 2 accumulator slots x 256 columns
constexpr int kTcThreadsBf16 = 160;          // warps 0..4
constexpr int kTcThreadsTf32 = 384;          // + 7 more converter warps
constexpr int kTcConvWarps = 8;
// kind::tf32 reads the upper 19 bits of a 32-bit operand and drops the rest, which is exactly the
// hi half of the split: the raw slab serves as hi and the converters only write lo.  (The parity
// tests would fail by orders of magnitude if an operand were rounded instead; true = mask hi explicitly.)
constexpr bool kTcStoreHi = false;
constexpr int kTcBatchItems = 64;            // work items whose metadata is staged at once
constexpr int kTcBatchBlocks = 1024;         // block columns staged per batch
constexpr uint32_t kTcSpinLimit = 1u << 20;  // mbarrier polls before a wait gives up

// shared-memory bytes of one block inside a ring slot
constexpr int kTcSlabBytesBf16 = 8192;           // slab 16 x 256 bf16
constexpr int kTcSlabBytesTf32 = 16384 + 16384;  // slab hi (in place of the raw fp32 slab), slab lo
constexpr int kTcImgBytesBf16 = 512;             // block image
constexpr int kTcImgBytesTf32 = 2048;            // block image: two k steps of 1 KB, each the hi block over the lo block
// a slot is `sb` slabs followed by the `sb` images, rounded so that every slot stays 1024-byte aligned
// ring slots a staged batch can span
__host__ __device__ constexpr int tc_mask_words(int sb) { return (kTcBatchBlocks + sb - 1) / sb + 1; }
__host__ __device__ constexpr int tc_stage_bytes(bool tf32, int sb) {
    return sb * (tf32 ? kTcSlabBytesTf32 : kTcSlabBytesBf16) +
           ((sb * (tf32 ? kTcImgBytesTf32 : kTcImgBytesBf16) + 1023) / 1024) * 1024;
}

// The M = 64 / 128 instruction shapes read block-image rows that do not exist: 768 bytes (bf16: six more 8-row
// cores of both k halves) or 1,536 bytes (fp32: twelve more per k step) past the end of a block's image.  For
// every block but the last of the last ring slot that is the next image or the next slot; for that last one it
// is what follows the ring in the dynamic allocation: the barrier words and the staged metadata (sized in
// run_bsr_tc as 8 * (3 * kTcMaxStages + 8) + 4 * (2 * kTcBatchItems + kTcBatchBlocks + masks) bytes, plus at
// least 1,025 bytes of alignment slack).  The products of those rows land in accumulator rows nobody reads.
constexpr int kTcOverReadBf16 = 768, kTcOverReadTf32 = 1536;
static_assert(8 * (3 * kTcMaxStages + 8) + 4 * (2 * kTcBatchItems + kTcBatchBlocks) >= kTcOverReadTf32 &&
                  kTcOverReadTf32 >= kTcOverReadBf16,
              "the operand over-read of the last block image must stay inside the kernel's own shared memory");

struct TcArgs {
    const int32_t *browptr;
    const int32_t *bcol;
    const void *bmma;       // [nnzb] MMA-ready block images (bf16: 512 B, fp32: hi 1 KB + lo 1 KB)
    float *C;
    int64_t ldc;
    int64_t M;
    int32_t Mb;
    int32_t N;
    int32_t nslab;          // ceil(N / 256)
    const int32_t *part;    // [gridDim.x + 1] first block-row of every CTA
    float alpha, beta;
    int32_t *error;         // device word: 0 = fine, else the first wait that expired
    int32_t box_bytes;      // bytes one TMA box copy delivers
    int32_t stages;         // ring slots in use
    int32_t sb;             // blocks per ring slot
    int32_t wide_store;     // C and ldc allow 32-byte stores
};

// ---- PTX wrappers -------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait.  Returns false when the limit ran out or another warp already gave up.
// (The limit is a compile-time constant on purpose: as a kernel argument it cost the fp32 kernel 18 %.)
template <uint32_t LIMIT>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *error,
                                          int code) {
    for (uint32_t i = 0; i < LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(error, 0, code);
    return false;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
template <bool TF32>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    if constexpr (TF32) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    }
}
// 32 consecutive accumulator columns of this thread's TMEM lane.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&r)[32]) {
    uint32_t u[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
          "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]),
          "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]),
          "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) r[i] = __uint_as_float(u[i]);
}

// Shared-memory matrix descriptor: start address, leading / stride byte offsets (all >> 4),
// the fixed field of this architecture, and the swizzle mode (0 none, 1 = 128 B with 32-byte
// atoms, 2 = 128 B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo, uint32_t swizzle) {
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo >> 4) << 16) |
           (static_cast<uint64_t>(sbo >> 4) << 32) | (1ull << 46) | (static_cast<uint64_t>(swizzle) << 61);
}

// Instruction descriptors without the N field: D = f32, A K-major, B MN-major;
// kind::f16 with A = B = bf16 (format 1), M = 64 (accumulator row r < 16 sits in TMEM lane r);
// kind::tf32 with A = B = tf32 (format 2), M = 128 (row r in lane r for all 128 rows: the lo block's
// rows 16..31 must share the epilogue warp's lane quarter, which M = 64 would spread over two).
constexpr uint32_t kIdescBf16 = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((64u >> 4) << 24);
constexpr uint32_t kIdescTf32 = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 16) | ((128u >> 4) << 24);
__device__ __forceinline__ uint32_t idesc_n(uint32_t base, int ncols) {
    return base | (static_cast<uint32_t>(ncols >> 3) << 17);
}

// Non-blocking look at a barrier phase (the result is used a ring slot later, so its latency hides).
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Progress counters in shared memory (a plain flag costs a fraction of a barrier round trip).
__device__ __forceinline__ void st_release(uint32_t addr, uint32_t v) {
    asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
// Bounded wait until the counter at `addr` has reached `target`.
template <uint32_t LIMIT>
__device__ __forceinline__ bool counter_wait(uint32_t addr, uint32_t target, volatile int *abort_flag, int32_t *error,
                                             int code) {
    for (uint32_t i = 0; i < LIMIT; ++i) {
        if (static_cast<int32_t>(ld_acquire(addr) - target) >= 0) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(error, 0, code);
    return false;
}

// EXPIRY_TEST: the instance behind sd_plan_desc_t.test_wait_expiry (short spin limit, CTA 0 never copies anything in).
template <bool TF32, bool EXPIRY_TEST>
__global__ void __launch_bounds__(TF32 ? kTcThreadsTf32 : kTcThreadsBf16, 1)
bsr_tc_kernel(const __grid_constant__ CUtensorMap tmapB, const TcArgs a) {
    constexpr uint32_t kLimit = EXPIRY_TEST ? 4096u : kTcSpinLimit;
    constexpr int kThreads = TF32 ? kTcThreadsTf32 : kTcThreadsBf16;
    constexpr int kSlab = TF32 ? kTcSlabBytesTf32 : kTcSlabBytesBf16;   // slab bytes of one block in a ring slot
    constexpr int kImgBytes = TF32 ? kTcImgBytesTf32 : kTcImgBytesBf16;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // stage ring first (1024-byte aligned for the 128-byte swizzle), barriers and metadata after it
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    // a ring slot: the slabs of its `sb` blocks, then their images (contiguous, as in global memory)
    const uint32_t img_off = static_cast<uint32_t>(a.sb) * kSlab;
    const int stage_bytes = tc_stage_bytes(TF32, a.sb);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + a.stages * stage_bytes);
    uint64_t *full = bars, *empty = bars + kTcMaxStages, *conv = bars + 2 * kTcMaxStages, *acc_full = bars + 3 * kTcMaxStages;
    uint64_t *drain = acc_full + 2;   // after an expired wait: the issuer's outstanding tensor-core work arrives here
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * kTcMaxStages + 3);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    uint32_t *epi_done = tmem_slot + 2;                                 // [2] rows whose accumulator each epilogue warp has read
    int32_t *meta_b0 = reinterpret_cast<int32_t *>(tmem_slot + 4);      // [kTcBatchItems + 1] block-row pointers
    int32_t *meta_col = meta_b0 + 2 * kTcBatchItems;                     // [kTcBatchBlocks] block columns
    uint32_t *first_mask = reinterpret_cast<uint32_t *>(meta_col + kTcBatchBlocks);   // [tc_mask_words] per ring slot:
    uint32_t *last_mask = first_mask + tc_mask_words(a.sb);              // blocks that open / close a block-row

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < a.stages; ++s) {
            mbar_init(smem_u32(full + s), 1);
            mbar_init(smem_u32(empty + s), 1);
            mbar_init(smem_u32(conv + s), kTcConvWarps);
        }
        for (int s = 0; s < 2; ++s) mbar_init(smem_u32(acc_full + s), 1);
        mbar_init(smem_u32(drain), 1);
        epi_done[0] = 0;
        epi_done[1] = 0;
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTcTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // This CTA owns the block-rows [r_begin, r_end) (plan-time partition of about equal cost) and
    // runs them once per 256-column slab of B.  Their blocks are contiguous in bcol and in the
    // image array.  Block-row pointers and block columns live in global memory; a dependent global
    // load between two blocks would serialise the pipeline on memory latency, so the CTA first
    // brings the metadata of a batch of block-rows into shared memory (all threads, two coalesced
    // round trips), then the roles run through the batch from there.
    //
    // What bounds this kernel is the latency of the single threads that issue the copies and the
    // tensor-core instructions: a dependent mbarrier wait costs about 180 cycles even when the
    // phase completed long ago.  So both look one ring slot ahead with a non-blocking test, the
    // per-block decisions (does this block open / close a block-row) are bit masks prepared by all
    // threads, and the epilogue hands accumulator slots back through plain counters.
    const int r_begin = __ldg(a.part + blockIdx.x), r_end = __ldg(a.part + blockIdx.x + 1);
    uint32_t p_stage = 0, p_phase = 0, p_issued = 0;                     // producer ring state
    uint32_t m_stage = 0, m_phase = 0;                                   // consumer ring state (MMA, converters)
    uint32_t it = 0;                                                      // block-rows with blocks done (accumulator slot / parity)
    bool ok = true, first = true, live = true;
    const int sb = a.sb;

    for (int slab = 0; slab < a.nslab && live; ++slab) {
    const int n0 = slab * kTcSlabCols;
    const int ncols = min(kTcSlabCols, a.N - n0);
    const int nhalves = ncols > 128 ? 2 : 1;   // epilogue warps with columns in this slab
    for (int row0 = r_begin; row0 < r_end;) {
        const int cand = min(kTcBatchItems, r_end - row0);
        if (!first) {
            __syncthreads();                       // everybody is done with the previous batch's metadata
            if (*abort_flag) { live = false; break; }   // uniform: read after the barrier
        }
        first = false;
        for (int j = threadIdx.x; j <= cand; j += kThreads) meta_b0[j] = __ldg(a.browptr + row0 + j);
        __syncthreads();
        // block-rows of this batch: as many as fit the staged column list (one oversized row goes alone)
        const int base = meta_b0[0];
        int bn = 1;
        while (bn < cand && meta_b0[bn + 1] - base <= kTcBatchBlocks) ++bn;
        const int total = meta_b0[bn] - base;   // blocks of the batch
        const int nstages = (total + sb - 1) / sb;
        const bool masks_staged = total <= kTcBatchBlocks;   // else: one oversized block-row, masks are implicit
        uint32_t nonempty = 0;
        for (int j = 0; j < bn; ++j) nonempty += meta_b0[j + 1] != meta_b0[j];
        for (int f = threadIdx.x; f < min(total, kTcBatchBlocks); f += kThreads) meta_col[f] = __ldg(a.bcol + base + f);
        if (masks_staged) {
            for (int f = threadIdx.x; f < nstages; f += kThreads) {
                first_mask[f] = 0;
                last_mask[f] = 0;
            }
            __syncthreads();
            for (int j = threadIdx.x; j < bn; j += kThreads) {
                const int s0 = meta_b0[j] - base, s1 = meta_b0[j + 1] - base;
                if (s1 > s0) {
                    atomicOr(first_mask + s0 / sb, 1u << (s0 % sb));
                    atomicOr(last_mask + (s1 - 1) / sb, 1u << ((s1 - 1) % sb));
                }
            }
        }
        __syncthreads();

        if (warp == 1) {
            // -------------------------------------------------------------- TMA producer
            // The whole warp: lane 0 waits for the slot, arms its barrier with the slot's byte count and copies the
            // images; then lane u issues the slab copy of the slot's block u, so the copies of a slot are issued side
            // by side instead of one after the other by a single thread (which cost about 200 cycles per block).
            {
                const uint8_t *img = static_cast<const uint8_t *>(a.bmma) + static_cast<int64_t>(base) * kImgBytes;
                const int zc = n0 / (TF32 ? 32 : 64);
                const uint32_t ring0 = smem_u32(smem), full0 = smem_u32(full), empty0 = smem_u32(empty);
                const uint32_t tx1 = static_cast<uint32_t>(a.box_bytes + kImgBytes);
                uint32_t ahead = lane == 0 ? mbar_test_wait(empty0 + p_stage * 8, p_phase ^ 1) : 0u;
                for (int fb = 0; fb < total && ok; fb += sb) {
                    if (EXPIRY_TEST && blockIdx.x == 0) break;   // wait-expiry test: nothing is ever copied in
                    const int cnt = min(sb, total - fb);
                    uint32_t ns = p_stage + 1, np = p_phase;
                    if (ns == static_cast<uint32_t>(a.stages)) {
                        ns = 0;
                        np ^= 1;
                    }
                    uint32_t ahead_next = 0;
                    const uint32_t dst = ring0 + p_stage * stage_bytes;
                    const uint32_t fbar = full0 + p_stage * 8;
                    if (lane == 0) {
                        ahead_next = mbar_test_wait(empty0 + ns * 8, np ^ 1);   // a look at the next slot
                        if (!ahead) ok = mbar_wait<kLimit>(empty0 + p_stage * 8, p_phase ^ 1, abort_flag, a.error, 1);
                        if (ok) {
                            mbar_expect_tx(fbar, cnt * tx1);
                            bulk_load(dst + img_off, img, cnt * kImgBytes, fbar);   // the images of cnt consecutive blocks
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;   // also orders the arming before the copies below
                    if (!ok) break;
                    ++p_issued;
                    img += cnt * kImgBytes;
                    if (lane < cnt) {
                        const int flat = fb + lane;
                        const int krow = ((flat < kTcBatchBlocks) ? meta_col[flat] : __ldg(a.bcol + base + flat)) * 16;
                        // one copy brings all column groups of the slab: [group][16 rows][128 B]
                        tma_load_3d(dst + lane * kSlab, &tmapB, 0, krow, zc, fbar);
                    }
                    p_stage = ns;
                    p_phase = np;
                    ahead = ahead_next;
                }
            }
        } else if (warp == 2) {
            // -------------------------------------------------------------- MMA issuer
            if (lane == 0) {
                uint32_t ms = m_stage, mp = m_phase;
                uint32_t n = it;   // block-rows with blocks before the one in hand
                // descriptors differ from block to block only in their start-address field:
                // block image (operand "A", K-major): 8-row cores 128 bytes apart; bf16: k halves 256 bytes
                // apart; fp32: hi block (rows 0..15) and lo block (rows 16..31) stacked, k halves 512 bytes apart;
                // slab (operand "B", MN-major): 128-byte column groups 2048 bytes apart; bf16: 128-byte
                // swizzle, 8-row k groups 1024 bytes apart; fp32: the 128-byte swizzle with 32-byte atoms
                // (layout type 1, which MN-major 32-bit operands need), 4-row k groups 512 bytes apart
                const uint64_t a0 = smem_desc(0, TF32 ? 512 : 256, 128, 0);
                const uint64_t b0 = smem_desc(0, 2048, TF32 ? 512 : 1024, TF32 ? 1 : 2);
                const uint32_t ring0 = smem_u32(smem), wait0 = smem_u32(TF32 ? conv : full), empty0 = smem_u32(empty);
                const uint32_t accf0 = smem_u32(acc_full), done0 = smem_u32(epi_done);
                const uint32_t idesc = idesc_n(TF32 ? kIdescTf32 : kIdescBf16, ncols);
                uint32_t as = 0, d0 = 0;
                uint32_t ahead = mbar_test_wait(wait0 + ms * 8, mp);
                for (int si = 0; si < nstages && ok; ++si) {
                    const int cnt = min(sb, total - si * sb);
                    uint32_t ns = ms + 1, np = mp;
                    if (ns == static_cast<uint32_t>(a.stages)) {
                        ns = 0;
                        np ^= 1;
                    }
                    const uint32_t ahead_next = mbar_test_wait(wait0 + ns * 8, np);   // a look at the next slot
                    uint32_t fm, lm;
                    if (masks_staged) {
                        fm = first_mask[si];
                        lm = last_mask[si];
                    } else {
                        fm = si == 0 ? 1u : 0u;
                        lm = si == nstages - 1 ? 1u << (cnt - 1) : 0u;
                    }
                    if (!ahead && !(ok = mbar_wait<kLimit>(wait0 + ms * 8, mp, abort_flag, a.error, 3))) break;
                    tc_fence_after();
                    const uint32_t stage0 = ring0 + ms * stage_bytes;
                    uint64_t slab16 = static_cast<uint64_t>((stage0 & 0x3FFFFu) >> 4);
                    uint64_t img16 = static_cast<uint64_t>(((stage0 + img_off) & 0x3FFFFu) >> 4);
                    // the slot's blocks as runs of one block-row each: the per-row decisions (which accumulator, is it
                    // free, is the row complete) are taken once per run, the loop over a run's blocks only issues
                    for (int u = 0; u < cnt && ok;) {
                        const uint32_t rest = lm >> u;                                   // row ends at or after block u
                        const int e = rest ? u + __ffs(rest) - 1 : cnt - 1;              // last block of the run inside this slot
                        uint32_t opens = (fm >> u) & 1u;
                        if (opens) {
                            // the accumulator slot of this block-row was last read for block-row n - 2
                            as = n & 1u;
                            d0 = tmem_base + as * kTcSlabCols;
                            if (n >= 2) {
                                for (int h = 0; h < nhalves && ok; ++h)
                                    ok = counter_wait<kLimit>(done0 + h * 4, n - 1, abort_flag, a.error, 2);
                                if (!ok) break;
                                tc_fence_after();
                            }
                        }
                        for (; u <= e; ++u, slab16 += kSlab >> 4, img16 += kImgBytes >> 4, opens = 0u) {
                        if constexpr (TF32) {
                            // k step = 8 block columns: 1 KB of the image (hi over lo), 8 rows = 1024 bytes of the slab;
                            // accumulator rows 0..15 collect hi*hi + hi*lo, rows 16..31 lo*hi + lo*lo
#pragma unroll
                            for (int ks = 0; ks < 2; ++ks) {
                                const uint64_t a_ks = a0 + img16 + ((ks * 1024) >> 4);
                                const uint64_t b_hi = b0 + slab16 + ((ks * 1024) >> 4);
                                const uint64_t b_lo = b_hi + (16384 >> 4);
                                tc_mma<true>(d0, a_ks, b_hi, idesc, (!opens || ks > 0) ? 1u : 0u);
                                tc_mma<true>(d0, a_ks, b_lo, idesc, 1u);
                            }
                        } else {
                            tc_mma<false>(d0, a0 + img16, b0 + slab16, idesc, opens ^ 1u);
                        }
                        }
                        if (rest) {
                            tc_commit(accf0 + as * 8);   // the block-row's accumulator is complete
                            ++n;
                        }
                    }
                    if (!ok) break;
                    tc_commit(empty0 + ms * 8);   // the slot is free once these MMAs retire
                    ms = ns;
                    mp = np;
                    ahead = ahead_next;
                }
                if (!ok) {
                    // a wait ran out: tensor-core instructions issued before it may still be reading shared memory and
                    // writing TMEM; let them retire (bounded) before the CTA gives both back
                    tc_commit(smem_u32(drain));
                    for (uint32_t i = 0; i < 65536 && !mbar_try_wait(smem_u32(drain), 0); ++i) {
                    }
                }
            }
        } else if (warp == 0 || warp == 4) {
            // -------------------------------------------------------------- epilogue warps
            // lane r < 16 holds row 16I + r of C (fp32: lane r + 16 holds the second half of its sum);
            // this warp takes columns [half*128, half*128 + 128) of the slab
            const int half = warp >> 2;
            uint32_t n = it;
            for (int j = 0; j < bn && ok && half < nhalves; ++j) {
                const int I = row0 + j;
                const bool has_blocks = meta_b0[j + 1] > meta_b0[j];
                const int64_t row = static_cast<int64_t>(I) * 16 + (lane & 15);
                const bool mine = lane < 16 && row < a.M;
                float *crow = a.C + row * a.ldc + n0;
                const uint32_t as = n & 1u, aphase = (n >> 1) & 1u;
                if (has_blocks) {
                    // one lane polls the barrier (spinning threads would crowd the barrier unit)
                    if (lane == 0) ok = mbar_wait<kLimit>(smem_u32(acc_full + as), aphase, abort_flag, a.error, 4);
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                    if (!ok) break;
                    tc_fence_after();
                }
#pragma unroll 1
                for (int ch = 0; ch < 4; ++ch) {
                    const int c0 = half * 128 + ch * 32;
                    if (c0 >= ncols) break;   // warp-uniform
                    float r[32];
                    if (has_blocks) {
                        tc_ld32(tmem_base + as * kTcSlabCols + c0, r);
                        if (ch == 3 || c0 + 32 >= ncols) {   // last read of the slot: the issuer may overwrite it
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) st_release(smem_u32(epi_done + half), n + 1);
                        }
                        if constexpr (TF32) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) r[i] += __shfl_down_sync(0xffffffffu, r[i], 16);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = 0.f;
                    }
                    if (mine && a.wide_store && a.beta == 0.f) {
                        // 32-byte stores: every instruction fills whole 32-byte sectors of 16 different rows (the 16-byte
                        // form writes half sectors, twice as many instructions and L2 write requests for the same bytes)
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            float *p = crow + c0 + 8 * q;
                            asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p),
                                         "f"(a.alpha * r[8 * q]), "f"(a.alpha * r[8 * q + 1]), "f"(a.alpha * r[8 * q + 2]),
                                         "f"(a.alpha * r[8 * q + 3]), "f"(a.alpha * r[8 * q + 4]), "f"(a.alpha * r[8 * q + 5]),
                                         "f"(a.alpha * r[8 * q + 6]), "f"(a.alpha * r[8 * q + 7])
                                         : "memory");
                        }
                    } else if (mine) {
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            float4 *p = reinterpret_cast<float4 *>(crow + c0) + q;
                            float4 v = make_float4(a.alpha * r[4 * q], a.alpha * r[4 * q + 1], a.alpha * r[4 * q + 2],
                                                   a.alpha * r[4 * q + 3]);
                            if (a.beta != 0.f) {
                                const float4 o = *p;
                                v.x = fmaf(a.beta, o.x, v.x); v.y = fmaf(a.beta, o.y, v.y);
                                v.z = fmaf(a.beta, o.z, v.z); v.w = fmaf(a.beta, o.w, v.w);
                            }
                            *p = v;
                        }
                    }
                }
                n += has_blocks ? 1u : 0u;
            }
        } else if constexpr (TF32) {
            // -------------------------------------------------------------- converter warps (3, 5..11)
            // split the fp32 slab of every block of the slot: the raw slab is the hi operand, lo goes beside it
            const int ct = (warp == 3 ? 0 : warp - 4) * 32 + lane;   // 0..255
            uint32_t cs = m_stage, cp = m_phase;
            for (int fb = 0; fb < total && ok; fb += sb) {
                const int cnt = min(sb, total - fb);
                if (lane == 0) ok = mbar_wait<kLimit>(smem_u32(full + cs), cp, abort_flag, a.error, 5);
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                uint8_t *sbp = smem + cs * stage_bytes;
                for (int u = 0; u < cnt; ++u) {
                    float4 *hi = reinterpret_cast<float4 *>(sbp + u * kSlab);
                    float4 *lo = reinterpret_cast<float4 *>(sbp + u * kSlab + 16384);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float4 x = hi[i * 256 + ct];
                        float4 h;
                        h.x = __uint_as_float(__float_as_uint(x.x) & 0xFFFFE000u);
                        h.y = __uint_as_float(__float_as_uint(x.y) & 0xFFFFE000u);
                        h.z = __uint_as_float(__float_as_uint(x.z) & 0xFFFFE000u);
                        h.w = __uint_as_float(__float_as_uint(x.w) & 0xFFFFE000u);
                        if (kTcStoreHi) hi[i * 256 + ct] = h;
                        lo[i * 256 + ct] = make_float4(x.x - h.x, x.y - h.y, x.z - h.z, x.w - h.w);
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(conv + cs));
                if (++cs == static_cast<uint32_t>(a.stages)) {
                    cs = 0;
                    cp ^= 1;
                }
            }
        }
        // every thread advances its copy of the ring positions and of the row count past the batch,
        // so that all roles enter the next batch at the same slot
        {
            const uint32_t adv = m_stage + static_cast<uint32_t>(nstages);
            m_phase ^= (adv / static_cast<uint32_t>(a.stages)) & 1;
            m_stage = adv % static_cast<uint32_t>(a.stages);
        }
        it += nonempty;
        row0 += bn;
    }
    }
    if (warp == 1 && lane == 0 && *abort_flag) {
        // give the copies this thread issued a bounded time to land before shared memory is released:
        // slot s was last filled by issue number i = s (mod stages), whose ring pass gives the parity
        for (uint32_t s2 = 0; s2 < static_cast<uint32_t>(a.stages) && s2 < p_issued; ++s2) {
            const uint32_t last = p_issued - 1 - ((p_issued - 1 - s2) % static_cast<uint32_t>(a.stages));
            const uint32_t parity = (last / static_cast<uint32_t>(a.stages)) & 1;
            for (uint32_t i = 0; i < 65536 && !mbar_try_wait(smem_u32(full + s2), parity); ++i) {
            }
        }
    }

    // ---- teardown: everybody meets here, also after an expired wait --------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTcTmemCols) : "memory");
    }
}

// Permutes row-major 16x16 bf16 blocks into the K-major, unswizzled operand image:
// 8x8 core matrices of 128 contiguous bytes, ordered [k group][row group].
static __global__ void bsr_mma_image_bf16_kernel(const uint16_t *__restrict__ bval, uint16_t *__restrict__ img,
                                                 int64_t nnzb) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= nnzb * 256) return;
    const int64_t b = i >> 8;
    const int r = (i >> 4) & 15, c = i & 15;
    const int off = (((c >> 3) * 2 + (r >> 3)) * 8 + (r & 7)) * 8 + (c & 7);
    img[b * 256 + off] = bval[i];
}

// fp32 blocks: hi / lo split and the K-major image: per k step (8 block columns) 1 KB holding the
// hi block (rows 0..15) over the lo block (rows 16..31) as core matrices of 8 rows x 4 floats, ordered
// [k half][row group: hi 0..7, hi 8..15, lo 0..7, lo 8..15].
static __global__ void bsr_mma_image_tf32_kernel(const float *__restrict__ bval, float *__restrict__ img, int64_t nnzb) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= nnzb * 256) return;
    const int64_t b = i >> 8;
    const int r = (i >> 4) & 15, c = i & 15;
    const int off = (c >> 3) * 256 + ((c & 7) >> 2) * 128 + (r >> 3) * 32 + (r & 7) * 4 + (c & 3);
    const float x = bval[i];
    const float h = __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
    img[b * 512 + off] = h;
    img[b * 512 + off + 64] = x - h;
}

}  // namespace sd
