// Family (c): BSR-16 on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM,
// operands brought to shared memory by TMA).
//
// A block-row I of A is a list of dense 16x16 blocks (I, J).  Its 16 output rows are
//     C[16I..16I+15, n0..n0+255] = sum_J  Ablk(I,J) * B[16J..16J+15, n0..n0+255]
// One tcgen05.mma per block and 256-column slab of B:
//     M = 64   MMA operand "A" = the block, K-major, unswizzled 8-row cores.  Only its first 16
//              rows exist: the tensor core reads rows 16..63 from whatever follows the block
//              image in shared memory and leaves their products in accumulator rows that nobody
//              reads (M = 64 is the smallest shape; the tensor pipe has time to spare here).
//     N = 256  MMA operand "B" = a 16 x 256 slab of B, MN-major, 128-byte swizzle: exactly the
//              image a TMA box load leaves in shared memory.
//     K = 16 (bf16, kind::f16) or 8 (fp32 as tf32, kind::tf32: two steps per block).
// The accumulator sits in TMEM with the row of C on the lane axis (lanes 0..15) and the dense
// column on the column axis: one instruction per block keeps the single issuing thread, whose
// per-instruction latency bounds this kernel, as idle as possible.
//
// fp32 values cannot go through one tf32 pass (10 mantissa bits: 2^-11 operand rounding, far
// outside the 1e-5 tolerance).  Both operands are split x = hi + lo with hi = x with its low 13
// mantissa bits cleared (exact in tf32) and lo = x - hi (exact in fp32); three products
// hi*hi + lo*hi + hi*lo are accumulated in fp32, the dropped lo*lo term is below 2^-22 |x||y|.
// The blocks are split at plan time; the slab of B is split in shared memory by converter warps.
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
constexpr int kTcBatchItems = 64;            // work items whose metadata is staged at once
constexpr int kTcBatchBlocks = 2048;         // block columns staged per batch
constexpr uint32_t kTcSpinLimit = 1u << 20;  // mbarrier polls before a wait gives up

// shared-memory bytes of one block inside a ring slot
constexpr int kTcSlabBytesBf16 = 8192;           // slab 16 x 256 bf16
constexpr int kTcSlabBytesTf32 = 16384 + 16384;  // slab hi (in place of the raw fp32 slab), slab lo
constexpr int kTcImgBytesBf16 = 512;             // block image
constexpr int kTcImgBytesTf32 = 2048;            // block image hi (two k steps of 512 B), then lo
// a slot is `sb` slabs followed by the `sb` images, rounded so that every slot stays 1024-byte aligned
__host__ __device__ constexpr int tc_stage_bytes(bool tf32, int sb) {
    return sb * (tf32 ? kTcSlabBytesTf32 : kTcSlabBytesBf16) +
           ((sb * (tf32 ? kTcImgBytesTf32 : kTcImgBytesBf16) + 1023) / 1024) * 1024;
}

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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *error,
                                          int code) {
    for (uint32_t i = 0; i < kTcSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(error, 0, code);
    return false;
}
// The same wait for a whole warp: lane 0 polls, every lane gets the outcome.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *error,
                                               int code) {
    int r = 1;
    if ((threadIdx.x & 31) == 0) r = mbar_wait(bar, parity, abort_flag, error, code) ? 1 : 0;
    return __shfl_sync(0xffffffffu, r, 0) != 0;
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

// Instruction descriptors without the N field: D = f32, A K-major, B MN-major, M = 64;
// kind::f16 with A = B = bf16 (format 1), kind::tf32 with A = B = tf32 (format 2).
constexpr uint32_t kIdescBf16 = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((64u >> 4) << 24);
constexpr uint32_t kIdescTf32 = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 16) | ((64u >> 4) << 24);
__device__ __forceinline__ uint32_t idesc_n(uint32_t base, int ncols) {
    return base | (static_cast<uint32_t>(ncols >> 3) << 17);
}

template <bool TF32>
__global__ void __launch_bounds__(TF32 ? kTcThreadsTf32 : kTcThreadsBf16, 1)
bsr_tc_kernel(const __grid_constant__ CUtensorMap tmapB, const TcArgs a) {
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
    uint64_t *full = bars, *empty = bars + kTcMaxStages, *conv = bars + 2 * kTcMaxStages,
             *acc_full = bars + 3 * kTcMaxStages, *acc_empty = bars + 3 * kTcMaxStages + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * kTcMaxStages + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    int32_t *meta_b0 = reinterpret_cast<int32_t *>(tmem_slot + 2);   // [kTcBatchItems + 1] block-row pointers
    int32_t *meta_col = meta_b0 + 2 * kTcBatchItems;                  // [kTcBatchBlocks] block columns

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < a.stages; ++s) {
            mbar_init(smem_u32(full + s), 1);
            mbar_init(smem_u32(empty + s), 1);
            mbar_init(smem_u32(conv + s), kTcConvWarps);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(acc_full + s), 1);
            mbar_init(smem_u32(acc_empty + s), 2);
        }
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
    const int r_begin = __ldg(a.part + blockIdx.x), r_end = __ldg(a.part + blockIdx.x + 1);
    uint32_t p_stage = 0, p_phase = 0, p_issued = 0;                     // producer ring state
    uint32_t m_stage = 0, m_phase = 0;                                   // consumer ring state (MMA, converters)
    uint32_t it = 0;                                                      // items done (accumulator slot / parity)
    bool ok = true, first = true, live = true;

    for (int slab = 0; slab < a.nslab && live; ++slab) {
    const int n0 = slab * kTcSlabCols;
    const int ncols = min(kTcSlabCols, a.N - n0);
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
        for (int f = threadIdx.x; f < min(total, kTcBatchBlocks); f += kThreads) meta_col[f] = __ldg(a.bcol + base + f);
        __syncthreads();

        if (warp == 1) {
            // -------------------------------------------------------------- TMA producer
            {
                // The whole warp runs the loop (uniform control flow and addresses); lane 0 issues the
                // copies: one slab copy per block, one image copy per ring slot.
                const bool leader = lane == 0;
                const uint8_t *img = static_cast<const uint8_t *>(a.bmma) + static_cast<int64_t>(base) * kImgBytes;
                const int zc = n0 / (TF32 ? 32 : 64);
                const uint32_t ring0 = smem_u32(smem), full0 = smem_u32(full), empty0 = smem_u32(empty);
                const uint32_t tx1 = static_cast<uint32_t>(a.box_bytes + kImgBytes);
                for (int fb = 0; fb < total && ok; fb += a.sb) {
                    const int cnt = min(a.sb, total - fb);
                    if (!(ok = mbar_wait_warp(empty0 + p_stage * 8, p_phase ^ 1, abort_flag, a.error, 1))) break;
                    ++p_issued;
                    uint32_t dst = ring0 + p_stage * stage_bytes;
                    const uint32_t fbar = full0 + p_stage * 8;
                    if (leader) {
                        mbar_expect_tx(fbar, cnt * tx1);
                        bulk_load(dst + img_off, img, cnt * kImgBytes, fbar);
                    }   // the images of cnt consecutive blocks
                    img += cnt * kImgBytes;
                    for (int u = 0; u < cnt; ++u, dst += kSlab) {
                        const int flat = fb + u;
                        const int krow = ((flat < kTcBatchBlocks) ? meta_col[flat] : __ldg(a.bcol + base + flat)) * 16;
                        // one copy brings all column groups of the slab: [group][16 rows][128 B]
                        if (leader) tma_load_3d(dst, &tmapB, 0, krow, zc, fbar);
                    }
                    if (++p_stage == static_cast<uint32_t>(a.stages)) {
                        p_stage = 0;
                        p_phase ^= 1;
                    }
                }
            }
        } else if (warp == 2) {
            // -------------------------------------------------------------- MMA issuer
            {
                // the whole warp runs the loop; lane 0 issues the tensor-core instructions
                const bool leader = lane == 0;
                int j = 0, k = 0;
                uint32_t ms = m_stage, mp = m_phase;
                const uint32_t accf0 = smem_u32(acc_full), acce0 = smem_u32(acc_empty);
                // block-rows without blocks produce no MMA: their accumulator is simply declared ready
                auto skip_empty_items = [&]() {
                    while (ok && j < bn && meta_b0[j + 1] == meta_b0[j]) {
                        const uint32_t as = (it + j) & 1, aphase = ((it + j) >> 1) & 1;
                        if (!(ok = mbar_wait_warp(acce0 + as * 8, aphase ^ 1, abort_flag, a.error, 2))) break;
                        if (leader) mbar_arrive(accf0 + as * 8);
                        ++j;
                    }
                };
                skip_empty_items();
                // descriptors differ from block to block only in their start-address field:
                // block image (operand "A", K-major): 8-row cores 128 bytes apart, k halves 256 bytes apart;
                // slab (operand "B", MN-major): 128-byte column groups 2048 bytes apart; bf16: 128-byte
                // swizzle, 8-row k groups 1024 bytes apart; fp32: the 128-byte swizzle with 32-byte atoms
                // (layout type 1, which MN-major 32-bit operands need), 4-row k groups 512 bytes apart
                const uint64_t a0 = smem_desc(0, 256, 128, 0);
                const uint64_t b0 = smem_desc(0, 2048, TF32 ? 512 : 1024, TF32 ? 1 : 2);
                const uint32_t ring0 = smem_u32(smem), wait0 = smem_u32(TF32 ? conv : full), empty0 = smem_u32(empty);
                const uint32_t idesc = idesc_n(TF32 ? kIdescTf32 : kIdescBf16, ncols);
                int nbj = 0;
                uint32_t as = 0, d0 = 0;
                auto enter_item = [&]() {   // per-item values, when the first block of block-row j comes up
                    as = (it + j) & 1;
                    d0 = tmem_base + as * kTcSlabCols;
                    nbj = meta_b0[j + 1] - meta_b0[j];
                    return mbar_wait_warp(acce0 + as * 8, (((it + j) >> 1) & 1) ^ 1, abort_flag, a.error, 2);
                };
                for (int fb = 0; fb < total && ok; fb += a.sb) {
                    const int cnt = min(a.sb, total - fb);
                    if (!(ok = mbar_wait_warp(wait0 + ms * 8, mp, abort_flag, a.error, 3))) break;
                    tc_fence_after();
                    const uint32_t stage0 = ring0 + ms * stage_bytes;
                    uint64_t slab16 = static_cast<uint64_t>((stage0 & 0x3FFFFu) >> 4);
                    uint64_t img16 = static_cast<uint64_t>(((stage0 + img_off) & 0x3FFFFu) >> 4);
                    for (int u = 0; u < cnt && ok; ++u, slab16 += kSlab >> 4, img16 += kImgBytes >> 4) {
                        if (k == 0) {
                            if (!(ok = enter_item())) break;
                            tc_fence_after();
                        }
                        if constexpr (TF32) {
                            // k step = 8 block columns: 512 bytes of the image, 8 rows = 1024 bytes of the slab
#pragma unroll
                            for (int ks = 0; ks < 2; ++ks) {
                                const uint64_t a_hi = a0 + img16 + ((ks * 512) >> 4);
                                const uint64_t a_lo = a_hi + (1024 >> 4);
                                const uint64_t b_hi = b0 + slab16 + ((ks * 1024) >> 4);
                                const uint64_t b_lo = b_hi + (16384 >> 4);
                                if (leader) {
                                    tc_mma<true>(d0, a_hi, b_hi, idesc, (k > 0 || ks > 0) ? 1u : 0u);
                                    tc_mma<true>(d0, a_lo, b_hi, idesc, 1u);
                                    tc_mma<true>(d0, a_hi, b_lo, idesc, 1u);
                                }
                            }
                        } else {
                            if (leader) tc_mma<false>(d0, a0 + img16, b0 + slab16, idesc, k > 0 ? 1u : 0u);
                        }
                        if (++k == nbj) {
                            if (leader) tc_commit(accf0 + as * 8);   // the block-row's accumulator is complete
                            ++j;
                            k = 0;
                            skip_empty_items();
                        }
                    }
                    if (!ok) break;
                    if (leader) tc_commit(empty0 + ms * 8);   // the slot is free once these MMAs retire
                    if (++ms == static_cast<uint32_t>(a.stages)) {
                        ms = 0;
                        mp ^= 1;
                    }
                }
            }
        } else if (warp == 0 || warp == 4) {
            // -------------------------------------------------------------- epilogue warps
            // lane r < 16 holds row 16I + r of C; this warp takes columns [half*128, half*128 + 128) of the slab
            const int half = warp >> 2;
            uint32_t eit = it;
            for (int j = 0; j < bn && ok; ++j, ++eit) {
                const int I = row0 + j;
                const bool has_blocks = meta_b0[j + 1] > meta_b0[j];
                const uint32_t as = eit & 1, aphase = (eit >> 1) & 1;
                const int64_t row = static_cast<int64_t>(I) * 16 + lane;
                const bool mine = lane < 16 && row < a.M;
                float *crow = a.C + row * a.ldc + n0;
                // one lane polls the barrier (spinning threads would crowd the barrier unit)
                if (lane == 0) ok = mbar_wait(smem_u32(acc_full + as), aphase, abort_flag, a.error, 4);
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                tc_fence_after();
#pragma unroll 1
                for (int ch = 0; ch < 4; ++ch) {
                    const int c0 = half * 128 + ch * 32;
                    if (c0 >= ncols) break;   // warp-uniform
                    float r[32];
                    if (has_blocks) {
                        tc_ld32(tmem_base + as * kTcSlabCols + c0, r);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = 0.f;
                    }
                    if (ch == 3 || c0 + 32 >= ncols) {   // last read of the slot: it may be overwritten
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(acc_empty + as));
                    }
                    if (mine) {
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
                if (half * 128 >= ncols) {   // this warp has no columns in a narrow slab: just release the slot
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(acc_empty + as));
                }
            }
        } else if constexpr (TF32) {
            // -------------------------------------------------------------- converter warps (3, 5..11)
            // split the fp32 slab of every block of the slot: hi stays in place, lo goes beside it
            const int ct = (warp == 3 ? 0 : warp - 4) * 32 + lane;   // 0..255
            uint32_t cs = m_stage, cp = m_phase;
            for (int fb = 0; fb < total && ok; fb += a.sb) {
                const int cnt = min(a.sb, total - fb);
                if (lane == 0) ok = mbar_wait(smem_u32(full + cs), cp, abort_flag, a.error, 5);
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
                        hi[i * 256 + ct] = h;
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
        // every thread advances its copy of the consumer ring position past the batch, so that
        // the MMA issuer and the converter warps enter the next batch at the same slot
        {
            const uint32_t adv = m_stage + static_cast<uint32_t>((total + a.sb - 1) / a.sb);
            m_phase ^= (adv / static_cast<uint32_t>(a.stages)) & 1;
            m_stage = adv % static_cast<uint32_t>(a.stages);
        }
        it += bn;
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

// fp32 blocks: hi / lo split and the K-major image of each half: per k step (8 block columns)
// four core matrices of 8 rows x 4 floats, ordered [k step][k half][row group]; hi image first
// (1 KB), lo image after it.
static __global__ void bsr_mma_image_tf32_kernel(const float *__restrict__ bval, float *__restrict__ img, int64_t nnzb) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= nnzb * 256) return;
    const int64_t b = i >> 8;
    const int r = (i >> 4) & 15, c = i & 15;
    const int off = (c >> 3) * 128 + ((c & 7) >> 2) * 64 + (r >> 3) * 32 + (r & 7) * 4 + (c & 3);
    const float x = bval[i];
    const float h = __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
    img[b * 512 + off] = h;
    img[b * 512 + 256 + off] = x - h;
}

}  // namespace sd
