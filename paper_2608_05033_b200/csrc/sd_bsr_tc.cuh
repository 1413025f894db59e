// Family (c): BSR-16 on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM,
// operands brought to shared memory by TMA).
//
// A block-row I of A is a list of dense 16x16 blocks (I, J).  Its 16 output rows are
//     C[16I..16I+15, :] = sum_J  Ablk(I,J) * B[16J..16J+15, :]
// tcgen05.mma needs M = 64 or 128, while a block is only 16 rows high, so the product is
// taken transposed: D[c, r] = sum_k  B[16J + k, n0 + c] * Ablk[r, k]  with
//     M = 128 dense columns c   (MMA operand "A" = a 16 x 128 slab of B, MN-major, 128B swizzle,
//                                exactly the image a TMA box load leaves in shared memory)
//     N = 16 block rows r       (MMA operand "B" = the block, K-major, unswizzled 8-row cores)
//     K = 16 (bf16, kind::f16) or 8 (fp32 as tf32, kind::tf32: two steps per block).
// The accumulator D sits in TMEM with the dense column on the lane axis, so an epilogue warp
// reading lane l, column r holds C[16I + r, n0 + l]: for a fixed r the 32 lanes of a warp write
// 32 consecutive floats of C.
//
// fp32 values cannot go through one tf32 pass (10 mantissa bits: 2^-11 operand rounding, far
// outside the 1e-5 tolerance).  Both operands are split x = hi + lo with hi = x with its low 13
// mantissa bits cleared (exact in tf32) and lo = x - hi (exact in fp32); three products
// hi*hi + lo*hi + hi*lo are accumulated in fp32, the dropped lo*lo term is below 2^-22 |x||y|.
// The blocks are split at plan time; the slab of B is split in shared memory by converter warps.
//
// Persistent CTAs.  Warp 0: TMA producer.  Warp 1: TMEM owner + MMA issuer.  Warps 2..5:
// epilogue (TMEM -> registers -> alpha/beta -> C).  Warps 6..9 (fp32 only): converters.  A ring
// slot ("stage") holds up to `sb` blocks that share one barrier round trip.  Every wait is
// bounded: on expiry the CTA records an error word, drains, frees its TMEM and returns.
#pragma once

#include <cuda.h>

#include "sd_common.cuh"
#include "sd_launch.cuh"

namespace sd {

constexpr int kTcMaxStages = 24;             // most ring slots a CTA may use
constexpr int kTcSlabCols = 256;             // dense columns per work item (two M = 128 tiles)
constexpr int kTcTmemCols = 64;              // 2 accumulator slots x 2 tiles x 16 columns
constexpr int kTcBatchItems = 64;            // work items whose metadata is staged at once
constexpr int kTcBatchBlocks = 2048;         // block columns staged per batch
constexpr uint32_t kTcSpinLimit = 1u << 20;  // mbarrier polls before a wait gives up

// shared-memory bytes of one block inside a stage
constexpr int kTcBlkBytesBf16 = 8192 + 1024;          // slab 16 x 256 bf16, block image (512 B, padded)
constexpr int kTcBlkBytesTf32 = 16384 + 16384 + 2048; // slab hi (in place of raw), slab lo, block hi + lo

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
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&r)[16]) {
    uint32_t u[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
          "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) r[i] = __uint_as_float(u[i]);
}

// Shared-memory matrix descriptor: start address, leading / stride byte offsets (all >> 4),
// the fixed field of this architecture, and the swizzle mode (0 none, 1 = 128 B with 32-byte
// atoms, 2 = 128 B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo, uint32_t swizzle) {
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo >> 4) << 16) |
           (static_cast<uint64_t>(sbo >> 4) << 32) | (1ull << 46) | (static_cast<uint64_t>(swizzle) << 61);
}

// Instruction descriptors: D = f32, A MN-major, B K-major, N = 16, M = 128;
// kind::f16 with A = B = bf16 (format 1), kind::tf32 with A = B = tf32 (format 2).
constexpr uint32_t kIdescBf16 = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescTf32 = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | ((16u >> 3) << 17) | ((128u >> 4) << 24);

template <bool TF32>
__global__ void __launch_bounds__(TF32 ? 320 : 192, TF32 ? 1 : 2)
bsr_tc_kernel(const __grid_constant__ CUtensorMap tmapB, const TcArgs a) {
    constexpr int kThreads = TF32 ? 320 : 192;
    constexpr int kBlk = TF32 ? kTcBlkBytesTf32 : kTcBlkBytesBf16;   // bytes of one block in a stage
    constexpr int kImgOff = TF32 ? 32768 : 8192;                       // block image inside a block's bytes
    constexpr int kImgBytes = TF32 ? 2048 : 512;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // stage ring first (1024-byte aligned for the 128-byte swizzle), barriers and metadata after it
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int stage_bytes = a.sb * kBlk;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + a.stages * stage_bytes);
    uint64_t *full = bars, *empty = bars + kTcMaxStages, *conv = bars + 2 * kTcMaxStages,
             *acc_full = bars + 3 * kTcMaxStages, *acc_empty = bars + 3 * kTcMaxStages + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 3 * kTcMaxStages + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    int32_t *meta_b0 = reinterpret_cast<int32_t *>(tmem_slot + 2);
    int32_t *meta_nblk = meta_b0 + kTcBatchItems;
    int32_t *meta_col = meta_nblk + kTcBatchItems;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < a.stages; ++s) {
            mbar_init(smem_u32(full + s), 1);
            mbar_init(smem_u32(empty + s), 1);
            mbar_init(smem_u32(conv + s), 4);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(acc_full + s), 1);
            mbar_init(smem_u32(acc_empty + s), 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTcTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int nitems = a.Mb * a.nslab;
    // Block-row pointers and block columns live in global memory.  A dependent global load
    // between two blocks would serialise the pipeline on memory latency, so the CTA first
    // brings the metadata of a batch of its work items into shared memory (all threads, two
    // overlapped round trips), then the roles run through the batch from there.
    const int my_items = (nitems - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    uint32_t p_stage = 0, p_phase = 0, p_issued = 0;                     // producer ring state
    uint32_t m_stage = 0, m_phase = 0;                                   // consumer ring state (MMA, converters)
    uint32_t it = 0;                                                      // items done (accumulator slot / parity)
    bool ok = true;

    for (int batch0 = 0; batch0 < my_items; batch0 += kTcBatchItems) {
        const int bn = min(kTcBatchItems, my_items - batch0);
        if (batch0 != 0) {
            __syncthreads();                       // everybody is done with the previous batch's metadata
            if (*abort_flag) break;                // uniform: read after the barrier
        }
        for (int j = threadIdx.x; j < bn; j += kThreads) {
            const int I = (blockIdx.x + (batch0 + j) * gridDim.x) / a.nslab;
            const int b0 = __ldg(a.browptr + I);
            meta_b0[j] = b0;
            meta_nblk[j] = __ldg(a.browptr + I + 1) - b0;
        }
        __syncthreads();
        int total = 0;   // blocks of the batch (every thread computes it)
        for (int j = 0; j < bn; ++j) {
            const int nb = meta_nblk[j], b0 = meta_b0[j];
            for (int k = threadIdx.x; k < nb && total + k < kTcBatchBlocks; k += kThreads)
                meta_col[total + k] = __ldg(a.bcol + b0 + k);
            total += nb;
        }
        __syncthreads();

        if (warp == 0) {
            // -------------------------------------------------------------- TMA producer
            if (lane == 0) {
                // This thread runs alone in its warp, so every instruction of the per-block path costs
                // its full issue latency: per-item values are computed when the item changes, and
                // addresses advance by addition.
                int j = -1, k = 0, nbj = 0, zc = 0;
                const uint8_t *img = nullptr;
                const uint32_t ring0 = smem_u32(smem), full0 = smem_u32(full), empty0 = smem_u32(empty);
                const uint32_t tx1 = static_cast<uint32_t>(a.box_bytes + kImgBytes);
                for (int fb = 0; fb < total && ok; fb += a.sb) {
                    const int cnt = min(a.sb, total - fb);
                    if (!(ok = mbar_wait(empty0 + p_stage * 8, p_phase ^ 1, abort_flag, a.error, 1))) break;
                    ++p_issued;
                    uint32_t dst = ring0 + p_stage * stage_bytes;
                    const uint32_t fbar = full0 + p_stage * 8;
                    mbar_expect_tx(fbar, cnt * tx1);
                    for (int u = 0; u < cnt; ++u) {
                        while (k == nbj) {   // next item with blocks
                            ++j;
                            k = 0;
                            nbj = meta_nblk[j];
                            const int item = blockIdx.x + (batch0 + j) * gridDim.x;
                            zc = (a.nslab == 1 ? 0 : (item % a.nslab) * kTcSlabCols) / (TF32 ? 32 : 64);
                            img = static_cast<const uint8_t *>(a.bmma) + static_cast<int64_t>(meta_b0[j]) * kImgBytes;
                        }
                        const int flat = fb + u;
                        const int krow = ((flat < kTcBatchBlocks) ? meta_col[flat] : __ldg(a.bcol + meta_b0[j] + k)) * 16;
                        // one copy brings all column groups of the slab: [group][16 rows][128 B]
                        tma_load_3d(dst, &tmapB, 0, krow, zc, fbar);
                        bulk_load(dst + kImgOff, img, kImgBytes, fbar);
                        img += kImgBytes;
                        dst += kBlk;
                        ++k;
                    }
                    if (++p_stage == static_cast<uint32_t>(a.stages)) {
                        p_stage = 0;
                        p_phase ^= 1;
                    }
                }
            }
        } else if (warp == 1) {
            // -------------------------------------------------------------- MMA issuer
            if (lane == 0) {
                int j = 0, k = 0;
                uint32_t ms = m_stage, mp = m_phase;
                // items without blocks produce no MMA: their accumulator is simply declared ready
                auto skip_empty_items = [&]() {
                    while (ok && j < bn && meta_nblk[j] == 0) {
                        const uint32_t as = (it + j) & 1, aphase = ((it + j) >> 1) & 1;
                        if (!(ok = mbar_wait(smem_u32(acc_empty + as), aphase ^ 1, abort_flag, a.error, 2))) break;
                        mbar_arrive(smem_u32(acc_full + as));
                        ++j;
                    }
                };
                skip_empty_items();
                // descriptors differ from block to block only in their start-address field
                const uint64_t a_hi0 = smem_desc(0, 2048, TF32 ? 512 : 1024, TF32 ? 1 : 2);
                const uint64_t b_hi0 = smem_desc(0, 256, 128, 0);
                const uint32_t ring0 = smem_u32(smem), wait0 = smem_u32(TF32 ? conv : full), empty0 = smem_u32(empty);
                const uint32_t accf0 = smem_u32(acc_full), acce0 = smem_u32(acc_empty);
                int mt_n = 2, nbj = (j < bn) ? meta_nblk[j] : 0;
                uint32_t as = 0, d0 = 0;
                auto enter_item = [&]() {   // per-item values, when the first block of item j comes up
                    as = (it + j) & 1;
                    d0 = tmem_base + as * 32;
                    nbj = meta_nblk[j];
                    if (a.nslab == 1) {
                        mt_n = min(2, (a.N + 127) / 128);
                    } else {
                        const int item = blockIdx.x + (batch0 + j) * gridDim.x;
                        mt_n = min(2, (a.N - (item % a.nslab) * kTcSlabCols + 127) / 128);
                    }
                    return mbar_wait(acce0 + as * 8, (((it + j) >> 1) & 1) ^ 1, abort_flag, a.error, 2);
                };
                for (int fb = 0; fb < total && ok; fb += a.sb) {
                    const int cnt = min(a.sb, total - fb);
                    if (!(ok = mbar_wait(wait0 + ms * 8, mp, abort_flag, a.error, 3))) break;
                    tc_fence_after();
                    uint32_t blk = ring0 + ms * stage_bytes;
                    for (int u = 0; u < cnt && ok; ++u, blk += kBlk) {
                        if (k == 0) {
                            if (!(ok = enter_item())) break;
                            tc_fence_after();
                        }
                        const uint64_t blk16 = static_cast<uint64_t>((blk & 0x3FFFFu) >> 4);
                        for (int mt = 0; mt < mt_n; ++mt) {
                            const uint32_t d = d0 + mt * 16;
                            if constexpr (TF32) {
                                // operand "A", MN-major 32-bit elements: the 128-byte swizzle with 32-byte
                                // atoms (layout type 1; its atom is 4 k rows of 128 bytes); 32-column groups
                                // 2048 bytes apart, 4-row k groups 512 bytes apart, k step = 8 rows = 1024 bytes
#pragma unroll
                                for (int ks = 0; ks < 2; ++ks) {
                                    const uint64_t a_hi = a_hi0 + blk16 + ((mt * 8192 + ks * 1024) >> 4);
                                    const uint64_t a_lo = a_hi + (16384 >> 4);
                                    const uint64_t b_hi = b_hi0 + blk16 + ((kImgOff + ks * 512) >> 4);
                                    const uint64_t b_lo = b_hi + (1024 >> 4);
                                    tc_mma<true>(d, a_hi, b_hi, kIdescTf32, (k > 0 || ks > 0) ? 1u : 0u);
                                    tc_mma<true>(d, a_lo, b_hi, kIdescTf32, 1u);
                                    tc_mma<true>(d, a_hi, b_lo, kIdescTf32, 1u);
                                }
                            } else {
                                // operand "A": 64-column atoms 2048 bytes apart, 8-row k groups 1024 bytes apart
                                tc_mma<false>(d, a_hi0 + blk16 + ((mt * 4096) >> 4), b_hi0 + blk16 + (kImgOff >> 4), kIdescBf16,
                                              k > 0 ? 1u : 0u);
                            }
                        }
                        if (++k == nbj) {
                            tc_commit(accf0 + as * 8);   // the item's accumulator is complete
                            ++j;
                            k = 0;
                            skip_empty_items();
                        }
                    }
                    if (!ok) break;
                    tc_commit(empty0 + ms * 8);   // the slot is free once these MMAs retire
                    if (++ms == static_cast<uint32_t>(a.stages)) {
                        ms = 0;
                        mp ^= 1;
                    }
                }
            }
        } else if (warp < 6) {
            // -------------------------------------------------------------- epilogue warps
            const int q = warp & 3;   // TMEM lane quarter this warp may read
            uint32_t eit = it;
            for (int j = 0; j < bn && ok; ++j, ++eit) {
                const int item = blockIdx.x + (batch0 + j) * gridDim.x;
                const int I = item / a.nslab, n0 = (item % a.nslab) * kTcSlabCols;
                const int mt_n = min(2, (a.N - n0 + 127) / 128);
                const bool has_blocks = meta_nblk[j] > 0;
                const uint32_t as = eit & 1, aphase = (eit >> 1) & 1;
                // beta != 0: fetch the old C values while the accumulator is still being produced
                float cold[2][16];
                if (a.beta != 0.f) {
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
                        const int col = n0 + mt * 128 + q * 32 + lane;
#pragma unroll
                        for (int rr = 0; rr < 16; ++rr) {
                            const int64_t row = static_cast<int64_t>(I) * 16 + rr;
                            cold[mt][rr] = (mt < mt_n && col < a.N && row < a.M) ? a.C[row * a.ldc + col] : 0.f;
                        }
                    }
                }
                // one lane polls the barrier (128 spinning threads would crowd the barrier unit)
                if (lane == 0) ok = mbar_wait(smem_u32(acc_full + as), aphase, abort_flag, a.error, 4);
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                tc_fence_after();
                float r[2][16];
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    if (mt < mt_n && has_blocks) {
                        tc_ld16(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + as * 32 + mt * 16, r[mt]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) r[mt][i] = 0.f;
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(acc_empty + as));   // accumulator slot may be overwritten
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    const int col = n0 + mt * 128 + q * 32 + lane;
                    if (mt < mt_n && col < a.N) {
#pragma unroll
                        for (int rr = 0; rr < 16; ++rr) {
                            const int64_t row = static_cast<int64_t>(I) * 16 + rr;
                            if (row < a.M) {
                                float v = a.alpha * r[mt][rr];
                                if (a.beta != 0.f) v = fmaf(a.beta, cold[mt][rr], v);
                                a.C[row * a.ldc + col] = v;
                            }
                        }
                    }
                }
            }
        } else if constexpr (TF32) {
            // -------------------------------------------------------------- converter warps
            // split the fp32 slab of every block of the slot: hi stays in place, lo goes beside it
            const int ct = threadIdx.x - 192;   // 0..127
            uint32_t cs = m_stage, cp = m_phase;
            for (int fb = 0; fb < total && ok; fb += a.sb) {
                const int cnt = min(a.sb, total - fb);
                if (lane == 0) ok = mbar_wait(smem_u32(full + cs), cp, abort_flag, a.error, 5);
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                uint8_t *sbp = smem + cs * stage_bytes;
                for (int u = 0; u < cnt; ++u) {
                    float4 *hi = reinterpret_cast<float4 *>(sbp + u * kBlk);
                    float4 *lo = reinterpret_cast<float4 *>(sbp + u * kBlk + 16384);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 x = hi[i * 128 + ct];
                        float4 h;
                        h.x = __uint_as_float(__float_as_uint(x.x) & 0xFFFFE000u);
                        h.y = __uint_as_float(__float_as_uint(x.y) & 0xFFFFE000u);
                        h.z = __uint_as_float(__float_as_uint(x.z) & 0xFFFFE000u);
                        h.w = __uint_as_float(__float_as_uint(x.w) & 0xFFFFE000u);
                        hi[i * 128 + ct] = h;
                        lo[i * 128 + ct] = make_float4(x.x - h.x, x.y - h.y, x.z - h.z, x.w - h.w);
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
    }
    if (warp == 0 && lane == 0 && *abort_flag) {
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
    if (warp == 1) {
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
