// Family (c): BSR-16 on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM,
// operands brought to shared memory by TMA).
//
// A block-row I of A is a list of dense 16x16 blocks (I, J).  Its 16 output rows are
//     C[16I..16I+15, :] = sum_J  Ablk(I,J) * B[16J..16J+15, :]
// tcgen05.mma needs M = 64 or 128, while a block is only 16 rows high, so the product is
// taken transposed: D[c, r] = sum_k  B[16J + k, n0 + c] * Ablk[r, k]  with
//     M = 128 dense columns c   (MMA operand "A" = a 16 x 128 slab of B, MN-major, 128B swizzle,
//                                exactly the image a 2-D TMA box load leaves in shared memory)
//     N = 16 block rows r       (MMA operand "B" = the block, K-major)
//     K = 16 block columns k    (one instruction per block for bf16).
// The accumulator D sits in TMEM with the dense column on the lane axis, so an epilogue warp
// reading lane l, column r holds C[16I + r, n0 + l]: for a fixed r the 32 lanes of a warp write
// 32 consecutive floats of C.
//
// Persistent CTAs, two per SM.  Warp 0: TMA producer.  Warp 1: TMEM owner + MMA issuer.
// Warps 2..5: epilogue (TMEM -> registers -> alpha/beta -> C).  Every wait is bounded: on
// expiry the CTA records an error word, drains, frees its TMEM and returns.
#pragma once

#include <cuda.h>

#include "sd_common.cuh"
#include "sd_launch.cuh"

namespace sd {

constexpr int kTcThreads = 192;
constexpr int kTcStages = 22;                // most ring slots a CTA may use
constexpr int kTcDefaultStages = 10;         // ring slots per CTA: two CTAs share an SM, because one
constexpr int kTcCtasPerSm = 2;              // producer/issuer pair is bound by its own handshake latency

constexpr int kTcStageBytes = 9 * 1024;      // 4 boxes of 2 KB (B slab, 256 columns) + the block image
constexpr int kTcBlockOff = 8 * 1024;        // offset of the block image inside a stage
constexpr int kTcSlabCols = 256;             // dense columns per work item (two M = 128 tiles)
constexpr int kTcTmemCols = 64;              // 2 accumulator slots x 2 tiles x 16 columns
constexpr int kTcBatchItems = 64;             // work items whose metadata is staged at once
constexpr int kTcBatchBlocks = 2048;          // block columns staged per batch
constexpr uint32_t kTcSpinLimit = 1u << 20;  // mbarrier polls before a wait gives up

struct TcArgs {
    const int32_t *browptr;
    const int32_t *bcol;
    const void *bmma;       // [nnzb] MMA-ready block images
    float *C;
    int64_t ldc;
    int64_t M;
    int32_t Mb;
    int32_t N;
    int32_t nslab;          // ceil(N / 256)
    float alpha, beta;
    int32_t *error;         // device word: 0 = fine, else the first wait that expired
    uint32_t lbo_a, sbo_a, lbo_b, sbo_b;   // shared-memory descriptor strides (bytes)
    int32_t map3d;          // the tensor map is the 3-D view {64 columns, K rows, N/64 groups}
    int32_t box_bytes;      // bytes one 3-D box copy delivers
    int32_t debug;          // bench-only experiment switches (0 in production)
    int32_t stages;         // ring slots in use (<= kTcStages)
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
__device__ int g_tc_test_wait = 0;
// Bounded wait.  Returns false when the limit ran out or another warp already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *error,
                                          int code) {
    for (uint32_t i = 0; i < kTcSpinLimit; ++i) {
        if (g_tc_test_wait ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(error, 0, code);
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
        : "memory");
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
__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
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
// the fixed field of this architecture, and the swizzle mode (0 none, 2 = 128 B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo, uint32_t swizzle) {
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo >> 4) << 16) |
           (static_cast<uint64_t>(sbo >> 4) << 32) | (1ull << 46) | (static_cast<uint64_t>(swizzle) << 61);
}

// Instruction descriptor, kind::f16 with bf16 inputs: D = f32, A = B = bf16, A MN-major,
// B K-major, N = 16, M = 128.
constexpr uint32_t kIdescBf16 = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (0u << 16) | ((16u >> 3) << 17) |
                                ((128u >> 4) << 24);

__global__ void __launch_bounds__(kTcThreads, 2)
bsr_tc_bf16_kernel(const __grid_constant__ CUtensorMap tmapB, const TcArgs a) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // stage ring first (1024-byte aligned for the 128-byte swizzle), barriers after it
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + a.stages * kTcStageBytes);
    uint64_t *full = bars, *empty = bars + kTcStages, *acc_full = bars + 2 * kTcStages,
             *acc_empty = bars + 2 * kTcStages + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kTcStages + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    int32_t *meta_b0 = reinterpret_cast<int32_t *>(tmem_slot + 2);
    int32_t *meta_nblk = meta_b0 + kTcBatchItems;
    int32_t *meta_col = meta_nblk + kTcBatchItems;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < a.stages; ++s) {
            mbar_init(smem_u32(full + s), 1);
            mbar_init(smem_u32(empty + s), 1);
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
    // overlapped round trips), then the three roles run through the batch from there.
    const int my_items = (nitems - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    uint32_t p_stage = 0, p_phase = 0, p_filled = 0, p_fill_parity = 0;   // producer ring state
    uint32_t m_stage = 0, m_phase = 0;                                   // MMA ring state
    uint32_t it = 0;                                                      // items done (accumulator slot / parity)
    bool ok = true;

    for (int batch0 = 0; batch0 < my_items; batch0 += kTcBatchItems) {
        const int bn = min(kTcBatchItems, my_items - batch0);
        if (batch0 != 0) {
            __syncthreads();                       // everybody is done with the previous batch's metadata
            if (*abort_flag) break;                // uniform: read after the barrier
        }
        for (int j = threadIdx.x; j < bn; j += kTcThreads) {
            const int I = (blockIdx.x + (batch0 + j) * gridDim.x) / a.nslab;
            const int b0 = __ldg(a.browptr + I);
            meta_b0[j] = b0;
            meta_nblk[j] = __ldg(a.browptr + I + 1) - b0;
        }
        __syncthreads();
        {
            int off = 0;
            for (int j = 0; j < bn; ++j) {
                const int nb = meta_nblk[j], b0 = meta_b0[j];
                for (int k = threadIdx.x; k < nb && off + k < kTcBatchBlocks; k += kTcThreads)
                    meta_col[off + k] = __ldg(a.bcol + b0 + k);
                off += nb;
            }
        }
        __syncthreads();

        if (warp == 0) {
            // -------------------------------------------------------------- TMA producer
            if (lane == 0) {
                int off = 0;
                for (int j = 0; j < bn && ok; ++j) {
                    const int item = blockIdx.x + (batch0 + j) * gridDim.x;
                    const int n0 = (item % a.nslab) * kTcSlabCols;
                    const int mt_n = min(2, (a.N - n0 + 127) / 128);
                    const int nb = meta_nblk[j], b0 = meta_b0[j];
                    for (int k = 0; k < nb; ++k) {
                        const int krow = ((off + k < kTcBatchBlocks) ? meta_col[off + k] : __ldg(a.bcol + b0 + k)) * 16;
                        if (!(ok = mbar_wait(smem_u32(empty + p_stage), p_phase ^ 1, abort_flag, a.error, 1))) break;
                        p_filled |= 1u << p_stage;
                        p_fill_parity = (p_fill_parity & ~(1u << p_stage)) | (p_phase << p_stage);
                        const uint32_t sbase = smem_u32(smem + p_stage * kTcStageBytes);
                        const uint32_t fb = smem_u32(full + p_stage);
                        const uint32_t slab_bytes = (a.debug & 8) ? 0u : (a.map3d ? a.box_bytes : mt_n * 4096);
                        mbar_expect_tx(fb, slab_bytes + ((a.debug & 4) ? 0u : 512u));
                        if (a.debug & 8) {
                        } else if (a.map3d) {
                            // one copy brings all 64-column groups of the slab: [group][16 rows][128 B]
                            tma_load_3d(sbase, &tmapB, 0, krow, n0 / 64, fb);
                        } else {
                            for (int h = 0; h < 2 * mt_n; ++h) tma_load_2d(sbase + h * 2048, &tmapB, n0 + h * 64, krow, fb);
                        }
                        if (!(a.debug & 4))
                            bulk_load(sbase + kTcBlockOff,
                                      static_cast<const uint8_t *>(a.bmma) + static_cast<int64_t>(b0 + k) * 512, 512, fb);
                        if (++p_stage == a.stages) {
                            p_stage = 0;
                            p_phase ^= 1;
                        }
                    }
                    off += nb;
                }
            }
        } else if (warp == 1) {
            // -------------------------------------------------------------- MMA issuer
            if (lane == 0) {
                uint32_t mit = it;
                for (int j = 0; j < bn && ok; ++j, ++mit) {
                    const int item = blockIdx.x + (batch0 + j) * gridDim.x;
                    const int n0 = (item % a.nslab) * kTcSlabCols;
                    const int mt_n = min(2, (a.N - n0 + 127) / 128);
                    const int nb = meta_nblk[j];
                    const uint32_t as = mit & 1, aphase = (mit >> 1) & 1;
                    if (!(ok = mbar_wait(smem_u32(acc_empty + as), aphase ^ 1, abort_flag, a.error, 2))) break;
                    tc_fence_after();
                    for (int b = 0; b < nb; ++b) {
                        if (!(ok = mbar_wait(smem_u32(full + m_stage), m_phase, abort_flag, a.error, 3))) break;
                        tc_fence_after();
                        const uint32_t sbase = smem_u32(smem + m_stage * kTcStageBytes);
                        const uint64_t bdesc = smem_desc(sbase + kTcBlockOff, a.lbo_b, a.sbo_b, 0);
                        for (int mt = 0; mt < mt_n; ++mt) {
                            const uint64_t adesc = smem_desc(sbase + mt * 4096, a.lbo_a, a.sbo_a, 2);
                            if (!(a.debug & 1)) tc_mma_f16(tmem_base + as * 32 + mt * 16, adesc, bdesc, kIdescBf16, b > 0 ? 1u : 0u);
                        }
                        if (a.debug & 32) mbar_arrive(smem_u32(empty + m_stage));
                        else tc_commit(smem_u32(empty + m_stage));   // the stage is free once these MMAs retire
                        if (++m_stage == a.stages) {
                            m_stage = 0;
                            m_phase ^= 1;
                        }
                    }
                    if (!ok) break;
                    if (nb > 0) tc_commit(smem_u32(acc_full + as));
                    else mbar_arrive(smem_u32(acc_full + as));   // block-row without blocks: nothing to wait for
                }
            }
        } else {
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
                            if (row < a.M && !(a.debug & 2)) {
                                float v = a.alpha * r[mt][rr];
                                if (a.beta != 0.f) v = fmaf(a.beta, cold[mt][rr], v);
                                a.C[row * a.ldc + col] = v;
                            }
                        }
                    }
                }
            }
        }
        it += bn;
    }
    if (warp == 0 && lane == 0 && *abort_flag) {
        // give the copies this thread issued a bounded time to land before shared memory is released
        for (int s2 = 0; s2 < a.stages; ++s2)
            if (p_filled & (1u << s2))
                for (uint32_t i = 0; i < 65536 && !mbar_try_wait(smem_u32(full + s2), (p_fill_parity >> s2) & 1); ++i) {
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

}  // namespace sd
