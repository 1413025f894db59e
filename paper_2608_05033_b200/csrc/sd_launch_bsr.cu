#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "sd_launch.cuh"
#include "sd_bsr_simt.cuh"
#include "sd_bsr_tc.cuh"

namespace sd {

cudaError_t run_bsr_simt(const BsrArgs &a, int dtype, bool vec, cudaStream_t st) {
    if (dtype == SD_F32) return launch_bsr_simt<float>(a, vec, st);
    return launch_bsr_simt<__nv_bfloat16>(a, vec, st);
}

cudaError_t build_bsr_mma_image(const void *bval, void *img, int64_t nnzb, int dtype, cudaStream_t st) {
    if (nnzb == 0) return cudaSuccess;
    const int64_t n = nnzb * 256;
    const unsigned blocks = static_cast<unsigned>((n + 255) / 256);
    if (dtype == SD_BF16)
        bsr_mma_image_bf16_kernel<<<blocks, 256, 0, st>>>(static_cast<const uint16_t *>(bval), static_cast<uint16_t *>(img),
                                                          nnzb);
    else
        bsr_mma_image_tf32_kernel<<<blocks, 256, 0, st>>>(static_cast<const float *>(bval), static_cast<float *>(img), nnzb);
    return cudaGetLastError();
}

// Block-row ranges of about equal cost for the CTAs of the tensor-core kernel: a block-row costs
// 8 units per block plus 2 for its accumulator hand-over, so the running cost up to block-row I is
// F(I) = 8*browptr[I] + 2*I; part[c] is the first I with F(I) >= c*F(Mb)/nparts.
static __global__ void bsr_partition_kernel(const int32_t *__restrict__ browptr, int32_t Mb, int32_t nparts,
                                            int32_t *__restrict__ part) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c > nparts) return;
    if (c == nparts) {
        part[c] = Mb;
        return;
    }
    const int64_t total = 8ll * browptr[Mb] + 2ll * Mb;
    const int64_t target = total / nparts * c + total % nparts * c / nparts;
    int lo = 0, hi = Mb;   // first I in [0, Mb] with F(I) >= target
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (8ll * browptr[mid] + 2ll * mid >= target) hi = mid;
        else lo = mid + 1;
    }
    part[c] = lo;
}

cudaError_t build_bsr_partition(const int32_t *browptr, int32_t Mb, int32_t nparts, int32_t *part, cudaStream_t st) {
    bsr_partition_kernel<<<(nparts + 256) / 256, 256, 0, st>>>(browptr, Mb, nparts, part);
    return cudaGetLastError();
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// The tensor-core kernel reads B through a 3-D TMA view {one 128-byte column group, K rows,
// N / group columns}: N must be a multiple of the group (64 bf16 / 32 fp32 columns), the base
// 16-byte aligned and the row pitch a multiple of 16 bytes.  Its epilogue stores 16-byte vectors
// of C: base 16-byte aligned, ldc a multiple of 4.
bool bsr_tc_usable(const BsrArgs &a, int dtype) {
    if (a.bval_mma == nullptr || a.part == nullptr || a.nparts < 1) return false;
    const int group = dtype == SD_BF16 ? 64 : 32;
    const int es = dtype == SD_BF16 ? 2 : 4;
    if (a.N < group || a.N % group != 0 || (a.ldb * es) % 16 != 0) return false;
    if (reinterpret_cast<uintptr_t>(a.B) & 15u) return false;
    if ((reinterpret_cast<uintptr_t>(a.C) & 15u) || a.ldc % 4 != 0) return false;
    return encode_tiled() != nullptr;
}

cudaError_t run_bsr_tc(const BsrArgs &a, int dtype, int32_t *error_word, int sm_count, cudaStream_t st) {
    const bool tf32 = dtype == SD_F32;
    const int group = tf32 ? 32 : 64, es = tf32 ? 4 : 2;
    const int groups = a.N / group, box_groups = groups < 256 / group ? groups : 256 / group;
    static_assert(sizeof(CUtensorMap) == sizeof(TcMapCache::map), "the plan keeps a CUtensorMap as 128 opaque bytes");
    CUtensorMap map;
    TcMapCache *mc = a.map_cache;
    const bool cached = mc && mc->valid && mc->B == a.B && mc->ldb == a.ldb && mc->K == a.K && mc->N == a.N;
    if (cached) memcpy(&map, mc->map, sizeof map);
    // 3-D view {columns of a group, K rows, groups}: one copy fetches a whole 16 x 256 slab as
    // [group][row][128 bytes], which is the tensor-core operand image
    const cuuint64_t gdim[3] = {static_cast<cuuint64_t>(group), static_cast<cuuint64_t>(a.K), static_cast<cuuint64_t>(groups)};
    const cuuint64_t gstride[2] = {static_cast<cuuint64_t>(a.ldb) * es, 128};
    const cuuint32_t box[3] = {static_cast<cuuint32_t>(group), 16, static_cast<cuuint32_t>(box_groups)};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (!cached) {
        const CUresult r = encode_tiled()(&map, tf32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                                          const_cast<void *>(a.B), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                          tf32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
        if (mc) {
            memcpy(mc->map, &map, sizeof map);
            mc->B = a.B;
            mc->ldb = a.ldb;
            mc->K = a.K;
            mc->N = a.N;
            mc->valid = 1;
        }
    }

    TcArgs t;
    t.browptr = a.browptr;
    t.bcol = a.bcol;
    t.bmma = a.bval_mma;
    t.C = a.C;
    t.ldc = a.ldc;
    t.M = a.M;
    t.Mb = a.Mb;
    t.N = a.N;
    t.nslab = (a.N + kTcSlabCols - 1) / kTcSlabCols;
    t.part = a.part;
    t.alpha = a.alpha;
    t.beta = a.beta;
    t.error = error_word;
    t.box_bytes = box_groups * 2048;
    t.wide_store = ((reinterpret_cast<uintptr_t>(a.C) & 31u) == 0 && a.ldc % 8 == 0) ? 1 : 0;
    // ring geometry (bench-only overrides through the environment); one CTA per SM, its ring
    // takes most of the shared memory: bf16 3 slots of 8 blocks (8.5 KB per block), fp32 3 slots
    // of 2 blocks (34 KB per block).  A barrier round trip costs far more than a block's work,
    // so slots hold several blocks.
    const Switches &sw = switches();
    t.sb = tf32 ? (sw.tc32_sb ? sw.tc32_sb : 2) : (sw.tc_sb ? sw.tc_sb : 8);
    t.stages = tf32 ? (sw.tc32_stages ? sw.tc32_stages : 3) : (sw.tc_stages ? sw.tc_stages : 3);
    if (t.sb < 1) t.sb = 1;
    if (t.sb > 32) t.sb = 32;   // one mask bit per block of a ring slot
    if (t.stages < 1) t.stages = 1;
    if (t.stages > kTcMaxStages) t.stages = kTcMaxStages;
    const int smem = t.stages * tc_stage_bytes(tf32, t.sb) + 2048 + 8 * (3 * kTcMaxStages + 8) + 4 * (2 * kTcBatchItems + kTcBatchBlocks + 2 * tc_mask_words(t.sb));
    if (smem > 227 * 1024) return cudaErrorInvalidValue;
    // the opt-in to more than 48 KB of dynamic shared memory is a per-device attribute of the kernel
    static std::atomic<int> attr_set[kMaxDevices][2];
    const int dev = current_device();
    if (dev >= kMaxDevices || attr_set[dev][tf32].load(std::memory_order_acquire) < smem) {
        cudaError_t e = tf32 ? cudaFuncSetAttribute(bsr_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)
                             : cudaFuncSetAttribute(bsr_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        e = tf32 ? cudaFuncSetAttribute(bsr_tc_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)
                 : cudaFuncSetAttribute(bsr_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev < kMaxDevices) attr_set[dev][tf32].store(smem, std::memory_order_release);
    }
    const int grid = a.nparts;
    (void)sm_count;
    if (a.test_wait_expiry) {
        if (tf32) bsr_tc_kernel<true, true><<<grid, kTcThreadsTf32, smem, st>>>(map, t);
        else bsr_tc_kernel<false, true><<<grid, kTcThreadsBf16, smem, st>>>(map, t);
    } else if (tf32) {
        bsr_tc_kernel<true, false><<<grid, kTcThreadsTf32, smem, st>>>(map, t);
    } else {
        bsr_tc_kernel<false, false><<<grid, kTcThreadsBf16, smem, st>>>(map, t);
    }
    return cudaGetLastError();
}

}  // namespace sd
