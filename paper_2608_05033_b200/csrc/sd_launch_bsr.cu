#include <cstdio>
#include <cstdlib>

#include "sd_launch.cuh"
#include "sd_bsr_simt.cuh"
#include "sd_bsr_tc.cuh"

namespace sd {

cudaError_t run_bsr_simt(const BsrArgs &a, int dtype, bool vec, cudaStream_t st) {
    if (dtype == SD_F32) return launch_bsr_simt<float>(a, vec, st);
    return launch_bsr_simt<__nv_bfloat16>(a, vec, st);
}

cudaError_t build_bsr_mma_image(const void *bval, void *img, int64_t nnzb, int dtype, cudaStream_t st) {
    if (dtype != SD_BF16 || nnzb == 0) return cudaSuccess;
    const int64_t n = nnzb * 256;
    bsr_mma_image_bf16_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(
        static_cast<const uint16_t *>(bval), static_cast<uint16_t *>(img), nnzb);
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

bool bsr_tc_usable(const BsrArgs &a, int dtype) {
    if (dtype != SD_BF16 || a.bval_mma == nullptr) return false;
    if (a.N < 64 || a.N % 8 != 0 || a.ldb % 8 != 0) return false;
    if (reinterpret_cast<uintptr_t>(a.B) & 15u) return false;
    return encode_tiled() != nullptr;
}

cudaError_t run_bsr_tc(const BsrArgs &a, int dtype, int32_t *error_word, int sm_count, cudaStream_t st) {
    (void)dtype;
    CUtensorMap map;
    // N a multiple of 64: a 3-D view {64 columns of a group, K rows, N/64 groups} lets one TMA
    // copy fetch a whole 16 x 256 slab as [group][row][128 bytes], the tensor-core operand image.
    // Otherwise the plain 2-D view is read with one 64-column box per copy (out-of-range columns
    // come back as zeros).
    const bool map3d = a.N % 64 == 0 && !getenv("SD_TC_MAP2D");
    CUresult r;
    if (map3d) {
        const int groups = a.N / 64;
        const cuuint64_t gdim[3] = {64, static_cast<cuuint64_t>(a.K), static_cast<cuuint64_t>(groups)};
        const cuuint64_t gstride[2] = {static_cast<cuuint64_t>(a.ldb) * 2, 128};
        const cuuint32_t box[3] = {64, 16, static_cast<cuuint32_t>(groups < 4 ? groups : 4)};
        const cuuint32_t estr[3] = {1, 1, 1};
        r = encode_tiled()(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(a.B), gdim, gstride, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(a.N), static_cast<cuuint64_t>(a.K)};
        const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(a.ldb) * 2};
        const cuuint32_t box[2] = {64, 16};
        const cuuint32_t estr[2] = {1, 1};
        r = encode_tiled()(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(a.B), gdim, gstride, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;

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
    t.alpha = a.alpha;
    t.beta = a.beta;
    t.error = error_word;
    t.map3d = map3d ? 1 : 0;
    t.stages = getenv("SD_TC_STAGES") ? atoi(getenv("SD_TC_STAGES")) : kTcDefaultStages;
    if (t.stages < 1 || t.stages > kTcStages) t.stages = kTcStages;
    t.debug = getenv("SD_TC_DEBUG") ? atoi(getenv("SD_TC_DEBUG")) : 0;
    t.box_bytes = map3d ? 2048 * ((a.N / 64) < 4 ? (a.N / 64) : 4) : 0;
    // operand "A" (slab of B): MN-major, 128-byte swizzle; 64-column atoms 2048 bytes apart,
    // 8-row k-groups 1024 bytes apart.  Operand "B" (the block): K-major, unswizzled 8x8 cores.
    t.lbo_a = 2048;
    t.sbo_a = 1024;
    t.lbo_b = 256;
    t.sbo_b = 128;
    if (const char *e = getenv("SD_TC_DESC")) {   // bench-only override of the descriptor strides
        unsigned v[4];
        if (sscanf(e, "%u,%u,%u,%u", &v[0], &v[1], &v[2], &v[3]) == 4) {
            t.lbo_a = v[0]; t.sbo_a = v[1]; t.lbo_b = v[2]; t.sbo_b = v[3];
        }
    }
    const int smem = t.stages * kTcStageBytes + 2048 + 4 * (2 * kTcBatchItems + kTcBatchBlocks);
    const int ctas_per_sm = getenv("SD_TC_CTAS") ? atoi(getenv("SD_TC_CTAS")) : kTcCtasPerSm;
    static int attr_set = 0;
    if (attr_set < smem) {
        cudaError_t e = cudaFuncSetAttribute(bsr_tc_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        attr_set = smem;
    }
    if (t.debug & 64) {
        int one = 1;
        cudaMemcpyToSymbol(g_tc_test_wait, &one, sizeof one);
    }
    const int items = t.Mb * t.nslab;
    const int grid = items < sm_count * ctas_per_sm ? items : sm_count * ctas_per_sm;
    bsr_tc_bf16_kernel<<<grid, kTcThreads, smem, st>>>(map, t);
    return cudaGetLastError();
}

}  // namespace sd
