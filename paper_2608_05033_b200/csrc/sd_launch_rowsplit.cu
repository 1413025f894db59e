#include "sd_launch.cuh"
#include "sd_rowsplit.cuh"
#include "sd_light.cuh"
#include "sd_rowsplit_narrow.cuh"
#include "sd_segment.cuh"

namespace sd {

cudaError_t run_rowsplit(const SpmmArgs &a, int dtype, bool vec, cudaStream_t st) {
    if (a.N >= 1 && a.N <= 4 && !switches().no_narrow) {   // one to four columns: lanes share a row, not its columns
        if (dtype == SD_F32) return launch_rowsplit_narrow<float>(a, vec, st);
        return launch_rowsplit_narrow<__nv_bfloat16>(a, vec, st);
    }
    // 8 to 64 columns (fp32; 8 to 128 bf16) as whole 16-byte vectors and long rows: several lane sets per row
    const int vw = dtype == SD_F32 ? 4 : 8;
    if (vec && a.N % vw == 0 && a.N / vw <= 16 && ((a.N / vw) & (a.N / vw - 1)) == 0) {
        const int lpr = a.N / vw;
        const int g = ksplit_group(a.mean_len, lpr);
        if (g > 1) {
            if (dtype == SD_F32) return launch_rowsplit_ksplit<float>(a, lpr, g, st);
            return launch_rowsplit_ksplit<__nv_bfloat16>(a, lpr, g, st);
        }
    }
    if (dtype == SD_F32) return launch_rowsplit<float>(a, vec, st);
    return launch_rowsplit<__nv_bfloat16>(a, vec, st);
}

// Hybrid family in one launch: chunks of the heavy rows (ca), rows of medium length (ma), short rows (la).
cudaError_t run_hybrid_fused(const SpmmArgs &ca, const SpmmArgs &ma, const SpmmArgs &la, int dtype, bool vec, cudaStream_t st) {
    if (dtype == SD_F32) return launch_hybrid<float>(ca, ma, la, vec, st);
    return launch_hybrid<__nv_bfloat16>(ca, ma, la, vec, st);
}

cudaError_t run_segments(const SpmmArgs &a, int dtype, bool vec, bool scratch, cudaStream_t st) {
    if (dtype == SD_F32) return launch_seg<float>(a, vec, scratch ? 1 : 0, st);
    return launch_seg<__nv_bfloat16>(a, vec, scratch ? 1 : 0, st);
}

cudaError_t run_single(const SpmmArgs &a, int dtype, bool vec, cudaStream_t st) {
    if (dtype == SD_F32) return launch_single<float>(a, vec, st);
    return launch_single<__nv_bfloat16>(a, vec, st);
}

cudaError_t run_chunk_reduce(const float *chunk_out, const int32_t *seg_chunk, const int32_t *seg_row, int64_t seg_begin,
                             int64_t seg_end, float *C, int64_t ldc, int32_t N, float alpha, float beta, cudaStream_t st,
                             int32_t skip_above) {
    const int64_t n = seg_end - seg_begin;
    if (N % 4 == 0)   // scratch rows are then 16-byte aligned
        chunk_reduce_kernel<4><<<static_cast<unsigned>((n + 7) / 8), 256, 0, st>>>(chunk_out, seg_chunk, seg_row, seg_begin,
                                                                                 seg_end, C, ldc, N, alpha, beta, skip_above);
    else
        chunk_reduce_kernel<1><<<static_cast<unsigned>((n + 7) / 8), 256, 0, st>>>(chunk_out, seg_chunk, seg_row, seg_begin,
                                                                                 seg_end, C, ldc, N, alpha, beta, skip_above);
    return cudaGetLastError();
}

cudaError_t run_chunk_reduce_wide(const float *chunk_out, const int32_t *seg_chunk, const int32_t *seg_row,
                                  const int32_t *list, int64_t count, float *C, int64_t ldc, int32_t N, float alpha,
                                  float beta, cudaStream_t st) {
    if (N % 4 == 0)
        chunk_reduce_wide_kernel<4><<<static_cast<unsigned>(count), 256, 0, st>>>(chunk_out, seg_chunk, seg_row, list, C, ldc,
                                                                                 N, alpha, beta);
    else
        chunk_reduce_wide_kernel<1><<<static_cast<unsigned>(count), 256, 0, st>>>(chunk_out, seg_chunk, seg_row, list, C, ldc,
                                                                                 N, alpha, beta);
    return cudaGetLastError();
}

// Loads every kernel instance that the multi-stream schedules of a plan of this value type and dense width can launch
// (both the 16-byte-vector and the scalar forms: which one runs depends on the operands' alignment at call time).
// With lazy module loading a kernel is otherwise loaded at its first launch; when that happens in the middle of a
// call that has just forked the plan's side streams, that plan's calls queued back to back stay 25 % slower for its
// whole life (measured on an earlier multi-stream form of the hybrid family: 0.311 against 0.246 ms at 8 columns on
// the R-MAT matrix; loading eagerly or at plan creation removes it).
cudaError_t preload_stream_kernels(int dtype, int32_t N) {
    SpmmArgs a{};
    a.N = N;
    a.load_only = true;
    const int vw = dtype == SD_F32 ? 4 : 8;
    for (int v = 0; v < 2; ++v) {
        const bool vec = v == 1;
        if (vec && N % vw != 0) continue;
        cudaError_t e = run_segments(a, dtype, vec, true, nullptr);
        if (e == cudaSuccess) e = run_segments(a, dtype, vec, false, nullptr);
        if (e == cudaSuccess) e = run_single(a, dtype, vec, nullptr);
        if (e != cudaSuccess) return e;
    }
    cudaFuncAttributes at;
    cudaError_t e = cudaFuncGetAttributes(&at, chunk_reduce_kernel<4>);
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&at, chunk_reduce_kernel<1>);
    return e;
}

cudaError_t run_scale_c(float *C, int64_t ldc, int64_t M, int32_t N, float beta, cudaStream_t st) {
    const int64_t total = M * N;
    const int blocks = static_cast<int>(std::min<int64_t>((total + 255) / 256, 148 * 16));
    scale_c_kernel<<<blocks, 256, 0, st>>>(C, ldc, M, N, beta);
    return cudaGetLastError();
}

}  // namespace sd
