#include "sd_launch.cuh"
#include "sd_rowsplit.cuh"

namespace sd {

cudaError_t run_rowsplit(const SpmmArgs &a, int dtype, bool vec, cudaStream_t st) {
    if (dtype == SD_F32) return launch_rowsplit<float>(a, vec, st);
    return launch_rowsplit<__nv_bfloat16>(a, vec, st);
}

cudaError_t run_scale_c(float *C, int64_t ldc, int64_t M, int32_t N, float beta, cudaStream_t st) {
    const int64_t total = M * N;
    const int blocks = static_cast<int>(std::min<int64_t>((total + 255) / 256, 148 * 16));
    scale_c_kernel<<<blocks, 256, 0, st>>>(C, ldc, M, N, beta);
    return cudaGetLastError();
}

}  // namespace sd
