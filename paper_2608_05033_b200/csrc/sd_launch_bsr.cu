#include "sd_launch.cuh"
#include "sd_bsr_simt.cuh"

namespace sd {

cudaError_t run_bsr_simt(const BsrArgs &a, int dtype, bool vec, cudaStream_t st) {
    if (dtype == SD_F32) return launch_bsr_simt<float>(a, vec, st);
    return launch_bsr_simt<__nv_bfloat16>(a, vec, st);
}

}  // namespace sd
