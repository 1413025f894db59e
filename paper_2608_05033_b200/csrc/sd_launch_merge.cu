#include "sd_launch.cuh"
#include "sd_merge.cuh"
#include "sd_rowsplit.cuh"

namespace sd {

cudaError_t run_merge(const MergeArgs &m, int dtype, bool vec, const int32_t *fix_tiles, int32_t nfix,
                      cudaStream_t st) {
    const int vecw = dtype == SD_F32 ? 4 : 8;
    const LaneGeom g = lane_geometry(m.s.N, vec, vecw);
    cudaError_t e = (dtype == SD_F32) ? launch_merge<float>(m, vec, g.lpr, st)
                                      : launch_merge<__nv_bfloat16>(m, vec, g.lpr, st);
    if (e != cudaSuccess) return e;
    if (nfix > 0) {
        merge_fixup_kernel<<<nfix, 32 * kFixChains, 0, st>>>(m, fix_tiles, nfix, kMergeTile);
        e = cudaGetLastError();
    }
    return e;
}

}  // namespace sd
