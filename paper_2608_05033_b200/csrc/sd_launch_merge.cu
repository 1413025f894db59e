#include "sd_launch.cuh"
#include "sd_merge.cuh"
#include "sd_rowsplit.cuh"

namespace sd {

cudaError_t run_merge(const MergeArgs &m, int dtype, bool vec, const int32_t *fix_short, int32_t nshort,
                      const int32_t *fix_long, int32_t nlong, cudaStream_t st) {
    const int vecw = dtype == SD_F32 ? 4 : 8;
    const LaneGeom g = lane_geometry(m.s.N, vec, vecw, false);
    cudaError_t e = (dtype == SD_F32) ? launch_merge<float>(m, vec, g.lpr, g.nv, st)
                                      : launch_merge<__nv_bfloat16>(m, vec, g.lpr, g.nv, st);
    if (e != cudaSuccess) return e;
    if (nshort > 0) {
        merge_fixup_short_kernel<<<(nshort + 7) / 8, 256, 0, st>>>(m, fix_short, nshort, kMergeTile);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (nlong > 0) {
        merge_fixup_long_kernel<<<nlong, 32 * kFixChains, 0, st>>>(m, fix_long, nlong, kMergeTile);
        e = cudaGetLastError();
    }
    return e;
}

}  // namespace sd
