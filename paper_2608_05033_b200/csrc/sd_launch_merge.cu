#include "sd_launch.cuh"
#include "sd_merge.cuh"
#include "sd_coo.cuh"
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

// ---- narrow dense operands: COO segmented reduction --------------------------------------------
template <typename T, int N>
static cudaError_t launch_coo_n(const CooPlan &cp, const SpmmArgs &s, bool vec, int sm_count, cudaStream_t st) {
    const int64_t chunks1 = (cp.nnz + coo_chunk(N) - 1) / coo_chunk(N);
    const int64_t count2 = 2 * chunks1;
    const int64_t chunks2 = (count2 + kCooCarryChunk - 1) / kCooCarryChunk;
    const int64_t count3 = 2 * chunks2;
    // persistent grid: the CTAs that are resident together (the registers of the instance decide)
    static std::atomic<int> occ_vec[kMaxDevices], occ_plain[kMaxDevices];
    const int occ = vec ? occupancy_cached(occ_vec, coo_reduce_kernel<T, N, true, false>, 256)
                        : occupancy_cached(occ_plain, coo_reduce_kernel<T, N, false, false>, 256);
    auto grid_for = [&](int64_t chunks) {
        const int64_t want = (chunks + 7) / 8;   // 8 warps per CTA, one chunk per warp step
        const int64_t cap = static_cast<int64_t>(sm_count) * occ;
        return static_cast<unsigned>(want < cap ? (want > 0 ? want : 1) : cap);
    };
    CooArgs a;
    a.row = cp.row;
    a.colind = s.colind;
    a.vals = s.vals;
    a.B = s.B;
    a.ldb_bytes = s.ldb_bytes;
    a.count = cp.nnz;
    a.C = s.C;
    a.ldc = s.ldc;
    a.alpha = s.alpha;
    a.beta = s.beta;
    a.rowptr = cp.rowptr;
    a.M = cp.M;
    a.carry_row = cp.c1_row;
    a.carry_val = cp.c1_val;
    if (vec) coo_reduce_kernel<T, N, true, false><<<grid_for(chunks1), 256, 0, st>>>(a);
    else coo_reduce_kernel<T, N, false, false><<<grid_for(chunks1), 256, 0, st>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int32_t *frow = cp.c1_row;
    const float *fval = cp.c1_val;
    int64_t fcount = count2;
    if (count2 > kCooDirectFinal) {   // level 2: the carry list is reduced the same way
        CooArgs b = a;
        b.row = cp.c1_row;
        b.colind = nullptr;
        b.vals = cp.c1_val;
        b.B = nullptr;
        b.count = count2;
        b.carry_row = cp.c2_row;
        b.carry_val = cp.c2_val;
        coo_reduce_kernel<float, N, false, true><<<grid_for(chunks2), 256, 0, st>>>(b);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        frow = cp.c2_row;
        fval = cp.c2_val;
        fcount = count3;
    }
    coo_final_kernel<N><<<static_cast<unsigned>((fcount + 255) / 256), 256, 0, st>>>(frow, fval, fcount, s.C, s.ldc, s.alpha, s.beta);
    return cudaGetLastError();
}

template <typename T>
static cudaError_t launch_coo(const CooPlan &cp, const SpmmArgs &s, bool vec, int sm_count, cudaStream_t st) {
    switch (s.N) {
    case 1: return launch_coo_n<T, 1>(cp, s, false, sm_count, st);
    case 2: return launch_coo_n<T, 2>(cp, s, false, sm_count, st);
    case 3: return launch_coo_n<T, 3>(cp, s, false, sm_count, st);
    case 4: return launch_coo_n<T, 4>(cp, s, vec && sizeof(T) == 4, sm_count, st);
    default: return cudaErrorInvalidValue;
    }
}

// `vec`: B is 16-byte aligned and its row pitch a multiple of 16 bytes.
cudaError_t run_coo(const CooPlan &cp, const SpmmArgs &s, int dtype, bool vec, int sm_count, cudaStream_t st) {
    return dtype == SD_F32 ? launch_coo<float>(cp, s, vec, sm_count, st) : launch_coo<__nv_bfloat16>(cp, s, vec, sm_count, st);
}

cudaError_t build_coo_rows(const int32_t *rowptr, int64_t M, int64_t nnz, int32_t *row, cudaStream_t st) {
    if (nnz == 0) return cudaSuccess;
    coo_rows_kernel<<<static_cast<unsigned>((nnz + 255) / 256), 256, 0, st>>>(rowptr, M, nnz, row);
    return cudaGetLastError();
}

}  // namespace sd
