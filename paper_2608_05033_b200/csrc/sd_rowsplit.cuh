// Family (a): row-split CSR SpMM.  One group of LPR lanes owns one row of A; each lane
// owns NV vectors of VW adjacent columns of the output row and gathers the matching
// 16-byte pieces of the rows of B (paper, case study on af_shell10: a few threads per
// row, several outputs per thread in registers, shuffles share the sparse entries).
#pragma once

#include "sd_common.cuh"

namespace sd {

constexpr int kRowsplitThreads = 256;

template <typename T, int VW, int LPR, int NV>
__global__ void __launch_bounds__(kRowsplitThreads)
rowsplit_kernel(const SpmmArgs a) {
    constexpr unsigned FULL = 0xffffffffu;
    const int lg = threadIdx.x % LPR;  // lane inside the group
    const int64_t row = (static_cast<int64_t>(blockIdx.x) * kRowsplitThreads + threadIdx.x) / LPR;
    const int cbase = blockIdx.y * (LPR * NV * VW);
    const T *__restrict__ vals = static_cast<const T *>(a.vals);
    const T *__restrict__ B = static_cast<const T *>(a.B);

    int p0 = 0, len = 0;
    if (row < a.S) {
        p0 = __ldg(a.ptr + row);
        len = __ldg(a.ptr + row + 1) - p0;
    }
    // trip counts are made warp-uniform so that the shuffles below are always converged
    const int maxlen = (LPR == 32) ? len : __reduce_max_sync(FULL, len);

    // two-level accumulation: `acc` takes at most 32*LPR terms before it is folded into
    // `tot`, so that a very long row is summed in blocks rather than as one running sum
    float acc[NV][VW], tot[NV][VW];
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
        for (int e = 0; e < VW; ++e) acc[v][e] = tot[v][e] = 0.f;

    bool colok[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) colok[v] = cbase + (v * LPR + lg) * VW < a.N;

    for (int base = 0; base < maxlen; base += LPR) {
        if (base != 0 && (base / LPR) % 32 == 0) {
#pragma unroll
            for (int v = 0; v < NV; ++v)
#pragma unroll
                for (int e = 0; e < VW; ++e) {
                    tot[v][e] += acc[v][e];
                    acc[v][e] = 0.f;
                }
        }
        // the group fetches LPR (column, value) pairs with one coalesced load each ...
        int myc = 0;
        float myv = 0.f;
        if (base + lg < len) {
            myc = __ldg(a.colind + p0 + base + lg);
            myv = to_float(vals[p0 + base + lg]);
        }
        const int cnt = min(LPR, maxlen - base);
        // ... and hands them round by shuffle
#pragma unroll 4
        for (int q = 0; q < cnt; ++q) {
            const int c = (LPR == 1) ? myc : __shfl_sync(FULL, myc, q, LPR);
            const float av = (LPR == 1) ? myv : __shfl_sync(FULL, myv, q, LPR);
            if (base + q < len) {
                const T *brow = B + static_cast<int64_t>(c) * a.ldb + cbase;
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    if (colok[v]) {
                        float b[VW];
                        RowLoad<T, VW>::ld(brow + (v * LPR + lg) * VW, b);
#pragma unroll
                        for (int e = 0; e < VW; ++e) acc[v][e] = fmaf(av, b[e], acc[v][e]);
                    }
                }
            }
        }
    }

    if (row < a.S) {
        float *crow = a.C + row * a.ldc + cbase;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
#pragma unroll
            for (int e = 0; e < VW; ++e) tot[v][e] += acc[v][e];
            if (colok[v]) store_cols<VW>(crow + (v * LPR + lg) * VW, tot[v], a.alpha, a.beta, 0);
        }
    }
}

// C = beta * C for an M x N matrix (alpha == 0, or a matrix without nonzeros).
static __global__ void scale_c_kernel(float *C, int64_t ldc, int64_t M, int32_t N, float beta) {
    const int64_t total = M * N;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        float *p = C + (i / N) * ldc + (i % N);
        *p = (beta == 0.f) ? 0.f : beta * *p;
    }
}

template <typename T, int VW, int LPR, int NV>
cudaError_t launch_rowsplit_one(const SpmmArgs &a, cudaStream_t st) {
    const int rows_per_cta = kRowsplitThreads / LPR;
    dim3 grid(static_cast<unsigned>((a.S + rows_per_cta - 1) / rows_per_cta),
              static_cast<unsigned>((a.N + LPR * NV * VW - 1) / (LPR * NV * VW)));
    rowsplit_kernel<T, VW, LPR, NV><<<grid, kRowsplitThreads, 0, st>>>(a);
    return cudaGetLastError();
}

// Lane geometry for a dense width: VW elements per 16-byte load when `vec`, LPR lanes per
// row (a power of two), NV vectors per lane; wider rows are covered by grid.y slabs.
struct LaneGeom {
    int vw, lpr, nv;
};
inline LaneGeom lane_geometry(int64_t N, bool vec, int vecw) {
    LaneGeom g;
    g.vw = vec ? vecw : 1;
    int64_t units = (N + g.vw - 1) / g.vw;
    int lpr = 1;
    while (lpr < 32 && lpr < units) lpr <<= 1;
    g.lpr = lpr;
    g.nv = (units > 32) ? (vec ? 2 : 4) : 1;
    return g;
}

template <typename T>
cudaError_t launch_rowsplit(const SpmmArgs &a, bool vec, cudaStream_t st) {
    constexpr int VWV = vec_width<T>::value;
    const LaneGeom g = lane_geometry(a.N, vec, VWV);
#define SD_RS_CASE(L)                                                                  \
    case L:                                                                            \
        if (vec) return (g.nv == 2) ? launch_rowsplit_one<T, VWV, 32, 2>(a, st)        \
                                    : launch_rowsplit_one<T, VWV, L, 1>(a, st);        \
        return (g.nv == 4) ? launch_rowsplit_one<T, 1, 32, 4>(a, st)                   \
                           : launch_rowsplit_one<T, 1, L, 1>(a, st);
    switch (g.lpr) {
        SD_RS_CASE(1)
        SD_RS_CASE(2)
        SD_RS_CASE(4)
        SD_RS_CASE(8)
        SD_RS_CASE(16)
        SD_RS_CASE(32)
    }
#undef SD_RS_CASE
    return cudaErrorInvalidValue;
}

}  // namespace sd
