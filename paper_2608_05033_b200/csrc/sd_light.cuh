// Short rows of the hybrid family (a handful of nonzeros, most of them one or two), named by a list
// that is sorted by falling length.  A group of LPR lanes owns R consecutive list entries at once, so
// that R gathers (one per row) are in flight per lane at every step; rows of similar length share a
// warp.  Every list entry is a plan-time descriptor {row, first nonzero, column of the first nonzero,
// length}: the first gather of a row depends on nothing but its descriptor (two dependent memory
// round trips per one-nonzero row: descriptor, row of B; four without it: list, row pointer, column
// index, row of B), and the (column, value) pair of step j + 1 is requested before the gathers of step j.
// The lanes of a group read the same pair with one broadcast load: at these lengths that is cheaper
// than loading LPR pairs and shuffling them.  Rows without nonzeros are written too (C = beta * C).
#pragma once

#include "sd_common.cuh"
#include "sd_rowsplit.cuh"

namespace sd {

constexpr int kLightThreads = 256;

template <typename T, int VW, int LPR, int NV, int R>
__global__ void __launch_bounds__(kLightThreads)
light_rows_kernel(const SpmmArgs a) {
    const int lg = threadIdx.x % LPR;
    const int64_t g = (static_cast<int64_t>(blockIdx.x) * kLightThreads + threadIdx.x) / LPR;
    const int64_t r0 = g * R;
    if (r0 >= a.S) return;
    const int cbase = blockIdx.y * (LPR * NV * VW);
    const T *__restrict__ vals = static_cast<const T *>(a.vals);
    const T *__restrict__ Bl = static_cast<const T *>(a.B) + cbase + lg * VW;
    bool colok[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) colok[v] = cbase + (v * LPR + lg) * VW < a.N;

    int p[R], len[R], cn[R], maxlen = 0;
    float vn[R];
    int64_t row[R];
    bool mine[R];
#pragma unroll
    for (int u = 0; u < R; ++u) {
        mine[u] = r0 + u < a.S;
        const int4 d = mine[u] ? __ldg(a.desc + r0 + u) : make_int4(0, 0, 0, 0);
        row[u] = d.x;
        p[u] = d.y;
        cn[u] = d.z;
        len[u] = d.w;
        maxlen = max(maxlen, len[u]);
    }
#pragma unroll
    for (int u = 0; u < R; ++u) vn[u] = len[u] > 0 ? to_float(vals[p[u]]) : 0.f;
    float acc[R][NV][VW];
#pragma unroll
    for (int u = 0; u < R; ++u)
#pragma unroll
        for (int v = 0; v < NV; ++v)
#pragma unroll
            for (int e = 0; e < VW; ++e) acc[u][v][e] = 0.f;

    for (int j = 0; j < maxlen; ++j) {
        int c[R];
        float av[R];
#pragma unroll
        for (int u = 0; u < R; ++u) {
            c[u] = cn[u];
            av[u] = vn[u];
            const bool more = j + 1 < len[u];   // the next step's pair, requested before this step's gathers
            cn[u] = more ? __ldg(a.colind + p[u] + j + 1) : 0;
            vn[u] = more ? to_float(vals[p[u] + j + 1]) : 0.f;
        }
        float b[R][NV][VW];
#pragma unroll
        for (int u = 0; u < R; ++u) {
            const T *brow = b_row(Bl, c[u], a.ldb_bytes);
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                if (j < len[u] && colok[v]) {   // a row that has ended gathers nothing (its pair is (0, 0): row 0 of B may hold non-finite values)
                    RowLoad<T, VW>::ld(brow + v * LPR * VW, b[u][v]);
                } else {
#pragma unroll
                    for (int e = 0; e < VW; ++e) b[u][v][e] = 0.f;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < R; ++u)
#pragma unroll
            for (int v = 0; v < NV; ++v)
#pragma unroll
                for (int e = 0; e < VW; ++e) acc[u][v][e] = fmaf(av[u], b[u][v][e], acc[u][v][e]);
    }
#pragma unroll
    for (int u = 0; u < R; ++u) {
        if (!mine[u]) continue;
        float *crow = a.C + row[u] * a.ldc + cbase;
#pragma unroll
        for (int v = 0; v < NV; ++v)
            if (colok[v]) store_cols<VW>(crow + (v * LPR + lg) * VW, acc[u][v], a.alpha, a.beta, 0);
    }
}

template <typename T, int VW, int LPR, int NV>
cudaError_t launch_light_one(const SpmmArgs &a, cudaStream_t st) {
    constexpr int R = (NV * VW >= 8) ? 2 : 4;
    if (a.load_only) {
        cudaFuncAttributes at;
        return cudaFuncGetAttributes(&at, light_rows_kernel<T, VW, LPR, NV, R>);
    }
    const int64_t groups = (a.S + R - 1) / R;
    const int per_cta = kLightThreads / LPR;
    dim3 grid(static_cast<unsigned>((groups + per_cta - 1) / per_cta),
              static_cast<unsigned>((a.N + LPR * NV * VW - 1) / (LPR * NV * VW)));
    light_rows_kernel<T, VW, LPR, NV, R><<<grid, kLightThreads, 0, st>>>(a);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_light(const SpmmArgs &a, bool vec, cudaStream_t st) {
    constexpr int VWV = vec_width<T>::value;
    const LaneGeom g = lane_geometry(a.N, vec, VWV, false);
    if (vec && g.nv == 2) {
        switch (g.lpr) {
        case 8: return launch_light_one<T, VWV, 8, 2>(a, st);
        case 16: return launch_light_one<T, VWV, 16, 2>(a, st);
        case 32: return launch_light_one<T, VWV, 32, 2>(a, st);
        }
        return cudaErrorInvalidValue;
    }
#define SD_LT_CASE(L)                                               \
    case L:                                                         \
        if (vec) return launch_light_one<T, VWV, L, 1>(a, st);      \
        return (g.nv == 4) ? launch_light_one<T, 1, 32, 4>(a, st)   \
                           : launch_light_one<T, 1, L, 1>(a, st);
    switch (g.lpr) {
        SD_LT_CASE(1)
        SD_LT_CASE(2)
        SD_LT_CASE(4)
        SD_LT_CASE(8)
        SD_LT_CASE(16)
        SD_LT_CASE(32)
    }
#undef SD_LT_CASE
    return cudaErrorInvalidValue;
}

}  // namespace sd
