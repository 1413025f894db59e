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
#include "sd_segment.cuh"

namespace sd {

constexpr int kLightThreads = 256;

template <typename T, int VW, int LPR, int NV, int R>
__device__ __forceinline__ void light_rows_body(const SpmmArgs &a, const unsigned bx) {
    const int lg = threadIdx.x % LPR;
    const int64_t g = (static_cast<int64_t>(bx) * kLightThreads + threadIdx.x) / LPR;
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

// The hybrid family in one launch: the first `gc` CTAs walk the chunks of the heavy rows (persistent, grid-stride), the
// next `gm` the rows of medium length (likewise), the rest the short rows (a batch of rows per lane group each).  CTAs
// are placed in index order, so the chunk CTAs take the SMs first and the others fill in as they retire: what side
// streams and a high stream priority would give, without depending on how streams map to the GPU's hardware queues
// (two of a plan's streams landing on the same queue serialised them: 0.20 against 0.15 ms per call for every third
// and fourth plan instance of a process) and without an order race between the kernels of calls queued back to back.
template <typename T, int VW, int LPR, int NV, int R>
__global__ void __launch_bounds__(kSegThreads, 4)
hybrid_fused_kernel(const SpmmArgs chunks, const SpmmArgs medium, const SpmmArgs light, const unsigned gc, const unsigned gm) {
    static_assert(kSegThreads == kLightThreads, "one CTA size for all roles");
    if (blockIdx.x < gc) seg_body<T, VW, LPR, NV, 1>(chunks, blockIdx.x, gc);
    else if (blockIdx.x < gc + gm) seg_body<T, VW, LPR, NV, 2>(medium, blockIdx.x - gc, gm);
    else light_rows_body<T, VW, LPR, NV, R>(light, blockIdx.x - gc - gm);
}

template <typename T, int VW, int LPR, int NV>
cudaError_t launch_hybrid_one(const SpmmArgs &ca, const SpmmArgs &ma, const SpmmArgs &la, cudaStream_t st) {
    // four rows per lane group at four CTAs per SM (64 registers, a few spilled words in the short-row role): measured
    // against 2, 6 and 8 rows and against 3 and 5 CTAs per SM, 4 to 20 % ahead of each on four workloads (fp32 values, one
    // 16-byte vector per lane); lanes that hold eight accumulators per row take two rows
    constexpr int R = (NV * VW >= 8) ? 2 : 4;
    auto kernel = hybrid_fused_kernel<T, VW, LPR, NV, R>;
    if (ca.load_only) {
        cudaFuncAttributes at;
        return cudaFuncGetAttributes(&at, kernel);
    }
    static std::atomic<int> occ_cache[kMaxDevices];
    const int64_t cap = static_cast<int64_t>(sm_count_cached()) * occupancy_cached(occ_cache, kernel, kSegThreads);
    const int per_cta = kSegThreads / LPR;
    const int64_t need_c = (ca.S + per_cta - 1) / per_cta, need_m = (ma.S + per_cta - 1) / per_cta;
    const int64_t need_l = ((la.S + R - 1) / R + per_cta - 1) / per_cta;
    const unsigned gc = static_cast<unsigned>(need_c < cap ? need_c : cap), gm = static_cast<unsigned>(need_m < cap ? need_m : cap);
    const int64_t total = static_cast<int64_t>(gc) + gm + need_l;
    if (total == 0) return cudaSuccess;
    if (total > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    dim3 grid(static_cast<unsigned>(total), static_cast<unsigned>((ca.N + LPR * NV * VW - 1) / (LPR * NV * VW)));
    kernel<<<grid, kSegThreads, 0, st>>>(ca, ma, la, gc, gm);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_hybrid(const SpmmArgs &ca, const SpmmArgs &ma, const SpmmArgs &la, bool vec, cudaStream_t st) {
    constexpr int VWV = vec_width<T>::value;
    const LaneGeom g = lane_geometry(ca.N, vec, VWV, false);
    if (vec && g.nv == 2) {
        switch (g.lpr) {
        case 8: return launch_hybrid_one<T, VWV, 8, 2>(ca, ma, la, st);
        case 16: return launch_hybrid_one<T, VWV, 16, 2>(ca, ma, la, st);
        case 32: return launch_hybrid_one<T, VWV, 32, 2>(ca, ma, la, st);
        }
        return cudaErrorInvalidValue;
    }
#define SD_HY_CASE(L)                                                        \
    case L:                                                                  \
        if (vec) return launch_hybrid_one<T, VWV, L, 1>(ca, ma, la, st);     \
        return (g.nv == 4) ? launch_hybrid_one<T, 1, 32, 4>(ca, ma, la, st)  \
                           : launch_hybrid_one<T, 1, L, 1>(ca, ma, la, st);
    switch (g.lpr) {
        SD_HY_CASE(1)
        SD_HY_CASE(2)
        SD_HY_CASE(4)
        SD_HY_CASE(8)
        SD_HY_CASE(16)
        SD_HY_CASE(32)
    }
#undef SD_HY_CASE
    return cudaErrorInvalidValue;
}

}  // namespace sd
