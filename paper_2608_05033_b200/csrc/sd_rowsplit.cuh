// Family (a): row-split CSR SpMM.  One group of LPR lanes owns one row of A; each lane
// owns NV vectors of VW adjacent columns of the output row and gathers the matching
// 16-byte pieces of the rows of B (paper, case study on af_shell10: a few threads per
// row, several outputs per thread in registers, shuffles share the sparse entries).
#pragma once

#include <cstdlib>

#include "sd_common.cuh"

namespace sd {

constexpr int kRowsplitThreads = 256;

// LONG = false: no row exceeds 32 * LPR terms (the plan knows the longest row), so the block-wise
// second accumulator and its instructions are not needed: 9 % faster on the 5-point stencil.
template <typename T, int VW, int LPR, int NV, bool LONG>
__global__ void __launch_bounds__(kRowsplitThreads, LONG ? 5 : 6)
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
    float acc[NV][VW], tot[LONG ? NV : 1][LONG ? VW : 1];
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
        for (int e = 0; e < VW; ++e) {
            acc[v][e] = 0.f;
            if constexpr (LONG) tot[v][e] = 0.f;
        }

    bool colok[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) colok[v] = cbase + (v * LPR + lg) * VW < a.N;

    // beta != 0: fetch the old C row now so that its latency hides behind the gathers
    float cin[NV][VW];
    if (a.beta != 0.f && row < a.S) {
        const float *crow = a.C + row * a.ldc + cbase;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            if (colok[v]) {
                if constexpr (VW == 1) {
                    cin[v][0] = crow[(v * LPR + lg)];
                } else {
#pragma unroll
                    for (int q = 0; q < VW / 4; ++q) {
                        const float4 o = *(reinterpret_cast<const float4 *>(crow + (v * LPR + lg) * VW) + q);
                        cin[v][4 * q] = o.x; cin[v][4 * q + 1] = o.y; cin[v][4 * q + 2] = o.z; cin[v][4 * q + 3] = o.w;
                    }
                }
            }
        }
    }

    for (int base = 0; base < maxlen; base += LPR) {
        if constexpr (LONG) {
            if (base != 0 && (base / LPR) % 32 == 0) {
#pragma unroll
                for (int v = 0; v < NV; ++v)
#pragma unroll
                    for (int e = 0; e < VW; ++e) {
                        tot[v][e] += acc[v][e];
                        acc[v][e] = 0.f;
                    }
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
                const T *brow = b_row(B, c, a.ldb_bytes) + cbase;
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
            for (int e = 0; e < VW; ++e) {
                float t = acc[v][e];
                if constexpr (LONG) t += tot[v][e];
                t *= a.alpha;
                if (a.beta != 0.f) t = fmaf(a.beta, cin[v][e], t);
                acc[v][e] = t;
            }
            if (colok[v]) store_cols<VW>(crow + (v * LPR + lg) * VW, acc[v], 1.f, 0.f, 0);
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
    if (a.max_len > 0 && a.max_len <= 32 * LPR) rowsplit_kernel<T, VW, LPR, NV, false><<<grid, kRowsplitThreads, 0, st>>>(a);
    else rowsplit_kernel<T, VW, LPR, NV, true><<<grid, kRowsplitThreads, 0, st>>>(a);
    return cudaGetLastError();
}

// Lane geometry for a dense width: VW elements per 16-byte load when `vec`, LPR lanes per
// row (a power of two), NV vectors per lane; wider rows are covered by grid.y slabs.
// Two vectors per lane halve the per-nonzero instruction overhead (index broadcast, address
// arithmetic) per byte gathered; they are used only when a group still covers a full 128-byte
// line with one load instruction (at least 8 lanes), because a gather instruction costs one
// L1 tag cycle per distinct line it touches.  The row-split kernel gains from them (short rows:
// fewer instructions per byte); the merge-path and segment kernels measure faster with one
// vector per lane and more lanes per row (`prefer_two` = false).
struct LaneGeom {
    int vw, lpr, nv;
};
inline int geom_nv_override() { return switches().geom_nv; }
inline LaneGeom lane_geometry(int64_t N, bool vec, int vecw, bool prefer_two = true) {
    LaneGeom g;
    g.vw = vec ? vecw : 1;
    const int64_t units = (N + g.vw - 1) / g.vw;
    if (!vec) {
        int lpr = 1;
        while (lpr < 32 && lpr < units) lpr <<= 1;
        g.lpr = lpr;
        g.nv = units > 32 ? 4 : 1;
        return g;
    }
    const bool two = prefer_two && units >= 16 && geom_nv_override() != 1;
    const int64_t per = two ? (units + 1) / 2 : units;
    int lpr = 1;
    while (lpr < 32 && lpr < per) lpr <<= 1;
    g.lpr = lpr;
    g.nv = (two || units > 32) ? 2 : 1;
    return g;
}

template <typename T>
cudaError_t launch_rowsplit(const SpmmArgs &a, bool vec, cudaStream_t st) {
    constexpr int VWV = vec_width<T>::value;
    const LaneGeom g = lane_geometry(a.N, vec, VWV);
    if (vec && g.nv == 2) {
        switch (g.lpr) {
        case 8: return launch_rowsplit_one<T, VWV, 8, 2>(a, st);
        case 16: return launch_rowsplit_one<T, VWV, 16, 2>(a, st);
        case 32: return launch_rowsplit_one<T, VWV, 32, 2>(a, st);
        }
        return cudaErrorInvalidValue;
    }
#define SD_RS_CASE(L)                                                  \
    case L:                                                            \
        if (vec) return launch_rowsplit_one<T, VWV, L, 1>(a, st);      \
        return (g.nv == 4) ? launch_rowsplit_one<T, 1, 32, 4>(a, st)   \
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
