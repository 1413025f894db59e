// Family (a) at dense widths up to 4 (SpMV included).  The wide kernel gives every lane a vector of
// output columns; with one to four columns there is nothing to split, and a thread per row would read
// its (column, value) pairs with a stride of one row length between neighbouring lanes.  Here G lanes
// share a row (the CSR-vector scheme of the SpMV literature the paper's template set builds on,
// Sec. 3.2): lane g takes the nonzeros p0 + g, p0 + g + G, ..., so a warp's loads of A are contiguous;
// every lane gathers the N-column row of B of its own nonzero; the G partial sums meet in log2(G)
// xor-shuffle steps and lane 0 writes the row.  G follows the mean row length (G = 1: a thread per row).  The order of every sum
// is fixed by (G, row length): results are run-to-run bit-identical.
#pragma once

#include "sd_coo.cuh"
#include "sd_common.cuh"

namespace sd {

constexpr int kNarrowThreads = 256;
constexpr int kNarrowFold = 64;   // terms a lane adds before its partial sum is folded into a second accumulator

template <typename T, int N, int G, bool VEC, bool LONG>
__global__ void __launch_bounds__(kNarrowThreads)
rowsplit_narrow_kernel(const SpmmArgs a) {
    constexpr unsigned FULL = 0xffffffffu;
    const int g = threadIdx.x % G;
    const int64_t row = (static_cast<int64_t>(blockIdx.x) * kNarrowThreads + threadIdx.x) / G;
    const T *__restrict__ vals = static_cast<const T *>(a.vals);
    int p0 = 0, p1 = 0;
    if (row < a.S) {
        p0 = __ldg(a.ptr + row);
        p1 = __ldg(a.ptr + row + 1);
    }
    float acc[N], tot[LONG ? N : 1];
#pragma unroll
    for (int e = 0; e < N; ++e) {
        acc[e] = 0.f;
        if constexpr (LONG) tot[e] = 0.f;
    }
    int p = p0 + g;
    [[maybe_unused]] int folded = 0;
    // four nonzeros per step while the row lasts: the index loads first, then the gathers, all in flight together
    for (; p + 3 * G < p1; p += 4 * G) {
        int c[4];
        float v[4], b[4][N];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            c[u] = __ldg(a.colind + p + u * G);
            v[u] = to_float(vals[p + u * G]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) coo_gather<T, N, VEC>(a.B, c[u], a.ldb_bytes, b[u]);
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int e = 0; e < N; ++e) acc[e] = fmaf(v[u], b[u][e], acc[e]);
        if constexpr (LONG) {
            folded += 2;
            if (folded >= kNarrowFold / 2) {
                folded = 0;
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    tot[e] += acc[e];
                    acc[e] = 0.f;
                }
            }
        }
    }
    // then two per step
    for (; p + G < p1; p += 2 * G) {
        const int c0 = __ldg(a.colind + p), c1 = __ldg(a.colind + p + G);
        const float v0 = to_float(vals[p]), v1 = to_float(vals[p + G]);
        float b0[N], b1[N];
        coo_gather<T, N, VEC>(a.B, c0, a.ldb_bytes, b0);
        coo_gather<T, N, VEC>(a.B, c1, a.ldb_bytes, b1);
#pragma unroll
        for (int e = 0; e < N; ++e) acc[e] = fmaf(v1, b1[e], fmaf(v0, b0[e], acc[e]));
        if constexpr (LONG) {
            if (++folded == kNarrowFold / 2) {
                folded = 0;
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    tot[e] += acc[e];
                    acc[e] = 0.f;
                }
            }
        }
    }
    if (p < p1) {
        const int c0 = __ldg(a.colind + p);
        const float v0 = to_float(vals[p]);
        float b0[N];
        coo_gather<T, N, VEC>(a.B, c0, a.ldb_bytes, b0);
#pragma unroll
        for (int e = 0; e < N; ++e) acc[e] = fmaf(v0, b0[e], acc[e]);
    }
#pragma unroll
    for (int e = 0; e < N; ++e) {
        if constexpr (LONG) acc[e] += tot[e];
#pragma unroll
        for (int d = G / 2; d >= 1; d >>= 1) acc[e] += __shfl_xor_sync(FULL, acc[e], d);
    }
    if (g == 0 && row < a.S) {
        float *crow = a.C + row * a.ldc;
        if constexpr (VEC && N == 4) {
            float4 r = make_float4(a.alpha * acc[0], a.alpha * acc[1], a.alpha * acc[2], a.alpha * acc[3]);
            if (a.beta != 0.f) {
                const float4 o = *reinterpret_cast<const float4 *>(crow);
                r.x = fmaf(a.beta, o.x, r.x); r.y = fmaf(a.beta, o.y, r.y);
                r.z = fmaf(a.beta, o.z, r.z); r.w = fmaf(a.beta, o.w, r.w);
            }
            *reinterpret_cast<float4 *>(crow) = r;
        } else {
#pragma unroll
            for (int e = 0; e < N; ++e) {
                float r = a.alpha * acc[e];
                if (a.beta != 0.f) r = fmaf(a.beta, crow[e], r);
                crow[e] = r;
            }
        }
    }
}

// The same scheme at 8 to 64 columns (one 16-byte vector per lane, LPR = 2..16 lanes across the columns):
// G such lane sets share a row, set k takes the nonzeros p0 + k, p0 + k + G, ...; the G partial rows meet by
// xor shuffles over the set index.  Pays when rows are long enough to keep G sets busy (the paper's
// af_shell10 case: a few threads per row, each holding several outputs); short rows keep the plain kernel.
template <typename T, int VW, int LPR, int G, bool LONG>
__global__ void __launch_bounds__(kNarrowThreads)
rowsplit_ksplit_kernel(const SpmmArgs a) {
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int LANES = LPR * G;                 // lanes per row
    const int lc = threadIdx.x % LPR;              // column vector of this lane
    const int gk = (threadIdx.x / LPR) % G;        // which share of the row's nonzeros
    const int64_t row = (static_cast<int64_t>(blockIdx.x) * kNarrowThreads + threadIdx.x) / LANES;
    const T *__restrict__ vals = static_cast<const T *>(a.vals);
    const T *__restrict__ Bl = static_cast<const T *>(a.B) + lc * VW;
    int p0 = 0, p1 = 0;
    if (row < a.S) {
        p0 = __ldg(a.ptr + row);
        p1 = __ldg(a.ptr + row + 1);
    }
    float acc[VW], tot[LONG ? VW : 1];
#pragma unroll
    for (int e = 0; e < VW; ++e) {
        acc[e] = 0.f;
        if constexpr (LONG) tot[e] = 0.f;
    }
    int p = p0 + gk;
    [[maybe_unused]] int folded = 0;
    for (; p + 3 * G < p1; p += 4 * G) {
        int c[4];
        float v[4], b[4][VW];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            c[u] = __ldg(a.colind + p + u * G);
            v[u] = to_float(vals[p + u * G]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) RowLoad<T, VW>::ld(b_row(Bl, c[u], a.ldb_bytes), b[u]);
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int e = 0; e < VW; ++e) acc[e] = fmaf(v[u], b[u][e], acc[e]);
        if constexpr (LONG) {
            if (++folded == kNarrowFold / 4) {
                folded = 0;
#pragma unroll
                for (int e = 0; e < VW; ++e) {
                    tot[e] += acc[e];
                    acc[e] = 0.f;
                }
            }
        }
    }
    for (; p < p1; p += G) {
        const int c0 = __ldg(a.colind + p);
        const float v0 = to_float(vals[p]);
        float b0[VW];
        RowLoad<T, VW>::ld(b_row(Bl, c0, a.ldb_bytes), b0);
#pragma unroll
        for (int e = 0; e < VW; ++e) acc[e] = fmaf(v0, b0[e], acc[e]);
    }
#pragma unroll
    for (int e = 0; e < VW; ++e) {
        if constexpr (LONG) acc[e] += tot[e];
#pragma unroll
        for (int d = LANES / 2; d >= LPR; d >>= 1) acc[e] += __shfl_xor_sync(FULL, acc[e], d);
    }
    if (gk == 0 && row < a.S) store_cols<VW>(a.C + row * a.ldc + lc * VW, acc, a.alpha, a.beta, 0);
}

inline int ksplit_override() { return switches().ksplit_g; }

// Lane sets per row for the kernel above: 1 (= use the plain row-split kernel) unless rows are long.
// Swept on uniform rows of 16 to 131 nonzeros at 8, 16 and 32 columns: about one set per eight nonzeros of
// the mean row, at most 16 lanes per row below a mean of 128 nonzeros and a whole warp from there.
inline int ksplit_group(int64_t mean_len, int lpr) {
    int g = 1;
    // 16 lanes across the columns (64 fp32 / 128 bf16 columns): two sets from a mean of 32 nonzeros
    const int lanes = (mean_len >= 128 || lpr >= 16) ? 32 : 16;
    const int64_t per_set = lpr >= 16 ? 16 : 8;
    if (const int o = ksplit_override()) g = o;
    else while (2 * g * lpr <= lanes && 2 * g <= mean_len / per_set) g <<= 1;
    while (g > 1 && g * lpr > 32) g >>= 1;
    return g;
}

template <typename T, int VW, int LPR, int G>
cudaError_t launch_ksplit_g(const SpmmArgs &a, cudaStream_t st) {
    if constexpr (LPR * G > 32) {
        return cudaErrorInvalidValue;
    } else {
        const int rows_per_cta = kNarrowThreads / (LPR * G);
        const unsigned grid = static_cast<unsigned>((a.S + rows_per_cta - 1) / rows_per_cta);
        const bool is_long = !(a.max_len > 0 && a.max_len <= static_cast<int64_t>(kNarrowFold) * G);
        if (is_long) rowsplit_ksplit_kernel<T, VW, LPR, G, true><<<grid, kNarrowThreads, 0, st>>>(a);
        else rowsplit_ksplit_kernel<T, VW, LPR, G, false><<<grid, kNarrowThreads, 0, st>>>(a);
        return cudaGetLastError();
    }
}

// N * sizeof(T) = 16 * LPR bytes exactly, LPR in {1, 2, 4, 8, 16}; g from ksplit_group (> 1).
template <typename T>
cudaError_t launch_rowsplit_ksplit(const SpmmArgs &a, int lpr, int g, cudaStream_t st) {
    constexpr int VWV = vec_width<T>::value;
#define SD_KS_CASE(L, GG) \
    if (lpr == L && g == GG) return launch_ksplit_g<T, VWV, L, GG>(a, st);
    SD_KS_CASE(1, 2) SD_KS_CASE(1, 4) SD_KS_CASE(1, 8) SD_KS_CASE(1, 16) SD_KS_CASE(1, 32)
    SD_KS_CASE(2, 2) SD_KS_CASE(2, 4) SD_KS_CASE(2, 8) SD_KS_CASE(2, 16)
    SD_KS_CASE(4, 2) SD_KS_CASE(4, 4) SD_KS_CASE(4, 8)
    SD_KS_CASE(8, 2) SD_KS_CASE(8, 4)
    SD_KS_CASE(16, 2)
#undef SD_KS_CASE
    return cudaErrorInvalidValue;
}

inline int narrow_group_override() { return switches().narrow_g; }

// Lanes per row from the mean row length: the largest power of two up to a quarter of it, 1..16
// (measured on uniform rows of 5 to 128 nonzeros: each lane should keep about four to eight gathers of
// its own; more lanes per row only add idle lanes and shuffle steps).  Unknown mean: 4.
inline int narrow_group(int64_t mean_len) {
    if (const int o = narrow_group_override()) return o;
    if (mean_len <= 0) return 4;
    int g = 1;
    while (g < 16 && 2 * g <= mean_len / 4) g <<= 1;
    return g;
}

template <typename T, int N, int G>
cudaError_t launch_narrow_g(const SpmmArgs &a, bool vec, cudaStream_t st) {
    const int rows_per_cta = kNarrowThreads / G;
    const unsigned grid = static_cast<unsigned>((a.S + rows_per_cta - 1) / rows_per_cta);
    const bool is_long = !(a.max_len > 0 && a.max_len <= static_cast<int64_t>(kNarrowFold) * G);
    constexpr bool CAN_VEC = sizeof(T) == 4 && N == 4;
    if constexpr (CAN_VEC) {
        if (vec) {
            if (is_long) rowsplit_narrow_kernel<T, N, G, true, true><<<grid, kNarrowThreads, 0, st>>>(a);
            else rowsplit_narrow_kernel<T, N, G, true, false><<<grid, kNarrowThreads, 0, st>>>(a);
            return cudaGetLastError();
        }
    }
    if (is_long) rowsplit_narrow_kernel<T, N, G, false, true><<<grid, kNarrowThreads, 0, st>>>(a);
    else rowsplit_narrow_kernel<T, N, G, false, false><<<grid, kNarrowThreads, 0, st>>>(a);
    return cudaGetLastError();
}

template <typename T, int N>
cudaError_t launch_narrow_n(const SpmmArgs &a, bool vec, cudaStream_t st) {
    switch (narrow_group(a.mean_len)) {
    case 1: return launch_narrow_g<T, N, 1>(a, vec, st);
    case 2: return launch_narrow_g<T, N, 2>(a, vec, st);
    case 4: return launch_narrow_g<T, N, 4>(a, vec, st);
    case 8: return launch_narrow_g<T, N, 8>(a, vec, st);
    case 16: return launch_narrow_g<T, N, 16>(a, vec, st);
    case 32: return launch_narrow_g<T, N, 32>(a, vec, st);
    }
    return cudaErrorInvalidValue;
}

template <typename T>
cudaError_t launch_rowsplit_narrow(const SpmmArgs &a, bool vec, cudaStream_t st) {
    switch (a.N) {
    case 1: return launch_narrow_n<T, 1>(a, vec, st);
    case 2: return launch_narrow_n<T, 2>(a, vec, st);
    case 3: return launch_narrow_n<T, 3>(a, vec, st);
    case 4: return launch_narrow_n<T, 4>(a, vec, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace sd
