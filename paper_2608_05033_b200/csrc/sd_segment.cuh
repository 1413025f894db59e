// Group-per-segment kernels of the window-major schedule (family (b) with column windows):
//   seg_kernel     one lane group per segment, or per chunk of a long segment
//   single_kernel  segments of exactly one nonzero, without a pointer array
//   chunk_reduce   adds the chunk sums of every long segment in order and updates C
// Groups are independent: their shuffles name only the group's own lanes, so two groups of a
// warp may run different trip counts, and the grid-stride loops need no warp-wide agreement.
#pragma once

#include <type_traits>

#include "sd_common.cuh"
#include "sd_rowsplit.cuh"

namespace sd {

constexpr int kSegThreads = 256;

// MODE 1 (SCRATCH): the segments are chunks; chunk c writes its plain sum to row c of a.C (the scratch
// matrix).  MODE 0: a.seg_row gives the output row and whether an earlier window wrote it.
// MODE 2: the segments are whole rows of the caller's CSR arrays named by the descriptors a.desc (hybrid
// family, rows of medium length); walked like chunks, written like segments.
// Up to four lanes per row: six CTAs per SM (40 registers) measure 6 % faster; wider groups lose with that cap.
// seg_body is the kernel's body for CTA number `bx` of `nbx` (a kernel of its own, or one role of the fused kernel
// of the hybrid family).
template <typename T, int VW, int LPR, int NV, int MODE>
__device__ __forceinline__ void seg_body(const SpmmArgs &a, const unsigned bx, const unsigned nbx) {
    constexpr bool SCRATCH = MODE == 1;   // output: scratch rows
    constexpr bool STREAM = MODE != 0;    // walk: whole steps untested, next step's pairs requested ahead
    const int lane = threadIdx.x & 31;
    const int lg = threadIdx.x % LPR;
    const unsigned gmask = (LPR == 32) ? 0xffffffffu : (((1u << LPR) - 1u) << (lane & ~(LPR - 1)));
    const int cbase = blockIdx.y * (LPR * NV * VW);
    const T *__restrict__ vals = static_cast<const T *>(a.vals);
    const T *__restrict__ Bl = static_cast<const T *>(a.B) + cbase + lg * VW;
    bool colok[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) colok[v] = cbase + (v * LPR + lg) * VW < a.N;
    // gathers in flight per lane: the chunk kernel, which runs ahead of the rest on its own stream and is
    // bound by gather latency, takes all LPR of a step (measured: 12 % less time for the window-major
    // call); the short-segment kernel measures better with four and the higher occupancy
    constexpr int QW = (NV * VW >= 8) ? 2 : (STREAM ? 8 : 4);
    constexpr int QU = LPR < QW ? LPR : QW;

    const int64_t gstride = static_cast<int64_t>(nbx) * (kSegThreads / LPR);
    for (int64_t s = (static_cast<int64_t>(bx) * kSegThreads + threadIdx.x) / LPR; s < a.S; s += gstride) {
        int p0, p1;
        int64_t out_row = s;   // SCRATCH: scratch row of this chunk
        if (SCRATCH && a.ranges) {
            // hybrid family: work item s is chunk order[s], a sub-range of one long row inside one column window
            out_row = a.order ? __ldg(a.order + s) : s;
            const int2 pr = __ldg(a.ranges + out_row);
            p0 = pr.x;
            p1 = pr.y;
        } else if (MODE == 2) {
            const int4 d = __ldg(a.desc + s);   // {row, first nonzero, its column, length}
            out_row = d.x;
            p0 = d.y;
            p1 = d.y + d.w;
        } else {
            p0 = __ldg(a.ptr + s);
            p1 = __ldg(a.ptr + s + 1);
        }
        int32_t r = 0;
        if (MODE == 0) r = __ldg(a.seg_row + s);
        if (MODE == 2) r = static_cast<int32_t>(out_row);
        float acc[NV][VW];
#pragma unroll
        for (int v = 0; v < NV; ++v)
#pragma unroll
            for (int e = 0; e < VW; ++e) acc[v][e] = 0.f;
        // A step takes LPR (or 2 LPR) nonzeros.  Whole steps run without any test; only a segment's last, partly
        // filled step tests every entry: its entries beyond the end have column 0 and value 0, and neither their
        // gather nor their product may happen, or a non-finite row 0 of B would reach rows that never name
        // column 0 (0 * Inf is NaN).
        if constexpr (SCRATCH && LPR <= 2 && NV * VW < 8) {
            // chunks with one or two lanes per row: a lane fetches two (column, value) pairs per step, so that twice
            // as many gathers are in flight per lane (skewed matrix at 8 columns 0.689 -> 0.642 ms; with four lanes it loses)
            constexpr int STEP = 2 * LPR;
            auto step = [&](int p, auto whole_tag) {
                constexpr bool WHOLE = decltype(whole_tag)::value;
                int myc[2];
                float myv[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const bool ok = WHOLE || p + h * LPR + lg < p1;
                    myc[h] = ok ? __ldg(a.colind + p + h * LPR + lg) : 0;
                    myv[h] = ok ? to_float(vals[p + h * LPR + lg]) : 0.f;
                }
                int cq[STEP];
                float aq[STEP], b[STEP][VW];
#pragma unroll
                for (int i = 0; i < STEP; ++i) {
                    cq[i] = (LPR == 1) ? myc[i / LPR] : __shfl_sync(gmask, myc[i / LPR], i % LPR, LPR);
                    aq[i] = (LPR == 1) ? myv[i / LPR] : __shfl_sync(gmask, myv[i / LPR], i % LPR, LPR);
                }
#pragma unroll
                for (int i = 0; i < STEP; ++i) {
                    if (colok[0] && (WHOLE || p + i < p1)) {
                        RowLoad<T, VW>::ld(b_row(Bl, cq[i], a.ldb_bytes), b[i]);
                    } else {
#pragma unroll
                        for (int e = 0; e < VW; ++e) b[i][e] = 0.f;
                    }
                }
#pragma unroll
                for (int i = 0; i < STEP; ++i)
#pragma unroll
                    for (int e = 0; e < VW; ++e) acc[0][e] = fmaf(aq[i], b[i][e], acc[0][e]);
            };
            int p = p0;
            for (; p + STEP <= p1; p += STEP) step(p, std::true_type{});
            if (p < p1) step(p, std::false_type{});
        } else {
            int myc = 0;
            float myv = 0.f;
            auto fetch = [&](int p, auto whole_tag) {   // the group's (column, value) pairs of the step that starts at p
                constexpr bool WHOLE = decltype(whole_tag)::value;
                myc = 0;
                myv = 0.f;
                if (WHOLE || p + lg < p1) {
                    myc = __ldg(a.colind + p + lg);
                    myv = to_float(vals[p + lg]);
                }
            };
            auto step = [&](int p, auto whole_tag) {
                constexpr bool WHOLE = decltype(whole_tag)::value;
                int curc = myc;
                float curv = myv;
                if constexpr (STREAM) {
                    // chunks: the next step's pairs are requested before this step's gathers, so that a step costs one
                    // memory round trip instead of two (the chunk kernel is bound by that latency)
                    fetch(p + LPR, std::false_type{});
                } else {
                    fetch(p, whole_tag);
                    curc = myc;
                    curv = myv;
                }
                for (int q0 = 0; q0 < LPR && (WHOLE || p + q0 < p1); q0 += QU) {
                    int cq[QU];
                    float aq[QU];
#pragma unroll
                    for (int qq = 0; qq < QU; ++qq) {
                        cq[qq] = (LPR == 1) ? curc : __shfl_sync(gmask, curc, q0 + qq, LPR);
                        aq[qq] = (LPR == 1) ? curv : __shfl_sync(gmask, curv, q0 + qq, LPR);
                    }
                    float b[QU][NV][VW];
#pragma unroll
                    for (int qq = 0; qq < QU; ++qq) {
                        const bool valid = WHOLE || (p + q0 + qq < p1);
                        const T *brow = b_row(Bl, cq[qq], a.ldb_bytes);
#pragma unroll
                        for (int v = 0; v < NV; ++v) {
                            if (valid && colok[v]) {
                                RowLoad<T, VW>::ld(brow + v * LPR * VW, b[qq][v]);
                            } else {
#pragma unroll
                                for (int e = 0; e < VW; ++e) b[qq][v][e] = 0.f;
                            }
                        }
                    }
#pragma unroll
                    for (int qq = 0; qq < QU; ++qq)
#pragma unroll
                        for (int v = 0; v < NV; ++v)
#pragma unroll
                            for (int e = 0; e < VW; ++e) acc[v][e] = fmaf(aq[qq], b[qq][v][e], acc[v][e]);
                }
            };
            int p = p0;
            if constexpr (STREAM) {
                fetch(p0, std::false_type{});
                for (; p + LPR <= p1; p += LPR) step(p, std::true_type{});
                if (p < p1) step(p, std::false_type{});
            } else {
                // short segments are mostly shorter than a step: one tested form (two copies of the loop cost 14 % here)
                for (; p < p1; p += LPR) step(p, std::false_type{});
            }
        }
        if (SCRATCH) {
            float *crow = a.C + out_row * a.ldc + cbase;
#pragma unroll
            for (int v = 0; v < NV; ++v)
                if (colok[v]) store_cols<VW>(crow + (v * LPR + lg) * VW, acc[v], 1.f, 0.f, 0);
        } else {
            float *crow = a.C + static_cast<int64_t>(r & 0x7FFFFFFF) * a.ldc + cbase;
#pragma unroll
            for (int v = 0; v < NV; ++v)
                if (colok[v]) store_cols<VW>(crow + (v * LPR + lg) * VW, acc[v], a.alpha, a.beta, r < 0 ? 1 : 0);
        }
    }
}

template <typename T, int VW, int LPR, int NV, int MODE>
__global__ void __launch_bounds__(kSegThreads, (LPR <= 4 && NV * VW < 8) ? 6 : 1)
seg_kernel(const SpmmArgs a) {
    seg_body<T, VW, LPR, NV, MODE>(a, blockIdx.x, gridDim.x);
}

constexpr int kSingleBatch = 4;   // segments per lane group: their loads are all in flight together

template <typename T, int VW, int LPR, int NV>
__global__ void __launch_bounds__(kSegThreads)
single_kernel(const SpmmArgs a) {
    const int lg = threadIdx.x % LPR;
    const int64_t g = (static_cast<int64_t>(blockIdx.x) * kSegThreads + threadIdx.x) / LPR;
    const int cbase = blockIdx.y * (LPR * NV * VW);
    const int64_t s0 = g * kSingleBatch;
    if (s0 >= a.S) return;
    const T *__restrict__ vals = static_cast<const T *>(a.vals);
    int32_t r[kSingleBatch];
    int c[kSingleBatch];
    float av[kSingleBatch];
#pragma unroll
    for (int u = 0; u < kSingleBatch; ++u) {
        const bool ok = s0 + u < a.S;
        r[u] = ok ? __ldg(a.seg_row + s0 + u) : 0;
        c[u] = ok ? __ldg(a.colind + s0 + u) : 0;
        av[u] = ok ? a.alpha * to_float(vals[s0 + u]) : 0.f;
    }
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int col = (v * LPR + lg) * VW;
        if (cbase + col >= a.N) continue;
        float b[kSingleBatch][VW], o[kSingleBatch][VW];
#pragma unroll
        for (int u = 0; u < kSingleBatch; ++u) {
            RowLoad<T, VW>::ld(b_row(static_cast<const T *>(a.B), c[u], a.ldb_bytes) + cbase + col, b[u]);
            const bool need_c = (s0 + u < a.S) && (r[u] < 0 || a.beta != 0.f);
            const float *crow = a.C + static_cast<int64_t>(r[u] & 0x7FFFFFFF) * a.ldc + cbase + col;
            if constexpr (VW == 1) {
                o[u][0] = need_c ? *crow : 0.f;
            } else {
#pragma unroll
                for (int q = 0; q < VW / 4; ++q) {
                    const float4 t = need_c ? *(reinterpret_cast<const float4 *>(crow) + q) : make_float4(0.f, 0.f, 0.f, 0.f);
                    o[u][4 * q] = t.x; o[u][4 * q + 1] = t.y; o[u][4 * q + 2] = t.z; o[u][4 * q + 3] = t.w;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kSingleBatch; ++u) {
            if (s0 + u >= a.S) continue;
            const float beta = r[u] < 0 ? 1.f : a.beta;
#pragma unroll
            for (int e = 0; e < VW; ++e) b[u][e] = fmaf(beta, o[u][e], av[u] * b[u][e]);
            store_cols<VW>(a.C + static_cast<int64_t>(r[u] & 0x7FFFFFFF) * a.ldc + cbase + col, b[u], 1.f, 0.f, 0);
        }
    }
}

// One warp per long segment: chain q of the warp adds every nchain-th chunk row, the chains
// are then added in a fixed order (no atomics: repeated runs give identical bits).  CW columns
// per lane (4 when N is a multiple of 4: 16-byte loads of the scratch rows).
template <int CW>
__global__ void __launch_bounds__(256)
chunk_reduce_kernel(const float *__restrict__ chunk_out, const int32_t *__restrict__ seg_chunk,
                    const int32_t *__restrict__ seg_row, int64_t seg_begin, int64_t seg_end, float *__restrict__ C,
                    int64_t ldc, int32_t N, float alpha, float beta, int32_t skip_above) {
    const int lane = threadIdx.x & 31;
    const int64_t s = seg_begin + static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5);
    if (s >= seg_end) return;
    const int units = (N + CW - 1) / CW;
    int lpc = 1;                       // lanes per chain: a power of two covering min(units, 32)
    while (lpc < 32 && lpc < units) lpc <<= 1;
    const int nchain = 32 / lpc, chain = lane / lpc, cl = lane % lpc;
    const int32_t c0 = __ldg(seg_chunk + s), c1 = __ldg(seg_chunk + s + 1);
    if (skip_above > 0 && c1 - c0 > skip_above) return;   // left to chunk_reduce_wide_kernel
    const int32_t r = __ldg(seg_row + s);
    const bool accumulate = r < 0;
    float *crow = C + static_cast<int64_t>(r & 0x7FFFFFFF) * ldc;
    for (int ub = 0; ub < units; ub += lpc) {
        const int col = (ub + cl) * CW;
        float sum[CW];
#pragma unroll
        for (int e = 0; e < CW; ++e) sum[e] = 0.f;
        if (col < N) {
#pragma unroll 4
            for (int32_t c = c0 + chain; c < c1; c += nchain) {
                const float *p = chunk_out + static_cast<int64_t>(c) * N + col;
                if constexpr (CW == 4) {
                    const float4 t = *reinterpret_cast<const float4 *>(p);
                    sum[0] += t.x; sum[1] += t.y; sum[2] += t.z; sum[3] += t.w;
                } else {
                    sum[0] += *p;
                }
            }
        }
        for (int off = lpc; off < 32; off <<= 1)
#pragma unroll
            for (int e = 0; e < CW; ++e) sum[e] += __shfl_xor_sync(0xffffffffu, sum[e], off);
        if (chain == 0 && col < N) {
#pragma unroll
            for (int e = 0; e < CW; ++e) {
                float v = alpha * sum[e];
                if (accumulate) v += crow[col + e];
                else if (beta != 0.f) v = fmaf(beta, crow[col + e], v);
                crow[col + e] = v;
            }
        }
    }
}

// Segments of very many chunks (list[]: their positions in seg_chunk / seg_row): one CTA each.  Warp w adds the chunks
// c0 + w, c0 + w + 8, ... with the same chains as above; the eight warp sums meet in shared memory and warp 0 adds them
// in warp order: a fixed order again.
template <int CW>
__global__ void __launch_bounds__(256)
chunk_reduce_wide_kernel(const float *__restrict__ chunk_out, const int32_t *__restrict__ seg_chunk,
                         const int32_t *__restrict__ seg_row, const int32_t *__restrict__ list, float *__restrict__ C,
                         int64_t ldc, int32_t N, float alpha, float beta) {
    __shared__ float part[8][32 * CW];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t s = __ldg(list + blockIdx.x);
    const int units = (N + CW - 1) / CW;
    int lpc = 1;
    while (lpc < 32 && lpc < units) lpc <<= 1;
    const int nchain = 32 / lpc, chain = lane / lpc, cl = lane % lpc;
    const int32_t c0 = __ldg(seg_chunk + s), c1 = __ldg(seg_chunk + s + 1);
    const int32_t r = __ldg(seg_row + s);
    const bool accumulate = r < 0;
    float *crow = C + static_cast<int64_t>(r & 0x7FFFFFFF) * ldc;
    for (int ub = 0; ub < units; ub += lpc) {
        const int col = (ub + cl) * CW;
        float sum[CW];
#pragma unroll
        for (int e = 0; e < CW; ++e) sum[e] = 0.f;
        if (col < N) {
#pragma unroll 4
            for (int32_t c = c0 + warp * nchain + chain; c < c1; c += 8 * nchain) {
                const float *p = chunk_out + static_cast<int64_t>(c) * N + col;
                if constexpr (CW == 4) {
                    const float4 t = *reinterpret_cast<const float4 *>(p);
                    sum[0] += t.x; sum[1] += t.y; sum[2] += t.z; sum[3] += t.w;
                } else {
                    sum[0] += *p;
                }
            }
        }
        for (int off = lpc; off < 32; off <<= 1)
#pragma unroll
            for (int e = 0; e < CW; ++e) sum[e] += __shfl_xor_sync(0xffffffffu, sum[e], off);
        if (chain == 0)
#pragma unroll
            for (int e = 0; e < CW; ++e) part[warp][cl * CW + e] = sum[e];
        __syncthreads();
        if (warp == 0 && chain == 0 && col < N) {
#pragma unroll
            for (int e = 0; e < CW; ++e) {
                float t = part[0][cl * CW + e];
#pragma unroll
                for (int w = 1; w < 8; ++w) t += part[w][cl * CW + e];
                float v = alpha * t;
                if (accumulate) v += crow[col + e];
                else if (beta != 0.f) v = fmaf(beta, crow[col + e], v);
                crow[col + e] = v;
            }
        }
        __syncthreads();
    }
}

template <typename T, int VW, int LPR, int NV>
cudaError_t launch_seg_one(const SpmmArgs &a, int mode, cudaStream_t st) {
    if (a.load_only) {
        cudaFuncAttributes at;
        return mode == 1 ? cudaFuncGetAttributes(&at, seg_kernel<T, VW, LPR, NV, 1>)
             : mode == 2 ? cudaFuncGetAttributes(&at, seg_kernel<T, VW, LPR, NV, 2>)
                         : cudaFuncGetAttributes(&at, seg_kernel<T, VW, LPR, NV, 0>);
    }
    const int per_cta = kSegThreads / LPR;
    const int64_t need = (a.S + per_cta - 1) / per_cta;
    // persistent grid: exactly the CTAs that are resident together (the registers of an instance decide how
    // many of the eight 256-thread CTAs an SM takes); a larger grid would run a thin second wave
    static std::atomic<int> occ_scratch[kMaxDevices], occ_plain[kMaxDevices], occ_rows[kMaxDevices];
    const int occ = mode == 1 ? occupancy_cached(occ_scratch, seg_kernel<T, VW, LPR, NV, 1>, kSegThreads)
                  : mode == 2 ? occupancy_cached(occ_rows, seg_kernel<T, VW, LPR, NV, 2>, kSegThreads)
                              : occupancy_cached(occ_plain, seg_kernel<T, VW, LPR, NV, 0>, kSegThreads);
    const int64_t cap = static_cast<int64_t>(sm_count_cached()) * occ;
    dim3 grid(static_cast<unsigned>(need < cap ? need : cap),
              static_cast<unsigned>((a.N + LPR * NV * VW - 1) / (LPR * NV * VW)));
    if (mode == 1) seg_kernel<T, VW, LPR, NV, 1><<<grid, kSegThreads, 0, st>>>(a);
    else if (mode == 2) seg_kernel<T, VW, LPR, NV, 2><<<grid, kSegThreads, 0, st>>>(a);
    else seg_kernel<T, VW, LPR, NV, 0><<<grid, kSegThreads, 0, st>>>(a);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_seg(const SpmmArgs &a, bool vec, int mode, cudaStream_t st) {
    constexpr int VWV = vec_width<T>::value;
    const LaneGeom g = lane_geometry(a.N, vec, VWV, false);
    if (vec && g.nv == 2) {
        switch (g.lpr) {
        case 8: return launch_seg_one<T, VWV, 8, 2>(a, mode, st);
        case 16: return launch_seg_one<T, VWV, 16, 2>(a, mode, st);
        case 32: return launch_seg_one<T, VWV, 32, 2>(a, mode, st);
        }
        return cudaErrorInvalidValue;
    }
#define SD_SEG_CASE(L)                                                       \
    case L:                                                                  \
        if (vec) return launch_seg_one<T, VWV, L, 1>(a, mode, st);        \
        return (g.nv == 4) ? launch_seg_one<T, 1, 32, 4>(a, mode, st)     \
                           : launch_seg_one<T, 1, L, 1>(a, mode, st);
    switch (g.lpr) {
        SD_SEG_CASE(1)
        SD_SEG_CASE(2)
        SD_SEG_CASE(4)
        SD_SEG_CASE(8)
        SD_SEG_CASE(16)
        SD_SEG_CASE(32)
    }
#undef SD_SEG_CASE
    return cudaErrorInvalidValue;
}

template <typename T, int VW, int LPR, int NV>
cudaError_t launch_single_one(const SpmmArgs &a, cudaStream_t st) {
    if (a.load_only) {
        cudaFuncAttributes at;
        return cudaFuncGetAttributes(&at, single_kernel<T, VW, LPR, NV>);
    }
    const int per_cta = kSegThreads / LPR * kSingleBatch;
    dim3 grid(static_cast<unsigned>((a.S + per_cta - 1) / per_cta),
              static_cast<unsigned>((a.N + LPR * NV * VW - 1) / (LPR * NV * VW)));
    single_kernel<T, VW, LPR, NV><<<grid, kSegThreads, 0, st>>>(a);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_single(const SpmmArgs &a, bool vec, cudaStream_t st) {
    constexpr int VWV = vec_width<T>::value;
    const LaneGeom g = lane_geometry(a.N, vec, VWV, false);
    if (vec && g.nv == 2) {
        switch (g.lpr) {
        case 8: return launch_single_one<T, VWV, 8, 2>(a, st);
        case 16: return launch_single_one<T, VWV, 16, 2>(a, st);
        case 32: return launch_single_one<T, VWV, 32, 2>(a, st);
        }
        return cudaErrorInvalidValue;
    }
#define SD_SG_CASE(L)                                                \
    case L:                                                          \
        if (vec) return launch_single_one<T, VWV, L, 1>(a, st);      \
        return (g.nv == 4) ? launch_single_one<T, 1, 32, 4>(a, st)   \
                           : launch_single_one<T, 1, L, 1>(a, st);
    switch (g.lpr) {
        SD_SG_CASE(1)
        SD_SG_CASE(2)
        SD_SG_CASE(4)
        SD_SG_CASE(8)
        SD_SG_CASE(16)
        SD_SG_CASE(32)
    }
#undef SD_SG_CASE
    return cudaErrorInvalidValue;
}

}  // namespace sd
