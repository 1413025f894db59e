// Family (b): merge-path (nnz-balanced) CSR SpMM with a segmented warp-shuffle scan of
// partial rows and a deterministic carry-out fix-up.
//
// The merged list interleaves the S segment ends with the nonzeros: after i ends and j
// nonzeros the next item is the end of segment i iff ptr[i+1] <= j, else nonzero j.  Equal
// slices of that list go to CTAs ("tiles", kMergeTile items) and, inside a tile, to groups of LPR
// lanes (IPG items each), so a 200,000-nonzero row and 200,000 one-nonzero rows cost the
// same (the paper's Sec. 3.1 names merge-based decomposition as the remedy for row-length
// imbalance; its own long-row kernel uses 256-nonzero chunks and float atomics instead).
//
// A segment is a row of A, or -- when the plan uses column windows -- the part of a row that
// falls into one window; seg_row then maps it to its output row.
#pragma once

#include "sd_common.cuh"
#include "sd_launch.cuh"

namespace sd {

constexpr int kMergeThreads = 256;
constexpr int kMergeEnd = -1;  // column value that marks a segment end in the staged item list

template <typename T, int VW, int LPR, int NV>
__global__ void __launch_bounds__(kMergeThreads)
merge_tile_kernel(const MergeArgs m) {
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int G = kMergeThreads / LPR;   // groups per tile
    constexpr int TILE = kMergeTile;         // items per tile
    constexpr int IPG = TILE / G;            // items per group
    constexpr int IPT = TILE / kMergeThreads;  // items per thread in the staging scan
    constexpr int CPL = NV * VW;             // columns per lane
    constexpr int COLS = LPR * CPL;          // columns per CTA slab
    constexpr int CP = COLS + 1;             // padded row pitch of head_s / tail_s

    __shared__ int2 items[TILE];              // (column | kMergeEnd, value bits)
    __shared__ int32_t ptr_s[TILE + 2];       // ptr[seg0 .. seg0 + ends]
    __shared__ uint16_t eb_s[TILE];           // ends before item k; bit 15: item k is an end
    __shared__ float head_s[G * CP];
    __shared__ float tail_s[G * CP];
    __shared__ int32_t warp_cnt[kMergeThreads / 32];
    __shared__ uint8_t has_end_s[G], open_s[G];
    __shared__ int32_t first_end_s;

    const SpmmArgs &a = m.s;
    const T *__restrict__ vals = static_cast<const T *>(a.vals);
    const T *__restrict__ B = static_cast<const T *>(a.B);
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int t = blockIdx.x;
    const int cbase = blockIdx.y * COLS;

    // ---- tile coordinates ------------------------------------------------------------
    const int64_t sb = m.seg_begin;
    const int64_t nzb = __ldg(a.ptr + sb);
    const int64_t total = (m.seg_end - sb) + (__ldg(a.ptr + m.seg_end) - nzb);
    const int64_t seg0 = __ldg(m.tile_seg + t);
    const int64_t seg1 = __ldg(m.tile_seg + t + 1);
    const int64_t d0 = static_cast<int64_t>(t) * TILE;
    const int count = static_cast<int>(min(static_cast<int64_t>(TILE), total - d0));
    const int64_t nz0 = nzb + d0 - (seg0 - sb);
    const int ends = static_cast<int>(seg1 - seg0);

    // ---- stage the tile: segment pointers, end markers, merged item list -----------------
    for (int i = tid; i <= ends; i += kMergeThreads) ptr_s[i] = __ldg(a.ptr + seg0 + i);
    for (int k = tid; k < TILE; k += kMergeThreads) eb_s[k] = 0;
    if (tid == 0) first_end_s = G;
    __syncthreads();
    // end of segment seg0+e sits at merged position (ptr[seg0+e+1] - nzb) + (seg0+e - sb)
    for (int e = tid; e < ends; e += kMergeThreads) {
        const int k = static_cast<int>((ptr_s[e + 1] - nzb) + (seg0 + e - sb) - d0);
        eb_s[k] = 0x8000u;
    }
    __syncthreads();
    {   // exclusive scan of the end markers: thread -> IPT consecutive items
        int local = 0;
        uint16_t f[IPT];
#pragma unroll
        for (int i = 0; i < IPT; ++i) {
            f[i] = eb_s[tid * IPT + i];
            local += f[i] >> 15;
        }
        int incl = local;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int n = __shfl_up_sync(FULL, incl, off);
            if (lane >= off) incl += n;
        }
        if (lane == 31) warp_cnt[tid >> 5] = incl;
        __syncthreads();
        int before = incl - local;
        for (int w = 0; w < (tid >> 5); ++w) before += warp_cnt[w];
#pragma unroll
        for (int i = 0; i < IPT; ++i) {
            eb_s[tid * IPT + i] = static_cast<uint16_t>(before) | f[i];
            before += f[i] >> 15;
        }
    }
    __syncthreads();
    for (int k = tid; k < count; k += kMergeThreads) {   // coalesced fill of the item list
        const uint16_t e = eb_s[k];
        int2 it;
        if (e & 0x8000u) {
            it = make_int2(kMergeEnd, 0);
        } else {
            const int64_t j = nz0 + k - e;
            it = make_int2(__ldg(a.colind + j), __float_as_int(to_float(vals[j])));
        }
        items[k] = it;
    }
    __syncthreads();

    // ---- each group walks its IPG items ----------------------------------------------------
    const int g = tid / LPR;
    const int lg = tid % LPR;
    const int k0 = g * IPG;
    const int nit = max(0, min(IPG, count - k0));
    bool colok[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) colok[v] = cbase + (v * LPR + lg) * VW < a.N;

    float acc[NV][VW];
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
        for (int e = 0; e < VW; ++e) acc[v][e] = 0.f;

    int seg_off = 0;      // segment index relative to seg0
    bool open = false;    // the segment at the group's start began before the group
    bool seen_end = false;
    if (nit > 0) {
        seg_off = eb_s[k0] & 0x7FFF;
        open = (nz0 + k0 - seg_off) > ptr_s[seg_off];
    }
    for (int k = 0; k < nit; ++k) {
        const int2 it = items[k0 + k];
        if (it.x != kMergeEnd) {
            const float av = __int_as_float(it.y);
            const T *brow = B + static_cast<int64_t>(it.x) * a.ldb + cbase;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                if (colok[v]) {
                    float b[VW];
                    RowLoad<T, VW>::ld(brow + (v * LPR + lg) * VW, b);
#pragma unroll
                    for (int e = 0; e < VW; ++e) acc[v][e] = fmaf(av, b[e], acc[v][e]);
                }
            }
        } else {
            if (open && !seen_end) {
                // tail end of a segment begun earlier: completed after the scan below
#pragma unroll
                for (int v = 0; v < NV; ++v)
#pragma unroll
                    for (int e = 0; e < VW; ++e) head_s[g * CP + (v * LPR + lg) * VW + e] = acc[v][e];
            } else {
                // the group saw this segment from its first nonzero: finished here
                const int64_t s = seg0 + seg_off;
                int64_t row = s;
                int accumulate = 0;
                if (a.seg_row) {
                    const int32_t r = __ldg(a.seg_row + s);
                    row = r & 0x7FFFFFFF;
                    accumulate = (r >> 31) & 1;
                }
                float *crow = a.C + row * a.ldc + cbase;
#pragma unroll
                for (int v = 0; v < NV; ++v)
                    if (colok[v]) store_cols<VW>(crow + (v * LPR + lg) * VW, acc[v], a.alpha, a.beta, accumulate);
            }
            seen_end = true;
            ++seg_off;
#pragma unroll
            for (int v = 0; v < NV; ++v)
#pragma unroll
                for (int e = 0; e < VW; ++e) acc[v][e] = 0.f;
        }
    }
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
        for (int e = 0; e < VW; ++e) tail_s[g * CP + (v * LPR + lg) * VW + e] = acc[v][e];
    if (lg == 0) {
        has_end_s[g] = seen_end;
        open_s[g] = open;
        if (seen_end) atomicMin(&first_end_s, g);
    }
    __syncthreads();

    // ---- segmented scan of the group tails across the tile (warp shuffles) --------------------
    // I[g] = (has_end[g] ? 0 : I[g-1]) + tail[g];  carry-in of group g is I[g-1].
    for (int c = tid >> 5; c < COLS; c += kMergeThreads / 32) {
        float run = 0.f;
        for (int ch = 0; ch < G; ch += 32) {
            const int gg = ch + lane;
            const bool valid = gg < G;
            float v = valid ? tail_s[gg * CP + c] : 0.f;
            int f = valid ? has_end_s[gg] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const float v2 = __shfl_up_sync(FULL, v, off);
                const int f2 = __shfl_up_sync(FULL, f, off);
                if (lane >= off && !f) {
                    v += v2;
                    f = f2;
                }
            }
            if (!f) v += run;
            float ex = __shfl_up_sync(FULL, v, 1);
            if (lane == 0) ex = run;
            run = __shfl_sync(FULL, v, 31);
            if (valid) tail_s[gg * CP + c] = ex;   // now the carry-in of group gg
        }
        // what is still open at the end of the tile goes to the carry-out slot
        if (lane == 0 && cbase + c < a.N) m.tile_tail[static_cast<int64_t>(t) * a.N + cbase + c] = run;
    }
    __syncthreads();

    // ---- finish the segments whose tail end a group held -----------------------------------------
    if (nit > 0 && open && seen_end) {
        const int first_end = first_end_s;
        const bool tile_open = open_s[0];
        const int64_t s = seg0 + (eb_s[k0] & 0x7FFF);
        float r[NV][VW];
#pragma unroll
        for (int v = 0; v < NV; ++v)
#pragma unroll
            for (int e = 0; e < VW; ++e) {
                const int c = (v * LPR + lg) * VW + e;
                r[v][e] = tail_s[g * CP + c] + head_s[g * CP + c];
            }
        if (g == first_end && tile_open) {
            // begun in an earlier tile: leave it to the fix-up pass
#pragma unroll
            for (int v = 0; v < NV; ++v)
                if (colok[v])
#pragma unroll
                    for (int e = 0; e < VW; ++e)
                        m.tile_head[static_cast<int64_t>(t) * a.N + cbase + (v * LPR + lg) * VW + e] = r[v][e];
        } else {
            int64_t row = s;
            int accumulate = 0;
            if (a.seg_row) {
                const int32_t rr = __ldg(a.seg_row + s);
                row = rr & 0x7FFFFFFF;
                accumulate = (rr >> 31) & 1;
            }
            float *crow = a.C + row * a.ldc + cbase;
#pragma unroll
            for (int v = 0; v < NV; ++v)
                if (colok[v]) store_cols<VW>(crow + (v * LPR + lg) * VW, r[v], a.alpha, a.beta, accumulate);
        }
    }
}

// Fix-up: tile `t` closed a segment that began in an earlier tile.  Its total is the sum of
// the carry-outs of the tiles since the one holding its first nonzero, plus this tile's head,
// added in a fixed order (no atomics, so repeated runs give identical bits).
constexpr int kFixChains = 8;

static __global__ void __launch_bounds__(32 * kFixChains)
merge_fixup_kernel(const MergeArgs m, const int32_t *__restrict__ fix_tiles, int32_t nfix, int32_t tile_items) {
    __shared__ float part[kFixChains][33];
    const SpmmArgs &a = m.s;
    const int f = blockIdx.x;
    if (f >= nfix) return;
    const int t = fix_tiles[f];
    const int64_t s = m.tile_seg[t];
    const int64_t nzb = a.ptr[m.seg_begin];
    const int64_t first_item = (a.ptr[s] - nzb) + (s - m.seg_begin);
    const int ta = static_cast<int>(first_item / tile_items);
    int64_t row = s;
    int accumulate = 0;
    if (a.seg_row) {
        const int32_t rr = a.seg_row[s];
        row = rr & 0x7FFFFFFF;
        accumulate = (rr >> 31) & 1;
    }
    const int x = threadIdx.x & 31, y = threadIdx.x >> 5;
    for (int c0 = 0; c0 < a.N; c0 += 32) {
        const int c = c0 + x;
        float sum = 0.f;
        if (c < a.N)
            for (int tt = ta + y; tt < t; tt += kFixChains) sum += m.tile_tail[static_cast<int64_t>(tt) * a.N + c];
        part[y][x] = sum;
        __syncthreads();
        if (y == 0 && c < a.N) {
            float tot = part[0][x];
#pragma unroll
            for (int q = 1; q < kFixChains; ++q) tot += part[q][x];
            tot += m.tile_head[static_cast<int64_t>(t) * a.N + c];
            float *p = a.C + row * a.ldc + c;
            float r = a.alpha * tot;
            if (accumulate) r += *p;
            else if (a.beta != 0.f) r += a.beta * *p;
            *p = r;
        }
        __syncthreads();
    }
}

template <typename T, int VW, int LPR, int NV>
cudaError_t launch_merge_one(const MergeArgs &m, cudaStream_t st) {
    dim3 grid(static_cast<unsigned>(m.ntiles),
              static_cast<unsigned>((m.s.N + LPR * NV * VW - 1) / (LPR * NV * VW)));
    merge_tile_kernel<T, VW, LPR, NV><<<grid, kMergeThreads, 0, st>>>(m);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_merge(const MergeArgs &m, bool vec, int lpr, cudaStream_t st) {
    constexpr int VWV = vec_width<T>::value;
    const int64_t units = (m.s.N + (vec ? VWV : 1) - 1) / (vec ? VWV : 1);
    const bool wide = units > 32;
#define SD_MG_CASE(L)                                                                   \
    case L:                                                                             \
        if (vec) return (wide && L == 32) ? launch_merge_one<T, VWV, 32, 2>(m, st)      \
                                          : launch_merge_one<T, VWV, L, 1>(m, st);      \
        return (wide && L == 32) ? launch_merge_one<T, 1, 32, 4>(m, st)                 \
                                 : launch_merge_one<T, 1, L, 1>(m, st);
    switch (lpr) {
        SD_MG_CASE(1)
        SD_MG_CASE(2)
        SD_MG_CASE(4)
        SD_MG_CASE(8)
        SD_MG_CASE(16)
        SD_MG_CASE(32)
    }
#undef SD_MG_CASE
    return cudaErrorInvalidValue;
}

}  // namespace sd
