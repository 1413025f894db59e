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

// FULL: every lane's columns are inside N (N is a multiple of the slab width), so the
// per-vector column tests disappear from the inner loop.
// One vector per lane: eight CTAs per SM (32 registers; the few spilled bytes cost less than the lost
// occupancy).  Two vectors per lane need more registers: four CTAs.
template <typename T, int VW, int LPR, int NV, bool FULL>
__global__ void __launch_bounds__(kMergeThreads, NV == 1 ? 8 : 4)
merge_tile_kernel(const MergeArgs m) {
    constexpr unsigned FULLMASK = 0xffffffffu;
    constexpr int G = kMergeThreads / LPR;   // groups per tile
    constexpr int TILE = kMergeTile;         // merged items per tile
    constexpr int IPG = TILE / G;            // merged items per group
    constexpr int CPL = NV * VW;             // columns per lane
    constexpr int COLS = LPR * CPL;          // columns per CTA slab
    constexpr int CP = COLS + 1;             // padded row pitch of head_s / tail_s

    // (column, value bits) of the tile's nonzeros.  Eight or more groups share a warp when LPR <= 4 and read
    // their own nonzeros in lock step, IPG items apart: one pad slot per IPG items moves neighbouring
    // groups to different banks.
    constexpr bool SKEW = LPR <= 4;   // measured: -7 to -9 % at 8 and 16 columns; with 8 or 16 lanes per row the extra index arithmetic costs more than the conflicts
    constexpr int IPG_SHIFT = (IPG == 4) ? 2 : (IPG == 8) ? 3 : (IPG == 16) ? 4 : (IPG == 32) ? 5 : (IPG == 64) ? 6 : 7;
    static_assert((1 << IPG_SHIFT) == IPG, "items per group must be a power of two");
    auto phys = [](int k) { return SKEW ? k + (k >> IPG_SHIFT) : k; };
    __shared__ int2 nz_s[TILE + (SKEW ? G : 0)];
    __shared__ int32_t ptr_s[TILE + 2];       // ptr[seg0 .. seg0 + ends + 1]
    __shared__ float head_s[G * CP];
    __shared__ float tail_s[G * CP];
    __shared__ int32_t gseg_s[G + 1];         // segment coordinate (relative to seg0) of each group start
    __shared__ uint8_t has_end_s[G], open_s[G];
    __shared__ int32_t first_end_s;

    // head_s / tail_s rows are stored element-major, slot(v, e) = e * (LPR * NV) + v * LPR + lg: for a
    // fixed element the lanes of a group touch consecutive words (no bank conflicts); slot k holds
    // column (k % (LPR * NV)) * VW + k / (LPR * NV) of the slab
    constexpr int LN = LPR * NV;
    const SpmmArgs &a = m.s;
    const T *__restrict__ vals = static_cast<const T *>(a.vals);
    const int tid = threadIdx.x;
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
    const int ends = static_cast<int>(seg1 - seg0);
    const int32_t nz0 = static_cast<int32_t>(nzb + d0 - (seg0 - sb));   // first nonzero of the tile
    const int nnz_t = count - ends;                                       // nonzeros in the tile

    // ---- stage segment pointers and the tile's nonzeros (coalesced) ------------------------
    for (int i = tid; i <= ends + 1; i += kMergeThreads)
        ptr_s[i] = __ldg(a.ptr + min(seg0 + i, m.seg_end));
    for (int k = tid; k < nnz_t; k += kMergeThreads)
        nz_s[phys(k)] = make_int2(__ldcs(a.colind + nz0 + k), __float_as_int(to_float(__ldcs(vals + nz0 + k))));   // A streams through
    if (tid == 0) first_end_s = G;
    __syncthreads();

    // ---- merge-path coordinate of every group start: ends e with (ptr[e+1]-nz0)+e < k -----
    for (int gi = tid; gi <= G; gi += kMergeThreads) {
        const int k = min(gi * IPG, count);
        int lo = 0, hi = ends;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if ((ptr_s[mid + 1] - nz0) + mid < k) lo = mid + 1;
            else hi = mid;
        }
        gseg_s[gi] = lo;
    }
    __syncthreads();

    // ---- each group walks its slice: whole segments in a tight loop -------------------------
    const int g = tid / LPR;
    const int lg = tid % LPR;
    const int s0 = gseg_s[g], s1 = gseg_s[g + 1];
    const int j0 = min(g * IPG, count) - s0;          // tile-relative nonzero coordinates
    const int j1 = min((g + 1) * IPG, count) - s1;
    const bool open = (nz0 + j0) > ptr_s[s0];         // segment s0 began before this group
    const bool seen_end = s1 > s0;

    bool colok[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) colok[v] = FULL || (cbase + (v * LPR + lg) * VW < a.N);
    const T *__restrict__ Bl = static_cast<const T *>(a.B) + cbase + lg * VW;   // this lane's columns

    float acc[NV][VW];
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
        for (int e = 0; e < VW; ++e) acc[v][e] = 0.f;

    const uint64_t keep = l2_keep_policy();
    int j = j0;
    for (int s = s0;; ++s) {
        const int jend = (s < s1) ? (ptr_s[s + 1] - nz0) : j1;
        // batches of WB nonzeros: their gathers are all in flight together
        constexpr int WB = 4;
        for (; j + WB <= jend; j += WB) {
            int2 it[WB];
#pragma unroll
            for (int u = 0; u < WB; ++u) it[u] = nz_s[phys(j + u)];
            float b[WB][NV][VW];
#pragma unroll
            for (int u = 0; u < WB; ++u) {
                const T *brow = b_row(Bl, it[u].x, a.ldb_bytes);
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    if (colok[v]) {
                        RowLoadKeep<T, VW>::ld(brow + v * LPR * VW, b[u][v], keep);
                    } else {
#pragma unroll
                        for (int e = 0; e < VW; ++e) b[u][v][e] = 0.f;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < WB; ++u)
#pragma unroll
                for (int v = 0; v < NV; ++v)
#pragma unroll
                    for (int e = 0; e < VW; ++e) acc[v][e] = fmaf(__int_as_float(it[u].y), b[u][v][e], acc[v][e]);
        }
        for (; j < jend; ++j) {
            const int2 it = nz_s[phys(j)];
            const float av = __int_as_float(it.y);
            const T *brow = b_row(Bl, it.x, a.ldb_bytes);
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                if (colok[v]) {
                    float b[VW];
                    RowLoadKeep<T, VW>::ld(brow + v * LPR * VW, b, keep);
#pragma unroll
                    for (int e = 0; e < VW; ++e) acc[v][e] = fmaf(av, b[e], acc[v][e]);
                }
            }
        }
        if (s == s1) break;
        if (s == s0 && open) {
            // tail end of a segment begun earlier: completed after the combine step below
#pragma unroll
            for (int v = 0; v < NV; ++v)
#pragma unroll
                for (int e = 0; e < VW; ++e) head_s[g * CP + e * LN + v * LPR + lg] = acc[v][e];
        } else {
            // the group saw this segment from its first nonzero: finished here
            const int64_t sg = seg0 + s;
            int64_t row = sg;
            int accumulate = 0;
            if (a.seg_row) {
                const int32_t r = __ldg(a.seg_row + sg);
                row = r & 0x7FFFFFFF;
                accumulate = (r >> 31) & 1;
            }
            float *crow = a.C + row * a.ldc + cbase;
#pragma unroll
            for (int v = 0; v < NV; ++v)
                if (colok[v]) store_cols<VW>(crow + (v * LPR + lg) * VW, acc[v], a.alpha, a.beta, accumulate);
        }
#pragma unroll
        for (int v = 0; v < NV; ++v)
#pragma unroll
            for (int e = 0; e < VW; ++e) acc[v][e] = 0.f;
    }
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
        for (int e = 0; e < VW; ++e) tail_s[g * CP + e * LN + v * LPR + lg] = acc[v][e];
    if (lg == 0) {
        has_end_s[g] = seen_end;
        open_s[g] = open;
        if (seen_end) atomicMin(&first_end_s, g);
    }
    __syncthreads();

    // ---- combine the group tails across the tile -------------------------------------------------
    // I[g] = (has_end[g] ? 0 : I[g-1]) + tail[g];  carry-in of group g is I[g-1].
    if constexpr (COLS >= 16) {
        // enough columns to keep the threads busy: one thread per column, groups in order
        if (tid < COLS) {
            float run = 0.f;
#pragma unroll 4
            for (int gg = 0; gg < G; ++gg) {
                const float tv = tail_s[gg * CP + tid];
                tail_s[gg * CP + tid] = run;
                run = has_end_s[gg] ? tv : run + tv;
            }
            const int col = (tid % LN) * VW + tid / LN;   // the column this slot holds
            if (cbase + col < a.N) m.tile_tail[static_cast<int64_t>(t) * a.N + cbase + col] = run;
        }
    } else {
        // few columns, many groups: segmented scan across groups with warp shuffles
        const int lane = tid & 31;
        for (int c = tid >> 5; c < COLS; c += kMergeThreads / 32) {
            float run = 0.f;
            for (int ch = 0; ch < G; ch += 32) {
                const int gg = ch + lane;
                float v = tail_s[gg * CP + c];
                // the groups that saw a segment end restart the sum: one ballot gives every lane the
                // start of its run, so only the values travel through the shuffles
                const unsigned restarts = __ballot_sync(FULLMASK, has_end_s[gg] != 0) & (FULLMASK >> (31 - lane));
                const int reach = restarts ? lane - (31 - __clz(restarts)) : lane;   // lanes below that belong to this lane's run
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const float v2 = __shfl_up_sync(FULLMASK, v, off);
                    if (off <= reach) v += v2;
                }
                if (!restarts) v += run;
                float ex = __shfl_up_sync(FULLMASK, v, 1);
                if (lane == 0) ex = run;
                run = __shfl_sync(FULLMASK, v, 31);
                tail_s[gg * CP + c] = ex;   // now the carry-in of group gg
            }
            const int col = (c % LN) * VW + c / LN;   // the column this slot holds
            if (lane == 0 && cbase + col < a.N) m.tile_tail[static_cast<int64_t>(t) * a.N + cbase + col] = run;
        }
    }
    __syncthreads();

    // ---- finish the segments whose tail end a group held -----------------------------------------
    if (open && seen_end) {
        const int first_end = first_end_s;
        const bool tile_open = open_s[0];
        const int64_t sg = seg0 + s0;
        float r[NV][VW];
#pragma unroll
        for (int v = 0; v < NV; ++v)
#pragma unroll
            for (int e = 0; e < VW; ++e) {
                const int c = e * LN + v * LPR + lg;
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
            int64_t row = sg;
            int accumulate = 0;
            if (a.seg_row) {
                const int32_t rr = __ldg(a.seg_row + sg);
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
// added in a fixed order (no atomics, so repeated runs give identical bits).  Chains shorter
// than kFixLongChain tiles are handled one per warp, longer ones one per CTA.
constexpr int kFixChains = 8;
constexpr int kFixLongChain = 8;

struct FixTarget {
    int64_t row;
    int accumulate;
    int ta;   // first tile of the chain
};

__device__ __forceinline__ FixTarget fix_target(const MergeArgs &m, int t, int32_t tile_items) {
    const SpmmArgs &a = m.s;
    const int64_t s = m.tile_seg[t];
    const int64_t nzb = a.ptr[m.seg_begin];
    const int64_t first_item = (a.ptr[s] - nzb) + (s - m.seg_begin);
    FixTarget f;
    f.ta = static_cast<int>(first_item / tile_items);
    f.row = s;
    f.accumulate = 0;
    if (a.seg_row) {
        const int32_t rr = a.seg_row[s];
        f.row = rr & 0x7FFFFFFF;
        f.accumulate = (rr >> 31) & 1;
    }
    return f;
}

__device__ __forceinline__ void fix_store(const SpmmArgs &a, const FixTarget &f, int c, float tot) {
    float *p = a.C + f.row * a.ldc + c;
    float r = a.alpha * tot;
    if (f.accumulate) r += *p;
    else if (a.beta != 0.f) r += a.beta * *p;
    *p = r;
}

static __global__ void __launch_bounds__(256)
merge_fixup_short_kernel(const MergeArgs m, const int32_t *__restrict__ fix_tiles, int32_t nfix, int32_t tile_items) {
    const int f = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (f >= nfix) return;
    const int lane = threadIdx.x & 31;
    const int t = fix_tiles[f];
    const FixTarget ft = fix_target(m, t, tile_items);
    for (int c = lane; c < m.s.N; c += 32) {
        float sum = 0.f;
        for (int tt = ft.ta; tt < t; ++tt) sum += m.tile_tail[static_cast<int64_t>(tt) * m.s.N + c];
        sum += m.tile_head[static_cast<int64_t>(t) * m.s.N + c];
        fix_store(m.s, ft, c, sum);
    }
}

static __global__ void __launch_bounds__(32 * kFixChains)
merge_fixup_long_kernel(const MergeArgs m, const int32_t *__restrict__ fix_tiles, int32_t nfix, int32_t tile_items) {
    __shared__ float part[kFixChains][33];
    const SpmmArgs &a = m.s;
    const int f = blockIdx.x;
    if (f >= nfix) return;
    const int t = fix_tiles[f];
    const FixTarget ft = fix_target(m, t, tile_items);
    const int x = threadIdx.x & 31, y = threadIdx.x >> 5;
    for (int c0 = 0; c0 < a.N; c0 += 32) {
        const int c = c0 + x;
        float sum = 0.f;
        if (c < a.N) {
#pragma unroll 4
            for (int tt = ft.ta + y; tt < t; tt += kFixChains) sum += m.tile_tail[static_cast<int64_t>(tt) * a.N + c];
        }
        part[y][x] = sum;
        __syncthreads();
        if (y == 0 && c < a.N) {
            float tot = part[0][x];
#pragma unroll
            for (int q = 1; q < kFixChains; ++q) tot += part[q][x];
            tot += m.tile_head[static_cast<int64_t>(t) * a.N + c];
            fix_store(a, ft, c, tot);
        }
        __syncthreads();
    }
}

template <typename T, int VW, int LPR, int NV>
cudaError_t launch_merge_one(const MergeArgs &m, cudaStream_t st) {
    constexpr int COLS = LPR * NV * VW;
    dim3 grid(static_cast<unsigned>(m.ntiles), static_cast<unsigned>((m.s.N + COLS - 1) / COLS));
    if (m.s.N % COLS == 0) merge_tile_kernel<T, VW, LPR, NV, true><<<grid, kMergeThreads, 0, st>>>(m);
    else merge_tile_kernel<T, VW, LPR, NV, false><<<grid, kMergeThreads, 0, st>>>(m);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_merge(const MergeArgs &m, bool vec, int lpr, int nv, cudaStream_t st) {
    constexpr int VWV = vec_width<T>::value;
    if (vec && nv == 2) {
        switch (lpr) {
        case 8: return launch_merge_one<T, VWV, 8, 2>(m, st);
        case 16: return launch_merge_one<T, VWV, 16, 2>(m, st);
        case 32: return launch_merge_one<T, VWV, 32, 2>(m, st);
        }
        return cudaErrorInvalidValue;
    }
#define SD_MG_CASE(L)                                                \
    case L:                                                          \
        if (vec) return launch_merge_one<T, VWV, L, 1>(m, st);       \
        return (nv == 4) ? launch_merge_one<T, 1, 32, 4>(m, st)      \
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
