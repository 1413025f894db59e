// Narrow dense operands (N <= 4, SpMV included) of family (b): a segmented reduction over the
// nonzeros in storage order with an explicit row index per nonzero (the COO form that the paper's
// Sec. 3.1 lists for SpMV-like widths).
//
// With one to eight columns a lane group per row has nothing to share: the generic merge kernel
// spends its time on per-lane searches and block-wide phases.  Here a warp owns 128 consecutive
// nonzeros (256 at one or two columns: four or eight coalesced loads of row, column and value per lane, as many
// gathers of B in flight),
// multiplies, and reduces equal-row runs with warp shuffles; no shared memory, no block barrier.
//
// Rows are ascending in storage order, so a row is one run.  A run that lies strictly inside a
// warp's 128 nonzeros is complete: its lane writes alpha * sum + beta * C.
// The first and the last run of a chunk may continue in the neighbours: their sums go to a carry
// list, two entries per chunk in chunk order, (first row, sum) and (last row, sum) -- a chunk
// that is one single run writes (row, sum) and (row, 0), so that entries of one row stay
// adjacent.  The carry list is itself a row-sorted list of values: the same kernel reduces it
// (level 2), and the few entries that level leaves over are added one run per thread (level 3).
// Rows without nonzeros are found from the row pointers by the first level and get beta * C.
// Every row is written by exactly one thread and every sum has a fixed order: results are
// reproducible bit for bit, no float atomics.
#pragma once

#include "sd_common.cuh"
#include "sd_launch.cuh"

namespace sd {

struct CooArgs {
    const int32_t *row;      // [count] row of every item (ascending)
    const int32_t *colind;   // level 1: [count] column of every nonzero
    const void *vals;        // level 1: [count] values of A; level 2: [count][N] float partial sums
    const void *B;           // level 1
    uint32_t ldb_bytes;
    int64_t count;           // items
    float *C;
    int64_t ldc;
    float alpha, beta;
    const int32_t *rowptr;   // level 1: [M + 1], to find the rows without nonzeros (they get beta * C)
    int64_t M;
    int32_t *carry_row;      // [2 * chunks] out
    float *carry_val;        // [2 * chunks][N] out
};

// N floats of row `col` of B, widened.  VEC: 16-byte loads are allowed (fp32, N = 4).
template <typename T, int N, bool VEC>
__device__ __forceinline__ void coo_gather(const void *B, int col, uint32_t ldb_bytes, float (&b)[N]) {
    const T *p = b_row(static_cast<const T *>(B), col, ldb_bytes);
    if constexpr (VEC && sizeof(T) == 4 && N % 4 == 0) {
#pragma unroll
        for (int q = 0; q < N / 4; ++q) {
            float t[4];
            RowLoad<T, 4>::ld(p + 4 * q, t);
#pragma unroll
            for (int e = 0; e < 4; ++e) b[4 * q + e] = t[e];
        }
    } else if constexpr (VEC && sizeof(T) == 2 && N == 8) {
        RowLoad<T, 8>::ld(p, b);
    } else {
#pragma unroll
        for (int e = 0; e < N; ++e) {
            float t[1];
            RowLoad<T, 1>::ld(p + e, t);
            b[e] = t[0];
        }
    }
}

// LEVEL2: the items are carry entries (row, N partial sums); otherwise nonzeros of A.
template <typename T, int N, bool VEC, bool LEVEL2>
__global__ void __launch_bounds__(256)
coo_reduce_kernel(const CooArgs a) {
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    constexpr int kCooChunk = LEVEL2 ? kCooCarryChunk : coo_chunk(N);
    constexpr int kCooU = kCooChunk / 32;   // items per lane and warp step
    const int64_t chunks = (a.count + kCooChunk - 1) / kCooChunk;
    const T *__restrict__ vals = static_cast<const T *>(a.vals);
    const float *__restrict__ pvals = static_cast<const float *>(a.vals);

    for (int64_t c = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; c < chunks; c += warps) {
        if constexpr (!LEVEL2) {
            // rows without nonzeros have no writer among the runs: this chunk looks after its share of them
            const int64_t rpc = (a.M + chunks - 1) / chunks;
            for (int64_t rr = c * rpc + lane; rr < min(a.M, (c + 1) * rpc); rr += 32) {
                if (__ldg(a.rowptr + rr) == __ldg(a.rowptr + rr + 1)) {
#pragma unroll
                    for (int e = 0; e < N; ++e) {
                        float *pc = a.C + rr * a.ldc + e;
                        *pc = (a.beta != 0.f) ? a.beta * *pc : 0.f;
                    }
                }
            }
        }
        const int64_t k0 = c * kCooChunk + lane;
        const bool whole = (c + 1) * kCooChunk <= a.count;   // warp-uniform: no item of the chunk is past the end
        // ---- four items per lane: loads first, all gathers in flight together ------------------
        int r[kCooU];
        float p[kCooU][N];
        if constexpr (LEVEL2) {
#pragma unroll
            for (int u = 0; u < kCooU; ++u) {
                const int64_t k = k0 + u * 32;
                const bool ok = whole || k < a.count;
                r[u] = ok ? __ldg(a.row + k) : -1;
#pragma unroll
                for (int e = 0; e < N; ++e) p[u][e] = ok ? __ldg(pvals + k * N + e) : 0.f;
            }
        } else {
            int col[kCooU];
            float av[kCooU];
#pragma unroll
            for (int u = 0; u < kCooU; ++u) {
                const int64_t k = k0 + u * 32;
                const bool ok = whole || k < a.count;
                r[u] = ok ? __ldg(a.row + k) : -1;
                col[u] = ok ? __ldg(a.colind + k) : 0;
                av[u] = ok ? to_float(vals[k]) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < kCooU; ++u) coo_gather<T, N, VEC>(a.B, col[u], a.ldb_bytes, p[u]);
#pragma unroll
            for (int u = 0; u < kCooU; ++u)
#pragma unroll
                for (int e = 0; e < N; ++e) p[u][e] = (r[u] >= 0) ? p[u][e] * av[u] : 0.f;   // items past the end gathered row 0: never let its contents (Inf, NaN) in
        }
        if (!whole) {   // items past the end of the list continue the last row with zeros
            const int64_t last = a.count - 1;
            const int last_u = static_cast<int>((last - c * kCooChunk) >> 5), last_l = static_cast<int>(last & 31);
            int pad_row = 0;
#pragma unroll
            for (int u = 0; u < kCooU; ++u) {
                const int t = __shfl_sync(FULL, r[u], last_l);
                if (u == last_u) pad_row = t;
            }
#pragma unroll
            for (int u = 0; u < kCooU; ++u)
                if (r[u] < 0) r[u] = pad_row;
        }

        // A run is written when it closes: the run of the chunk's first row goes to the carry
        // list (it may have begun in an earlier chunk), every other one is a complete row.
        const int first_row = __shfl_sync(FULL, r[0], 0);
        auto emit = [&](int row, const float (&v)[N]) {
            if (row == first_row) {
                a.carry_row[2 * c] = row;
#pragma unroll
                for (int e = 0; e < N; ++e) a.carry_val[(2 * c) * N + e] = v[e];
            } else {
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    float *pc = a.C + static_cast<int64_t>(row) * a.ldc + e;
                    *pc = (a.beta != 0.f) ? fmaf(a.beta, *pc, a.alpha * v[e]) : a.alpha * v[e];
                }
            }
        };
        int crow = first_row;   // the run that reached the end of the previous 32 items ...
        float cval[N];          // ... and its sum so far (both warp-uniform)
#pragma unroll
        for (int e = 0; e < N; ++e) cval[e] = 0.f;

#pragma unroll
        for (int u = 0; u < kCooU; ++u) {
            // where runs start among these 32 items: one ballot replaces a row exchange per scan step
            const int rp = __shfl_up_sync(FULL, r[u], 1);
            const unsigned starts = __ballot_sync(FULL, lane == 0 || rp != r[u]);
            const int my_start = 31 - __clz(starts & (FULL >> (31 - lane)));   // first lane of this lane's run
            const int dist = lane - my_start;
            // inclusive segmented scan over equal rows
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    const float vu = __shfl_up_sync(FULL, p[u][e], d);
                    if (dist >= d) p[u][e] += vu;
                }
            }
            const bool cont = __shfl_sync(FULL, r[u], 0) == crow;
            if (cont) {                 // the open run continues in the lanes of lane 0's run
                if (my_start == 0) {
#pragma unroll
                    for (int e = 0; e < N; ++e) p[u][e] += cval[e];
                }
            } else if (lane == 0) {     // it ended exactly at the 32-item boundary
                emit(crow, cval);
            }
            if (lane < 31 && ((starts >> (lane + 1)) & 1u)) emit(r[u], p[u]);   // runs that end inside these 32 items
            crow = __shfl_sync(FULL, r[u], 31);                                  // the run reaching lane 31 stays open
#pragma unroll
            for (int e = 0; e < N; ++e) cval[e] = __shfl_sync(FULL, p[u][e], 31);
        }
        // ---- what is still open at the end of the chunk --------------------------------------
        if (lane == 0) {
            a.carry_row[2 * c + 1] = crow;
            if (crow == first_row) {   // the whole chunk is one run: (row, sum), (row, 0)
                a.carry_row[2 * c] = crow;
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    a.carry_val[(2 * c) * N + e] = cval[e];
                    a.carry_val[(2 * c + 1) * N + e] = 0.f;
                }
            } else {
#pragma unroll
                for (int e = 0; e < N; ++e) a.carry_val[(2 * c + 1) * N + e] = cval[e];
            }
        }
    }
}

// Level 3: one thread per run of equal rows in a short carry list.
template <int N>
__global__ void coo_final_kernel(const int32_t *__restrict__ row, const float *__restrict__ val, int64_t count, float *C,
                                 int64_t ldc, float alpha, float beta) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= count) return;
    const int r = row[i];
    if (i > 0 && row[i - 1] == r) return;
    float s[N];
#pragma unroll
    for (int e = 0; e < N; ++e) s[e] = 0.f;
    for (int64_t j = i; j < count && row[j] == r; ++j)
#pragma unroll
        for (int e = 0; e < N; ++e) s[e] += val[j * N + e];
#pragma unroll
    for (int e = 0; e < N; ++e) {
        float *pc = C + static_cast<int64_t>(r) * ldc + e;
        *pc = (beta != 0.f) ? fmaf(beta, *pc, alpha * s[e]) : alpha * s[e];
    }
}

// Row index of every nonzero (plan time).
static __global__ void coo_rows_kernel(const int32_t *__restrict__ rowptr, int64_t M, int64_t nnz, int32_t *__restrict__ row) {
    const int64_t k = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (k >= nnz) return;
    int64_t lo = 0, hi = M;   // last row with rowptr[row] <= k
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (rowptr[mid] <= k) lo = mid;
        else hi = mid;
    }
    row[k] = static_cast<int32_t>(lo);
}

}  // namespace sd
