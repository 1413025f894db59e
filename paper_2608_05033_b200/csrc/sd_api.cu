// C ABI of the SpMM library: plan creation (structure scan, decision, representation
// build), execution dispatch, teardown.  See include/sd.h for the contract.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include <cub/cub.cuh>

#include "sd_common.cuh"
#include "sd_launch.cuh"

// =====================================================================================
// error state
// =====================================================================================
namespace sd {

static thread_local char g_err_text[512] = "";
static thread_local int g_err_code = SD_OK;

void set_error(sd_status_t code, const char *fmt, ...) {
    g_err_code = code;
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err_text, sizeof g_err_text, fmt, ap);
    va_end(ap);
}

sd_status_t cuda_fail(cudaError_t e, const char *what) {
    set_error(SD_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
    return SD_ERR_CUDA;
}

static int env_int(const char *name, int dflt) {
    const char *e = getenv(name);
    return e ? atoi(e) : dflt;
}

const Switches &switches() {
    static const Switches sw = [] {
        Switches s;
        s.no_coo = getenv("SD_NO_COO") != nullptr;
        s.no_side_streams = getenv("SD_NO_SIDE_STREAMS") != nullptr;
        s.no_chunk_ahead = getenv("SD_NO_CHUNK_AHEAD") != nullptr;
        s.bsr_simt = getenv("SD_BSR_SIMT") != nullptr;
        s.no_narrow = getenv("SD_NO_NARROW") != nullptr;
        s.geom_nv = env_int("SD_GEOM_NV", 0);
        s.ksplit_g = env_int("SD_KSPLIT_G", 0);
        s.narrow_g = env_int("SD_NARROW_G", 0);
        s.tc_sb = env_int("SD_TC_SB", 0);
        s.tc_stages = env_int("SD_TC_STAGES", 0);
        s.tc32_sb = env_int("SD_TC32_SB", 0);
        s.tc32_stages = env_int("SD_TC32_STAGES", 0);
        return s;
    }();
    return sw;
}

// =====================================================================================
// structure scan kernels (Sec. 3.1, intrinsic pattern features; integers only)
// =====================================================================================
struct ScanAccum {
    unsigned long long row_hist[32];
    unsigned long long sum_r2, empty_rows, sum_span, sum_gap, diag, unsorted_rows, long_rows, nnz_long_rows;
    unsigned long long max_r, max_span;
    unsigned long long blk_hist[9];
    unsigned long long nnz_dense_blocks;
    unsigned long long bad_csr;   // validation: number of offending rows / entries
};

__device__ __forceinline__ int hist_bin(long long v) { return v <= 0 ? 0 : 64 - __clzll(v); }

// One warp per row.  Optionally writes the 16x16 block key of every nonzero.
__global__ void __launch_bounds__(256)
scan_rows_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colind, int64_t M,
                 int64_t Kb, unsigned long long *__restrict__ keys, ScanAccum *__restrict__ out) {
    constexpr unsigned FULL = 0xffffffffu;
    __shared__ unsigned long long s_hist[32];
    __shared__ unsigned long long s_sum[8];
    __shared__ unsigned long long s_max[2];
    if (threadIdx.x < 32) s_hist[threadIdx.x] = 0;
    if (threadIdx.x < 8) s_sum[threadIdx.x] = 0;
    if (threadIdx.x < 2) s_max[threadIdx.x] = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    unsigned long long l_r2 = 0, l_empty = 0, l_span = 0, l_gap = 0, l_diag = 0, l_uns = 0, l_long = 0,
                       l_nnzlong = 0, l_maxr = 0, l_maxspan = 0;
    for (int64_t row = warp0; row < M; row += nwarps) {
        const int p0 = rowptr[row], p1 = rowptr[row + 1];
        const long long r = static_cast<long long>(p1) - p0;
        int mn = INT_MAX, mx = INT_MIN, dg = 0, uns = 0;
        for (int p = p0 + lane; p < p1; p += 32) {
            const int c = colind[p];
            mn = min(mn, c);
            mx = max(mx, c);
            dg += (c == row);
            if (p + 1 < p1) uns |= (colind[p + 1] <= c);
            if (keys) keys[p] = static_cast<unsigned long long>(row >> 4) * Kb + static_cast<unsigned>(c >> 4);
        }
        mn = __reduce_min_sync(FULL, mn);
        mx = __reduce_max_sync(FULL, mx);
        dg = __reduce_add_sync(FULL, dg);
        uns = __reduce_or_sync(FULL, uns);
        if (lane == 0) {
            atomicAdd(&s_hist[hist_bin(r)], 1ULL);
            l_r2 += static_cast<unsigned long long>(r) * static_cast<unsigned long long>(r);
            l_maxr = max(l_maxr, static_cast<unsigned long long>(r));
            if (r == 0) {
                l_empty += 1;
            } else {
                const unsigned long long span = static_cast<unsigned long long>(static_cast<long long>(mx) - mn + 1);
                l_span += span;
                l_gap += span - 1;
                l_maxspan = max(l_maxspan, span);
                l_diag += dg;
                l_uns += uns ? 1 : 0;
                if (r >= 256) {
                    l_long += 1;
                    l_nnzlong += r;
                }
            }
        }
    }
    if (lane == 0) {
        atomicAdd(&s_sum[0], l_r2);
        atomicAdd(&s_sum[1], l_empty);
        atomicAdd(&s_sum[2], l_span);
        atomicAdd(&s_sum[3], l_gap);
        atomicAdd(&s_sum[4], l_diag);
        atomicAdd(&s_sum[5], l_uns);
        atomicAdd(&s_sum[6], l_long);
        atomicAdd(&s_sum[7], l_nnzlong);
        atomicMax(&s_max[0], l_maxr);
        atomicMax(&s_max[1], l_maxspan);
    }
    __syncthreads();
    if (threadIdx.x < 32 && s_hist[threadIdx.x]) atomicAdd(&out->row_hist[threadIdx.x], s_hist[threadIdx.x]);
    if (threadIdx.x == 0) {
        atomicAdd(&out->sum_r2, s_sum[0]);
        atomicAdd(&out->empty_rows, s_sum[1]);
        atomicAdd(&out->sum_span, s_sum[2]);
        atomicAdd(&out->sum_gap, s_sum[3]);
        atomicAdd(&out->diag, s_sum[4]);
        atomicAdd(&out->unsorted_rows, s_sum[5]);
        atomicAdd(&out->long_rows, s_sum[6]);
        atomicAdd(&out->nnz_long_rows, s_sum[7]);
        atomicMax(&out->max_r, s_max[0]);
        atomicMax(&out->max_span, s_max[1]);
    }
}

// Histogram of the entry count of each occupied block.
__global__ void block_fill_kernel(const int32_t *__restrict__ counts, int64_t nnzb, ScanAccum *__restrict__ out) {
    __shared__ unsigned long long s_h[9];
    __shared__ unsigned long long s_dense;
    if (threadIdx.x < 9) s_h[threadIdx.x] = 0;
    if (threadIdx.x == 0) s_dense = 0;
    __syncthreads();
    for (int64_t b = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; b < nnzb;
         b += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int c = counts[b];
        atomicAdd(&s_h[min(hist_bin(c) - 1, 8)], 1ULL);
        if (c >= 128) atomicAdd(&s_dense, static_cast<unsigned long long>(c));
    }
    __syncthreads();
    if (threadIdx.x < 9 && s_h[threadIdx.x]) atomicAdd(&out->blk_hist[threadIdx.x], s_h[threadIdx.x]);
    if (threadIdx.x == 0 && s_dense) atomicAdd(&out->nnz_dense_blocks, s_dense);
}

// CSR validation: rowptr[0] == 0, rowptr non-decreasing, 0 <= col < K.
__global__ void validate_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colind, int64_t M,
                                int64_t K, int64_t nnz, ScanAccum *__restrict__ out) {
    unsigned long long bad = 0;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    const int64_t i0 = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    for (int64_t i = i0; i < M; i += stride) bad += (rowptr[i + 1] < rowptr[i]);
    for (int64_t p = i0; p < nnz; p += stride) bad += (colind[p] < 0 || colind[p] >= K);
    if (i0 == 0) bad += (rowptr[0] != 0);
    if (bad) atomicAdd(&out->bad_csr, bad);
}

// =====================================================================================
// representation builders
// =====================================================================================
// BSR-16 block-row pointers from the sorted distinct block keys.
__global__ void bsr_browptr_kernel(const unsigned long long *__restrict__ ukeys, int64_t nnzb, int64_t Kb,
                                   int32_t Mb, int32_t *__restrict__ browptr) {
    const int64_t I = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (I > Mb) return;
    const unsigned long long want = static_cast<unsigned long long>(I) * Kb;
    int64_t lo = 0, hi = nnzb;
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (ukeys[mid] < want) lo = mid + 1;
        else hi = mid;
    }
    browptr[I] = static_cast<int32_t>(lo);
}

__global__ void bsr_bcol_kernel(const unsigned long long *__restrict__ ukeys, int64_t nnzb, int64_t Kb,
                                int32_t *__restrict__ bcol) {
    const int64_t b = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (b < nnzb) bcol[b] = static_cast<int32_t>(ukeys[b] % Kb);
}

// Scatter the values into row-major 16x16 blocks (copies only: bit-exact).  Warp per row.
template <typename T>
__global__ void __launch_bounds__(256)
bsr_fill_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colind, const T *__restrict__ vals,
                int64_t M, const int32_t *__restrict__ browptr, const int32_t *__restrict__ bcol, T *__restrict__ bval) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    for (int64_t row = warp0; row < M; row += nwarps) {
        const int b0 = browptr[row >> 4], b1 = browptr[(row >> 4) + 1];
        for (int p = rowptr[row] + lane; p < rowptr[row + 1]; p += 32) {
            const int c = colind[p];
            const int J = c >> 4;
            int lo = b0, hi = b1;
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (bcol[mid] < J) lo = mid + 1;
                else hi = mid;
            }
            bval[static_cast<int64_t>(lo) * 256 + (row & 15) * 16 + (c & 15)] = vals[p];
        }
    }
}

// Merge-path tile table: tile_seg[t] = seg_begin + #{ r : (ptr[r+1]-nzb) + (r-seg_begin) < t*tile }.
__global__ void merge_table_kernel(const int32_t *__restrict__ ptr, int64_t seg_begin, int64_t seg_end, int32_t tile,
                                   int32_t ntiles, int32_t *__restrict__ tile_seg) {
    const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t > ntiles) return;
    const int64_t S = seg_end - seg_begin;
    const int64_t nzb = ptr[seg_begin];
    const int64_t total = S + (ptr[seg_end] - nzb);
    const int64_t d = min(t * tile, total);
    int64_t lo = 0, hi = S;   // number of segment ends placed before position d
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if ((ptr[seg_begin + mid + 1] - nzb) + mid < d) lo = mid + 1;
        else hi = mid;
    }
    tile_seg[t] = static_cast<int32_t>(seg_begin + lo);
}

// A tile needs the fix-up pass iff a segment was open at its start and ends inside it.  The
// chain of carry-outs to add starts at the tile holding the segment's first nonzero.
__global__ void merge_fixflag_kernel(const int32_t *__restrict__ ptr, const int32_t *__restrict__ tile_seg,
                                     int64_t seg_begin, int32_t tile, int32_t ntiles, uint8_t *__restrict__ flag_short,
                                     uint8_t *__restrict__ flag_long) {
    const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t >= ntiles) return;
    const int64_t s0 = tile_seg[t], s1 = tile_seg[t + 1];
    const int64_t nzb = ptr[seg_begin];
    const int64_t nz0 = nzb + t * tile - (s0 - seg_begin);
    const bool fix = (s1 > s0) && (nz0 > ptr[s0]);
    const int64_t ta = ((ptr[s0] - nzb) + (s0 - seg_begin)) / tile;
    const bool is_long = fix && (t - ta >= kMergeLongChain);
    flag_short[t] = fix && !is_long;
    flag_long[t] = is_long;
}

// ---- column windows (the paper's "packed column windows" for SpMM, Sec. 3.4) ------------------
// The column range is cut into W windows of wcols columns.  Nonzeros are re-bucketed by window
// (stable, so rows stay ascending inside a window); a segment is the run of one row inside one
// window.  Windows are executed one after the other, so the slab of B a window touches can stay
// in L2 while every nonzero of that window is processed.
__global__ void __launch_bounds__(256)
window_keys_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colind, int64_t M, int32_t wcols,
                   uint32_t *__restrict__ wkey, int32_t *__restrict__ rowid) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    for (int64_t row = warp0; row < M; row += nwarps)
        for (int p = rowptr[row] + lane; p < rowptr[row + 1]; p += 32) {
            wkey[p] = static_cast<uint32_t>(colind[p] / wcols);
            rowid[p] = static_cast<int32_t>(row);
        }
}

__global__ void window_rows_kernel(const int32_t *__restrict__ perm, const int32_t *__restrict__ rowid, int64_t nnz,
                                   int32_t *__restrict__ w_row) {
    const int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (q < nnz) w_row[q] = rowid[perm[q]];
}

__global__ void window_headflag_kernel(const uint32_t *__restrict__ wkey_sorted, const int32_t *__restrict__ w_row,
                                       int64_t nnz, uint8_t *__restrict__ flag) {
    const int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (q >= nnz) return;
    flag[q] = (q == 0) || (w_row[q] != w_row[q - 1]) || (wkey_sorted[q] != wkey_sorted[q - 1]);
}

__global__ void window_emptyflag_kernel(const int32_t *__restrict__ rowptr, int64_t M, uint8_t *__restrict__ flag) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < M) flag[i] = rowptr[i + 1] == rowptr[i];
}

// First ordering of the segments: the E empty rows (their ids are already in seg_row[0..E)),
// then the runs of (window, row) in window-major order.  Each gets its start and length in
// the window-sorted nonzero order, its output row with the "already written" bit, and the
// sort key 3 * window + class (class 0: more than `short_len` nonzeros, class 1: 0 or
// 2..short_len nonzeros, class 2: exactly one).
__global__ void window_segments_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colind,
                                       const uint32_t *__restrict__ wkey_sorted, const int32_t *__restrict__ w_row,
                                       const int32_t *__restrict__ heads, int32_t wcols, int32_t short_len, int64_t E,
                                       int64_t S, int64_t nnz, int32_t *__restrict__ seg_start,
                                       int32_t *__restrict__ seg_len, int32_t *__restrict__ seg_row,
                                       uint32_t *__restrict__ seg_key) {
    const int64_t s = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (s >= S) return;
    if (s < E) {
        seg_start[s] = 0;
        seg_len[s] = 0;
        seg_key[s] = 1;   // window 0, short class
        return;
    }
    const int64_t h = s - E;
    const int32_t q = heads[h];
    const int32_t len = static_cast<int32_t>((h + 1 < S - E ? heads[h + 1] : nnz) - q);
    const int32_t row = w_row[q];
    const uint32_t win = wkey_sorted[q];
    const uint32_t first_win = static_cast<uint32_t>(colind[rowptr[row]] / wcols);
    seg_start[s] = q;
    seg_len[s] = len;
    seg_row[s] = row | (win != first_win ? static_cast<int32_t>(0x80000000u) : 0);
    seg_key[s] = 3 * win + (len > short_len ? 0u : (len == 1 ? 2u : 1u));
}

__global__ void window_reorder_kernel(const int32_t *__restrict__ order, const int32_t *__restrict__ seg_len,
                                      const int32_t *__restrict__ seg_row, int64_t S, int32_t *__restrict__ len2,
                                      int32_t *__restrict__ row2) {
    const int64_t s = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (s >= S) return;
    len2[s] = seg_len[order[s]];
    row2[s] = seg_row[order[s]];
}

// Final gather of the nonzeros: output position q belongs to the segment found by binary
// search in the new segment pointers; its source is that segment's run in window-sorted order.
template <typename T>
__global__ void window_gather_kernel(const int32_t *__restrict__ seg_ptr2, const int32_t *__restrict__ order,
                                     const int32_t *__restrict__ seg_start, const int32_t *__restrict__ perm,
                                     const int32_t *__restrict__ colind, const T *__restrict__ vals, int64_t S, int64_t nnz,
                                     int32_t *__restrict__ w_col, T *__restrict__ w_val, int32_t *__restrict__ w_src) {
    const int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (q >= nnz) return;
    int64_t lo = 0, hi = S;   // last segment with seg_ptr2[s] <= q and a non-zero length covers q
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (seg_ptr2[mid + 1] <= q) lo = mid + 1;
        else hi = mid;
    }
    const int32_t p = perm[seg_start[order[lo]] + (q - seg_ptr2[lo])];
    w_col[q] = colind[p];
    w_val[q] = vals[p];
    w_src[q] = p;
}

// New values for an unchanged pattern: the re-bucketed copy is refreshed from the caller's array.
template <typename T>
__global__ void window_revalue_kernel(const int32_t *__restrict__ w_src, const T *__restrict__ vals, int64_t nnz,
                                      T *__restrict__ w_val) {
    const int64_t q = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (q < nnz) w_val[q] = vals[w_src[q]];
}

// Chunks of the long segments: segment s (class 0) is cut into ceil(len / chunk) pieces.
__global__ void chunk_count_kernel(const uint32_t *__restrict__ key_sorted, const int32_t *__restrict__ len2, int64_t S,
                                   int32_t chunk, int32_t *__restrict__ nch) {
    const int64_t s = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (s > S) return;
    nch[s] = (s < S && key_sorted[s] % 3 == 0) ? (len2[s] + chunk - 1) / chunk : 0;
}

// chunk_ptr of window w starts at seg_chunk[first long segment] + w and holds one terminator.
__global__ void chunk_fill_kernel(const int32_t *__restrict__ seg_ptr, const int32_t *__restrict__ seg_chunk,
                                  int64_t seg_begin, int64_t seg_end, int32_t chunk, int32_t w,
                                  int32_t *__restrict__ chunk_ptr) {
    const int64_t s = seg_begin + static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (s >= seg_end) return;
    const int32_t c0 = seg_chunk[s], c1 = seg_chunk[s + 1];
    for (int32_t c = c0; c < c1; ++c) chunk_ptr[c + w] = seg_ptr[s] + (c - c0) * chunk;
    if (s == seg_end - 1) chunk_ptr[c1 + w] = seg_ptr[s + 1];
}

// bounds[k] = first segment (in the final order) whose key is >= k, for k = 0..2W.
__global__ void window_bounds_kernel(const uint32_t *__restrict__ key_sorted, int64_t S, int32_t nkeys,
                                     int64_t *__restrict__ bounds) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k > nkeys) return;
    int64_t lo = 0, hi = S;
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (key_sorted[mid] < static_cast<uint32_t>(k)) lo = mid + 1;
        else hi = mid;
    }
    bounds[k] = lo;
}

}  // namespace sd

// =====================================================================================
// the plan object
// =====================================================================================
struct sd_plan {
    const int32_t *rowptr = nullptr;
    const int32_t *colind = nullptr;
    const void *vals = nullptr;
    int64_t M = 0, K = 0, N = 0, nnz = 0;
    int dtype = SD_F32;
    int device = 0;
    sd_plan_info_t info{};

    // MERGE: segment arrays the kernels read (the caller's CSR when windows == 1)
    const int32_t *m_ptr = nullptr;
    const int32_t *m_col = nullptr;
    const void *m_vals = nullptr;
    const int32_t *m_seg_row = nullptr;
    int32_t *w_ptr = nullptr;      // plan-owned when windows > 1
    int32_t *w_col = nullptr;
    void *w_vals = nullptr;
    int32_t *w_src = nullptr;   // position in the caller's arrays of every re-bucketed nonzero
    int32_t *w_seg_row = nullptr;
    int64_t num_segments = 0;
    int32_t *seg_chunk = nullptr;   // [S + 1] first chunk of every segment (long segments own chunks)
    int32_t *chunk_ptr = nullptr;   // per window: nonzero boundaries of its chunks, one terminator each
    float *chunk_out = nullptr;     // [chunks][N] partial sums of the chunks
    int64_t num_chunks = 0;
    // window-major plans run the three independent segment classes of a window side by side
    cudaStream_t aux[2] = {nullptr, nullptr};
    cudaEvent_t ev_fork = nullptr, ev_join[2] = {nullptr, nullptr};
    cudaStream_t chunk_stream = nullptr;     // the chunk kernels of all windows run ahead on a stream of their own
    std::vector<cudaEvent_t> ev_chunk;       // one per window: its chunk sums are complete
    struct Window {
        int64_t seg_begin, seg_end;     // segments of the merge-path kernel (all of them without windows)
        int64_t short_begin, short_end; // segments of the group-per-segment kernel (windows only)
        int64_t single_begin, single_end; // one-nonzero segments (windows only)
        int32_t single_nz;              // position of the first of them in the re-bucketed nonzeros
        int64_t chunk_begin, chunk_end; // chunks of the long segments (windows only)
        int64_t tile_base;              // first tile of the window in the concatenated tile numbering
        int32_t ntiles, nshort, nlong;
    };
    std::vector<Window> wins;
    int32_t *tile_seg = nullptr;
    int32_t *fix_short = nullptr;
    int32_t *fix_long = nullptr;
    float *tile_head = nullptr;
    float *tile_tail = nullptr;
    int64_t ntiles = 0;

    // HYBRID: rows of at least h_T nonzeros ("heavy") run as chunks of the caller's CSR arrays, the rest row-wise
    int32_t *h_rows = nullptr;       // [h_nl] heavy rows, ascending
    int32_t *h_chunk_ptr = nullptr;  // [h_nl + 1] first chunk of every heavy row (chunks are numbered row by row)
    int2 *h_ranges = nullptr;        // [h_nc] nonzero range of every chunk
    int32_t *h_order = nullptr;      // [h_nc] chunk ids in the order the chunk kernel takes them: by column window
    int32_t *h_giant = nullptr;      // [h_ng] positions in h_rows of the rows of more than kGiantChunks chunks (a CTA sums each)
    int64_t h_ng = 0;
    int32_t *h_light = nullptr;      // [M - h_nl] light rows, longest first, ascending inside a length
    int64_t h_nm = 0;                // the first h_nm of them have at least kHybridMedium nonzeros: one lane group per row
    int4 *h_desc = nullptr;          // [M - h_nl] per light row, in list order: {row, first nonzero, its column, length} (rebuilt at load)
    int64_t h_nl = 0, h_nc = 0;
    int32_t h_T = 0;

    // narrow dense operands (N <= kCooMaxN) of the merge family
    int32_t *coo_row = nullptr;
    int32_t *coo_c1_row = nullptr, *coo_c2_row = nullptr;
    float *coo_c1_val = nullptr, *coo_c2_val = nullptr;

    // BSR
    int32_t *browptr = nullptr;
    int32_t *bcol = nullptr;
    void *bval = nullptr;
    void *bval_mma = nullptr;   // tensor-core operand images of the blocks
    int32_t *bsr_part = nullptr; // block-row ranges of the tensor-core kernel's CTAs
    int32_t bsr_nparts = 0;
    int32_t *dev_error = nullptr;
    int64_t nnzb = 0;
    mutable sd::TcMapCache tc_map;   // descriptor of the last dense operand (sd_spmm takes the plan as const)
    int32_t test_wait_expiry = 0;

    // host-buffer entry point
    void *stage_B = nullptr;
    float *stage_C = nullptr;
    cudaStream_t host_stream = nullptr;

    int64_t owned = 0;

    sd_features_t feat{};       // extended analysis, computed at the first sd_plan_get_features
    bool have_feat = false;
};

namespace sd {

static sd_status_t dev_alloc(sd_plan *p, void **out, size_t bytes, const char *what) {
    *out = nullptr;
    if (bytes == 0) bytes = 16;
    cudaError_t e = cudaMalloc(out, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        set_error(SD_ERR_ALLOC, "cudaMalloc(%zu bytes) for %s failed: %s", bytes, what, cudaGetErrorString(e));
        return SD_ERR_ALLOC;
    }
    if (p) p->owned += static_cast<int64_t>(bytes);
    return SD_OK;
}

struct TempBuf {   // frees temporary device memory on every exit path
    void *p = nullptr;
    ~TempBuf() { if (p) cudaFree(p); }
    sd_status_t get(size_t bytes, const char *what) { return dev_alloc(nullptr, &p, bytes, what); }
};

// Family rule on the integer summary.  The paper ranks templates with a learned model and a
// measured search (Sec. 3.2-3.3) and prints no thresholds; these are fixed integer rules:
//   BSR-TC    rows strictly ascending, N >= 64 and a multiple of 32 (fp32) / 64 (bf16) columns, and
//             rho_BSR(16) = 256 nnzb / nnz <= rho_max(dtype, N) (Eq. 4)
//   MERGE     (max r >= 256 and rows >= 256 hold >= 10 % of nnz) or CV(r)^2 >= 4
//   ROWSPLIT  otherwise
// rho_max is where the block form stops paying on this GPU (Sec. 3.1: dense tiles pay "when
// useful arithmetic outweighs compaction and fill-in costs").  The tensor-core kernel's time
// depends on the number of blocks only, the CSR kernels' time on the number of nonzeros; the
// measured cross-over (random 16x16 blocks thinned to a given fill) by width and value type:
//              N < 128   128 <= N < 256   N >= 256
//     fp32       9/8          2              3
//     bf16       3            7              10
static int decide_family(const sd_plan_info_t &s, int dtype) {
    int64_t num, den = 1;
    if (dtype == SD_BF16) {
        num = s.N < 128 ? 3 : (s.N < 256 ? 7 : 10);
    } else if (s.N < 128) {
        num = 9;
        den = 8;
    } else {
        num = s.N < 256 ? 2 : 3;
    }
    // the tensor-core kernel serves dense widths that are whole 128-byte groups of columns; at any other
    // width the block form would run its SIMT kernel, which is slower than the CSR kernels at every width
    const int64_t group = dtype == SD_BF16 ? 64 : 32;
    const bool tc_width = s.N >= 64 && s.N % group == 0;   // 32 fp32 columns: the row-split kernel is ahead even on full blocks
    if (tc_width && s.nnz > 0 && s.unsorted_rows == 0 && den * 256 * s.nnzb16 <= num * s.nnz) return SD_BSR_TC;
    const unsigned __int128 lhs = static_cast<unsigned __int128>(static_cast<uint64_t>(s.M)) * s.sum_r2;
    const unsigned __int128 rhs =
        static_cast<unsigned __int128>(5) * static_cast<uint64_t>(s.nnz) * static_cast<uint64_t>(s.nnz);
    const bool skew = (s.max_r >= 256 && 10 * s.nnz_long_rows >= s.nnz) || (s.nnz > 0 && lhs >= rhs);
    return skew ? SD_MERGE : SD_ROWSPLIT;
}

// Number of column windows: none unless the rows are short on average (nnz < 16 M, so the
// extra read-modify-write of C per (row, window) pair stays below the gather traffic saved),
// the columns are sorted, and B does not fit in 60 % of L2; then the smallest power of two
// that makes one window's slab of B fit.
static int decide_windows(const sd_plan_info_t &s, int dtype) {
    const int64_t es = dtype == SD_F32 ? 4 : 2;
    const int64_t bbytes = s.K * s.N * es;
    const int64_t budget = s.l2_bytes / 10 * 6;
    if (s.unsorted_rows != 0 || s.nnz >= 16 * s.M || budget <= 0 || bbytes <= budget) return 1;
    int w = 1;
    while (w < 64 && bbytes > budget * w) w <<= 1;
    return w;
}

// One window, but still the class split (long segments as chunks, short ones one lane group each,
// one-nonzero rows flat) instead of merge-path tiles: measured on R-MAT and rank-size matrices, the split
// is ahead from 16 fp32 / 8 bf16 columns up to 64 fp32 / 32 bf16 columns (0.68 to 0.94 of the tile kernel's
// time; 0.80 at 8 bf16 columns) and behind or level at 8 fp32 columns and beyond those widths (the sweep of
// `bench.py --regret`).  Needs ascending columns like the windows.
static bool decide_class_split(const sd_plan_info_t &s, int dtype) {
    const int64_t widest = dtype == SD_BF16 ? 32 : 64;
    const int64_t narrowest = dtype == SD_BF16 ? 8 : 16;
    return s.unsorted_rows == 0 && s.nnz > 0 && s.N >= narrowest && s.N <= widest;
}

// The hybrid family in place of the merge family's own schedules, for matrices with ascending columns (measured,
// `bench.py --regret`; fp32 values allow wider rows than bf16 values, whose lanes hold eight accumulators per row):
//   without column windows: from 5 columns up to rows of B of 384 bytes with fp32 values (96 columns) and 256 bytes with
//     bf16 values (128 columns), when the call gathers at least 256 MiB (nnz x bytes of a row of B): below that its
//     launches weigh too much (R-MAT scale 18 at 8 columns, 126 / 252 MB gathered: 1.27 / 1.04 to 1.13 of the tiles'
//     time).  On the R-MAT matrix it takes 0.70 to 0.90 of the better of merge-path tiles and class split up to 256-byte
//     rows (bf16 at 256 bytes: level), 0.87 of the tiles' time at 96 fp32 columns, and is behind them at 128 fp32
//     columns (1.06) and 192 bf16 columns (1.16).
//   with column windows: where one row of B is 64 to 192 bytes with fp32 values (16 to 48 columns) and 64 to 128 bytes
//     with bf16 values (32 to 64 columns): on the rank-size matrix 0.84 to 0.93 of the windowed class split's time at 96
//     and 128 bytes and level with it (0.99 to 1.01) at the ends of the band, with 3 launches instead of 16 to 64 and a
//     quarter of the plan memory; behind it at 64 fp32 columns (1.07) and 96 or 128 bf16 columns (1.2), where the light
//     rows gather wide rows of B from DRAM that the windowed schedule finds in L2.
static bool decide_hybrid(const sd_plan_info_t &s, int dtype, int windows) {
    const bool f32 = dtype == SD_F32;
    const int64_t row_bytes = s.N * (f32 ? 4 : 2);
    if (s.unsorted_rows != 0) return false;
    if (windows > 1) return row_bytes >= 64 && row_bytes <= (f32 ? 192 : 128);
    return s.N > kCooMaxN && row_bytes <= (f32 ? 384 : 256) && s.nnz * row_bytes >= (int64_t{1} << 28);
}

__global__ void iota_kernel(int32_t *out, int64_t n) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) out[i] = static_cast<int32_t>(i);
}

constexpr int kChunkNnz = 128;      // long segments are cut into pieces of at most this many nonzeros
constexpr int kShortSegment = 32;   // segments up to this many nonzeros go to the group-per-segment kernel
constexpr int kHybridHeavy = 256;   // hybrid family: rows of at least this many nonzeros run as chunks: the long-row threshold
                                    // of the paper's appendix listing; measured on the rank-size matrix at 128-byte rows of
                                    // B, 64 / 128 / 192 / 256 give 1.054 / 0.987 / 0.956 / 0.950 ms
constexpr int kHybridMedium = 4;    // light rows of at least this many nonzeros take one lane group each, a step of nonzeros
                                    // at a time; shorter ones run several rows per lane group, a nonzero at a time
                                    // (2 / 3 / 4 / 8 / 16 / 32 measured on six workloads: 4 is best or level on five)
constexpr int kHybridHeavyMax = 256;   // upper limit: a light row is one running sum

// Re-buckets the nonzeros by column window and builds the (row, window) segment list, ordered by
// (window, class, row): inside a window the long segments come first (merge-path kernel), then the
// short ones (group-per-segment kernel), then those of exactly one nonzero (flat kernel).
// bounds[3w .. 3w+3] delimit the three classes of window w.
static sd_status_t build_windows(sd_plan *p, int W, std::vector<int64_t> &bounds, cudaStream_t st) {
    const int64_t nnz = p->nnz, M = p->M;
    const int32_t wcols = static_cast<int32_t>((p->K + W - 1) / W);
    const size_t es = p->dtype == SD_F32 ? 4 : 2;
    const int64_t E = p->info.empty_rows;
    sd_status_t s;
    TempBuf wkey, wkey_sorted, rowid, w_row, ids, perm, tmp, flag, nsel, heads;
    if ((s = wkey.get(4 * nnz, "window keys"))) return s;
    if ((s = wkey_sorted.get(4 * nnz, "window keys"))) return s;
    if ((s = rowid.get(4 * nnz, "row ids"))) return s;
    if ((s = w_row.get(4 * nnz, "row ids"))) return s;
    if ((s = ids.get(4 * nnz, "positions"))) return s;
    if ((s = perm.get(4 * nnz, "permutation"))) return s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->w_col), 4 * nnz, "window-major colind"))) return s;
    if ((s = dev_alloc(p, &p->w_vals, es * nnz, "window-major values"))) return s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->w_src), 4 * nnz, "window-major source positions"))) return s;

    window_keys_kernel<<<148 * 8, 256, 0, st>>>(p->rowptr, p->colind, M, wcols, static_cast<uint32_t *>(wkey.p),
                                               static_cast<int32_t *>(rowid.p));
    SD_CUDA_TRY(cudaGetLastError());
    iota_kernel<<<ceil_div(nnz, 256), 256, 0, st>>>(static_cast<int32_t *>(ids.p), nnz);
    SD_CUDA_TRY(cudaGetLastError());
    int bits = 1;
    while ((1 << bits) < W) ++bits;
    size_t tb = 0;
    SD_CUDA_TRY(cub::DeviceRadixSort::SortPairs(nullptr, tb, static_cast<uint32_t *>(wkey.p),
                                                static_cast<uint32_t *>(wkey_sorted.p), static_cast<int32_t *>(ids.p),
                                                static_cast<int32_t *>(perm.p), nnz, 0, bits, st));
    if ((s = tmp.get(tb, "sort scratch"))) return s;
    SD_CUDA_TRY(cub::DeviceRadixSort::SortPairs(tmp.p, tb, static_cast<uint32_t *>(wkey.p),
                                                static_cast<uint32_t *>(wkey_sorted.p), static_cast<int32_t *>(ids.p),
                                                static_cast<int32_t *>(perm.p), nnz, 0, bits, st));
    window_rows_kernel<<<ceil_div(nnz, 256), 256, 0, st>>>(static_cast<int32_t *>(perm.p), static_cast<int32_t *>(rowid.p),
                                                          nnz, static_cast<int32_t *>(w_row.p));
    SD_CUDA_TRY(cudaGetLastError());
    // runs of (window, row): head flags -> head positions
    const int64_t nflag = nnz > M ? nnz : M;
    if ((s = flag.get(nflag, "segment flags"))) return s;
    if ((s = nsel.get(sizeof(int32_t), "segment count"))) return s;
    if ((s = heads.get(4 * nnz, "segment heads"))) return s;
    window_headflag_kernel<<<ceil_div(nnz, 256), 256, 0, st>>>(static_cast<uint32_t *>(wkey_sorted.p),
                                                              static_cast<int32_t *>(w_row.p), nnz,
                                                              static_cast<uint8_t *>(flag.p));
    SD_CUDA_TRY(cudaGetLastError());
    cub::CountingInputIterator<int32_t> cnt(0);
    size_t tb2 = 0;
    SD_CUDA_TRY(cub::DeviceSelect::Flagged(nullptr, tb2, cnt, static_cast<uint8_t *>(flag.p), static_cast<int32_t *>(heads.p),
                                           static_cast<int32_t *>(nsel.p), static_cast<int>(nflag), st));
    TempBuf tmp2;
    if ((s = tmp2.get(tb2, "select scratch"))) return s;
    SD_CUDA_TRY(cub::DeviceSelect::Flagged(tmp2.p, tb2, cnt, static_cast<uint8_t *>(flag.p), static_cast<int32_t *>(heads.p),
                                           static_cast<int32_t *>(nsel.p), static_cast<int>(nnz), st));
    int32_t nheads = 0;
    SD_CUDA_TRY(cudaMemcpyAsync(&nheads, nsel.p, sizeof nheads, cudaMemcpyDeviceToHost, st));
    SD_CUDA_TRY(cudaStreamSynchronize(st));
    const int64_t S = E + nheads;
    p->num_segments = S;

    TempBuf seg_start, seg_len, seg_row1, seg_key, seg_key_sorted, seg_ids, order, len2, dbounds;
    if ((s = seg_start.get(4 * S, "segment starts"))) return s;
    if ((s = seg_len.get(4 * S, "segment lengths"))) return s;
    if ((s = seg_row1.get(4 * S, "segment rows"))) return s;
    if ((s = seg_key.get(4 * S, "segment keys"))) return s;
    if ((s = seg_key_sorted.get(4 * S, "segment keys"))) return s;
    if ((s = seg_ids.get(4 * S, "segment ids"))) return s;
    if ((s = order.get(4 * S, "segment order"))) return s;
    if ((s = len2.get(4 * (S + 1), "segment lengths"))) return s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->w_ptr), 4 * (S + 1), "segment pointers"))) return s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->w_seg_row), 4 * (S + 1), "segment rows"))) return s;
    if (E > 0) {   // ids of the empty rows, ascending, at the front of the first ordering
        window_emptyflag_kernel<<<ceil_div(M, 256), 256, 0, st>>>(p->rowptr, M, static_cast<uint8_t *>(flag.p));
        SD_CUDA_TRY(cudaGetLastError());
        SD_CUDA_TRY(cub::DeviceSelect::Flagged(tmp2.p, tb2, cnt, static_cast<uint8_t *>(flag.p),
                                               static_cast<int32_t *>(seg_row1.p), static_cast<int32_t *>(nsel.p),
                                               static_cast<int>(M), st));
    }
    window_segments_kernel<<<ceil_div(S, 256), 256, 0, st>>>(
        p->rowptr, p->colind, static_cast<uint32_t *>(wkey_sorted.p), static_cast<int32_t *>(w_row.p),
        static_cast<int32_t *>(heads.p), wcols, kShortSegment, E, S, nnz, static_cast<int32_t *>(seg_start.p),
        static_cast<int32_t *>(seg_len.p), static_cast<int32_t *>(seg_row1.p), static_cast<uint32_t *>(seg_key.p));
    SD_CUDA_TRY(cudaGetLastError());
    // stable sort of the segments by (window, class)
    iota_kernel<<<ceil_div(S, 256), 256, 0, st>>>(static_cast<int32_t *>(seg_ids.p), S);
    SD_CUDA_TRY(cudaGetLastError());
    int kbits = 1;
    while ((1 << kbits) < 3 * W) ++kbits;
    size_t tb3 = 0;
    SD_CUDA_TRY(cub::DeviceRadixSort::SortPairs(nullptr, tb3, static_cast<uint32_t *>(seg_key.p),
                                                static_cast<uint32_t *>(seg_key_sorted.p),
                                                static_cast<int32_t *>(seg_ids.p), static_cast<int32_t *>(order.p), S, 0,
                                                kbits, st));
    TempBuf tmp3;
    if ((s = tmp3.get(tb3, "sort scratch"))) return s;
    SD_CUDA_TRY(cub::DeviceRadixSort::SortPairs(tmp3.p, tb3, static_cast<uint32_t *>(seg_key.p),
                                                static_cast<uint32_t *>(seg_key_sorted.p),
                                                static_cast<int32_t *>(seg_ids.p), static_cast<int32_t *>(order.p), S, 0,
                                                kbits, st));
    window_reorder_kernel<<<ceil_div(S, 256), 256, 0, st>>>(static_cast<int32_t *>(order.p),
                                                           static_cast<int32_t *>(seg_len.p),
                                                           static_cast<int32_t *>(seg_row1.p), S,
                                                           static_cast<int32_t *>(len2.p), p->w_seg_row);
    SD_CUDA_TRY(cudaGetLastError());
    SD_CUDA_TRY(cudaMemsetAsync(static_cast<int32_t *>(len2.p) + S, 0, 4, st));
    size_t tb4 = 0;
    SD_CUDA_TRY(cub::DeviceScan::ExclusiveSum(nullptr, tb4, static_cast<int32_t *>(len2.p), p->w_ptr,
                                              static_cast<int>(S + 1), st));
    TempBuf tmp4;
    if ((s = tmp4.get(tb4, "scan scratch"))) return s;
    SD_CUDA_TRY(cub::DeviceScan::ExclusiveSum(tmp4.p, tb4, static_cast<int32_t *>(len2.p), p->w_ptr,
                                              static_cast<int>(S + 1), st));
    if (p->dtype == SD_F32)
        window_gather_kernel<float><<<ceil_div(nnz, 256), 256, 0, st>>>(
            p->w_ptr, static_cast<int32_t *>(order.p), static_cast<int32_t *>(seg_start.p), static_cast<int32_t *>(perm.p),
            p->colind, static_cast<const float *>(p->vals), S, nnz, p->w_col, static_cast<float *>(p->w_vals), p->w_src);
    else
        window_gather_kernel<uint16_t><<<ceil_div(nnz, 256), 256, 0, st>>>(
            p->w_ptr, static_cast<int32_t *>(order.p), static_cast<int32_t *>(seg_start.p), static_cast<int32_t *>(perm.p),
            p->colind, static_cast<const uint16_t *>(p->vals), S, nnz, p->w_col, static_cast<uint16_t *>(p->w_vals), p->w_src);
    SD_CUDA_TRY(cudaGetLastError());
    if ((s = dbounds.get(sizeof(int64_t) * (3 * W + 1), "window bounds"))) return s;
    window_bounds_kernel<<<1, 256, 0, st>>>(static_cast<uint32_t *>(seg_key_sorted.p), S, 3 * W,
                                           static_cast<int64_t *>(dbounds.p));
    SD_CUDA_TRY(cudaGetLastError());
    bounds.assign(3 * W + 1, 0);
    SD_CUDA_TRY(cudaMemcpyAsync(bounds.data(), dbounds.p, sizeof(int64_t) * (3 * W + 1), cudaMemcpyDeviceToHost, st));
    SD_CUDA_TRY(cudaStreamSynchronize(st));

    // chunks of the long segments: counts -> exclusive scan -> boundaries
    TempBuf nch;
    if ((s = nch.get(4 * (S + 1), "chunk counts"))) return s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->seg_chunk), 4 * (S + 1), "segment chunks"))) return s;
    chunk_count_kernel<<<ceil_div(S + 1, 256), 256, 0, st>>>(static_cast<uint32_t *>(seg_key_sorted.p),
                                                            static_cast<int32_t *>(len2.p), S, kChunkNnz,
                                                            static_cast<int32_t *>(nch.p));
    SD_CUDA_TRY(cudaGetLastError());
    SD_CUDA_TRY(cub::DeviceScan::ExclusiveSum(tmp4.p, tb4, static_cast<int32_t *>(nch.p), p->seg_chunk,
                                              static_cast<int>(S + 1), st));
    int32_t total_chunks = 0;
    SD_CUDA_TRY(cudaMemcpyAsync(&total_chunks, p->seg_chunk + S, 4, cudaMemcpyDeviceToHost, st));
    SD_CUDA_TRY(cudaStreamSynchronize(st));
    p->num_chunks = total_chunks;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->chunk_ptr), 4 * (static_cast<int64_t>(total_chunks) + W + 1),
                       "chunk boundaries")))
        return s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->chunk_out), sizeof(float) * total_chunks * p->N, "chunk sums")))
        return s;
    for (int w = 0; w < W; ++w) {
        const int64_t sb = bounds[3 * w], se = bounds[3 * w + 1];
        if (se > sb) {
            chunk_fill_kernel<<<ceil_div(se - sb, 256), 256, 0, st>>>(p->w_ptr, p->seg_chunk, sb, se, kChunkNnz, w,
                                                                     p->chunk_ptr);
            SD_CUDA_TRY(cudaGetLastError());
        }
    }
    SD_CUDA_TRY(cudaStreamSynchronize(st));
    return SD_OK;
}

static sd_status_t create_split_streams(sd_plan *p, int W);

// `split`: the segments are re-bucketed by (window, class) and run through the chunk / segment / single
// kernels; always so with W > 1, and with W = 1 when the class split alone pays (decide_class_split).
static sd_status_t build_merge(sd_plan *p, int W, bool split, cudaStream_t st) {
    sd_status_t s;
    std::vector<int64_t> win_seg;   // per window: start of the long class, start of the short class
    if (W < 1) W = 1;
    if (W > 1) split = true;
    if (split) {
        if ((s = build_windows(p, W, win_seg, st))) return s;
        p->m_ptr = p->w_ptr;
        p->m_col = p->w_col;
        p->m_vals = p->w_vals;
        p->m_seg_row = p->w_seg_row;
    } else {
        W = 1;
        p->m_ptr = p->rowptr;
        p->m_col = p->colind;
        p->m_vals = p->vals;
        p->m_seg_row = nullptr;
        p->num_segments = p->M;
        win_seg = {0, p->M, p->M, p->M};
    }
    // nonzero positions of the class boundaries
    std::vector<int32_t> win_nz(3 * W + 1, 0);
    for (int k = 0; k <= 3 * W; ++k)
        SD_CUDA_TRY(cudaMemcpyAsync(&win_nz[k], p->m_ptr + win_seg[k], sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    SD_CUDA_TRY(cudaStreamSynchronize(st));
    int64_t ntiles = 0;
    p->wins.clear();
    for (int w = 0; w < W; ++w) {
        sd_plan::Window win;
        win.seg_begin = win_seg[3 * w];
        win.seg_end = win_seg[3 * w + 1];
        win.short_begin = win_seg[3 * w + 1];
        win.short_end = win_seg[3 * w + 2];
        win.single_begin = win_seg[3 * w + 2];
        win.single_end = win_seg[3 * w + 3];
        win.single_nz = win_nz[3 * w + 2];
        win.chunk_begin = win.chunk_end = 0;
        int64_t total = (win.seg_end - win.seg_begin) + (win_nz[3 * w + 1] - win_nz[3 * w]);
        if (split) total = 0;   // with windows the long segments run as chunks, not as merge-path tiles
        win.ntiles = static_cast<int32_t>((total + kMergeTile - 1) / kMergeTile);
        win.tile_base = ntiles;
        win.nshort = win.nlong = 0;
        ntiles += win.ntiles;
        p->wins.push_back(win);
    }
    if (ntiles > INT32_MAX / 2) {
        set_error(SD_ERR_UNSUPPORTED, "too many merge tiles");
        return SD_ERR_UNSUPPORTED;
    }
    p->ntiles = ntiles;
    // tile tables are concatenated: window w owns entries [tile_base + w, tile_base + w + ntiles_w]
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->tile_seg), sizeof(int32_t) * (ntiles + W), "tile table")))
        return s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->fix_short), sizeof(int32_t) * (ntiles + 1), "fix-up list")))
        return s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->fix_long), sizeof(int32_t) * (ntiles + 1), "fix-up list")))
        return s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->tile_head), sizeof(float) * ntiles * p->N, "tile heads")))
        return s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->tile_tail), sizeof(float) * ntiles * p->N, "tile tails")))
        return s;
    int32_t max_tiles = 1;
    for (auto &win : p->wins) max_tiles = std::max(max_tiles, win.ntiles);
    TempBuf flags_s, flags_l, nsel, tmp;
    if ((s = flags_s.get(max_tiles, "fix-up flags"))) return s;
    if ((s = flags_l.get(max_tiles, "fix-up flags"))) return s;
    if ((s = nsel.get(2 * sizeof(int32_t), "fix-up counts"))) return s;
    size_t tb = 0;
    cub::CountingInputIterator<int32_t> ids(0);
    int32_t *dn = static_cast<int32_t *>(nsel.p);
    SD_CUDA_TRY(cub::DeviceSelect::Flagged(nullptr, tb, ids, static_cast<uint8_t *>(flags_s.p), p->fix_short, dn, max_tiles,
                                           st));
    if ((s = tmp.get(tb, "select scratch"))) return s;
    int launches = 0;
    if (split && (s = create_split_streams(p, W))) return s;
    if (split) {   // chunk ranges of the long segments
        std::vector<int32_t> cb(2 * W, 0);
        for (int w = 0; w < W; ++w) {
            SD_CUDA_TRY(cudaMemcpyAsync(&cb[2 * w], p->seg_chunk + p->wins[w].seg_begin, 4, cudaMemcpyDeviceToHost, st));
            SD_CUDA_TRY(cudaMemcpyAsync(&cb[2 * w + 1], p->seg_chunk + p->wins[w].seg_end, 4, cudaMemcpyDeviceToHost, st));
        }
        SD_CUDA_TRY(cudaStreamSynchronize(st));
        for (int w = 0; w < W; ++w) {
            p->wins[w].chunk_begin = cb[2 * w];
            p->wins[w].chunk_end = cb[2 * w + 1];
            if (cb[2 * w + 1] > cb[2 * w]) launches += 2;
        }
    }
    for (int w = 0; w < W; ++w) {
        sd_plan::Window &win = p->wins[w];
        if (win.short_end > win.short_begin) launches += 1;
        if (win.single_end > win.single_begin) launches += 1;
        int32_t *table = p->tile_seg + win.tile_base + w;
        merge_table_kernel<<<ceil_div(win.ntiles + 1, 256), 256, 0, st>>>(p->m_ptr, win.seg_begin, win.seg_end, kMergeTile,
                                                                         win.ntiles, table);
        SD_CUDA_TRY(cudaGetLastError());
        if (win.ntiles == 0) continue;
        merge_fixflag_kernel<<<ceil_div(win.ntiles, 256), 256, 0, st>>>(p->m_ptr, table, win.seg_begin, kMergeTile,
                                                                       win.ntiles, static_cast<uint8_t *>(flags_s.p),
                                                                       static_cast<uint8_t *>(flags_l.p));
        SD_CUDA_TRY(cudaGetLastError());
        SD_CUDA_TRY(cub::DeviceSelect::Flagged(tmp.p, tb, ids, static_cast<uint8_t *>(flags_s.p),
                                               p->fix_short + win.tile_base, dn, win.ntiles, st));
        SD_CUDA_TRY(cub::DeviceSelect::Flagged(tmp.p, tb, ids, static_cast<uint8_t *>(flags_l.p),
                                               p->fix_long + win.tile_base, dn + 1, win.ntiles, st));
        int32_t hn[2] = {0, 0};
        SD_CUDA_TRY(cudaMemcpyAsync(hn, dn, sizeof hn, cudaMemcpyDeviceToHost, st));
        SD_CUDA_TRY(cudaStreamSynchronize(st));
        win.nshort = hn[0];
        win.nlong = hn[1];
        launches += 1 + (win.nshort > 0) + (win.nlong > 0);
    }
    p->info.tile_items = kMergeTile;
    p->info.num_tiles = ntiles;
    p->info.num_segments = p->num_segments;
    p->info.windows = W;
    p->info.class_split = split ? 1 : 0;
    p->info.launches = launches;
    // Narrow dense operands take the COO segmented reduction instead of the tile kernel (the tile
    // table above stays valid and inspectable): one row index per nonzero and two carry lists.
    if (!split && p->N >= 1 && p->N <= kCooMaxN && p->nnz > 0 && !switches().no_coo) {
        const int cchunk = coo_chunk(static_cast<int>(p->N));
        const int64_t chunks1 = (p->nnz + cchunk - 1) / cchunk, count2 = 2 * chunks1;
        const int64_t chunks2 = (count2 + kCooCarryChunk - 1) / kCooCarryChunk, count3 = 2 * chunks2;
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->coo_row), sizeof(int32_t) * p->nnz, "row index per nonzero"))) return s;
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->coo_c1_row), sizeof(int32_t) * count2, "carry rows"))) return s;
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->coo_c1_val), sizeof(float) * count2 * p->N, "carry sums"))) return s;
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->coo_c2_row), sizeof(int32_t) * count3, "carry rows (level 2)"))) return s;
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->coo_c2_val), sizeof(float) * count3 * p->N, "carry sums (level 2)"))) return s;
        SD_CUDA_TRY(build_coo_rows(p->rowptr, p->M, p->nnz, p->coo_row, st));
        SD_CUDA_TRY(cudaStreamSynchronize(st));
        p->info.launches = 2 + (count2 > kCooDirectFinal);
    }
    return SD_OK;
}

// ---- HYBRID: light rows row-wise, heavy rows as chunks inside column windows --------------------------------
struct GiantRow {
    const int32_t *chunk_ptr;
    __device__ bool operator()(int32_t i) const { return chunk_ptr[i + 1] - chunk_ptr[i] > kGiantChunks; }
};

struct HeavyRow {
    const int32_t *rowptr;
    int32_t T;
    __device__ bool operator()(int32_t r) const { return rowptr[r + 1] - rowptr[r] >= T; }
};

__device__ __forceinline__ int32_t first_not_below(const int32_t *__restrict__ colind, int32_t lo, int32_t hi, int64_t col) {
    while (lo < hi) {
        const int32_t mid = lo + ((hi - lo) >> 1);
        if (colind[mid] < col) lo = mid + 1;
        else hi = mid;
    }
    return lo;
}

// One thread per (heavy row i, window w): the nonzeros of the row whose columns fall in the window are a contiguous
// range (columns ascend); counts its chunks into a row-major and a window-major table.
__global__ void __launch_bounds__(256)
hybrid_count_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colind, const int32_t *__restrict__ rows,
                    int64_t nl, int32_t W, int64_t wcols, int32_t *__restrict__ start, int32_t *__restrict__ by_row,
                    int32_t *__restrict__ by_win) {
    const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t >= nl * W) return;
    const int64_t i = t / W;
    const int32_t w = static_cast<int32_t>(t % W);
    const int32_t r = rows[i], p0 = rowptr[r], p1 = rowptr[r + 1];
    const int32_t lo = w == 0 ? p0 : first_not_below(colind, p0, p1, w * wcols);
    const int32_t hi = w == W - 1 ? p1 : first_not_below(colind, lo, p1, (w + 1) * wcols);
    const int32_t n = (hi - lo + kChunkNnz - 1) / kChunkNnz;
    start[2 * t] = lo;
    start[2 * t + 1] = hi;
    by_row[t] = n;
    by_win[static_cast<int64_t>(w) * nl + i] = n;
}

__global__ void __launch_bounds__(256)
hybrid_fill_kernel(const int32_t *__restrict__ start, const int32_t *__restrict__ row_off, const int32_t *__restrict__ win_off,
                   int64_t nl, int32_t W, int2 *__restrict__ ranges, int32_t *__restrict__ order,
                   int32_t *__restrict__ chunk_ptr) {
    const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t > nl * W) return;
    if (t == nl * W) {
        chunk_ptr[nl] = row_off[t];
        return;
    }
    const int64_t i = t / W;
    const int32_t w = static_cast<int32_t>(t % W);
    const int32_t c = row_off[t], o = win_off[static_cast<int64_t>(w) * nl + i];
    if (w == 0) chunk_ptr[i] = c;
    const int32_t lo = start[2 * t], hi = start[2 * t + 1];
    for (int32_t j = 0, x = lo; x < hi; ++j, x += kChunkNnz) {
        ranges[c + j] = make_int2(x, min(x + kChunkNnz, hi));
        order[o + j] = c + j;
    }
}

// Sort key of the light-row list: heavy rows first (they are not part of the list), then light rows by falling length.
__global__ void __launch_bounds__(256)
hybrid_light_key_kernel(const int32_t *__restrict__ rowptr, int64_t M, int32_t T, int32_t *__restrict__ key,
                        int32_t *__restrict__ id) {
    const int64_t r = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (r >= M) return;
    const int32_t len = rowptr[r + 1] - rowptr[r];
    key[r] = len >= T ? 0 : T - len;
    id[r] = static_cast<int32_t>(r);
}

// Descriptors of the light rows: everything the first gather of a row needs, in one 16-byte load.
__global__ void __launch_bounds__(256)
hybrid_desc_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colind, const int32_t *__restrict__ rows,
                   int64_t n, int4 *__restrict__ desc) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int32_t r = rows[i], p0 = rowptr[r], len = rowptr[r + 1] - p0;
    desc[i] = make_int4(r, p0, len > 0 ? colind[p0] : 0, len);
}

static sd_status_t build_light_desc(sd_plan *p, cudaStream_t st) {
    const int64_t n = p->M - p->h_nl;
    if (n <= 0) return SD_OK;
    sd_status_t s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->h_desc), sizeof(int4) * n, "light row descriptors"))) return s;
    hybrid_desc_kernel<<<ceil_div(n, 256), 256, 0, st>>>(p->rowptr, p->colind, p->h_light, n, p->h_desc);
    SD_CUDA_TRY(cudaGetLastError());
    SD_CUDA_TRY(cudaStreamSynchronize(st));
    return SD_OK;
}

// Number of entries of the ascending array `key` that are <= v (one thread).
__global__ void count_not_above_kernel(const int32_t *__restrict__ key, int64_t n, int32_t v, int64_t *__restrict__ out) {
    int64_t lo = 0, hi = n;
    while (lo < hi) {
        const int64_t mid = lo + ((hi - lo) >> 1);
        if (key[mid] <= v) lo = mid + 1;
        else hi = mid;
    }
    *out = lo;
}

static sd_status_t build_hybrid(sd_plan *p, int W, int32_t T, cudaStream_t st) {
    sd_status_t s;
    if (W < 1) W = 1;
    if (T < 2) T = 2;
    if (T > kHybridHeavyMax) T = kHybridHeavyMax;
    p->h_T = T;
    TempBuf sel, nsel, tmp, start, by_row, by_win, row_off, win_off;
    if ((s = sel.get(sizeof(int32_t) * p->M, "heavy rows"))) return s;
    if ((s = nsel.get(sizeof(int64_t), "heavy row count"))) return s;
    size_t tb = 0;
    cub::CountingInputIterator<int32_t> ids(0);
    HeavyRow pred{p->rowptr, T};
    SD_CUDA_TRY(cub::DeviceSelect::If(nullptr, tb, ids, static_cast<int32_t *>(sel.p), static_cast<int32_t *>(nsel.p),
                                      static_cast<int32_t>(p->M), pred, st));
    if ((s = tmp.get(tb, "select scratch"))) return s;
    SD_CUDA_TRY(cub::DeviceSelect::If(tmp.p, tb, ids, static_cast<int32_t *>(sel.p), static_cast<int32_t *>(nsel.p),
                                      static_cast<int32_t>(p->M), pred, st));
    int32_t nl = 0;
    SD_CUDA_TRY(cudaMemcpyAsync(&nl, nsel.p, sizeof nl, cudaMemcpyDeviceToHost, st));
    SD_CUDA_TRY(cudaStreamSynchronize(st));
    p->h_nl = nl;
    p->h_nc = 0;
    p->info.windows = W;
    p->info.launches = 1;
    if (nl > 0) {
        const int64_t cells = static_cast<int64_t>(nl) * W;
        if (cells + 1 > INT32_MAX) {
            set_error(SD_ERR_UNSUPPORTED, "too many (heavy row, window) pairs");
            return SD_ERR_UNSUPPORTED;
        }
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->h_rows), sizeof(int32_t) * nl, "heavy rows"))) return s;
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->h_chunk_ptr), sizeof(int32_t) * (nl + 1), "chunk pointers"))) return s;
        SD_CUDA_TRY(cudaMemcpyAsync(p->h_rows, sel.p, sizeof(int32_t) * nl, cudaMemcpyDeviceToDevice, st));
        if ((s = start.get(sizeof(int32_t) * 2 * cells, "window ranges"))) return s;
        if ((s = by_row.get(sizeof(int32_t) * (cells + 1), "chunk counts"))) return s;
        if ((s = by_win.get(sizeof(int32_t) * (cells + 1), "chunk counts"))) return s;
        if ((s = row_off.get(sizeof(int32_t) * (cells + 1), "chunk offsets"))) return s;
        if ((s = win_off.get(sizeof(int32_t) * (cells + 1), "chunk offsets"))) return s;
        SD_CUDA_TRY(cudaMemsetAsync(static_cast<int32_t *>(by_row.p) + cells, 0, sizeof(int32_t), st));
        SD_CUDA_TRY(cudaMemsetAsync(static_cast<int32_t *>(by_win.p) + cells, 0, sizeof(int32_t), st));
        const int64_t wcols = (p->K + W - 1) / W;
        hybrid_count_kernel<<<ceil_div(cells, 256), 256, 0, st>>>(p->rowptr, p->colind, p->h_rows, nl, W, wcols,
                                                                 static_cast<int32_t *>(start.p),
                                                                 static_cast<int32_t *>(by_row.p),
                                                                 static_cast<int32_t *>(by_win.p));
        SD_CUDA_TRY(cudaGetLastError());
        size_t tb2 = 0;
        SD_CUDA_TRY(cub::DeviceScan::ExclusiveSum(nullptr, tb2, static_cast<int32_t *>(by_row.p),
                                                  static_cast<int32_t *>(row_off.p), static_cast<int32_t>(cells + 1), st));
        TempBuf tmp2;
        if ((s = tmp2.get(tb2, "scan scratch"))) return s;
        SD_CUDA_TRY(cub::DeviceScan::ExclusiveSum(tmp2.p, tb2, static_cast<int32_t *>(by_row.p),
                                                  static_cast<int32_t *>(row_off.p), static_cast<int32_t>(cells + 1), st));
        SD_CUDA_TRY(cub::DeviceScan::ExclusiveSum(tmp2.p, tb2, static_cast<int32_t *>(by_win.p),
                                                  static_cast<int32_t *>(win_off.p), static_cast<int32_t>(cells + 1), st));
        int32_t nc = 0;
        SD_CUDA_TRY(cudaMemcpyAsync(&nc, static_cast<int32_t *>(row_off.p) + cells, sizeof nc, cudaMemcpyDeviceToHost, st));
        SD_CUDA_TRY(cudaStreamSynchronize(st));
        p->h_nc = nc;
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->h_ranges), sizeof(int2) * nc, "chunk ranges"))) return s;
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->h_order), sizeof(int32_t) * nc, "chunk order"))) return s;
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->chunk_out), sizeof(float) * nc * p->N, "chunk sums"))) return s;
        hybrid_fill_kernel<<<ceil_div(cells + 1, 256), 256, 0, st>>>(static_cast<int32_t *>(start.p),
                                                                    static_cast<int32_t *>(row_off.p),
                                                                    static_cast<int32_t *>(win_off.p), nl, W, p->h_ranges,
                                                                    p->h_order, p->h_chunk_ptr);
        SD_CUDA_TRY(cudaGetLastError());
        // rows of very many chunks: summed by a whole CTA each
        GiantRow giant{p->h_chunk_ptr};
        SD_CUDA_TRY(cub::DeviceSelect::If(tmp.p, tb, ids, static_cast<int32_t *>(sel.p), static_cast<int32_t *>(nsel.p), nl,
                                          giant, st));
        int32_t ng = 0;
        SD_CUDA_TRY(cudaMemcpyAsync(&ng, nsel.p, sizeof ng, cudaMemcpyDeviceToHost, st));
        SD_CUDA_TRY(cudaStreamSynchronize(st));
        p->h_ng = ng;
        if (ng > 0) {
            if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->h_giant), sizeof(int32_t) * ng, "giant rows"))) return s;
            SD_CUDA_TRY(cudaMemcpyAsync(p->h_giant, sel.p, sizeof(int32_t) * ng, cudaMemcpyDeviceToDevice, st));
            SD_CUDA_TRY(cudaStreamSynchronize(st));
        }
        p->info.launches = 2 + (ng > 0 ? 1 : 0);   // the fused kernel, the chunk sums, the chunk sums of very long rows
    }
    if (nl < p->M) {   // the light rows, longest first
        TempBuf key, key_out, id, id_out, tmp3;
        if ((s = key.get(sizeof(int32_t) * p->M, "light keys"))) return s;
        if ((s = key_out.get(sizeof(int32_t) * p->M, "light keys"))) return s;
        if ((s = id.get(sizeof(int32_t) * p->M, "row ids"))) return s;
        if ((s = id_out.get(sizeof(int32_t) * p->M, "row ids"))) return s;
        hybrid_light_key_kernel<<<ceil_div(p->M, 256), 256, 0, st>>>(p->rowptr, p->M, T, static_cast<int32_t *>(key.p),
                                                                    static_cast<int32_t *>(id.p));
        SD_CUDA_TRY(cudaGetLastError());
        int bits = 1;
        while ((1 << bits) <= T) ++bits;
        size_t tb3 = 0;
        SD_CUDA_TRY(cub::DeviceRadixSort::SortPairs(nullptr, tb3, static_cast<int32_t *>(key.p), static_cast<int32_t *>(key_out.p),
                                                    static_cast<int32_t *>(id.p), static_cast<int32_t *>(id_out.p),
                                                    static_cast<int32_t>(p->M), 0, bits, st));
        if ((s = tmp3.get(tb3, "sort scratch"))) return s;
        SD_CUDA_TRY(cub::DeviceRadixSort::SortPairs(tmp3.p, tb3, static_cast<int32_t *>(key.p), static_cast<int32_t *>(key_out.p),
                                                    static_cast<int32_t *>(id.p), static_cast<int32_t *>(id_out.p),
                                                    static_cast<int32_t>(p->M), 0, bits, st));
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->h_light), sizeof(int32_t) * (p->M - nl), "light rows"))) return s;
        SD_CUDA_TRY(cudaMemcpyAsync(p->h_light, static_cast<int32_t *>(id_out.p) + nl, sizeof(int32_t) * (p->M - nl),
                                    cudaMemcpyDeviceToDevice, st));
        // sorted keys: 0 for the heavy rows, then T - length ascending; lengths of at least kHybridMedium have keys up to T - kHybridMedium
        int64_t upto = nl;
        if (T > kHybridMedium) {
            count_not_above_kernel<<<1, 1, 0, st>>>(static_cast<int32_t *>(key_out.p), p->M, T - kHybridMedium,
                                                    static_cast<int64_t *>(nsel.p));
            SD_CUDA_TRY(cudaGetLastError());
            SD_CUDA_TRY(cudaMemcpyAsync(&upto, nsel.p, sizeof upto, cudaMemcpyDeviceToHost, st));
        }
        SD_CUDA_TRY(cudaStreamSynchronize(st));
        p->h_nm = upto - nl;
        if ((s = build_light_desc(p, st))) return s;
    }
    p->num_chunks = p->h_nc;
    p->info.num_segments = p->h_nc;
    p->info.num_tiles = p->h_nl;
    p->info.heavy_len = T;
    return SD_OK;
}

template <typename T>
static cudaError_t fill_bsr(sd_plan *p, cudaStream_t st) {
    bsr_fill_kernel<T><<<148 * 8, 256, 0, st>>>(p->rowptr, p->colind, static_cast<const T *>(p->vals), p->M,
                                                p->browptr, p->bcol, static_cast<T *>(p->bval));
    return cudaGetLastError();
}

static sd_status_t build_bsr(sd_plan *p, const unsigned long long *ukeys, int64_t nnzb, cudaStream_t st) {
    const int64_t Mb = (p->M + 15) / 16, Kb = (p->K + 15) / 16;
    const size_t es = p->dtype == SD_F32 ? 4 : 2;
    p->nnzb = nnzb;
    sd_status_t s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->browptr), sizeof(int32_t) * (Mb + 1), "browptr"))) return s;
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->bcol), sizeof(int32_t) * nnzb, "bcol"))) return s;
    if ((s = dev_alloc(p, &p->bval, es * 256 * nnzb, "bval"))) return s;
    SD_CUDA_TRY(cudaMemsetAsync(p->bval, 0, es * 256 * nnzb, st));
    bsr_browptr_kernel<<<ceil_div(Mb + 1, 256), 256, 0, st>>>(ukeys, nnzb, Kb, static_cast<int32_t>(Mb), p->browptr);
    SD_CUDA_TRY(cudaGetLastError());
    bsr_bcol_kernel<<<ceil_div(nnzb, 256), 256, 0, st>>>(ukeys, nnzb, Kb, p->bcol);
    SD_CUDA_TRY(cudaGetLastError());
    SD_CUDA_TRY(p->dtype == SD_F32 ? fill_bsr<float>(p, st) : fill_bsr<__nv_bfloat16>(p, st));
    // tensor-core operand images: bf16 512 bytes per block, fp32 a hi and a lo image of 1 KB each
    if ((s = dev_alloc(p, &p->bval_mma, (p->dtype == SD_BF16 ? 512 : 2048) * static_cast<size_t>(nnzb),
                       "bval (tensor-core image)")))
        return s;
    SD_CUDA_TRY(build_bsr_mma_image(p->bval, p->bval_mma, nnzb, p->dtype, st));
    // one persistent CTA per SM, each with a contiguous range of block-rows of about equal cost
    p->bsr_nparts = static_cast<int32_t>(Mb < p->info.sm_count ? Mb : p->info.sm_count);
    if (p->bsr_nparts > 0) {
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->bsr_part), sizeof(int32_t) * (p->bsr_nparts + 1), "block-row partition")))
            return s;
        SD_CUDA_TRY(build_bsr_partition(p->browptr, static_cast<int32_t>(Mb), p->bsr_nparts, p->bsr_part, st));
    }
    if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->dev_error), sizeof(int32_t), "error word"))) return s;
    SD_CUDA_TRY(cudaMemsetAsync(p->dev_error, 0, sizeof(int32_t), st));
    SD_CUDA_TRY(cudaStreamSynchronize(st));
    return SD_OK;
}

static sd_status_t create_plan(const sd_plan_desc_t *d, sd_plan *p) {
    cudaStream_t st = static_cast<cudaStream_t>(d->stream);
    p->rowptr = d->rowptr;
    p->colind = d->colind;
    p->vals = d->vals;
    p->M = d->M;
    p->K = d->K;
    p->N = d->N;
    p->dtype = d->dtype;
    p->test_wait_expiry = d->test_wait_expiry;
    SD_CUDA_TRY(cudaGetDevice(&p->device));
    cudaDeviceProp prop;
    SD_CUDA_TRY(cudaGetDeviceProperties(&prop, p->device));
    sd_plan_info_t &info = p->info;
    memset(&info, 0, sizeof info);
    info.M = p->M;
    info.K = p->K;
    info.N = p->N;
    info.dtype = p->dtype;
    info.sm_count = prop.multiProcessorCount;
    info.l2_bytes = prop.l2CacheSize;
    info.windows = 1;

    if (p->M > 0) {
        int32_t last = 0;
        SD_CUDA_TRY(cudaMemcpyAsync(&last, p->rowptr + p->M, sizeof last, cudaMemcpyDeviceToHost, st));
        SD_CUDA_TRY(cudaStreamSynchronize(st));
        if (last < 0) {
            set_error(SD_ERR_INVALID_ARG, "rowptr[M] = %d is negative", last);
            return SD_ERR_INVALID_ARG;
        }
        p->nnz = last;
    }
    info.nnz = p->nnz;
    if (p->nnz > 0 && (!p->colind || !p->vals)) {
        set_error(SD_ERR_INVALID_ARG, "colind / vals are null but rowptr[M] = %lld", (long long)p->nnz);
        return SD_ERR_INVALID_ARG;
    }

    sd_status_t s;
    TempBuf accum;
    if ((s = accum.get(sizeof(ScanAccum), "scan accumulators"))) return s;
    ScanAccum *dacc = static_cast<ScanAccum *>(accum.p);
    SD_CUDA_TRY(cudaMemsetAsync(dacc, 0, sizeof(ScanAccum), st));

    if (d->validate && p->M > 0) {
        validate_kernel<<<148 * 8, 256, 0, st>>>(p->rowptr, p->colind, p->M, p->K, p->nnz, dacc);
        SD_CUDA_TRY(cudaGetLastError());
        ScanAccum h;
        SD_CUDA_TRY(cudaMemcpyAsync(&h, dacc, sizeof h, cudaMemcpyDeviceToHost, st));
        SD_CUDA_TRY(cudaStreamSynchronize(st));
        if (h.bad_csr) {
            set_error(SD_ERR_INVALID_ARG, "malformed CSR: %llu offending rowptr / colind entries", h.bad_csr);
            return SD_ERR_INVALID_ARG;
        }
    }

    // ---- scan: row statistics + 16x16 block keys -> sort -> run-length encode ----------------
    const int64_t Kb = (p->K + 15) / 16, Mb = (p->M + 15) / 16;
    TempBuf keys_a, keys_b, counts, nruns, cubtmp;
    int64_t nnzb = 0;
    if (p->M > 0) {
        if (p->nnz > 0) {
            if ((s = keys_a.get(sizeof(unsigned long long) * p->nnz, "block keys"))) return s;
            if ((s = keys_b.get(sizeof(unsigned long long) * p->nnz, "sorted block keys"))) return s;
        }
        const int blocks = static_cast<int>(std::min<int64_t>((p->M + 7) / 8, 148 * 16));
        scan_rows_kernel<<<blocks, 256, 0, st>>>(p->rowptr, p->colind, p->M, Kb,
                                                static_cast<unsigned long long *>(keys_a.p), dacc);
        SD_CUDA_TRY(cudaGetLastError());
    }
    if (p->nnz > 0) {
        int bits = 1;
        while (bits < 64 && (static_cast<unsigned __int128>(1) << bits) < static_cast<unsigned __int128>(Mb) * Kb) ++bits;
        auto *ka = static_cast<unsigned long long *>(keys_a.p);
        auto *kb = static_cast<unsigned long long *>(keys_b.p);
        size_t tb = 0;
        SD_CUDA_TRY(cub::DeviceRadixSort::SortKeys(nullptr, tb, ka, kb, p->nnz, 0, bits, st));
        if ((s = cubtmp.get(tb, "sort scratch"))) return s;
        SD_CUDA_TRY(cub::DeviceRadixSort::SortKeys(cubtmp.p, tb, ka, kb, p->nnz, 0, bits, st));
        if ((s = counts.get(sizeof(int32_t) * p->nnz, "block fill counts"))) return s;
        if ((s = nruns.get(sizeof(int64_t), "block count"))) return s;
        size_t tb2 = 0;
        SD_CUDA_TRY(cub::DeviceRunLengthEncode::Encode(nullptr, tb2, kb, ka, static_cast<int32_t *>(counts.p),
                                                       static_cast<int64_t *>(nruns.p), p->nnz, st));
        if (tb2 > tb) {
            cudaFree(cubtmp.p);
            cubtmp.p = nullptr;
            if ((s = cubtmp.get(tb2, "rle scratch"))) return s;
        }
        // distinct keys land in keys_a (its contents are no longer needed)
        SD_CUDA_TRY(cub::DeviceRunLengthEncode::Encode(cubtmp.p, tb2, kb, ka, static_cast<int32_t *>(counts.p),
                                                       static_cast<int64_t *>(nruns.p), p->nnz, st));
        SD_CUDA_TRY(cudaMemcpyAsync(&nnzb, nruns.p, sizeof nnzb, cudaMemcpyDeviceToHost, st));
        SD_CUDA_TRY(cudaStreamSynchronize(st));
        block_fill_kernel<<<static_cast<int>(std::min<int64_t>((nnzb + 255) / 256, 148 * 8)), 256, 0, st>>>(
            static_cast<int32_t *>(counts.p), nnzb, dacc);
        SD_CUDA_TRY(cudaGetLastError());
    }
    ScanAccum h;
    SD_CUDA_TRY(cudaMemcpyAsync(&h, dacc, sizeof h, cudaMemcpyDeviceToHost, st));
    SD_CUDA_TRY(cudaStreamSynchronize(st));
    for (int i = 0; i < 32; ++i) info.row_hist[i] = static_cast<int64_t>(h.row_hist[i]);
    info.sum_r2 = h.sum_r2;
    info.max_r = static_cast<int64_t>(h.max_r);
    info.empty_rows = static_cast<int64_t>(h.empty_rows);
    info.sum_span = h.sum_span;
    info.max_span = static_cast<int64_t>(h.max_span);
    info.sum_gap = h.sum_gap;
    info.diag = static_cast<int64_t>(h.diag);
    info.unsorted_rows = static_cast<int64_t>(h.unsorted_rows);
    info.long_rows = static_cast<int64_t>(h.long_rows);
    info.nnz_long_rows = static_cast<int64_t>(h.nnz_long_rows);
    info.nnzb16 = nnzb;
    for (int i = 0; i < 9; ++i) info.blk_hist[i] = static_cast<int64_t>(h.blk_hist[i]);
    info.nnz_dense_blocks = static_cast<int64_t>(h.nnz_dense_blocks);

    // ---- decision ------------------------------------------------------------------------------
    int family = d->family == SD_AUTO ? decide_family(info, p->dtype) : d->family;
    if (d->family == SD_AUTO && family == SD_MERGE && d->windows == 0 && p->M > 0 && p->nnz > 0 &&
        decide_hybrid(info, p->dtype, decide_windows(info, p->dtype)))
        family = SD_HYBRID;
    if (family == SD_HYBRID && info.unsorted_rows != 0) {   // the chunks of a window are ranges of the rows only if columns ascend
        if (d->family == SD_HYBRID) {
            set_error(SD_ERR_UNSUPPORTED, "the hybrid family needs ascending columns in every row (%lld rows are not)",
                      (long long)info.unsorted_rows);
            return SD_ERR_UNSUPPORTED;
        }
        family = SD_MERGE;
    }
    if (family == SD_BSR_TC && (info.unsorted_rows != 0 || p->nnz == 0)) {
        if (d->family == SD_BSR_TC && info.unsorted_rows != 0) {
            set_error(SD_ERR_UNSUPPORTED, "BSR needs strictly ascending columns in every row (%lld rows are not)",
                      (long long)info.unsorted_rows);
            return SD_ERR_UNSUPPORTED;
        }
        family = SD_ROWSPLIT;
    }
    info.family = family;

    // ---- representation -----------------------------------------------------------------------
    info.launches = 1;
    if (family == SD_MERGE && p->M > 0 && p->nnz > 0) {
        int W = d->windows == 0 ? decide_windows(info, p->dtype) : d->windows;
        bool split = W > 1 || W == -1 || (d->windows == 0 && decide_class_split(info, p->dtype));
        if (W < 1) W = 1;
        if (info.unsorted_rows != 0) {   // windows and the class split need ascending columns
            W = 1;
            split = false;
        }
        if ((s = build_merge(p, W, split, st))) return s;
    } else if (family == SD_BSR_TC) {
        if ((s = build_bsr(p, static_cast<unsigned long long *>(keys_a.p), nnzb, st))) return s;
    } else if (family == SD_HYBRID && p->M > 0 && p->nnz > 0) {
        int W = d->windows == 0 ? decide_windows(info, p->dtype) : d->windows;
        const int32_t T = d->heavy_len > 0 ? d->heavy_len : kHybridHeavy;
        if ((s = build_hybrid(p, W, T, st))) return s;
    }
    info.plan_bytes = p->owned;
    return SD_OK;
}

static void free_plan(sd_plan *p) {
    if (!p) return;
    cudaFree(p->w_ptr);
    cudaFree(p->w_col);
    cudaFree(p->w_vals);
    cudaFree(p->w_src);
    cudaFree(p->w_seg_row);
    cudaFree(p->seg_chunk);
    cudaFree(p->chunk_ptr);
    cudaFree(p->chunk_out);
    cudaFree(p->tile_seg);
    cudaFree(p->fix_short);
    cudaFree(p->fix_long);
    cudaFree(p->tile_head);
    cudaFree(p->tile_tail);
    cudaFree(p->h_rows);
    cudaFree(p->h_chunk_ptr);
    cudaFree(p->h_ranges);
    cudaFree(p->h_order);
    cudaFree(p->h_light);
    cudaFree(p->h_desc);
    cudaFree(p->h_giant);
    cudaFree(p->coo_row);
    cudaFree(p->coo_c1_row);
    cudaFree(p->coo_c1_val);
    cudaFree(p->coo_c2_row);
    cudaFree(p->coo_c2_val);
    cudaFree(p->browptr);
    cudaFree(p->bcol);
    cudaFree(p->bval);
    cudaFree(p->bval_mma);
    cudaFree(p->bsr_part);
    cudaFree(p->dev_error);
    cudaFree(p->stage_B);
    cudaFree(p->stage_C);
    if (p->host_stream) cudaStreamDestroy(p->host_stream);
    for (int i = 0; i < 2; ++i) {
        if (p->aux[i]) cudaStreamDestroy(p->aux[i]);
        if (p->ev_join[i]) cudaEventDestroy(p->ev_join[i]);
    }
    if (p->ev_fork) cudaEventDestroy(p->ev_fork);
    if (p->chunk_stream) cudaStreamDestroy(p->chunk_stream);
    for (cudaEvent_t e : p->ev_chunk)
        if (e) cudaEventDestroy(e);
    delete p;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- plan serialisation ---------------------------------------------------------------------------
// Position-dependent 64-bit hash of an int32 array: the sum over i of mix(i, x[i]) (a sum, so the order in which
// the threads add does not matter and the value is the same on every run and every grid size).
__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__global__ void __launch_bounds__(256)
hash_array_kernel(const int32_t *__restrict__ x, int64_t n, unsigned long long salt, unsigned long long *__restrict__ out) {
    unsigned long long h = 0;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x)
        h += mix64((static_cast<unsigned long long>(i) + 1) * 0x9E3779B97F4A7C15ull ^
                   (static_cast<unsigned long long>(static_cast<uint32_t>(x[i])) + salt));
    for (int off = 16; off > 0; off >>= 1) h += __shfl_xor_sync(0xffffffffu, h, off);
    if ((threadIdx.x & 31) == 0 && h) atomicAdd(out, h);
}

// Hash of the sparsity pattern (rowptr and colind; the values are not part of it).
static sd_status_t pattern_hash(const int32_t *rowptr, const int32_t *colind, int64_t M, int64_t nnz, cudaStream_t st,
                                uint64_t *out) {
    TempBuf acc;
    sd_status_t s;
    if ((s = acc.get(sizeof(unsigned long long), "pattern hash"))) return s;
    SD_CUDA_TRY(cudaMemsetAsync(acc.p, 0, sizeof(unsigned long long), st));
    auto *d = static_cast<unsigned long long *>(acc.p);
    if (M >= 0 && rowptr) {
        hash_array_kernel<<<static_cast<unsigned>(std::min<int64_t>((M + 256) / 256, 148 * 8)), 256, 0, st>>>(rowptr, M + 1, 0x51ull, d);
        SD_CUDA_TRY(cudaGetLastError());
    }
    if (nnz > 0) {
        hash_array_kernel<<<static_cast<unsigned>(std::min<int64_t>((nnz + 255) / 256, 148 * 8)), 256, 0, st>>>(colind, nnz, 0xC0ull, d);
        SD_CUDA_TRY(cudaGetLastError());
    }
    unsigned long long h = 0;
    SD_CUDA_TRY(cudaMemcpyAsync(&h, d, sizeof h, cudaMemcpyDeviceToHost, st));
    SD_CUDA_TRY(cudaStreamSynchronize(st));
    *out = h;
    return SD_OK;
}

constexpr uint64_t kBlobMagic = 0x31304E414C504453ull;   // "SDPLAN01"
constexpr uint32_t kBlobVersion = 2;
constexpr int kBlobArrays = 19;

struct BlobHeader {
    uint64_t magic;
    uint32_t version, header_bytes;
    uint64_t pattern;           // pattern_hash of (rowptr, colind)
    int64_t M, K, N, nnz;
    int32_t dtype, family;
    char device_name[128];      // the plan was tuned on this GPU model (grid sizes, window count, thresholds)
    int32_t sm_count, nwins;
    int64_t l2_bytes;
    sd_plan_info_t info;
    int64_t num_segments, num_chunks, ntiles, nnzb;
    int32_t bsr_nparts, has_coo;
    int64_t h_nl, h_nc, h_ng, h_nm;
    int32_t h_T, reserved;
    uint64_t array_bytes[kBlobArrays];   // payload sizes, in the order of blob_arrays(); each padded to 16 bytes in the blob
};

struct BlobArray {
    void **field;
    size_t bytes;
    const char *what;
};

static size_t pad16(size_t b) { return (b + 15) & ~static_cast<size_t>(15); }

// The structure-only device arrays of a plan, in blob order.  Value copies (re-bucketed values, 16x16 blocks and their
// tensor-core images) and scratch are not part of the blob: they are rebuilt from the caller's values at load time.
static void blob_arrays(sd_plan *p, BlobArray (&arr)[kBlobArrays]) {
    const int64_t S = p->num_segments, nnz = p->nnz, W = static_cast<int64_t>(p->wins.size());
    const bool merge = p->info.family == SD_MERGE && !p->wins.empty();
    const bool split = merge && p->info.class_split;
    const bool bsr = p->info.family == SD_BSR_TC;
    const int64_t Mb = (p->M + 15) / 16;
    auto set = [&](int i, void *field, size_t bytes, const char *what) { arr[i] = {static_cast<void **>(field), bytes, what}; };
    set(0, &p->w_ptr, split ? 4 * (S + 1) : 0, "segment pointers");
    set(1, &p->w_col, split ? 4 * nnz : 0, "window-major colind");
    set(2, &p->w_src, split ? 4 * nnz : 0, "window-major source positions");
    set(3, &p->w_seg_row, split ? 4 * (S + 1) : 0, "segment rows");
    set(4, &p->seg_chunk, split ? 4 * (S + 1) : 0, "segment chunks");
    set(5, &p->chunk_ptr, split ? 4 * (p->num_chunks + W + 1) : 0, "chunk boundaries");
    set(6, &p->tile_seg, merge ? 4 * (p->ntiles + W) : 0, "tile table");
    set(7, &p->fix_short, merge ? 4 * (p->ntiles + 1) : 0, "fix-up list");
    set(8, &p->fix_long, merge ? 4 * (p->ntiles + 1) : 0, "fix-up list");
    set(9, &p->coo_row, (merge && p->coo_row) ? 4 * nnz : 0, "row index per nonzero");
    set(10, &p->browptr, bsr ? 4 * (Mb + 1) : 0, "browptr");
    set(11, &p->bcol, bsr ? 4 * p->nnzb : 0, "bcol");
    set(12, &p->bsr_part, (bsr && p->bsr_nparts > 0) ? 4 * (static_cast<int64_t>(p->bsr_nparts) + 1) : 0, "block-row partition");
    const bool hyb = p->info.family == SD_HYBRID && p->h_T > 0;
    const bool heavy = hyb && p->h_nl > 0;
    set(13, &p->h_rows, heavy ? 4 * p->h_nl : 0, "heavy rows");
    set(14, &p->h_chunk_ptr, heavy ? 4 * (p->h_nl + 1) : 0, "chunk pointers");
    set(15, &p->h_ranges, heavy ? 8 * p->h_nc : 0, "chunk ranges");
    set(16, &p->h_order, heavy ? 4 * p->h_nc : 0, "chunk order");
    set(17, &p->h_giant, (heavy && p->h_ng > 0) ? 4 * p->h_ng : 0, "giant rows");
    set(18, &p->h_light, (hyb && p->h_nl < p->M) ? 4 * (p->M - p->h_nl) : 0, "light rows");
}

static sd_status_t create_split_streams(sd_plan *p, int W) {
    SD_CUDA_TRY(preload_stream_kernels(p->dtype, static_cast<int32_t>(p->N)));   // before the streams exist
    for (int i = 0; i < 2; ++i) {
        SD_CUDA_TRY(cudaStreamCreateWithFlags(&p->aux[i], cudaStreamNonBlocking));
        SD_CUDA_TRY(cudaEventCreateWithFlags(&p->ev_join[i], cudaEventDisableTiming));
    }
    SD_CUDA_TRY(cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming));
    SD_CUDA_TRY(cudaStreamCreateWithFlags(&p->chunk_stream, cudaStreamNonBlocking));
    p->ev_chunk.assign(W, nullptr);
    for (int w = 0; w < W; ++w) SD_CUDA_TRY(cudaEventCreateWithFlags(&p->ev_chunk[w], cudaEventDisableTiming));
    return SD_OK;
}

}  // namespace sd

// =====================================================================================
// extern "C"
// =====================================================================================
using namespace sd;

extern "C" {
#pragma GCC visibility push(default)

const char *sd_version(void) { return "0.1"; }

int sd_last_error(char *buf, size_t n) {
    if (buf && n) {
        strncpy(buf, g_err_text, n - 1);
        buf[n - 1] = '\0';
    }
    return g_err_code;
}

sd_status_t sd_plan_create_ex(const sd_plan_desc_t *d, sd_plan_t **out) {
    if (out) *out = nullptr;
    if (!d || !out) {
        set_error(SD_ERR_INVALID_ARG, "desc and out must not be null");
        return SD_ERR_INVALID_ARG;
    }
    if (d->M < 0 || d->K < 0 || d->N < 0 || d->M > INT32_MAX - 1 || d->K > INT32_MAX - 1 || d->N > INT32_MAX / 2) {
        set_error(SD_ERR_INVALID_ARG, "M, K, N must be in [0, 2^31)");
        return SD_ERR_INVALID_ARG;
    }
    if (d->M > 0 && !d->rowptr) {
        set_error(SD_ERR_INVALID_ARG, "rowptr is null");
        return SD_ERR_INVALID_ARG;
    }
    if (d->dtype != SD_F32 && d->dtype != SD_BF16) {
        set_error(SD_ERR_INVALID_ARG, "unknown dtype %d", d->dtype);
        return SD_ERR_INVALID_ARG;
    }
    if (d->family < SD_AUTO || d->family > SD_HYBRID) {
        set_error(SD_ERR_INVALID_ARG, "unknown family %d", d->family);
        return SD_ERR_INVALID_ARG;
    }
    if (d->windows < -1 || d->windows > 64) {
        set_error(SD_ERR_INVALID_ARG, "windows must be in [-1, 64]");
        return SD_ERR_INVALID_ARG;
    }
    sd_plan *p = new (std::nothrow) sd_plan;
    if (!p) {
        set_error(SD_ERR_ALLOC, "host allocation failed");
        return SD_ERR_ALLOC;
    }
    const sd_status_t s = create_plan(d, p);
    if (s != SD_OK) {
        free_plan(p);
        return s;
    }
    *out = p;
    return SD_OK;
}

sd_plan_t *sd_plan_create(const int32_t *rowptr, const int32_t *colind, const float *vals, int64_t M, int64_t K,
                          int64_t N) {
    sd_plan_desc_t d;
    memset(&d, 0, sizeof d);
    d.rowptr = rowptr;
    d.colind = colind;
    d.vals = vals;
    d.M = M;
    d.K = K;
    d.N = N;
    d.dtype = SD_F32;
    d.family = SD_AUTO;
    sd_plan_t *p = nullptr;
    sd_plan_create_ex(&d, &p);
    return p;
}

void sd_plan_destroy(sd_plan_t *plan) { free_plan(plan); }

sd_status_t sd_plan_get_info(const sd_plan_t *plan, sd_plan_info_t *out) {
    if (!plan || !out) {
        set_error(SD_ERR_INVALID_ARG, "plan and out must not be null");
        return SD_ERR_INVALID_ARG;
    }
    *out = plan->info;
    return SD_OK;
}

// Row-length shape class on the integers of the summary (Sec. 3.1 names five classes and gives no
// cut-offs; the rule is stated beside sd_shape_t).  CV^2 = M sum r^2 / nnz^2 - 1.
static int shape_class_of(const sd_plan_info_t &s) {
    if (s.nnz <= 0 || s.M <= 0) return SD_SHAPE_UNIFORM;
    using u128 = unsigned __int128;
    const u128 m_r2 = static_cast<u128>(static_cast<uint64_t>(s.M)) * s.sum_r2;
    const u128 nnz2 = static_cast<u128>(static_cast<uint64_t>(s.nnz)) * static_cast<uint64_t>(s.nnz);
    if (16 * m_r2 <= 17 * nnz2) return SD_SHAPE_UNIFORM;
    const int64_t nonempty = s.M - s.empty_rows;
    int first = -1, last = -1;
    for (int b = 1; b < 32; ++b) {
        if (4 * s.row_hist[b] >= nonempty) {
            if (first < 0) first = b;
            last = b;
        }
    }
    if (first >= 0 && last - first >= 3) return SD_SHAPE_BIMODAL;
    if (m_r2 >= 5 * nnz2 && static_cast<u128>(static_cast<uint64_t>(s.max_r)) * static_cast<uint64_t>(s.M) >=
                                static_cast<u128>(64) * static_cast<uint64_t>(s.nnz))
        return SD_SHAPE_POWERLAW;
    if (m_r2 >= 2 * nnz2) return SD_SHAPE_SKEWED;
    return SD_SHAPE_MODERATE;
}

sd_status_t sd_plan_get_features(sd_plan_t *plan, sd_features_t *out) {
    if (!plan || !out) {
        set_error(SD_ERR_INVALID_ARG, "sd_plan_get_features: null argument");
        return SD_ERR_INVALID_ARG;
    }
    if (!plan->have_feat) {
        int prev = 0;
        SD_CUDA_TRY(cudaGetDevice(&prev));
        SD_CUDA_TRY(cudaSetDevice(plan->device));
        FeatureCounts fc;
        const sd_status_t s = compute_feature_counts(plan->rowptr, plan->colind, plan->M, plan->K, plan->nnz, nullptr, &fc);
        cudaSetDevice(prev);
        if (s) return s;
        const sd_plan_info_t &info = plan->info;
        sd_features_t f{};
        for (int k = 0; k < 3; ++k) {
            f.row_q[k] = fc.row_q[k];
            f.col_q[k] = fc.col_q[k];
            f.sell_slots[k] = fc.sell_slots[k];
        }
        f.col_max = fc.col_max;
        f.col_empty = fc.col_empty;
        f.sum_d2 = fc.sum_d2;
        f.ell_slots = info.M * info.max_r;
        f.nnzb[0] = fc.nnzb4;
        f.nnzb[1] = fc.nnzb8;
        f.nnzb[2] = info.nnzb16;
        const int64_t vb = plan->dtype == SD_BF16 ? 2 : 4;
        f.value_bytes = static_cast<int32_t>(vb);
        f.rep_bytes[0] = (vb + 4) * info.nnz + 4 * (info.M + 1);
        f.rep_bytes[1] = (vb + 4) * f.ell_slots;
        const int64_t heights[3] = {16, 32, 512};
        for (int k = 0; k < 3; ++k)
            f.rep_bytes[2 + k] = (vb + 4) * f.sell_slots[k] + 4 * ((info.M + heights[k] - 1) / heights[k] + 1);
        const int64_t bs[3] = {4, 8, 16};
        for (int k = 0; k < 3; ++k)
            f.rep_bytes[5 + k] = (vb * bs[k] * bs[k] + 4) * f.nnzb[k] + 4 * ((info.M + bs[k] - 1) / bs[k] + 1);
        f.shape_class = shape_class_of(info);
        const bool reads_csr = info.family == SD_ROWSPLIT || info.family == SD_HYBRID ||
                               (info.family == SD_MERGE && !info.class_split);
        f.borrowed_bytes = reads_csr ? f.rep_bytes[0] : 0;
        f.plan_bytes = info.plan_bytes;
        f.d_r = info.K * info.N * vb;
        f.d_s = 4 * info.M * info.N;
        f.m_r = f.borrowed_bytes + f.plan_bytes + f.d_r;
        f.m_t = f.m_r + f.d_s;
        f.work_units = info.family == SD_MERGE ? (info.class_split ? info.num_segments : info.num_tiles)
                     : info.family == SD_BSR_TC ? (info.M + 15) / 16
                     : info.family == SD_HYBRID ? info.num_segments + (info.M - info.num_tiles)
                                                : info.M;
        f.sm_count = info.sm_count;
        f.l2_bytes = info.l2_bytes;
        plan->feat = f;
        plan->have_feat = true;
    }
    *out = plan->feat;
    return SD_OK;
}

sd_status_t sd_plan_get_bsr(const sd_plan_t *plan, int32_t *browptr, int32_t *bcol, void *bval) {
    if (!plan) {
        set_error(SD_ERR_INVALID_ARG, "plan is null");
        return SD_ERR_INVALID_ARG;
    }
    if (plan->info.family != SD_BSR_TC) {
        set_error(SD_ERR_UNSUPPORTED, "the plan holds no BSR representation");
        return SD_ERR_UNSUPPORTED;
    }
    const int64_t Mb = (plan->M + 15) / 16;
    const size_t es = plan->dtype == SD_F32 ? 4 : 2;
    if (browptr) SD_CUDA_TRY(cudaMemcpy(browptr, plan->browptr, sizeof(int32_t) * (Mb + 1), cudaMemcpyDeviceToHost));
    if (bcol && plan->nnzb)
        SD_CUDA_TRY(cudaMemcpy(bcol, plan->bcol, sizeof(int32_t) * plan->nnzb, cudaMemcpyDeviceToHost));
    if (bval && plan->nnzb) SD_CUDA_TRY(cudaMemcpy(bval, plan->bval, es * 256 * plan->nnzb, cudaMemcpyDeviceToHost));
    return SD_OK;
}

sd_status_t sd_plan_get_hybrid(const sd_plan_t *plan, int32_t *heavy_rows, int32_t *chunk_ptr, int32_t *ranges,
                               int32_t *order, int32_t *light_rows) {
    if (!plan) {
        set_error(SD_ERR_INVALID_ARG, "plan is null");
        return SD_ERR_INVALID_ARG;
    }
    if (plan->info.family != SD_HYBRID) {
        set_error(SD_ERR_UNSUPPORTED, "the plan's family is not SD_HYBRID");
        return SD_ERR_UNSUPPORTED;
    }
    const int64_t nl = plan->h_nl, nc = plan->h_nc, nlight = plan->h_T > 0 ? plan->M - nl : 0;
    if (heavy_rows && nl > 0) SD_CUDA_TRY(cudaMemcpy(heavy_rows, plan->h_rows, 4 * nl, cudaMemcpyDeviceToHost));
    if (chunk_ptr) {
        if (nl > 0) SD_CUDA_TRY(cudaMemcpy(chunk_ptr, plan->h_chunk_ptr, 4 * (nl + 1), cudaMemcpyDeviceToHost));
        else chunk_ptr[0] = 0;
    }
    if (ranges && nc > 0) SD_CUDA_TRY(cudaMemcpy(ranges, plan->h_ranges, 8 * nc, cudaMemcpyDeviceToHost));
    if (order && nc > 0) SD_CUDA_TRY(cudaMemcpy(order, plan->h_order, 4 * nc, cudaMemcpyDeviceToHost));
    if (light_rows && nlight > 0) SD_CUDA_TRY(cudaMemcpy(light_rows, plan->h_light, 4 * nlight, cudaMemcpyDeviceToHost));
    return SD_OK;
}

sd_status_t sd_plan_device_status(sd_plan_t *plan, int32_t *status) {
    if (!plan || !status) {
        set_error(SD_ERR_INVALID_ARG, "plan and status must not be null");
        return SD_ERR_INVALID_ARG;
    }
    *status = 0;
    SD_CUDA_TRY(cudaDeviceSynchronize());
    if (plan->dev_error) {
        SD_CUDA_TRY(cudaMemcpy(status, plan->dev_error, sizeof(int32_t), cudaMemcpyDeviceToHost));
        if (*status) SD_CUDA_TRY(cudaMemset(plan->dev_error, 0, sizeof(int32_t)));
    }
    return SD_OK;
}

sd_status_t sd_plan_get_tiles(const sd_plan_t *plan, int32_t *tile_seg, int64_t cap, int64_t *count) {
    if (!plan || !count) {
        set_error(SD_ERR_INVALID_ARG, "plan and count must not be null");
        return SD_ERR_INVALID_ARG;
    }
    if (plan->info.family != SD_MERGE) {
        set_error(SD_ERR_UNSUPPORTED, "the plan holds no merge-path tile table");
        return SD_ERR_UNSUPPORTED;
    }
    const int64_t n = plan->wins.empty() ? 0 : plan->ntiles + static_cast<int64_t>(plan->wins.size());
    *count = n;
    if (tile_seg && cap >= n && n > 0)
        SD_CUDA_TRY(cudaMemcpy(tile_seg, plan->tile_seg, sizeof(int32_t) * n, cudaMemcpyDeviceToHost));
    return SD_OK;
}

sd_status_t sd_plan_get_segments(const sd_plan_t *plan, int32_t *seg_ptr, int32_t *seg_row, int32_t *colind,
                                 void *vals, int64_t *win_seg) {
    if (!plan) {
        set_error(SD_ERR_INVALID_ARG, "plan is null");
        return SD_ERR_INVALID_ARG;
    }
    if (plan->info.family != SD_MERGE || !plan->info.class_split) {
        set_error(SD_ERR_UNSUPPORTED, "the plan holds no window-major segment list");
        return SD_ERR_UNSUPPORTED;
    }
    const int64_t S = plan->num_segments;
    const size_t es = plan->dtype == SD_F32 ? 4 : 2;
    if (seg_ptr) SD_CUDA_TRY(cudaMemcpy(seg_ptr, plan->w_ptr, 4 * (S + 1), cudaMemcpyDeviceToHost));
    if (seg_row) SD_CUDA_TRY(cudaMemcpy(seg_row, plan->w_seg_row, 4 * S, cudaMemcpyDeviceToHost));
    if (colind) SD_CUDA_TRY(cudaMemcpy(colind, plan->w_col, 4 * plan->nnz, cudaMemcpyDeviceToHost));
    if (vals) SD_CUDA_TRY(cudaMemcpy(vals, plan->w_vals, es * plan->nnz, cudaMemcpyDeviceToHost));
    if (win_seg) {
        for (size_t w = 0; w < plan->wins.size(); ++w) {
            win_seg[3 * w] = plan->wins[w].seg_begin;
            win_seg[3 * w + 1] = plan->wins[w].short_begin;
            win_seg[3 * w + 2] = plan->wins[w].single_begin;
        }
        win_seg[3 * plan->wins.size()] = S;
    }
    return SD_OK;
}

sd_status_t sd_spmm(const sd_plan_t *plan, const void *B, int64_t ldb, float *C, int64_t ldc, float alpha, float beta,
                    void *stream) {
    if (!plan) {
        set_error(SD_ERR_INVALID_ARG, "plan is null");
        return SD_ERR_INVALID_ARG;
    }
    const int64_t M = plan->M, N = plan->N;
    if (M == 0 || N == 0) return SD_OK;
    if (!C || ldc < N) {
        set_error(SD_ERR_INVALID_ARG, "C is null or ldc < N");
        return SD_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (alpha == 0.f || plan->nnz == 0) {
        SD_CUDA_TRY(run_scale_c(C, ldc, M, static_cast<int32_t>(N), beta, st));
        return SD_OK;
    }
    if (!B || ldb < N) {
        set_error(SD_ERR_INVALID_ARG, "B is null or ldb < N");
        return SD_ERR_INVALID_ARG;
    }
    if (ldb * (plan->dtype == SD_F32 ? 4 : 2) > static_cast<int64_t>(UINT32_MAX)) {
        set_error(SD_ERR_UNSUPPORTED, "row pitch of B must be below 4 GiB");
        return SD_ERR_UNSUPPORTED;
    }
    const int vw = plan->dtype == SD_F32 ? 4 : 8;
    const bool vec = aligned16(B) && aligned16(C) && N % vw == 0 && ldb % vw == 0 && ldc % 4 == 0;

    SpmmArgs a;
    a.ptr = plan->rowptr;
    a.colind = plan->colind;
    a.vals = plan->vals;
    a.seg_row = nullptr;
    a.B = B;
    a.C = C;
    a.ldb = ldb;
    a.ldc = ldc;
    a.ldb_bytes = static_cast<uint32_t>(ldb * (plan->dtype == SD_F32 ? 4 : 2));
    a.S = M;
    a.max_len = plan->info.max_r;
    a.mean_len = M > 0 ? (plan->nnz + M - 1) / M : 0;
    a.N = static_cast<int32_t>(N);
    a.alpha = alpha;
    a.beta = beta;

    switch (plan->info.family) {
    case SD_ROWSPLIT:
        SD_CUDA_TRY(run_rowsplit(a, plan->dtype, vec, st));
        return SD_OK;
    case SD_MERGE: {
        if (plan->coo_row) {   // narrow dense operand: one writer per row
            a.colind = plan->colind;
            a.vals = plan->vals;
            CooPlan cp;
            cp.row = plan->coo_row;
            cp.rowptr = plan->rowptr;
            cp.M = plan->info.empty_rows > 0 ? M : 0;   // no search for rows without nonzeros when the scan found none
            cp.nnz = plan->nnz;
            cp.c1_row = plan->coo_c1_row;
            cp.c1_val = plan->coo_c1_val;
            cp.c2_row = plan->coo_c2_row;
            cp.c2_val = plan->coo_c2_val;
            const bool bvec = aligned16(B) && (ldb * (plan->dtype == SD_F32 ? 4 : 2)) % 16 == 0;
            SD_CUDA_TRY(run_coo(cp, a, plan->dtype, bvec, plan->info.sm_count, st));
            return SD_OK;
        }
        a.ptr = plan->m_ptr;
        a.colind = plan->m_col;
        a.vals = plan->m_vals;
        a.seg_row = plan->m_seg_row;
        a.S = plan->num_segments;
        const bool side = plan->aux[0] && !switches().no_side_streams;
        // The chunk kernels only read A and B and write their own scratch rows: they run on a stream of
        // their own, up to `depth` windows ahead of the kernels that update C, which wait for their
        // window's event.
        const bool ahead = side && plan->chunk_stream && !switches().no_chunk_ahead;
        auto launch_chunks = [&](size_t w, cudaStream_t cs) -> sd_status_t {
            const sd_plan::Window &win = plan->wins[w];
            SpmmArgs ca = a;
            ca.ptr = plan->chunk_ptr + win.chunk_begin + w;
            ca.seg_row = nullptr;
            ca.S = win.chunk_end - win.chunk_begin;
            ca.C = plan->chunk_out + win.chunk_begin * N;
            ca.ldc = N;
            ca.alpha = 1.f;
            ca.beta = 0.f;
            SD_CUDA_TRY(run_segments(ca, plan->dtype, vec, true, cs));
            return SD_OK;
        };
        const size_t depth = 2;   // windows the chunk stream may be ahead (measured: 2 is as good as all of them, and keeps
                                  // fewer slabs of B competing for L2)
        size_t chunks_issued = 0;
        auto issue_chunks_upto = [&](size_t upto) -> sd_status_t {   // windows [chunks_issued, upto)
            for (; chunks_issued < upto && chunks_issued < plan->wins.size(); ++chunks_issued) {
                const size_t w = chunks_issued;
                if (plan->wins[w].chunk_end > plan->wins[w].chunk_begin) {
                    sd_status_t cs = launch_chunks(w, plan->chunk_stream);
                    if (cs) return cs;
                }
                SD_CUDA_TRY(cudaEventRecord(plan->ev_chunk[w], plan->chunk_stream));
            }
            return SD_OK;
        };
        if (ahead) {
            SD_CUDA_TRY(cudaEventRecord(plan->ev_fork, st));
            SD_CUDA_TRY(cudaStreamWaitEvent(plan->chunk_stream, plan->ev_fork, 0));
            sd_status_t cs = issue_chunks_upto(depth);
            if (cs) return cs;
        }
        for (size_t w = 0; w < plan->wins.size(); ++w) {   // windows run in order
            const sd_plan::Window &win = plan->wins[w];
            // Inside a window every row belongs to one segment, so the three classes touch disjoint
            // rows of C and may run side by side: short and one-nonzero segments go to two plan-owned
            // streams forked from the caller's stream and joined before the next window.
            const bool has_short = win.short_end > win.short_begin, has_single = win.single_end > win.single_begin;
            cudaStream_t s_short = st, s_single = st;
            if (side && (has_short || has_single)) {
                SD_CUDA_TRY(cudaEventRecord(plan->ev_fork, st));
                if (has_short) {
                    s_short = plan->aux[0];
                    SD_CUDA_TRY(cudaStreamWaitEvent(s_short, plan->ev_fork, 0));
                }
                if (has_single) {
                    s_single = plan->aux[1];
                    SD_CUDA_TRY(cudaStreamWaitEvent(s_single, plan->ev_fork, 0));
                }
            }
            if (win.chunk_end > win.chunk_begin) {
                // long segments: every chunk is summed by one lane group into its own scratch row,
                // then each segment adds its chunks in order and updates its row of C
                if (ahead) {
                    SD_CUDA_TRY(cudaStreamWaitEvent(st, plan->ev_chunk[w], 0));
                } else {
                    sd_status_t cs = launch_chunks(w, st);
                    if (cs) return cs;
                }
                SD_CUDA_TRY(run_chunk_reduce(plan->chunk_out, plan->seg_chunk, a.seg_row, win.seg_begin, win.seg_end, C,
                                             ldc, static_cast<int32_t>(N), alpha, beta, st));
            }
            if (has_short) {   // short segments: one lane group per segment
                SpmmArgs sa = a;
                sa.ptr = a.ptr + win.short_begin;
                sa.seg_row = a.seg_row + win.short_begin;
                sa.S = win.short_end - win.short_begin;
                SD_CUDA_TRY(run_segments(sa, plan->dtype, vec, false, s_short));
            }
            if (has_single) {   // one-nonzero segments: flat
                SpmmArgs sa = a;
                sa.seg_row = a.seg_row + win.single_begin;
                sa.colind = a.colind + win.single_nz;
                sa.vals = static_cast<const uint8_t *>(a.vals) + static_cast<size_t>(win.single_nz) * (plan->dtype == SD_F32 ? 4 : 2);
                sa.S = win.single_end - win.single_begin;
                SD_CUDA_TRY(run_single(sa, plan->dtype, vec, s_single));
            }
            if (s_short != st) {
                SD_CUDA_TRY(cudaEventRecord(plan->ev_join[0], s_short));
                SD_CUDA_TRY(cudaStreamWaitEvent(st, plan->ev_join[0], 0));
            }
            if (s_single != st) {
                SD_CUDA_TRY(cudaEventRecord(plan->ev_join[1], s_single));
                SD_CUDA_TRY(cudaStreamWaitEvent(st, plan->ev_join[1], 0));
            }
            if (ahead && chunks_issued < plan->wins.size()) {   // window w is done: the chunk stream may go one further
                SD_CUDA_TRY(cudaEventRecord(plan->ev_join[0], st));
                SD_CUDA_TRY(cudaStreamWaitEvent(plan->chunk_stream, plan->ev_join[0], 0));
                sd_status_t cs = issue_chunks_upto(chunks_issued + 1);
                if (cs) return cs;
            }
            if (win.ntiles == 0) continue;
            MergeArgs m;
            m.s = a;
            m.tile_seg = plan->tile_seg + win.tile_base + w;
            m.tile_head = plan->tile_head + win.tile_base * N;
            m.tile_tail = plan->tile_tail + win.tile_base * N;
            m.seg_begin = win.seg_begin;
            m.seg_end = win.seg_end;
            m.ntiles = win.ntiles;
            SD_CUDA_TRY(run_merge(m, plan->dtype, vec, plan->fix_short + win.tile_base, win.nshort,
                                  plan->fix_long + win.tile_base, win.nlong, st));
        }
        if (ahead) SD_CUDA_TRY(cudaStreamWaitEvent(st, plan->ev_chunk.back(), 0));   // the caller's stream covers everything
        return SD_OK;
    }
    case SD_HYBRID: {
        // one launch for the chunks of the heavy rows, the rows of medium length and the short rows; then the chunk sums
        SpmmArgs ca = a, ma = a, la = a;
        ca.ranges = plan->h_ranges;
        ca.order = plan->h_order;
        ca.S = plan->h_nc;
        ca.C = plan->chunk_out;
        ca.ldc = N;
        ca.alpha = 1.f;
        ca.beta = 0.f;
        ma.desc = plan->h_desc;
        ma.S = plan->h_nm;
        la.desc = plan->h_desc + plan->h_nm;
        la.S = M - plan->h_nl - plan->h_nm;
        SD_CUDA_TRY(run_hybrid_fused(ca, ma, la, plan->dtype, vec, st));
        if (plan->h_nl > 0) {
            SD_CUDA_TRY(run_chunk_reduce(plan->chunk_out, plan->h_chunk_ptr, plan->h_rows, 0, plan->h_nl, C, ldc,
                                         static_cast<int32_t>(N), alpha, beta, st, plan->h_ng > 0 ? kGiantChunks : 0));
            if (plan->h_ng > 0)
                SD_CUDA_TRY(run_chunk_reduce_wide(plan->chunk_out, plan->h_chunk_ptr, plan->h_rows, plan->h_giant,
                                                  plan->h_ng, C, ldc, static_cast<int32_t>(N), alpha, beta, st));
        }
        return SD_OK;
    }
    case SD_BSR_TC: {
        BsrArgs b;
        b.browptr = plan->browptr;
        b.bcol = plan->bcol;
        b.bval = plan->bval;
        b.bval_mma = plan->bval_mma;
        b.part = plan->bsr_part;
        b.nparts = plan->bsr_nparts;
        b.B = B;
        b.C = C;
        b.ldb = ldb;
        b.ldc = ldc;
        b.M = M;
        b.K = plan->K;
        b.Mb = static_cast<int32_t>((M + 15) / 16);
        b.N = static_cast<int32_t>(N);
        b.alpha = alpha;
        b.beta = beta;
        b.map_cache = &plan->tc_map;
        b.test_wait_expiry = plan->test_wait_expiry;
        const bool vec4 = aligned16(B) && aligned16(C) && N % 4 == 0 && ldb % 4 == 0 && ldc % 4 == 0 &&
                          (plan->dtype == SD_F32 || (reinterpret_cast<uintptr_t>(B) & 7u) == 0);
        if (bsr_tc_usable(b, plan->dtype) && !switches().bsr_simt)
            SD_CUDA_TRY(run_bsr_tc(b, plan->dtype, plan->dev_error, plan->info.sm_count, st));
        else
            SD_CUDA_TRY(run_bsr_simt(b, plan->dtype, vec4, st));
        return SD_OK;
    }
    default:
        set_error(SD_ERR_INTERNAL, "plan has no family");
        return SD_ERR_INTERNAL;
    }
}

sd_status_t sd_plan_update_values(sd_plan_t *plan, const void *vals, void *stream) {
    if (!plan) {
        set_error(SD_ERR_INVALID_ARG, "plan is null");
        return SD_ERR_INVALID_ARG;
    }
    if (plan->nnz == 0) return SD_OK;
    if (!vals) {
        set_error(SD_ERR_INVALID_ARG, "vals is null");
        return SD_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool same_copy = plan->m_vals == plan->vals;   // the kernels read the caller's array directly
    plan->vals = vals;
    switch (plan->info.family) {
    case SD_MERGE:
        if (same_copy) {
            plan->m_vals = vals;
        } else if (plan->w_src) {
            const unsigned blocks = static_cast<unsigned>(ceil_div(plan->nnz, 256));
            if (plan->dtype == SD_F32)
                window_revalue_kernel<float><<<blocks, 256, 0, st>>>(plan->w_src, static_cast<const float *>(vals), plan->nnz,
                                                                     static_cast<float *>(plan->w_vals));
            else
                window_revalue_kernel<uint16_t><<<blocks, 256, 0, st>>>(plan->w_src, static_cast<const uint16_t *>(vals),
                                                                        plan->nnz, static_cast<uint16_t *>(plan->w_vals));
            SD_CUDA_TRY(cudaGetLastError());
        }
        return SD_OK;
    case SD_BSR_TC: {
        const size_t es = plan->dtype == SD_F32 ? 4 : 2;
        SD_CUDA_TRY(cudaMemsetAsync(plan->bval, 0, es * 256 * plan->nnzb, st));
        SD_CUDA_TRY(plan->dtype == SD_F32 ? fill_bsr<float>(plan, st) : fill_bsr<__nv_bfloat16>(plan, st));
        SD_CUDA_TRY(build_bsr_mma_image(plan->bval, plan->bval_mma, plan->nnzb, plan->dtype, st));
        return SD_OK;
    }
    default:
        return SD_OK;   // row-split reads the caller's array
    }
}

sd_status_t sd_spmm_host_async(sd_plan_t *plan, const void *B_host, int64_t ldb, float *C_host, int64_t ldc, float alpha,
                         float beta) {
    if (!plan) {
        set_error(SD_ERR_INVALID_ARG, "plan is null");
        return SD_ERR_INVALID_ARG;
    }
    const int64_t M = plan->M, N = plan->N, K = plan->K;
    if (M == 0 || N == 0) return SD_OK;
    if (!C_host || ldc < N || !B_host || ldb < N) {
        set_error(SD_ERR_INVALID_ARG, "null host buffer or leading dimension < N");
        return SD_ERR_INVALID_ARG;
    }
    const size_t es = plan->dtype == SD_F32 ? 4 : 2;
    sd_status_t s;
    if (!plan->host_stream) SD_CUDA_TRY(cudaStreamCreateWithFlags(&plan->host_stream, cudaStreamNonBlocking));
    if (!plan->stage_B && (s = dev_alloc(plan, &plan->stage_B, es * K * N, "B staging"))) return s;
    if (!plan->stage_C && (s = dev_alloc(plan, reinterpret_cast<void **>(&plan->stage_C), sizeof(float) * M * N,
                                         "C staging")))
        return s;
    cudaStream_t st = plan->host_stream;
    SD_CUDA_TRY(cudaMemcpy2DAsync(plan->stage_B, es * N, B_host, es * ldb, es * N, K, cudaMemcpyHostToDevice, st));
    if (beta != 0.f)
        SD_CUDA_TRY(cudaMemcpy2DAsync(plan->stage_C, 4 * N, C_host, 4 * ldc, 4 * N, M, cudaMemcpyHostToDevice, st));
    if ((s = sd_spmm(plan, plan->stage_B, N, plan->stage_C, N, alpha, beta, st))) return s;
    SD_CUDA_TRY(cudaMemcpy2DAsync(C_host, 4 * ldc, plan->stage_C, 4 * N, 4 * N, M, cudaMemcpyDeviceToHost, st));
    return SD_OK;
}

sd_status_t sd_plan_sync(sd_plan_t *plan) {
    if (!plan) {
        set_error(SD_ERR_INVALID_ARG, "plan is null");
        return SD_ERR_INVALID_ARG;
    }
    if (plan->host_stream) SD_CUDA_TRY(cudaStreamSynchronize(plan->host_stream));
    return SD_OK;
}

sd_status_t sd_spmm_host(sd_plan_t *plan, const void *B_host, int64_t ldb, float *C_host, int64_t ldc, float alpha,
                         float beta) {
    const sd_status_t s = sd_spmm_host_async(plan, B_host, ldb, C_host, ldc, alpha, beta);
    return s ? s : sd_plan_sync(plan);
}

sd_status_t sd_plan_save(const sd_plan_t *plan, void *buf, size_t cap, size_t *bytes) {
    if (!plan || !bytes) {
        set_error(SD_ERR_INVALID_ARG, "sd_plan_save: plan and bytes must not be null");
        return SD_ERR_INVALID_ARG;
    }
    sd_plan *p = const_cast<sd_plan *>(plan);   // only read
    BlobArray arr[kBlobArrays];
    blob_arrays(p, arr);
    const size_t nwins = p->wins.size();
    size_t need = pad16(sizeof(BlobHeader)) + pad16(nwins * sizeof(sd_plan::Window));
    for (const BlobArray &a : arr) need += pad16(a.bytes);
    *bytes = need;
    if (!buf) return SD_OK;   // size query
    if (cap < need) {
        set_error(SD_ERR_INVALID_ARG, "sd_plan_save: the buffer holds %zu bytes, the plan needs %zu", cap, need);
        return SD_ERR_INVALID_ARG;
    }
    int prev = 0;
    SD_CUDA_TRY(cudaGetDevice(&prev));
    SD_CUDA_TRY(cudaSetDevice(p->device));
    BlobHeader h;
    memset(&h, 0, sizeof h);
    h.magic = kBlobMagic;
    h.version = kBlobVersion;
    h.header_bytes = static_cast<uint32_t>(sizeof(BlobHeader));
    sd_status_t s = pattern_hash(p->rowptr, p->colind, p->M, p->nnz, nullptr, &h.pattern);
    if (s == SD_OK) {
        cudaDeviceProp prop;
        cudaError_t e = cudaGetDeviceProperties(&prop, p->device);
        if (e != cudaSuccess) s = cuda_fail(e, "cudaGetDeviceProperties");
        else strncpy(h.device_name, prop.name, sizeof h.device_name - 1);
    }
    if (s != SD_OK) {
        cudaSetDevice(prev);
        return s;
    }
    h.M = p->M; h.K = p->K; h.N = p->N; h.nnz = p->nnz;
    h.dtype = p->dtype;
    h.family = p->info.family;
    h.sm_count = p->info.sm_count;
    h.nwins = static_cast<int32_t>(nwins);
    h.l2_bytes = p->info.l2_bytes;
    h.info = p->info;
    h.num_segments = p->num_segments;
    h.num_chunks = p->num_chunks;
    h.ntiles = p->ntiles;
    h.nnzb = p->nnzb;
    h.bsr_nparts = p->bsr_nparts;
    h.has_coo = p->coo_row ? 1 : 0;
    h.h_nl = p->h_nl; h.h_nc = p->h_nc; h.h_ng = p->h_ng; h.h_nm = p->h_nm; h.h_T = p->h_T;
    for (int i = 0; i < kBlobArrays; ++i) h.array_bytes[i] = arr[i].bytes;
    unsigned char *out = static_cast<unsigned char *>(buf);
    memset(out, 0, need);
    memcpy(out, &h, sizeof h);
    size_t off = pad16(sizeof(BlobHeader));
    if (nwins) memcpy(out + off, p->wins.data(), nwins * sizeof(sd_plan::Window));
    off += pad16(nwins * sizeof(sd_plan::Window));
    for (const BlobArray &a : arr) {
        if (a.bytes) {
            cudaError_t e = cudaMemcpy(out + off, *a.field, a.bytes, cudaMemcpyDeviceToHost);
            if (e != cudaSuccess) {
                cudaSetDevice(prev);
                return cuda_fail(e, a.what);
            }
        }
        off += pad16(a.bytes);
    }
    cudaSetDevice(prev);
    return SD_OK;
}

sd_status_t sd_plan_load(const void *blob, size_t bytes, const int32_t *rowptr, const int32_t *colind, const void *vals,
                         sd_plan_t **out) {
    if (out) *out = nullptr;
    if (!blob || !out || bytes < sizeof(BlobHeader)) {
        set_error(SD_ERR_INVALID_ARG, "sd_plan_load: null argument or a blob shorter than its header");
        return SD_ERR_INVALID_ARG;
    }
    BlobHeader h;
    memcpy(&h, blob, sizeof h);
    if (h.magic != kBlobMagic || h.version != kBlobVersion || h.header_bytes != sizeof(BlobHeader) || h.nwins < 0 ||
        h.M < 0 || h.nnz < 0 || (h.dtype != SD_F32 && h.dtype != SD_BF16)) {
        set_error(SD_ERR_INVALID_ARG, "sd_plan_load: not a plan blob of this library version");
        return SD_ERR_INVALID_ARG;
    }
    size_t need = pad16(sizeof(BlobHeader)) + pad16(static_cast<size_t>(h.nwins) * sizeof(sd_plan::Window));
    for (int i = 0; i < kBlobArrays; ++i) need += pad16(h.array_bytes[i]);
    if (bytes < need) {
        set_error(SD_ERR_INVALID_ARG, "sd_plan_load: the blob is truncated (%zu of %zu bytes)", bytes, need);
        return SD_ERR_INVALID_ARG;
    }
    if ((h.M > 0 && !rowptr) || (h.nnz > 0 && (!colind || !vals))) {
        set_error(SD_ERR_INVALID_ARG, "sd_plan_load: the CSR arrays the plan was made for must be given again");
        return SD_ERR_INVALID_ARG;
    }
    // key: device model, then the pattern itself
    int dev = 0;
    SD_CUDA_TRY(cudaGetDevice(&dev));
    cudaDeviceProp prop;
    SD_CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
    if (strncmp(prop.name, h.device_name, sizeof h.device_name) != 0 || prop.multiProcessorCount != h.sm_count ||
        static_cast<int64_t>(prop.l2CacheSize) != h.l2_bytes) {
        set_error(SD_ERR_UNSUPPORTED, "sd_plan_load: the plan was made on '%s' (%d SMs), this device is '%s' (%d SMs)",
                  h.device_name, h.sm_count, prop.name, prop.multiProcessorCount);
        return SD_ERR_UNSUPPORTED;
    }
    if (h.M > 0) {
        int32_t last = 0;
        SD_CUDA_TRY(cudaMemcpy(&last, rowptr + h.M, sizeof last, cudaMemcpyDeviceToHost));
        if (last != h.nnz) {
            set_error(SD_ERR_INVALID_ARG, "sd_plan_load: rowptr[M] = %d, the plan was made for %lld nonzeros", last,
                      (long long)h.nnz);
            return SD_ERR_INVALID_ARG;
        }
    }
    uint64_t pat = 0;
    sd_status_t s = pattern_hash(rowptr, colind, h.M, h.nnz, nullptr, &pat);
    if (s != SD_OK) return s;
    if (pat != h.pattern) {
        set_error(SD_ERR_INVALID_ARG, "sd_plan_load: the sparsity pattern differs from the one the plan was made for");
        return SD_ERR_INVALID_ARG;
    }
    sd_plan *p = new (std::nothrow) sd_plan;
    if (!p) {
        set_error(SD_ERR_ALLOC, "host allocation failed");
        return SD_ERR_ALLOC;
    }
    auto fail = [&](sd_status_t code) {
        free_plan(p);
        return code;
    };
    p->rowptr = rowptr;
    p->colind = colind;
    p->vals = vals;
    p->M = h.M; p->K = h.K; p->N = h.N; p->nnz = h.nnz;
    p->dtype = h.dtype;
    p->device = dev;
    p->info = h.info;
    p->num_segments = h.num_segments;
    p->num_chunks = h.num_chunks;
    p->ntiles = h.ntiles;
    p->nnzb = h.nnzb;
    p->bsr_nparts = h.bsr_nparts;
    p->h_nl = h.h_nl; p->h_nc = h.h_nc; p->h_ng = h.h_ng; p->h_nm = h.h_nm; p->h_T = h.h_T;
    const unsigned char *in = static_cast<const unsigned char *>(blob);
    size_t off = pad16(sizeof(BlobHeader));
    p->wins.resize(h.nwins);
    if (h.nwins) memcpy(p->wins.data(), in + off, static_cast<size_t>(h.nwins) * sizeof(sd_plan::Window));
    off += pad16(static_cast<size_t>(h.nwins) * sizeof(sd_plan::Window));
    // the array list depends on coo_row being set: mark it before sizing, allocate below
    BlobArray arr[kBlobArrays];
    if (h.has_coo) p->coo_row = reinterpret_cast<int32_t *>(1);
    blob_arrays(p, arr);
    p->coo_row = nullptr;
    for (int i = 0; i < kBlobArrays; ++i) {
        if (arr[i].bytes != h.array_bytes[i]) {
            set_error(SD_ERR_INVALID_ARG, "sd_plan_load: the blob's array sizes do not fit its header");
            return fail(SD_ERR_INVALID_ARG);
        }
        if (arr[i].bytes) {
            if ((s = dev_alloc(p, arr[i].field, arr[i].bytes, arr[i].what))) return fail(s);
            cudaError_t e = cudaMemcpy(*arr[i].field, in + off, arr[i].bytes, cudaMemcpyHostToDevice);
            if (e != cudaSuccess) return fail(cuda_fail(e, arr[i].what));
        }
        off += pad16(arr[i].bytes);
    }
    // scratch and value copies, as plan creation allocates them
    const size_t es = p->dtype == SD_F32 ? 4 : 2;
    if (p->info.family == SD_MERGE && !p->wins.empty()) {
        const int W = static_cast<int>(p->wins.size());
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->tile_head), sizeof(float) * p->ntiles * p->N, "tile heads"))) return fail(s);
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->tile_tail), sizeof(float) * p->ntiles * p->N, "tile tails"))) return fail(s);
        if (p->info.class_split) {
            if ((s = dev_alloc(p, &p->w_vals, es * p->nnz, "window-major values"))) return fail(s);
            if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->chunk_out), sizeof(float) * p->num_chunks * p->N, "chunk sums"))) return fail(s);
            if ((s = create_split_streams(p, W))) return fail(s);
            p->m_ptr = p->w_ptr;
            p->m_col = p->w_col;
            p->m_vals = p->w_vals;
            p->m_seg_row = p->w_seg_row;
        } else {
            p->m_ptr = p->rowptr;
            p->m_col = p->colind;
            p->m_vals = p->vals;
            p->m_seg_row = nullptr;
        }
        if (h.has_coo) {
            const int cchunk = coo_chunk(static_cast<int>(p->N));
            const int64_t chunks1 = (p->nnz + cchunk - 1) / cchunk, count2 = 2 * chunks1;
            const int64_t chunks2 = (count2 + kCooCarryChunk - 1) / kCooCarryChunk, count3 = 2 * chunks2;
            if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->coo_c1_row), sizeof(int32_t) * count2, "carry rows"))) return fail(s);
            if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->coo_c1_val), sizeof(float) * count2 * p->N, "carry sums"))) return fail(s);
            if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->coo_c2_row), sizeof(int32_t) * count3, "carry rows (level 2)"))) return fail(s);
            if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->coo_c2_val), sizeof(float) * count3 * p->N, "carry sums (level 2)"))) return fail(s);
        }
    } else if (p->info.family == SD_HYBRID && p->h_T > 0) {
        if (p->h_nl > 0 &&
            (s = dev_alloc(p, reinterpret_cast<void **>(&p->chunk_out), sizeof(float) * p->h_nc * p->N, "chunk sums")))
            return fail(s);
        if ((s = build_light_desc(p, nullptr))) return fail(s);
    } else if (p->info.family == SD_BSR_TC) {
        if ((s = dev_alloc(p, &p->bval, es * 256 * p->nnzb, "bval"))) return fail(s);
        if ((s = dev_alloc(p, &p->bval_mma, (p->dtype == SD_BF16 ? 512 : 2048) * static_cast<size_t>(p->nnzb), "bval (tensor-core image)"))) return fail(s);
        if ((s = dev_alloc(p, reinterpret_cast<void **>(&p->dev_error), sizeof(int32_t), "error word"))) return fail(s);
        cudaError_t e = cudaMemset(p->dev_error, 0, sizeof(int32_t));
        if (e != cudaSuccess) return fail(cuda_fail(e, "cudaMemset"));
    }
    // the value copies come from the values given now (the blob is keyed by the pattern only)
    if ((s = sd_plan_update_values(p, vals, nullptr))) return fail(s);
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return fail(cuda_fail(e, "cudaDeviceSynchronize"));
    p->info = h.info;
    *out = p;
    return SD_OK;
}

#pragma GCC visibility pop
}  // extern "C"
