// sd_spmm_merge_static: the merge-path SpMM for callers that must not allocate.
//
// Some callers cannot let a library call cudaMalloc: a serving process whose framework has
// already handed every free byte of the GPU to its own caching pool (a late cudaMalloc then
// fails or fragments that pool), a latency-critical loop where cudaMalloc's implicit
// device-wide synchronisation is unacceptable, or code that holds a hard memory budget.  A
// plan (sd_plan_create) allocates its tile table and carry-out buffers, so such callers cannot
// use it.  This entry point keeps all of that in one fixed array that lives in the library's
// device image, and so performs no allocation at all, at the price of a size limit.
#include <cstdio>

#include "sd_common.cuh"
#include "sd_launch.cuh"
#include "sd_merge.cuh"

namespace sd {

// The whole scratch of one call: tile table, then the per-tile head rows, then the per-tile
// tail rows.  Every GPU that loads the library carries these 4 MiB until the process exits.
constexpr size_t kStaticScratchBytes = 4u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// device address of g_static_scratch, per device; published with release / acquire so that two host
// threads making their first call on a device together both end up with the complete address
static std::atomic<void *> g_scratch_addr[kMaxDevices];

// In host code the name g_static_scratch is only a handle for the runtime, not an address a
// kernel could use; the real device address has to be asked for, once per device, with that
// device current.
static sd_status_t static_scratch(void **out) {
    int dev = 0;
    SD_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) {
        set_error(SD_ERR_UNSUPPORTED, "device ordinal %d is beyond the %d this entry point tracks", dev, kMaxDevices);
        return SD_ERR_UNSUPPORTED;
    }
    void *p = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!p) {
        SD_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        g_scratch_addr[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return SD_OK;
}

// Fix-up without a precomputed list: one warp looks at one tile, decides by itself whether the
// tile closed a row that an earlier tile began, and if so adds the carry-outs of the tiles
// since the row's first nonzero (four chains per warp, combined in a fixed order) to the head.
static __global__ void __launch_bounds__(256)
merge_fixup_scan_kernel(const MergeArgs m, int32_t tile_items) {
    const SpmmArgs &a = m.s;
    const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (t >= m.ntiles) return;
    const int lane = threadIdx.x & 31;
    const int64_t s0 = m.tile_seg[t], s1 = m.tile_seg[t + 1];
    const int64_t nz0 = static_cast<int64_t>(t) * tile_items - s0;   // rows start at 0 here: nzb = 0
    if (!(s1 > s0 && nz0 > a.ptr[s0])) return;
    const int ta = static_cast<int>((a.ptr[s0] + s0) / tile_items);
    float *crow = a.C + s0 * a.ldc;
    for (int c0 = 0; c0 < a.N; c0 += 8) {
        const int c = c0 + (lane & 7), chain = lane >> 3;
        float sum = 0.f;
        if (c < a.N)
            for (int tt = ta + chain; tt < t; tt += 4) sum += m.tile_tail[static_cast<int64_t>(tt) * a.N + c];
        sum += __shfl_xor_sync(0xffffffffu, sum, 8);
        sum += __shfl_xor_sync(0xffffffffu, sum, 16);
        if (chain == 0 && c < a.N) {
            const float tot = sum + m.tile_head[static_cast<int64_t>(t) * a.N + c];
            float r = a.alpha * tot;
            if (a.beta != 0.f) r = fmaf(a.beta, crow[c], r);
            crow[c] = r;
        }
    }
}

static __global__ void static_table_kernel(const int32_t *__restrict__ ptr, int64_t S, int32_t tile, int32_t ntiles,
                                           int32_t *__restrict__ tile_seg) {
    const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t > ntiles) return;
    const int64_t total = S + ptr[S];
    const int64_t d = min(t * tile, total);
    int64_t lo = 0, hi = S;   // number of row ends placed before merged position d
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (ptr[mid + 1] + mid < d) lo = mid + 1;
        else hi = mid;
    }
    tile_seg[t] = static_cast<int32_t>(lo);
}

}  // namespace sd

using namespace sd;

extern "C" {
#pragma GCC visibility push(default)

sd_status_t sd_spmm_merge_static(const int32_t *rowptr, const int32_t *colind, const float *vals, int64_t M, int64_t K,
                                 int64_t N, int64_t nnz, const float *B, int64_t ldb, float *C, int64_t ldc, float alpha,
                                 float beta, void *stream) {
    if (M < 0 || K < 0 || N < 0 || nnz < 0 || M > INT32_MAX - 1 || nnz > INT32_MAX - 1 || N > INT32_MAX / 2) {
        set_error(SD_ERR_INVALID_ARG, "M, K, N, nnz must be in [0, 2^31)");
        return SD_ERR_INVALID_ARG;
    }
    if (M == 0 || N == 0) return SD_OK;
    if (!rowptr || !C || ldc < N) {
        set_error(SD_ERR_INVALID_ARG, "rowptr or C is null, or ldc < N");
        return SD_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (alpha == 0.f || nnz == 0) {
        SD_CUDA_TRY(run_scale_c(C, ldc, M, static_cast<int32_t>(N), beta, st));
        return SD_OK;
    }
    if (!colind || !vals || !B || ldb < N) {
        set_error(SD_ERR_INVALID_ARG, "colind, vals or B is null, or ldb < N");
        return SD_ERR_INVALID_ARG;
    }
    if (ldb * 4 > static_cast<int64_t>(UINT32_MAX)) {
        set_error(SD_ERR_UNSUPPORTED, "row pitch of B must be below 4 GiB");
        return SD_ERR_UNSUPPORTED;
    }
    // layout of the fixed array: [tile table | head rows | tail rows]
    const int64_t ntiles = (M + nnz + kMergeTile - 1) / kMergeTile;
    const size_t table_bytes = ((static_cast<size_t>(ntiles) + 1) * sizeof(int32_t) + 255) & ~static_cast<size_t>(255);
    const size_t rows_bytes = static_cast<size_t>(ntiles) * static_cast<size_t>(N) * sizeof(float);
    const size_t need = table_bytes + 2 * rows_bytes;
    if (need > kStaticScratchBytes) {
        set_error(SD_ERR_UNSUPPORTED,
                  "sd_spmm_merge_static: (M + nnz) = %lld with N = %lld needs %zu bytes of scratch, the fixed array holds "
                  "%zu; use a plan (sd_plan_create) for this size",
                  (long long)(M + nnz), (long long)N, need, kStaticScratchBytes);
        return SD_ERR_UNSUPPORTED;
    }
    void *base = nullptr;
    const sd_status_t s = static_scratch(&base);
    if (s != SD_OK) return s;
    unsigned char *p = static_cast<unsigned char *>(base);

    SpmmArgs a;
    a.ptr = rowptr;
    a.colind = colind;
    a.vals = vals;
    a.seg_row = nullptr;
    a.B = B;
    a.C = C;
    a.ldb = ldb;
    a.ldc = ldc;
    a.ldb_bytes = static_cast<uint32_t>(ldb * 4);
    a.S = M;
    a.N = static_cast<int32_t>(N);
    a.alpha = alpha;
    a.beta = beta;
    a.max_len = 0;
    a.mean_len = 0;
    MergeArgs m;
    m.s = a;
    m.tile_seg = reinterpret_cast<int32_t *>(p);
    m.tile_head = reinterpret_cast<float *>(p + table_bytes);
    m.tile_tail = reinterpret_cast<float *>(p + table_bytes + rows_bytes);
    m.seg_begin = 0;
    m.seg_end = M;
    m.ntiles = static_cast<int32_t>(ntiles);

    // The array still holds whatever the previous call left.  The table and the tail rows are
    // rewritten in full below; the head rows are written only by tiles that close a row, so they
    // are cleared first.
    SD_CUDA_TRY(cudaMemsetAsync(m.tile_head, 0, rows_bytes, st));
    static_table_kernel<<<ceil_div(ntiles + 1, 256), 256, 0, st>>>(rowptr, M, kMergeTile, m.ntiles,
                                                                 reinterpret_cast<int32_t *>(p));
    SD_CUDA_TRY(cudaGetLastError());
    const bool vec = ((reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(C)) & 15u) == 0 && N % 4 == 0 &&
                     ldb % 4 == 0 && ldc % 4 == 0;
    SD_CUDA_TRY(run_merge(m, SD_F32, vec, nullptr, 0, nullptr, 0, st));   // tile kernel only: no lists
    merge_fixup_scan_kernel<<<ceil_div(ntiles, 8), 256, 0, st>>>(m, kMergeTile);
    SD_CUDA_TRY(cudaGetLastError());
    return SD_OK;
}

#pragma GCC visibility pop
}  // extern "C"
