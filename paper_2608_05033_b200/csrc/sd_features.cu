// Extended structure analysis (paper Sec. 3.1: row-length quartiles, column-degree statistics,
// value-slot expansion of ELL / SELL / BSR, Eq. 4).  Exact integer counts, computed on the device
// on request; nothing here is on the sd_spmm path.
#include <algorithm>

#include <cub/cub.cuh>

#include "sd_common.cuh"
#include "sd_launch.cuh"

namespace sd {

namespace {

struct FeatAccum {
    unsigned long long col_max, col_empty, sum_d2;
    unsigned long long sell[3];
    unsigned long long distinct;
};

__global__ void feat_row_len_kernel(const int32_t *__restrict__ rowptr, int64_t M, int32_t *__restrict__ len) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < M) len[i] = rowptr[i + 1] - rowptr[i];
}

__global__ void feat_col_count_kernel(const int32_t *__restrict__ colind, int64_t nnz, int32_t *__restrict__ deg) {
    for (int64_t p = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; p < nnz;
         p += static_cast<int64_t>(gridDim.x) * blockDim.x)
        atomicAdd(deg + colind[p], 1);   // integer atomics: the counts do not depend on the order
}

__global__ void __launch_bounds__(256)
feat_col_stats_kernel(const int32_t *__restrict__ deg, int64_t K, FeatAccum *__restrict__ out) {
    using Reduce = cub::BlockReduce<unsigned long long, 256>;
    __shared__ typename Reduce::TempStorage tmp;
    unsigned long long mx = 0, empty = 0, d2 = 0;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < K;
         j += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const unsigned long long d = static_cast<unsigned long long>(deg[j]);
        mx = max(mx, d);
        empty += (d == 0);
        d2 += d * d;
    }
    mx = Reduce(tmp).Reduce(mx, cub::Max());
    __syncthreads();
    empty = Reduce(tmp).Sum(empty);
    __syncthreads();
    d2 = Reduce(tmp).Sum(d2);
    if (threadIdx.x == 0) {
        atomicMax(&out->col_max, mx);
        atomicAdd(&out->col_empty, empty);
        atomicAdd(&out->sum_d2, d2);
    }
}

// One warp per slice of c consecutive rows: |s| * max r over the slice.
__global__ void __launch_bounds__(256)
feat_sell_kernel(const int32_t *__restrict__ rowptr, int64_t M, int32_t c, int which, FeatAccum *__restrict__ out) {
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int64_t nslices = (M + c - 1) / c;
    const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    unsigned long long local = 0;
    for (int64_t s = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; s < nslices; s += warps) {
        const int64_t r0 = s * c, r1 = min(M, r0 + c);
        int mx = 0;
        for (int64_t i = r0 + lane; i < r1; i += 32) mx = max(mx, rowptr[i + 1] - rowptr[i]);
        mx = __reduce_max_sync(FULL, mx);
        local += static_cast<unsigned long long>(r1 - r0) * static_cast<unsigned long long>(mx);
    }
    if (lane == 0 && local) atomicAdd(&out->sell[which], local);
}

// b x b block key of every nonzero (b = 1 << shift); one warp per row.
__global__ void __launch_bounds__(256)
feat_block_keys_kernel(const int32_t *__restrict__ rowptr, const int32_t *__restrict__ colind, int64_t M, int shift,
                       unsigned long long Kb, unsigned long long *__restrict__ keys) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    for (int64_t row = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; row < M; row += warps) {
        const unsigned long long base = static_cast<unsigned long long>(row >> shift) * Kb;
        for (int p = rowptr[row] + lane; p < rowptr[row + 1]; p += 32)
            keys[p] = base + static_cast<unsigned long long>(colind[p] >> shift);
    }
}

__global__ void __launch_bounds__(256)
feat_distinct_kernel(const unsigned long long *__restrict__ sorted, int64_t n, FeatAccum *__restrict__ out) {
    using Reduce = cub::BlockReduce<unsigned long long, 256>;
    __shared__ typename Reduce::TempStorage tmp;
    unsigned long long cnt = 0;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x)
        cnt += (i == 0 || sorted[i] != sorted[i - 1]);
    cnt = Reduce(tmp).Sum(cnt);
    if (threadIdx.x == 0 && cnt) atomicAdd(&out->distinct, cnt);
}

struct Tmp {   // temporary device memory, freed on every exit path
    void *p = nullptr;
    ~Tmp() { if (p) cudaFree(p); }
    cudaError_t get(size_t bytes) { return cudaMalloc(&p, bytes ? bytes : 16); }
};

int grid_for(int64_t n, int per_block) {
    return static_cast<int>(std::max<int64_t>(1, std::min<int64_t>((n + per_block - 1) / per_block, 148 * 16)));
}

// Nearest-rank quartiles of n int32 values (destroys nothing: sorts into a copy).
sd_status_t quartiles(const int32_t *vals, int64_t n, int64_t (&q)[3], cudaStream_t st) {
    q[0] = q[1] = q[2] = 0;
    if (n <= 0) return SD_OK;
    Tmp sorted, scratch;
    SD_CUDA_TRY(sorted.get(sizeof(int32_t) * n));
    size_t tb = 0;
    SD_CUDA_TRY(cub::DeviceRadixSort::SortKeys(nullptr, tb, vals, static_cast<int32_t *>(sorted.p), n, 0, 32, st));
    SD_CUDA_TRY(scratch.get(tb));
    SD_CUDA_TRY(cub::DeviceRadixSort::SortKeys(scratch.p, tb, vals, static_cast<int32_t *>(sorted.p), n, 0, 32, st));
    for (int k = 1; k <= 3; ++k) {
        const int64_t rank = (k * n + 3) / 4;   // ceil(k n / 4), 1-based
        int32_t v = 0;
        SD_CUDA_TRY(cudaMemcpyAsync(&v, static_cast<int32_t *>(sorted.p) + (rank - 1), sizeof v, cudaMemcpyDeviceToHost, st));
        SD_CUDA_TRY(cudaStreamSynchronize(st));
        q[k - 1] = v;
    }
    return SD_OK;
}

}  // namespace

sd_status_t compute_feature_counts(const int32_t *rowptr, const int32_t *colind, int64_t M, int64_t K, int64_t nnz,
                                   cudaStream_t st, FeatureCounts *out) {
    *out = FeatureCounts{};
    Tmp acc;
    SD_CUDA_TRY(acc.get(sizeof(FeatAccum)));
    FeatAccum *dacc = static_cast<FeatAccum *>(acc.p);
    SD_CUDA_TRY(cudaMemsetAsync(dacc, 0, sizeof(FeatAccum), st));
    sd_status_t s;

    // ---- row-length quartiles and SELL slots ------------------------------------------------------
    if (M > 0) {
        Tmp len;
        SD_CUDA_TRY(len.get(sizeof(int32_t) * M));
        feat_row_len_kernel<<<static_cast<unsigned>((M + 255) / 256), 256, 0, st>>>(rowptr, M, static_cast<int32_t *>(len.p));
        SD_CUDA_TRY(cudaGetLastError());
        if ((s = quartiles(static_cast<int32_t *>(len.p), M, out->row_q, st))) return s;
        const int32_t heights[3] = {16, 32, 512};
        for (int w = 0; w < 3; ++w) {
            feat_sell_kernel<<<grid_for((M + heights[w] - 1) / heights[w], 8), 256, 0, st>>>(rowptr, M, heights[w], w, dacc);
            SD_CUDA_TRY(cudaGetLastError());
        }
    }

    // ---- column degrees ---------------------------------------------------------------------------
    if (K > 0) {
        Tmp deg;
        SD_CUDA_TRY(deg.get(sizeof(int32_t) * K));
        SD_CUDA_TRY(cudaMemsetAsync(deg.p, 0, sizeof(int32_t) * K, st));
        if (nnz > 0) {
            feat_col_count_kernel<<<grid_for(nnz, 1024), 256, 0, st>>>(colind, nnz, static_cast<int32_t *>(deg.p));
            SD_CUDA_TRY(cudaGetLastError());
        }
        feat_col_stats_kernel<<<grid_for(K, 1024), 256, 0, st>>>(static_cast<int32_t *>(deg.p), K, dacc);
        SD_CUDA_TRY(cudaGetLastError());
        if ((s = quartiles(static_cast<int32_t *>(deg.p), K, out->col_q, st))) return s;
    }

    // ---- occupied 4x4 and 8x8 blocks: keys -> sort -> count the distinct ones -----------------------
    int64_t nnzb[2] = {0, 0};
    if (nnz > 0 && M > 0) {
        Tmp ka, kb, scratch;
        SD_CUDA_TRY(ka.get(sizeof(unsigned long long) * nnz));
        SD_CUDA_TRY(kb.get(sizeof(unsigned long long) * nnz));
        auto *a = static_cast<unsigned long long *>(ka.p);
        auto *b = static_cast<unsigned long long *>(kb.p);
        size_t cap = 0;
        for (int w = 0; w < 2; ++w) {
            const int shift = w == 0 ? 2 : 3;
            const unsigned long long Kb = (static_cast<unsigned long long>(K) + (1u << shift) - 1) >> shift;
            const unsigned long long Mb = (static_cast<unsigned long long>(M) + (1u << shift) - 1) >> shift;
            int bits = 1;
            while (bits < 64 && (static_cast<unsigned __int128>(1) << bits) < static_cast<unsigned __int128>(Mb) * Kb) ++bits;
            feat_block_keys_kernel<<<grid_for(M, 8), 256, 0, st>>>(rowptr, colind, M, shift, Kb, a);
            SD_CUDA_TRY(cudaGetLastError());
            size_t tb = 0;
            SD_CUDA_TRY(cub::DeviceRadixSort::SortKeys(nullptr, tb, a, b, nnz, 0, bits, st));
            if (tb > cap || !scratch.p) {
                if (scratch.p) SD_CUDA_TRY(cudaFree(scratch.p));
                scratch.p = nullptr;
                SD_CUDA_TRY(scratch.get(tb));
                cap = tb;
            }
            SD_CUDA_TRY(cub::DeviceRadixSort::SortKeys(scratch.p, tb, a, b, nnz, 0, bits, st));
            SD_CUDA_TRY(cudaMemsetAsync(&dacc->distinct, 0, sizeof(unsigned long long), st));
            feat_distinct_kernel<<<grid_for(nnz, 1024), 256, 0, st>>>(b, nnz, dacc);
            SD_CUDA_TRY(cudaGetLastError());
            unsigned long long d = 0;
            SD_CUDA_TRY(cudaMemcpyAsync(&d, &dacc->distinct, sizeof d, cudaMemcpyDeviceToHost, st));
            SD_CUDA_TRY(cudaStreamSynchronize(st));
            nnzb[w] = static_cast<int64_t>(d);
        }
    }
    FeatAccum h;
    SD_CUDA_TRY(cudaMemcpyAsync(&h, dacc, sizeof h, cudaMemcpyDeviceToHost, st));
    SD_CUDA_TRY(cudaStreamSynchronize(st));
    out->col_max = static_cast<int64_t>(h.col_max);
    out->col_empty = static_cast<int64_t>(h.col_empty);
    out->sum_d2 = h.sum_d2;
    for (int w = 0; w < 3; ++w) out->sell_slots[w] = static_cast<int64_t>(h.sell[w]);
    out->nnzb4 = nnzb[0];
    out->nnzb8 = nnzb[1];
    return SD_OK;
}

}  // namespace sd
