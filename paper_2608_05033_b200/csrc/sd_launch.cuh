// Host entry points of the kernel families, one translation unit each.
#pragma once

#include "sd_common.cuh"

namespace sd {

// Every tile holds the same number of merged items whatever the lane geometry, so one tile
// table serves every dense width and both the vector and the scalar kernels.
constexpr int kMergeTile = 1024;

struct MergeArgs {
    SpmmArgs s;
    const int32_t *tile_seg;  // [ntiles + 1] segment coordinate of each tile start (global seg ids)
    float *tile_head;         // [ntiles][N]  partial of the segment open at tile start, if it ends here
    float *tile_tail;         // [ntiles][N]  partial of the segment still open at tile end
    int64_t seg_begin;        // first segment of this window
    int64_t seg_end;          // one past the last segment of this window
    int32_t ntiles;
};


// Family (a).  `vec`: B, C, ldb, ldc and N allow 16-byte accesses.
cudaError_t run_rowsplit(const SpmmArgs &a, int dtype, bool vec, cudaStream_t st);
cudaError_t run_hybrid_fused(const SpmmArgs &ca, const SpmmArgs &ma, const SpmmArgs &la, int dtype, bool vec, cudaStream_t st);

// One lane group per segment (a.seg_row: output rows), or per chunk of a long segment
// (`scratch`: chunk c writes its plain sum to row c of a.C).
cudaError_t run_segments(const SpmmArgs &a, int dtype, bool vec, bool scratch, cudaStream_t st);

// One-nonzero segments: segment s is nonzero s of a.colind / a.vals, a.seg_row[s] its output row.
cudaError_t run_single(const SpmmArgs &a, int dtype, bool vec, cudaStream_t st);

// Long segments of a window-major plan: segment s owns the scratch rows seg_chunk[s] ..
// seg_chunk[s+1]-1 of chunk_out ([chunks][N]); their sum, taken in order, updates C[seg_row[s]].
cudaError_t run_chunk_reduce(const float *chunk_out, const int32_t *seg_chunk, const int32_t *seg_row, int64_t seg_begin,
                             int64_t seg_end, float *C, int64_t ldc, int32_t N, float alpha, float beta, cudaStream_t st,
                             int32_t skip_above = 0);
constexpr int kGiantChunks = 64;   // segments of more chunks than this are summed by a whole CTA
cudaError_t run_chunk_reduce_wide(const float *chunk_out, const int32_t *seg_chunk, const int32_t *seg_row,
                                  const int32_t *list, int64_t count, float *C, int64_t ldc, int32_t N, float alpha,
                                  float beta, cudaStream_t st);

// C = beta * C.
cudaError_t preload_stream_kernels(int dtype, int32_t N);
cudaError_t run_scale_c(float *C, int64_t ldc, int64_t M, int32_t N, float beta, cudaStream_t st);

// Family (b): tile kernel, then the carry-out fix-up for the listed tiles (short chains one per
// warp, long chains one per CTA).
cudaError_t run_merge(const MergeArgs &m, int dtype, bool vec, const int32_t *fix_short, int32_t nshort,
                      const int32_t *fix_long, int32_t nlong, cudaStream_t st);
constexpr int kMergeLongChain = 8;   // chains of at least this many tiles go to the per-CTA fix-up

// Family (b) for dense widths up to kCooMaxN (beyond it the shuffles per nonzero outweigh the
// gain; measured cross-over between 4 and 8 columns): segmented reduction over the nonzeros with an
// explicit row index per nonzero, carries reduced in two more levels.
constexpr int kCooMaxN = 4;
// nonzeros per warp step: 8 per lane at one or two columns (the gathers are 4 or 8 bytes: more of them
// must be in flight; measured), 4 per lane at three or four; carry lists are always cut into 128-entry chunks
constexpr int coo_chunk(int N) { return N <= 2 ? 256 : 128; }
constexpr int kCooCarryChunk = 128;
constexpr int64_t kCooDirectFinal = 4096;  // carry lists up to this length skip the second level
struct CooPlan {
    const int32_t *row;   // [nnz] row of every nonzero
    const int32_t *rowptr; // [M + 1]
    int64_t M;             // rows to search for empty ones (0: the matrix has none)
    int64_t nnz;
    int32_t *c1_row;      // [2 * ceil(nnz / coo_chunk(N))] first-level carries
    float *c1_val;        // ... x N
    int32_t *c2_row;      // [2 * ceil(len(c1) / kCooCarryChunk)] second-level carries
    float *c2_val;
};
cudaError_t run_coo(const CooPlan &cp, const SpmmArgs &s, int dtype, bool vec, int sm_count, cudaStream_t st);
cudaError_t build_coo_rows(const int32_t *rowptr, int64_t M, int64_t nnz, int32_t *row, cudaStream_t st);

// Family (c).
// The TMA descriptor of B as the tensor-core kernel reads it, kept by the plan for the last (B, ldb) it ran with:
// encoding one costs a driver call on the host, and a serving loop calls sd_spmm with the same operand buffer.
struct alignas(64) TcMapCache {
    unsigned char map[128];   // a CUtensorMap
    const void *B = nullptr;
    int64_t ldb = 0, K = 0;
    int32_t N = 0;
    int32_t valid = 0;
};
struct BsrArgs {
    const int32_t *browptr;  // [Mb + 1]
    const int32_t *bcol;     // [nnzb]
    const void *bval;        // [nnzb][16][16] row-major, plan dtype
    const void *bval_mma;    // [nnzb] tensor-core operand images of the same blocks
    const int32_t *part;     // [nparts + 1] block-row ranges of the tensor-core kernel's CTAs
    int32_t nparts;
    const void *B;
    float *C;
    int64_t ldb, ldc;
    int64_t M, K;
    int32_t Mb;
    int32_t N;
    float alpha, beta;
    TcMapCache *map_cache;      // may be null: the descriptor is then encoded for this call only
    int32_t test_wait_expiry;   // see sd_plan_desc_t
};
cudaError_t run_bsr_simt(const BsrArgs &a, int dtype, bool vec, cudaStream_t st);
// Tensor-core form.  bsr_tc_usable: dtype, dense width and the TMA alignment rules allow it.
bool bsr_tc_usable(const BsrArgs &a, int dtype);
cudaError_t run_bsr_tc(const BsrArgs &a, int dtype, int32_t *error_word, int sm_count, cudaStream_t st);
// Counts behind sd_plan_get_features (row-length / column-degree quartiles, column-degree moments,
// SELL slots for slice heights 16 / 32 / 512, occupied 4x4 and 8x8 blocks).  Synchronous.
struct FeatureCounts {
    int64_t row_q[3], col_q[3], col_max, col_empty;
    uint64_t sum_d2;
    int64_t sell_slots[3];
    int64_t nnzb4, nnzb8;
};
sd_status_t compute_feature_counts(const int32_t *rowptr, const int32_t *colind, int64_t M, int64_t K, int64_t nnz,
                                   cudaStream_t st, FeatureCounts *out);

cudaError_t build_bsr_partition(const int32_t *browptr, int32_t Mb, int32_t nparts, int32_t *part, cudaStream_t st);
cudaError_t build_bsr_mma_image(const void *bval, void *img, int64_t nnzb, int dtype, cudaStream_t st);

}  // namespace sd
