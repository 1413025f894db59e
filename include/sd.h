/*
 * sd.h -- C ABI of the structure-adaptive SpMM library for NVIDIA B200 (sm_100a).
 *
 *     C = alpha * A * B + beta * C
 *
 * A is an M x K sparse matrix in CSR (32-bit indices; fp32 values, or bf16 values
 * that are multiplied exactly and accumulated in fp32), B is a row-major dense
 * K x N matrix in the same dtype as A's values, C is a row-major dense M x N fp32
 * matrix.  This is the SpMM of the paper's Sec. 2.1 ("SpMM computes C = AB with a
 * dense matrix B of width K"; the paper's dense width K is called N here, and K is
 * the column count of A).  N = 1 is SpMV.  alpha and beta follow the BLAS
 * convention; the paper's operator is alpha = 1, beta = 0.
 *
 * The three calls mirror the preprocess / compute / cleanup harness of the
 * paper's generated implementations (Appendix "A Generated SpMM Implementation"):
 * sd_plan_create analyses the sparsity pattern once (Sec. 3.1: row-length
 * statistics, column spread, occupied 16x16 tiles), chooses a representation and a
 * schedule -- the compilation plan <R, S, theta_H> of Sec. 3, Eq. 2, with fixed
 * integer rules in place of the paper's learned ranking and search -- and builds
 * it; sd_spmm executes it any number of times with different dense operands;
 * sd_plan_destroy releases it.
 *
 * Conventions for every call
 *  - Pointers named rowptr, colind, vals, B, C are DEVICE pointers on the current
 *    CUDA device unless the parameter says "host".  Sizes are element counts.
 *  - Errors are return codes.  Nothing throws, aborts or traps.  The last error
 *    message of the calling thread is kept for sd_last_error().
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 */
#ifndef SD_H_
#define SD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sd_plan sd_plan_t; /* opaque, library-owned */

typedef enum {
    SD_OK = 0,
    SD_ERR_INVALID_ARG = 1, /* null pointer, negative size, ld < N, bad enum, invalid CSR */
    SD_ERR_UNSUPPORTED = 2, /* valid request this build cannot serve */
    SD_ERR_ALLOC = 3,       /* device or host allocation failed */
    SD_ERR_CUDA = 4,        /* a CUDA call failed; text in sd_last_error */
    SD_ERR_INTERNAL = 5
} sd_status_t;

typedef enum { SD_F32 = 0, SD_BF16 = 1 } sd_dtype_t; /* dtype of vals AND of B */

/* Kernel families (paper Sec. 3.2 lists the SpMM template set CSR, COO, BSR-4/8/16,
 * Blocked-ELL, DTC; this library keeps a row-wise CSR family, an nnz-balanced
 * family in the spirit of COO / merge-based decompositions, and BSR-16). */
typedef enum {
    SD_AUTO = 0,     /* decide from the structure summary */
    SD_ROWSPLIT = 1, /* sub-warp per row, vectorised gathers of B rows */
    SD_MERGE = 2,    /* merge-path split of (row ends + nonzeros), segmented reduction,
                        deterministic carry-out fix-up; or its class split (sd_plan_info_t.class_split:
                        the (row, column window) segments re-bucketed window by window, long ones as
                        128-nonzero chunks, short ones one lane group each, one-nonzero ones flat),
                        chosen by dense width and forced with windows = -1 */
    SD_BSR_TC = 3,   /* 16x16 blocks on the tensor cores (tcgen05 / TMEM / TMA) */
    SD_HYBRID = 4    /* the schedule of the paper's appendix listing (light rows row-wise, heavy rows in
                        chunks), without its atomics: rows below heavy_len nonzeros are summed row-wise,
                        several rows per lane group, longest first; every heavy row is cut, column window by
                        column window, into chunks of at most 128 nonzeros of the caller's own CSR arrays
                        (no re-bucketed copy of A), the chunks are summed window-major into scratch rows
                        and one warp (or CTA) per heavy row adds its scratch rows in order.  Three launches
                        at most (one kernel for all rows, then the chunk sums), on the caller's stream only;
                        plan memory of a few tens of bytes per row.  Needs ascending columns.  AUTO takes
                        it in place of SD_MERGE (measured rule): without column windows from 5 columns up to
                        rows of B of 384 bytes (fp32 values) or 256 bytes (bf16 values) when the call gathers
                        at least 256 MiB, with column windows where a row of B is 64 to 192 (128) bytes */
} sd_family_t;

/* Options of sd_plan_create_ex.  Zero-initialise, then set fields. */
typedef struct {
    const int32_t *rowptr; /* device, [M+1], non-decreasing, rowptr[0] == 0 */
    const int32_t *colind; /* device, [nnz], 0 <= col < K */
    const void *vals;      /* device, [nnz], float or bf16 per `dtype` */
    int64_t M, K, N;       /* N: dense width the plan is tuned for (other widths still run) */
    int32_t dtype;         /* sd_dtype_t */
    int32_t family;        /* sd_family_t; SD_AUTO applies the rule */
    int32_t windows;       /* column windows of the MERGE family: 0 = automatic, 1 = off, 2..64;
                              -1 = one window, but with the class split of the window-major schedule */
    int32_t validate;      /* != 0: check rowptr monotone and 0 <= col < K on the device first */
    void *stream;          /* stream for the analysis kernels (plan creation still synchronises) */
    int32_t test_wait_expiry; /* TEST ONLY, leave 0.  != 0: in the tensor-core kernel of an SD_BSR_TC plan the first CTA's
                              copy thread never fills its ring, and every wait gives up after a few thousand polls
                              instead of a million: the kernel must return by itself, sd_plan_device_status must
                              report a non-zero code, C is left incomplete */
    int32_t heavy_len;     /* SD_HYBRID: rows of at least this many nonzeros run as chunks; 0 = the library's default
                              (256, the long-row threshold of the paper's appendix listing); clamped to 2 .. 256 */
} sd_plan_desc_t;

/* Integer structure summary (Sec. 3.1 "Intrinsic pattern features", Eq. 4) and the
 * decision taken from it.  All counts are exact integers. */
typedef struct {
    int64_t M, K, N, nnz;
    int64_t row_hist[32];   /* bin 0: r == 0; bin b >= 1: 2^(b-1) <= r < 2^b   (r = row length) */
    uint64_t sum_r2;        /* sum of r_i^2 */
    int64_t max_r;
    int64_t empty_rows;
    uint64_t sum_span;      /* sum over non-empty rows of (max col - min col + 1) */
    int64_t max_span;
    uint64_t sum_gap;       /* sum over non-empty rows of (max col - min col) */
    int64_t diag;           /* stored entries with col == row */
    int64_t unsorted_rows;  /* rows with an adjacent pair col[p+1] <= col[p] */
    int64_t long_rows;      /* rows with r >= 256 */
    int64_t nnz_long_rows;  /* nonzeros in those rows */
    int64_t nnzb16;         /* occupied 16x16 blocks (Eq. 4, nnzb_16) */
    int64_t blk_hist[9];    /* per-block entry count: [1],[2,3],[4,7],...,[128,255],[256+] */
    int64_t nnz_dense_blocks; /* nonzeros in blocks holding >= 128 entries */
    /* decision and schedule parameters (theta_H of Eq. 2) */
    int32_t family;         /* sd_family_t actually built */
    int32_t dtype;
    int32_t windows;        /* column windows in use (1 = none) */
    int32_t tile_items;     /* merge items (row ends + nonzeros) per CTA tile, MERGE only */
    int64_t num_tiles;      /* MERGE: total tiles over all windows.  HYBRID: number of heavy rows */
    int64_t num_segments;   /* MERGE: rows, or (row, window) pairs with the class split.  HYBRID: number of chunks */
    int64_t plan_bytes;     /* device memory owned by the plan */
    int32_t sm_count;       /* hardware context read at plan time (Sec. 3.1) */
    int32_t launches;       /* kernel launches one sd_spmm call issues on the vectorised path */
    int64_t l2_bytes;
    int32_t class_split;    /* MERGE: 1 when the segments run by class (long ones as chunks, short ones one
                               lane group each, one-nonzero ones flat) instead of merge-path tiles: always
                               with windows > 1, and with one window where that alone pays */
    int32_t heavy_len;      /* HYBRID: rows of at least this many nonzeros run as chunks (0 for the other families) */
} sd_plan_info_t;

/* sd_plan_create -- Sec. 3 (task <X, o, H> in, specialised implementation out) and
 * the `preprocess` entry of the paper's harness.  fp32 values, automatic family.
 *   rowptr, colind, vals  device pointers, BORROWED: they must stay allocated and
 *                         unchanged until sd_plan_destroy.
 *   M, K                  shape of A;  N  dense width to tune for.
 * Synchronous; allocates device memory owned by the plan.  Returns NULL on failure
 * (reason through sd_last_error). */
sd_plan_t *sd_plan_create(const int32_t *rowptr, const int32_t *colind, const float *vals,
                          int64_t M, int64_t K, int64_t N);

/* sd_plan_create_ex -- same, with dtype, forced family, window count, validation.
 * *out receives the plan.  SD_ERR_INVALID_ARG for null desc/out, negative sizes,
 * null CSR pointers with M > 0, unknown enums, or (validate != 0) a malformed CSR. */
sd_status_t sd_plan_create_ex(const sd_plan_desc_t *desc, sd_plan_t **out);

/* sd_spmm -- the `compute` entry: C = alpha*A*B + beta*C on `stream`.
 *   B    device, row-major [K, ldb], dtype of the plan, read-only, must not alias C
 *   C    device, row-major [M, ldc] fp32, in/out; columns N..ldc-1 are never touched
 *   ldb, ldc >= N (elements).  N is the width given at plan creation.
 * beta == 0: C is not read (NaN/Inf in it do not propagate).  alpha == 0: C = beta*C
 * without reading A or B.  M == 0 or N == 0: SD_OK, nothing launched.  Empty rows
 * get beta*C.  Asynchronous: launches only, no allocation, no synchronisation.
 * 16-byte aligned B/C with N, ldb, ldc multiples of the vector width take the
 * vectorised kernels; anything else takes scalar kernels (never an error).
 * With column windows the call issues one kernel sequence per window, in order, and C is
 * updated window by window.  Window-major plans run part of their kernels on plan-owned
 * streams that are forked from `stream` and joined back into it before the call returns, so that
 * everything is ordered after what `stream` held before the call and before what is queued on it
 * afterwards (a stream capture of `stream` therefore takes the whole call into its graph).  A plan
 * must not run concurrently on two streams or from two host threads (it owns scratch, streams and
 * events).
 * Results are run-to-run bit-identical (no floating-point atomics). */
sd_status_t sd_spmm(const sd_plan_t *plan, const void *B, int64_t ldb, float *C, int64_t ldc,
                    float alpha, float beta, void *stream);

/* sd_plan_update_values -- new values for the SAME sparsity pattern (paper, Appendix "A Generated
 * SpMM Implementation": the structure-only part of the preprocessing is reusable; e.g. edge weights
 * that change between the epochs of a graph network).
 *   vals   device [nnz], dtype of the plan, in the order of the colind array given at creation;
 *          borrowed from now on in place of the previous array (which may be freed once the
 *          work queued on `stream` has run)
 * Row-split and row-ordered merge plans only swap the pointer; window-major plans refresh
 * their re-bucketed copy, block plans refill the 16x16 blocks and the tensor-core images, both
 * with kernels on `stream`: order the call before the next sd_spmm (same stream, or an event).
 * The family, the windows and every structural decision stay as they are. */
sd_status_t sd_plan_update_values(sd_plan_t *plan, const void *vals, void *stream);

/* sd_spmm_host -- same operation with HOST buffers: B (and C when beta != 0) are
 * copied to plan-owned device staging buffers, sd_spmm runs, C is copied back, and
 * the call returns after the copy completed.  The staging buffers are allocated by
 * the first such call on a plan.  Pinned host memory gives full PCIe speed. */
sd_status_t sd_spmm_host(sd_plan_t *plan, const void *B_host, int64_t ldb, float *C_host,
                         int64_t ldc, float alpha, float beta);

/* sd_spmm_host_async / sd_plan_sync -- sd_spmm_host in two halves.  The first queues the
 * copies and the kernels on the plan's own stream and returns; B_host and C_host must stay
 * valid and untouched until sd_plan_sync(plan) has returned, which waits for everything
 * queued on that stream.  Calls on DIFFERENT plans overlap on the GPU and on the bus: one
 * plan's result travels to the host while the next plan's operand travels to the device
 * (pinned host memory is needed for that).  Several calls on the same plan run one after the
 * other; they share its staging buffers. */
sd_status_t sd_spmm_host_async(sd_plan_t *plan, const void *B_host, int64_t ldb, float *C_host,
                               int64_t ldc, float alpha, float beta);
sd_status_t sd_plan_sync(sd_plan_t *plan);

/* sd_plan_save / sd_plan_load -- keep the outcome of the analysis across processes (paper Sec. 3.4, last
 * paragraph: the winning implementation is cached per sparsity pattern, operator, platform and dense width, so
 * that later calls skip the search; here the "implementation" is the plan: family, schedule parameters and the
 * structure-only representation -- tile tables, window-major segment lists, block lists).
 * The blob is keyed by (hash of rowptr and colind, N, value type, device model): sd_plan_load recomputes the
 * hash of the arrays it is given (one pass over them on the device, no sort) and refuses a blob made for
 * another pattern (SD_ERR_INVALID_ARG) or another GPU model (SD_ERR_UNSUPPORTED).  Values are NOT in the
 * blob: the loaded plan takes them from `vals` as sd_plan_update_values would, so a pattern whose weights
 * changed since the save loads fine.
 *   sd_plan_save   buf == NULL: only *bytes (the size needed) is set.  Else `cap` >= that size; host buffer.
 *                  Synchronous (device-to-host copies).
 *   sd_plan_load   blob: host.  rowptr / colind / vals: device, borrowed like at creation, dtype and shapes as
 *                  saved.  *out receives a plan equivalent to the saved one: same sd_plan_get_info, same
 *                  representation, bit-identical sd_spmm results. */
sd_status_t sd_plan_save(const sd_plan_t *plan, void *buf, size_t cap, size_t *bytes);
sd_status_t sd_plan_load(const void *blob, size_t bytes, const int32_t *rowptr, const int32_t *colind,
                         const void *vals, sd_plan_t **out);

/* sd_plan_destroy -- the `cleanup` entry.  Frees everything the plan owns.  NULL is a no-op. */
void sd_plan_destroy(sd_plan_t *plan);

/* sd_plan_get_info -- structure summary and decision (host struct out). */
sd_status_t sd_plan_get_info(const sd_plan_t *plan, sd_plan_info_t *out);

/* Extended structure analysis (Sec. 3.1: row-length quartiles, column-degree statistics,
 * the value-slot expansion of padded and blocked layouts of Eq. 4 with their storage
 * estimates; Sec. 3.3, Eq. 10-13: footprint, working sets, work units).  Exact integers;
 * ratios (rho = slots / nnz, q_R = m_r / l2_bytes, ...) are left to the caller.
 * Quartiles are nearest-rank: the ceil(q*n/4)-th smallest of n values, q = 1, 2, 3
 * (0 when n == 0).  SELL slices are c consecutive rows in storage order (no sorting
 * window); the last slice may be shorter and counts its own rows only. */
typedef enum {
    SD_SHAPE_UNIFORM = 0,  /* CV^2 <= 1/16 */
    SD_SHAPE_MODERATE = 1, /* none of the others */
    SD_SHAPE_SKEWED = 2,   /* CV^2 >= 1 */
    SD_SHAPE_POWERLAW = 3, /* CV^2 >= 4 and max r >= 64 x mean r */
    SD_SHAPE_BIMODAL = 4   /* two row_hist bins at least 3 apart hold >= 1/4 of the non-empty rows each */
} sd_shape_t;              /* tested in the order UNIFORM, BIMODAL, POWERLAW, SKEWED, MODERATE */

typedef struct {
    int64_t row_q[3];      /* quartiles of the row length r_i over the M rows */
    int64_t col_q[3];      /* quartiles of the column degree d_j over the K columns */
    int64_t col_max;       /* max_j d_j */
    int64_t col_empty;     /* columns without a stored entry */
    uint64_t sum_d2;       /* sum of d_j^2 */
    int64_t ell_slots;     /* M * max_i r_i                          (rho_ELL numerator) */
    int64_t sell_slots[3]; /* sum over slices |s| max_{i in s} r_i,  c = 16, 32, 512 */
    int64_t nnzb[3];       /* occupied b x b blocks,                 b = 4, 8, 16 */
    /* storage estimates, value type of the plan, 32-bit indices:
     * [0] CSR (vb+4) nnz + 4 (M+1);  [1] ELL (vb+4) slots;
     * [2..4] SELL-16/32/512 (vb+4) slots + 4 (slices+1);
     * [5..7] BSR-4/8/16 (vb b^2 + 4) nnzb + 4 (ceil(M/b)+1) */
    int64_t rep_bytes[8];
    int32_t shape_class;   /* sd_shape_t */
    int32_t value_bytes;   /* vb: 4 or 2 */
    /* the plan as built (Eq. 10-13) */
    int64_t borrowed_bytes; /* caller's CSR arrays that sd_spmm reads: all three for SD_ROWSPLIT and for
                               SD_MERGE without the class split, none otherwise */
    int64_t plan_bytes;     /* device memory owned by the plan: representation, tables, scratch */
    int64_t d_r, d_s;       /* dense B: K N vb;  dense C: 4 M N */
    int64_t m_r, m_t;       /* m_r = borrowed + plan + d_r;  m_t = m_r + d_s */
    int64_t work_units;     /* rows (SD_ROWSPLIT), tiles (SD_MERGE), (row, window) segments (SD_MERGE with
                               the class split), block-rows (SD_BSR_TC) */
    int32_t sm_count;
    int32_t reserved;
    int64_t l2_bytes;
} sd_features_t;

/* sd_plan_get_features -- computes the analysis above on the device at the first call
 * (a few sorts over M, K and nnz keys: temporary device memory of about 40 bytes per nonzero,
 * freed before returning; synchronous) and keeps it in the plan.  Needs the CSR arrays given
 * at creation to be still valid.  Not thread-safe against other calls on the same plan. */
sd_status_t sd_plan_get_features(sd_plan_t *plan, sd_features_t *out);

/* sd_plan_get_bsr -- copy the BSR-16 representation (Sec. 3.1, Eq. 4) to HOST arrays:
 * browptr int32 [ceil(M/16)+1], bcol int32 [nnzb16] ascending inside a block-row,
 * bval [nnzb16][16][16] row-major in the plan dtype, absent slots +0.  Any pointer may
 * be NULL to skip it.  SD_ERR_UNSUPPORTED if the plan's family is not SD_BSR_TC. */
sd_status_t sd_plan_get_bsr(const sd_plan_t *plan, int32_t *browptr, int32_t *bcol, void *bval);

/* sd_plan_get_tiles -- MERGE family: copy the merge-path tile start coordinates to a HOST
 * array.  For window w (w = 0 when the plan uses no column windows) the merged list
 * interleaves the ends of that window's segments with its nonzeros; table entry t is the
 * (global) index of the first segment whose end lies at or after merged position
 * t * tile_items.  Window w owns ntiles_w + 1 consecutive entries and the windows are
 * concatenated.  `cap` is the capacity of tile_seg in elements; *count receives the number
 * of entries (also when tile_seg is NULL or too small).  SD_ERR_UNSUPPORTED for other
 * families. */
sd_status_t sd_plan_get_tiles(const sd_plan_t *plan, int32_t *tile_seg, int64_t cap, int64_t *count);

/* sd_plan_get_segments -- MERGE family with column windows (the paper's "packed column
 * windows", Sec. 3.4): copy the window-major representation to HOST arrays.  The columns are
 * cut into `windows` ranges of ceil(K / windows) columns; a segment is the part of one row
 * that falls into one window.  Inside a window the segments with more than 32 nonzeros come
 * first (they go to the merge-path kernel), then those with none or 2..32 (one lane group per
 * segment), then those with exactly one; rows ascend inside each class, except that the empty
 * rows are zero-length segments at the head of window 0's middle class.
 *   seg_ptr  int32 [num_segments + 1]  start of each segment in the re-bucketed arrays
 *   seg_row  int32 [num_segments]      output row; bit 31 set when an earlier window already
 *                                      wrote the row (this segment then adds to C)
 *   colind   int32 [nnz], vals [nnz]   nonzeros in window-major order (plan dtype)
 *   win_seg  int64 [3*windows + 1]     per window: first segment of each of the three classes;
 *                                      last entry = num_segments
 * Any pointer may be NULL.  SD_ERR_UNSUPPORTED when the plan does not use the class split. */
sd_status_t sd_plan_get_segments(const sd_plan_t *plan, int32_t *seg_ptr, int32_t *seg_row, int32_t *colind,
                                 void *vals, int64_t *win_seg);

/* sd_plan_get_hybrid -- HYBRID family: copy the schedule to HOST arrays (nl = info.num_tiles heavy rows,
 * nc = info.num_segments chunks, W = info.windows, window of a column = col / ceil(K / W)).
 *   heavy_rows  int32 [nl]       rows of at least info.heavy_len nonzeros, ascending
 *   chunk_ptr   int32 [nl + 1]   first chunk of every heavy row; chunks are numbered row by row, inside a row
 *                                window by window, inside a (row, window) piece by position
 *   ranges      int32 [nc][2]    nonzero range [begin, end) of every chunk in the caller's colind / vals:
 *                                a (row, window) piece of n nonzeros makes ceil(n / 128) chunks, all of 128
 *                                nonzeros but the last
 *   order       int32 [nc]       chunk numbers in the order the chunk kernel takes them: by window, then row,
 *                                then position
 *   light_rows  int32 [M - nl]   the other rows, longest first, ascending inside a length (rows without
 *                                nonzeros last)
 * Any pointer may be NULL.  SD_ERR_UNSUPPORTED for other families. */
sd_status_t sd_plan_get_hybrid(const sd_plan_t *plan, int32_t *heavy_rows, int32_t *chunk_ptr, int32_t *ranges,
                               int32_t *order, int32_t *light_rows);

/* sd_plan_device_status -- every wait inside the library's kernels (mbarrier waits of the
 * tensor-core kernel) is bounded; a wait that runs out makes its CTA record a non-zero code
 * in a plan-owned device word, release its resources and return, so the context stays
 * usable but C is then incomplete.  This call synchronises the device, copies the word to
 * *status (0 = no wait ever expired) and clears it. */
sd_status_t sd_plan_device_status(sd_plan_t *plan, int32_t *status);

/* sd_spmm_merge_static -- (no counterpart in the paper: an addition of this library.)
 * C = alpha*A*B + beta*C with the merge-path kernels, fp32, straight from the CSR arrays and
 * WITHOUT ANY ALLOCATION.  It is meant for callers that cannot let a library allocate device
 * memory: processes whose framework has already claimed the GPU's free memory for its own
 * pool, so that a late cudaMalloc fails or fragments it; latency-critical loops that cannot
 * take cudaMalloc's device-wide synchronisation; code under a fixed memory budget.  A plan
 * allocates its tile table and carry-out rows; here they live in one fixed 4 MiB array inside
 * the library's device image (every GPU that loads the library holds it until exit).
 *   rowptr [M+1], colind [nnz], vals [nnz]   device, as for sd_plan_create (rowptr[0] == 0 is
 *                                            relied upon, not checked); nnz = rowptr[M] is passed
 *                                            in so that nothing is read back
 *   B device [K, ldb] fp32, C device [M, ldc] fp32, ldb, ldc >= N; alpha/beta as sd_spmm.
 * Size limit: with T = ceil((M + nnz) / 1024) tiles, 4*(T+1) rounded up to 256, plus 8*T*N
 * bytes, must fit in 4 MiB (N = 32: about 16 million rows + nonzeros); beyond that the call
 * returns SD_ERR_UNSUPPORTED with the numbers in sd_last_error and launches nothing.
 * The first call on each device looks up the array's device address; make that first call
 * before any stream capture begins on the device.  All calls share the one array, which keeps
 * the previous call's contents (the call clears the part that must start from zero): two calls
 * whose kernels overlap on the GPU -- different streams, or different host threads -- race on
 * it and corrupt each other's results, so serialise them.  Asynchronous on `stream`. */
sd_status_t sd_spmm_merge_static(const int32_t *rowptr, const int32_t *colind, const float *vals,
                                 int64_t M, int64_t K, int64_t N, int64_t nnz, const float *B,
                                 int64_t ldb, float *C, int64_t ldc, float alpha, float beta,
                                 void *stream);

/* sd_last_error -- copy the calling thread's last error text into buf (NUL-terminated,
 * at most n bytes); returns the last status code. */
int sd_last_error(char *buf, size_t n);

/* sd_version -- "major.minor" text of this build. */
const char *sd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SD_H_ */
