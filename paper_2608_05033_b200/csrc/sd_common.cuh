// Shared device/host helpers of the SpMM library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <atomic>

#include "../../include/sd.h"

namespace sd {

// ---- error reporting (thread-local text + code) --------------------------------
void set_error(sd_status_t code, const char *fmt, ...);
sd_status_t cuda_fail(cudaError_t e, const char *what);

#define SD_CUDA_TRY(expr)                                   \
    do {                                                    \
        cudaError_t e__ = (expr);                           \
        if (e__ != cudaSuccess) return cuda_fail(e__, #expr); \
    } while (0)

// ---- element access -------------------------------------------------------------
__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// Vector width in elements of a 16-byte load of T.
template <typename T> struct vec_width;
template <> struct vec_width<float> { static constexpr int value = 4; };
template <> struct vec_width<__nv_bfloat16> { static constexpr int value = 8; };

// Load VW consecutive elements of T (read-only path) and widen to float.
template <typename T, int VW> struct RowLoad;

template <> struct RowLoad<float, 4> {
    __device__ __forceinline__ static void ld(const float *p, float (&o)[4]) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(p));
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
};
template <> struct RowLoad<float, 1> {
    __device__ __forceinline__ static void ld(const float *p, float (&o)[1]) { o[0] = __ldg(p); }
};
template <> struct RowLoad<__nv_bfloat16, 8> {
    __device__ __forceinline__ static void ld(const __nv_bfloat16 *p, float (&o)[8]) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(p));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {       // bf16 is the upper half of a float
            o[2 * i] = __uint_as_float(w[i] << 16);
            o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
};
template <> struct RowLoad<__nv_bfloat16, 1> {
    __device__ __forceinline__ static void ld(const __nv_bfloat16 *p, float (&o)[1]) {
        o[0] = __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short *>(p))) << 16);
    }
};

// Rows of B are what the kernels re-read: an L2 policy that evicts them last keeps more of B
// resident against the streams of A and C (measured on the GCN workload: 5 to 19 % less time).
__device__ __forceinline__ uint64_t l2_keep_policy() {
    uint64_t pol;
    asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// RowLoad with that policy.
template <typename T, int VW> struct RowLoadKeep;
template <> struct RowLoadKeep<float, 4> {
    __device__ __forceinline__ static void ld(const float *p, float (&o)[4], uint64_t pol) {
        asm("ld.global.nc.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
            : "=f"(o[0]), "=f"(o[1]), "=f"(o[2]), "=f"(o[3])
            : "l"(p), "l"(pol));
    }
};
template <> struct RowLoadKeep<float, 1> {
    __device__ __forceinline__ static void ld(const float *p, float (&o)[1], uint64_t pol) {
        asm("ld.global.nc.L2::cache_hint.f32 %0, [%1], %2;" : "=f"(o[0]) : "l"(p), "l"(pol));
    }
};
template <> struct RowLoadKeep<__nv_bfloat16, 8> {
    __device__ __forceinline__ static void ld(const __nv_bfloat16 *p, float (&o)[8], uint64_t pol) {
        uint32_t w[4];
        asm("ld.global.nc.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
            : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3])
            : "l"(p), "l"(pol));
#pragma unroll
        for (int i = 0; i < 4; ++i) {       // bf16 is the upper half of a float
            o[2 * i] = __uint_as_float(w[i] << 16);
            o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
};
template <> struct RowLoadKeep<__nv_bfloat16, 1> {
    __device__ __forceinline__ static void ld(const __nv_bfloat16 *p, float (&o)[1], uint64_t pol) {
        unsigned short h;
        asm("ld.global.nc.L2::cache_hint.u16 %0, [%1], %2;" : "=h"(h) : "l"(p), "l"(pol));
        o[0] = __uint_as_float(static_cast<uint32_t>(h) << 16);
    }
};

// How one output row leaves the registers.
//   mode 0: C = alpha*acc + beta*C   (first and only write of the row; beta == 0 never reads C)
//   mode 1: C = C + alpha*acc        (later column window of a row already written)
template <int VW>
__device__ __forceinline__ void store_cols(float *c, const float (&acc)[VW], float alpha, float beta,
                                           int accumulate) {
    if constexpr (VW == 1) {
        float r = alpha * acc[0];
        if (accumulate) r += *c;
        else if (beta != 0.f) r += beta * *c;
        *c = r;
    } else {
#pragma unroll
        for (int q = 0; q < VW / 4; ++q) {
            float4 *p = reinterpret_cast<float4 *>(c) + q;
            float4 r = make_float4(alpha * acc[4 * q], alpha * acc[4 * q + 1], alpha * acc[4 * q + 2],
                                   alpha * acc[4 * q + 3]);
            if (accumulate) {
                const float4 o = *p;
                r.x += o.x; r.y += o.y; r.z += o.z; r.w += o.w;
            } else if (beta != 0.f) {
                const float4 o = *p;
                r.x += beta * o.x; r.y += beta * o.y; r.z += beta * o.z; r.w += beta * o.w;
            }
            __stcs(p, r);   // C is written once and not read again: streaming store, first to leave L2
        }
    }
}

// Address of row `col` of B given a per-lane base pointer: one 32 x 32 -> 64 bit multiply-add
// (column indices are non-negative and the row pitch in bytes is below 2^32, checked on the host).
template <typename T>
__device__ __forceinline__ const T *b_row(const T *base, int col, uint32_t ldb_bytes) {
    return reinterpret_cast<const T *>(reinterpret_cast<const char *>(base) +
                                       static_cast<uint64_t>(static_cast<uint32_t>(col)) * ldb_bytes);
}

// Arguments common to the CSR kernels.
struct SpmmArgs {
    const int32_t *ptr;     // row (or segment) pointer array, [S+1]
    const int32_t *colind;  // [nnz]
    const void *vals;       // [nnz] float or bf16
    const int32_t *seg_row; // nullptr: segment s is row s.  Else output row of segment s;
                            // bit 31 set: the row was already written by an earlier window.
    const void *B;
    float *C;
    int64_t ldb, ldc;
    uint32_t ldb_bytes;     // ldb * sizeof(element of B)
    int64_t S;              // number of rows / segments
    int32_t N;
    float alpha, beta;
    int64_t max_len;        // longest row / segment if known (0: unknown); lets the row-split kernel drop its second accumulator
    int64_t mean_len;       // mean row length rounded up if known (0: unknown): lanes per row of the narrow row-split kernel
    // hybrid family (light rows row-wise, heavy rows as chunks):
    bool load_only = false;          // host side only: the launcher loads the kernel instance it would launch and returns
    const int4 *desc = nullptr;      // light-rows kernel: {row, first nonzero, its column, length} of every row it takes
    const int2 *ranges = nullptr;    // chunk kernel: nonzero range [x, y) of every chunk (in the caller's CSR arrays) ...
    const int32_t *order = nullptr;  // ... and the order in which the chunks are taken (column-window-major); work item i is chunk order[i]
};

// A/B measurement switches (none is needed in normal use).  The environment is read once, at the
// first use in the process (thread-safe), never on the sd_spmm path.
struct Switches {
    bool no_coo;           // SD_NO_COO: generic merge kernel at one to four columns
    bool no_side_streams;  // SD_NO_SIDE_STREAMS: the classes of a window on one stream
    bool no_chunk_ahead;   // SD_NO_CHUNK_AHEAD: chunk kernels in window order
    bool bsr_simt;         // SD_BSR_SIMT: SIMT block kernel instead of the tensor-core one
    bool no_narrow;        // SD_NO_NARROW: wide row-split kernel at one to four columns
    int geom_nv;           // SD_GEOM_NV: 1 forces one vector per lane
    int ksplit_g;          // SD_KSPLIT_G: lane sets per row (0: rule, 1: off)
    int narrow_g;          // SD_NARROW_G: lanes per row of the narrow row-split kernel (0: rule)
    int tc_sb, tc_stages, tc32_sb, tc32_stages;   // SD_TC_SB / SD_TC_STAGES / SD_TC32_SB / SD_TC32_STAGES: ring geometry (0: default)
};
const Switches &switches();

// Per-device caches of launch facts (SM count, resident CTAs of a kernel instance, attributes already set):
// one slot per device ordinal, published with atomics, so that a process driving several GPUs, or several
// host threads making their first call together, never reads another device's value or a torn one.
constexpr int kMaxDevices = 64;
inline int current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) dev = 0;
    return dev;
}
inline int sm_count_cached() {
    static std::atomic<int> cache[kMaxDevices];
    const int dev = current_device();
    int v = dev < kMaxDevices ? cache[dev].load(std::memory_order_relaxed) : 0;
    if (v > 0) return v;
    v = 148;
    cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    if (dev < kMaxDevices) cache[dev].store(v, std::memory_order_relaxed);
    return v;
}
// CTAs of `kernel` (threads per CTA, no dynamic shared memory) that are resident together on one SM of the current device.
template <typename Kernel>
inline int occupancy_cached(std::atomic<int> (&cache)[kMaxDevices], Kernel kernel, int threads) {
    const int dev = current_device();
    int v = dev < kMaxDevices ? cache[dev].load(std::memory_order_relaxed) : 0;
    if (v > 0) return v;
    v = 8;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, kernel, threads, 0) != cudaSuccess || v < 1) v = v < 1 ? 1 : 8;
    if (dev < kMaxDevices) cache[dev].store(v, std::memory_order_relaxed);
    return v;
}

inline int ceil_div(int64_t a, int64_t b) { return static_cast<int>((a + b - 1) / b); }

}  // namespace sd
