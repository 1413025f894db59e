// Family (c), SIMT form: BSR-16 block-row kernel on the ordinary FP32 pipes.  It serves the
// BSR representation whenever the tensor-core kernel cannot (operands that break the TMA
// alignment rules, dense widths it does not cover) -- the paper's nemeth26 case keeps such
// a SIMT block-row plan beside its tensor-core candidate.
#pragma once

#include "sd_common.cuh"
#include "sd_launch.cuh"

namespace sd {

template <> struct RowLoad<__nv_bfloat16, 4> {
    __device__ __forceinline__ static void ld(const __nv_bfloat16 *p, float (&o)[4]) {
        const uint2 v = __ldg(reinterpret_cast<const uint2 *>(p));
        o[0] = __uint_as_float(v.x << 16);
        o[1] = __uint_as_float(v.x & 0xFFFF0000u);
        o[2] = __uint_as_float(v.y << 16);
        o[3] = __uint_as_float(v.y & 0xFFFF0000u);
    }
};

constexpr int kBsrSimtThreads = 64;

// One CTA per (block-row, slab of 64*VW columns); a thread owns VW columns of all 16 rows.
template <typename T, int VW>
__global__ void __launch_bounds__(kBsrSimtThreads)
bsr_simt_kernel(const BsrArgs a) {
    __shared__ __align__(16) float As[16][16];
    const int I = blockIdx.x;
    const int c0 = (blockIdx.y * kBsrSimtThreads + threadIdx.x) * VW;
    const bool colok = c0 < a.N;
    const T *__restrict__ bval = static_cast<const T *>(a.bval);
    const T *__restrict__ B = static_cast<const T *>(a.B);

    float acc[16][VW];
#pragma unroll
    for (int r = 0; r < 16; ++r)
#pragma unroll
        for (int e = 0; e < VW; ++e) acc[r][e] = 0.f;

    const int b0 = __ldg(a.browptr + I), b1 = __ldg(a.browptr + I + 1);
    for (int b = b0; b < b1; ++b) {
        __syncthreads();
        for (int i = threadIdx.x; i < 256; i += kBsrSimtThreads)
            As[i >> 4][i & 15] = to_float(bval[static_cast<int64_t>(b) * 256 + i]);
        __syncthreads();
        const int64_t krow0 = static_cast<int64_t>(__ldg(a.bcol + b)) * 16;
        if (colok) {
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                if (krow0 + k < a.K) {
                    float bv[VW];
                    RowLoad<T, VW>::ld(B + (krow0 + k) * a.ldb + c0, bv);
#pragma unroll
                    for (int r = 0; r < 16; ++r) {
                        const float av = As[r][k];
#pragma unroll
                        for (int e = 0; e < VW; ++e) acc[r][e] = fmaf(av, bv[e], acc[r][e]);
                    }
                }
            }
        }
    }
    if (colok) {
#pragma unroll
        for (int r = 0; r < 16; ++r) {
            const int64_t row = static_cast<int64_t>(I) * 16 + r;
            if (row < a.M) store_cols<VW>(a.C + row * a.ldc + c0, acc[r], a.alpha, a.beta, 0);
        }
    }
}

template <typename T>
cudaError_t launch_bsr_simt(const BsrArgs &a, bool vec, cudaStream_t st) {
    const int vw = vec ? 4 : 1;
    dim3 grid(static_cast<unsigned>(a.Mb), static_cast<unsigned>((a.N + kBsrSimtThreads * vw - 1) / (kBsrSimtThreads * vw)));
    if (vec) bsr_simt_kernel<T, 4><<<grid, kBsrSimtThreads, 0, st>>>(a);
    else bsr_simt_kernel<T, 1><<<grid, kBsrSimtThreads, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace sd
