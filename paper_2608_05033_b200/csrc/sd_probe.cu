// sd_probe_gather: a measurement aid.  It replays a stream of row indices (for instance the
// colind array of a CSR matrix) as bare row gathers from a dense table -- the memory access
// pattern of SpMM with everything else removed (no values of A, no multiply, no output rows) --
// so that the time of an SpMM kernel can be set against the rate at which the memory system can
// deliver that very gather stream.
#include "sd_common.cuh"

namespace sd {

// A group of LPR lanes fetches one row of LPR*16 bytes per index; groups stride over the index
// array; four gathers are in flight per lane; the sums keep the loads alive.
template <int LPR>
__global__ void __launch_bounds__(256)
probe_gather_kernel(const int32_t *__restrict__ idx, int64_t count, const float4 *__restrict__ table, uint32_t row_bytes,
                    float4 *__restrict__ sink) {
    const int lg = threadIdx.x % LPR;
    const int64_t g = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) / LPR;
    const int64_t G = (static_cast<int64_t>(gridDim.x) * blockDim.x) / LPR;
    const char *base = reinterpret_cast<const char *>(table + lg);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    // consecutive groups take consecutive runs of 4 indices, as consecutive lane groups of an
    // SpMM kernel take consecutive nonzeros
    for (int64_t i = g * 4; i < count; i += G * 4) {
        int r[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) r[u] = (i + u < count) ? __ldg(idx + i + u) : 0;
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
            v[u] = __ldg(reinterpret_cast<const float4 *>(base + static_cast<uint64_t>(static_cast<uint32_t>(r[u])) * row_bytes));
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (i + u < count) {   // the tail's stand-in loads of row 0 do not count
                acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w;
            }
        }
    }
    sink[(static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x)] = acc;
}

}  // namespace sd

using namespace sd;

extern "C" {
#pragma GCC visibility push(default)

sd_status_t sd_probe_gather(const int32_t *idx, int64_t count, const void *table, int32_t row_bytes, float *sink,
                            int32_t *sink_floats_needed, void *stream) {
    int dev = 0, sms = 148;
    SD_CUDA_TRY(cudaGetDevice(&dev));
    SD_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int blocks = sms * 8;   // 8 CTAs of 256 threads fill an SM
    if (sink_floats_needed) *sink_floats_needed = blocks * 256 * 4;
    if (!idx && !table && !sink) return SD_OK;   // size query
    if (!idx || !table || !sink || count < 0 ||
        !(row_bytes == 16 || row_bytes == 32 || row_bytes == 64 || row_bytes == 128 || row_bytes == 256 ||
          row_bytes == 512)) {
        set_error(SD_ERR_INVALID_ARG, "sd_probe_gather: null pointer, negative count, or row_bytes not in {16,...,512}");
        return SD_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float4 *t = static_cast<const float4 *>(table);
    float4 *s = reinterpret_cast<float4 *>(sink);
    const uint32_t rb = static_cast<uint32_t>(row_bytes);
    switch (row_bytes / 16) {
    case 1: probe_gather_kernel<1><<<blocks, 256, 0, st>>>(idx, count, t, rb, s); break;
    case 2: probe_gather_kernel<2><<<blocks, 256, 0, st>>>(idx, count, t, rb, s); break;
    case 4: probe_gather_kernel<4><<<blocks, 256, 0, st>>>(idx, count, t, rb, s); break;
    case 8: probe_gather_kernel<8><<<blocks, 256, 0, st>>>(idx, count, t, rb, s); break;
    case 16: probe_gather_kernel<16><<<blocks, 256, 0, st>>>(idx, count, t, rb, s); break;
    default: probe_gather_kernel<32><<<blocks, 256, 0, st>>>(idx, count, t, rb, s); break;
    }
    SD_CUDA_TRY(cudaGetLastError());
    return SD_OK;
}

#pragma GCC visibility pop
}  // extern "C"
