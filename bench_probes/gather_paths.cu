// Gather-path probes for bench.py (--probe, --probe-paths): a measurement aid, not part of the SpMM
// library and not linked into it.  Each kernel replays a stream of row indices (for instance the
// colind array of a CSR matrix, in storage order) as bare row gathers from a dense table -- the
// memory access pattern of SpMM with the values of A, the multiply-adds and the output removed --
// through one fetch path, so that the time of an SpMM kernel can be set against the rate at which
// the memory system delivers that very gather stream, and the fetch paths against one another.
//
// Every wait in here is bounded: on expiry the CTA records a code in *err, waits (bounded) for
// its own copies in flight and returns.
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <stdint.h>
namespace cg = cooperative_groups;

namespace {

__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
    asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
// MODE 0: plain read-only load   1: L2 evict-last hint   2: L1 no-allocate
template <int MODE>
__device__ __forceinline__ float4 load_vec(const char *p, uint64_t pol) {
    float4 v;
    if constexpr (MODE == 0) {
        v = __ldg(reinterpret_cast<const float4 *>(p));
    } else if constexpr (MODE == 1) {
        asm volatile("ld.global.nc.L2::cache_hint.v4.f32 {%0,%1,%2,%3}, [%4], %5;"
                     : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p), "l"(pol));
    } else {
        asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                     : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    }
    return v;
}
__device__ __forceinline__ void add4(float4 &a, const float4 &v) { a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w; }

// ---- grid-stride order: a group of LPR lanes fetches one row of LPR * 16 bytes per index; every group takes WB
// consecutive indices (all WB gathers in flight together), groups stride over the stream -----------------------
template <int LPR, int WB, int MODE, int OCC>
__global__ void __launch_bounds__(256, OCC) stride_kernel(const int *__restrict__ idx, long count, const char *__restrict__ table,
                                                          uint32_t row_bytes, float4 *__restrict__ sink) {
    const int lg = threadIdx.x % LPR;
    const long g = ((long)blockIdx.x * blockDim.x + threadIdx.x) / LPR;
    const long G = ((long)gridDim.x * blockDim.x) / LPR;
    const char *base = table + lg * 16;
    const uint64_t pol = policy_evict_last();
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (long i = g * WB; i < count; i += G * WB) {
        int r[WB];
#pragma unroll
        for (int u = 0; u < WB; ++u) r[u] = (i + u < count) ? __ldg(idx + i + u) : 0;
        float4 v[WB];
#pragma unroll
        for (int u = 0; u < WB; ++u) v[u] = load_vec<MODE>(base + (uint64_t)(uint32_t)r[u] * row_bytes, pol);
#pragma unroll
        for (int u = 0; u < WB; ++u)
            if (i + u < count) add4(acc, v[u]);   // the tail's stand-in loads of row 0 do not count
    }
    sink[(long)blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

// ---- tile order (512-byte rows): CTA t takes the 1,024-index tiles t, t + grid, ...; a warp takes 128 contiguous
// indices of a tile, staged in shared memory and read back as broadcasts, as the merge-path SpMM kernel does -----
template <int MODE>
__global__ void __launch_bounds__(256, 8) tile_kernel(const int *__restrict__ idx, long count, const char *__restrict__ table,
                                                      float4 *__restrict__ sink) {
    __shared__ int s_idx[1024];
    const int lg = threadIdx.x & 31, w = threadIdx.x >> 5;
    const char *base = table + lg * 16;
    const uint64_t pol = policy_evict_last();
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const long ntiles = (count + 1023) / 1024;
    for (long t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const long t0 = t * 1024;
        const int n = (int)min(1024L, count - t0);
        __syncthreads();
        for (int k = threadIdx.x; k < 1024; k += 256) s_idx[k] = (k < n) ? __ldcs(idx + t0 + k) : 0;
        __syncthreads();
        const int j1 = min((w + 1) * 128, n);
        for (int j = w * 128; j < j1; j += 4) {
            int r[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) r[u] = s_idx[min(j + u, 1023)];
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = load_vec<MODE>(base + (uint64_t)(uint32_t)r[u] * 512u, pol);
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (j + u < j1) add4(acc, v[u]);
        }
    }
    sink[(long)blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

// ---- half a warp per 512-byte row, two 16-byte vectors per lane: one load instruction of a warp touches two rows ----
__global__ void __launch_bounds__(256, 4) half_warp_kernel(const int *__restrict__ idx, long count, const char *__restrict__ table,
                                                           float4 *__restrict__ sink) {
    constexpr int WB = 4;
    const int lg = threadIdx.x & 15, h = (threadIdx.x >> 4) & 1;
    const long g = ((long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long G = ((long)gridDim.x * blockDim.x) >> 5;
    const char *base = table + lg * 16;
    float4 acc0 = make_float4(0.f, 0.f, 0.f, 0.f), acc1 = acc0;
    for (long i = g * 2 * WB; i < count; i += G * 2 * WB) {
        int r[WB];
#pragma unroll
        for (int u = 0; u < WB; ++u) r[u] = (i + 2 * u + h < count) ? __ldg(idx + i + 2 * u + h) : 0;
        float4 v[WB][2];
#pragma unroll
        for (int u = 0; u < WB; ++u) {
            v[u][0] = __ldg(reinterpret_cast<const float4 *>(base + (uint64_t)(uint32_t)r[u] * 512u));
            v[u][1] = __ldg(reinterpret_cast<const float4 *>(base + (uint64_t)(uint32_t)r[u] * 512u + 256));
        }
#pragma unroll
        for (int u = 0; u < WB; ++u)
            if (i + 2 * u + h < count) {
                add4(acc0, v[u][0]);
                add4(acc1, v[u][1]);
            }
    }
    // sink slot layout of this kernel: thread t holds columns (t % 16) * 4 .. +3 in [0] and 64 + the same in [1]
    sink[2 * ((long)blockIdx.x * blockDim.x + threadIdx.x)] = acc0;
    sink[2 * ((long)blockIdx.x * blockDim.x + threadIdx.x) + 1] = acc1;
}

// ---- bulk copies (cp.async.bulk, one 512-byte row each) into a shared-memory ring; eight consumer warps read the
// rows back with 16-byte shared loads -------------------------------------------------------------------------
constexpr int kBulkRows = 32;   // rows per ring slot
constexpr int kBulkCons = 8;    // consumer warps
constexpr int kBulkStages = 6;
constexpr uint32_t kSpin = 1u << 20;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {   // bounded
    for (uint32_t i = 0; i < kSpin; ++i) {
        uint32_t ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); }
__device__ __forceinline__ void mbar_expect(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__global__ void __launch_bounds__(32 * (kBulkCons + 1)) bulk_ring_kernel(const int *__restrict__ idx, long count,
                                                                        const char *__restrict__ table,
                                                                        float4 *__restrict__ sink, int *err) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t full[kBulkStages], empty[kBulkStages];
    __shared__ int s_err;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        for (int s = 0; s < kBulkStages; ++s) {
            mbar_init(smem_u32(&full[s]), 1);
            mbar_init(smem_u32(&empty[s]), kBulkCons);
        }
        s_err = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const long nb = (count + kBulkRows - 1) / kBulkRows;   // batches of 32 rows, CTA-strided
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (warp == kBulkCons) {
        // producer warp: every lane copies one row of the batch
        int armed = 0;
        bool ok = true;
        for (long b = blockIdx.x; b < nb; b += gridDim.x, ++armed) {
            const int s = armed % kBulkStages, it = armed / kBulkStages;
            if (it > 0) ok = mbar_wait(smem_u32(&empty[s]), (it - 1) & 1);
            ok = __all_sync(0xffffffffu, ok) && !*(volatile int *)&s_err;
            if (!ok) break;
            const long i = b * kBulkRows + lane;
            const int r = (i < count) ? __ldg(idx + i) : 0;
            if (lane == 0) mbar_expect(smem_u32(&full[s]), kBulkRows * 512);
            __syncwarp();
            const uint32_t dst = smem_u32(smem + (size_t)s * kBulkRows * 512 + lane * 512);
            const char *src = table + (uint64_t)(uint32_t)r * 512u;
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(dst), "l"(src), "r"(512), "r"(smem_u32(&full[s])) : "memory");
        }
        if (!ok && lane == 0) {
            s_err = 1;
            atomicExch(err, 1);
        }
        // copies in flight: wait (bounded) until every armed slot has landed before the CTA may leave
        if (lane == 0) {
            const int first = armed > kBulkStages ? armed - kBulkStages : 0;
            for (int a = first; a < armed; ++a) (void)mbar_wait(smem_u32(&full[a % kBulkStages]), (a / kBulkStages) & 1);
        }
    } else {
        int done = 0;
        for (long b = blockIdx.x; b < nb; b += gridDim.x, ++done) {
            const int s = done % kBulkStages, it = done / kBulkStages;
            const bool ok = mbar_wait(smem_u32(&full[s]), it & 1);
            if (!ok || *(volatile int *)&s_err) {
                if (lane == 0) {
                    s_err = 2;
                    atomicExch(err, 2);
                }
                break;
            }
            const float4 *rows = reinterpret_cast<const float4 *>(smem + (size_t)s * kBulkRows * 512);
#pragma unroll
            for (int q = 0; q < kBulkRows / kBulkCons; ++q) {
                const int rr = warp + q * kBulkCons;
                if (b * kBulkRows + rr < count) add4(acc, rows[rr * 32 + lane]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&empty[s]));
        }
    }
    sink[(long)blockIdx.x * blockDim.x + tid] = acc;
}

// ---- asynchronous 16-byte copies (cp.async) into a per-warp shared-memory ring: a gather in flight holds a ring slot
// instead of registers, so a warp can keep D rows (D * 512 bytes) in flight; every lane copies and later reads back
// its own 16 bytes of a row, so the warp needs no barrier.  Batches of WB rows are one commit group; NB = D / WB
// groups are in flight.  CG: copies bypass L1 (cp.async.cg), else they allocate in it (cp.async.ca) -----------------
template <int D, int WB, bool CG>
__global__ void __launch_bounds__(256) async_ring_kernel(const int *__restrict__ idx, long count, const char *__restrict__ table,
                                                        float4 *__restrict__ sink) {
    extern __shared__ __align__(16) char ring_mem[];
    constexpr int NB = D / WB;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    char *ring = ring_mem + (size_t)w * D * 512 + lane * 16;
    const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);
    const char *base = table + lane * 16;
    const long g = (long)blockIdx.x * 8 + w, G = (long)gridDim.x * 8;
    const long nbatch_all = (count + WB - 1) / WB;
    const long nb = nbatch_all > g ? (nbatch_all - g + G - 1) / G : 0;   // batches of this warp: g, g + G, ...
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    auto issue = [&](long k) {
        if (k < nb) {
            const long i = (g + k * G) * WB;
            int r[WB];
#pragma unroll
            for (int u = 0; u < WB; ++u) r[u] = (i + u < count) ? __ldg(idx + i + u) : -1;
#pragma unroll
            for (int u = 0; u < WB; ++u) {
                if (r[u] < 0) continue;
                const uint32_t dst = ring_s + (uint32_t)(((k % NB) * WB + u) * 512);
                const char *src = base + (uint64_t)(uint32_t)r[u] * 512u;
                if constexpr (CG) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
                else asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");   // one group per call, also when empty: uniform counting
    };
    for (long k = 0; k < NB; ++k) issue(k);
    for (long k = 0; k < nb; ++k) {
        asm volatile("cp.async.wait_group %0;" ::"n"(NB - 1) : "memory");   // batch k has landed
        const long i = (g + k * G) * WB;
#pragma unroll
        for (int u = 0; u < WB; ++u)
            if (i + u < count) add4(acc, *reinterpret_cast<const float4 *>(ring + ((k % NB) * WB + u) * 512));
        issue(k + NB);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    sink[(long)blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

// ---- hub rows in distributed shared memory: a cluster of CL CTAs (one per SM) keeps CL * kHubRows hot rows; an
// index with bit 31 set names hub slot (idx & 0x7fffffff), held by CTA slot / kHubRows of the cluster ------------
constexpr int kHubRows = 256;   // 128 KB of 512-byte rows per CTA
__global__ void __launch_bounds__(1024, 1) hub_cluster_kernel(const int *__restrict__ idx, long count, const char *__restrict__ table,
                                                              const int *__restrict__ hubrows, float4 *__restrict__ sink) {
    extern __shared__ __align__(128) unsigned char smem[];
    cg::cluster_group cl = cg::this_cluster();
    const unsigned rank = cl.block_rank();
    const int lg = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int r = w; r < kHubRows; r += 32) {
        const int row = hubrows[rank * kHubRows + r];
        reinterpret_cast<float4 *>(smem)[r * 32 + lg] = __ldg(reinterpret_cast<const float4 *>(table + (uint64_t)(uint32_t)row * 512u) + lg);
    }
    cl.sync();
    constexpr int WB = 4;
    const long g = ((long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long G = ((long)gridDim.x * blockDim.x) >> 5;
    const char *base = table + lg * 16;
    const uint32_t sbase = smem_u32(smem) + lg * 16;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (long i = g * WB; i < count; i += G * WB) {
        int r[WB];
#pragma unroll
        for (int u = 0; u < WB; ++u) r[u] = (i + u < count) ? __ldg(idx + i + u) : 0;
        float4 v[WB];
#pragma unroll
        for (int u = 0; u < WB; ++u) {
            if (r[u] < 0) {
                const uint32_t slot = (uint32_t)r[u] & 0x7fffffffu;
                uint32_t ra;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(sbase + (slot % kHubRows) * 512u), "r"(slot / kHubRows));
                asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v[u].x), "=f"(v[u].y), "=f"(v[u].z), "=f"(v[u].w) : "r"(ra));
            } else {
                v[u] = __ldg(reinterpret_cast<const float4 *>(base + (uint64_t)(uint32_t)r[u] * 512u));
            }
        }
#pragma unroll
        for (int u = 0; u < WB; ++u)
            if (i + u < count) add4(acc, v[u]);
    }
    sink[(long)blockIdx.x * blockDim.x + threadIdx.x] = acc;
    cl.sync();   // nobody leaves while a peer may still read its rows
}

int sm_count() {
    int d = 0, n = 148;
    cudaGetDevice(&d);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, d);
    return n;
}
template <typename K>
int resident(K k, int threads, size_t smem) {
    int n = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k, threads, smem) != cudaSuccess || n < 1) n = 1;
    return n;
}
template <int LPR>
void launch_stride_any(const int *idx, long count, const char *table, uint32_t rb, float4 *sink, cudaStream_t st) {
    stride_kernel<LPR, 4, 0, 8><<<sm_count() * 8, 256, 0, st>>>(idx, count, table, rb, sink);
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

// Paths: 0 plain loads, 4 in flight per lane (any row size 16..512 bytes); the others take 512-byte rows only:
//   1 plain x8   2 plain x16   3 L2 evict-last x4   4 L1 no-allocate x4   5 tile order, staged indices, evict-last
//   6 half warp per row, two vectors per lane   7 bulk-copy ring   8 / 9 / 10 hub rows in a cluster of 4 / 8 / 16 CTAs
//   11 / 12 cp.async ring, 16 rows in flight per warp, bypassing / through L1   13 the same with 32 rows (L1 bypassed)
// Floats the sink must hold for any path.
long gp_sink_floats(void) { return (long)sm_count() * 8 * 1024 * 4; }

// idx [count] device int32; table device, row pitch = row_bytes; sink device (gp_sink_floats() floats); err device
// int32 (bulk ring: non-zero when a wait ran out); hubrows device int32 [CL * 256] (paths 8..10: the rows the cluster
// keeps, hub slot order).  *info receives the resident CTAs per SM (clusters on the GPU for paths 8..10).
// Returns 0, -1 for a bad argument, or the cudaError_t of the launch.
int gp_gather(int path, const int *idx, long count, const void *table_, int row_bytes, float *sink_, int *err,
              const int *hubrows, int *info, void *stream) {
    cudaStream_t st = (cudaStream_t)stream;
    const char *table = static_cast<const char *>(table_);
    float4 *sink = reinterpret_cast<float4 *>(sink_);
    if (!idx || !table || !sink || count < 0) return -1;
    if (info) *info = 8;
    if (path == 0) {
        const uint32_t rb = (uint32_t)row_bytes;
        switch (row_bytes) {
        case 16: launch_stride_any<1>(idx, count, table, rb, sink, st); break;
        case 32: launch_stride_any<2>(idx, count, table, rb, sink, st); break;
        case 64: launch_stride_any<4>(idx, count, table, rb, sink, st); break;
        case 128: launch_stride_any<8>(idx, count, table, rb, sink, st); break;
        case 256: launch_stride_any<16>(idx, count, table, rb, sink, st); break;
        case 512: launch_stride_any<32>(idx, count, table, rb, sink, st); break;
        default: return -1;
        }
        return (int)cudaGetLastError();
    }
    if (row_bytes != 512) return -1;
#define GP_STRIDE(WB, MODE, OCC)                                      \
    {                                                                 \
        auto k = stride_kernel<32, WB, MODE, OCC>;                    \
        const int o = resident(k, 256, 0);                            \
        if (info) *info = o;                                          \
        k<<<sm_count() * o, 256, 0, st>>>(idx, count, table, 512u, sink); \
    }
    switch (path) {
    case 1: GP_STRIDE(8, 0, 4) break;
    case 2: GP_STRIDE(16, 0, 2) break;
    case 3: GP_STRIDE(4, 1, 8) break;
    case 4: GP_STRIDE(4, 2, 8) break;
    case 5: tile_kernel<1><<<sm_count() * 8, 256, 0, st>>>(idx, count, table, sink); break;
    case 6:
        if (info) *info = 4;
        half_warp_kernel<<<sm_count() * 4, 256, 0, st>>>(idx, count, table, sink);
        break;
    case 7: {
        if (!err) return -1;
        const size_t sm = (size_t)kBulkStages * kBulkRows * 512;
        cudaFuncSetAttribute(bulk_ring_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
        const int o = resident(bulk_ring_kernel, 32 * (kBulkCons + 1), sm);
        if (info) *info = o;
        bulk_ring_kernel<<<sm_count() * o, 32 * (kBulkCons + 1), sm, st>>>(idx, count, table, sink, err);
        break;
    }
    case 8: case 9: case 10: {
        if (!hubrows) return -1;
        const int CL = path == 8 ? 4 : (path == 9 ? 8 : 16);
        const size_t sm = (size_t)kHubRows * 512;
        cudaFuncSetAttribute(hub_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
        if (CL > 8) cudaFuncSetAttribute(hub_cluster_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        cudaLaunchConfig_t cfg = {};
        cfg.blockDim = dim3(1024);
        cfg.dynamicSmemBytes = sm;
        cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = CL;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        cfg.gridDim = dim3(CL);
        int ncl = 0;
        cudaError_t e = cudaOccupancyMaxActiveClusters(&ncl, hub_cluster_kernel, &cfg);
        if (e != cudaSuccess || ncl < 1) return (int)(e != cudaSuccess ? e : cudaErrorLaunchOutOfResources);
        if (info) *info = ncl;
        cfg.gridDim = dim3(ncl * CL);
        e = cudaLaunchKernelEx(&cfg, hub_cluster_kernel, idx, count, table, hubrows, sink);
        if (e != cudaSuccess) return (int)e;
        break;
    }
#define GP_ASYNC(D, CGF)                                                                           \
    {                                                                                              \
        auto k = async_ring_kernel<D, 4, CGF>;                                                     \
        const size_t sm = (size_t)8 * D * 512;                                                     \
        cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);             \
        const int o = resident(k, 256, sm);                                                        \
        if (info) *info = o;                                                                       \
        k<<<sm_count() * o, 256, sm, st>>>(idx, count, table, sink);                               \
    }
    case 11: GP_ASYNC(16, true) break;
    case 12: GP_ASYNC(16, false) break;
    case 13: GP_ASYNC(32, true) break;
#undef GP_ASYNC
    default: return -1;
    }
#undef GP_STRIDE
    return (int)cudaGetLastError();
}

#pragma GCC visibility pop
}
