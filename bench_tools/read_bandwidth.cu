// Read-bandwidth test for sm_100a: how fast one pass over a large fp32 array streams from HBM with plain 16-byte
// loads and with the tile pipeline of the encoder (per-warp stages filled by 2-D TMA tile copies or contiguous bulk
// copies), for several tile heights, stage counts and resident CTAs.  Stand-alone program (no library code):
//     read_bandwidth [elements]      default: a 102 MB array; rotates over six arrays so that nothing stays in L2
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <cuda.h>
#include <cuda_runtime.h>

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < (1u << 20); ++it) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_rows(uint32_t dst, const CUtensorMap* tmap, uint32_t bar, int32_t row0)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"((uint64_t)tmap), "r"(bar), "r"(0), "r"(row0) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// plain loads: every thread streams float4s, grid-stride, UNROLL independent loads in flight
template <int UNROLL>
__global__ void __launch_bounds__(256) k_ldg(const float4* __restrict__ p, uint64_t n4, float* sink)
{
    float acc = 0.f;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + (UNROLL - 1) * stride < n4; i += UNROLL * stride) {
        float4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) v[u] = __ldg(p + i + u * stride);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) acc += v[u].x + v[u].y + v[u].z + v[u].w;
    }
    if (acc == 12345.678f) sink[0] = acc;
}

// per-warp pipeline of STAGES tiles of ROWS rows x 128 B (TMA 2-D, 128B swizzle) or 1-D bulk copies of the same size
template <int ROWS, int STAGES, bool BULK1D, int WARPS>
__global__ void __launch_bounds__(WARPS * 32) k_tma(const __grid_constant__ CUtensorMap tmap, const float* base, uint32_t num_tiles,
                                                    float* sink)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[WARPS][STAGES];
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t kBytes = ROWS * 128;
    const uint32_t sbase = ((smem_u32(smem_raw) + 1023u) & ~1023u) + warp * STAGES * kBytes;
    const uint32_t bar0 = smem_u32(&bars[warp][0]);
    const uint32_t stride = gridDim.x * WARPS;
    const uint32_t first = blockIdx.x * WARPS + warp;
    if (lane == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(bar0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        for (int s = 0; s < STAGES; ++s) {
            const uint64_t t = (uint64_t)first + (uint64_t)s * stride;
            if (t < num_tiles) {
                mbar_expect_tx(bar0 + 8 * s, kBytes);
                if (BULK1D) bulk_load(sbase + s * kBytes, base + t * (kBytes / 4), kBytes, bar0 + 8 * s);
                else tma_load_rows(sbase + s * kBytes, &tmap, bar0 + 8 * s, (int32_t)(t * ROWS));
            }
        }
    }
    __syncwarp();
    float acc = 0.f;
    uint32_t k = 0;
    for (uint64_t t = first; t < num_tiles; t += stride, ++k) {
        const uint32_t s = k % STAGES, use = k / STAGES;
        mbar_wait(bar0 + 8 * s, use & 1);
        float v;
        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(sbase + s * kBytes + lane * 4) : "memory");
        acc += v;
        __syncwarp();
        if (lane == 0) {
            const uint64_t nt = t + (uint64_t)STAGES * stride;
            if (nt < num_tiles) {
                mbar_expect_tx(bar0 + 8 * s, kBytes);
                if (BULK1D) bulk_load(sbase + s * kBytes, base + nt * (kBytes / 4), kBytes, bar0 + 8 * s);
                else tma_load_rows(sbase + s * kBytes, &tmap, bar0 + 8 * s, (int32_t)(nt * ROWS));
            }
        }
    }
    if (acc == 12345.678f) sink[0] = acc;
}

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static bool make_map(CUtensorMap* map, const float* base, uint64_t rows, uint32_t box_rows, CUtensorMapL2promotion prom)
{
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || !p) return false;
    const cuuint64_t dims[2] = {32u, rows};
    const cuuint64_t strides[1] = {128u};
    const cuuint32_t box[2] = {32u, box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    return ((encode_tiled_fn)p)(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2u, (void*)base, dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, prom,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename F>
static double time_it(F launch, int iters)
{
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0); cudaEventCreate(&e1);
    for (int i = 0; i < 3; ++i) launch(i);
    cudaDeviceSynchronize();
    cudaEventRecord(e0);
    for (int i = 0; i < iters; ++i) launch(i);
    cudaEventRecord(e1);
    cudaDeviceSynchronize();
    float ms = 0;
    cudaEventElapsedTime(&ms, e0, e1);
    return ms / iters;
}

template <int ROWS, int STAGES, bool BULK1D, int WARPS>
static void run_tma(const char* name, float** bufs, int nbuf, uint64_t n, int ctas_per_sm, float* sink, CUtensorMapL2promotion prom)
{
    auto k = k_tma<ROWS, STAGES, BULK1D, WARPS>;
    const size_t smem = (size_t)WARPS * STAGES * ROWS * 128 + 1024;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) { printf("%s: smem attr failed\n", name); return; }
    CUtensorMap maps[8];
    const uint64_t rows = n / 32;
    for (int b = 0; b < nbuf; ++b)
        if (!make_map(&maps[b], bufs[b], rows, ROWS, prom)) { printf("%s: map failed\n", name); return; }
    const uint32_t tiles = (uint32_t)(rows / ROWS);
    const int grid = 148 * ctas_per_sm;
    double ms = time_it([&](int i) { k<<<grid, WARPS * 32, smem>>>(maps[i % nbuf], bufs[i % nbuf], tiles, sink); }, 20);
    cudaError_t e = cudaGetLastError();
    printf("%-44s ctas/sm %d smem %6zu: %8.2f us  %7.1f GB/s %s\n", name, ctas_per_sm, smem, ms * 1e3, 4.0 * n / ms / 1e6,
           e == cudaSuccess ? "" : cudaGetErrorString(e));
    fflush(stdout);
}

int main(int argc, char** argv)
{
    const uint64_t n = (argc > 1) ? strtoull(argv[1], nullptr, 10) : 25557032ull / 2048 * 2048;
    const int nbuf = 6;
    float* bufs[8];
    for (int b = 0; b < nbuf; ++b) {
        if (cudaMalloc(&bufs[b], n * 4) != cudaSuccess) { printf("alloc failed\n"); return 1; }
        cudaMemset(bufs[b], 0, n * 4);
    }
    float* sink;
    cudaMalloc(&sink, 4);
    printf("n = %llu floats (%.1f MB), %d rotating buffers\n", (unsigned long long)n, n * 4 / 1e6, nbuf);
    for (int cps : {2, 4, 8}) {
        double ms = time_it([&](int i) { k_ldg<4><<<148 * cps, 256>>>((const float4*)bufs[i % nbuf], n / 4, sink); }, 20);
        printf("ldg.128 x4 in flight, %d CTAs/SM of 256: %8.2f us %7.1f GB/s\n", cps, ms * 1e3, 4.0 * n / ms / 1e6);
        ms = time_it([&](int i) { k_ldg<8><<<148 * cps, 256>>>((const float4*)bufs[i % nbuf], n / 4, sink); }, 20);
        printf("ldg.128 x8 in flight, %d CTAs/SM of 256: %8.2f us %7.1f GB/s\n", cps, ms * 1e3, 4.0 * n / ms / 1e6);
    }
    const auto P128 = CU_TENSOR_MAP_L2_PROMOTION_L2_128B, P256 = CU_TENSOR_MAP_L2_PROMOTION_L2_256B, PN = CU_TENSOR_MAP_L2_PROMOTION_NONE;
    run_tma<32, 2, false, 8>("tma 32 rows x2 stages, 8 warps (encoder)", bufs, nbuf, n, 3, sink, P128);
    run_tma<32, 2, false, 8>("tma 32 rows x2 stages, 8 warps, promo 256", bufs, nbuf, n, 3, sink, P256);
    run_tma<32, 2, false, 8>("tma 32 rows x2 stages, 8 warps, promo none", bufs, nbuf, n, 3, sink, PN);
    run_tma<32, 3, false, 8>("tma 32 rows x3 stages, 8 warps", bufs, nbuf, n, 2, sink, P128);
    run_tma<32, 2, false, 8>("tma 32 rows x2 stages, 8 warps", bufs, nbuf, n, 2, sink, P128);
    run_tma<32, 2, false, 8>("tma 32 rows x2 stages, 8 warps", bufs, nbuf, n, 1, sink, P128);
    run_tma<32, 2, false, 4>("tma 32 rows x2 stages, 4 warps", bufs, nbuf, n, 4, sink, P128);
    run_tma<32, 2, false, 4>("tma 32 rows x2 stages, 4 warps", bufs, nbuf, n, 2, sink, P128);
    run_tma<64, 2, false, 8>("tma 64 rows x2 stages, 8 warps", bufs, nbuf, n, 1, sink, P128);
    run_tma<64, 2, false, 4>("tma 64 rows x2 stages, 4 warps", bufs, nbuf, n, 3, sink, P128);
    run_tma<128, 2, false, 4>("tma 128 rows x2 stages, 4 warps", bufs, nbuf, n, 1, sink, P128);
    run_tma<256, 2, false, 2>("tma 256 rows x2 stages, 2 warps", bufs, nbuf, n, 1, sink, P128);
    run_tma<256, 2, false, 1>("tma 256 rows x2 stages, 1 warp", bufs, nbuf, n, 3, sink, P128);
    run_tma<32, 2, true, 8>("bulk1d 4 KB x2 stages, 8 warps", bufs, nbuf, n, 3, sink, P128);
    run_tma<128, 2, true, 4>("bulk1d 16 KB x2 stages, 4 warps", bufs, nbuf, n, 1, sink, P128);
    run_tma<256, 2, true, 2>("bulk1d 32 KB x2 stages, 2 warps", bufs, nbuf, n, 1, sink, P128);
    return 0;
}
