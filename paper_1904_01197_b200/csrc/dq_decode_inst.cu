// Instantiation of decode_aggregate_kernel for one dither width and one side-information mode (DQ_INST_DITH,
// DQ_INST_RUN = a DecSide value, given on the compiler's command line).
#include <atomic>

#include "dq_decode.cuh"
#include "dq_launch.h"

#ifndef DQ_INST_DITH
#error "compile with -DDQ_INST_DITH=<32|16|0> -DDQ_INST_RUN=<0|1|2>"
#endif

namespace dq {

#define DQ_NAME2(D, R) launch_decode_d##D##_r##R
#define DQ_NAME(D, R) DQ_NAME2(D, R)

cudaError_t DQ_NAME(DQ_INST_DITH, DQ_INST_RUN)(const CUtensorMap& side_map, const CUtensorMap& out_map,
                                               const DecodeArgs& a, int sm_count, cudaStream_t st)
{
    auto k = decode_aggregate_kernel<DQ_INST_DITH, DQ_INST_RUN>;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    // per device: the shared-memory attribute and the resident CTAs per SM
    static std::atomic<uint64_t> configured{0};
    static std::atomic<int> per_sm[64];
    if (!(configured.load(std::memory_order_acquire) & (1ull << dev))) {
        cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecSmemBytes);
        if (e != cudaSuccess) return e;
        int blocks = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks, k, kDecThreads, kDecSmemBytes);
        if (e != cudaSuccess) return e;
        if (blocks < 1) return cudaErrorLaunchOutOfResources;
        per_sm[dev].store(blocks);
        configured.fetch_or(1ull << dev, std::memory_order_release);
    }
    const uint32_t smem = kDecSmemBytes;
    const int blocks = per_sm[dev].load();
    const uint64_t want = ((uint64_t)a.num_units + kDecTeamWarps - 1u) / kDecTeamWarps;   // one team-unit each at least
    const uint64_t room = (uint64_t)blocks * (uint64_t)sm_count;
    const uint32_t grid = (uint32_t)(want < room ? want : room);
    return launch_overlapped(k, grid, (uint32_t)kDecThreads, smem, st, side_map, out_map, a);
}

}  // namespace dq
