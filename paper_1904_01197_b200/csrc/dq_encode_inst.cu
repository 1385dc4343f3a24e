// Instantiations of encode_kernel for one encoder mode and one dither width (DQ_INST_MODE, DQ_INST_DITH, given on
// the compiler's command line) and all eight code widths.
#include <atomic>

#include "dq_encode.cuh"
#include "dq_launch.h"

#ifndef DQ_INST_MODE
#error "compile with -DDQ_INST_MODE=<EncMode> -DDQ_INST_DITH=<32|16>"
#endif

namespace dq {
namespace {

template <int BITS>
cudaError_t launch_one(const CUtensorMap& map, const EncodeArgs& a, uint32_t grid, cudaStream_t st)
{
    auto k = encode_kernel<BITS, DQ_INST_MODE, DQ_INST_DITH>;
    // the attribute is per device and idempotent; one bit per device that has it
    static std::atomic<uint64_t> configured{0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!(configured.load(std::memory_order_acquire) & (1ull << dev))) {
        cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kEncSmemBytes);
        if (e != cudaSuccess) return e;
        configured.fetch_or(1ull << dev, std::memory_order_release);
    }
    return launch_overlapped(k, grid, (uint32_t)kEncThreads, kEncSmemBytes, st, map, a);
}

}  // namespace

#define DQ_NAME2(M, D) launch_encode_m##M##_d##D
#define DQ_NAME(M, D) DQ_NAME2(M, D)

cudaError_t DQ_NAME(DQ_INST_MODE, DQ_INST_DITH)(uint32_t bits, const CUtensorMap& map, const EncodeArgs& a,
                                                 uint32_t grid, cudaStream_t st)
{
    switch (bits) {
        case 1: return launch_one<1>(map, a, grid, st);
        case 2: return launch_one<2>(map, a, grid, st);
        case 3: return launch_one<3>(map, a, grid, st);
        case 4: return launch_one<4>(map, a, grid, st);
        case 5: return launch_one<5>(map, a, grid, st);
        case 6: return launch_one<6>(map, a, grid, st);
        case 7: return launch_one<7>(map, a, grid, st);
        default: return launch_one<8>(map, a, grid, st);
    }
}

}  // namespace dq
