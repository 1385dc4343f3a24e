// Launch interface between the host side of the C ABI (dq_b200.cu) and the translation units that hold the
// kernel instantiations.  The encode and decode kernels are templates with dozens of instantiations; they are
// compiled as separate translation units (one per encoder mode and dither width, one per decoder variant) so that
// the library builds in parallel.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace dq {

struct EncodeArgs;
struct DecodeArgs;

// Launch with programmatic stream serialization allowed: every kernel of this library executes
// griddepcontrol.wait before it writes anything, and before it reads anything that the previous kernel of the
// stream may have produced, so letting the next launch become resident while this one drains only hides launch
// latency.
template <typename... KArgs, typename... Args>
cudaError_t launch_overlapped(void (*kernel)(KArgs...), uint32_t grid, uint32_t block, size_t smem, cudaStream_t st,
                              Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Encoder: mode = EncMode, dith = 32 or 16.  One function per (mode, dith) translation unit; launch_encode picks.
#define DQ_DECLARE_ENCODE(MODE, DITH)                                                                              \
    cudaError_t launch_encode_m##MODE##_d##DITH(uint32_t bits, const CUtensorMap& map, const EncodeArgs& a,        \
                                                uint32_t grid, cudaStream_t st);
DQ_DECLARE_ENCODE(0, 32) DQ_DECLARE_ENCODE(1, 32) DQ_DECLARE_ENCODE(2, 32) DQ_DECLARE_ENCODE(3, 32)
DQ_DECLARE_ENCODE(0, 16) DQ_DECLARE_ENCODE(1, 16) DQ_DECLARE_ENCODE(2, 16) DQ_DECLARE_ENCODE(3, 16)
#undef DQ_DECLARE_ENCODE

// Decoder: dith = 32, 16 or 0 (no dither at the receiver); run = DecSide (0 given vector or none, 1 running mean,
// 2 reconstruction of message 0).
// The grid (persistent CTAs) follows from a.num_units and the device.
#define DQ_DECLARE_DECODE(DITH, RUN)                                                                               \
    cudaError_t launch_decode_d##DITH##_r##RUN(const CUtensorMap& side_map, const CUtensorMap& out_map,            \
                                               const DecodeArgs& a, int sm_count, cudaStream_t st);
DQ_DECLARE_DECODE(32, 0) DQ_DECLARE_DECODE(32, 1) DQ_DECLARE_DECODE(16, 0) DQ_DECLARE_DECODE(16, 1)
DQ_DECLARE_DECODE(32, 2) DQ_DECLARE_DECODE(16, 2)
DQ_DECLARE_DECODE(0, 0)
#undef DQ_DECLARE_DECODE

}  // namespace dq
