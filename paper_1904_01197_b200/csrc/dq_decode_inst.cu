// Instantiation of decode_aggregate_kernel for one dither width and one side-information mode (DQ_INST_DITH,
// DQ_INST_RUN, given on the compiler's command line).
#include "dq_decode.cuh"
#include "dq_launch.h"

#ifndef DQ_INST_DITH
#error "compile with -DDQ_INST_DITH=<32|16|0> -DDQ_INST_RUN=<0|1>"
#endif

namespace dq {

#define DQ_NAME2(D, R) launch_decode_d##D##_r##R
#define DQ_NAME(D, R) DQ_NAME2(D, R)

cudaError_t DQ_NAME(DQ_INST_DITH, DQ_INST_RUN)(const DecodeArgs& a, uint32_t grid, cudaStream_t st)
{
    return launch_overlapped(decode_aggregate_kernel<DQ_INST_DITH, (DQ_INST_RUN != 0)>, grid, (uint32_t)kDecThreads,
                             0, st, a);
}

}  // namespace dq
