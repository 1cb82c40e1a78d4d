// One (gradient dtype, fused or not, statistics mode) combination of the streaming norm-test
// kernels: this file is compiled once per combination (see build.py), each time with
//   -DABS_INST_GT=F32|BF16  -DABS_INST_ADAM=0|1  -DABS_INST_STAT=0|1|2
// and instantiates launch_stream for it -- about fifty kernels, one per worker count.
#include "launch.cuh"

#ifndef ABS_INST_GT
#define ABS_INST_GT BF16
#endif
#ifndef ABS_INST_ADAM
#define ABS_INST_ADAM 1
#endif
#ifndef ABS_INST_STAT
#define ABS_INST_STAT 0
#endif

namespace absnt {
template cudaError_t launch_stream<ABS_INST_GT, ABS_INST_ADAM != 0, ABS_INST_STAT>(
    const StreamParams&, const WideTable*, cudaStream_t);
}  // namespace absnt
