// Launch interface of the bounded-wait probe and the int8 tensor-peak microbenchmark (selftest.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace iodf {

// One warp waits `tries` suspended tries on an mbarrier nobody arrives on, then sets *status_dev.
cudaError_t launch_timeout_probe(uint32_t* status_dev, uint32_t tries, cudaStream_t stream);
// `sms` CTAs each issue mma_groups * 8 tcgen05.mma kind::i8 128x256x32; *ops_out = int8 OPs of the launch.
cudaError_t launch_int8_mma_peak(uint32_t* status_dev, uint32_t mma_groups, int sms, cudaStream_t stream,
                                 unsigned long long* ops_out);

}  // namespace iodf
