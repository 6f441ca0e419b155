// Launch interface of the level kernel that splits a tile's work by role (level_pipe.cu), for levels
// whose plan has LevelPlan::pipe set.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "level_kernel.h"

namespace iodf {

constexpr int kPipeThreads = 736;    // 16 requantising warps, 4 im2col / shifted-sum warps, 3 control warps

cudaError_t configure_pipe_kernels(uint32_t max_smem_bytes);
cudaError_t launch_level_pipe(const LevelArgs& args, bool inverse, int grid, uint32_t smem_bytes, cudaStream_t stream);

}  // namespace iodf
