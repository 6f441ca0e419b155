// Launch interface of the per-level flow kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "iodf_dev.h"

namespace iodf {

struct LevelArgs {
  const LevelPlan* plan;   // device
  const uint8_t* blob;     // device: the level's packed blocks
  // encode: the level's input before the squeeze: uint8 image batch (first level) or the int32
  //         kept channels of the previous level, [B][c/4][2h][2w]
  // decode: the int32 kept channels coming back from the deeper level (or z's final block),
  //         image b at in + b*in_stride, [keep_c][h][w]
  const void* in;
  long long in_stride;
  int32_t* z;              // [B][d]
  int32_t* prior;          // [B][2][d_fact] or null
  // encode: int32 kept channels for the next level [B][keep_c][h][w] (unused on the last level)
  // decode: the level's output after depth-to-space, [B][c/4][2h][2w]: uint8 on the first level,
  //         int32 otherwise
  void* out;
  uint32_t* oor;           // decode, first level: count of recovered values outside 0..255, or null
  uint32_t* status;        // device status word (non-zero: a bounded wait gave up)
  int batch;
  // decode only: 0 = the whole level; 1 = prior head only (reads the kept channels, writes prior
  // parameters, stores nothing else); 2 = couplings only (no prior head)
  int phase;
  // first level only, img_w > 0: the batch is the grid of in_h x in_w patches of one image
  // [c][img_h][img_w] (patch b = row b / patches_x, column b % patches_x), read (encode) or written
  // (decode) in place of the [B][c][in_h][in_w] batch. mul_patches_x = ceil(2^32 / patches_x), 0 for 1.
  int img_h, img_w, patches_x;
  uint32_t mul_patches_x;
};

cudaError_t configure_level_kernels(uint32_t max_smem_bytes);
// lean: the kernel variant for levels whose hidden layers all use the folded requantisation flavour with the
// 0..127 clip and whose weights are not streamed (LevelPlan::lean)
cudaError_t launch_level(const LevelArgs& args, bool inverse, bool lean, int grid, uint32_t smem_bytes,
                         cudaStream_t stream);

}  // namespace iodf
