// Launch interface of the entropy-coding kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace iodf {

constexpr int kMaxRansBlocks = 9;      // one per flow level plus the final block

struct RansBlock {
  long long z_off;         // offset of the block in an image's z
  long long n;             // elements
  long long prior_off;     // offset in mu (and in the log-scale plane), or -1: mu = 0, scale index final_ls
  int first_stream;        // number of the block's first stream within an image
  int n_streams;           // ceil(n / elems_per_stream)
};

struct RansArgs {
  const uint16_t* G;       // device: sigmoid table, 2 * umax + 1 entries
  const uint32_t* R;       // device: reciprocal scales, n_scales entries
  int umax, n_scales, final_ls;
  int n_blocks, n_streams; // per image
  int cap;                 // words per stream in the container (3 * elems_per_stream + 2)
  int batch;
  long long d, d_fact;
  uint32_t* errors;        // device counter or null: streams with an out-of-range scale index or a
                           // malformed word sequence
  RansBlock blocks[kMaxRansBlocks];
};

cudaError_t launch_rans_encode(const RansArgs& a, const int32_t* z, const int32_t* prior, uint16_t* words,
                               uint32_t* counts, cudaStream_t stream);
cudaError_t launch_rans_decode(const RansArgs& a, int block, const uint16_t* words, const uint32_t* counts,
                               const int32_t* prior, int32_t* z, cudaStream_t stream);

// Container <-> compact byte stream ([B + 1] uint32 record offsets, then per image uint16 counts and the
// streams' words back to back). `sizes` is a scratch array of batch uint32. Unpacking checks every
// record against `payload_bytes` and its own counts; a bad record gives zero counts and is counted in
// a.errors.
cudaError_t launch_rans_pack(const RansArgs& a, const uint16_t* words, const uint32_t* counts, uint32_t* sizes,
                             uint8_t* packed, cudaStream_t stream);
cudaError_t launch_rans_unpack(const RansArgs& a, const uint8_t* packed, unsigned long long payload_bytes,
                               uint16_t* words, uint32_t* counts, cudaStream_t stream);

}  // namespace iodf
