// Two small kernels beside the flow kernels (entry points: iodf_selftest_timeout, iodf_int8_mma_peak):
//
//  * timeout_probe_kernel: one warp waits, with the library's bounded wait and a caller-given number
//    of tries, on an mbarrier that nothing ever arrives on. The wait runs out, sets the device
//    status word and the kernel returns normally: the path that iodf_check reports as IODF_ETIMEOUT,
//    exercised without a fault, a trap or an endless loop. No tensor memory, no MMA, no bulk copy.
//
//  * int8_mma_peak_kernel: the denominator of the tensor roofline. One CTA per SM issues a fixed
//    number of tcgen05.mma kind::i8 instructions of shape 128 x 256 x 32 from operands resident in
//    shared memory into two alternating 256-column accumulators in tensor memory. Nothing else
//    runs, so OPs / time is what the int8 tensor pipe of this GPU sustains at the clocks and power
//    it is given.
#include <cuda_runtime.h>

#include "selftest.h"
#include "iodf_dev.h"
#include "ptx.cuh"

namespace iodf {
namespace {

__global__ void __launch_bounds__(32, 1) timeout_probe_kernel(uint32_t* status, uint32_t tries) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    ptx::mbar_init_fence();
    abort_flag = 0;
  }
  __syncwarp();
  // phase 0 of a barrier that expects one arrival and never gets it
  if (threadIdx.x == 0) ptx::bounded_wait(&abort_flag, status, &bar, 0u, tries);
  __syncwarp();
  // a second wait after the first gave up must return at once (the abort flag is set)
  if (threadIdx.x == 1) ptx::bounded_wait(&abort_flag, status, &bar, 0u, tries);
}

constexpr int kPeakN = 256;              // MMA N
constexpr int kPeakKSteps = 4;           // 32-byte K steps resident in shared memory
constexpr int kPeakABytes = kTileM * 32 * kPeakKSteps;    // 16 KB
constexpr int kPeakBBytes = kPeakN * 32 * kPeakKSteps;    // 32 KB

__global__ void __launch_bounds__(128, 1) int8_mma_peak_kernel(uint32_t* status, uint32_t groups) {
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ __align__(8) uint64_t done;
  __shared__ uint32_t tmem_base, abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  // operands: pseudo-random bytes (a multiplicative hash of the byte index), so that the data
  // paths toggle as they do on real activations and weights
  for (int i = tid; i < (kPeakABytes + kPeakBBytes) / 4; i += 128)
    reinterpret_cast<uint32_t*>(smem)[i] = (uint32_t)(i + 1 + blockIdx.x * 7919) * 2654435761u;
  if (tid == 0) {
    ptx::mbar_init(ptx::smem_u32(&done), 1);
    ptx::mbar_init_fence();
    abort_flag = 0;
  }
  if (warp == 0) ptx::tmem_alloc(ptx::smem_u32(&tmem_base), 512u);
  ptx::fence_async_smem();
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = tmem_base;
  if (tid == 0) {
    const uint32_t idesc = ptx::umma_idesc_i8((uint32_t)kPeakN, false);
    const uint32_t sa = ptx::smem_u32(smem), sb = sa + kPeakABytes;
    uint32_t da[kPeakKSteps], db[kPeakKSteps];
#pragma unroll
    for (int k = 0; k < kPeakKSteps; ++k) {
      da[k] = ptx::umma_desc_lo(sa + (uint32_t)k * 2u * kTileM * 16u, kTileM * 16u);
      db[k] = ptx::umma_desc_lo(sb + (uint32_t)k * 2u * kPeakN * 16u, kPeakN * 16u);
    }
    // one group = 2 accumulators x kPeakKSteps MMAs; the first K step of a group overwrites its
    // accumulator, so the int32 sums stay small whatever the number of groups
    for (uint32_t g = 0; g < groups; ++g) {
#pragma unroll
      for (int acc = 0; acc < 2; ++acc)
#pragma unroll
        for (int k = 0; k < kPeakKSteps; ++k)
          ptx::umma_i8_lo(tmem + (uint32_t)(acc * kPeakN), da[k], db[k], idesc, k ? 1u : 0u);
    }
    ptx::umma_commit(ptx::smem_u32(&done));
    ptx::bounded_wait(&abort_flag, status, &done, 0u, kSpinLimit);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 0) ptx::tmem_dealloc(tmem, 512u);
}

}  // namespace
}  // namespace iodf

namespace iodf {

cudaError_t launch_timeout_probe(uint32_t* status_dev, uint32_t tries, cudaStream_t stream) {
  timeout_probe_kernel<<<1, 32, 0, stream>>>(status_dev, tries);
  return cudaGetLastError();
}

cudaError_t launch_int8_mma_peak(uint32_t* status_dev, uint32_t mma_groups, int sms, cudaStream_t stream,
                                 unsigned long long* ops_out) {
  const int smem = kPeakABytes + kPeakBBytes;
  cudaError_t e = cudaFuncSetAttribute(int8_mma_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  int8_mma_peak_kernel<<<sms, 128, smem, stream>>>(status_dev, mma_groups);
  if (ops_out)
    *ops_out = 2ull * kTileM * kPeakN * 32ull * 2ull * kPeakKSteps * (unsigned long long)mma_groups * (unsigned long long)sms;
  return cudaGetLastError();
}

}  // namespace iodf
