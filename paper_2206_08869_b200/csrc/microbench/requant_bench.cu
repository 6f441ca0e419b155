// Microbenchmark behind the epilogue's design: how many hidden activations per clock one SM can
// requantise (y = clip(hi32(acc * m0 + 2^(30+s)) >> (s-1), 0, 127), Eq. "quant_conv" of Sec. 4.1 in
// the library's fixed-point form), for a few instruction sequences, with the accumulators in
// registers and read from tensor memory, at 1 to 8 warps per scheduler, and for a form that goes
// through the fp64 pipe. Not part of the library.
//
//   nvcc -O3 -std=c++17 -gencode arch=compute_100a,code=sm_100a -o requant_bench requant_bench.cu && ./requant_bench
#include <cstdio>
#include <cstdint>
#include <cmath>
#include <cuda_runtime.h>

#include "../ptx.cuh"
using namespace iodf;
__device__ __forceinline__ uint32_t pack4_sat(int y0, int y1, int y2, int y3) {
  uint32_t t, w;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(y3), "r"(y2), "r"(0));
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(y1), "r"(y0), "r"(t));
  return w;
}
__device__ __forceinline__ uint32_t relu4(uint32_t w) {
  uint32_t neg;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(neg) : "r"(w), "r"(0u), "r"(0xBA98u));
  return w & ~neg;
}

template <int V>
__device__ __forceinline__ int rq1(int acc, int m0, int sh, long long rnd64, int rnd_hi) {
  if (V == 0) {   // 64-bit multiply-add, high word, shift
    const long long p = (long long)acc * (long long)m0 + rnd64;
    return ((int)(p >> 32)) >> sh;
  } else if (V == 1) {   // high multiply + add + shift
    return (__mulhi(acc, m0) + rnd_hi) >> sh;
  } else if (V == 2) {   // mul.wide then 64-bit add via PTX
    long long p;
    asm("mad.wide.s32 %0, %1, %2, %3;" : "=l"(p) : "r"(acc), "r"(m0), "l"(rnd64));
    return ((int)(p >> 32)) >> sh;
  } else {               // float (not exact; speed reference)
    return (int)floorf(__int2float_rn(acc) * __int_as_float(m0) + 0.5f);
  }
}

template <int V, bool kSmemConst>
__global__ void bench_regs(const int* __restrict__ gm0, int iters, int sh, unsigned long long* out_clk, uint32_t* out_sum) {
  __shared__ __align__(16) int sm0[256];
  __shared__ __align__(16) uint4 sout[1024];
  for (int i = threadIdx.x; i < 256; i += blockDim.x) sm0[i] = gm0[i];
  __syncthreads();
  const long long rnd64 = 1ll << (31 + sh);
  const int rnd_hi = 1 << (sh - 1);
  int acc[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) acc[i] = (threadIdx.x * 977 + i * 131071) ^ 0x5a5a;
  uint32_t sum = 0;
  int regc[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) regc[i] = gm0[i];
  const unsigned long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
    const int ch0 = (it * 16) & 255;
    uint32_t wd[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      int4 c;
      if (kSmemConst) c = *reinterpret_cast<const int4*>(&sm0[(ch0 + 4 * q) & 255]);
      else c = make_int4(regc[4 * q], regc[4 * q + 1], regc[4 * q + 2], regc[4 * q + 3]);
      const int y0 = rq1<V>(acc[4 * q], c.x, sh, rnd64, rnd_hi), y1 = rq1<V>(acc[4 * q + 1], c.y, sh, rnd64, rnd_hi);
      const int y2 = rq1<V>(acc[4 * q + 2], c.z, sh, rnd64, rnd_hi), y3 = rq1<V>(acc[4 * q + 3], c.w, sh, rnd64, rnd_hi);
      wd[q] = relu4(pack4_sat(y0, y1, y2, y3));
    }
    sout[threadIdx.x & 1023] = make_uint4(wd[0], wd[1], wd[2], wd[3]);
    // next iteration's inputs depend on nothing computed here except cheaply (keeps the loop honest)
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] += 0x01010101 * (it + 1);
    sum ^= wd[0] + wd[3];
  }
  const unsigned long long t1 = clock64();
  if (threadIdx.x == 0) out_clk[blockIdx.x] = t1 - t0;
  out_sum[blockIdx.x * blockDim.x + threadIdx.x] = sum + sout[(threadIdx.x * 7) & 1023].x;
}

template <int V, bool S>
void run_regs(const char* name, const int* dm0, unsigned long long* dclk, uint32_t* dsum) {
  const int iters = 2000;
  for (int warps : {1, 4, 8, 16, 32}) {
    bench_regs<V, S><<<1, warps * 32>>>(dm0, iters, 7, dclk, dsum);
    cudaDeviceSynchronize();
    bench_regs<V, S><<<1, warps * 32>>>(dm0, iters, 7, dclk, dsum);
    cudaError_t e = cudaDeviceSynchronize();
    unsigned long long clk = 0;
    cudaMemcpy(&clk, dclk, sizeof(clk), cudaMemcpyDeviceToHost);
    printf("%-28s warps/SM %2d: %7.1f clk per chunk per warp, %6.2f activations/clk/SM  (%s)\n", name, warps,
           (double)clk / iters, 16.0 * 32 * warps * iters / (double)clk, cudaGetErrorString(e));
  }
}

__device__ __forceinline__ int rq1w(int acc, int m0, int sh, long long rnd64) {
  const long long p = (long long)acc * (long long)m0 + rnd64;
  return ((int)(p >> 32)) >> sh;
}
__device__ __forceinline__ uint4 chunk(const uint32_t* r, const int* sm0, int ch0, int sh, long long rnd64) {
  uint32_t wd[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int4 c = *reinterpret_cast<const int4*>(&sm0[(ch0 + 4 * q) & 255]);
    wd[q] = relu4(pack4_sat(rq1w((int)r[4 * q], c.x, sh, rnd64), rq1w((int)r[4 * q + 1], c.y, sh, rnd64),
                            rq1w((int)r[4 * q + 2], c.z, sh, rnd64), rq1w((int)r[4 * q + 3], c.w, sh, rnd64)));
  }
  return make_uint4(wd[0], wd[1], wd[2], wd[3]);
}

// V: 0 = ld16, wait with operands, compute; 1 = ld16, plain wait; 2 = two ld8; 3 = pipelined ping-pong (as the kernel);
//    4 = ld32 then two chunks
template <int V>
__global__ void __launch_bounds__(512, 1) bench_tmem(const int* __restrict__ gm0, int iters, int sh, unsigned long long* out_clk, uint32_t* out_sum) {
  __shared__ __align__(16) int sm0[256];
  __shared__ __align__(16) uint4 sout[512];
  __shared__ uint32_t tmem_base;
  for (int i = threadIdx.x; i < 256; i += blockDim.x) sm0[i] = gm0[i];
  const int warp = __shfl_sync(0xFFFFFFFFu, threadIdx.x >> 5, 0);
  if (warp == 0) ptx::tmem_alloc(ptx::smem_u32(&tmem_base), 512u);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
  const long long rnd64 = 1ll << (31 + sh);
  uint32_t sum = 0;
  const unsigned long long t0 = clock64();
  if (V == 3) {
    uint32_t ra[16], rb[16];
    ptx::tmem_ld16(taddr, ra);
    for (int it = 0; it < iters; it += 2) {
      const int col = (it * 16) & 255;
      ptx::tmem_ld_wait();
      ptx::tmem_ld16(taddr + (uint32_t)((col + 16) & 255), rb);
      uint4 v = chunk(ra, sm0, col, sh, rnd64);
      sout[threadIdx.x] = v; sum ^= v.x + v.w;
      ptx::tmem_ld_wait();
      ptx::tmem_ld16(taddr + (uint32_t)((col + 32) & 255), ra);
      v = chunk(rb, sm0, col + 16, sh, rnd64);
      sout[threadIdx.x] = v; sum ^= v.x + v.w;
    }
    ptx::tmem_ld_wait();
  } else if (V == 4) {
    for (int it = 0; it < iters; it += 2) {
      const int col = (it * 16) & 255;
      uint32_t r[32];
      ptx::tmem_ld32(taddr + (uint32_t)col, r);
      ptx::tmem_ld_wait();
      uint4 v = chunk(r, sm0, col, sh, rnd64);
      sout[threadIdx.x] = v; sum ^= v.x + v.w;
      v = chunk(r + 16, sm0, col + 16, sh, rnd64);
      sout[threadIdx.x] = v; sum ^= v.x + v.w;
    }
  } else {
    for (int it = 0; it < iters; ++it) {
      const int col = (it * 16) & 255;
      uint32_t r[16];
      if (V == 2) {
        uint32_t a[8], b[8];
        ptx::tmem_ld8(taddr + (uint32_t)col, a);
        ptx::tmem_ld8(taddr + (uint32_t)col + 8, b);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 8; ++i) { r[i] = a[i]; r[8 + i] = b[i]; }
      } else {
        ptx::tmem_ld16(taddr + (uint32_t)col, r);
        if (V == 0) ptx::tmem_ld_wait16(r); else ptx::tmem_ld_wait();
      }
      const uint4 v = chunk(r, sm0, col, sh, rnd64);
      sout[threadIdx.x] = v;
      sum ^= v.x + v.w;
    }
  }
  const unsigned long long t1 = clock64();
  if (threadIdx.x == 0) out_clk[blockIdx.x] = t1 - t0;
  out_sum[blockIdx.x * blockDim.x + threadIdx.x] = sum + sout[(threadIdx.x * 7) & 511].x;
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 0) ptx::tmem_dealloc(tmem_base, 512u);
}

template <int V>
void run_tmem(const char* name, const int* dm0, unsigned long long* dclk, uint32_t* dsum) {
  const int iters = 2000;
  for (int warps : {4, 16}) {
    bench_tmem<V><<<1, warps * 32>>>(dm0, iters, 7, dclk, dsum);
    cudaDeviceSynchronize();
    bench_tmem<V><<<1, warps * 32>>>(dm0, iters, 7, dclk, dsum);
    cudaError_t e = cudaDeviceSynchronize();
    unsigned long long clk = 0;
    cudaMemcpy(&clk, dclk, sizeof(clk), cudaMemcpyDeviceToHost);
    printf("%-32s warps/SM %2d: %7.1f clk per chunk per warp, %6.2f activations/clk/SM  (%s)\n", name, warps,
           (double)clk / iters, 16.0 * 32 * warps * iters / (double)clk, cudaGetErrorString(e));
  }
}

// ---- the same requantisation through the fp64 pipe ---------------------------------------------------
// y = floor((acc * m0 + 2^(31+sh)) / 2^(32+sh)) in double precision, exact while |acc * m0| + 2^(31+sh)
// < 2^53: acc becomes a double by the exponent trick (2^52 + 2^31 + acc as the low word of 0x43300000),
// one fused multiply-add with ms = m0 * 2^-(32+sh) and c = 0.5 - (2^52 + 2^31) * ms gives
// (acc * m0 + 2^(31+sh)) / 2^(32+sh) without rounding, and a round-down add of 1.5 * 2^52 leaves its
// floor in the low word. Is the otherwise idle fp64 pipe a second lane for the epilogue?
__device__ __forceinline__ int rq_f64(int acc, double ms, double c) {
  const double d = __hiloint2double(0x43300000, acc ^ 0x80000000);
  return __double2loint(__dadd_rd(fma(d, ms, c), 6755399441055744.0));
}

// kF of every 16 columns go through the fp64 form (0: none, 16: all)
template <int kF>
__global__ void bench_f64(const int* __restrict__ gm0, int iters, int sh, unsigned long long* out_clk, uint32_t* out_sum) {
  __shared__ __align__(16) int sm0[256];
  __shared__ __align__(16) double2 smc[256];
  __shared__ __align__(16) uint4 sout[1024];
  for (int i = threadIdx.x; i < 256; i += blockDim.x) {
    sm0[i] = gm0[i];
    const double ms = ldexp((double)gm0[i], -(32 + sh));
    smc[i] = make_double2(ms, 0.5 - 4503601774854144.0 * ms);
  }
  __syncthreads();
  const long long rnd64 = 1ll << (31 + sh);
  int acc[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) acc[i] = ((threadIdx.x * 977 + i * 131071) ^ 0x5a5a) & 0x1FFFFF;
  uint32_t sum = 0;
  const unsigned long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
    const int ch0 = (it * 16) & 255;
    int y[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const bool f = (i * kF) / 16 != ((i + 1) * kF) / 16;
      if (f) { const double2 k = smc[ch0 + i]; y[i] = rq_f64(acc[i] - (1 << 20), k.x, k.y); }
      else y[i] = rq1w(acc[i] - (1 << 20), sm0[ch0 + i], sh, rnd64);
    }
    uint32_t wd[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) wd[q] = relu4(pack4_sat(y[4 * q], y[4 * q + 1], y[4 * q + 2], y[4 * q + 3]));
    sout[threadIdx.x & 1023] = make_uint4(wd[0], wd[1], wd[2], wd[3]);
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = (acc[i] + 0x10101 * (it + 1)) & 0x1FFFFF;     // |acc - 2^20| stays below 2^21
    sum += wd[0] + wd[3] * 3u + wd[1] * 5u + wd[2] * 7u;
  }
  const unsigned long long t1 = clock64();
  if (threadIdx.x == 0) out_clk[blockIdx.x] = t1 - t0;
  out_sum[blockIdx.x * blockDim.x + threadIdx.x] = sum;      // a function of the requantised values alone
}

// both forms on every accumulator in [-2^21, 2^21) for a few multipliers and shifts; the constants of
// the fp64 form come from the host
struct F64Case { int m0, sh; double ms, c; };
__global__ void check_f64(const F64Case* __restrict__ cases, int n, unsigned long long* bad) {
  const int a = (int)(blockIdx.x * blockDim.x + threadIdx.x) - (1 << 21);
  unsigned long long nb = 0;
  for (int j = 0; j < n; ++j) {
    const F64Case k = cases[j];
    nb += rq1w(a, k.m0, k.sh, 1ll << (31 + k.sh)) != rq_f64(a, k.ms, k.c);
  }
  if (nb) atomicAdd(bad, nb);
}

template <int kF>
void run_f64(const char* name, const int* dm0, unsigned long long* dclk, uint32_t* dsum, uint32_t* ref) {
  const int iters = 2000;
  for (int warps : {4, 16, 20}) {
    bench_f64<kF><<<1, warps * 32>>>(dm0, iters, 7, dclk, dsum);
    cudaDeviceSynchronize();
    bench_f64<kF><<<1, warps * 32>>>(dm0, iters, 7, dclk, dsum);
    cudaError_t e = cudaDeviceSynchronize();
    unsigned long long clk = 0;
    cudaMemcpy(&clk, dclk, sizeof(clk), cudaMemcpyDeviceToHost);
    uint32_t h[1024];
    cudaMemcpy(h, dsum, 4 * warps * 32, cudaMemcpyDeviceToHost);
    uint32_t x = 0;
    for (int i = 0; i < warps * 32; ++i) x = x * 31 + h[i];
    const char* same = "";
    if (kF == 0) ref[warps] = x; else same = ref[warps] == x ? "same results" : "DIFFERENT results";
    printf("%-32s warps/SM %2d: %7.1f clk per chunk per warp, %6.2f activations/clk/SM  (%s) %s\n", name, warps,
           (double)clk / iters, 16.0 * 32 * warps * iters / (double)clk, cudaGetErrorString(e), same);
  }
}

int main() {
  int hm0[256];
  for (int i = 0; i < 256; ++i) hm0[i] = (1 << 30) + i * 3000017;
  int* dm0; unsigned long long* dclk; uint32_t* dsum;
  cudaMalloc(&dm0, sizeof(hm0)); cudaMalloc(&dclk, 1024); cudaMalloc(&dsum, 4 * 2048);
  cudaMemcpy(dm0, hm0, sizeof(hm0), cudaMemcpyHostToDevice);
  run_regs<0, true>("regs: wide mad, smem consts", dm0, dclk, dsum);
  run_regs<0, false>("regs: wide mad, reg consts", dm0, dclk, dsum);
  run_regs<1, true>("regs: mulhi + add", dm0, dclk, dsum);
  run_regs<3, true>("regs: float (not exact)", dm0, dclk, dsum);
  run_tmem<1>("tmem: ld16, wait, compute", dm0, dclk, dsum);
  run_tmem<3>("tmem: load of the next piece in flight", dm0, dclk, dsum);
  // the fp64 form: exact? and does the fp64 pipe add throughput beside the integer pipes?
  F64Case cases[12 * 13];
  for (int i = 0; i < 12; ++i)
    for (int sh = 0; sh <= 12; ++sh) {
      const int m0 = i == 0 ? 1 << 30 : (i == 1 ? (1 << 30) + 1 : (i == 2 ? 0x7FFFFFFF : hm0[i]));
      const double ms = ldexp((double)m0, -(32 + sh));
      cases[i * 13 + sh] = F64Case{m0, sh, ms, 0.5 - 4503601774854144.0 * ms};
    }
  F64Case* dcases;
  cudaMalloc(&dcases, sizeof(cases));
  cudaMemcpy(dcases, cases, sizeof(cases), cudaMemcpyHostToDevice);
  cudaMemset(dclk, 0, 8);
  check_f64<<<(1 << 22) / 256, 256>>>(dcases, 12 * 13, dclk);
  unsigned long long bad = 1;
  cudaDeviceSynchronize();
  cudaMemcpy(&bad, dclk, 8, cudaMemcpyDeviceToHost);
  printf("fp64 form against the integer form, 2^22 accumulators x 12 multipliers x 13 shifts: %llu mismatches\n", bad);
  cudaMemcpy(dm0, hm0, sizeof(hm0), cudaMemcpyHostToDevice);
  uint32_t ref[64] = {0};
  run_f64<0>("regs: integer form (same loop)", dm0, dclk, dsum, ref);
  run_f64<16>("regs: fp64 form, all columns", dm0, dclk, dsum, ref);
  run_f64<4>("regs: 4 of 16 columns fp64", dm0, dclk, dsum, ref);
  run_f64<8>("regs: 8 of 16 columns fp64", dm0, dclk, dsum, ref);
  run_f64<12>("regs: 12 of 16 columns fp64", dm0, dclk, dsum, ref);
  return 0;
}
