// One flow level of the integer-only discrete flow on sm_100a, one CTA per group of images.
//
// The CTA keeps the level's flow variable v (int32, planar [channel][pixel]) in shared memory for
// all couplings of the level, so global memory is touched only for the level's input, its outputs
// and the packed weights (which stay in L2). Per coupling (Eq. 2, Sec. 3):
//
//   x_a -> int8 (input requant)                                     workers, exact 64-bit rq
//   per 128-pixel tile:
//     A1 = im2col(x_a)            [128 x 9*cpad]                    workers -> shared memory
//     D1 = A1 * W1^T              tcgen05.mma kind::i8, int32 in TMEM (control thread issues)
//     A2 = clip(ReLU(rq(D1)))     TMEM -> registers -> shared memory (int8, MMA operand layout)
//     D2 = A2 * W2^T ; A3 = clip(ReLU(rq(D2)))                      (the 1x1 conv)
//     D3 = A3 * W3'^T             W3' has one row per (tap, out channel): the nine per-tap partial
//                                 products of the last 3x3 conv for the tile's pixels
//     acc[q] += D3[p][tap]        each partial product is added to the output pixel q = p - tap
//                                 offset (zero padding = dropped terms), int32 atomics in shared
//   x_b +/-= rq(acc + bias)       exact 64-bit rq; + encodes, - decodes
//
// Computing the last conv as "GEMM to per-tap partials, then shifted sum" needs no halo of the
// hidden activations, which therefore never leave the SM. Integer addition is associative, so the
// result is bit-identical to the direct sum of Eq. 5.
//
// Squeeze, channel permutation and split are index maps: v is loaded in squeeze order, each
// coupling addresses v through its table of physical columns (the composition of all permutations
// so far), and the level's outputs are written through the final table.
//
// Execution structure: 16 worker warps and one control warp. All workers work on the same phase
// of one tile (four warps per TMEM lane quarter split the columns four ways). Two tiles are in
// flight, each with its own A-operand buffer and TMEM columns, and their phases alternate:
// build(A) build(B) epi1(A) epi1(B) epi2(A) epi2(B) scatter(A) scatter(B). A worker that has
// finished its part of a phase arrives on the tile's "A ready" mbarrier and goes straight on to the
// other tile's phase (after waiting for that tile's accumulator); the control thread waits for the
// arrivals, issues the tile's next MMAs and commits them to the tile's "D ready" mbarrier. So the
// tensor core always works under a requantisation phase and no worker waits for an MMA issue. The
// control thread also issues the bulk copies that bring the next coupling's weights in.
#include "iodf_dev.h"
#include "level_kernel.h"
#include "ptx.cuh"

namespace iodf {

namespace {

struct __align__(16) Ctl {
  uint64_t a_ready[2];    // workers -> control: the tile slot's A operand is written (count = worker warps)
  uint64_t d_ready[2];    // tensor core -> workers: the tile slot's accumulator is complete
  uint64_t w_full[3];     // bulk copy -> control: weight slot (or ring slot) filled
  uint64_t w_empty[3];    // tensor core -> control: the MMAs reading a ring slot have completed
  uint64_t meta_full[2];  // bulk copy -> everyone: meta block of step (i & 1) has landed
  uint32_t tmem_base;
  uint32_t abort;
};

struct Ctx {
  uint8_t* smem;
  Ctl* ctl;
  uint32_t* status;
  int tid, warp, lane;
  int wq;                 // TMEM lane quarter of this warp
  int cs, ncs;            // column-split index and count of the epilogues (all replicas together)
  int bcs, bncs;          // column-split index and count of the im2col build (within one lane quarter)
  int row;                // tile row (= TMEM lane) of this thread
  int rep, rrows;         // row replication (see LevelPlan::rep) and rows per replica (128 / rep)
  uint32_t tmem_base;     // first allocated TMEM column, lane field 0
  uint32_t tmem_slot;     // current tile slot's first column, this warp's lane quarter
};

// Bounded wait of this kernel: see ptx::bounded_wait.
__device__ __forceinline__ bool wait_bar(Ctl* ctl, uint32_t* status, uint64_t* bar, uint32_t parity) {
  return ptx::bounded_wait(&ctl->abort, status, bar, parity, kSpinLimit);
}

// The control thread's waits are short and on the critical path of every tile phase: it polls
// inline first (no call, no suspension) and only then falls back to the bounded blocking wait.
__device__ __forceinline__ void spin_then_wait(Ctl* ctl, uint32_t* status, uint64_t* bar, uint32_t b, uint32_t parity) {
  for (int it = 0; it < 2048; ++it)
    if (ptx::mbar_test_wait(b, parity)) return;
  wait_bar(ctl, status, bar, parity);
}
__device__ __forceinline__ void spin_then_wait(Ctl* ctl, uint32_t* status, uint64_t* bar, uint32_t parity) {
  spin_then_wait(ctl, status, bar, ptx::smem_u32(bar), parity);
}

__device__ __forceinline__ void cta_barrier() { __syncthreads(); }


__device__ __forceinline__ int32_t rq_exact(int32_t a, int32_t m0, int32_t s) {
  const long long p = (long long)a * (long long)m0 + (1ll << (30 + s));
  if (s >= 1) return ((int32_t)(p >> 32)) >> (s - 1);   // same value, one 32-bit shift
  return (int32_t)(p >> 31);
}

// rq(acc + bias) with the channel's precomputed c64 = bias * m0 + 2^(30+s): one 64-bit multiply-add,
// then the high word shifted by s - 1 (s >= 1) or the 64-bit value shifted by 31 (s = 0).
__device__ __forceinline__ int32_t rq_out(int32_t acc, const OutRq o) {
  const long long c64 = (long long)(((unsigned long long)o.c_hi << 32) | (unsigned long long)o.c_lo);
  const long long p = (long long)acc * (long long)o.m0 + c64;
  const int32_t hi = (int32_t)(p >> 32);
  return o.s >= 1 ? (hi >> (o.s - 1)) : (int32_t)__funnelshift_r((uint32_t)p, (uint32_t)hi, 31);
}

__device__ __forceinline__ int clampi(int v, int lo, int hi) { return min(max(v, lo), hi); }

// n / d with the plan's magic multiplier ceil(2^32 / d) (0 stands for d = 1); exact while n * d < 2^32
__device__ __forceinline__ int fdiv(int n, uint32_t mul) { return mul ? (int)__umulhi((uint32_t)n, mul) : n; }

__device__ __forceinline__ uint32_t pack4(int y0, int y1, int y2, int y3) {
  const uint32_t a = __byte_perm((uint32_t)y0, (uint32_t)y1, 0x0040);
  const uint32_t b = __byte_perm((uint32_t)y2, (uint32_t)y3, 0x0040);
  return __byte_perm(a, b, 0x5410);
}

// Pixel bookkeeping of one tile row.
struct RowPos {
  int p;            // pixel slot in the CTA (group-local)
  bool valid;
  uint32_t gmask;   // bit t=(u*3+v): input pixel (i+u-1, j+v-1) is inside the image   (gather)
  uint32_t smask;   // bit t: output pixel (i-u+1, j-v+1) is inside the image           (scatter)
};

// Packed row record: bit 0 valid, bits 1..9 gather mask, bits 10..18 scatter mask.
__device__ __forceinline__ uint32_t row_record(int p, int pvalid, int px, int h, int w, uint32_t mul_px,
                                               uint32_t mul_w) {
  if (p >= pvalid) return 0u;
  uint32_t r = 1u;
  const int q = p - fdiv(p, mul_px) * px;
  const int i = fdiv(q, mul_w), j = q - i * w;
#pragma unroll
  for (int u = 0; u < 3; ++u)
#pragma unroll
    for (int v = 0; v < 3; ++v) {
      const bool gi = (i + u - 1 >= 0) && (i + u - 1 < h) && (j + v - 1 >= 0) && (j + v - 1 < w);
      const bool si = (i - u + 1 >= 0) && (i - u + 1 < h) && (j - v + 1 >= 0) && (j - v + 1 < w);
      r |= (gi ? 1u : 0u) << (1 + u * 3 + v);
      r |= (si ? 1u : 0u) << (10 + u * 3 + v);
    }
  return r;
}

// row: the thread's tile row; prow: its row within the replica (the same unless rows are replicated)
__device__ __forceinline__ RowPos row_pos(const uint32_t* rowinfo, int tile, int row, int prow) {
  RowPos r;
  r.p = tile * kTileM + prow;
  const uint32_t rec = rowinfo[tile * kTileM + row];
  r.valid = (rec & 1u) != 0;
  r.gmask = (rec >> 1) & 0x1FFu;
  r.smask = (rec >> 10) & 0x1FFu;
  return r;
}

// A[row][tap*cpad + c] = xa[p + tap offset][c] (0 outside the image), as aligned 8-byte granules,
// followed by the granule of bias columns (where K has room for it), written in 16-byte chunks into
// the MMA operand layout [K/16][128][16]. Where each granule comes from is a property of the level,
// not of the pixel: the host tabulates, per granule, the byte offset of its source relative to the
// pixel's own xa record and the bit of the row's gather mask that validates it (9: the bias
// granule, 10: padding), so a granule costs one table read, one mask test and one predicated load.
// kPairs: cpad is a multiple of 16, so the two granules of a chunk belong to one tap and come with
// one 16-byte load.
template <bool kPairs>
__device__ __forceinline__ uint4 im2col_chunk(const int8_t* __restrict__ base, const int2* __restrict__ tab, int jc,
                                              uint32_t gmask) {
  if (kPairs) {
    const int2 e = tab[2 * jc];
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if ((gmask >> e.y) & 1u) v = *reinterpret_cast<const uint4*>(base + e.x);
    if (e.y == kGranBias) v = make_uint4(kBiasColumnsLo, kBiasColumnsHi, 0u, 0u);
    return v;
  }
  const int4 e = *reinterpret_cast<const int4*>(tab + 2 * jc);       // both granules' entries
  uint2 g0 = make_uint2(0u, 0u), g1 = make_uint2(0u, 0u);
  if ((gmask >> e.y) & 1u) g0 = *reinterpret_cast<const uint2*>(base + e.x);
  if ((gmask >> e.w) & 1u) g1 = *reinterpret_cast<const uint2*>(base + e.z);
  if (e.y == kGranBias) g0 = make_uint2(kBiasColumnsLo, kBiasColumnsHi);
  if (e.w == kGranBias) g1 = make_uint2(kBiasColumnsLo, kBiasColumnsHi);
  return make_uint4(g0.x, g0.y, g1.x, g1.y);
}

template <bool kPairs>
__device__ __forceinline__ void build_im2col_t(const Ctx& cx, uint8_t* __restrict__ sA, const int8_t* __restrict__ xa,
                                               const int2* __restrict__ tab, int cpad, int kd, const RowPos rp) {
  const int nchunks = kd >> 4;
  const int8_t* base = xa + (size_t)rp.p * cpad;
  uint8_t* out = sA + cx.row * 16;
  int jc = cx.bcs;
  for (; jc + cx.bncs < nchunks; jc += 2 * cx.bncs) {          // two chunks at a time: independent loads
    const uint4 c0 = im2col_chunk<kPairs>(base, tab, jc, rp.gmask);
    const uint4 c1 = im2col_chunk<kPairs>(base, tab, jc + cx.bncs, rp.gmask);
    *reinterpret_cast<uint4*>(out + (size_t)jc * (kTileM * 16)) = c0;
    *reinterpret_cast<uint4*>(out + (size_t)(jc + cx.bncs) * (kTileM * 16)) = c1;
  }
  if (jc < nchunks)
    *reinterpret_cast<uint4*>(out + (size_t)jc * (kTileM * 16)) = im2col_chunk<kPairs>(base, tab, jc, rp.gmask);
}

__device__ __forceinline__ void build_im2col(const Ctx& cx, uint8_t* __restrict__ sA, const int8_t* __restrict__ xa,
                                             const int2* __restrict__ tab, int cpad, int kd, const RowPos rp) {
  if ((cpad & 15) == 0) build_im2col_t<true>(cx, sA, xa, tab, cpad, kd, rp);
  else build_im2col_t<false>(cx, sA, xa, tab, cpad, kd, rp);
}

// Requantisation flavours of a hidden layer (chosen per layer when the model is packed):
//   kModeFolded   the same shift s >= 1 for every channel and the bias already in the accumulator
//                 (bias rows of the GEMM): constant m0 per channel, y = hi32(acc * m0 + 2^(30+s)) >> (s-1)
//   kModeUniform  every channel has the same shift s >= 1: constants {m0, bias} per channel,
//                 y = hi32((acc + bias) * m0 + 2^(30+s)) >> (s-1)
//   kModeFast     per-channel shifts, all s >= 1: y = hi32(acc * m0 + c64) >> (s-1)
//   kModeExact    any s: y = (acc * m0 + c64) >> (31 + s) in 64 bits
// All three are exact: for s >= 1, floor(x / 2^(31+s)) = floor(floor(x / 2^32) / 2^(s-1)).
constexpr int kModeFolded = 3, kModeUniform = 2, kModeFast = 1, kModeExact = 0;

// Clip flavours: kClipS8Relu is the common ReLU + clip to [0, 127]: the saturating 32->8 bit pack
// clips to [-128, 127] and the negative bytes are then cleared; kClipU8Relu is ReLU + clip to
// [0, 255] (unsigned activations, Sec. 4.1), which the unsigned saturating pack does by itself;
// kClipAny is max/min with the layer's bounds.
constexpr int kClipS8Relu = 1, kClipU8Relu = 2, kClipAny = 0;

// d = {sat8(y3), sat8(y2), sat8(y1), sat8(y0)} (y0 in the lowest byte)
__device__ __forceinline__ uint32_t pack4_sat(int y0, int y1, int y2, int y3) {
  uint32_t t, w;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(y3), "r"(y2), "r"(0));
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(y1), "r"(y0), "r"(t));
  return w;
}
// d = {satu8(y3), satu8(y2), satu8(y1), satu8(y0)}: clip(y, 0, 255) of four values
__device__ __forceinline__ uint32_t pack4_sat_u8(int y0, int y1, int y2, int y3) {
  uint32_t t, w;
  asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(y3), "r"(y2), "r"(0));
  asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(y1), "r"(y0), "r"(t));
  return w;
}
// clip(y, 0, 127) of four values: saturate to int8 while packing, then clear the negative bytes
// (a byte permute with sign replication builds the mask): two instructions for the four ReLUs.
__device__ __forceinline__ uint32_t pack4_relu_sat(int y0, int y1, int y2, int y3) {
  const uint32_t w = pack4_sat(y0, y1, y2, y3);
  uint32_t neg;          // every byte replaced by eight copies of its sign bit
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(neg) : "r"(w), "r"(0u), "r"(0xBA98u));
  return w & ~neg;
}

template <int kMode, int kClip>
struct Requant {
  const HiddenRq* __restrict__ rq;     // kModeFast / kModeExact
  const int2* __restrict__ mb;         // kModeUniform: {m0, bias}
  int lo, hi, sh;
  long long rnd64;

  __device__ __forceinline__ int one(int acc, int ch) const {
    int y;
    if (kMode == kModeUniform) {
      const int2 c = mb[ch];
      const long long p = (long long)(acc + c.y) * (long long)c.x + rnd64;
      y = ((int)(p >> 32)) >> sh;
    } else {
      const HiddenRq r = rq[ch];
      const long long c64 = (long long)(((unsigned long long)r.c_hi << 32) | (unsigned long long)r.c_lo);
      const long long p = (long long)acc * (long long)r.m0 + c64;
      if (kMode == kModeFast) y = ((int)(p >> 32)) >> r.sh;
      else y = (int)(p >> (32 + r.sh));
    }
    return kClip != kClipAny ? y : clampi(y, lo, hi);        // otherwise clipped while packing
  }
  // 16 accumulator columns starting at channel ch0 -> one 16-byte chunk of the next A operand
  __device__ __forceinline__ uint4 chunk(const uint32_t* r, int ch0) const {
    uint32_t wd[4];
    if (kMode == kModeFolded) {
      // multipliers of four channels per 16-byte shared-memory load
      const int4* q = reinterpret_cast<const int4*>(reinterpret_cast<const int32_t*>(mb) + ch0);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int4 c = q[i];
        const int y0 = uniform_one((int)r[4 * i], c.x, 0), y1 = uniform_one((int)r[4 * i + 1], c.y, 0);
        const int y2 = uniform_one((int)r[4 * i + 2], c.z, 0), y3 = uniform_one((int)r[4 * i + 3], c.w, 0);
        wd[i] = pack_clipped(y0, y1, y2, y3);
      }
    } else if (kMode == kModeUniform) {
      // {m0, bias} pairs of two channels per 16-byte shared-memory load (the table is 16-byte aligned)
      const int4* q = reinterpret_cast<const int4*>(mb + ch0);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int4 c01 = q[2 * i], c23 = q[2 * i + 1];
        const int y0 = uniform_one((int)r[4 * i], c01.x, c01.y), y1 = uniform_one((int)r[4 * i + 1], c01.z, c01.w);
        const int y2 = uniform_one((int)r[4 * i + 2], c23.x, c23.y), y3 = uniform_one((int)r[4 * i + 3], c23.z, c23.w);
        wd[i] = pack_clipped(y0, y1, y2, y3);
      }
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int y0 = one((int)r[4 * i], ch0 + 4 * i), y1 = one((int)r[4 * i + 1], ch0 + 4 * i + 1);
        const int y2 = one((int)r[4 * i + 2], ch0 + 4 * i + 2), y3 = one((int)r[4 * i + 3], ch0 + 4 * i + 3);
        wd[i] = pack_clipped(y0, y1, y2, y3);
      }
    }
    return make_uint4(wd[0], wd[1], wd[2], wd[3]);
  }
  __device__ __forceinline__ int uniform_one(int acc, int m0, int bias) const {
    const long long p = (long long)(acc + bias) * (long long)m0 + rnd64;
    const int y = ((int)(p >> 32)) >> sh;
    return kClip != kClipAny ? y : clampi(y, lo, hi);
  }
  __device__ __forceinline__ uint32_t pack_clipped(int y0, int y1, int y2, int y3) const {
    return kClip == kClipS8Relu ? pack4_relu_sat(y0, y1, y2, y3)
                                : (kClip == kClipU8Relu ? pack4_sat_u8(y0, y1, y2, y3) : pack4(y0, y1, y2, y3));
  }
};

// TMEM accumulator -> requantised int8 activations in the next GEMM's A layout. n is a multiple
// of 16; kd (the next GEMM's K) is n rounded up to 32, the extra chunk being zero. The unit of work
// is one 16-column chunk (= one 16-byte piece of the A row), dealt round-robin to the column
// splits so that they differ by at most one chunk; a warp takes its chunks two at a time.
template <int kMode, int kClip>
__device__ __forceinline__ void epilogue_hidden_t(const Ctx& cx, int n, int kd, const Requant<kMode, kClip> q,
                                                  uint32_t pad_lo, uint32_t pad_hi, uint8_t* __restrict__ sOut) {
  const int nch = n >> 4;
  // A chunk goes to this thread's row in every replica of the tile (one replica: the row itself).
  uint8_t* out = sOut + cx.row * 16;
  const bool replicated = cx.rep > 1;
  auto put = [&](int chunk, const uint4 val) {
    *reinterpret_cast<uint4*>(out + (size_t)chunk * (kTileM * 16)) = val;
    if (replicated) {
      uint8_t* base = sOut + (size_t)chunk * (kTileM * 16);
      for (int k = 1; k < cx.rep; ++k)
        *reinterpret_cast<uint4*>(base + ((cx.row + k * cx.rrows) & (kTileM - 1)) * 16) = val;
    }
  };
  // chunks past the data: the first one starts with the bias columns of the next GEMM (pad_lo,
  // pad_hi; zero if it has none), the others are zero
  for (int j = nch + ((cx.cs - nch) & (cx.ncs - 1)); j < (kd >> 4); j += cx.ncs)
    put(j, j == nch ? make_uint4(pad_lo, pad_hi, 0u, 0u) : make_uint4(0u, 0u, 0u, 0u));
  int ch = cx.cs;
  for (; ch + cx.ncs < nch; ch += 2 * cx.ncs) {
    const int ch2 = ch + cx.ncs;
    uint32_t ra[16], rb[16];
    ptx::tmem_ld16(cx.tmem_slot + (uint32_t)(ch << 4), ra);
    ptx::tmem_ld16(cx.tmem_slot + (uint32_t)(ch2 << 4), rb);
    ptx::tmem_ld_wait16(ra);
    ptx::tmem_ld_wait16(rb);
    put(ch, q.chunk(ra, ch << 4));
    put(ch2, q.chunk(rb, ch2 << 4));
  }
  if (ch < nch) {
    uint32_t ra[16];
    ptx::tmem_ld16(cx.tmem_slot + (uint32_t)(ch << 4), ra);
    ptx::tmem_ld_wait16(ra);
    put(ch, q.chunk(ra, ch << 4));
  }
}

// mode: layer flavour (see above); us: the layer's uniform shift (kModeUniform only).
__device__ __forceinline__ void epilogue_hidden(const Ctx& cx, int mode, int us, int n, int kd, const HiddenRq* rq,
                                                const int2* mb, int lo, int hi, uint32_t pad_lo, uint32_t pad_hi,
                                                uint8_t* sOut) {
  const bool s8relu = lo == 0 && hi == 127, u8relu = lo == 0 && hi == 255;
  if (mode >= kModeUniform) {
    const long long rnd64 = 1ll << (30 + us);
    if (mode == kModeFolded) {
      if (s8relu) epilogue_hidden_t(cx, n, kd, Requant<kModeFolded, kClipS8Relu>{rq, mb, lo, hi, us - 1, rnd64}, pad_lo, pad_hi, sOut);
      else if (u8relu) epilogue_hidden_t(cx, n, kd, Requant<kModeFolded, kClipU8Relu>{rq, mb, lo, hi, us - 1, rnd64}, pad_lo, pad_hi, sOut);
      else epilogue_hidden_t(cx, n, kd, Requant<kModeFolded, kClipAny>{rq, mb, lo, hi, us - 1, rnd64}, pad_lo, pad_hi, sOut);
    } else {
      if (s8relu) epilogue_hidden_t(cx, n, kd, Requant<kModeUniform, kClipS8Relu>{rq, mb, lo, hi, us - 1, rnd64}, pad_lo, pad_hi, sOut);
      else epilogue_hidden_t(cx, n, kd, Requant<kModeUniform, kClipAny>{rq, mb, lo, hi, us - 1, rnd64}, pad_lo, pad_hi, sOut);
    }
  } else if (mode == kModeFast) {
    epilogue_hidden_t(cx, n, kd, Requant<kModeFast, kClipAny>{rq, mb, lo, hi, 0, 0}, pad_lo, pad_hi, sOut);
  } else {
    epilogue_hidden_t(cx, n, kd, Requant<kModeExact, kClipAny>{rq, mb, lo, hi, 0, 0}, pad_lo, pad_hi, sOut);
  }
}

// Per-tap partial products -> shifted sum into the translation accumulator.
// Column granule (tap, gq) holds out channels gq*8 .. gq*8+8 of that tap. The partial product of
// pixel p and tap (du, dv) belongs to output pixel p - (du-1)*w - (dv-1). Consecutive lanes hold
// consecutive pixels, so the three dv-contributions that meet in one output pixel sit in lanes
// L-1, L, L+1: they are summed with two warp shuffles, and one shared-memory atomic per (du,
// channel) adds the row sum. A warp's two edge lanes add their outward contribution themselves.
// Masked contributions (target outside the image) are zero before the shuffle. Work unit =
// (du, gq); units are dealt round-robin to the column splits.
__device__ void epilogue_scatter(const Ctx& cx, int cb, int cbp, int32_t* __restrict__ acc, int pg, int w,
                                 const RowPos rp) {
  const int gpt = cbp >> 3;
  const int nunits = 3 * gpt;
  const uint32_t sm = rp.valid ? rp.smask : 0u;
  const bool rows_align = (32 % w) == 0;     // every image row lies inside one warp's 32 pixels
  for (int u = cx.cs; u < nunits; u += cx.ncs) {
    const int du = (u >= 2 * gpt) ? 2 : ((u >= gpt) ? 1 : 0);
    const int gq = u - du * gpt;
    uint32_t r0[8], r1[8], r2[8];
    ptx::tmem_ld8(cx.tmem_slot + (uint32_t)(((du * 3 + 0) * gpt + gq) << 3), r0);
    ptx::tmem_ld8(cx.tmem_slot + (uint32_t)(((du * 3 + 1) * gpt + gq) << 3), r1);
    ptx::tmem_ld8(cx.tmem_slot + (uint32_t)(((du * 3 + 2) * gpt + gq) << 3), r2);
    ptx::tmem_ld_wait8(r0);
    ptx::tmem_ld_wait8(r1);
    ptx::tmem_ld_wait8(r2);
    const bool ok_m = ((sm >> (du * 3 + 0)) & 1u) != 0;   // dv = -1: target column j + 1
    const bool ok_0 = ((sm >> (du * 3 + 1)) & 1u) != 0;   // dv =  0: target column j
    const bool ok_p = ((sm >> (du * 3 + 2)) & 1u) != 0;   // dv = +1: target column j - 1
    const int c0 = gq << 3;
    // this lane's own output pixel for this du; the row sum is zero whenever that pixel is
    // outside the image (all three contributions share its row, hence its vertical validity)
    const uint32_t dst = ptx::smem_u32(acc + c0 * pg + rp.p - (du - 1) * w);
    const uint32_t plane = (uint32_t)pg * 4u;
    if (rows_align) {
      // Image rows never straddle a warp (w divides 32): the lane that a rotating shuffle wraps to
      // holds the first (last) pixel of a row, whose dv = +1 (-1) contribution is masked, i.e.
      // zero. So no edge handling is needed at all.
      // Masks are applied at the receiver as 0/1 multipliers (the neighbours' mask bits come over
      // with one shuffle per unit), so each channel costs two shuffles and three multiply-adds.
      const int k_0 = ok_0 ? 1 : 0;
      const int k_p = __shfl_sync(0xFFFFFFFFu, ok_p ? 1 : 0, (cx.lane + 1) & 31);
      const int k_m = __shfl_sync(0xFFFFFFFFu, ok_m ? 1 : 0, (cx.lane + 31) & 31);
      int sum[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int n_p = __shfl_sync(0xFFFFFFFFu, (int)r2[i], (cx.lane + 1) & 31);
        const int n_m = __shfl_sync(0xFFFFFFFFu, (int)r0[i], (cx.lane + 31) & 31);
        sum[i] = (int)r1[i] * k_0 + n_p * k_p + n_m * k_m;
      }
      if (ok_0) {      // the row sum is zero otherwise
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (c0 + i < cb) ptx::red_add_s32_always(dst + (uint32_t)i * plane, sum[i]);
      }
    } else {
      const bool edge_hi = cx.lane == 31 && ok_m, edge_lo = cx.lane == 0 && ok_p;
      int sum[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {                        // branch-free: eight independent chains
        const int v_m = ok_m ? (int)r0[i] : 0;
        const int v_0 = ok_0 ? (int)r1[i] : 0;
        const int v_p = ok_p ? (int)r2[i] : 0;
        const int from_next = __shfl_down_sync(0xFFFFFFFFu, v_p, 1);   // lane L+1's dv=+1 lands here
        const int from_prev = __shfl_up_sync(0xFFFFFFFFu, v_m, 1);     // lane L-1's dv=-1 lands here
        sum[i] = v_0 + (cx.lane < 31 ? from_next : 0) + (cx.lane > 0 ? from_prev : 0);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const bool ch = c0 + i < cb;
        ptx::red_add_s32(dst + (uint32_t)i * plane, sum[i], ch && ok_0);
        ptx::red_add_s32(dst + (uint32_t)i * plane + 4u, (int)r0[i], ch && edge_hi);
        ptx::red_add_s32(dst + (uint32_t)i * plane - 4u, (int)r2[i], ch && edge_lo);
      }
    }
  }
}

// Prior head accumulator -> (mu, log-scale index) in global memory.
__device__ void epilogue_prior(const Ctx& cx, const LevelPlan& P, const LevelArgs& a, const PriorMeta& M,
                               const OutRq* orq, int img0, const RowPos rp) {
  const int cb = P.cb, px = P.px;
  const int g = rp.valid ? rp.p / px : 0;
  const int q = rp.p - g * px;
  int32_t* mu = a.prior + (size_t)(img0 + g) * 2u * P.d_fact + P.prior_off + q;
  int32_t* ls = mu + P.d_fact;
  const int ngran = (2 * cb + 7) >> 3;
  for (int gi = cx.cs; gi < ngran; gi += cx.ncs) {
    uint32_t r[8];
    ptx::tmem_ld8(cx.tmem_slot + (uint32_t)(gi << 3), r);
    ptx::tmem_ld_wait8(r);
    if (rp.valid) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int col = (gi << 3) + i;
        if (col < 2 * cb) {
          const OutRq o = orq[col];
          const int32_t y = rq_out((int32_t)r[i], o);
          if (col < cb) mu[(size_t)col * px] = y;
          else ls[(size_t)(col - cb) * px] = clampi(y, M.ls_lo, M.ls_hi);
        }
      }
    }
  }
}

// ---- step bookkeeping shared by workers and control -------------------------------------------
struct Steps {
  int n_couplings, nsteps;
  bool do_prior, inverse;
  __device__ bool is_prior(int i) const { return do_prior && (inverse ? i == 0 : i == nsteps - 1); }
  __device__ int coupling_index(int i) const {
    return inverse ? (n_couplings - 1 - (i - (do_prior ? 1 : 0))) : i;
  }
};

__device__ __forceinline__ const BlockRef& step_ref(const LevelPlan& P, const Steps& st, int i) {
  return st.is_prior(i) ? P.prior : P.coupling[st.coupling_index(i)];
}

// ---- MMA issue and weight traffic (elected threads) --------------------------------------------
// D[128 x n] (+)= A[128 x kd] * B[n x kd]^T for B rows n0..n0+n of a matrix with n_total rows.
// The control thread competes for issue slots with sixteen busy worker warps, so the loop body is
// kept to the MMA and two descriptor increments (K advances by 32 bytes = two 16-byte chunks).
__device__ __forceinline__ void issue_gemm(uint32_t d_tmem, uint32_t sa, uint32_t sb, int n_total, int n0, int n,
                                           int kd, bool a_unsigned) {
  const uint32_t idesc = ptx::umma_idesc_i8((uint32_t)n, a_unsigned);
  const uint32_t lbo_b = (uint32_t)n_total * 16u;
  uint64_t da = ptx::umma_desc(sa, kTileM * 16, 128);
  uint64_t db = ptx::umma_desc(sb + (uint32_t)n0 * 16u, lbo_b, 128);
  const uint64_t da_step = (uint64_t)((2u * kTileM * 16u) >> 4);
  const uint64_t db_step = (uint64_t)((2u * lbo_b) >> 4);
  const int ksteps = kd >> 5;
  ptx::umma_i8_first(d_tmem, da, db, idesc);
  for (int k = 1; k < ksteps; ++k) {
    da += da_step;
    db += db_step;
    ptx::umma_i8_acc(d_tmem, da, db, idesc);
  }
}

__device__ __forceinline__ void bulk_load(const Ctx& cx, const uint8_t* blob, uint32_t off, uint32_t bytes,
                                          uint32_t s_dst, uint64_t* bar) {
  const uint32_t b = ptx::smem_u32(bar);
  ptx::mbar_expect_tx(b, bytes);
  ptx::bulk_g2s(ptx::smem_u32(cx.smem + s_dst), blob + off, bytes, b);
}

// Weight bookkeeping. Slots hold, in order of use: S0 the first matrix of every step (W1 of a
// coupling, the prior head's matrix), S1 every coupling's W2, S2 every coupling's W3. A slot's
// k-th load completes phase k of its mbarrier, so a consumer that knows k knows the parity to wait
// for. With `alias` (one group only) S0 instead alternates W1 and W3 for every tile, S2 is unused,
// and the single elected thread counts S0's loads itself.
struct Weights {
  int cur_step[3];        // loader: step whose matrix the slot holds or is receiving (-1: none)
  uint32_t s0_loads;      // alias mode: loads requested into S0
  uint32_t s0_used;       // alias mode: loads consumed from S0
};

__device__ __forceinline__ bool slot_used_by(const Steps& st, int s, int step) {
  return s == 0 || !st.is_prior(step);
}
// ordinal of step i among the loads of slot s
__device__ __forceinline__ int load_ordinal(const Steps& st, int s, int i) {
  return (s == 0) ? i : i - ((st.inverse && st.do_prior) ? 1 : 0);
}

// Loader: every slot whose matrix belongs to a finished step (<= done) receives the matrix of the
// next step that uses it.
__device__ void top_up(const Ctx& cx, const LevelPlan& P, const LevelArgs& a, const Steps& st, Weights& W, int done,
                       bool alias) {
  for (int s = alias ? 1 : 0; s < (alias ? 2 : 3); ++s) {
    if (W.cur_step[s] > done) continue;
    int j = W.cur_step[s] + 1;
    while (j < st.nsteps && !slot_used_by(st, s, j)) ++j;
    if (j >= st.nsteps) { W.cur_step[s] = st.nsteps; continue; }
    const BlockRef& br = step_ref(P, st, j);
    bulk_load(cx, a.blob, br.w_off[s], br.w_bytes[s], P.s_w[s], &cx.ctl->w_full[s]);
    W.cur_step[s] = j;
  }
}

// ---- control thread -----------------------------------------------------------------------------
// Issues, in the fixed order in which the workers produce them, the MMAs of every tile phase, and
// keeps the weight and meta slots filled. Takes part in the two CTA barriers of every step.
__device__ void run_control(const Ctx& cx, const LevelPlan& P, const LevelArgs& a, const Steps& st, int ntv) {
  uint8_t* smem = cx.smem;
  Ctl* ctl = cx.ctl;
  const bool lead = cx.lane == 0;
  const bool alias = P.w13_alias != 0;
  const int nslots = P.nslots;
  uint32_t apar[2] = {0u, 0u}, dpar[2] = {0u, 0u};
  Weights W;
  W.cur_step[0] = W.cur_step[1] = W.cur_step[2] = -1;
  W.s0_loads = W.s0_used = 0;

  if (lead) {
    for (int i = 0; i < st.nsteps && i < 2; ++i) {
      const BlockRef& br = step_ref(P, st, i);
      bulk_load(cx, a.blob, br.meta_off, br.meta_bytes, P.s_meta[i], &ctl->meta_full[i]);
    }
    top_up(cx, P, a, st, W, -1, alias);
    if (alias && st.nsteps > 0) {
      const BlockRef& br = step_ref(P, st, 0);
      bulk_load(cx, a.blob, br.w_off[0], br.w_bytes[0], P.s_w[0], &ctl->w_full[0]);
      W.s0_loads = 1;
    }
  }
  __syncwarp();
  cta_barrier();                         // the workers have loaded the flow variable
  // wait for tile slot sl's A operand, then D = A * W^T into the slot's TMEM columns
  auto mma = [&](int sl, int wslot, bool wait_w, uint32_t wpar, int n, int kd, bool au) {
    spin_then_wait(ctl, a.status, &ctl->a_ready[sl], apar[sl]);
    apar[sl] ^= 1u;
    if (wait_w) spin_then_wait(ctl, a.status, &ctl->w_full[wslot], wpar);
    ptx::tc_fence_after();
    const uint32_t sa = ptx::smem_u32(smem + P.s_a[sl]), sb = ptx::smem_u32(smem + P.s_w[wslot]);
    const uint32_t d = cx.tmem_base + (uint32_t)(sl * kSlotCols);
    for (int n0 = 0; n0 < n; n0 += 256) issue_gemm(d + (uint32_t)n0, sa, sb, n, n0, min(256, n - n0), kd, au);
    ptx::umma_commit(ptx::smem_u32(&ctl->d_ready[sl]));
  };
  // alias mode only: wait until the MMA just issued for slot 0 has completed, then refill S0
  auto s0_refill = [&](const BlockRef& br, int which) {
    wait_bar(ctl, a.status, &ctl->d_ready[0], dpar[0]);
    bulk_load(cx, a.blob, br.w_off[which], br.w_bytes[which], P.s_w[0], &ctl->w_full[0]);
    ++W.s0_loads;
  };

  for (int i = 0; i < st.nsteps; ++i) {
    const bool prior = st.is_prior(i);
    int n[3] = {0, 0, 0}, kd[3] = {0, 0, 0};
    bool au[3] = {false, false, false};      // A operand unsigned: hidden activations clipped above 127
    if (lead) {
      wait_bar(ctl, a.status, &ctl->meta_full[i & 1], (uint32_t)((i >> 1) & 1));
      const uint8_t* mb = smem + P.s_meta[i & 1];
      if (prior) {
        const PriorMeta* M = reinterpret_cast<const PriorMeta*>(mb);
        n[0] = M->n; kd[0] = M->kd;
      } else {
        const CouplingMeta* M = reinterpret_cast<const CouplingMeta*>(mb);
        n[0] = M->n1; n[1] = M->n2; n[2] = M->n3;
        kd[0] = M->kd1; kd[1] = M->kd2; kd[2] = M->kd3;
        au[1] = M->hi1 > 127; au[2] = M->hi2 > 127;
      }
    }
    cta_barrier();     // the workers have finished the pixel pass: step i-1's meta slot is free
    if (lead) {
      if (i >= 1 && i + 1 < st.nsteps) {
        const BlockRef& br = step_ref(P, st, i + 1);
        bulk_load(cx, a.blob, br.meta_off, br.meta_bytes, P.s_meta[(i + 1) & 1], &ctl->meta_full[(i + 1) & 1]);
      }
      const uint32_t par0 = (uint32_t)(load_ordinal(st, 0, i) & 1), par12 = (uint32_t)(load_ordinal(st, 1, i) & 1);
      const BlockRef& br = step_ref(P, st, i);
      const int nstages = prior ? 1 : 3;
      bool first = true;
      // Common case (a coupling, every matrix resident, no accumulator wider than one MMA): every
      // instruction of this thread between a tile's last arrival and its commit delays the tile, so
      // the descriptors of the step's three GEMMs are built once and the issue path is unrolled.
      const bool lean = !alias && !prior && n[0] <= 256 && n[1] <= 256 && n[2] <= 256;
      if (lean) {
        uint32_t idesc[3], db_lo[3], db_step[3];
        int ks[3];
#pragma unroll
        for (int sg = 0; sg < 3; ++sg) {
          const uint32_t lbo_b = (uint32_t)n[sg] * 16u;
          idesc[sg] = ptx::umma_idesc_i8((uint32_t)n[sg], au[sg]);
          db_lo[sg] = ptx::umma_desc_lo(ptx::smem_u32(smem + P.s_w[sg]), lbo_b);
          db_step[sg] = (2u * lbo_b) >> 4;
          ks[sg] = kd[sg] >> 5;
        }
        const uint32_t da_lo[2] = {ptx::umma_desc_lo(ptx::smem_u32(smem + P.s_a[0]), kTileM * 16),
                                   ptx::umma_desc_lo(ptx::smem_u32(smem + P.s_a[1]), kTileM * 16)};
        const uint32_t da_step = (2u * kTileM * 16u) >> 4;
        const uint32_t abar[2] = {ptx::smem_u32(&ctl->a_ready[0]), ptx::smem_u32(&ctl->a_ready[1])};
        const uint32_t dbar[2] = {ptx::smem_u32(&ctl->d_ready[0]), ptx::smem_u32(&ctl->d_ready[1])};
        // The step's matrices were requested when the previous step ended and are normally here by
        // now; waiting for them before the first arrival keeps the waits off the tiles' critical path.
#pragma unroll
        for (int sg = 0; sg < 3; ++sg) spin_then_wait(ctl, a.status, &ctl->w_full[sg], sg == 0 ? par0 : par12);
        for (int t0 = 0; t0 < ntv; t0 += nslots) {
          const int nt = min(nslots, ntv - t0);
#pragma unroll
          for (int sg = 0; sg < 3; ++sg) {
#pragma unroll
            for (int sl = 0; sl < 2; ++sl) {
              if (sl < nt) {
                spin_then_wait(ctl, a.status, &ctl->a_ready[sl], abar[sl], apar[sl]);
                apar[sl] ^= 1u;
                ptx::tc_fence_after();
                const uint32_t d = cx.tmem_base + (uint32_t)(sl * kSlotCols);
                uint32_t da = da_lo[sl], db = db_lo[sg];
                ptx::umma_i8_lo(d, da, db, idesc[sg], 0u);
                for (int k = 1; k < ks[sg]; ++k) {
                  da += da_step;
                  db += db_step[sg];
                  ptx::umma_i8_lo(d, da, db, idesc[sg], 1u);
                }
                ptx::umma_commit(dbar[sl]);
              }
            }
          }
        }
      } else
      for (int t0 = 0; t0 < ntv; t0 += nslots) {
        const int nt = min(nslots, ntv - t0);
        const bool last_tile = t0 + nslots >= ntv;
        for (int stage = 0; stage < nstages; ++stage) {
          for (int sl = 0; sl < nt; ++sl) {
            if (!alias) {
              const int wslot = prior ? 0 : stage;
              mma(sl, wslot, first && sl == 0, wslot == 0 ? par0 : par12, n[stage], kd[stage], au[stage]);
              dpar[sl] ^= 1u;
            } else if (stage == 1) {
              mma(sl, 1, first, par12, n[1], kd[1], au[1]);
              dpar[sl] ^= 1u;
            } else {
              // S0 holds, in turn: W1, W3 of every tile (coupling) or the prior matrix for all tiles
              const bool ww = prior ? first : true;
              mma(sl, 0, ww, W.s0_used & 1u, n[stage], kd[stage], au[stage]);
              if (ww) ++W.s0_used;
              if (prior) {
                if (last_tile && i + 1 < st.nsteps) s0_refill(step_ref(P, st, i + 1), 0);
              } else if (stage == 0) {
                s0_refill(br, 2);
              } else if (!last_tile) {
                s0_refill(br, 0);
              } else if (i + 1 < st.nsteps) {
                s0_refill(step_ref(P, st, i + 1), 0);
              }
              dpar[sl] ^= 1u;
            }
          }
        }
        first = false;
      }
    }
    __syncwarp();
    cta_barrier();     // every MMA of step i has completed (the workers waited for each accumulator)
    if (lead) top_up(cx, P, a, st, W, i, alias);
  }
  if (st.nsteps > 0 && !st.is_prior(st.nsteps - 1)) cta_barrier();   // trailing translation pass
}

// ---- control thread, streamed weights --------------------------------------------------------------
// For hidden widths above 256 no weight matrix stays resident: every tile re-reads W1, W2, W3 from
// L2 in K-slices of 32 bytes (one MMA K step: N x 32 bytes, contiguous in the packed matrix) through
// a ring of kRingDepth slots. The thread runs a producer cursor (bulk copies, up to kRingDepth
// slices ahead, across stage, tile and step boundaries) and a consumer cursor (MMAs) over the same
// fixed sequence of slices. Slice g uses ring slot g % depth; its load completes phase g / depth of
// that slot's "full" barrier, and the MMAs that read it commit to the slot's "empty" barrier.
struct SliceCursor {
  int step, tile, stage, k;
  uint32_t g;            // running slice number
};

__device__ void run_control_streamed(const Ctx& cx, const LevelPlan& P, const LevelArgs& a, const Steps& st, int ntv) {
  uint8_t* smem = cx.smem;
  Ctl* ctl = cx.ctl;
  const bool lead = cx.lane == 0;
  uint32_t apar = 0u;
  SliceCursor prod{0, 0, 0, 0, 0u};

  auto stages_of = [&](int step) { return st.is_prior(step) ? 1 : 3; };
  // advance a cursor to the next slice of the fixed sequence; false when the level is finished
  auto advance = [&](SliceCursor& c) {
    const BlockRef& br = step_ref(P, st, c.step);
    ++c.g;
    if (++c.k < (int)br.k_slices[c.stage]) return true;
    c.k = 0;
    if (++c.stage < stages_of(c.step)) return true;
    c.stage = 0;
    if (++c.tile < ntv) return true;
    c.tile = 0;
    return ++c.step < st.nsteps;
  };
  bool prod_live = st.nsteps > 0 && ntv > 0;
  // issue the loads of every slice up to `limit` slices ahead of consumer slice number g_cons
  auto produce = [&](uint32_t g_cons) {
    while (prod_live && prod.g < g_cons + (uint32_t)kRingDepth) {
      const uint32_t slot = prod.g % (uint32_t)kRingDepth, round = prod.g / (uint32_t)kRingDepth;
      if (round > 0) wait_bar(ctl, a.status, &ctl->w_empty[slot], (round - 1u) & 1u);
      const BlockRef& br = step_ref(P, st, prod.step);
      const uint32_t bytes = br.w_bytes[prod.stage] / br.k_slices[prod.stage];
      bulk_load(cx, a.blob, br.w_off[prod.stage] + (uint32_t)prod.k * bytes, bytes,
                P.s_w[0] + slot * P.ring_slot_bytes, &ctl->w_full[slot]);
      prod_live = advance(prod);
    }
  };

  if (lead) {
    for (int i = 0; i < st.nsteps && i < 2; ++i) {
      const BlockRef& br = step_ref(P, st, i);
      bulk_load(cx, a.blob, br.meta_off, br.meta_bytes, P.s_meta[i], &ctl->meta_full[i]);
    }
    produce(0u);
  }
  uint32_t g = 0u;       // consumer slice number
  for (int i = 0; i < st.nsteps; ++i) {
    const bool prior = st.is_prior(i);
    int n[3] = {0, 0, 0};
    bool au[3] = {false, false, false};
    if (lead) {
      wait_bar(ctl, a.status, &ctl->meta_full[i & 1], (uint32_t)((i >> 1) & 1));
      const uint8_t* mb = smem + P.s_meta[i & 1];
      if (prior) {
        n[0] = reinterpret_cast<const PriorMeta*>(mb)->n;
      } else {
        const CouplingMeta* M = reinterpret_cast<const CouplingMeta*>(mb);
        n[0] = M->n1; n[1] = M->n2; n[2] = M->n3;
        au[1] = M->hi1 > 127; au[2] = M->hi2 > 127;
      }
    }
    cta_barrier();     // the workers have finished the pixel pass: step i-1's meta slot is free
    if (lead) {
      if (i >= 1 && i + 1 < st.nsteps) {
        const BlockRef& br = step_ref(P, st, i + 1);
        bulk_load(cx, a.blob, br.meta_off, br.meta_bytes, P.s_meta[(i + 1) & 1], &ctl->meta_full[(i + 1) & 1]);
      }
      const BlockRef& br = step_ref(P, st, i);
      const int nstages = prior ? 1 : 3;
      const uint32_t sa = ptx::smem_u32(smem + P.s_a[0]);
      for (int t = 0; t < ntv; ++t) {
        for (int stage = 0; stage < nstages; ++stage) {
          wait_bar(ctl, a.status, &ctl->a_ready[0], apar);
          apar ^= 1u;
          ptx::tc_fence_after();
          const int nn = n[stage];
          const uint32_t lbo_b = (uint32_t)nn * 16u;
          for (int k = 0; k < (int)br.k_slices[stage]; ++k, ++g) {
            produce(g);
            const uint32_t slot = g % (uint32_t)kRingDepth;
            wait_bar(ctl, a.status, &ctl->w_full[slot], (g / (uint32_t)kRingDepth) & 1u);
            const uint32_t sb = ptx::smem_u32(smem + P.s_w[0] + slot * P.ring_slot_bytes);
            const uint64_t da = ptx::umma_desc(sa + (uint32_t)k * 2u * (kTileM * 16), kTileM * 16, 128);
            for (int n0 = 0; n0 < nn; n0 += 256) {
              const uint64_t db = ptx::umma_desc(sb + (uint32_t)n0 * 16u, lbo_b, 128);
              const uint32_t idesc = ptx::umma_idesc_i8((uint32_t)min(256, nn - n0), au[stage]);
              if (k == 0) ptx::umma_i8_first(cx.tmem_base + (uint32_t)n0, da, db, idesc);
              else ptx::umma_i8_acc(cx.tmem_base + (uint32_t)n0, da, db, idesc);
            }
            ptx::umma_commit(ptx::smem_u32(&ctl->w_empty[slot]));
          }
          ptx::umma_commit(ptx::smem_u32(&ctl->d_ready[0]));
          produce(g);   // keep the ring full while the workers requantise
        }
      }
    }
    __syncwarp();
    cta_barrier();     // every MMA of step i has completed (the workers waited for each accumulator)
  }
  if (st.nsteps > 0 && !st.is_prior(st.nsteps - 1)) cta_barrier();   // trailing translation pass
}

// ---- workers ----------------------------------------------------------------------------------
template <bool kInv>
__device__ __forceinline__ void run_workers(Ctx& cx, const LevelPlan& P, const LevelArgs& a, const Steps& st, int img0, int pvalid,
                            int ntv) {
  uint8_t* smem = cx.smem;
  Ctl* ctl = cx.ctl;
  int32_t* v = reinterpret_cast<int32_t*>(smem + P.s_v);
  int8_t* xa = reinterpret_cast<int8_t*>(smem + P.s_xa);
  int32_t* acc = reinterpret_cast<int32_t*>(smem + P.s_acc);
  uint8_t* sA = smem + P.s_a[0];          // A-operand buffer of the current tile slot
  const uint32_t* rowinfo = reinterpret_cast<const uint32_t*>(smem + P.s_rowinfo);
  const int pg = P.pg, ca = P.ca, cb = P.cb, w = P.w, cpad = P.cpad, cbp = P.cbp;
  const int2* gtab = reinterpret_cast<const int2*>(smem + P.s_gran);
  uint32_t dpar[2] = {0u, 0u};
  const int nslots = P.nslots;
  const CouplingMeta* prevM = nullptr;       // coupling whose translation is still to be applied

  auto use_slot = [&](int sl) {
    sA = smem + P.s_a[sl];
    cx.tmem_slot = cx.tmem_base + (uint32_t)(sl * kSlotCols) + ((uint32_t)(cx.wq * 32) << 16);
  };
  // this warp's part of tile slot sl's A operand is written (and its TMEM reads are done): every
  // lane fences its own writes towards the async proxy, the warp synchronises, one lane arrives
  auto arrive_a = [&](int sl) {
    ptx::tc_fence_before();
    ptx::fence_async_smem();
    __syncwarp();
    if (cx.lane == 0)
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(ptx::smem_u32(&ctl->a_ready[sl])) : "memory");
  };
  auto wait_d = [&](int sl) {
    // often already complete: test inline before the call
    {
      const uint32_t b = ptx::smem_u32(&ctl->d_ready[sl]);
      // already complete (common), or complete within one suspended try: no call; else the bounded wait
      if (!ptx::mbar_test_wait(b, dpar[sl]) && !ptx::mbar_try_wait(b, dpar[sl]))
        wait_bar(ctl, a.status, &ctl->d_ready[sl], dpar[sl]);
    }
    dpar[sl] ^= 1u;
    ptx::tc_fence_after();
  };

  // n / pvalid for the work-item maps below (n * pvalid < 2^32)
  const uint32_t mul_pv = pvalid > 1 ? (uint32_t)((0xFFFFFFFFull / (uint32_t)pvalid) + 1ull) : 0u;
  // x_b +/-= rq(acc + bias) of the previous coupling. Work item = (channel, pixel), channel-major, so
  // that levels with few pixels per CTA still use every thread and the load is even; two items at
  // a time for independent instruction chains.
  auto apply_translation_all = [&]() {
    const uint8_t* pm = reinterpret_cast<const uint8_t*>(prevM);
    const int32_t* colB = reinterpret_cast<const int32_t*>(pm + prevM->off_colB);
    const OutRq* orq = reinterpret_cast<const OutRq*>(pm + prevM->off_out);
    const int items = cb * pvalid;
    auto one = [&](int it) {
      const int c = fdiv(it, mul_pv), p = it - c * pvalid;
      const OutRq o = orq[c];
      int32_t* ap = acc + c * pg + p;
      const uint32_t t = (uint32_t)rq_out(*ap, o);
      *ap = 0;
      uint32_t* vv = reinterpret_cast<uint32_t*>(&v[colB[c] * pg + p]);
      *vv = kInv ? (*vv - t) : (*vv + t);
    };
    int it = cx.tid;
    for (; it + kWorkers < items; it += 2 * kWorkers) {
      one(it);
      one(it + kWorkers);
    }
    if (it < items) one(it);
  };
  // network input: ca channels requantised to int8, padded to cpad bytes per pixel. Work item =
  // (group of four channels, pixel).
  auto requant_input_all = [&](const int32_t* cols, int32_t m0, int32_t s) {
    const int items = (cpad >> 2) * pvalid;
    for (int it = cx.tid; it < items; it += kWorkers) {
      const int g = fdiv(it, mul_pv), p = it - g * pvalid;
      const int g0 = g << 2;
      int y[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        y[i] = 0;
        if (g0 + i < ca) y[i] = clampi(rq_exact(v[cols[g0 + i] * pg + p], m0, s), -128, 127);
      }
      *reinterpret_cast<uint32_t*>(xa + (size_t)p * cpad + g0) = pack4(y[0], y[1], y[2], y[3]);
    }
  };
  auto worker_barrier = [&]() { asm volatile("bar.sync 1, %0;" ::"n"(kWorkers) : "memory"); };

  for (int i = 0; i < st.nsteps; ++i) {
    if (!ptx::mbar_test_wait(ptx::smem_u32(&ctl->meta_full[i & 1]), (uint32_t)((i >> 1) & 1)))
      wait_bar(ctl, a.status, &ctl->meta_full[i & 1], (uint32_t)((i >> 1) & 1));
    const uint8_t* mb = smem + P.s_meta[i & 1];
    const bool prior = st.is_prior(i);
    const CouplingMeta* Mp = reinterpret_cast<const CouplingMeta*>(mb);
    const PriorMeta* Pp = reinterpret_cast<const PriorMeta*>(mb);
    {
      const int32_t* cols = prior ? P.col_out : reinterpret_cast<const int32_t*>(mb + Mp->off_colA);
      const int32_t in_m0 = prior ? Pp->in_m0 : Mp->in_m0, in_s = prior ? Pp->in_s : Mp->in_s;
      if (prevM) {
        apply_translation_all();
        worker_barrier();            // the network input may read channels that were just updated
      }
      requant_input_all(cols, in_m0, in_s);
    }
    prevM = prior ? nullptr : Mp;
    cta_barrier();
    RowPos rp[2];
    if (prior) {
      const PriorMeta M = *Pp;
      const OutRq* orq = reinterpret_cast<const OutRq*>(mb + M.off_out);
      for (int t0 = 0; t0 < ntv; t0 += nslots) {
        const int nt = min(nslots, ntv - t0);
        for (int sl = 0; sl < nt; ++sl) {
          use_slot(sl);
          rp[sl] = row_pos(rowinfo, t0 + sl, cx.row, cx.row & (cx.rrows - 1));
          build_im2col(cx, sA, xa, gtab, cpad, M.kd, rp[sl]);
          arrive_a(sl);
        }
        for (int sl = 0; sl < nt; ++sl) {
          wait_d(sl);
          use_slot(sl);
          epilogue_prior(cx, P, a, M, orq, img0, rp[sl]);
        }
      }
    } else {
      const CouplingMeta M = *Mp;
      const HiddenRq* h1 = reinterpret_cast<const HiddenRq*>(mb + M.off_h1);
      const HiddenRq* h2 = reinterpret_cast<const HiddenRq*>(mb + M.off_h2);
      const int2* u1 = reinterpret_cast<const int2*>(mb + M.off_u1);
      const int2* u2 = reinterpret_cast<const int2*>(mb + M.off_u2);
      for (int t0 = 0; t0 < ntv; t0 += nslots) {
        const int nt = min(nslots, ntv - t0);
        for (int sl = 0; sl < nt; ++sl) {                     // conv 3x3: input -> hidden 1
          use_slot(sl);
          rp[sl] = row_pos(rowinfo, t0 + sl, cx.row, cx.row & (cx.rrows - 1));
          build_im2col(cx, sA, xa, gtab, cpad, M.kd1, rp[sl]);
          arrive_a(sl);
        }
        for (int sl = 0; sl < nt; ++sl) {                     // requant, conv 1x1
          wait_d(sl);
          use_slot(sl);
          epilogue_hidden(cx, M.mode1, M.us1, M.n1, M.kd2, h1, u1, M.lo1, M.hi1, kBiasColumnsLo, kBiasColumnsHi, sA);
          arrive_a(sl);
        }
        for (int sl = 0; sl < nt; ++sl) {                     // requant, conv 3x3 as per-tap partials
          wait_d(sl);
          use_slot(sl);
          epilogue_hidden(cx, M.mode2, M.us2, M.n2, M.kd3, h2, u2, M.lo2, M.hi2, 0u, 0u, sA);
          arrive_a(sl);
        }
        for (int sl = 0; sl < nt; ++sl) {                     // shifted sum into the accumulator
          wait_d(sl);
          use_slot(sl);
          epilogue_scatter(cx, cb, cbp, acc, pg, w, rp[sl]);
        }
      }
    }
    ptx::tc_fence_before();
    cta_barrier();
  }
  if (prevM) {
    apply_translation_all();
    cta_barrier();
  }
}

template <bool kInv>
__global__ void __launch_bounds__(kThreads, 1) level_kernel(const LevelArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ Ctl ctl;
  const LevelPlan& P = *a.plan;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  ptx::grid_launch_dependents();         // the next kernel in the stream may start its prologue
  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(ptx::smem_u32(&ctl.a_ready[s]), (uint32_t)kWorkerWarps);
      ptx::mbar_init(ptx::smem_u32(&ctl.d_ready[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl.meta_full[s]), 1);
    }
    for (int s = 0; s < 3; ++s) {
      ptx::mbar_init(ptx::smem_u32(&ctl.w_full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl.w_empty[s]), 1);
    }
    ptx::mbar_init_fence();
    ctl.abort = 0;
  }
  if (warp == 0) ptx::tmem_alloc(ptx::smem_u32(&ctl.tmem_base), (uint32_t)P.tmem_cols);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = ctl.tmem_base;

  const int c = P.c, px = P.px, pg = P.pg, w = P.w;
  const int img0 = blockIdx.x * P.group;
  const int nimg = min(P.group, a.batch - img0);
  const int pvalid = nimg * px;
  const int ntv = (pvalid + kTileM - 1) / kTileM;
  const int per_img = c * px;                    // elements per image at this level
  int32_t* v = reinterpret_cast<int32_t*>(smem + P.s_v);

  Steps st;
  st.n_couplings = (kInv && a.phase == 1) ? 0 : P.n_couplings;
  st.do_prior = P.has_prior && a.prior != nullptr && !(kInv && a.phase == 2);
  st.nsteps = st.n_couplings + (st.do_prior ? 1 : 0);
  st.inverse = kInv;

  Ctx cx;
  cx.smem = smem;
  cx.ctl = &ctl;
  cx.status = a.status;
  cx.tid = tid;
  cx.warp = warp;
  cx.lane = lane;
  cx.wq = warp & 3;
  cx.rep = P.rep;
  cx.rrows = kTileM / P.rep;
  cx.bcs = warp >> 2;
  cx.bncs = kWorkerWarps >> 2;
  cx.cs = ((cx.wq * P.rep) >> 2) * cx.bncs + cx.bcs;     // replica index * 4 + split within the quarter
  cx.ncs = cx.bncs * P.rep;
  cx.row = cx.wq * 32 + lane;
  cx.tmem_base = tmem;
  cx.tmem_slot = tmem + ((uint32_t)(cx.wq * 32) << 16);

  if (warp >= kWorkerWarps) {
    // The packed blocks are written once at model creation, so the first copies need not wait for
    // the previous kernel; run_control starts them before it joins the workers' first barrier.
    if (P.streamed) {
      cta_barrier();                     // the workers have loaded the flow variable
      run_control_streamed(cx, P, a, st, ntv);
    } else {
      run_control(cx, P, a, st, ntv);
    }
  } else {
    int32_t* acc = reinterpret_cast<int32_t*>(smem + P.s_acc);
    for (int idx = tid; idx < P.cb * pg; idx += kWorkers) acc[idx] = 0;
    uint32_t* rowinfo = reinterpret_cast<uint32_t*>(smem + P.s_rowinfo);
    for (int idx = tid; idx < P.tiles * kTileM; idx += kWorkers) rowinfo[idx] = row_record(P.rep > 1 ? (idx & (kTileM / P.rep - 1)) : idx, pvalid, px, P.h, w, P.mul_px, P.mul_w);
    int32_t* gran = reinterpret_cast<int32_t*>(smem + P.s_gran);
    for (int idx = tid; idx < 2 * P.n_gran; idx += kWorkers) gran[idx] = P.gran_tab[idx];
    // Everything above used only the plan; from here on the kernel reads what the previous kernel
    // in the stream wrote and writes what it may still be reading.
    ptx::grid_dependency_wait();
    if (!kInv) {
      // space-to-depth on load: plane c*4 + dy*2 + dx, pixel (i, j) <- in[c][2i+dy][2j+dx]
      const int w2 = 2 * w;
#pragma unroll 4
      for (int e = tid; e < nimg * per_img; e += kWorkers) {
        const int g = fdiv(e, P.mul_per_img), r = e - g * per_img;
        const int ci = fdiv(r, P.mul_4px), r2 = r - ci * 4 * px;
        const int y = fdiv(r2, P.mul_w2), x = r2 - y * w2;
        size_t src = (size_t)(img0 + g) * per_img + r;
        if (P.is_first && a.img_w > 0) {                 // patch (by, bx) of one large image
          const int by = fdiv(img0 + g, a.mul_patches_x), bx = img0 + g - by * a.patches_x;
          src = ((size_t)ci * a.img_h + (size_t)(by * 2 * P.h + y)) * a.img_w + (size_t)(bx * w2 + x);
        }
        const int32_t val = P.is_first ? (int32_t) reinterpret_cast<const uint8_t*>(a.in)[src]
                                       : reinterpret_cast<const int32_t*>(a.in)[src];
        v[(ci * 4 + (y & 1) * 2 + (x & 1)) * pg + g * px + (y >> 1) * w + (x >> 1)] = val;
      }
    } else {
      // merge: logical channel k < keep_c from the deeper level, the rest from z's block of this level
#pragma unroll 4
      for (int e = tid; e < nimg * per_img; e += kWorkers) {
        const int g = fdiv(e, P.mul_per_img), r = e - g * per_img;
        const int k = fdiv(r, P.mul_px), q = r - k * px;
        const size_t b = (size_t)(img0 + g);
        if (a.phase == 1 && k >= P.keep_c) continue;     // prior head only: z's block is not read
        const int32_t val =
            (k < P.keep_c) ? reinterpret_cast<const int32_t*>(a.in)[b * (size_t)a.in_stride + (size_t)k * px + q]
                           : a.z[b * P.d + P.z_off + (size_t)(k - P.keep_c) * px + q];
        v[P.col_out[k] * pg + g * px + q] = val;
      }
    }
    cta_barrier();

    run_workers<kInv>(cx, P, a, st, img0, pvalid, ntv);

    if (!kInv) {
      // split on store: factored-out half -> z block of this level; kept half -> next level (or
      // the final z block)
      int32_t* keep_out = reinterpret_cast<int32_t*>(a.out);
#pragma unroll 4
      for (int e = tid; e < nimg * per_img; e += kWorkers) {
        const int g = fdiv(e, P.mul_per_img), r = e - g * per_img;
        const int k = fdiv(r, P.mul_px), q = r - k * px;
        const size_t b = (size_t)(img0 + g);
        const int32_t val = v[P.col_out[k] * pg + g * px + q];
        if (k >= P.keep_c) a.z[b * P.d + P.z_off + (size_t)(k - P.keep_c) * px + q] = val;
        else if (P.is_last) a.z[b * P.d + P.z_final_off + (size_t)k * px + q] = val;
        else keep_out[(b * P.keep_c + k) * (size_t)px + q] = val;
      }
    } else if (a.phase != 1) {
      // depth-to-space on store
      const int w2 = 2 * w;
      uint32_t bad = 0;
#pragma unroll 4
      for (int e = tid; e < nimg * per_img; e += kWorkers) {
        const int g = fdiv(e, P.mul_per_img), r = e - g * per_img;
        const int ci = fdiv(r, P.mul_4px), r2 = r - ci * 4 * px;
        const int y = fdiv(r2, P.mul_w2), x = r2 - y * w2;
        const int32_t val = v[(ci * 4 + (y & 1) * 2 + (x & 1)) * pg + g * px + (y >> 1) * w + (x >> 1)];
        size_t dst = (size_t)(img0 + g) * per_img + r;
        if (P.is_first && a.img_w > 0) {
          const int by = fdiv(img0 + g, a.mul_patches_x), bx = img0 + g - by * a.patches_x;
          dst = ((size_t)ci * a.img_h + (size_t)(by * 2 * P.h + y)) * a.img_w + (size_t)(bx * w2 + x);
        }
        if (P.is_first) {
          reinterpret_cast<uint8_t*>(a.out)[dst] = (uint8_t)((uint32_t)val & 0xFFu);
          bad += (val < 0 || val > 255) ? 1u : 0u;
        } else {
          reinterpret_cast<int32_t*>(a.out)[dst] = val;
        }
      }
      if (P.is_first && a.oor != nullptr) {
        bad = __reduce_add_sync(0xFFFFFFFFu, bad);
        if (lane == 0 && bad) atomicAdd(a.oor, bad);
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 0) ptx::tmem_dealloc(tmem, (uint32_t)P.tmem_cols);
}

}  // namespace

cudaError_t launch_level(const LevelArgs& args, bool inverse, int grid, uint32_t smem_bytes, cudaStream_t stream) {
  // Programmatic dependent launch: the CTAs of this level may start (barrier set-up, TMEM
  // allocation, index records) while the previous kernel in the stream drains; the kernel itself
  // waits for that kernel's completion before it touches anything a kernel writes.
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)kThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (inverse) return cudaLaunchKernelEx(&cfg, level_kernel<true>, args);
  return cudaLaunchKernelEx(&cfg, level_kernel<false>, args);
}

cudaError_t configure_level_kernels(uint32_t max_smem_bytes) {
  cudaError_t e = cudaFuncSetAttribute(level_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)max_smem_bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(level_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem_bytes);
}

}  // namespace iodf
