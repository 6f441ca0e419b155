// Device code shared by the flow-level kernels (level_kernel.cu: every level shape; level_pipe.cu:
// the stage-pipelined kernel for levels of several tiles): requantisation, im2col, the epilogues,
// step bookkeeping, MMA issue and weight copies, and the index maps of a level's load and store.
#pragma once
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
// All are exact: for s >= 1, floor(x / 2^(31+s)) = floor(floor(x / 2^32) / 2^(s-1)).
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
  const int2* __restrict__ mb;         // kModeUniform: {m0, bias}; kModeFolded: int32 m0 per channel
  int lo, hi, sh;
  long long rnd64;                     // 2^(30+s) (kModeFolded, kModeUniform)

  __device__ __forceinline__ int one(int acc, int ch) const {
    const HiddenRq r = rq[ch];
    const long long c64 = (long long)(((unsigned long long)r.c_hi << 32) | (unsigned long long)r.c_lo);
    const long long p = (long long)acc * (long long)r.m0 + c64;
    const int y = kMode == kModeFast ? (((int)(p >> 32)) >> r.sh) : (int)(p >> (32 + r.sh));
    return kClip != kClipAny ? y : clampi(y, lo, hi);        // otherwise clipped while packing
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
  // four accumulator columns starting at channel ch0 (a multiple of 4) -> four bytes of the next A operand
  __device__ __forceinline__ uint32_t quad(const uint32_t* r, int ch0) const {
    if (kMode >= kModeFolded) {
      const int4 c = *reinterpret_cast<const int4*>(reinterpret_cast<const int32_t*>(mb) + ch0);
      return pack_clipped(uniform_one((int)r[0], c.x, 0), uniform_one((int)r[1], c.y, 0),
                          uniform_one((int)r[2], c.z, 0), uniform_one((int)r[3], c.w, 0));
    } else if (kMode == kModeUniform) {
      const int4* q = reinterpret_cast<const int4*>(mb + ch0);     // {m0, bias} pairs, 16-byte aligned
      const int4 c01 = q[0], c23 = q[1];
      return pack_clipped(uniform_one((int)r[0], c01.x, c01.y), uniform_one((int)r[1], c01.z, c01.w),
                          uniform_one((int)r[2], c23.x, c23.y), uniform_one((int)r[3], c23.z, c23.w));
    }
    return pack_clipped(one((int)r[0], ch0), one((int)r[1], ch0 + 1), one((int)r[2], ch0 + 2), one((int)r[3], ch0 + 3));
  }
  // 16 accumulator columns starting at channel ch0 -> one 16-byte chunk of the next A operand
  __device__ __forceinline__ uint4 chunk(const uint32_t* r, int ch0) const {
    return make_uint4(quad(r, ch0), quad(r + 4, ch0 + 4), quad(r + 8, ch0 + 8), quad(r + 12, ch0 + 12));
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

// mode: layer flavour (see above); us: the layer's uniform shift (kModeFolded, kModeUniform).
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

// ---- im2col without the granule table ---------------------------------------------------------------
// im2col of this thread's tile row by taps: split `cs` of `ncs` (a power of two) takes the taps t
// with t % ncs == cs, one predicated load per 8-byte granule straight from the pixel-major network
// input (the tap's bit of the row's gather mask says whether its source pixel is inside the image),
// and one split also writes what follows the nine taps: the eight bias columns and zeros up to kd.
// kCpad = bytes per pixel of the network input (C/2 rounded up to 8). The bytes are those of
// build_im2col; only the way to them differs.
template <int kCpad>
__device__ __forceinline__ void build_im2col_taps(uint8_t* __restrict__ a_row, const int8_t* __restrict__ xa, int w,
                                                   int kd, const RowPos rp, int cs, int ncs) {
  constexpr int kG = kCpad / 8;          // granules per tap
  const int8_t* base = xa + (size_t)rp.p * kCpad;
  auto at = [&](int g) { return a_row + (size_t)(g >> 1) * (kTileM * 16) + (g & 1) * 8; };
#pragma unroll
  for (int t = 0; t < 9; ++t) {
    if ((t & (ncs - 1)) != cs) continue;
    const int8_t* src = base + (((t / 3) - 1) * w + (t % 3) - 1) * kCpad;
    const bool ok = ((rp.gmask >> t) & 1u) != 0;
    if (kG % 2 == 0) {                   // whole 16-byte chunks
#pragma unroll
      for (int gi = 0; gi < kG; gi += 2) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (ok) v = *reinterpret_cast<const uint4*>(src + gi * 8);
        *reinterpret_cast<uint4*>(at(t * kG + gi)) = v;
      }
    } else {
#pragma unroll
      for (int gi = 0; gi < kG; ++gi) {
        uint2 v = make_uint2(0u, 0u);
        if (ok) v = *reinterpret_cast<const uint2*>(src + gi * 8);
        *reinterpret_cast<uint2*>(at(t * kG + gi)) = v;
      }
    }
  }
  if (cs == (9 & (ncs - 1))) {
    const int ng = kd >> 3;
    if (9 * kG < ng) *reinterpret_cast<uint2*>(at(9 * kG)) = make_uint2(kBiasColumnsLo, kBiasColumnsHi);
    for (int g = 9 * kG + 1; g < ng; ++g) *reinterpret_cast<uint2*>(at(g)) = make_uint2(0u, 0u);
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


// ---- pixel pass: work of all worker threads between two couplings ---------------------------------
struct PixelPass {
  int32_t* v;            // flow variable, planar [column][pg]
  int32_t* acc;          // translation accumulator, planar [cb][pg]
  int8_t* xa;            // network input, pixel-major [pg][cpad]
  int pg, ca, cb, cpad, pvalid;
  uint32_t mul_pv;       // magic multiplier of pvalid (0: pvalid = 1)
  int tid, nthreads;     // this thread among the threads that share the pass
  // pvalid and pg multiples of four: four pixels of a plane per 16-byte access
  __device__ __forceinline__ bool by_four() const { return ((pvalid | pg) & 3) == 0; }
  __device__ __forceinline__ uint32_t mul_pv4() const {
    return pvalid > 4 ? (uint32_t)((0xFFFFFFFFull / (uint32_t)(pvalid >> 2)) + 1ull) : 0u;
  }
};

// x_b +/-= rq(acc + bias) of the coupling whose meta block is M. Work item = (channel, pixel),
// channel-major, so that levels with few pixels per CTA still use every thread and the load is even;
// two items at a time for independent instruction chains.
template <bool kInv>
__device__ __forceinline__ void apply_translation(const PixelPass& pp, const CouplingMeta* M) {
  const uint8_t* pm = reinterpret_cast<const uint8_t*>(M);
  const int32_t* colB = reinterpret_cast<const int32_t*>(pm + M->off_colB);
  const OutRq* orq = reinterpret_cast<const OutRq*>(pm + M->off_out);
  if (pp.by_four()) {
    // work item = (channel, four neighbouring pixels): one 16-byte load and store per plane
    const int q = pp.pvalid >> 2, items4 = pp.cb * q;
    const uint32_t mul = pp.mul_pv4();
    for (int it = pp.tid; it < items4; it += pp.nthreads) {
      const int c = fdiv(it, mul), p = (it - c * q) << 2;
      const OutRq o = orq[c];
      int4* ap = reinterpret_cast<int4*>(pp.acc + c * pp.pg + p);
      uint4* vp = reinterpret_cast<uint4*>(&pp.v[colB[c] * pp.pg + p]);
      const int4 t = *ap;
      uint4 x = *vp;
      *ap = make_int4(0, 0, 0, 0);
      const uint32_t t0 = (uint32_t)rq_out(t.x, o), t1 = (uint32_t)rq_out(t.y, o);
      const uint32_t t2 = (uint32_t)rq_out(t.z, o), t3 = (uint32_t)rq_out(t.w, o);
      x.x = kInv ? x.x - t0 : x.x + t0;
      x.y = kInv ? x.y - t1 : x.y + t1;
      x.z = kInv ? x.z - t2 : x.z + t2;
      x.w = kInv ? x.w - t3 : x.w + t3;
      *vp = x;
    }
    return;
  }
  const int items = pp.cb * pp.pvalid;
  auto one = [&](int it) {
    const int c = fdiv(it, pp.mul_pv), p = it - c * pp.pvalid;
    const OutRq o = orq[c];
    int32_t* ap = pp.acc + c * pp.pg + p;
    const uint32_t t = (uint32_t)rq_out(*ap, o);
    *ap = 0;
    uint32_t* vv = reinterpret_cast<uint32_t*>(&pp.v[colB[c] * pp.pg + p]);
    *vv = kInv ? (*vv - t) : (*vv + t);
  };
  int it = pp.tid;
  for (; it + pp.nthreads < items; it += 2 * pp.nthreads) {
    one(it);
    one(it + pp.nthreads);
  }
  if (it < items) one(it);
}

// network input: ca channels requantised to int8, padded to cpad bytes per pixel. Work item =
// (group of four channels, pixel).
__device__ __forceinline__ void requant_input(const PixelPass& pp, const int32_t* cols, int32_t m0, int32_t s) {
  const int items = (pp.cpad >> 2) * pp.pvalid;
  for (int it = pp.tid; it < items; it += pp.nthreads) {
    const int g = fdiv(it, pp.mul_pv), p = it - g * pp.pvalid;
    const int g0 = g << 2;
    int y[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      y[i] = 0;
      if (g0 + i < pp.ca) y[i] = rq_exact(pp.v[cols[g0 + i] * pp.pg + p], m0, s);
    }
    // the clip to -128..127 is the pack's saturation
    *reinterpret_cast<uint32_t*>(pp.xa + (size_t)p * pp.cpad + g0) = pack4_sat(y[0], y[1], y[2], y[3]);
  }
}

// ---- a level's input and output index maps ---------------------------------------------------------
// Planes of at least this many bytes leave through bulk copies; smaller ones (the deep levels: 16 or 64
// pixels per image) are cheaper to store with the threads than to issue one copy each for.
constexpr int kBulkStoreMinBytes = 1024;

// Encode: space-to-depth on load (first level: uint8 images, or the patch grid of one image).
// Decode: merge of the channels that come back from the deeper level with this level's block of z.
template <bool kInv>
__device__ __forceinline__ void level_load(const LevelPlan& P, const LevelArgs& a, int32_t* v, int img0, int nimg, int tid,
                                           int nthreads) {
  const int c = P.c, px = P.px, pg = P.pg, w = P.w;
  const int per_img = c * px;
  if (!kInv) {
    // space-to-depth on load: plane c*4 + dy*2 + dx, pixel (i, j) <- in[c][2i+dy][2j+dx]
    const int w2 = 2 * w;
    if ((w & 1) == 0 && (a.img_w & 3) == 0) {
      // Four neighbours of an input row per thread and step: one 4-byte (uint8 images) or 16-byte
      // (int32 channels) load, and two 8-byte stores, one into the dx = 0 plane and one into the
      // dx = 1 plane. Every index below is a multiple of four, so the accesses are aligned.
#pragma unroll 2
      for (int e = 4 * tid; e < nimg * per_img; e += 4 * nthreads) {
        const int g = fdiv(e, P.mul_per_img), r = e - g * per_img;
        const int ci = fdiv(r, P.mul_4px), r2 = r - ci * 4 * px;
        const int y = fdiv(r2, P.mul_w2), x = r2 - y * w2;
        size_t src = (size_t)(img0 + g) * per_img + r;
        if (P.is_first && a.img_w > 0) {                 // patch (by, bx) of one large image
          const int by = fdiv(img0 + g, a.mul_patches_x), bx = img0 + g - by * a.patches_x;
          src = ((size_t)ci * a.img_h + (size_t)(by * 2 * P.h + y)) * a.img_w + (size_t)(bx * w2 + x);
        }
        int4 q;
        if (P.is_first) {
          const uint32_t b4 = *reinterpret_cast<const uint32_t*>(reinterpret_cast<const uint8_t*>(a.in) + src);
          q = make_int4((int)(b4 & 0xFFu), (int)((b4 >> 8) & 0xFFu), (int)((b4 >> 16) & 0xFFu), (int)(b4 >> 24));
        } else {
          q = *reinterpret_cast<const int4*>(reinterpret_cast<const int32_t*>(a.in) + src);
        }
        int32_t* d0 = v + (ci * 4 + (y & 1) * 2) * pg + g * px + (y >> 1) * w + (x >> 1);
        *reinterpret_cast<int2*>(d0) = make_int2(q.x, q.z);
        *reinterpret_cast<int2*>(d0 + pg) = make_int2(q.y, q.w);
      }
    } else
#pragma unroll 4
    for (int e = tid; e < nimg * per_img; e += nthreads) {
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
    for (int e = tid; e < nimg * per_img; e += nthreads) {
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
}

// Encode: split on store. Decode: depth-to-space on store (first level: uint8 with the out-of-range count).
template <bool kInv>
__device__ __forceinline__ void level_store(const LevelPlan& P, const LevelArgs& a, const int32_t* v, int img0, int nimg,
                                            int tid, int lane, int nthreads) {
  const int c = P.c, px = P.px, pg = P.pg, w = P.w;
  const int per_img = c * px;
  if (!kInv) {
    // split on store: factored-out half -> z block of this level; kept half -> next level (or
    // the final z block)
    int32_t* keep_out = reinterpret_cast<int32_t*>(a.out);
    if (px * 4 >= kBulkStoreMinBytes && (px & 3) == 0) {    // (16-byte granularity of the copies)
      // A channel plane of an image is px contiguous words both in shared memory and in every
      // destination layout: one bulk copy shared -> global per plane, issued by as many threads as
      // there are planes, instead of a pass of the threads over the elements. The planes were
      // written through the generic proxy: every thread fences its writes towards the async proxy
      // first, and the issuing threads wait until their copies have read shared memory.
      ptx::fence_async_smem();
      asm volatile("bar.sync 2, %0;" ::"r"(nthreads) : "memory");
      for (int pl = tid; pl < nimg * c; pl += nthreads) {
        const int g = pl / c, k = pl - g * c;
        const size_t b = (size_t)(img0 + g);
        int32_t* dst = k >= P.keep_c ? a.z + b * P.d + P.z_off + (size_t)(k - P.keep_c) * px
                       : (P.is_last ? a.z + b * P.d + P.z_final_off + (size_t)k * px
                                    : keep_out + (b * P.keep_c + k) * (size_t)px);
        ptx::bulk_s2g(dst, ptx::smem_u32(v + P.col_out[k] * pg + g * px), (uint32_t)px * 4u);
      }
      ptx::bulk_s2g_commit_and_wait_read();
      return;
    }
#pragma unroll 4
    for (int e = tid; e < nimg * per_img; e += nthreads) {
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
    for (int e = tid; e < nimg * per_img; e += nthreads) {
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
                       bool alias, uint64_t* w_full) {
  for (int s = alias ? 1 : 0; s < (alias ? 2 : 3); ++s) {
    if (W.cur_step[s] > done) continue;
    int j = W.cur_step[s] + 1;
    while (j < st.nsteps && !slot_used_by(st, s, j)) ++j;
    if (j >= st.nsteps) { W.cur_step[s] = st.nsteps; continue; }
    const BlockRef& br = step_ref(P, st, j);
    bulk_load(cx, a.blob, br.w_off[s], br.w_bytes[s], P.s_w[s], &w_full[s]);
    W.cur_step[s] = j;
  }
}

}  // namespace

}  // namespace iodf
