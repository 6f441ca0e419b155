// One flow level of the integer-only discrete flow on sm_100a, one CTA per group of images.
//
// The CTA keeps the level's flow variable v (int32, planar [channel][pixel]) in shared memory for
// all couplings of the level, so global memory is touched only for the level's input, its outputs
// and the packed weights (which stay in L2). Per coupling (Eq. 2, Sec. 3):
//
//   x_a -> int8 (input requant)                                     all threads, exact 64-bit rq
//   per 128-pixel tile:
//     A1 = im2col(x_a)            [128 x 9*ca]                      threads -> shared memory
//     D1 = A1 * W1^T              tcgen05.mma kind::i8, int32 in TMEM
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
#include "iodf_dev.h"
#include "level_kernel.h"
#include "ptx.cuh"

namespace iodf {

namespace {

struct __align__(16) Ctl {
  uint64_t bar_meta;
  uint64_t bar_w[3];
  uint64_t bar_mma;
  uint32_t tmem_base;
  uint32_t abort;
};

struct Ctx {
  uint8_t* smem;
  Ctl* ctl;
  uint32_t* status;
  int tid, warp, lane, wq, wh, row;
  uint32_t tmem;       // TMEM base address (lane 0, first allocated column)
  uint32_t tmem_row;   // the same with this warp's lane quarter in the lane field
};

// Bounded wait on an mbarrier phase. After one wait in the CTA has given up, every later wait
// returns at once, so a stuck CTA drains in bounded time, frees its TMEM and exits.
__device__ __noinline__ bool wait_bar(const Ctx& cx, uint64_t* bar, uint32_t parity) {
  volatile uint32_t* ab = &cx.ctl->abort;
  if (*ab) return false;
  const uint32_t b = ptx::smem_u32(bar);
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (ptx::mbar_try_wait(b, parity)) return true;
    if ((it & 255u) == 255u && *ab) return false;
  }
  *ab = 1;
  atomicExch(cx.status, 1u);
  return false;
}

__device__ __forceinline__ int32_t rq_exact(int32_t a, int32_t m0, int32_t s) {
  const long long p = (long long)a * (long long)m0 + (1ll << (30 + s));
  return (int32_t)(p >> (31 + s));
}

__device__ __forceinline__ int clampi(int v, int lo, int hi) { return min(max(v, lo), hi); }

template <bool kFast>
__device__ __forceinline__ int rq_hidden(int acc, const HiddenRq r, int lo, int hi) {
  const long long c64 = (long long)(((unsigned long long)r.c_hi << 32) | (unsigned long long)r.c_lo);
  const long long p = (long long)acc * (long long)r.m0 + c64;
  int y;
  if (kFast) y = ((int)(p >> 32)) >> r.sh;
  else y = (int)(p >> (32 + r.sh));
  return clampi(y, lo, hi);
}

// Pixel bookkeeping of one tile row.
struct RowPos {
  int p;            // pixel slot in the CTA (group-local)
  bool valid;
  uint32_t gmask;   // bit t=(u*3+v): input pixel (i+u-1, j+v-1) is inside the image   (gather)
  uint32_t smask;   // bit t: output pixel (i-u+1, j-v+1) is inside the image           (scatter)
};

__device__ __forceinline__ RowPos row_pos(int tile, int row, int pvalid, int px, int h, int w) {
  RowPos r;
  r.p = tile * kTileM + row;
  r.valid = r.p < pvalid;
  r.gmask = 0;
  r.smask = 0;
  if (r.valid) {
    const int q = r.p % px;
    const int i = q / w, j = q - i * w;
#pragma unroll
    for (int u = 0; u < 3; ++u)
#pragma unroll
      for (int v = 0; v < 3; ++v) {
        const bool gi = (i + u - 1 >= 0) && (i + u - 1 < h) && (j + v - 1 >= 0) && (j + v - 1 < w);
        const bool si = (i - u + 1 >= 0) && (i - u + 1 < h) && (j - v + 1 >= 0) && (j - v + 1 < w);
        r.gmask |= (gi ? 1u : 0u) << (u * 3 + v);
        r.smask |= (si ? 1u : 0u) << (u * 3 + v);
      }
  }
  return r;
}

// A[row][tap*ca + c] = xa[c][p + tap offset] (0 outside the image or beyond 9*ca), written as
// 16-byte chunks into the MMA operand layout [K/16][128][16].
__device__ void build_im2col(const Ctx& cx, uint8_t* sA, const int8_t* xa, int ca, int pg, int w, int kd,
                             const RowPos rp) {
  const int nchunks = kd >> 4;
  for (int jc = cx.wh; jc < nchunks; jc += kThreads / kTileM) {
    int k = jc << 4;
    int tap = k / ca;
    int c = k - tap * ca;
    uint32_t wd[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int b = 0; b < 16; ++b) {
      int val = 0;
      if (tap < 9 && ((rp.gmask >> tap) & 1u)) {
        const int du = tap / 3 - 1, dv = tap - (tap / 3) * 3 - 1;
        val = xa[c * pg + rp.p + du * w + dv];
      }
      wd[b >> 2] |= (uint32_t)(val & 0xFF) << (8 * (b & 3));
      if (++c == ca) { c = 0; ++tap; }
    }
    *reinterpret_cast<uint4*>(sA + (size_t)jc * (kTileM * 16) + cx.row * 16) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
  }
}

// D[128 x n] (+)= A[128 x kd] * B[n x kd]^T for B rows n0..n0+n of a matrix with n_total rows.
__device__ void issue_gemm(uint32_t d_tmem, uint32_t sa, uint32_t sb, int n_total, int n0, int n, int kd) {
  const uint32_t idesc = ptx::umma_idesc_s8((uint32_t)n);
  const uint32_t lbo_b = (uint32_t)n_total * 16u;
  for (int k = 0; k < (kd >> 5); ++k) {
    const uint64_t da = ptx::umma_desc(sa + (uint32_t)k * 2u * (kTileM * 16), kTileM * 16, 128);
    const uint64_t db = ptx::umma_desc(sb + (uint32_t)n0 * 16u + (uint32_t)k * 2u * lbo_b, lbo_b, 128);
    ptx::umma_i8(d_tmem, da, db, idesc, k > 0 ? 1u : 0u);
  }
}

// TMEM accumulator -> requantised int8 activations in the next GEMM's A layout.
template <bool kFast>
__device__ void epilogue_hidden(const Ctx& cx, uint32_t taddr, int n, int kd, const HiddenRq* rq, int lo, int hi,
                                uint8_t* sOut) {
  const int nblk = (n + 31) >> 5;
  for (int b = cx.wh; b < nblk; b += kThreads / kTileM) {
    const int c0 = b << 5;
    uint32_t r[32];
    if (n - c0 >= 32) {
      ptx::tmem_ld32(taddr + (uint32_t)c0, r);
    } else {
      uint32_t t[16];
      ptx::tmem_ld16(taddr + (uint32_t)c0, t);
#pragma unroll
      for (int i = 0; i < 16; ++i) { r[i] = t[i]; r[16 + i] = 0u; }
    }
    ptx::tmem_ld_wait();
    uint32_t wd[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) wd[i] = 0u;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      int y = 0;
      if (c0 + i < n) y = rq_hidden<kFast>((int)r[i], rq[c0 + i], lo, hi);
      wd[i >> 2] |= (uint32_t)(y & 0xFF) << (8 * (i & 3));
    }
    uint8_t* dst = sOut + (size_t)(2 * b) * (kTileM * 16) + cx.row * 16;
    *reinterpret_cast<uint4*>(dst) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
    if (c0 + 16 < kd) *reinterpret_cast<uint4*>(dst + kTileM * 16) = make_uint4(wd[4], wd[5], wd[6], wd[7]);
  }
}

// Per-tap partial products -> shifted sum into the translation accumulator.
__device__ void epilogue_scatter(const Ctx& cx, uint32_t taddr, int n3, int cb, int32_t* acc, int pg, int w,
                                 const RowPos rp) {
  const int nblk = n3 >> 4;
  for (int b = cx.wh; b < nblk; b += kThreads / kTileM) {
    uint32_t r[16];
    ptx::tmem_ld16(taddr + (uint32_t)(b << 4), r);
    ptx::tmem_ld_wait();
    if (rp.valid) {
      int col = b << 4;
      int tap = col / cb;
      int c = col - tap * cb;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        if (tap < 9 && ((rp.smask >> tap) & 1u)) {
          const int du = tap / 3 - 1, dv = tap - (tap / 3) * 3 - 1;
          atomicAdd(&acc[c * pg + rp.p - du * w - dv], (int32_t)r[i]);
        }
        if (++c == cb) { c = 0; ++tap; }
      }
    }
  }
}

struct WeightState {   // thread 0 only
  uint32_t ph[3];
};

__device__ __forceinline__ void load_part(const Ctx& cx, const uint8_t* blob, uint32_t off, uint32_t bytes,
                                          uint32_t s_dst, uint64_t* bar) {
  const uint32_t b = ptx::smem_u32(bar);
  ptx::mbar_expect_tx(b, bytes);
  ptx::bulk_g2s(ptx::smem_u32(cx.smem + s_dst), blob + off, bytes, b);
}

// One additive coupling over all tiles of the CTA. sign = +1 encodes, -1 decodes.
template <bool kInv>
__device__ void run_coupling(const Ctx& cx, const LevelPlan& P, const LevelArgs& a, const BlockRef& br, int pvalid,
                             uint32_t& ph_meta, uint32_t& ph_mma, WeightState& ws) {
  uint8_t* smem = cx.smem;
  int32_t* v = reinterpret_cast<int32_t*>(smem + P.s_v);
  int8_t* xa = reinterpret_cast<int8_t*>(smem + P.s_xa);
  int32_t* acc = reinterpret_cast<int32_t*>(smem + P.s_acc);
  uint8_t* sA13 = smem + P.s_a13;
  uint8_t* sA2 = smem + P.s_a2;
  const int pg = P.pg, ca = P.ca, cb = P.cb, w = P.w, h = P.h, px = P.px;
  const bool alias = P.w13_alias != 0;

  if (cx.tid == 0) {
    load_part(cx, a.blob, br.meta_off, br.meta_bytes, P.s_meta, &cx.ctl->bar_meta);
    load_part(cx, a.blob, br.w_off[0], br.w_bytes[0], P.s_w[0], &cx.ctl->bar_w[0]);
    load_part(cx, a.blob, br.w_off[1], br.w_bytes[1], P.s_w[1], &cx.ctl->bar_w[1]);
    if (!alias) load_part(cx, a.blob, br.w_off[2], br.w_bytes[2], P.s_w[2], &cx.ctl->bar_w[2]);
  }
  wait_bar(cx, &cx.ctl->bar_meta, ph_meta);
  ph_meta ^= 1u;
  const uint8_t* mb = smem + P.s_meta;
  const CouplingMeta M = *reinterpret_cast<const CouplingMeta*>(mb);
  const int32_t* colA = reinterpret_cast<const int32_t*>(mb + M.off_colA);
  const int32_t* colB = reinterpret_cast<const int32_t*>(mb + M.off_colB);
  const OutRq* orq = reinterpret_cast<const OutRq*>(mb + M.off_out);
  const HiddenRq* h1 = reinterpret_cast<const HiddenRq*>(mb + M.off_h1);
  const HiddenRq* h2 = reinterpret_cast<const HiddenRq*>(mb + M.off_h2);

  // network input: x_a requantised to int8
  for (int idx = cx.tid; idx < ca * pg; idx += kThreads) {
    const int c = idx / pg, p = idx - c * pg;
    int y = 0;
    if (p < pvalid) y = clampi(rq_exact(v[colA[c] * pg + p], M.in_m0, M.in_s), -128, 127);
    xa[idx] = (int8_t)y;
  }
  __syncthreads();

  bool w_ready[3] = {false, false, false};
  for (int tile = 0; tile < P.tiles; ++tile) {
    if (tile * kTileM >= pvalid) break;
    const RowPos rp = row_pos(tile, cx.row, pvalid, px, h, w);

    // conv 3x3: ca -> n1
    build_im2col(cx, sA13, xa, ca, pg, w, M.kd1, rp);
    ptx::fence_async_smem();
    __syncthreads();
    if (cx.tid == 0) {
      if (!w_ready[0] || alias) { wait_bar(cx, &cx.ctl->bar_w[0], ws.ph[0]); ws.ph[0] ^= 1u; w_ready[0] = true; }
      ptx::tc_fence_after();
      issue_gemm(cx.tmem, ptx::smem_u32(sA13), ptx::smem_u32(smem + P.s_w[0]), M.n1, 0, M.n1, M.kd1);
      ptx::umma_commit(ptx::smem_u32(&cx.ctl->bar_mma));
    }
    wait_bar(cx, &cx.ctl->bar_mma, ph_mma);
    ph_mma ^= 1u;
    ptx::tc_fence_after();
    if (alias && cx.tid == 0)
      load_part(cx, a.blob, br.w_off[2], br.w_bytes[2], P.s_w[2], &cx.ctl->bar_w[2]);
    if (M.fast1) epilogue_hidden<true>(cx, cx.tmem_row, M.n1, M.kd2, h1, M.lo1, M.hi1, sA2);
    else epilogue_hidden<false>(cx, cx.tmem_row, M.n1, M.kd2, h1, M.lo1, M.hi1, sA2);
    ptx::tc_fence_before();
    ptx::fence_async_smem();
    __syncthreads();

    // conv 1x1: n1 -> n2
    if (cx.tid == 0) {
      if (!w_ready[1]) { wait_bar(cx, &cx.ctl->bar_w[1], ws.ph[1]); ws.ph[1] ^= 1u; w_ready[1] = true; }
      ptx::tc_fence_after();
      issue_gemm(cx.tmem + (uint32_t)P.d2_col, ptx::smem_u32(sA2), ptx::smem_u32(smem + P.s_w[1]), M.n2, 0, M.n2,
                 M.kd2);
      ptx::umma_commit(ptx::smem_u32(&cx.ctl->bar_mma));
    }
    wait_bar(cx, &cx.ctl->bar_mma, ph_mma);
    ph_mma ^= 1u;
    ptx::tc_fence_after();
    if (M.fast2) epilogue_hidden<true>(cx, cx.tmem_row + (uint32_t)P.d2_col, M.n2, M.kd3, h2, M.lo2, M.hi2, sA13);
    else epilogue_hidden<false>(cx, cx.tmem_row + (uint32_t)P.d2_col, M.n2, M.kd3, h2, M.lo2, M.hi2, sA13);
    ptx::tc_fence_before();
    ptx::fence_async_smem();
    __syncthreads();

    // conv 3x3: n2 -> cb, as nine per-tap partial products
    if (cx.tid == 0) {
      if (!w_ready[2] || alias) { wait_bar(cx, &cx.ctl->bar_w[2], ws.ph[2]); ws.ph[2] ^= 1u; w_ready[2] = true; }
      ptx::tc_fence_after();
      for (int n0 = 0; n0 < M.n3; n0 += 256)
        issue_gemm(cx.tmem + (uint32_t)n0, ptx::smem_u32(sA13), ptx::smem_u32(smem + P.s_w[2]), M.n3, n0,
                   min(256, M.n3 - n0), M.kd3);
      ptx::umma_commit(ptx::smem_u32(&cx.ctl->bar_mma));
    }
    wait_bar(cx, &cx.ctl->bar_mma, ph_mma);
    ph_mma ^= 1u;
    ptx::tc_fence_after();
    if (alias && cx.tid == 0 && (tile + 1) * kTileM < pvalid)
      load_part(cx, a.blob, br.w_off[0], br.w_bytes[0], P.s_w[0], &cx.ctl->bar_w[0]);
    epilogue_scatter(cx, cx.tmem_row, M.n3, cb, acc, pg, w, rp);
    ptx::tc_fence_before();
    __syncthreads();
  }

  // z_b = x_b + t (encode) or x_b = z_b - t (decode); clear the accumulator for the next coupling
  for (int idx = cx.tid; idx < cb * pg; idx += kThreads) {
    const int c = idx / pg, p = idx - c * pg;
    if (p < pvalid) {
      const OutRq o = orq[c];
      const uint32_t t = (uint32_t)rq_exact(acc[idx] + o.bias, o.m0, o.s);
      uint32_t* vv = reinterpret_cast<uint32_t*>(&v[colB[c] * pg + p]);
      *vv = kInv ? (*vv - t) : (*vv + t);
    }
    acc[idx] = 0;
  }
  __syncthreads();
}

// Prior head on the kept channels: (mu, log-scale index) for every factored-out element.
__device__ void run_prior(const Ctx& cx, const LevelPlan& P, const LevelArgs& a, int img0, int pvalid,
                          uint32_t& ph_meta, uint32_t& ph_mma, WeightState& ws) {
  uint8_t* smem = cx.smem;
  const int32_t* v = reinterpret_cast<const int32_t*>(smem + P.s_v);
  int8_t* xa = reinterpret_cast<int8_t*>(smem + P.s_xa);
  uint8_t* sA = smem + P.s_a13;
  const int pg = P.pg, ca = P.ca, cb = P.cb, w = P.w, h = P.h, px = P.px;
  const BlockRef& br = P.prior;
  if (cx.tid == 0) {
    load_part(cx, a.blob, br.meta_off, br.meta_bytes, P.s_meta, &cx.ctl->bar_meta);
    load_part(cx, a.blob, br.w_off[0], br.w_bytes[0], P.s_w[0], &cx.ctl->bar_w[0]);
  }
  wait_bar(cx, &cx.ctl->bar_meta, ph_meta);
  ph_meta ^= 1u;
  const uint8_t* mb = smem + P.s_meta;
  const PriorMeta M = *reinterpret_cast<const PriorMeta*>(mb);
  const OutRq* orq = reinterpret_cast<const OutRq*>(mb + M.off_out);
  for (int idx = cx.tid; idx < ca * pg; idx += kThreads) {
    const int c = idx / pg, p = idx - c * pg;
    int y = 0;
    if (p < pvalid) y = clampi(rq_exact(v[P.col_out[c] * pg + p], M.in_m0, M.in_s), -128, 127);
    xa[idx] = (int8_t)y;
  }
  __syncthreads();
  bool w_ready = false;
  for (int tile = 0; tile < P.tiles; ++tile) {
    if (tile * kTileM >= pvalid) break;
    const RowPos rp = row_pos(tile, cx.row, pvalid, px, h, w);
    build_im2col(cx, sA, xa, ca, pg, w, M.kd, rp);
    ptx::fence_async_smem();
    __syncthreads();
    if (cx.tid == 0) {
      if (!w_ready) { wait_bar(cx, &cx.ctl->bar_w[0], ws.ph[0]); ws.ph[0] ^= 1u; w_ready = true; }
      ptx::tc_fence_after();
      issue_gemm(cx.tmem, ptx::smem_u32(sA), ptx::smem_u32(smem + P.s_w[0]), M.n, 0, M.n, M.kd);
      ptx::umma_commit(ptx::smem_u32(&cx.ctl->bar_mma));
    }
    wait_bar(cx, &cx.ctl->bar_mma, ph_mma);
    ph_mma ^= 1u;
    ptx::tc_fence_after();
    const int g = rp.valid ? rp.p / px : 0;
    const int q = rp.p - g * px;
    int32_t* mu = a.prior + (size_t)(img0 + g) * 2u * P.d_fact + P.prior_off + q;
    int32_t* ls = mu + P.d_fact;
    const int nblk = M.n >> 4;
    for (int b = cx.wh; b < nblk; b += kThreads / kTileM) {
      uint32_t r[16];
      ptx::tmem_ld16(cx.tmem_row + (uint32_t)(b << 4), r);
      ptx::tmem_ld_wait();
      if (rp.valid) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int col = (b << 4) + i;
          if (col < 2 * cb) {
            const OutRq o = orq[col];
            const int32_t y = rq_exact((int32_t)r[i] + o.bias, o.m0, o.s);
            if (col < cb) mu[(size_t)col * px] = y;
            else ls[(size_t)(col - cb) * px] = clampi(y, M.ls_lo, M.ls_hi);
          }
        }
      }
    }
    ptx::tc_fence_before();
    __syncthreads();
  }
}

template <bool kInv>
__global__ void __launch_bounds__(kThreads, 1) level_kernel(const LevelArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ Ctl ctl;
  const LevelPlan& P = *a.plan;
  Ctx cx;
  cx.smem = smem;
  cx.ctl = &ctl;
  cx.status = a.status;
  cx.tid = threadIdx.x;
  cx.warp = cx.tid >> 5;
  cx.lane = cx.tid & 31;
  cx.wq = cx.warp & 3;
  cx.wh = cx.warp >> 2;
  cx.row = cx.wq * 32 + cx.lane;

  if (cx.tid == 0) {
    ptx::mbar_init(ptx::smem_u32(&ctl.bar_meta), 1);
    for (int i = 0; i < 3; ++i) ptx::mbar_init(ptx::smem_u32(&ctl.bar_w[i]), 1);
    ptx::mbar_init(ptx::smem_u32(&ctl.bar_mma), 1);
    ptx::mbar_init_fence();
    ctl.abort = 0;
  }
  if (cx.warp == 0) ptx::tmem_alloc(ptx::smem_u32(&ctl.tmem_base), (uint32_t)P.tmem_cols);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  cx.tmem = ctl.tmem_base;
  cx.tmem_row = cx.tmem + ((uint32_t)(cx.wq * 32) << 16);

  const int c = P.c, px = P.px, pg = P.pg, w = P.w;
  const int img0 = blockIdx.x * P.group;
  const int nimg = min(P.group, a.batch - img0);
  const int pvalid = nimg * px;
  const int per_img = c * px;                    // elements per image at this level
  int32_t* v = reinterpret_cast<int32_t*>(smem + P.s_v);
  int32_t* acc = reinterpret_cast<int32_t*>(smem + P.s_acc);
  for (int idx = cx.tid; idx < P.cb * pg; idx += kThreads) acc[idx] = 0;

  if (!kInv) {
    // space-to-depth on load: plane c*4 + dy*2 + dx, pixel (i, j) <- in[c][2i+dy][2j+dx]
    const int w2 = 2 * w;
    for (int e = cx.tid; e < nimg * per_img; e += kThreads) {
      const int g = e / per_img, r = e - g * per_img;
      const int ci = r / (4 * px), r2 = r - ci * 4 * px;
      const int y = r2 / w2, x = r2 - y * w2;
      const size_t src = (size_t)(img0 + g) * per_img + r;
      const int32_t val = P.is_first ? (int32_t) reinterpret_cast<const uint8_t*>(a.in)[src]
                                     : reinterpret_cast<const int32_t*>(a.in)[src];
      v[(ci * 4 + (y & 1) * 2 + (x & 1)) * pg + g * px + (y >> 1) * w + (x >> 1)] = val;
    }
  } else {
    // merge: logical channel k < keep_c from the deeper level, the rest from z's block of this level
    for (int e = cx.tid; e < nimg * per_img; e += kThreads) {
      const int g = e / per_img, r = e - g * per_img;
      const int k = r / px, q = r - k * px;
      const size_t b = (size_t)(img0 + g);
      const int32_t val = (k < P.keep_c)
                              ? reinterpret_cast<const int32_t*>(a.in)[b * (size_t)a.in_stride + (size_t)k * px + q]
                              : a.z[b * P.d + P.z_off + (size_t)(k - P.keep_c) * px + q];
      v[P.col_out[k] * pg + g * px + q] = val;
    }
  }
  __syncthreads();

  uint32_t ph_meta = 0, ph_mma = 0;
  WeightState ws;
  ws.ph[0] = ws.ph[1] = ws.ph[2] = 0;

  if (kInv && P.has_prior && a.prior != nullptr) run_prior(cx, P, a, img0, pvalid, ph_meta, ph_mma, ws);

  for (int jj = 0; jj < P.n_couplings; ++jj) {
    const int j = kInv ? (P.n_couplings - 1 - jj) : jj;
    run_coupling<kInv>(cx, P, a, P.coupling[j], pvalid, ph_meta, ph_mma, ws);
  }

  if (!kInv) {
    // split on store: factored-out half -> z block of this level; kept half -> next level (or the
    // final z block)
    int32_t* keep_out = reinterpret_cast<int32_t*>(a.out);
    for (int e = cx.tid; e < nimg * per_img; e += kThreads) {
      const int g = e / per_img, r = e - g * per_img;
      const int k = r / px, q = r - k * px;
      const size_t b = (size_t)(img0 + g);
      const int32_t val = v[P.col_out[k] * pg + g * px + q];
      if (k >= P.keep_c) a.z[b * P.d + P.z_off + (size_t)(k - P.keep_c) * px + q] = val;
      else if (P.is_last) a.z[b * P.d + P.z_final_off + (size_t)k * px + q] = val;
      else keep_out[(b * P.keep_c + k) * (size_t)px + q] = val;
    }
    if (P.has_prior && a.prior != nullptr) run_prior(cx, P, a, img0, pvalid, ph_meta, ph_mma, ws);
  } else {
    // depth-to-space on store
    const int w2 = 2 * w;
    uint32_t bad = 0;
    for (int e = cx.tid; e < nimg * per_img; e += kThreads) {
      const int g = e / per_img, r = e - g * per_img;
      const int ci = r / (4 * px), r2 = r - ci * 4 * px;
      const int y = r2 / w2, x = r2 - y * w2;
      const int32_t val = v[(ci * 4 + (y & 1) * 2 + (x & 1)) * pg + g * px + (y >> 1) * w + (x >> 1)];
      const size_t dst = (size_t)(img0 + g) * per_img + r;
      if (P.is_first) {
        reinterpret_cast<uint8_t*>(a.out)[dst] = (uint8_t)((uint32_t)val & 0xFFu);
        bad += (val < 0 || val > 255) ? 1u : 0u;
      } else {
        reinterpret_cast<int32_t*>(a.out)[dst] = val;
      }
    }
    if (P.is_first && a.oor != nullptr) {
      bad = __reduce_add_sync(0xFFFFFFFFu, bad);
      if (cx.lane == 0 && bad) atomicAdd(a.oor, bad);
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (cx.warp == 0) ptx::tmem_dealloc(cx.tmem, (uint32_t)P.tmem_cols);
}

}  // namespace

cudaError_t launch_level(const LevelArgs& args, bool inverse, int grid, uint32_t smem_bytes, cudaStream_t stream) {
  if (inverse) level_kernel<true><<<grid, kThreads, smem_bytes, stream>>>(args);
  else level_kernel<false><<<grid, kThreads, smem_bytes, stream>>>(args);
  return cudaGetLastError();
}

cudaError_t configure_level_kernels(uint32_t max_smem_bytes) {
  cudaError_t e = cudaFuncSetAttribute(level_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)max_smem_bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(level_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem_bytes);
}

}  // namespace iodf
