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
// Execution structure: 16 worker warps and one control warp. The workers form one or two groups;
// each group owns a tile slot (an A-operand buffer in shared memory and a range of TMEM columns)
// and walks its tiles through build -> epilogue 1 -> epilogue 2 -> scatter, handing the slot to
// the control thread between stages through mbarriers. The control thread issues the bulk copies
// of weights and the MMAs, so while one group requantises, the tensor core works for the other.
#include "iodf_dev.h"
#include "level_kernel.h"
#include "ptx.cuh"

namespace iodf {

namespace {

struct __align__(16) Ctl {
  uint64_t a_ready[2];    // workers -> control: the slot's A operand is written (count = group threads)
  uint64_t d_ready[2];    // tensor core -> workers: the slot's accumulator is complete
  uint64_t w_full[3];     // bulk copy -> control: weight slot filled
  uint64_t w_free[3];     // tensor core -> control: last MMA reading the weight slot is complete
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
  int group, cs, ncs;     // tile slot, column-split index and count inside the group
  int row;                // tile row (= TMEM lane) of this thread
  uint32_t tmem_slot;     // TMEM address of the slot's first column, this warp's lane quarter
};

// Bounded wait on an mbarrier phase. After one wait in the CTA has given up, every later wait
// returns at once, so a stuck CTA drains in bounded time, frees its TMEM and exits.
__device__ __noinline__ bool wait_bar(Ctl* ctl, uint32_t* status, uint64_t* bar, uint32_t parity) {
  volatile uint32_t* ab = &ctl->abort;
  if (*ab) return false;
  const uint32_t b = ptx::smem_u32(bar);
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (ptx::mbar_try_wait(b, parity)) return true;
    if ((it & 255u) == 255u && *ab) return false;
  }
  *ab = 1;
  atomicExch(status, 1u);
  return false;
}

__device__ __forceinline__ void worker_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kWorkers) : "memory"); }

__device__ __forceinline__ int32_t rq_exact(int32_t a, int32_t m0, int32_t s) {
  const long long p = (long long)a * (long long)m0 + (1ll << (30 + s));
  return (int32_t)(p >> (31 + s));
}

__device__ __forceinline__ int clampi(int v, int lo, int hi) { return min(max(v, lo), hi); }

__device__ __forceinline__ int min_relu(int v, int hi) {
  int r;
  asm("min.relu.s32 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(hi));
  return r;
}

template <bool kFast, bool kLo0>
__device__ __forceinline__ int rq_hidden(int acc, const HiddenRq r, int lo, int hi) {
  const long long c64 = (long long)(((unsigned long long)r.c_hi << 32) | (unsigned long long)r.c_lo);
  const long long p = (long long)acc * (long long)r.m0 + c64;
  int y;
  if (kFast) y = ((int)(p >> 32)) >> r.sh;
  else y = (int)(p >> (32 + r.sh));
  return kLo0 ? min_relu(y, hi) : clampi(y, lo, hi);
}

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

__device__ __forceinline__ int tap_offset(int tap, int w) {
  const int u = (tap * 11) >> 5;            // tap / 3 for 0..8
  return (u - 1) * w + (tap - u * 3 - 1);
}

// A[row][tap*cpad + c] = xa[p + tap offset][c] (0 outside the image), as aligned 8-byte granules,
// written in 16-byte chunks into the MMA operand layout [K/16][128][16].
__device__ void build_im2col(const Ctx& cx, uint8_t* sA, const int8_t* xa, int cpad, int w, int kd, const RowPos rp) {
  const int nchunks = kd >> 4;
  const int gpt = cpad >> 3;                // granules per tap
  const int ngran = 9 * gpt;
  for (int jc = cx.cs; jc < nchunks; jc += cx.ncs) {
    uint2 g2[2];
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int g = 2 * jc + half;
      g2[half] = make_uint2(0u, 0u);
      if (g < ngran) {
        const int tap = g / gpt, i = g - tap * gpt;
        if ((rp.gmask >> tap) & 1u)
          g2[half] = *reinterpret_cast<const uint2*>(xa + (size_t)(rp.p + tap_offset(tap, w)) * cpad + 8 * i);
      }
    }
    *reinterpret_cast<uint4*>(sA + (size_t)jc * (kTileM * 16) + cx.row * 16) =
        make_uint4(g2[0].x, g2[0].y, g2[1].x, g2[1].y);
  }
}

// 16 accumulator columns -> requantised bytes -> one 16-byte chunk of the next A operand.
template <bool kFast, bool kLo0>
__device__ __forceinline__ uint4 requant16(const uint32_t* r, const HiddenRq* rq, int lo, int hi) {
  uint32_t wd[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int y0 = rq_hidden<kFast, kLo0>((int)r[4 * i + 0], rq[4 * i + 0], lo, hi);
    const int y1 = rq_hidden<kFast, kLo0>((int)r[4 * i + 1], rq[4 * i + 1], lo, hi);
    const int y2 = rq_hidden<kFast, kLo0>((int)r[4 * i + 2], rq[4 * i + 2], lo, hi);
    const int y3 = rq_hidden<kFast, kLo0>((int)r[4 * i + 3], rq[4 * i + 3], lo, hi);
    wd[i] = pack4(y0, y1, y2, y3);
  }
  return make_uint4(wd[0], wd[1], wd[2], wd[3]);
}

// TMEM accumulator -> requantised int8 activations in the next GEMM's A layout. n is a multiple
// of 16; kd (the next GEMM's K) is n rounded up to 32, the extra chunk being zero.
template <bool kFast, bool kLo0>
__device__ void epilogue_hidden_t(const Ctx& cx, int n, int kd, const HiddenRq* rq, int lo, int hi, uint8_t* sOut) {
  const int nblk = (n + 31) >> 5;
  for (int b = cx.cs; b < nblk; b += cx.ncs) {
    const int c0 = b << 5;
    uint8_t* dst = sOut + (size_t)(2 * b) * (kTileM * 16) + cx.row * 16;
    if (n - c0 >= 32) {
      uint32_t r[32];
      ptx::tmem_ld32(cx.tmem_slot + (uint32_t)c0, r);
      ptx::tmem_ld_wait();
      *reinterpret_cast<uint4*>(dst) = requant16<kFast, kLo0>(r, rq + c0, lo, hi);
      *reinterpret_cast<uint4*>(dst + kTileM * 16) = requant16<kFast, kLo0>(r + 16, rq + c0 + 16, lo, hi);
    } else {
      uint32_t r[16];
      ptx::tmem_ld16(cx.tmem_slot + (uint32_t)c0, r);
      ptx::tmem_ld_wait();
      *reinterpret_cast<uint4*>(dst) = requant16<kFast, kLo0>(r, rq + c0, lo, hi);
      if (c0 + 16 < kd) *reinterpret_cast<uint4*>(dst + kTileM * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

__device__ void epilogue_hidden(const Ctx& cx, int fast, int n, int kd, const HiddenRq* rq, int lo, int hi,
                                uint8_t* sOut) {
  if (fast) {
    if (lo == 0) epilogue_hidden_t<true, true>(cx, n, kd, rq, lo, hi, sOut);
    else epilogue_hidden_t<true, false>(cx, n, kd, rq, lo, hi, sOut);
  } else {
    epilogue_hidden_t<false, false>(cx, n, kd, rq, lo, hi, sOut);
  }
}

// Per-tap partial products -> shifted sum into the translation accumulator. Column granule gi
// (8 columns) belongs to tap gi / (cbp/8) and out channels (gi % (cbp/8))*8 .. +8.
__device__ void epilogue_scatter(const Ctx& cx, int cb, int cbp, int32_t* acc, int pg, int w, const RowPos rp) {
  const int gpt = cbp >> 3;
  const int ngran = 9 * gpt;
  for (int gi = cx.cs; gi < ngran; gi += cx.ncs) {
    uint32_t r[8];
    ptx::tmem_ld8(cx.tmem_slot + (uint32_t)(gi << 3), r);
    ptx::tmem_ld_wait();
    const int tap = gi / gpt;
    const int c0 = (gi - tap * gpt) << 3;
    if (rp.valid && ((rp.smask >> tap) & 1u)) {
      int32_t* dst = acc + c0 * pg + rp.p - tap_offset(tap, w);
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (c0 + i < cb) atomicAdd(dst + i * pg, (int32_t)r[i]);
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
    ptx::tmem_ld_wait();
    if (rp.valid) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int col = (gi << 3) + i;
        if (col < 2 * cb) {
          const OutRq o = orq[col];
          const int32_t y = rq_exact((int32_t)r[i] + o.bias, o.m0, o.s);
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

// ---- control thread ---------------------------------------------------------------------------
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

struct WSlot {
  uint32_t full_par, free_par;
  int uses_left, cur_uses;
  bool inflight, need_free, exhausted;
  int g_step, g_sub;      // position of the load-sequence generator
};

struct Control {
  const LevelPlan& P;
  const LevelArgs& a;
  uint8_t* smem;
  Ctl* ctl;
  Steps st;
  int ntv;                // valid tiles of this CTA
  bool alias;
  WSlot ws[3];

  __device__ bool wait(uint64_t* bar, uint32_t par) { return wait_bar(ctl, a.status, bar, par); }

  __device__ void bulk(uint32_t off, uint32_t bytes, uint32_t s_dst, uint64_t* bar) {
    const uint32_t b = ptx::smem_u32(bar);
    ptx::mbar_expect_tx(b, bytes);
    ptx::bulk_g2s(ptx::smem_u32(smem + s_dst), a.blob + off, bytes, b);
  }

  // Next matrix that weight slot s will hold, in the fixed order the MMAs consume them.
  __device__ bool next_load(int s, uint32_t* off, uint32_t* bytes, int* uses) {
    WSlot& w = ws[s];
    for (;;) {
      if (w.g_step >= st.nsteps) return false;
      const BlockRef& br = step_ref(P, st, w.g_step);
      if (st.is_prior(w.g_step)) {
        if (s != 0 || w.g_sub > 0) { ++w.g_step; w.g_sub = 0; continue; }
        *off = br.w_off[0]; *bytes = br.w_bytes[0]; *uses = ntv; w.g_sub = 1;
        return true;
      }
      if (alias && s == 0) {                      // W1, W3, W1, W3, ... once per tile
        if (w.g_sub >= 2 * ntv) { ++w.g_step; w.g_sub = 0; continue; }
        const int which = (w.g_sub & 1) ? 2 : 0;
        *off = br.w_off[which]; *bytes = br.w_bytes[which]; *uses = 1; ++w.g_sub;
        return true;
      }
      if (alias && s == 2) return false;
      if (w.g_sub > 0) { ++w.g_step; w.g_sub = 0; continue; }
      *off = br.w_off[s]; *bytes = br.w_bytes[s]; *uses = ntv; w.g_sub = 1;
      return true;
    }
  }

  __device__ void issue_next(int s) {
    uint32_t off, bytes;
    int uses;
    if (!next_load(s, &off, &bytes, &uses)) { ws[s].exhausted = true; return; }
    bulk(off, bytes, P.s_w[s], &ctl->w_full[s]);
    ws[s].inflight = true;
    ws[s].cur_uses = uses;
  }

  __device__ void try_prefetch(int s) {
    WSlot& w = ws[s];
    if (w.uses_left != 0 || w.inflight || w.exhausted) return;
    if (w.need_free) {
      if (!ptx::mbar_try_wait(ptx::smem_u32(&ctl->w_free[s]), w.free_par)) return;
      w.free_par ^= 1u;
      w.need_free = false;
    }
    issue_next(s);
  }

  __device__ void acquire(int s) {
    WSlot& w = ws[s];
    if (w.uses_left != 0) return;
    if (!w.inflight) {
      if (w.need_free) { wait(&ctl->w_free[s], w.free_par); w.free_par ^= 1u; w.need_free = false; }
      issue_next(s);
    }
    wait(&ctl->w_full[s], w.full_par);
    w.full_par ^= 1u;
    w.uses_left = w.cur_uses;
    w.inflight = false;
  }

  __device__ void release(int s) {
    WSlot& w = ws[s];
    if (--w.uses_left == 0) {
      ptx::umma_commit(ptx::smem_u32(&ctl->w_free[s]));
      w.need_free = true;
    }
  }

  __device__ void run(uint32_t tmem) {
    for (int s = 0; s < 3; ++s) {
      ws[s].full_par = ws[s].free_par = 0;
      ws[s].uses_left = ws[s].cur_uses = 0;
      ws[s].inflight = ws[s].need_free = ws[s].exhausted = false;
      ws[s].g_step = ws[s].g_sub = 0;
    }
    for (int i = 0; i < st.nsteps && i < 2; ++i) {
      const BlockRef& br = step_ref(P, st, i);
      bulk(br.meta_off, br.meta_bytes, P.s_meta[i], &ctl->meta_full[i]);
    }
    for (int s = 0; s < 3; ++s) try_prefetch(s);

    uint32_t apar[2] = {0u, 0u};
    const int nslots = P.nslots;
    for (int i = 0; i < st.nsteps; ++i) {
      if (!wait(&ctl->meta_full[i & 1], (uint32_t)((i >> 1) & 1))) return;
      const uint8_t* mb = smem + P.s_meta[i & 1];
      const bool prior = st.is_prior(i);
      int n[3], kd[3];
      if (prior) {
        const PriorMeta* M = reinterpret_cast<const PriorMeta*>(mb);
        n[0] = M->n; kd[0] = M->kd;
        n[1] = n[2] = kd[1] = kd[2] = 0;
      } else {
        const CouplingMeta* M = reinterpret_cast<const CouplingMeta*>(mb);
        n[0] = M->n1; n[1] = M->n2; n[2] = M->n3;
        kd[0] = M->kd1; kd[1] = M->kd2; kd[2] = M->kd3;
      }
      const int nstages = prior ? 1 : 3;
      int tcur[2] = {0, 1}, stg[2] = {0, 0};
      int remaining = ntv * nstages;
      bool first = true;
      uint32_t spin = 0;
      while (remaining > 0) {
        bool progress = false;
        for (int s = 0; s < nslots; ++s) {
          if (tcur[s] >= ntv) continue;
          if (!ptx::mbar_try_wait(ptx::smem_u32(&ctl->a_ready[s]), apar[s])) continue;
          apar[s] ^= 1u;
          ptx::tc_fence_after();
          if (first) {
            // every worker has left step i-1, so its meta slot can take step i+1
            first = false;
            if (i >= 1 && i + 1 < st.nsteps) {
              const BlockRef& br = step_ref(P, st, i + 1);
              bulk(br.meta_off, br.meta_bytes, P.s_meta[(i + 1) & 1], &ctl->meta_full[(i + 1) & 1]);
            }
          }
          const int stage = stg[s];
          const int phys = prior ? 0 : ((stage == 2 && alias) ? 0 : stage);
          acquire(phys);
          const uint32_t d = tmem + (uint32_t)(s * kSlotCols);
          const uint32_t sa = ptx::smem_u32(smem + P.s_a[s]);
          const uint32_t sb = ptx::smem_u32(smem + P.s_w[phys]);
          for (int n0 = 0; n0 < n[stage]; n0 += 256)
            issue_gemm(d + (uint32_t)n0, sa, sb, n[stage], n0, min(256, n[stage] - n0), kd[stage]);
          ptx::umma_commit(ptx::smem_u32(&ctl->d_ready[s]));
          release(phys);
          if (++stg[s] == nstages) { stg[s] = 0; tcur[s] += nslots; }
          --remaining;
          progress = true;
        }
        for (int s = 0; s < 3; ++s) try_prefetch(s);
        if (progress) spin = 0;
        else if (++spin > kSpinLimit || ctl->abort) {
          if (!ctl->abort) { ctl->abort = 1; atomicExch(a.status, 1u); }
          return;
        }
      }
    }
  }
};

// ---- workers ----------------------------------------------------------------------------------
template <bool kInv>
__device__ void run_workers(Ctx& cx, const LevelPlan& P, const LevelArgs& a, const Steps& st, int img0, int pvalid,
                            int ntv) {
  uint8_t* smem = cx.smem;
  Ctl* ctl = cx.ctl;
  int32_t* v = reinterpret_cast<int32_t*>(smem + P.s_v);
  int8_t* xa = reinterpret_cast<int8_t*>(smem + P.s_xa);
  int32_t* acc = reinterpret_cast<int32_t*>(smem + P.s_acc);
  uint8_t* sA = smem + P.s_a[cx.group];
  const int pg = P.pg, ca = P.ca, cb = P.cb, w = P.w, h = P.h, px = P.px, cpad = P.cpad, cbp = P.cbp;
  const int gthreads = (kWorkers / P.nslots);
  uint64_t* a_ready = &ctl->a_ready[cx.group];
  uint64_t* d_ready = &ctl->d_ready[cx.group];
  uint32_t dpar = 0;
  const CouplingMeta* prevM = nullptr;       // coupling whose translation is still to be applied

  auto arrive_a = [&]() {
    ptx::tc_fence_before();
    ptx::fence_async_smem();
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(ptx::smem_u32(a_ready)) : "memory");
  };
  auto wait_d = [&]() {
    wait_bar(ctl, a.status, d_ready, dpar);
    dpar ^= 1u;
    ptx::tc_fence_after();
  };
  // x_b +/-= rq(acc + bias) of the previous coupling for pixel p
  auto apply_translation = [&](int p) {
    const uint8_t* pm = reinterpret_cast<const uint8_t*>(prevM);
    const int32_t* colB = reinterpret_cast<const int32_t*>(pm + prevM->off_colB);
    const OutRq* orq = reinterpret_cast<const OutRq*>(pm + prevM->off_out);
    for (int c = 0; c < cb; ++c) {
      const OutRq o = orq[c];
      const uint32_t t = (uint32_t)rq_exact(acc[c * pg + p] + o.bias, o.m0, o.s);
      acc[c * pg + p] = 0;
      uint32_t* vv = reinterpret_cast<uint32_t*>(&v[colB[c] * pg + p]);
      *vv = kInv ? (*vv - t) : (*vv + t);
    }
  };
  // network input of pixel p: ca channels requantised to int8, padded to cpad bytes
  auto requant_input = [&](int p, const int32_t* cols, int32_t m0, int32_t s) {
    for (int g0 = 0; g0 < cpad; g0 += 8) {
      int y[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        y[i] = 0;
        if (g0 + i < ca) y[i] = clampi(rq_exact(v[cols[g0 + i] * pg + p], m0, s), -128, 127);
      }
      *reinterpret_cast<uint2*>(xa + (size_t)p * cpad + g0) =
          make_uint2(pack4(y[0], y[1], y[2], y[3]), pack4(y[4], y[5], y[6], y[7]));
    }
  };

  for (int i = 0; i < st.nsteps; ++i) {
    wait_bar(ctl, a.status, &ctl->meta_full[i & 1], (uint32_t)((i >> 1) & 1));
    const uint8_t* mb = smem + P.s_meta[i & 1];
    const bool prior = st.is_prior(i);
    if (prior) {
      const PriorMeta M = *reinterpret_cast<const PriorMeta*>(mb);
      const OutRq* orq = reinterpret_cast<const OutRq*>(mb + M.off_out);
      for (int p = cx.tid; p < pvalid; p += kWorkers) {
        if (prevM) apply_translation(p);
        requant_input(p, P.col_out, M.in_m0, M.in_s);
      }
      prevM = nullptr;
      worker_barrier();
      for (int t = cx.group; t < ntv; t += P.nslots) {
        const RowPos rp = row_pos(t, cx.row, pvalid, px, h, w);
        build_im2col(cx, sA, xa, cpad, w, M.kd, rp);
        arrive_a();
        wait_d();
        epilogue_prior(cx, P, a, M, orq, img0, rp);
      }
      worker_barrier();
      continue;
    }
    const CouplingMeta* Mp = reinterpret_cast<const CouplingMeta*>(mb);
    const CouplingMeta M = *Mp;
    const int32_t* colA = reinterpret_cast<const int32_t*>(mb + M.off_colA);
    const HiddenRq* h1 = reinterpret_cast<const HiddenRq*>(mb + M.off_h1);
    const HiddenRq* h2 = reinterpret_cast<const HiddenRq*>(mb + M.off_h2);
    for (int p = cx.tid; p < pvalid; p += kWorkers) {
      if (prevM) apply_translation(p);
      requant_input(p, colA, M.in_m0, M.in_s);
    }
    prevM = Mp;
    worker_barrier();
    for (int t = cx.group; t < ntv; t += P.nslots) {
      const RowPos rp = row_pos(t, cx.row, pvalid, px, h, w);
      build_im2col(cx, sA, xa, cpad, w, M.kd1, rp);
      arrive_a();
      wait_d();
      epilogue_hidden(cx, M.fast1, M.n1, M.kd2, h1, M.lo1, M.hi1, sA);
      arrive_a();
      wait_d();
      epilogue_hidden(cx, M.fast2, M.n2, M.kd3, h2, M.lo2, M.hi2, sA);
      arrive_a();
      wait_d();
      epilogue_scatter(cx, cb, cbp, acc, pg, w, rp);
    }
    ptx::tc_fence_before();
    worker_barrier();
  }
  if (prevM) {
    for (int p = cx.tid; p < pvalid; p += kWorkers) apply_translation(p);
    worker_barrier();
  }
  (void)gthreads;
}

template <bool kInv>
__global__ void __launch_bounds__(kThreads, 1) level_kernel(const LevelArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ Ctl ctl;
  const LevelPlan& P = *a.plan;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool is_worker = warp < kWorkerWarps;
  const int wpg = kWorkerWarps / P.nslots;       // warps per group

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(ptx::smem_u32(&ctl.a_ready[s]), (uint32_t)(wpg * 32));
      ptx::mbar_init(ptx::smem_u32(&ctl.d_ready[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl.meta_full[s]), 1);
    }
    for (int s = 0; s < 3; ++s) {
      ptx::mbar_init(ptx::smem_u32(&ctl.w_full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl.w_free[s]), 1);
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
  st.n_couplings = P.n_couplings;
  st.do_prior = P.has_prior && a.prior != nullptr;
  st.nsteps = P.n_couplings + (st.do_prior ? 1 : 0);
  st.inverse = kInv;

  if (!is_worker) {
    if (lane == 0) {
      Control ctrl{P, a, smem, &ctl, st, ntv, P.w13_alias != 0};
      ctrl.run(tmem);
    }
  } else {
    Ctx cx;
    cx.smem = smem;
    cx.ctl = &ctl;
    cx.status = a.status;
    cx.tid = tid;
    cx.warp = warp;
    cx.lane = lane;
    cx.wq = warp & 3;
    cx.group = warp / wpg;
    cx.cs = (warp % wpg) >> 2;
    cx.ncs = wpg >> 2;
    cx.row = cx.wq * 32 + lane;
    cx.tmem_slot = tmem + ((uint32_t)(cx.wq * 32) << 16) + (uint32_t)(cx.group * kSlotCols);

    int32_t* acc = reinterpret_cast<int32_t*>(smem + P.s_acc);
    for (int idx = tid; idx < P.cb * pg; idx += kWorkers) acc[idx] = 0;
    if (!kInv) {
      // space-to-depth on load: plane c*4 + dy*2 + dx, pixel (i, j) <- in[c][2i+dy][2j+dx]
      const int w2 = 2 * w;
      for (int e = tid; e < nimg * per_img; e += kWorkers) {
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
      for (int e = tid; e < nimg * per_img; e += kWorkers) {
        const int g = e / per_img, r = e - g * per_img;
        const int k = r / px, q = r - k * px;
        const size_t b = (size_t)(img0 + g);
        const int32_t val =
            (k < P.keep_c) ? reinterpret_cast<const int32_t*>(a.in)[b * (size_t)a.in_stride + (size_t)k * px + q]
                           : a.z[b * P.d + P.z_off + (size_t)(k - P.keep_c) * px + q];
        v[P.col_out[k] * pg + g * px + q] = val;
      }
    }
    worker_barrier();

    run_workers<kInv>(cx, P, a, st, img0, pvalid, ntv);

    if (!kInv) {
      // split on store: factored-out half -> z block of this level; kept half -> next level (or
      // the final z block)
      int32_t* keep_out = reinterpret_cast<int32_t*>(a.out);
      for (int e = tid; e < nimg * per_img; e += kWorkers) {
        const int g = e / per_img, r = e - g * per_img;
        const int k = r / px, q = r - k * px;
        const size_t b = (size_t)(img0 + g);
        const int32_t val = v[P.col_out[k] * pg + g * px + q];
        if (k >= P.keep_c) a.z[b * P.d + P.z_off + (size_t)(k - P.keep_c) * px + q] = val;
        else if (P.is_last) a.z[b * P.d + P.z_final_off + (size_t)k * px + q] = val;
        else keep_out[(b * P.keep_c + k) * (size_t)px + q] = val;
      }
    } else {
      // depth-to-space on store
      const int w2 = 2 * w;
      uint32_t bad = 0;
      for (int e = tid; e < nimg * per_img; e += kWorkers) {
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
