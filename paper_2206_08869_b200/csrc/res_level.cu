// One flow level whose couplings use the paper's residual-block network (Eq. 3, Sec. 4.1; scatter
// add, Sec. 4.5; App. B.1: conv 3x3 -> L blocks of two 3x3 convs -> conv 3x3, all on `hidden`
// channels), one CTA per image, images of at most 256 pixels at this level.
//
// Every conv here is a 3x3 conv over hidden activations, so a pixel needs its neighbours' hidden
// values: the activations of the whole image stay in shared memory (X: the block tensor, D channels;
// MID: the first conv's output; both unsigned 8-bit, pixel-major) and a conv is
//
//   for each 128-pixel tile, for each tap (u, v):
//     A slice  [128 x kpad]   rows = the tile's pixels shifted by the tap (zero outside the image),
//                             copied from the source buffer into the MMA operand layout
//     W slice  [n_pad x kpad] the tap's weights, bulk-copied from the packed blob (L2)
//     D[tile] (+)= A * W^T    tcgen05.mma kind::i8, K = kpad, accumulators of all tiles in TMEM
//   epilogue: TMEM -> exact 64-bit requantisation -> what the conv's kind says (see ResKind)
//
// Slices are double-buffered: while the tensor core works on slice g the builders write slice g+1,
// and the weights travel through a ring several slices ahead. A block is
//   MID = clip(ReLU(rq(conv_a(X))))                        kResHidden
//   X   = rq(X; M_r, s_r)      for all D channels          the shortcut Q(x), in place
//   X[idx[j]] = clip(max(X[idx[j]] + rq(conv_b(MID))[j], 0), 0, 255)   kResBranch: scatter add + ReLU
// which equals Eq. 3 with the scatter add because rq(X) of an 8-bit X with a multiplier below one
// is again in 0..255, and channels that the second conv does not keep only get the shortcut.
//
// Sixteen builder warps write the operand slices and requantise; one more warp's elected lane
// requests the weight slices and issues the MMAs, so building slice g+1 overlaps issuing slice g.
// This is a first version of the path: convs run one after another, a conv's epilogue does not
// overlap the next conv's MMAs.
#include "res_level.h"
#include "ptx.cuh"

namespace iodf {

namespace {

struct __align__(16) ResCtl {
  uint64_t w_full[kResMaxWSlots];   // bulk copy -> issuer: weight ring slot filled
  uint64_t slice_done[2];   // tensor core -> everyone: the MMAs that read A/W buffer b have completed
  uint64_t a_full[2];       // builders -> issuer: A slice buffer b written (one arrival per builder warp)
  uint32_t tmem_base;
  uint32_t abort;
};

// bounded wait on an mbarrier phase; after one wait has given up every later one returns at once
__device__ __noinline__ bool res_wait(ResCtl* ctl, uint32_t* status, uint64_t* bar, uint32_t parity) {
  volatile uint32_t* ab = &ctl->abort;
  if (*ab) return false;
  const uint32_t b = ptx::smem_u32(bar);
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (ptx::mbar_try_wait(b, parity)) return true;
    if (*ab) return false;
  }
  *ab = 1;
  atomicExch(status, 1u);
  return false;
}

// usually the phase has completed already: probe inline before the bounded blocking wait
__device__ __forceinline__ void res_wait_fast(ResCtl* ctl, uint32_t* status, uint64_t* bar, uint32_t parity) {
  const uint32_t b = ptx::smem_u32(bar);
  for (int it = 0; it < 64; ++it)
    if (ptx::mbar_test_wait(b, parity)) return;
  res_wait(ctl, status, bar, parity);
}

__device__ __forceinline__ int rdiv(int n, uint32_t mul) { return mul ? (int)__umulhi((uint32_t)n, mul) : n; }

__device__ __forceinline__ int32_t rq64(int32_t a, int32_t m0, int32_t s) {
  const long long p = (long long)a * (long long)m0 + (1ll << (30 + s));
  return (int32_t)(p >> (31 + s));
}

__device__ __forceinline__ int32_t rq_const(int32_t acc, const OutRq o) {     // c64 = bias * m0 + 2^(30+s)
  const long long c64 = (long long)(((unsigned long long)o.c_hi << 32) | (unsigned long long)o.c_lo);
  const long long p = (long long)acc * (long long)o.m0 + c64;
  return (int32_t)(p >> (31 + o.s));
}

__device__ __forceinline__ int clampi(int v, int lo, int hi) { return min(max(v, lo), hi); }

struct Geo {
  int px, h, w, pg;
  uint32_t mul_w;
};

// bit t = u*3+v of the mask: input pixel (i+u-1, j+v-1) is inside the image
__device__ __forceinline__ uint32_t gather_mask(int p, const Geo& g) {
  if (p >= g.px) return 0u;
  const int i = rdiv(p, g.mul_w), j = p - i * g.w;
  uint32_t m = 0;
#pragma unroll
  for (int u = 0; u < 3; ++u)
#pragma unroll
    for (int v = 0; v < 3; ++v)
      if (i + u - 1 >= 0 && i + u - 1 < g.h && j + v - 1 >= 0 && j + v - 1 < g.w) m |= 1u << (u * 3 + v);
  return m;
}

struct Run {
  uint8_t* smem;
  ResCtl* ctl;
  uint32_t* status;
  const uint8_t* blob;
  const ResHead* H;
  Geo g;
  int tid, warp, lane;
  int ntiles;
  uint32_t tmem;
  uint32_t gslice;          // slices issued so far (buffer = gslice & 1, use count = gslice >> 1)
  uint32_t gload;           // weight slices requested so far (ring slot = gload % n_wslots), issuing thread only
  int32_t* v;
  const uint32_t* rowinfo;
};

__device__ __forceinline__ uint8_t* buf_of(const Run& r, int which) {
  return r.smem + (which == 0 ? r.H->s_xa : (which == 1 ? r.H->s_x : r.H->s_mid));
}
__device__ __forceinline__ int pitch_of(const Run& r, int which) {
  return which == 0 ? r.H->xa_pitch : (which == 1 ? r.H->x_pitch : r.H->mid_pitch);
}

// All nine taps of all tiles: accumulators D[tile][0 .. n_pad) complete in TMEM on return.
__device__ void conv_mma(Run& r, const ResConv& c) {
  const uint8_t* src = buf_of(r, c.src);
  const int pitch = pitch_of(r, c.src);
  const int nchunks = c.kpad >> 4;
  const uint32_t idesc = ptx::umma_idesc_i8((uint32_t)c.n_pad, c.a_unsigned != 0);
  // Weight slices travel through a ring of n_wslots slots, requested n_wslots - 2 slices ahead of
  // their use so that the L2 latency of the copies is off the slice loop. Slice number `g` of the
  // kernel uses ring slot g % n_wslots; a slot is free once the MMAs of the slice that used it last
  // have completed, which the wait at the top of a slice guarantees for every slice up to g - 2.
  const int nslices = r.ntiles * 9;
  const uint32_t nws = (uint32_t)r.H->n_wslots, ahead = nws - 2u;
  const uint32_t g0 = r.gslice;
  if (r.warp == kResBuilderWarps) {
    // ---- issuing warp: weight copies and MMAs; the builders run one slice ahead of it ----
    if (r.lane == 0) {
      auto request = [&](int sidx) {                // weights of the conv's slice sidx
        const uint32_t slot = r.gload % nws;
        const uint32_t bar = ptx::smem_u32(&r.ctl->w_full[slot]);
        ptx::mbar_expect_tx(bar, c.slice_bytes);
        ptx::bulk_g2s(ptx::smem_u32(r.smem + r.H->s_wring + slot * r.H->w_slot_bytes),
                      r.blob + c.w_off + (size_t)(sidx % 9) * c.slice_bytes, c.slice_bytes, bar);
        ++r.gload;
      };
      // operand descriptors: low words (start address, leading-dimension offset) and their K steps
      const uint32_t lbo_b = (uint32_t)c.n_pad * 16u;
      const uint32_t da_lo[2] = {ptx::umma_desc_lo(ptx::smem_u32(r.smem + r.H->s_abuf[0]), kTileM * 16),
                                 ptx::umma_desc_lo(ptx::smem_u32(r.smem + r.H->s_abuf[1]), kTileM * 16)};
      const uint32_t db_lo0 = ptx::umma_desc_lo(ptx::smem_u32(r.smem + r.H->s_wring), lbo_b);
      const uint32_t db_slot = r.H->w_slot_bytes >> 4;
      const uint32_t da_step = (2u * kTileM * 16u) >> 4, db_step = (2u * lbo_b) >> 4;
      const int ksteps = c.kpad >> 5;
      // every earlier slice has completed (the previous conv ended with a CTA barrier): the ring is free
      for (int sidx = 0; sidx < nslices && sidx < (int)ahead; ++sidx) request(sidx);
      for (int tile = 0; tile < r.ntiles; ++tile)
        for (int tap = 0; tap < 9; ++tap) {
          const uint32_t g = r.gslice++;
          const int b = (int)(g & 1u);
          const uint32_t use = g >> 1;
          const int sidx = (int)(g - g0);
          if (sidx + (int)ahead < nslices) {
            // its ring slot was last read by slice g - 2
            if (use > 0) res_wait_fast(r.ctl, r.status, &r.ctl->slice_done[b], (use - 1u) & 1u);
            request(sidx + (int)ahead);
          }
          res_wait_fast(r.ctl, r.status, &r.ctl->a_full[b], use & 1u);
          const uint32_t wslot = g % nws;
          res_wait_fast(r.ctl, r.status, &r.ctl->w_full[wslot], (g / nws) & 1u);
          ptx::tc_fence_after();
          uint32_t da = da_lo[b], db = db_lo0 + wslot * db_slot;
          const uint32_t d = r.tmem + (uint32_t)(tile * kResMaxWidth);
          ptx::umma_i8_lo(d, da, db, idesc, tap > 0 ? 1u : 0u);
          for (int k = 1; k < ksteps; ++k) {
            da += da_step;
            db += db_step;
            ptx::umma_i8_lo(d, da, db, idesc, 1u);
          }
          ptx::umma_commit(ptx::smem_u32(&r.ctl->slice_done[b]));
        }
    } else {
      r.gslice += (uint32_t)nslices;
    }
    __syncwarp();
    return;
  }
  // ---- builders ----
  // the conv's requantisation constants and index list move to shared memory while the slices run
  // (the previous conv's epilogue, their last reader, ended with a CTA barrier)
  {
    uint4* tab = reinterpret_cast<uint4*>(r.smem + r.H->s_tab);
    const uint4* src_rq = reinterpret_cast<const uint4*>(r.blob + c.rq_off);
    for (int i = r.tid; i < c.n_pad; i += kResThreads) tab[i] = src_rq[i];
    if (c.kind == kResBranch) {
      int32_t* ti = reinterpret_cast<int32_t*>(tab + kResMaxWidth);
      const int32_t* si = reinterpret_cast<const int32_t*>(r.blob + c.idx_off);
      for (int i = r.tid; i < c.n; i += kResThreads) ti[i] = si[i];
    }
  }
  for (int tile = 0; tile < r.ntiles; ++tile) {
    for (int tap = 0; tap < 9; ++tap) {
      const uint32_t g = r.gslice++;
      const int b = (int)(g & 1u);
      const uint32_t use = g >> 1;                      // how often buffer b has been used before
      // the MMAs that last read buffer b must have completed before it is overwritten
      // (suspended wait: the builders run ahead of the issuing thread, and a spinning warp would take
      // issue slots from it)
      if (use > 0 && !ptx::mbar_test_wait(ptx::smem_u32(&r.ctl->slice_done[b]), (use - 1u) & 1u))
        res_wait(r.ctl, r.status, &r.ctl->slice_done[b], (use - 1u) & 1u);
      uint8_t* abuf = r.smem + r.H->s_abuf[b];
      const int off = ((tap * 11) >> 5) - 1;            // u - 1
      const int shift = off * r.g.w + (tap - (off + 1) * 3 - 1);
      for (int it = r.tid; it < kTileM * nchunks; it += kResThreads) {
        const int row = it & (kTileM - 1), ch = it >> 7;
        const int p = tile * kTileM + row;
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if ((r.rowinfo[p] >> tap) & 1u)
          val = *reinterpret_cast<const uint4*>(src + (size_t)(p + shift) * pitch + ch * 16);
        *reinterpret_cast<uint4*>(abuf + (size_t)ch * (kTileM * 16) + row * 16) = val;
      }
      ptx::fence_async_smem();
      __syncwarp();
      if (r.lane == 0)
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(ptx::smem_u32(&r.ctl->a_full[b])) : "memory");
    }
  }
  // the last two slices (one per buffer) close the conv
  const uint32_t g = r.gslice;
  if (g >= 1) res_wait_fast(r.ctl, r.status, &r.ctl->slice_done[(g - 1) & 1u], (((g - 1) >> 1)) & 1u);
  if (g >= 2) res_wait_fast(r.ctl, r.status, &r.ctl->slice_done[(g - 2) & 1u], (((g - 2) >> 1)) & 1u);
  ptx::tc_fence_after();
  asm volatile("bar.sync 1, %0;" ::"n"(kResThreads) : "memory");      // builders only: the staged tables are complete
}

struct StepIo {            // what the epilogue of the last conv / the prior head needs
  const int32_t* colB;     // physical column of x_b's logical channels
  int32_t* mu;             // global: this image's mu and ls planes of the level's block
  int32_t* ls;
  int ls_lo, ls_hi;
  bool subtract;
};

__device__ void conv_epilogue(Run& r, const ResConv& c, const StepIo& io) {
  const OutRq* orq = reinterpret_cast<const OutRq*>(r.smem + r.H->s_tab);          // staged by conv_mma
  const int32_t* idx = reinterpret_cast<const int32_t*>(r.smem + r.H->s_tab + kResMaxWidth * sizeof(OutRq));
  const int q = r.warp & 3, split = r.warp >> 2, nsplit = kResThreads / 128;
  const int nch = c.n_pad >> 4;
  uint8_t* dst = buf_of(r, c.dst);
  const int dpitch = pitch_of(r, c.dst);
  for (int tile = 0; tile < (r.warp < kResBuilderWarps ? r.ntiles : 0); ++tile) {
    const int p = tile * kTileM + q * 32 + r.lane;
    const bool valid = p < r.g.px;
    for (int ch = split; ch < nch; ch += nsplit) {
      uint32_t acc[16];
      __syncwarp();                                   // the tensor-memory load is a whole-warp instruction
      ptx::tmem_ld16(r.tmem + (uint32_t)(tile * kResMaxWidth + ch * 16) + ((uint32_t)(q * 32) << 16), acc);
      ptx::tmem_ld_wait16(acc);
      if (!valid) {
        // rows beyond the image: nothing to store
      } else if (c.kind == kResHidden) {
        uint32_t wd[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint32_t word = 0;
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const int col = ch * 16 + i * 4 + jj;
            const int y = clampi(rq_const((int32_t)acc[i * 4 + jj], orq[col]), 0, 255);
            word |= (uint32_t)y << (8 * jj);
          }
          wd[i] = word;
        }
        *reinterpret_cast<uint4*>(dst + (size_t)p * dpitch + ch * 16) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
      } else {
#pragma unroll 4
        for (int i = 0; i < 16; ++i) {
          const int col = ch * 16 + i;
          if (col >= c.n) continue;
          const int32_t y = rq_const((int32_t)acc[i], orq[col]);
          if (c.kind == kResBranch) {
            uint8_t* xp = dst + (size_t)p * dpitch + idx[col];
            *xp = (uint8_t)clampi((int)*xp + y, 0, 255);
          } else if (c.kind == kResOut) {
            uint32_t* vv = reinterpret_cast<uint32_t*>(&r.v[io.colB[col] * r.g.pg + p]);
            *vv = io.subtract ? (*vv - (uint32_t)y) : (*vv + (uint32_t)y);
          } else {   // kResPrior: first half mu, second half the clipped log-scale index
            const int half = c.n >> 1;
            if (col < half) io.mu[(size_t)col * r.g.px + p] = y;
            else io.ls[(size_t)(col - half) * r.g.px + p] = clampi(y, io.ls_lo, io.ls_hi);
          }
        }
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
}

// network input: logical channels cols[0 .. n) of the flow variable, requantised to int8, pixel-major
__device__ void requant_input(Run& r, const int32_t* cols, int n, int32_t m0, int32_t s) {
  int8_t* xa = reinterpret_cast<int8_t*>(r.smem + r.H->s_xa);
  const int pitch = r.H->xa_pitch;
  for (int it = r.tid; it < (r.warp < kResBuilderWarps ? n * r.g.px : 0); it += kResThreads) {
    const int c = it / r.g.px, p = it - c * r.g.px;
    xa[(size_t)p * pitch + c] = (int8_t)clampi(rq64(r.v[cols[c] * r.g.pg + p], m0, s), -128, 127);
  }
  __syncthreads();
}

template <bool kInv>
__global__ void __launch_bounds__(kResAllThreads, 1) res_level_kernel(const LevelArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ ResCtl ctl;
  const LevelPlan& P = *a.plan;
  const ResHead* H = reinterpret_cast<const ResHead*>(a.blob);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kResMaxWSlots; ++s) ptx::mbar_init(ptx::smem_u32(&ctl.w_full[s]), 1);
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(ptx::smem_u32(&ctl.slice_done[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl.a_full[s]), (uint32_t)kResBuilderWarps);
    }
    ptx::mbar_init_fence();
    ctl.abort = 0;
  }
  if (warp == 0) ptx::tmem_alloc(ptx::smem_u32(&ctl.tmem_base), (uint32_t)H->tmem_cols);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();

  Run r;
  r.smem = smem; r.ctl = &ctl; r.status = a.status; r.blob = a.blob; r.H = H;
  r.g.px = P.px; r.g.h = P.h; r.g.w = P.w; r.g.pg = P.pg; r.g.mul_w = P.mul_w;
  r.tid = tid; r.warp = warp; r.lane = lane;
  r.ntiles = (P.px + kTileM - 1) / kTileM;
  r.tmem = ctl.tmem_base;
  r.gslice = 0;
  r.gload = 0;
  r.v = reinterpret_cast<int32_t*>(smem + H->s_v);
  uint32_t* rowinfo = reinterpret_cast<uint32_t*>(smem + H->s_rowinfo);
  r.rowinfo = rowinfo;

  const int c = P.c, px = P.px, pg = P.pg, w = P.w;
  const int b = blockIdx.x;                       // one image per CTA
  const bool builder = warp < kResBuilderWarps;
  const int per_img = builder ? c * px : 0;       // the issuing warp takes no part in the element loops
  int32_t* v = r.v;
  for (int i = tid; i < (builder ? r.ntiles * kTileM : 0); i += kResThreads) rowinfo[i] = gather_mask(i, r.g);
  // activation buffers start at zero: padding channels and bytes beyond a conv's outputs stay zero
  // or meet zero weights
  for (uint32_t i = H->s_xa + tid * 16; builder && i < H->s_rowinfo; i += kResThreads * 16)
    *reinterpret_cast<uint4*>(smem + i) = make_uint4(0u, 0u, 0u, 0u);

  if (!kInv) {
    const int w2 = 2 * w;
    for (int e = tid; e < per_img; e += kResThreads) {
      const int ci = rdiv(e, P.mul_4px), r2 = e - ci * 4 * px;
      const int y = rdiv(r2, P.mul_w2), x = r2 - y * w2;
      size_t src = (size_t)b * per_img + e;
      if (P.is_first && a.img_w > 0) {
        const int by = rdiv(b, a.mul_patches_x), bx = b - by * a.patches_x;
        src = ((size_t)ci * a.img_h + (size_t)(by * 2 * P.h + y)) * a.img_w + (size_t)(bx * w2 + x);
      }
      const int32_t val = P.is_first ? (int32_t) reinterpret_cast<const uint8_t*>(a.in)[src]
                                     : reinterpret_cast<const int32_t*>(a.in)[src];
      v[(ci * 4 + (y & 1) * 2 + (x & 1)) * pg + (y >> 1) * w + (x >> 1)] = val;
    }
  } else {
    for (int e = tid; e < per_img; e += kResThreads) {
      const int k = rdiv(e, P.mul_px), q = e - k * px;
      if (a.phase == 1 && k >= P.keep_c) continue;
      const int32_t val =
          (k < P.keep_c) ? reinterpret_cast<const int32_t*>(a.in)[(size_t)b * (size_t)a.in_stride + (size_t)k * px + q]
                         : a.z[(size_t)b * P.d + P.z_off + (size_t)(k - P.keep_c) * px + q];
      v[P.col_out[k] * pg + q] = val;
    }
  }
  __syncthreads();

  const ResCouplingRec* cps = reinterpret_cast<const ResCouplingRec*>(a.blob + H->coupling_off);
  const ResConv* convs = reinterpret_cast<const ResConv*>(a.blob + H->conv_off);
  const int n_couplings = (kInv && a.phase == 1) ? 0 : H->n_couplings;
  const bool do_prior = H->prior_conv >= 0 && a.prior != nullptr && !(kInv && a.phase == 2);
  const int nsteps = n_couplings + (do_prior ? 1 : 0);
  for (int step = 0; step < nsteps; ++step) {
    const bool prior = do_prior && (kInv ? step == 0 : step == nsteps - 1);
    StepIo io{};
    io.subtract = kInv;
    if (prior) {
      const ResConv cv = convs[H->prior_conv];
      requant_input(r, P.col_out, P.ca, H->prior_in_m0, H->prior_in_s);
      io.mu = a.prior + (size_t)b * 2u * P.d_fact + P.prior_off;
      io.ls = io.mu + P.d_fact;
      io.ls_lo = H->ls_lo; io.ls_hi = H->ls_hi;
      conv_mma(r, cv);
      conv_epilogue(r, cv, io);
      continue;
    }
    const int ki = kInv ? (n_couplings - 1 - (step - (do_prior ? 1 : 0))) : step;
    const ResCouplingRec cp = cps[ki];
    io.colB = reinterpret_cast<const int32_t*>(a.blob + cp.colB_off);
    requant_input(r, reinterpret_cast<const int32_t*>(a.blob + cp.colA_off), P.ca, cp.in_m0, cp.in_s);
    for (int ci = 0; ci < cp.n_convs; ++ci) {
      const ResConv cv = convs[cp.conv0 + ci];
      conv_mma(r, cv);
      if (cv.kind == kResBranch) {
        // the shortcut Q(x) of all channels, in place (the first conv of the block has read X already)
        uint8_t* X = smem + H->s_x;
        const int words = H->x_pitch >> 2;
        for (int it = tid; it < (builder ? px * words : 0); it += kResThreads) {
          uint32_t* wp = reinterpret_cast<uint32_t*>(X) + it;
          const uint32_t in = *wp;
          uint32_t out = 0;
#pragma unroll
          for (int jj = 0; jj < 4; ++jj)
            out |= (uint32_t)clampi(rq64((int32_t)((in >> (8 * jj)) & 0xFFu), cv.short_m0, cv.short_s), 0, 255) << (8 * jj);
          *wp = out;
        }
        __syncthreads();
      }
      conv_epilogue(r, cv, io);
    }
  }

  if (!kInv) {
    int32_t* keep_out = reinterpret_cast<int32_t*>(a.out);
    for (int e = tid; e < per_img; e += kResThreads) {
      const int k = rdiv(e, P.mul_px), q = e - k * px;
      const int32_t val = v[P.col_out[k] * pg + q];
      if (k >= P.keep_c) a.z[(size_t)b * P.d + P.z_off + (size_t)(k - P.keep_c) * px + q] = val;
      else if (P.is_last) a.z[(size_t)b * P.d + P.z_final_off + (size_t)k * px + q] = val;
      else keep_out[((size_t)b * P.keep_c + k) * (size_t)px + q] = val;
    }
  } else if (a.phase != 1) {
    const int w2 = 2 * w;
    uint32_t bad = 0;
    for (int e = tid; e < per_img; e += kResThreads) {
      const int ci = rdiv(e, P.mul_4px), r2 = e - ci * 4 * px;
      const int y = rdiv(r2, P.mul_w2), x = r2 - y * w2;
      const int32_t val = v[(ci * 4 + (y & 1) * 2 + (x & 1)) * pg + (y >> 1) * w + (x >> 1)];
      size_t dst = (size_t)b * per_img + e;
      if (P.is_first && a.img_w > 0) {
        const int by = rdiv(b, a.mul_patches_x), bx = b - by * a.patches_x;
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

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 0) ptx::tmem_dealloc(ctl.tmem_base, (uint32_t)H->tmem_cols);
}

}  // namespace

cudaError_t launch_res_level(const LevelArgs& args, bool inverse, int grid, uint32_t smem_bytes, cudaStream_t stream) {
  if (inverse) res_level_kernel<true><<<grid, kResAllThreads, smem_bytes, stream>>>(args);
  else res_level_kernel<false><<<grid, kResAllThreads, smem_bytes, stream>>>(args);
  return cudaGetLastError();
}

cudaError_t configure_res_kernels(uint32_t max_smem_bytes) {
  cudaError_t e = cudaFuncSetAttribute(res_level_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)max_smem_bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(res_level_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem_bytes);
}

}  // namespace iodf
