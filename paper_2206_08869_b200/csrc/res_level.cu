// One flow level whose couplings use the paper's residual-block network (Eq. 3, Sec. 4.1; scatter
// add, Sec. 4.5; App. B.1: conv 3x3 -> L blocks of two 3x3 convs -> conv 3x3, all on `hidden`
// channels), one CTA per image of at most 256 pixels at this level; larger images (up to 2048 pixels)
// are cut into row bands, one CTA of a thread-block cluster each (see "Row bands" below), and small
// ones may share a CTA (ResHead::group images, their padded frames one after the other).
//
// Every conv here is a 3x3 conv over hidden activations, so a pixel needs its neighbours' hidden
// values: the activations of the whole image stay in shared memory (xa: the requantised network
// input, X: the block tensor of D channels, MID: the first conv's output; 8-bit). They are stored
// the way tcgen05.mma reads a K-major operand without swizzle, [channel chunk of 16][row][16 bytes],
// with the image laid out in rows of w + 2 positions (a zero column on either side, a zero row
// above and below, and w + 3 guard positions before and after). A conv tap (u, v) is then nothing
// but a row offset (u-1)(w+2) + (v-1) of the operand's start address: no operand is ever built.
//
//   for each tap, for each 128-position tile, for each 32 channels:
//       D[tile] (+)= A(buffer, tile rows shifted by the tap) * W(tap)^T      tcgen05.mma kind::i8
//   epilogue: TMEM -> exact 64-bit requantisation -> what the conv's kind says (see ResKind);
//   results are stored at the image's positions only, so the padding stays zero.
//
// The (h+2)(w+2) positions are computed in full (outputs at padding positions are discarded): a
// third more rows than pixels at 16x16, bought with tensor time that is idle anyway. One lane each
// of three more warps issues the MMAs of a conv back to back (tiles dealt between them, or the taps
// when there is one tile), one lane of a last warp streams the taps' weight
// slices from the packed blob through a ring, running ahead into the next conv; the 16 other warps
// requantise. A block is
//   MID = clip(ReLU(rq(conv_a(X))))                        kResHidden
//   X   = rq(X; M_r, s_r)      for all D channels          the shortcut Q(x), in place
//   X[idx[j]] = clip(max(X[idx[j]] + rq(conv_b(MID))[j], 0), 0, 255)   kResBranch: scatter add + ReLU
// which equals Eq. 3 with the scatter add because rq(X) of an 8-bit X with a multiplier below one
// is again in 0..255, and channels that the second conv does not keep only get the shortcut. The
// scatter itself happens when the level is packed: conv_b's filter j is stored as row idx[j] of a
// D-row weight matrix (zero rows, which requantise to 0, elsewhere), so the kernel's update is a
// plain 16-channel-wide add. The extra rows cost tensor time that is idle; byte-wise scattered
// updates cost shared-memory bank conflicts that were not.
//
// Row bands. A 3x3 conv needs the rows above and below a band. Each CTA of the cluster keeps its band
// in the same padded layout with two more rows: the band's own rows in the middle, the neighbouring
// bands' edge rows (or the zero padding at the image's border) above and below. Whatever writes
// activations (network input, every conv's epilogue) also writes a band's first and last row into
// the neighbours' edge rows through distributed shared memory, and the barrier that separates a
// conv from the next one is then a cluster barrier. The index lists of the level's load and store
// take the band's offset; nothing else changes.
//
// Convs run one after another: a conv's epilogue does not overlap the next conv's MMAs.
#include "res_level.h"
#include "ptx.cuh"

namespace iodf {

namespace {

struct __align__(16) ResCtl {
  uint64_t w_full[kResMaxWSlots];   // bulk copy -> issuer: weight ring slot filled
  uint64_t w_empty[kResMaxWSlots];  // tensor core -> issuer: the MMAs that read ring slot s have completed
  uint64_t conv_done;       // tensor core -> requantising warps: every MMA of the running conv has completed
  uint32_t tmem_base;
  uint32_t abort;
};

// bounded wait of this kernel: see ptx::bounded_wait
__device__ __forceinline__ bool res_wait(ResCtl* ctl, uint32_t* status, uint64_t* bar, uint32_t parity) {
  return ptx::bounded_wait(&ctl->abort, status, bar, parity, kSpinLimit);
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

// ---- thread-block cluster: rank, barrier, stores into a peer CTA's shared memory -------------------
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// every thread of every CTA of the cluster; orders shared-memory writes (local and remote) before it
// with reads after it
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t peer_addr(const void* p, uint32_t rank) {
  uint32_t a;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(ptx::smem_u32(p)), "r"(rank));
  return a;
}
__device__ __forceinline__ void peer_store16(uint32_t addr, const uint4 v) {
  asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void peer_store1(uint32_t addr, uint32_t byte) {
  asm volatile("st.shared::cluster.u8 [%0], %1;" ::"r"(addr), "r"(byte) : "memory");
}

struct Geo {
  int px, h, w, pg;        // the CTA's band: pixels, rows, width, pixel slots
  uint32_t mul_w;
};

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
  uint32_t gslice;          // weight slices consumed so far (ring slot = gslice % n_wslots), issuing lane only
  uint32_t gload;           // weight slices requested so far, loading lane only
  uint32_t nconv;           // convs run so far (parity of conv_done)
  uint32_t prefetched;      // weight slices of the coming conv that were requested already, loading lane only
  int32_t* v;
  const int32_t* pixel_of;  // pixel index (within the band) of a padded position, -1 at padding
  const int32_t* halo_of;   // 0, or where a position is mirrored in a neighbouring band: (its padded position there << 1) | (1: the band below)
  int bands, band;          // row bands of the image (CTAs of the cluster) and this CTA's
  int px_full;              // pixels of the whole image at this level (strides of the global layouts)
  int q0;                   // the band's first pixel
  // several images per CTA (bands = 1): their frames follow one another in the padded layout, their
  // pixels in the flow variable's planes (pixel index = image * px + pixel of the image)
  int nimg, frame, ptot;    // images of this CTA, padded positions per image, pixels of all its images
  uint32_t mul_px;          // magic multiplier of px
  size_t prior_img_stride;  // prior parameters: elements between two images
};

// padded position (0 = first computed position) of pixel p of the CTA (image-major)
__device__ __forceinline__ int position_of(const Run& r, int p) {
  const int g = r.nimg > 1 ? rdiv(p, r.mul_px) : 0, q = p - g * r.g.px;
  const int i = rdiv(q, r.g.mul_w), j = q - i * r.g.w;
  return g * r.frame + (i + 1) * r.H->w2 + (j + 1);
}

// End of a step that wrote activations: they must be visible to the tensor core's reads (this CTA's
// and, for edge rows, the neighbours') before the next conv is issued.
__device__ __forceinline__ void step_barrier(const Run& r) {
  ptx::fence_async_smem();
  ptx::tc_fence_before();
  if (r.bands > 1) {
    cluster_barrier();
    ptx::fence_async_smem();     // what the neighbours wrote here, towards the async proxy
  } else {
    __syncthreads();
  }
}
// the same 16 bytes / byte in the neighbouring band's edge row, if the position is one of this band's edge rows
__device__ __forceinline__ void mirror16(const Run& r, uint8_t* buf, int c, int rr, const uint4 v) {
  const int hrec = r.halo_of[rr];
  if (hrec) peer_store16(peer_addr(buf + ((size_t)(c >> 4) * r.H->rows + r.H->guard + (hrec >> 1)) * 16 + (c & 15),
                                   (uint32_t)(r.band + ((hrec & 1) ? 1 : -1))), v);
}
__device__ __forceinline__ void mirror1(const Run& r, uint8_t* buf, int c, int rr, uint32_t byte) {
  const int hrec = r.halo_of[rr];
  if (hrec) peer_store1(peer_addr(buf + ((size_t)(c >> 4) * r.H->rows + r.H->guard + (hrec >> 1)) * 16 + (c & 15),
                                  (uint32_t)(r.band + ((hrec & 1) ? 1 : -1))), byte);
}


__device__ __forceinline__ uint8_t* buf_of(const Run& r, int which) {
  return r.smem + (which == 0 ? r.H->s_xa : (which == 1 ? r.H->s_x : r.H->s_mid));
}
// byte address of channel c at padded position rr (0 = first computed position) of a buffer
__device__ __forceinline__ uint8_t* at(const Run& r, uint8_t* buf, int c, int rr) {
  return buf + ((size_t)(c >> 4) * r.H->rows + r.H->guard + rr) * 16 + (c & 15);
}

// All nine taps of all tiles: accumulators D[tile][0 .. n_pad) complete in TMEM on return (for the
// requantising warps; the issuing warp returns as soon as everything is issued).
__device__ void conv_mma(Run& r, const ResConv& c, const ResConv* next, const int32_t* colB) {
  const uint32_t parity = r.nconv & 1u;
  ++r.nconv;
  if (r.warp == kResBuilderWarps + kResIssuers) {
    // ---- loading warp: the conv's nine weight slices, then the first ones of the conv that follows.
    // A request blocks while the ring is full (and the copy instruction itself takes hundreds of
    // clocks to issue), which is why it has a lane of its own.
    if (r.lane == 0) {
      const uint32_t nws = (uint32_t)r.H->n_wslots;
      auto request = [&](const ResConv& c, int tap) {
        const uint32_t gl = r.gload++;
        const uint32_t slot = gl % nws, use = gl / nws;
        // the slice that used this slot last must have been consumed
        if (use > 0) res_wait_fast(r.ctl, r.status, &r.ctl->w_empty[slot], (use - 1u) & 1u);
        const uint32_t bar = ptx::smem_u32(&r.ctl->w_full[slot]);
        ptx::mbar_expect_tx(bar, c.slice_bytes);
        ptx::bulk_g2s(ptx::smem_u32(r.smem + r.H->s_wring + slot * r.H->w_slot_bytes),
                      r.blob + c.w_off + (size_t)tap * c.slice_bytes, c.slice_bytes, bar);
      };
      for (int tap = (int)r.prefetched; tap < 9; ++tap) request(c, tap);
      r.prefetched = 0;
      // Slices of the next conv travel while this one is multiplied and requantised. Never more than
      // the ring holds: their slots are freed by this conv's MMAs, which all complete before the CTA
      // barrier that this warp, too, has to reach.
      if (next) {
        const int npre = (int)(nws < 9u ? nws : 9u);
        for (int tap = 0; tap < npre; ++tap) request(*next, tap);
        r.prefetched = (uint32_t)npre;
      }
    }
    __syncwarp();
    return;
  }
  if (r.warp >= kResBuilderWarps) {
    // ---- issuing warps: the conv's MMAs, tap by tap as the weight slices land; issuer i takes the
    // tiles i, i + kResIssuers, ... (accumulators are per tile, so the issuers are independent; an MMA
    // costs its issuing lane ~100 clocks, the tensor core much less)
    const int me = r.warp - kResBuilderWarps;
    if (r.lane == 0) {
      const uint32_t nws = (uint32_t)r.H->n_wslots;
      const uint32_t idesc = ptx::umma_idesc_i8((uint32_t)c.n_pad, c.a_unsigned != 0);
      const uint32_t rows = (uint32_t)r.H->rows;
      // operand start addresses in 16-byte units
      const uint32_t a0 = (ptx::smem_u32(buf_of(r, c.src)) >> 4) + (uint32_t)r.H->guard;
      const uint32_t ring0 = ptx::smem_u32(r.smem + r.H->s_wring) >> 4, slot16 = r.H->w_slot_bytes >> 4;
      const uint32_t a_hi = (rows & 0x3FFFu) << 16, b_hi = ((uint32_t)c.n_pad & 0x3FFFu) << 16;
      const int ksteps = c.kpad >> 5;
      ptx::tc_fence_after();
      for (int tap = 0; tap < 9; ++tap) {
        const uint32_t g = r.gslice++;
        const uint32_t slot = g % nws;
        // one tile: the taps are dealt between the issuers, and a tap's slice is waited for and
        // released by its issuer alone (w_empty then counts one arrival)
        if (r.ntiles == 1 && tap % kResIssuers != me) continue;
        res_wait_fast(r.ctl, r.status, &r.ctl->w_full[slot], (g / nws) & 1u);
        ptx::tc_fence_after();
        const int u = (tap * 11) >> 5;
        const int shift = (u - 1) * r.H->w2 + (tap - u * 3 - 1);
        if (r.ntiles == 1) {
          // each issuer accumulates a partial sum over its taps in its own TMEM columns (integer
          // partial sums add up exactly in the epilogue)
          const uint32_t d = r.tmem + (uint32_t)(me * kResMaxWidth);
          uint32_t sa = a0 + (uint32_t)shift;
          uint32_t sb = ring0 + slot * slot16;
          for (int k = 0; k < ksteps; ++k) {
            ptx::umma_i8_lo(d, (sa & 0x3FFFu) | a_hi, (sb & 0x3FFFu) | b_hi, idesc, (tap >= kResIssuers || k > 0) ? 1u : 0u);
            sa += 2u * rows;
            sb += 2u * (uint32_t)c.n_pad;
          }
        } else {
          for (int tile = me; tile < r.ntiles; tile += kResIssuers) {
            const uint32_t d = r.tmem + (uint32_t)(tile * kResMaxWidth);
            uint32_t sa = a0 + (uint32_t)(tile * kTileM + shift);
            uint32_t sb = ring0 + slot * slot16;
            for (int k = 0; k < ksteps; ++k) {
              ptx::umma_i8_lo(d, (sa & 0x3FFFu) | a_hi, (sb & 0x3FFFu) | b_hi, idesc, (tap > 0 || k > 0) ? 1u : 0u);
              sa += 2u * rows;
              sb += 2u * (uint32_t)c.n_pad;
            }
          }
        }
        ptx::umma_commit(ptx::smem_u32(&r.ctl->w_empty[slot]));
      }
      ptx::umma_commit(ptx::smem_u32(&r.ctl->conv_done));
    }
    __syncwarp();
    return;
  }
  // requantising warps: the conv's constants and index list move to shared memory meanwhile (the
  // previous conv's epilogue, their last reader, ended with a CTA barrier)
  {
    uint4* tab = reinterpret_cast<uint4*>(r.smem + r.H->s_tab);
    const uint4* src_rq = reinterpret_cast<const uint4*>(r.blob + c.rq_off);
    for (int i = r.tid; i < c.n_pad; i += kResThreads) tab[i] = src_rq[i];
    if (c.kind == kResBranch) {
      // the block's shortcut rq(x; M_r, s_r) as a table over the 256 values of an 8-bit x
      uint8_t* lut = r.smem + r.H->s_tab + kResMaxWidth * (sizeof(OutRq) + sizeof(int32_t));
      if (r.tid < 256) lut[r.tid] = (uint8_t)clampi(rq64(r.tid, c.short_m0, c.short_s), 0, 255);
    } else if (c.kind == kResOut) {
      // the physical columns of x_b's channels, in place of the index list
      int32_t* ti = reinterpret_cast<int32_t*>(tab + kResMaxWidth);
      for (int i = r.tid; i < c.n; i += kResThreads) ti[i] = colB[i];
    }
  }
  asm volatile("bar.sync 1, %0;" ::"n"(kResThreads) : "memory");      // requantising warps: the staged tables are complete
  if (c.kind == kResBranch) {
    // The shortcut Q(x) of all channels, in place, at the image's positions, while the second conv is
    // being multiplied: its MMAs read MID, and the block's first conv has read X already.
    uint8_t* X = r.smem + r.H->s_x;
    const uint8_t* lut = r.smem + r.H->s_tab + kResMaxWidth * (sizeof(OutRq) + sizeof(int32_t));
    const int chunks = r.H->x_pitch >> 4, px = r.ptot;
    for (int it = r.tid; it < chunks * px; it += kResThreads) {
      const int ch = it / px, p = it - ch * px;
      const int rr = position_of(r, p);
      uint4* wp = reinterpret_cast<uint4*>(at(r, X, ch * 16, rr));
      uint4 val = *wp;
      uint32_t* wv = reinterpret_cast<uint32_t*>(&val);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t in = wv[k];
        uint32_t out = 0;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) out |= (uint32_t)lut[(in >> (8 * jj)) & 0xFFu] << (8 * jj);
        wv[k] = out;
      }
      *wp = val;
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kResThreads) : "memory");    // before the epilogue adds to X
  }
  if (!ptx::mbar_test_wait(ptx::smem_u32(&r.ctl->conv_done), parity))
    res_wait(r.ctl, r.status, &r.ctl->conv_done, parity);
  ptx::tc_fence_after();
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
  for (int tile = 0; tile < (r.warp < kResBuilderWarps ? r.ntiles : 0); ++tile) {
    const int rr = tile * kTileM + q * 32 + r.lane;       // padded position of this thread's row
    const int p = r.pixel_of[rr];                          // its pixel, or -1 at a padding position
    const bool valid = p >= 0;
    for (int ch = split; ch < nch; ch += nsplit) {
      uint32_t acc[16];
      __syncwarp();                                   // the tensor-memory load is a whole-warp instruction
      ptx::tmem_ld16(r.tmem + (uint32_t)(tile * kResMaxWidth + ch * 16) + ((uint32_t)(q * 32) << 16), acc);
      ptx::tmem_ld_wait16(acc);
      if (r.ntiles == 1) {                            // the issuers' partial sums over their taps
#pragma unroll
        for (int part = 1; part < kResIssuers; ++part) {
          uint32_t more[16];
          ptx::tmem_ld16(r.tmem + (uint32_t)(part * kResMaxWidth + ch * 16) + ((uint32_t)(q * 32) << 16), more);
          ptx::tmem_ld_wait16(more);
#pragma unroll
          for (int i = 0; i < 16; ++i) acc[i] += more[i];
        }
      }
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
        const uint4 val = make_uint4(wd[0], wd[1], wd[2], wd[3]);
        *reinterpret_cast<uint4*>(at(r, dst, ch * 16, rr)) = val;
        if (r.bands > 1) mirror16(r, dst, ch * 16, rr, val);
      } else if (c.kind == kResBranch) {
        // The conv's outputs sit at their channels of X already (the scatter add was done on the
        // weights, when the level was packed; a channel without a filter requantises 0 to 0), so the
        // update is sixteen adjacent bytes: one 16-byte read of the shortcut, one 16-byte write.
        uint4* xp = reinterpret_cast<uint4*>(at(r, dst, ch * 16, rr));
        const uint4 xv = *xp;
        const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
        uint32_t wd[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint32_t word = 0;
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const int col = ch * 16 + i * 4 + jj;
            // the branch value is clipped to +-255 first: the sum then stays far inside 32 bits for
            // any requantisation constants, and the clip to 0..255 below gives the same result
            const int br = clampi(rq_const((int32_t)acc[i * 4 + jj], orq[col]), -255, 255);
            const int y = clampi((int)((xw[i] >> (8 * jj)) & 0xFFu) + br, 0, 255);
            word |= (uint32_t)y << (8 * jj);
          }
          wd[i] = word;
        }
        const uint4 val = make_uint4(wd[0], wd[1], wd[2], wd[3]);
        *xp = val;
        if (r.bands > 1) mirror16(r, dst, ch * 16, rr, val);
      } else {
#pragma unroll 4
        for (int i = 0; i < 16; ++i) {
          const int col = ch * 16 + i;
          if (col >= c.n) continue;
          const int32_t y = rq_const((int32_t)acc[i], orq[col]);
          if (c.kind == kResOut) {
            uint32_t* vv = reinterpret_cast<uint32_t*>(&r.v[idx[col] * r.g.pg + p]);       // idx: staged columns of x_b
            *vv = io.subtract ? (*vv - (uint32_t)y) : (*vv + (uint32_t)y);
          } else {   // kResPrior: first half mu, second half the clipped log-scale index
            const int half = c.n >> 1;
            const int g = r.nimg > 1 ? rdiv(p, r.mul_px) : 0;          // image of the CTA, pixel of the image
            const size_t at_px = (size_t)g * r.prior_img_stride + (size_t)(p - g * r.g.px);
            if (col < half) io.mu[(size_t)col * r.px_full + at_px] = y;
            else io.ls[(size_t)(col - half) * r.px_full + at_px] = clampi(y, io.ls_lo, io.ls_hi);
          }
        }
      }
    }
  }
  step_barrier(r);               // the next conv's MMAs read what was stored here
}

// network input: logical channels cols[0 .. n) of the flow variable, requantised to int8, at the
// image's positions of the padded layout
__device__ void requant_input(Run& r, const int32_t* cols, int n, int32_t m0, int32_t s) {
  uint8_t* xa = r.smem + r.H->s_xa;
  for (int it = r.tid; it < (r.warp < kResBuilderWarps ? n * r.ptot : 0); it += kResThreads) {
    const int c = it / r.ptot, p = it - c * r.ptot;
    const int rr = position_of(r, p);
    const uint32_t byte = (uint32_t)(uint8_t)(int8_t)clampi(rq64(r.v[cols[c] * r.g.pg + p], m0, s), -128, 127);
    *at(r, xa, c, rr) = (uint8_t)byte;
    if (r.bands > 1) mirror1(r, xa, c, rr, byte);
  }
  step_barrier(r);
}

template <bool kInv>
__global__ void __launch_bounds__(kResAllThreads, 1) res_level_kernel(const LevelArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ ResCtl ctl;
  const LevelPlan& P = *a.plan;
  const ResHead* H = reinterpret_cast<const ResHead*>(a.blob);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kResMaxWSlots; ++s) {
      ptx::mbar_init(ptx::smem_u32(&ctl.w_full[s]), 1);
      // a slot is released by every issuer that read it: all of them, or the tap's one at single-tile levels
      ptx::mbar_init(ptx::smem_u32(&ctl.w_empty[s]), H->ntiles == 1 ? 1u : (uint32_t)kResIssuers);
    }
    ptx::mbar_init(ptx::smem_u32(&ctl.conv_done), (uint32_t)kResIssuers);
    ptx::mbar_init_fence();
    ctl.abort = 0;
  }
  if (warp == 0) ptx::tmem_alloc(ptx::smem_u32(&ctl.tmem_base), (uint32_t)H->tmem_cols);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();

  // one CTA per image, or per band of rows of an image (the CTAs of a cluster)
  const int bands = H->bands, hb = H->hb;
  const int band = bands > 1 ? (int)cluster_rank() : 0;
  const int group = bands > 1 ? 1 : H->group;     // images per CTA
  const int b = (blockIdx.x / bands) * group;     // (first) image
  const int nimg = min(group, a.batch - b);
  const int w = P.w, pg = P.pg, c = P.c;
  const int pxb = hb * w;                         // pixels of the band (of an image)
  const int q0 = band * pxb;                      // the band's first pixel in the image
  const int frame = (hb + 2) * H->w2;             // padded positions of an image

  Run r;
  r.smem = smem; r.ctl = &ctl; r.status = a.status; r.blob = a.blob; r.H = H;
  r.g.px = pxb; r.g.h = hb; r.g.w = w; r.g.pg = pg; r.g.mul_w = P.mul_w;
  r.tid = tid; r.warp = warp; r.lane = lane;
  r.ntiles = H->ntiles;
  r.tmem = ctl.tmem_base;
  r.gslice = 0;
  r.gload = 0;
  r.nconv = 0;
  r.prefetched = 0;
  r.v = reinterpret_cast<int32_t*>(smem + H->s_v);
  int32_t* pixel_of = reinterpret_cast<int32_t*>(smem + H->s_rowinfo);
  int32_t* halo_of = pixel_of + r.ntiles * kTileM;
  r.pixel_of = pixel_of;
  r.halo_of = halo_of;
  r.bands = bands; r.band = band; r.px_full = P.px; r.q0 = q0;
  r.nimg = nimg; r.frame = frame; r.ptot = nimg * pxb; r.mul_px = P.mul_px;
  r.prior_img_stride = (size_t)2 * P.d_fact;

  const bool builder = warp < kResBuilderWarps;
  const int per_band = c * pxb;                   // elements of an image's band
  const int n_el = builder ? nimg * per_band : 0; // the issuing warps take no part in the element loops
  int32_t* v = r.v;
  for (int rr = tid; rr < (builder ? r.ntiles * kTileM : 0); rr += kResThreads) {
    const int g = rr / frame, r0 = rr - g * frame;         // image of the CTA, position in its frame
    const int i = r0 / H->w2, j = r0 - i * H->w2;          // position (i, j) of the (hb+2) x (w+2) frame
    const bool own = g < nimg && i >= 1 && i <= hb && j >= 1 && j <= w;
    pixel_of[rr] = own ? g * pxb + (i - 1) * w + (j - 1) : -1;
    // the band's first row is the row below the band above's last one, and the other way round
    int hrec = 0;
    if (own && i == 1 && band > 0) hrec = ((rr + hb * H->w2) << 1) | 0;
    if (own && i == hb && band + 1 < bands) hrec = ((rr - hb * H->w2) << 1) | 1;
    halo_of[rr] = hrec;
  }
  // activation buffers start at zero: padding channels and bytes beyond a conv's outputs stay zero
  // or meet zero weights
  for (uint32_t i = H->s_xa + tid * 16; builder && i < H->s_rowinfo; i += kResThreads * 16)
    *reinterpret_cast<uint4*>(smem + i) = make_uint4(0u, 0u, 0u, 0u);

  // the level's input: pre-squeeze rows 2 * band * hb .. of [c/4][2h][2w] (encode), or the band's pixels
  // of the kept channels and of z's block (decode)
  const int px = P.px;
  if (!kInv) {
    const int w2 = 2 * w, rows2 = 2 * hb;
    for (int e0 = tid; e0 < n_el; e0 += kResThreads) {
      const int g = e0 / per_band, e = e0 - g * per_band, bi = b + g;      // image of the CTA, element of the image
      const int ci = e / (rows2 * w2), r2 = e - ci * rows2 * w2;
      const int y = r2 / w2, x = r2 - y * w2;
      const int gy = 2 * band * hb + y;                    // row of the whole pre-squeeze image
      size_t src = ((size_t)bi * (c / 4) + ci) * (size_t)(4 * px) + (size_t)gy * w2 + x;
      if (P.is_first && a.img_w > 0) {
        const int by = rdiv(bi, a.mul_patches_x), bx = bi - by * a.patches_x;
        src = ((size_t)ci * a.img_h + (size_t)(by * 2 * P.h + gy)) * a.img_w + (size_t)(bx * w2 + x);
      }
      const int32_t val = P.is_first ? (int32_t) reinterpret_cast<const uint8_t*>(a.in)[src]
                                     : reinterpret_cast<const int32_t*>(a.in)[src];
      v[(ci * 4 + (y & 1) * 2 + (x & 1)) * pg + g * pxb + (y >> 1) * w + (x >> 1)] = val;
    }
  } else {
    for (int e0 = tid; e0 < n_el; e0 += kResThreads) {
      const int g = e0 / per_band, e = e0 - g * per_band, bi = b + g;
      const int k = e / pxb, q = e - k * pxb;
      if (a.phase == 1 && k >= P.keep_c) continue;
      const int32_t val =
          (k < P.keep_c) ? reinterpret_cast<const int32_t*>(a.in)[(size_t)bi * (size_t)a.in_stride + (size_t)k * px + q0 + q]
                         : a.z[(size_t)bi * P.d + P.z_off + (size_t)(k - P.keep_c) * px + q0 + q];
      v[P.col_out[k] * pg + g * pxb + q] = val;
    }
  }
  // nobody writes into a neighbour's edge rows before that neighbour has cleared its buffers
  if (bands > 1) cluster_barrier(); else __syncthreads();

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
      io.mu = a.prior + (size_t)b * 2u * P.d_fact + P.prior_off + q0;
      io.ls = io.mu + P.d_fact;
      io.ls_lo = H->ls_lo; io.ls_hi = H->ls_hi;
      conv_mma(r, cv, nullptr, nullptr);
      conv_epilogue(r, cv, io);
      continue;
    }
    const int ki = kInv ? (n_couplings - 1 - (step - (do_prior ? 1 : 0))) : step;
    const ResCouplingRec cp = cps[ki];
    io.colB = reinterpret_cast<const int32_t*>(a.blob + cp.colB_off);
    requant_input(r, reinterpret_cast<const int32_t*>(a.blob + cp.colA_off), P.ca, cp.in_m0, cp.in_s);
    for (int ci = 0; ci < cp.n_convs; ++ci) {
      const ResConv cv = convs[cp.conv0 + ci];
      const bool has_next = ci + 1 < cp.n_convs;
      const ResConv nx = convs[cp.conv0 + (has_next ? ci + 1 : ci)];
      conv_mma(r, cv, has_next ? &nx : nullptr, io.colB);
      conv_epilogue(r, cv, io);
    }
  }

  if (!kInv) {
    int32_t* keep_out = reinterpret_cast<int32_t*>(a.out);
    for (int e0 = tid; e0 < n_el; e0 += kResThreads) {
      const int g = e0 / per_band, e = e0 - g * per_band, bi = b + g;
      const int k = e / pxb, q = e - k * pxb;
      const int32_t val = v[P.col_out[k] * pg + g * pxb + q];
      if (k >= P.keep_c) a.z[(size_t)bi * P.d + P.z_off + (size_t)(k - P.keep_c) * px + q0 + q] = val;
      else if (P.is_last) a.z[(size_t)bi * P.d + P.z_final_off + (size_t)k * px + q0 + q] = val;
      else keep_out[((size_t)bi * P.keep_c + k) * (size_t)px + q0 + q] = val;
    }
  } else if (a.phase != 1) {
    const int w2 = 2 * w, rows2 = 2 * hb;
    uint32_t bad = 0;
    for (int e0 = tid; e0 < n_el; e0 += kResThreads) {
      const int g = e0 / per_band, e = e0 - g * per_band, bi = b + g;
      const int ci = e / (rows2 * w2), r2 = e - ci * rows2 * w2;
      const int y = r2 / w2, x = r2 - y * w2;
      const int gy = 2 * band * hb + y;
      const int32_t val = v[(ci * 4 + (y & 1) * 2 + (x & 1)) * pg + g * pxb + (y >> 1) * w + (x >> 1)];
      size_t dst = ((size_t)bi * (c / 4) + ci) * (size_t)(4 * px) + (size_t)gy * w2 + x;
      if (P.is_first && a.img_w > 0) {
        const int by = rdiv(bi, a.mul_patches_x), bx = bi - by * a.patches_x;
        dst = ((size_t)ci * a.img_h + (size_t)(by * 2 * P.h + gy)) * a.img_w + (size_t)(bx * w2 + x);
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

cudaError_t launch_res_level(const LevelArgs& args, bool inverse, int images, int bands, uint32_t smem_bytes,
                             cudaStream_t stream) {
  // one CTA per image, or a cluster of `bands` CTAs per image
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(images * bands));
  cfg.blockDim = dim3((unsigned)kResAllThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)bands;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = bands > 1 ? 1 : 0;
  if (inverse) return cudaLaunchKernelEx(&cfg, res_level_kernel<true>, args);
  return cudaLaunchKernelEx(&cfg, res_level_kernel<false>, args);
}

cudaError_t configure_res_kernels(uint32_t max_smem_bytes) {
  cudaError_t e = cudaFuncSetAttribute(res_level_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)max_smem_bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(res_level_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem_bytes);
}

}  // namespace iodf
