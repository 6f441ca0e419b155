// One flow level of several 128-pixel tiles per CTA, with the work of a tile split by role.
//
// The arithmetic is that of level_kernel.cu (Eq. 2 with the three-conv network: im2col -> GEMM ->
// requantise -> GEMM -> requantise -> GEMM to per-tap partials -> shifted sum; pixel pass between
// couplings), and so are the two tile slots whose phases alternate. What differs is who does what:
//
//   16 requantising warps   R(slot) -> int8 operand of the slot's next GEMM, both hidden layers,
//                           alternating between the slots: epi1(A) epi1(B) epi2(A) epi2(B) ...
//   4 auxiliary warps       shifted sum of a tile's per-tap partials, then im2col of the tile
//                           after next into the same slot
//   3 control warps         one per GEMM of the chain: lane 0 waits (suspended by the hardware) for
//                           the slot's operand and for the accumulator region to be free, issues the
//                           K steps and commits them; it also keeps its weight slot filled
//
// In level_kernel.cu all sixteen workers build, requantise and sum, one phase at a time, and one
// thread issues every MMA; a tile phase there is a few hundred instructions per warp between
// latencies (barrier wake-up, tensor-memory load, MMA issue and completion) that nothing hides.
// Here the requantising warps, which are bound by the integer pipe, run one epilogue after the
// other: the im2col, the shifted sum and the three MMA round trips of a slot all happen while they
// requantise the other slot. Where the level's widths allow it (2 x widest hidden layer + 2 x nine
// taps x padded C/2 <= 512 columns) the per-tap partials have tensor-memory columns of their own, so
// that a slot's next tile does not wait for its shifted sum.
//
// All hand-overs are mbarriers, one per slot and kind, whose phases advance once per tile of the
// slot; a waiter never lags or leads a barrier by more than one phase (the next phase of a barrier
// needs a hand-over that the waiter itself produces, and every step ends with a CTA barrier after
// all of its MMAs have completed and all its sums have been added).
//
// Taken only for levels the host marks (LevelPlan::pipe): several tiles per CTA, all weight matrices
// resident, both hidden layers in the folded requantisation flavour with the 0..127 clip.
// Everything else runs in level_kernel.cu.
#include "level_device.cuh"
#include "level_pipe.h"

namespace iodf {

namespace {

constexpr int kEpiWarps = 16;                                  // four per lane quarter
constexpr int kAuxWarps = 4;                                   // one per lane quarter
constexpr int kPipeWorkerWarps = kEpiWarps + kAuxWarps;        // 20
constexpr int kPipeWorkers = kPipeWorkerWarps * 32;            // 640
static_assert(kPipeWorkers + 3 * 32 == kPipeThreads, "workers + one control warp per GEMM of the chain");

struct __align__(16) PipeCtl {
  uint64_t a1_full[2];    // aux warps -> control 0: the slot's im2col operand is built      (count kAuxWarps)
  uint64_t a2_full[2];    // requantising warps -> control 1: A2 written, first accumulator drained (count kEpiWarps)
  uint64_t a3_full[2];    // requantising warps -> control 2: A3 written, second accumulator drained
  uint64_t r3_free[2];    // aux warps -> control: the slot's per-tap partials have been summed (count kAuxWarps)
  uint64_t d_full[3][2];  // tensor core -> workers: accumulator of GEMM g of the slot's tile complete
  uint64_t w_full[3];     // bulk copy -> control g: weight slot g filled
  uint64_t meta_full[2];  // bulk copy -> everyone: meta block of step (i & 1) has landed
  uint32_t tmem_base;
  uint32_t abort;
};

struct Pipe {
  uint8_t* smem;
  PipeCtl* ctl;
  uint32_t* status;
  int tid, warp, lane;
};

__device__ __forceinline__ bool pipe_wait(const Pipe& pp, uint64_t* bar, uint32_t parity) {
  const uint32_t b = ptx::smem_u32(bar);
  if (ptx::mbar_test_wait(b, parity) || ptx::mbar_try_wait(b, parity)) return true;
  return ptx::bounded_wait(&pp.ctl->abort, pp.status, bar, parity, kSpinLimit);
}

// this warp's writes to an operand buffer (generic proxy) and its tensor-memory reads are done
__device__ __forceinline__ void pipe_arrive(const Pipe& pp, uint64_t* bar, bool wrote_operand) {
  ptx::tc_fence_before();
  if (wrote_operand) ptx::fence_async_smem();
  __syncwarp();
  if (pp.lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(ptx::smem_u32(bar)) : "memory");
}

// Tiles of a step go to the slots in turn (tile t: slot t & 1, the slot's (t >> 1)-th tile of the
// step). A barrier of slot s has completed `base[s]` phases before the step, so the phase that
// belongs to tile t has the parity below.
struct SlotCount {
  uint32_t all[2];   // tiles the slot has seen in all steps so far (a1_full, a2_full, first accumulator)
  uint32_t cpl[2];   // tiles of coupling steps only (a3_full, r3_free, second and third accumulator)
  __device__ __forceinline__ void advance(int ntv, bool prior) {
    const uint32_t n0 = (uint32_t)((ntv + 1) >> 1), n1 = (uint32_t)(ntv >> 1);
    all[0] += n0; all[1] += n1;
    if (!prior) { cpl[0] += n0; cpl[1] += n1; }
  }
};

// Columns [c0, c0 + m) of a tile's accumulator (this thread's row) -> requantised bytes of the next
// operand's row: y = clip(hi32(acc * m0 + 2^(30+s)) >> (s-1), 0, 127), the bias being part of the
// accumulator (folded flavour). c0 and m are multiples of 8. A tensor-memory load takes a few hundred
// clocks from issue to use and tcgen05.wait::ld waits for every load in flight, so the loop is
// pipelined by hand: the load of piece k+1 is issued right after the wait for piece k and travels
// while piece k is requantised; only the first load of a phase is exposed.
__device__ __forceinline__ void epilogue_lean(uint32_t taddr, int c0, int m, const int32_t* __restrict__ m0tab, int sh,
                                              long long rnd64, uint8_t* __restrict__ out_row) {
  const Requant<kModeFolded, kClipS8Relu> q{nullptr, reinterpret_cast<const int2*>(m0tab), 0, 127, sh, rnd64};
  const bool aligned = (c0 & 15) == 0;
  auto store16 = [&](int col, const uint4 v) {
    uint8_t* d = out_row + (size_t)(col >> 4) * (kTileM * 16);
    if (aligned) {
      *reinterpret_cast<uint4*>(d) = v;
    } else {       // the piece starts in the middle of a 16-byte chunk
      *reinterpret_cast<uint2*>(d + 8) = make_uint2(v.x, v.y);
      *reinterpret_cast<uint2*>(d + kTileM * 16) = make_uint2(v.z, v.w);
    }
  };
  const int np = m >> 4;
  uint32_t ra[16], rb[16];
  if (np > 0) {
    ptx::tmem_ld16(taddr + (uint32_t)c0, ra);
    for (int k = 0; k < np; k += 2) {
      const int col = c0 + (k << 4);
      ptx::tmem_ld_wait();
      if (k + 1 < np) ptx::tmem_ld16(taddr + (uint32_t)(col + 16), rb);
      store16(col, q.chunk(ra, col));
      if (k + 1 >= np) break;
      ptx::tmem_ld_wait();
      if (k + 2 < np) ptx::tmem_ld16(taddr + (uint32_t)(col + 32), ra);
      store16(col + 16, q.chunk(rb, col + 16));
    }
  }
  if (m & 8) {
    const int col = c0 + (np << 4);
    uint32_t r8[8];
    ptx::tmem_ld8(taddr + (uint32_t)col, r8);
    ptx::tmem_ld_wait();
    *reinterpret_cast<uint2*>(out_row + (size_t)(col >> 4) * (kTileM * 16) + (col & 15)) =
        make_uint2(q.quad(r8, col), q.quad(r8 + 4, col + 4));
  }
}

// Shifted sum of one tile's per-tap partial products (R3) into the translation accumulator, by
// direct reductions: the partial product of pixel p and tap (du, dv) belongs to output pixel
// p - (du-1) w - (dv-1) and is added there with one shared-memory reduction per (tap, channel),
// skipped when the tap's bit of the row's scatter mask is clear (target outside the image: zero
// padding). kCb = C/2 (8-column granules per tap: ceil(kCb / 8)); kPlane = bytes between channel
// planes of the accumulator, so that a channel's address is a compile-time offset inside the
// instruction and the loop has next to no integer arithmetic of its own (the requantising warps
// saturate the integer pipe).
template <int kPlane, int kCb>
__device__ __forceinline__ void scatter_lean(uint32_t taddr, int32_t* __restrict__ acc, int w, const RowPos rp) {
  constexpr int kGpt = (kCb + 7) / 8;
  const uint32_t sm = rp.valid ? rp.smask : 0u;
  const uint32_t base = ptx::smem_u32(acc + rp.p);
#pragma unroll
  for (int du = 0; du < 3; ++du) {
#pragma unroll
    for (int gq = 0; gq < kGpt; ++gq) {
      uint32_t r[3][8];
#pragma unroll
      for (int dv = 0; dv < 3; ++dv) ptx::tmem_ld8(taddr + (uint32_t)(((du * 3 + dv) * kGpt + gq) << 3), r[dv]);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int dv = 0; dv < 3; ++dv) {
        if ((sm >> (du * 3 + dv)) & 1u) {
          const uint32_t dst = base - (uint32_t)(((du - 1) * w + (dv - 1)) * 4) + (uint32_t)(gq * 8 * kPlane);
          if (gq * 8 + 0 < kCb) ptx::red_add_s32_at<0 * kPlane>(dst, (int)r[dv][0]);
          if (gq * 8 + 1 < kCb) ptx::red_add_s32_at<1 * kPlane>(dst, (int)r[dv][1]);
          if (gq * 8 + 2 < kCb) ptx::red_add_s32_at<2 * kPlane>(dst, (int)r[dv][2]);
          if (gq * 8 + 3 < kCb) ptx::red_add_s32_at<3 * kPlane>(dst, (int)r[dv][3]);
          if (gq * 8 + 4 < kCb) ptx::red_add_s32_at<4 * kPlane>(dst, (int)r[dv][4]);
          if (gq * 8 + 5 < kCb) ptx::red_add_s32_at<5 * kPlane>(dst, (int)r[dv][5]);
          if (gq * 8 + 6 < kCb) ptx::red_add_s32_at<6 * kPlane>(dst, (int)r[dv][6]);
          if (gq * 8 + 7 < kCb) ptx::red_add_s32_at<7 * kPlane>(dst, (int)r[dv][7]);
        }
      }
    }
  }
}

// ---- control warps -------------------------------------------------------------------------------
// Control warp g issues GEMM g of every tile, in tile order, and keeps weight slot g filled (g = 0
// also brings in the meta blocks). All waits are blocking, so a control warp takes no issue slots
// while it has nothing to do.
__device__ void pipe_control(const Pipe& pp, const LevelPlan& P, const LevelArgs& a, const Steps& st, int ntv, int sg) {
  uint8_t* smem = pp.smem;
  PipeCtl* ctl = pp.ctl;
  const bool lead = pp.lane == 0;
  Ctx cx{};                      // for the shared copy helper
  cx.smem = smem;
  int held = -1;                 // step whose matrix the weight slot holds or is receiving
  // the slot's next matrix, once the step `done` has finished with the slot
  auto refill = [&](int done) {
    if (held > done) return;
    int j = held + 1;
    while (j < st.nsteps && !slot_used_by(st, sg, j)) ++j;
    held = st.nsteps;
    if (j >= st.nsteps) return;
    const BlockRef& br = step_ref(P, st, j);
    bulk_load(cx, a.blob, br.w_off[sg], br.w_bytes[sg], P.s_w[sg], &ctl->w_full[sg]);
    held = j;
  };
  uint64_t* const a_full = sg == 0 ? ctl->a1_full : (sg == 1 ? ctl->a2_full : ctl->a3_full);
  const bool r3_separate = P.r_col[1] != 0;
  SlotCount sc{{0u, 0u}, {0u, 0u}};

  if (lead) {
    if (sg == 0)
      for (int i = 0; i < st.nsteps && i < 2; ++i) {
        const BlockRef& br = step_ref(P, st, i);
        bulk_load(cx, a.blob, br.meta_off, br.meta_bytes, P.s_meta[i], &ctl->meta_full[i]);
      }
    refill(-1);
  }
  __syncwarp();
  __syncthreads();                       // the workers have loaded the flow variable

  const uint32_t tmem = ctl->tmem_base;
  for (int i = 0; i < st.nsteps; ++i) {
    const bool prior = st.is_prior(i);
    const bool active = sg == 0 || !prior;       // the prior head is one GEMM: control 0 only
    int n = 0, kd = 0;
    if (lead && active) {
      pipe_wait(pp, &ctl->meta_full[i & 1], (uint32_t)((i >> 1) & 1));
      const uint8_t* mb = smem + P.s_meta[i & 1];
      if (prior) {
        const PriorMeta* M = reinterpret_cast<const PriorMeta*>(mb);
        n = M->n; kd = M->kd;
      } else {
        const CouplingMeta* M = reinterpret_cast<const CouplingMeta*>(mb);
        n = sg == 0 ? M->n1 : (sg == 1 ? M->n2 : M->n3);
        kd = sg == 0 ? M->kd1 : (sg == 1 ? M->kd2 : M->kd3);
      }
    }
    __syncthreads();     // the workers have finished the pixel pass: step i-1's meta slot is free
    if (lead) {
      if (sg == 0 && i >= 1 && i + 1 < st.nsteps) {
        const BlockRef& br = step_ref(P, st, i + 1);
        bulk_load(cx, a.blob, br.meta_off, br.meta_bytes, P.s_meta[(i + 1) & 1], &ctl->meta_full[(i + 1) & 1]);
      }
      if (active) {
        pipe_wait(pp, &ctl->w_full[sg], (uint32_t)(load_ordinal(st, sg, i) & 1));
        const uint32_t lbo_b = (uint32_t)n * 16u;
        const uint32_t idesc = ptx::umma_idesc_i8((uint32_t)n, false);
        const uint32_t db_lo = ptx::umma_desc_lo(ptx::smem_u32(smem + P.s_w[sg]), lbo_b);
        const uint32_t da_step = (2u * kTileM * 16u) >> 4, db_step = (2u * lbo_b) >> 4;
        const int ks = kd >> 5;
        // The accumulator region of this GEMM must be free of the slot's previous tile: GEMM 0 writes
        // the slot's main columns, last read by the second epilogue (per-tap partials elsewhere), by
        // the shifted sum (partials in the main columns) or by the prior head's epilogue; GEMM 2 with
        // columns of its own waits for the shifted sum; everything else follows from the operand.
        uint64_t* freed = nullptr;
        bool freed_cpl = true;
        if (sg == 0) {
          if (prior) { freed = ctl->a2_full; freed_cpl = false; }
          else freed = r3_separate ? ctl->a3_full : ctl->r3_free;
        } else if (sg == 2 && r3_separate) {
          freed = ctl->r3_free;
        }
        for (int t = 0; t < ntv; ++t) {
          const int sl = t & 1;
          const uint32_t u = (uint32_t)(t >> 1);
          const uint32_t ph_in = (sg == 2 ? sc.cpl[sl] : sc.all[sl]) + u;
          pipe_wait(pp, &a_full[sl], ph_in & 1u);                                   // the tile's operand is written
          if (freed && u > 0) pipe_wait(pp, &freed[sl], ((freed_cpl ? sc.cpl[sl] : sc.all[sl]) + u - 1u) & 1u);
          ptx::tc_fence_after();
          const uint32_t d = tmem + (uint32_t)(sg == 2 ? P.r_col[1] + sl * P.r_col[2] : sl * P.r_col[0]);
          uint32_t da = ptx::umma_desc_lo(ptx::smem_u32(smem + (sg == 0 ? P.s_a1[sl] : P.s_a[sl])), kTileM * 16), db = db_lo;
          ptx::umma_i8_lo(d, da, db, idesc, 0u);
          for (int k = 1; k < ks; ++k) {
            da += da_step;
            db += db_step;
            ptx::umma_i8_lo(d, da, db, idesc, 1u);
          }
          ptx::umma_commit(ptx::smem_u32(&ctl->d_full[sg][sl]));
        }
      }
    }
    sc.advance(ntv, prior);
    __syncwarp();
    __syncthreads();     // every MMA of step i has completed (the workers waited for each accumulator)
    if (lead) refill(i);
  }
  if (st.nsteps > 0 && !st.is_prior(st.nsteps - 1)) __syncthreads();   // trailing translation pass
}

// ---- workers ---------------------------------------------------------------------------------------
template <bool kInv>
__device__ __forceinline__ void pipe_workers(const Pipe& pp, const LevelPlan& P, const LevelArgs& a, const Steps& st,
                                             int img0, int pvalid, int ntv, uint32_t tmem) {
  uint8_t* smem = pp.smem;
  PipeCtl* ctl = pp.ctl;
  int32_t* v = reinterpret_cast<int32_t*>(smem + P.s_v);
  int8_t* xa = reinterpret_cast<int8_t*>(smem + P.s_xa);
  int32_t* acc = reinterpret_cast<int32_t*>(smem + P.s_acc);
  const uint32_t* rowinfo = reinterpret_cast<const uint32_t*>(smem + P.s_rowinfo);
  const int2* gtab = reinterpret_cast<const int2*>(smem + P.s_gran);
  const int pg = P.pg, ca = P.ca, cb = P.cb, w = P.w, cpad = P.cpad, cbp = P.cbp;
  const bool aux = pp.warp >= kEpiWarps;
  const bool a1_separate = P.s_a1[0] != P.s_a[0];  // the im2col operands have buffers of their own
  const int wq = pp.warp & 3;                      // TMEM lane quarter
  const int cs = (pp.warp >> 2) & 3;               // requantising warps: which quarter of the columns
  const int row = wq * 32 + pp.lane;
  const uint32_t lane_field = (uint32_t)(wq * 32) << 16;
  Ctx cx{};                                        // for the shared build / sum / prior routines
  cx.smem = smem; cx.status = a.status;
  cx.tid = pp.tid; cx.warp = pp.warp; cx.lane = pp.lane; cx.wq = wq;
  cx.row = row; cx.rep = 1; cx.rrows = kTileM;
  cx.bcs = 0; cx.bncs = 1;                         // an aux thread builds its whole row
  cx.cs = aux ? 0 : cs;                            // aux: every unit of the shifted sum; prior epilogue: a quarter of the granules
  cx.ncs = aux ? 1 : 4;
  cx.tmem_base = tmem;
  SlotCount sc{{0u, 0u}, {0u, 0u}};
  const CouplingMeta* prevM = nullptr;

  const uint32_t mul_pv = pvalid > 1 ? (uint32_t)((0xFFFFFFFFull / (uint32_t)pvalid) + 1ull) : 0u;
  const PixelPass px{v, acc, xa, pg, ca, cb, cpad, pvalid, mul_pv, pp.tid, kPipeWorkers};
  auto worker_barrier = [&]() { asm volatile("bar.sync 1, %0;" ::"n"(kPipeWorkers) : "memory"); };
  auto main_cols = [&](int sl) { return tmem + (uint32_t)(sl * P.r_col[0]) + lane_field; };

  for (int i = 0; i < st.nsteps; ++i) {
    pipe_wait(pp, &ctl->meta_full[i & 1], (uint32_t)((i >> 1) & 1));
    const uint8_t* mb = smem + P.s_meta[i & 1];
    const bool prior = st.is_prior(i);
    const CouplingMeta* Mp = reinterpret_cast<const CouplingMeta*>(mb);
    const PriorMeta* Pp = reinterpret_cast<const PriorMeta*>(mb);
    {
      const int32_t* cols = prior ? P.col_out : reinterpret_cast<const int32_t*>(mb + Mp->off_colA);
      const int32_t in_m0 = prior ? Pp->in_m0 : Mp->in_m0, in_s = prior ? Pp->in_s : Mp->in_s;
      if (prevM) {
        apply_translation<kInv>(px, prevM);
        worker_barrier();            // the network input may read channels that were just updated
      }
      requant_input(px, cols, in_m0, in_s);
    }
    prevM = prior ? nullptr : Mp;
    __syncthreads();

    if (aux) {
      // ---- auxiliary warps: the shifted sum of tile t, then the im2col of tile t + 2 into its slot
      const int kd1 = prior ? Pp->kd : Mp->kd1;
      auto build = [&](int t) {
        const RowPos r = row_pos(rowinfo, t, row, row);
        uint8_t* a_row = smem + P.s_a1[t & 1] + row * 16;
        if (cpad == 8) build_im2col_taps<8>(a_row, xa, w, kd1, r, 0, 1);
        else if (cpad == 16) build_im2col_taps<16>(a_row, xa, w, kd1, r, 0, 1);
        else build_im2col(cx, smem + P.s_a1[t & 1], xa, gtab, cpad, kd1, r);
        pipe_arrive(pp, &ctl->a1_full[t & 1], true);
      };
      for (int t = 0; t < ntv && t < 2; ++t) build(t);
      auto sum = [&](int t) {
        const int sl = t & 1;
        ptx::tc_fence_after();
        const RowPos r = row_pos(rowinfo, t, row, row);
        cx.tmem_slot = tmem + (uint32_t)(P.r_col[1] + sl * P.r_col[2]) + lane_field;
        if (cb == 6 && pg == 1024) scatter_lean<4096, 6>(cx.tmem_slot, acc, w, r);
        else if (cb == 6 && pg == 256) scatter_lean<1024, 6>(cx.tmem_slot, acc, w, r);
        else if (cb == 12 && pg == 256) scatter_lean<1024, 12>(cx.tmem_slot, acc, w, r);
        else epilogue_scatter(cx, cb, cbp, acc, pg, w, r);
        pipe_arrive(pp, &ctl->r3_free[sl], false);
      };
      // Two cursors: nb, the next tile to build (its slot's im2col buffer is free once the first GEMM
      // of the slot's previous tile has read it; with one operand buffer per slot, once the last GEMM
      // has), and ns, the next tile whose per-tap partials are to be summed. Building comes first: the
      // slot's next GEMM waits for it, nothing waits for a sum before the step ends (or, with shared
      // columns, before that same GEMM).
      const int g_read = (a1_separate || prior) ? 0 : 2;       // the GEMM whose completion frees the im2col buffer
      int nb = min(2, ntv), ns = prior ? ntv : 0;
      uint32_t idle = 0;
      volatile uint32_t* ab = &ctl->abort;
      while (nb < ntv || ns < ntv) {
        const int bs = nb & 1, ss = ns & 1;
        const uint32_t ph_b = ((g_read == 0 ? sc.all[bs] : sc.cpl[bs]) + (uint32_t)((nb - 2) >> 1)) & 1u;
        const uint32_t ph_s = (sc.cpl[ss] + (uint32_t)(ns >> 1)) & 1u;
        if (nb < ntv && ptx::mbar_test_wait(ptx::smem_u32(&ctl->d_full[g_read][bs]), ph_b)) {
          build(nb);
          ++nb;
          idle = 0;
        } else if (ns < ntv && ptx::mbar_test_wait(ptx::smem_u32(&ctl->d_full[2][ss]), ph_s)) {
          sum(ns);
          ++ns;
          idle = 0;
        } else {
          // nothing to do: sleep on the barrier that is due next, for a short while
          if (ns < ntv) ptx::mbar_try_wait_ns(ptx::smem_u32(&ctl->d_full[2][ss]), ph_s, 300u);
          else ptx::mbar_try_wait_ns(ptx::smem_u32(&ctl->d_full[g_read][bs]), ph_b, 300u);
          if (*ab) break;
          if (++idle > (1u << 22)) {       // bounded: a level that stops moving is reported, not awaited
            *ab = 1;
            atomicExch(a.status, 1u);
            break;
          }
        }
      }
    } else {
      // ---- requantising warps: both slots in turn, one hidden layer after the other
      for (int t0 = 0; t0 < ntv; t0 += 2) {
        const int nt = min(2, ntv - t0);
        const uint32_t u = (uint32_t)(t0 >> 1);
        if (prior) {
          const PriorMeta M = *Pp;
          const OutRq* orq = reinterpret_cast<const OutRq*>(mb + M.off_out);
          for (int sl = 0; sl < nt; ++sl) {
            pipe_wait(pp, &ctl->d_full[0][sl], (sc.all[sl] + u) & 1u);
            ptx::tc_fence_after();
            cx.tmem_slot = main_cols(sl);
            epilogue_prior(cx, P, a, M, orq, img0, row_pos(rowinfo, t0 + sl, row, row));
            pipe_arrive(pp, &ctl->a2_full[sl], false);                      // the slot's accumulator is drained
          }
          continue;
        }
#pragma unroll 1
        for (int layer = 0; layer < 2; ++layer) {
          const int n = layer ? Mp->n2 : Mp->n1, kd = layer ? Mp->kd3 : Mp->kd2, us = layer ? Mp->us2 : Mp->us1;
          const int32_t* m0tab = reinterpret_cast<const int32_t*>(mb + (layer ? Mp->off_u2 : Mp->off_u1));
          const long long rnd64 = 1ll << (30 + us);
          // this warp's share of the columns: a quarter of the 8-column units
          const int units = n >> 3;
          const int c0 = ((units * cs) >> 2) << 3, c1 = ((units * (cs + 1)) >> 2) << 3;
          for (int sl = 0; sl < nt; ++sl) {
            pipe_wait(pp, &ctl->d_full[layer][sl], ((layer ? sc.cpl[sl] : sc.all[sl]) + u) & 1u);
            // The first layer's output goes where the slot's previous tile had its third GEMM's operand:
            // that GEMM must have read it (with im2col buffers of their own nothing else orders the two).
            if (layer == 0 && u > 0) pipe_wait(pp, &ctl->d_full[2][sl], (sc.cpl[sl] + u - 1u) & 1u);
            ptx::tc_fence_after();
            uint8_t* out_row = smem + P.s_a[sl] + row * 16;
            // the columns beyond the layer's channels: bias columns of the next GEMM (first layer), zeros
            for (int j = (n >> 4) + cs; j < (kd >> 4); j += 4)
              *reinterpret_cast<uint4*>(out_row + (size_t)j * (kTileM * 16)) =
                  (layer == 0 && j == (n >> 4)) ? make_uint4(kBiasColumnsLo, kBiasColumnsHi, 0u, 0u) : make_uint4(0u, 0u, 0u, 0u);
            epilogue_lean(main_cols(sl), c0, c1 - c0, m0tab, us - 1, rnd64, out_row);
            pipe_arrive(pp, layer ? &ctl->a3_full[sl] : &ctl->a2_full[sl], true);
          }
        }
      }
    }
    sc.advance(ntv, prior);
    ptx::tc_fence_before();
    __syncthreads();
  }
  if (prevM) {
    apply_translation<kInv>(px, prevM);
    __syncthreads();
  }
}

template <bool kInv>
__global__ void __launch_bounds__(kPipeThreads, 1) level_pipe_kernel(const LevelArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ PipeCtl ctl;
  const LevelPlan& P = *a.plan;
  // the warp index through a shuffle: tells the compiler that it is the same in all lanes, so that
  // roles, tensor-memory addresses and operand descriptors live in uniform registers
  const int tid = threadIdx.x, warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0), lane = tid & 31;

  ptx::grid_launch_dependents();         // the next kernel in the stream may start its prologue
  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      ptx::mbar_init(ptx::smem_u32(&ctl.a1_full[s]), (uint32_t)kAuxWarps);
      ptx::mbar_init(ptx::smem_u32(&ctl.a2_full[s]), (uint32_t)kEpiWarps);
      ptx::mbar_init(ptx::smem_u32(&ctl.a3_full[s]), (uint32_t)kEpiWarps);
      ptx::mbar_init(ptx::smem_u32(&ctl.r3_free[s]), (uint32_t)kAuxWarps);
      for (int g = 0; g < 3; ++g) ptx::mbar_init(ptx::smem_u32(&ctl.d_full[g][s]), 1);
    }
    for (int s = 0; s < 3; ++s) ptx::mbar_init(ptx::smem_u32(&ctl.w_full[s]), 1);
    for (int s = 0; s < 2; ++s) ptx::mbar_init(ptx::smem_u32(&ctl.meta_full[s]), 1);
    ptx::mbar_init_fence();
    ctl.abort = 0;
  }
  if (warp == 0) ptx::tmem_alloc(ptx::smem_u32(&ctl.tmem_base), (uint32_t)P.tmem_cols);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = ctl.tmem_base;

  const int px = P.px, pg = P.pg, w = P.w;
  const int img0 = blockIdx.x * P.group;
  const int nimg = min(P.group, a.batch - img0);
  const int pvalid = nimg * px;
  const int ntv = (pvalid + kTileM - 1) / kTileM;
  int32_t* v = reinterpret_cast<int32_t*>(smem + P.s_v);

  Steps st;
  st.n_couplings = (kInv && a.phase == 1) ? 0 : P.n_couplings;
  st.do_prior = P.has_prior && a.prior != nullptr && !(kInv && a.phase == 2);
  st.nsteps = st.n_couplings + (st.do_prior ? 1 : 0);
  st.inverse = kInv;

  Pipe pp{smem, &ctl, a.status, tid, warp, lane};
  if (warp >= kPipeWorkerWarps) {
    pipe_control(pp, P, a, st, ntv, warp - kPipeWorkerWarps);
  } else {
    int32_t* acc = reinterpret_cast<int32_t*>(smem + P.s_acc);
    for (int idx = tid; idx < P.cb * pg; idx += kPipeWorkers) acc[idx] = 0;
    uint32_t* rowinfo = reinterpret_cast<uint32_t*>(smem + P.s_rowinfo);
    for (int idx = tid; idx < P.tiles * kTileM; idx += kPipeWorkers)
      rowinfo[idx] = row_record(idx, pvalid, px, P.h, w, P.mul_px, P.mul_w);
    int32_t* gran = reinterpret_cast<int32_t*>(smem + P.s_gran);
    for (int idx = tid; idx < 2 * P.n_gran; idx += kPipeWorkers) gran[idx] = P.gran_tab[idx];
    // Everything above used only the plan; from here on the kernel reads what the previous kernel
    // in the stream wrote and writes what it may still be reading.
    ptx::grid_dependency_wait();
    level_load<kInv>(P, a, v, img0, nimg, tid, kPipeWorkers);
    __syncthreads();

    pipe_workers<kInv>(pp, P, a, st, img0, pvalid, ntv, tmem);

    level_store<kInv>(P, a, v, img0, nimg, tid, lane, kPipeWorkers);
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 0) ptx::tmem_dealloc(tmem, (uint32_t)P.tmem_cols);
}

}  // namespace

cudaError_t launch_level_pipe(const LevelArgs& args, bool inverse, int grid, uint32_t smem_bytes, cudaStream_t stream) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)kPipeThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (inverse) return cudaLaunchKernelEx(&cfg, level_pipe_kernel<true>, args);
  return cudaLaunchKernelEx(&cfg, level_pipe_kernel<false>, args);
}

cudaError_t configure_pipe_kernels(uint32_t max_smem_bytes) {
  cudaError_t e = cudaFuncSetAttribute(level_pipe_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)max_smem_bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(level_pipe_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem_bytes);
}

}  // namespace iodf
