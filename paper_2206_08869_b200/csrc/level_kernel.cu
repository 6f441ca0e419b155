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

#include "level_device.cuh"

namespace iodf {

namespace {

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
    top_up(cx, P, a, st, W, -1, alias, ctl->w_full);
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
    if (lead) top_up(cx, P, a, st, W, i, alias, ctl->w_full);
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
// kLean: every hidden layer of the level is in the folded requantisation flavour with the 0..127
// clip (what the model packer produces for the usual layers), so that the epilogues need one code
// path instead of seven. The deep levels run every phase's code once per coupling, and what they
// wait for most, beside memory, is instruction fetch: the smaller the loop body, the better.
template <bool kInv, bool kLean>
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

  // n / pvalid for the work-item maps of the pixel pass (n * pvalid < 2^32)
  const uint32_t mul_pv = pvalid > 1 ? (uint32_t)((0xFFFFFFFFull / (uint32_t)pvalid) + 1ull) : 0u;
  const PixelPass pp{v, acc, xa, pg, ca, cb, cpad, pvalid, mul_pv, cx.tid, kWorkers};
  auto apply_translation_all = [&]() { apply_translation<kInv>(pp, prevM); };
  auto requant_input_all = [&](const int32_t* cols, int32_t m0, int32_t s) { requant_input(pp, cols, m0, s); };
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
          if (kLean) epilogue_hidden_t(cx, M.n1, M.kd2, Requant<kModeFolded, kClipS8Relu>{h1, u1, 0, 127, M.us1 - 1, 1ll << (30 + M.us1)},
                                       kBiasColumnsLo, kBiasColumnsHi, sA);
          else epilogue_hidden(cx, M.mode1, M.us1, M.n1, M.kd2, h1, u1, M.lo1, M.hi1, kBiasColumnsLo, kBiasColumnsHi, sA);
          arrive_a(sl);
        }
        for (int sl = 0; sl < nt; ++sl) {                     // requant, conv 3x3 as per-tap partials
          wait_d(sl);
          use_slot(sl);
          if (kLean) epilogue_hidden_t(cx, M.n2, M.kd3, Requant<kModeFolded, kClipS8Relu>{h2, u2, 0, 127, M.us2 - 1, 1ll << (30 + M.us2)}, 0u, 0u, sA);
          else epilogue_hidden(cx, M.mode2, M.us2, M.n2, M.kd3, h2, u2, M.lo2, M.hi2, 0u, 0u, sA);
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

template <bool kInv, bool kLean>
__global__ void __launch_bounds__(kThreads, 1) level_kernel(const LevelArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ Ctl ctl;
  const LevelPlan& P = *a.plan;
  // the warp index through a shuffle: tells the compiler that it is the same in all lanes, so that
  // roles, tensor-memory addresses and operand descriptors can live in uniform registers
  const int tid = threadIdx.x, warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0), lane = tid & 31;

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
    if (!kLean && P.streamed) {
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
    level_load<kInv>(P, a, v, img0, nimg, tid, kWorkers);
    cta_barrier();

    run_workers<kInv, kLean>(cx, P, a, st, img0, pvalid, ntv);

    level_store<kInv>(P, a, v, img0, nimg, tid, lane, kWorkers);
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 0) ptx::tmem_dealloc(tmem, (uint32_t)P.tmem_cols);
}

}  // namespace

cudaError_t launch_level(const LevelArgs& args, bool inverse, bool lean, int grid, uint32_t smem_bytes,
                         cudaStream_t stream) {
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
  if (lean) return inverse ? cudaLaunchKernelEx(&cfg, level_kernel<true, true>, args)
                           : cudaLaunchKernelEx(&cfg, level_kernel<false, true>, args);
  return inverse ? cudaLaunchKernelEx(&cfg, level_kernel<true, false>, args)
                 : cudaLaunchKernelEx(&cfg, level_kernel<false, false>, args);
}

cudaError_t configure_level_kernels(uint32_t max_smem_bytes) {
  cudaError_t e = cudaFuncSetAttribute(level_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem_bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(level_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem_bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(level_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem_bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(level_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem_bytes);
  return e;
}

}  // namespace iodf
