// Structures shared by the host-side packer and the sm_100a kernels.
//
// Memory layout on the device
//   * One "level blob" per flow level holds, back to back and 128-byte aligned, one packed block
//     per coupling and one for the prior head. A block is [meta | W1 | W2 | W3]; the kernel pulls
//     each part into shared memory with one bulk copy.
//   * Weight matrices are stored exactly as tcgen05.mma reads them from shared memory: K-major,
//     no swizzle, as [K/16][N][16 bytes]. A core matrix (8 rows x 16 bytes) is 128 contiguous
//     bytes; consecutive 8-row groups are 128 bytes apart (stride-dimension offset) and
//     consecutive 16-byte K chunks are N*16 bytes apart (leading-dimension offset).
//   * Activation tiles (128 pixels x K bytes) use the same scheme: [K/16][128][16 bytes].
//   * Bias columns: right after the data columns of the first two GEMMs' K (after the nine taps;
//     after the padded hidden channels) every A row carries the eight constants (1, 127, ..., 127), and a
//     layer whose biases fit has them decomposed over the matching eight weight rows
//     (bias = w0 * 1 + (w1 + ... + w7) * 127), so that its accumulator already includes the bias.
//   * K of a 3x3 conv over the coupling input is ordered tap-major with the channel count padded
//     to 8 (k = tap*cpad + c), so every im2col granule is an aligned 8-byte copy. N of the last
//     3x3 conv is one row per (tap, out channel) with the channel count padded to 8
//     (n = tap*cbp + c), so every 8-column accumulator granule belongs to one tap.
#pragma once
#include <stdint.h>

namespace iodf {

constexpr int kTileM = 128;          // pixels per MMA tile (UMMA M)
constexpr int kWorkerWarps = 16;     // four per TMEM lane quarter
constexpr int kWorkers = kWorkerWarps * 32;
constexpr int kThreads = kWorkers + 32;   // + one control warp (bulk copies and MMA issue)
constexpr int kMaxCouplings = 32;    // per level
constexpr int kMaxC = 256;           // flow channels per level
constexpr int kMaxHidden = 512;      // kept hidden channels per layer (padded): the TMEM column count
constexpr int kRingDepth = 3;        // weight K-slices in flight when weights are streamed
constexpr int kSlotCols = 256;       // TMEM columns per tile slot when two tiles are in flight
constexpr uint32_t kSpinLimit = 20000u;   // bounded waits: tries of up to 100 us each
// The eight constant A-operand bytes that multiply a layer's bias rows: 1, then seven times 127.
// im2col granule table: validity selectors beyond the nine taps' gather-mask bits
constexpr int kGranBias = 9, kGranPad = 10;
constexpr int kMaxGran = 152;        // 8-byte granules of the widest first-conv K: (9 * 128 + 8) / 8, rounded up to 32 bytes
constexpr uint32_t kBiasColumnsLo = 0x7F7F7F01u, kBiasColumnsHi = 0x7F7F7F7Fu;

// Per-hidden-channel constants of the fast requantisation path (16 bytes).
//   y = hi32(acc * m0 + c64) >> sh,  c64 = bias * m0 + 2^(30+s),  sh = s - 1   (needs s >= 1)
struct HiddenRq {
  int32_t m0;
  int32_t sh;
  uint32_t c_lo, c_hi;
};

// Per-output-channel constants of the translation and prior outputs (any shift 0..31):
//   y = (acc * m0 + c64) >> (31 + s),  c64 = bias * m0 + 2^(30+s)
struct OutRq {
  int32_t m0;
  int32_t s;
  uint32_t c_lo, c_hi;
};

// Meta part of a coupling block, followed in memory by
//   colA[ca] colB[cb] (int32 physical column of each logical channel), OutRq[cb],
//   HiddenRq[n1], HiddenRq[n2], {m0, bias}[n1], {m0, bias}[n2]; every array 16-byte aligned.
struct CouplingMeta {
  int32_t in_m0, in_s;
  int32_t n1, n2;                // hidden widths padded to 16 (MMA N)
  int32_t kd1, kd2, kd3;         // K bytes of the three GEMMs, padded to 32
  int32_t n3;                    // 9*cbp padded to 16 (per-tap partial outputs of the last conv)
  int32_t lo1, hi1, lo2, hi2;    // effective activation clips (ReLU folded in)
  int32_t mode1, mode2;          // requantisation flavour of the two hidden layers:
                                 //   3: one shift s >= 1 and the bias folded into the GEMM (m0 table)
                                 //   2: one shift s >= 1 for the whole layer ({m0, bias} table)
                                 //   1: per-channel shifts, all >= 1 (HiddenRq table, high-word path)
                                 //   0: any shift (HiddenRq table, full 64-bit shift)
  int32_t us1, us2;              // the uniform shift (modes 2 and 3)
  int32_t off_colA, off_colB, off_out, off_h1, off_h2;   // byte offsets from the meta start
  int32_t off_u1, off_u2;        // {m0, bias} tables (int2 per channel; mode 3: int32 m0 per channel)
  int32_t pad[9];
};
static_assert(sizeof(CouplingMeta) == 128, "meta header is 128 bytes");

// Meta part of a prior-head block, followed by OutRq[2*cb].
struct PriorMeta {
  int32_t in_m0, in_s;
  int32_t n;                     // 2*cb padded to 16
  int32_t kd;                    // 9*cpad padded to 32
  int32_t ls_lo, ls_hi;
  int32_t off_out;
  int32_t pad[25];
};
static_assert(sizeof(PriorMeta) == 128, "meta header is 128 bytes");

struct BlockRef {                // where a block's parts sit in the level blob (byte offsets)
  uint32_t meta_off, meta_bytes;
  uint32_t w_off[3], w_bytes[3];
  uint32_t k_slices[3];          // K / 32 of each matrix (a K-slice of 32 bytes is w_bytes / k_slices contiguous bytes)
};

// Everything a level kernel needs; lives in global memory.
struct LevelPlan {
  int32_t c, h, w, px;           // level shape after the squeeze
  int32_t ca, cb;
  int32_t cpad, cbp;             // ca, cb rounded up to 8
  int32_t group;                 // images per CTA
  int32_t pg;                    // pixel slots per CTA = group*px rounded up to 32
  int32_t tiles;                 // ceil(group*px / 128)
  int32_t n_couplings;
  int32_t split, has_prior, is_first, is_last;
  int32_t keep_c;                // channels that go on to the next level (c/2 if split else c)
  int32_t rep;                   // row replication, 1, 2 or 4: a CTA whose pixels fill at most 128/rep rows of
                                 // its single tile puts them in the tile rep times (rows r, r + 128/rep, ...),
                                 // so that every TMEM lane quarter holds a copy and the epilogues split the
                                 // accumulator columns over all 16 worker warps instead of 4 * (4 / rep)
  int32_t residual;              // 1: the level's couplings are residual-block networks (its own kernel; the
                                 //    level blob then starts with a ResHead and the fields on tiles, slots and
                                 //    the shared-memory layout below are unused)
  int32_t res_bands;             // residual levels: row bands per image (CTAs of a cluster), 1 = one CTA per image
  int32_t nslots;                // tiles in flight per CTA: 1 or 2
  int32_t tmem_cols;
  int32_t w13_alias;             // 1: W1 and W3 share a slot and are re-fetched per tile
  int32_t streamed;              // 1: weights are streamed per tile in 32-byte K-slices through a ring of
                                 //    kRingDepth slots at s_w[0] (hidden widths above 256, one tile in flight)
  uint32_t ring_slot_bytes;
  int32_t lean;                  // 1: every hidden layer in the folded requantisation flavour with the 0..127 clip,
                                 //    weights not streamed: the general kernel's small variant runs the level
  int32_t pipe;                  // 1: the level runs in the kernel that splits a tile's work by role (several
                                 //    tiles per CTA, two tile slots, resident weights, folded requantisation with
                                 //    the 0..127 clip)
  int32_t r_col[3];              // that kernel's tensor-memory columns: slot s has its hidden-layer accumulators
                                 //    at s * r_col[0] and its per-tap partials at r_col[1] + s * r_col[2]
                                 //    (r_col[1] = 0: the partials share the slot's main columns)
  // shared-memory byte offsets
  uint32_t s_v, s_xa, s_acc, s_rowinfo, s_gran, s_a[2], s_meta[2], s_w[3], s_total;
  uint32_t s_a1[2];              // role-split kernel: the slots' im2col operands (= s_a[] when they share the buffer)
  // magic multipliers for the index maps: n / d = umulhi(n, ceil(2^32 / d)) for n * d < 2^32 (0: d = 1)
  uint32_t mul_per_img, mul_4px, mul_w2, mul_px, mul_w;
  uint32_t recip_gpa, recip_gpb; // floor(g / (cpad/8)) = (g * recip_gpa) >> 16 for g < 4096; same for cbp/8
  // global layout
  uint64_t z_off, prior_off, z_final_off, d, d_fact;
  int32_t col_out[kMaxC];        // physical column of logical channel k after the last coupling
  // im2col granule g of the first conv's K (8 bytes): {byte offset of its source relative to the
  // pixel's xa record, validity selector: tap 0..8 = bit of the row's gather mask, kGranBias, kGranPad}
  int32_t n_gran;
  int32_t gran_tab[2 * kMaxGran];
  BlockRef coupling[kMaxCouplings];
  BlockRef prior;
};

}  // namespace iodf
