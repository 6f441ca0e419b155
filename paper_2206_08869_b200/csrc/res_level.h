// Flow levels whose couplings use the residual-block network (Eq. 3, Sec. 4.1; scatter add, Sec. 4.5;
// App. B.1): device-side records and the launch interface. The level's shape, index maps and
// latent layout are the LevelPlan's; everything about the networks sits in the level blob, headed
// by a ResHead.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "iodf_dev.h"
#include "level_kernel.h"

namespace iodf {

constexpr int kResBuilderWarps = 16;                         // the warps that requantise (and load / store the level)
constexpr int kResThreads = kResBuilderWarps * 32;           // their threads
constexpr int kResIssuers = 3;                               // warps whose elected lane issues MMAs (tiles dealt between them)
constexpr int kResAllThreads = kResThreads + 32 * (kResIssuers + 1);   // + the issuing warps and the warp that streams weights
constexpr int kResMaxWidth = 128;      // hidden channels of a residual network (conv outputs), padded to 16
constexpr int kResMaxPixels = 256;     // pixels of an image that one CTA holds at a residual level
constexpr int kResMaxBands = 8;        // row bands of an image (= CTAs of a thread-block cluster) at larger levels
constexpr int kResMaxWSlots = 8;       // depth of the weight-slice ring

// what a conv's epilogue does with its requantised outputs
enum ResKind : int32_t {
  kResHidden = 0,     // ReLU + clip to 0..255, written as bytes to the conv's destination buffer
  kResBranch = 1,     // second conv of a block, as wide as X (its filters sit at the rows idx[] names, zero
                      // rows elsewhere): added channel by channel to the (already requantised) shortcut in X
  kResOut = 2,        // last conv: the translation, added to / subtracted from the flow variable
  kResPrior = 3       // prior head: mu and clipped log-scale index to global memory
};

// One 3x3 conv. Its nine weight slices (one per tap) are [kpad/16][n_pad][16 bytes] each, back to back.
struct ResConv {
  uint32_t w_off;          // blob offset of slice 0
  uint32_t slice_bytes;    // n_pad * kpad
  uint32_t rq_off;         // blob offset of OutRq[n_pad] (padding channels requantise 0 to 0)
  uint32_t idx_off;        // unused (the index list of a block is applied when the level is packed)
  int32_t n, n_pad;        // outputs, and padded to 16
  int32_t kpad;            // input bytes per pixel and tap, a multiple of 32 (<= the source's pitch)
  int32_t a_unsigned;      // input is unsigned 8-bit (hidden activations) or signed (network / head input)
  int32_t kind;
  int32_t src, dst;        // buffers: 0 = network input (int8), 1 = X, 2 = MID
  int32_t short_m0, short_s;   // kResBranch: the block's shortcut requantisation
  int32_t pad[3];
};
static_assert(sizeof(ResConv) == 64, "64-byte records");

struct ResCouplingRec {
  int32_t in_m0, in_s;
  uint32_t colA_off, colB_off;   // blob offsets of the physical columns of the coupling's logical channels
  int32_t conv0, n_convs;        // its convs in the conv array
  int32_t pad[2];
};

struct ResHead {
  int32_t n_couplings, n_convs;
  int32_t prior_conv;            // index of the prior head's conv, or -1
  int32_t prior_in_m0, prior_in_s, ls_lo, ls_hi;
  int32_t xa_pitch, x_pitch, mid_pitch;      // bytes per pixel of the three activation buffers (multiples of 32)
  uint32_t coupling_off, conv_off;           // blob offsets of ResCouplingRec[] and ResConv[]
  uint32_t s_v, s_xa, s_x, s_mid, s_rowinfo, s_unused[2], s_wring, w_slot_bytes, s_total;   // shared-memory layout
  int32_t tmem_cols;
  int32_t n_wslots;              // weight slices in flight: ring of 2 .. kResMaxWSlots slots at s_wring
  uint32_t s_tab;                // the running conv's OutRq[kResMaxWidth], idx[kResMaxWidth] and 256-byte shortcut table
  // padded layout of the activation buffers: rows of w2 = w + 2 positions, (h + 2) * w2 positions
  // rounded up to ntiles * 128 computed ones, `guard` rows before them, `rows` rows per channel chunk
  int32_t w2, guard, rows, ntiles;
  // Levels of more than kResMaxPixels pixels per image: the image is cut into `bands` bands of hb rows,
  // one CTA of a thread-block cluster each (bands = 1, hb = h otherwise). Every CTA keeps its band in
  // the padded layout above with (hb + 2) rows; the row above and below hold the neighbouring bands'
  // edge rows, which the neighbours write through distributed shared memory after every conv.
  int32_t bands, hb;
  // Levels whose padded frame (h + 2)(w + 2) fits a 128-position tile several times over: `group` images
  // per CTA (throughput plan only, bands = 1), their frames one after the other in the padded layout. A
  // real pixel's taps stay inside its own frame and every frame's border is zero, so nothing else changes.
  int32_t group;
};
static_assert(sizeof(ResHead) == 128, "128-byte header");

cudaError_t configure_res_kernels(uint32_t max_smem_bytes);
// `images` images of `bands` row bands each (bands > 1: one thread-block cluster per image)
cudaError_t launch_res_level(const LevelArgs& args, bool inverse, int images, int bands, uint32_t smem_bytes,
                             cudaStream_t stream);

}  // namespace iodf
