// Host side of the IODF library: descriptor validation, weight repacking into the tensor-core
// operand layout, shared-memory planning per level, and the C entry points declared in iodf.h.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/iodf.h"
#include "iodf_dev.h"
#include "rans_kernel.h"
#include "res_level.h"
#include "level_kernel.h"
#include "level_pipe.h"
#include "selftest.h"

using namespace iodf;

namespace {

constexpr uint32_t kAlign = 128;

inline uint32_t up(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }

struct HostLevel {
  LevelPlan plan;
  std::vector<uint8_t> blob;
  int grid_group = 1;
  int32_t ls_lo = 0, ls_hi = 0;      // clip of the prior head's log-scale index (levels with a head)
};

}  // namespace

struct iodf_model {
  int device = 0;
  int last_cuda = 0;
  uint32_t max_batch = 0;
  uint32_t in_c = 0, in_h = 0, in_w = 0;
  iodf_layout layout{};
  std::vector<HostLevel> levels;
  std::vector<LevelPlan*> d_plan;
  std::vector<uint8_t*> d_blob;
  std::vector<int32_t*> d_keep;     // kept channels between level l and l+1
  uint32_t* d_status = nullptr;
  std::vector<cudaEvent_t> ev;      // n_levels + 1 events for the timed entry points
  // staging for the host-buffer entry points
  uint8_t* d_x = nullptr;
  int32_t* d_z = nullptr;
  int32_t* d_prior = nullptr;
};

struct iodf_codec {
  int device = 0;
  int last_cuda = 0;
  uint32_t max_batch = 0;
  uint32_t elems_per_stream = 0;
  uint8_t* d_tables = nullptr;      // R then G
  uint32_t* d_errors = nullptr;
  uint32_t* d_sizes = nullptr;      // max_batch record sizes (packing scratch)
  // staging of the host-buffer entry points, allocated by their first call
  uint16_t* d_words = nullptr;
  uint32_t* d_counts = nullptr;
  uint8_t* d_packed = nullptr;
  size_t packed_capacity = 0;
  iodf::RansArgs args{};
  iodf_codec_layout layout{};
};

namespace {

struct Blobs {
  const int8_t* w;
  size_t w_count;
  const int32_t* r;
  size_t r_count;
};

int check_layer(const iodf_layer_desc& L, const Blobs& B) {
  if ((L.k != 1 && L.k != 3) || L.c_in < 1 || L.c_out < 1) return IODF_EINVAL;
  const uint64_t wn = (uint64_t)L.c_out * L.k * L.k * L.c_in;
  if (L.weight_off > B.w_count || wn > B.w_count - L.weight_off) return IODF_EINVAL;
  if (L.requant_off > B.r_count || 3ull * L.c_out > B.r_count - L.requant_off) return IODF_EINVAL;
  const int32_t* m0 = B.r + L.requant_off + L.c_out;
  const int32_t* s = m0 + L.c_out;
  for (uint32_t i = 0; i < L.c_out; ++i)
    if (m0[i] < (1 << 30) || s[i] < 0 || s[i] > 31) return IODF_EINVAL;
  if (L.has_clamp && L.clamp_lo > L.clamp_hi) return IODF_EINVAL;
  return IODF_OK;
}

// Worst case |accumulator + bias| for inputs bounded by amax must fit int32.
int check_overflow(const iodf_layer_desc& L, const Blobs& B, int64_t amax) {
  const int8_t* w = B.w + L.weight_off;
  const int32_t* bias = B.r + L.requant_off;
  const size_t fan = (size_t)L.k * L.k * L.c_in;
  for (uint32_t o = 0; o < L.c_out; ++o) {
    int64_t sum = 0;
    for (size_t i = 0; i < fan; ++i) sum += std::abs((int)w[o * fan + i]);
    const int64_t worst = sum * amax + std::llabs((long long)bias[o]);
    if (worst > 0x7FFFFFFFll) return IODF_EOVERFLOW;
  }
  return IODF_OK;
}

struct Act { int lo, hi; };

// Effective range of a hidden layer's output; must be inside the signed (-128..127) or the unsigned
// (0..255, the format of Sec. 4.1 for non-negative tensors) 8-bit range.
int hidden_range(const iodf_layer_desc& L, Act* out) {
  if (!L.has_clamp) return IODF_EUNSUPPORTED;
  int lo = L.clamp_lo, hi = L.clamp_hi;
  if (L.relu) lo = std::max(lo, 0);
  if (lo > hi) { lo = hi; }
  const bool fits_signed = lo >= -128 && hi <= 127, fits_unsigned = lo >= 0 && hi <= 255;
  if (!fits_signed && !fits_unsigned) return IODF_EUNSUPPORTED;
  out->lo = lo;
  out->hi = hi;
  return IODF_OK;
}

// Bias folded into the GEMM: the A operand carries kBiasRows constant columns (1, 127, 127, ...)
// and the weight matrix one row per column with bias = w[0] + 127 * (w[1] + ... + w[kBiasRows-1]),
// every |w[j]| <= 127, so the accumulator already holds acc + bias and the epilogue needs the
// multiplier only. Exact (integer sums); possible while |bias| <= kFoldMaxBias.
constexpr int kBiasRows = 8;
constexpr int64_t kFoldMaxBias = 63 + 127ll * 127ll * (kBiasRows - 1);
void fold_bias(int32_t bias, int8_t w[kBiasRows]) {
  const int64_t b = bias;
  int64_t q = b >= 0 ? (b + 63) / 127 : -((-b + 63) / 127);
  w[0] = (int8_t)(b - 127 * q);
  for (int j = 1; j < kBiasRows; ++j) {
    const int64_t t = std::max<int64_t>(-127, std::min<int64_t>(127, q));
    w[j] = (int8_t)t;
    q -= t;
  }
}

// Fills the constant tables of a hidden layer and picks its requantisation flavour:
//   3: one shift s >= 1 for the whole layer and every bias foldable: table of multipliers (mb[i])
//   2: one shift s >= 1: table of {m0, bias} pairs (mb[2i], mb[2i+1])
//   1 / 0: per-channel shifts (HiddenRq table)
void put_hidden_rq(HiddenRq* dst, int32_t* mb, const iodf_layer_desc& L, const Blobs& B, int n_pad, int* mode,
                   int* uniform_s) {
  const int32_t* bias = B.r + L.requant_off;
  const int32_t* m0 = bias + L.c_out;
  const int32_t* s = m0 + L.c_out;
  bool fast = true, uniform = true, foldable = true;
  for (int i = 0; i < n_pad; ++i) {
    HiddenRq h;
    if (i < (int)L.c_out) {
      const long long c64 = (long long)bias[i] * (long long)m0[i] + (1ll << (30 + s[i]));
      h.m0 = m0[i];
      h.sh = s[i] - 1;
      h.c_lo = (uint32_t)((unsigned long long)c64 & 0xFFFFFFFFull);
      h.c_hi = (uint32_t)((unsigned long long)c64 >> 32);
      if (s[i] < 1) fast = false;
      if (s[i] != s[0] || s[i] < 1) uniform = false;
      if (std::llabs((long long)bias[i]) > kFoldMaxBias) foldable = false;
      mb[2 * i] = m0[i];
      mb[2 * i + 1] = bias[i];
    } else {  // padding channel: acc = 0 -> 0 (its weights in the next layer are zero anyway)
      h.m0 = 1 << 30;
      h.sh = 0;
      h.c_lo = 0x80000000u;
      h.c_hi = 0;
      mb[2 * i] = 1 << 30;
      mb[2 * i + 1] = 0;
    }
    dst[i] = h;
  }
  *mode = uniform ? (foldable ? 3 : 2) : (fast ? 1 : 0);
  *uniform_s = uniform ? s[0] : 0;
  if (*mode == 3)
    for (int i = 0; i < n_pad; ++i) mb[i] = i < (int)L.c_out ? m0[i] : (1 << 30);
}

void put_out_rq(OutRq* dst, const iodf_layer_desc& L, const Blobs& B) {
  const int32_t* bias = B.r + L.requant_off;
  const int32_t* m0 = bias + L.c_out;
  const int32_t* s = m0 + L.c_out;
  for (uint32_t i = 0; i < L.c_out; ++i) {
    const long long c64 = (long long)bias[i] * (long long)m0[i] + (1ll << (30 + s[i]));
    dst[i] = OutRq{m0[i], s[i], (uint32_t)((unsigned long long)c64 & 0xFFFFFFFFull),
                   (uint32_t)((unsigned long long)c64 >> 32)};
  }
}

// Weight matrix [n_pad rows][kd bytes], K-major, no swizzle: byte (n, k) at (k/16)*n_pad*16 + n*16 + k%16.
inline size_t wpos(int n_pad, int n, int k) { return (size_t)(k >> 4) * n_pad * 16 + (size_t)n * 16 + (k & 15); }

struct PackedBlock {
  std::vector<uint8_t> meta, w[3];
  uint32_t k_slices[3] = {0, 0, 0};
};

void append_block(std::vector<uint8_t>& blob, const PackedBlock& pb, BlockRef* ref) {
  auto add = [&](const std::vector<uint8_t>& part, uint32_t* off, uint32_t* bytes) {
    blob.resize(up((uint32_t)blob.size(), kAlign), 0);
    *off = (uint32_t)blob.size();
    *bytes = (uint32_t)part.size();
    blob.insert(blob.end(), part.begin(), part.end());
  };
  add(pb.meta, &ref->meta_off, &ref->meta_bytes);
  for (int i = 0; i < 3; ++i) {
    add(pb.w[i], &ref->w_off[i], &ref->w_bytes[i]);
    ref->k_slices[i] = pb.k_slices[i];
  }
  blob.resize(up((uint32_t)blob.size(), kAlign), 0);
}

struct Dims { int n1, n2, n3, kd1, kd2, kd3; };

PackedBlock pack_coupling(const iodf_coupling_desc& cp, const Blobs& B, int ca, int cb, const int* colA,
                          const int* colB, Act a1, Act a2, Dims* dims) {
  const iodf_layer_desc& L1 = cp.layers[0];
  const iodf_layer_desc& L2 = cp.layers[1];
  const iodf_layer_desc& L3 = cp.layers[2];
  const int k1 = (int)L1.c_out, k2 = (int)L2.c_out;
  const int cpad = (int)up(ca, 8), cbp = (int)up(cb, 8);
  Dims d;
  d.n1 = (int)up(k1, 16); d.n2 = (int)up(k2, 16); d.n3 = (int)up(9 * cbp, 16);
  // K of the first two GEMMs leaves room for the kBiasRows constant columns after the data
  d.kd1 = (int)up(9 * cpad + kBiasRows, 32); d.kd2 = (int)up(d.n1 + kBiasRows, 32); d.kd3 = (int)up(k2, 32);
  *dims = d;
  PackedBlock pb;
  CouplingMeta M{};
  M.in_m0 = cp.in_m0; M.in_s = cp.in_s;
  M.n1 = d.n1; M.n2 = d.n2; M.kd1 = d.kd1; M.kd2 = d.kd2; M.kd3 = d.kd3; M.n3 = d.n3;
  M.lo1 = a1.lo; M.hi1 = a1.hi; M.lo2 = a2.lo; M.hi2 = a2.hi;
  // requantisation tables: both flavours are built, only the one the layer's mode reads is kept
  std::vector<HiddenRq> h1(d.n1), h2(d.n2);
  std::vector<int32_t> u1(2 * d.n1), u2(2 * d.n2);
  put_hidden_rq(h1.data(), u1.data(), L1, B, d.n1, &M.mode1, &M.us1);
  put_hidden_rq(h2.data(), u2.data(), L2, B, d.n2, &M.mode2, &M.us2);
  uint32_t off = sizeof(CouplingMeta);
  M.off_colA = (int)off; off += up(4 * ca, 16);
  M.off_colB = (int)off; off += up(4 * cb, 16);
  M.off_out = (int)off;  off += (uint32_t)sizeof(OutRq) * cb;
  auto table_bytes = [](int mode, int n) { return mode == 3 ? 4u * n : mode == 2 ? 8u * n : (uint32_t)sizeof(HiddenRq) * n; };
  M.off_h1 = M.off_u1 = (int)off; off += table_bytes(M.mode1, d.n1);
  M.off_h2 = M.off_u2 = (int)off; off += table_bytes(M.mode2, d.n2);
  pb.meta.assign(off, 0);
  std::memcpy(pb.meta.data() + M.off_colA, colA, 4 * ca);
  std::memcpy(pb.meta.data() + M.off_colB, colB, 4 * cb);
  put_out_rq(reinterpret_cast<OutRq*>(pb.meta.data() + M.off_out), L3, B);
  if (M.mode1 >= 2) std::memcpy(pb.meta.data() + M.off_u1, u1.data(), table_bytes(M.mode1, d.n1));
  else std::memcpy(pb.meta.data() + M.off_h1, h1.data(), sizeof(HiddenRq) * d.n1);
  if (M.mode2 >= 2) std::memcpy(pb.meta.data() + M.off_u2, u2.data(), table_bytes(M.mode2, d.n2));
  else std::memcpy(pb.meta.data() + M.off_h2, h2.data(), sizeof(HiddenRq) * d.n2);
  std::memcpy(pb.meta.data(), &M, sizeof(M));

  pb.k_slices[0] = d.kd1 / 32; pb.k_slices[1] = d.kd2 / 32; pb.k_slices[2] = d.kd3 / 32;
  // W1: row = hidden channel, K index = tap*cpad + c
  pb.w[0].assign((size_t)d.n1 * d.kd1, 0);
  const int8_t* w1 = B.w + L1.weight_off;
  for (int n = 0; n < k1; ++n)
    for (int tap = 0; tap < 9; ++tap)
      for (int c = 0; c < ca; ++c)
        pb.w[0][wpos(d.n1, n, tap * cpad + c)] = (uint8_t)w1[((size_t)n * 9 + tap) * ca + c];
  if (M.mode1 == 3) {            // bias rows right after the nine taps
    const int32_t* b1 = B.r + L1.requant_off;
    for (int n = 0; n < k1; ++n) {
      int8_t bw[kBiasRows];
      fold_bias(b1[n], bw);
      for (int j = 0; j < kBiasRows; ++j) pb.w[0][wpos(d.n1, n, 9 * cpad + j)] = (uint8_t)bw[j];
    }
  }
  // W2: 1x1
  pb.w[1].assign((size_t)d.n2 * d.kd2, 0);
  const int8_t* w2 = B.w + L2.weight_off;
  for (int n = 0; n < k2; ++n)
    for (int k = 0; k < k1; ++k) pb.w[1][wpos(d.n2, n, k)] = (uint8_t)w2[(size_t)n * k1 + k];
  if (M.mode2 == 3) {            // bias rows right after the (padded) hidden channels
    const int32_t* b2 = B.r + L2.requant_off;
    for (int n = 0; n < k2; ++n) {
      int8_t bw[kBiasRows];
      fold_bias(b2[n], bw);
      for (int j = 0; j < kBiasRows; ++j) pb.w[1][wpos(d.n2, n, d.n1 + j)] = (uint8_t)bw[j];
    }
  }
  // W3': row = tap*cbp + c, K index = hidden channel
  pb.w[2].assign((size_t)d.n3 * d.kd3, 0);
  const int8_t* w3 = B.w + L3.weight_off;
  for (int c = 0; c < cb; ++c)
    for (int tap = 0; tap < 9; ++tap)
      for (int k = 0; k < k2; ++k)
        pb.w[2][wpos(d.n3, tap * cbp + c, k)] = (uint8_t)w3[((size_t)c * 9 + tap) * k2 + k];
  return pb;
}

PackedBlock pack_prior(const iodf_level_desc& lv, const Blobs& B, int ca, int cb, int* n_out, int* kd_out) {
  const iodf_layer_desc& L = lv.prior_layer;
  const int cpad = (int)up(ca, 8);
  PackedBlock pb;
  PriorMeta M{};
  M.in_m0 = lv.prior_in_m0; M.in_s = lv.prior_in_s;
  M.n = (int)up(2 * cb, 16);
  M.kd = (int)up(9 * cpad, 32);
  M.ls_lo = lv.ls_lo; M.ls_hi = lv.ls_hi;
  M.off_out = (int)sizeof(PriorMeta);
  pb.meta.assign(sizeof(PriorMeta) + sizeof(OutRq) * 2 * cb, 0);
  put_out_rq(reinterpret_cast<OutRq*>(pb.meta.data() + M.off_out), L, B);
  std::memcpy(pb.meta.data(), &M, sizeof(M));
  pb.k_slices[0] = M.kd / 32;
  pb.w[0].assign((size_t)M.n * M.kd, 0);
  const int8_t* w = B.w + L.weight_off;
  for (int o = 0; o < 2 * cb; ++o)
    for (int tap = 0; tap < 9; ++tap)
      for (int c = 0; c < ca; ++c)
        pb.w[0][wpos(M.n, o, tap * cpad + c)] = (uint8_t)w[((size_t)o * 9 + tap) * ca + c];
  *n_out = M.n;
  *kd_out = M.kd;
  return pb;
}

uint32_t pow2_cols(uint32_t need) {
  uint32_t c = 32;
  while (c < need) c <<= 1;
  return c;
}

// Levels of at least this many tiles per CTA run in the kernel that splits a tile's work by role
// (level_pipe.cu) when they are eligible for it. Measured on the ImageNet64-shaped flow: 5 % faster
// than the general kernel at eight tiles per image, 5 % slower at two (nothing follows the one
// pair of tiles that the role split could overlap with).
#ifndef IODF_PIPE_MIN_TILES
#define IODF_PIPE_MIN_TILES 4
#endif
constexpr int kPipeMinTiles = IODF_PIPE_MIN_TILES;

// What that kernel needs to know about a level.
struct PipeDims {
  bool eligible = false;           // every coupling in the folded flavour with the 0..127 clip
  uint32_t a1_bytes = 16;          // im2col operand of a tile (couplings and prior head)
  uint32_t n_hidden = 0;           // widest accumulator of the first two GEMMs (and of the prior head)
  uint32_t n_taps = 0;             // accumulator of the third GEMM: nine taps x padded C/2
};

// Choose images per CTA, tiles in flight and the shared-memory layout. Returns false if nothing fits.
//   pipe:   two tile slots, every weight matrix resident, the work of a tile split by role
//           (level_pipe.cu; needs an eligible level of several tiles per CTA)
//   mode 0: two tile slots, every weight matrix resident      (needs all N <= 256 and >= 2 tiles)
//   mode 1: one tile slot, every weight matrix resident
//   mode 2: one tile slot, W1 and W3 share a slot and are re-fetched per tile
//   mode 3: one tile slot, weights streamed per tile in 32-byte K-slices through a small ring
//           (the only mode for hidden widths above 256: a 512 x 512 matrix alone is 256 KB)
bool plan_smem(LevelPlan& P, uint32_t a_bytes, uint32_t meta_bytes, const uint32_t wmax[3], uint32_t n_max,
               uint32_t limit, uint32_t max_batch, int num_sms, const PipeDims& pd, bool throughput) {
  int group = P.px >= kTileM ? 1 : kTileM / P.px;
  group = std::max(1, std::min<int>(group, (int)max_batch));
  // A level's time is set by the serial chain of its couplings inside one CTA, not by how many
  // rows of the 128-row tile are filled: while the CTAs of a full batch would not fill the SMs,
  // smaller groups (more CTAs, emptier tiles) are faster. The throughput plan keeps the tile as
  // full as the resident-weight modes allow instead: the step is a little longer, but a launch takes
  // a half to a quarter of the CTAs, which leaves SMs to the other batches a caller has in flight.
  while (!throughput && group > 1 && ((int)max_batch + group - 1) / group < num_sms) group /= 2;
  for (; group >= 1; group = (group > 1 ? group / 2 : 0)) {
    const int tiles = (group * P.px + kTileM - 1) / kTileM;
    // the role-split kernel first with im2col buffers of its own (mode -2), then sharing the slot's buffer (-1)
    for (int mode = -2; mode < 4; ++mode) {
      const bool pipe = mode < 0;
      // per-tap partials in columns of their own when two slots of both kinds fit the 512 columns
      const bool r3_separate = 2u * pd.n_hidden + 2u * pd.n_taps <= 512u;
      if (pipe && (!pd.eligible || tiles < kPipeMinTiles || std::max(pd.n_hidden, pd.n_taps) > (uint32_t)kSlotCols)) continue;
      if (mode == 0 && (tiles < 2 || n_max > (uint32_t)kSlotCols)) continue;
      if (mode >= 0 && mode < 3 && n_max > 2u * kSlotCols) continue;
      if (mode == 3 && n_max <= (uint32_t)kSlotCols) continue;   // resident weights are faster when they fit
      if (mode == 3 && throughput && group > 1) continue;        // streamed weights cost more than the fuller tile saves
      const uint32_t pg = up((uint32_t)group * P.px, 32);
      uint32_t off = 0;
      auto take = [&](uint32_t bytes) { uint32_t o = off; off = up(off + bytes, kAlign); return o; };
      P.s_v = take((uint32_t)P.c * pg * 4);
      P.s_xa = take(pg * (uint32_t)P.cpad);
      P.s_acc = take((uint32_t)P.cb * pg * 4);
      P.s_rowinfo = take((uint32_t)tiles * kTileM * 4);
      P.s_gran = take((uint32_t)P.n_gran * 8);
      P.s_a[0] = take(a_bytes);
      P.s_a[1] = (pipe || mode == 0) ? take(a_bytes) : P.s_a[0];
      P.s_a1[0] = mode == -2 ? take(pd.a1_bytes) : P.s_a[0];
      P.s_a1[1] = mode == -2 ? take(pd.a1_bytes) : P.s_a[1];
      P.s_meta[0] = take(meta_bytes);
      P.s_meta[1] = take(meta_bytes);
      P.ring_slot_bytes = up(32u * n_max, kAlign);
      if (mode == 3) {
        P.s_w[0] = take(P.ring_slot_bytes * kRingDepth);
        P.s_w[1] = P.s_w[2] = P.s_w[0];
      } else {
        P.s_w[0] = take(mode == 2 ? std::max(wmax[0], wmax[2]) : wmax[0]);
        P.s_w[1] = take(wmax[1]);
        P.s_w[2] = mode == 2 ? P.s_w[0] : take(wmax[2]);
      }
      P.s_total = off;
      P.pipe = pipe ? 1 : 0;
      P.lean = (pd.eligible && mode != 3) ? 1 : 0;
      P.r_col[0] = r3_separate ? (int)pd.n_hidden : kSlotCols;
      P.r_col[1] = r3_separate ? 2 * (int)pd.n_hidden : 0;
      P.r_col[2] = r3_separate ? (int)pd.n_taps : kSlotCols;
      P.w13_alias = mode == 2;
      P.streamed = mode == 3;
      P.nslots = mode == 0 ? 2 : 1;
      P.tmem_cols = (int)(pipe ? 512 : (mode == 0 ? 2 * kSlotCols : pow2_cols(n_max)));
      P.group = group;
      P.pg = (int)pg;
      P.tiles = tiles;
      P.rep = tiles == 1 ? (group * P.px <= kTileM / 4 ? 4 : (group * P.px <= kTileM / 2 ? 2 : 1)) : 1;
      if (off <= limit) return true;
    }
    if (group == 1) break;
  }
  return false;
}

int cuda_fail(iodf_model* m, cudaError_t e) {
  if (m) m->last_cuda = (int)e;
  return e == cudaErrorMemoryAllocation ? IODF_ENOMEM : IODF_ECUDA;
}

#define CU(m, x)                                   \
  do {                                             \
    cudaError_t e__ = (x);                         \
    if (e__ != cudaSuccess) return cuda_fail(m, e__); \
  } while (0)

// Row bands of an image at a residual level: 1 while the whole image fits one CTA, otherwise the
// smallest power of two that brings a band down to kResMaxPixels pixels (bands of at least two rows;
// 0 if there is none up to kResMaxBands).
int residual_bands(uint32_t h, uint32_t w) {
  for (uint32_t nb = 1; nb <= (uint32_t)kResMaxBands; nb *= 2)
    if (h % nb == 0 && (nb == 1 || h / nb >= 2) && (h / nb) * w <= (uint32_t)kResMaxPixels) return (int)nb;
  return 0;
}

// A coupling with residual blocks (layers already checked one by one): shapes, ranges and what this
// build runs.
int check_residual(const iodf_coupling_desc& cp, const Blobs& B, uint32_t ca, uint32_t cb, uint32_t h, uint32_t w) {
  if (!cp.blocks || cp.n_layers != 2 + 2 * cp.n_blocks) return IODF_EINVAL;
  const iodf_layer_desc& cin = cp.layers[0];
  const iodf_layer_desc& cout = cp.layers[cp.n_layers - 1];
  const uint32_t D = cin.c_out;
  if (cin.c_in != ca || cout.c_in != D || cout.c_out != cb || cout.relu || cout.has_clamp) return IODF_EINVAL;
  for (uint32_t b = 0; b < cp.n_blocks; ++b) {
    const iodf_layer_desc& la = cp.layers[1 + 2 * b];
    const iodf_layer_desc& lb = cp.layers[2 + 2 * b];
    const iodf_resblock_desc& rb = cp.blocks[b];
    if (la.c_in != D || lb.c_in != la.c_out || lb.relu || lb.has_clamp) return IODF_EINVAL;
    if (!rb.idx || rb.n_idx != lb.c_out || rb.short_m0 < (1 << 30) || rb.short_s < 0 || rb.short_s > 31 ||
        rb.clamp_lo > rb.clamp_hi)
      return IODF_EINVAL;
    std::vector<char> used(D, 0);
    for (uint32_t j = 0; j < rb.n_idx; ++j) {
      if (rb.idx[j] < 0 || rb.idx[j] >= (int32_t)D || used[rb.idx[j]]) return IODF_EINVAL;
      used[rb.idx[j]] = 1;
    }
  }
  // what the residual kernel runs
  if (residual_bands(h, w) == 0) return IODF_EUNSUPPORTED;
  for (uint32_t q = 0; q < cp.n_layers; ++q) {
    const iodf_layer_desc& L = cp.layers[q];
    if (L.k != 3 || L.c_out > (uint32_t)kResMaxWidth || L.c_in > (uint32_t)kResMaxWidth) return IODF_EUNSUPPORTED;
    const bool hidden = q == 0 || (q + 1 < cp.n_layers && q % 2 == 1);      // conv_in and every conv_a
    if (hidden) {
      Act a;
      int rc = hidden_range(L, &a);
      if (rc) return rc;
      if (a.lo != 0 || a.hi != 255) return IODF_EUNSUPPORTED;
    }
    int rc = check_overflow(L, B, q == 0 ? 128 : 255);
    if (rc) return rc;
  }
  for (uint32_t b = 0; b < cp.n_blocks; ++b)
    if (cp.blocks[b].clamp_lo != 0 || cp.blocks[b].clamp_hi != 255) return IODF_EUNSUPPORTED;
  return IODF_OK;
}

// Level blob of a residual level: ResHead, coupling records, conv records, then tables and weights.
int pack_residual_level(const iodf_level_desc& lv, const Blobs& B, LevelPlan& P, std::vector<uint8_t>& blob,
                        const std::vector<std::vector<int>>& cols, uint32_t smem_limit, uint32_t max_batch,
                        bool throughput) {
  const int ca = P.ca, cb = P.cb, px = P.px;
  std::vector<ResCouplingRec> cps(lv.n_couplings);
  std::vector<ResConv> convs;
  int maxD = 32, maxK = 32, kmax = 32, nmax = 16;
  struct Src { const iodf_layer_desc* L; };
  std::vector<const iodf_layer_desc*> conv_layer;
  // `n`: outputs the kernel computes (a block's second conv is widened to the D channels it is added to)
  auto add_conv = [&](const iodf_layer_desc& L, int kind, int src, int dst, bool a_unsigned, uint32_t n = 0) {
    ResConv c{};
    if (n == 0) n = L.c_out;
    c.n = (int)n; c.n_pad = (int)up(n, 16); c.kpad = (int)up(L.c_in, 32);
    c.a_unsigned = a_unsigned; c.kind = kind; c.src = src; c.dst = dst;
    c.slice_bytes = (uint32_t)c.n_pad * (uint32_t)c.kpad;
    kmax = std::max(kmax, c.kpad); nmax = std::max(nmax, c.n_pad);
    convs.push_back(c);
    conv_layer.push_back(&L);
    return (int)convs.size() - 1;
  };
  for (uint32_t ki = 0; ki < lv.n_couplings; ++ki) {
    const iodf_coupling_desc& cp = lv.couplings[ki];
    cps[ki].in_m0 = cp.in_m0; cps[ki].in_s = cp.in_s;
    cps[ki].conv0 = (int)convs.size(); cps[ki].n_convs = (int)cp.n_layers;
    maxD = std::max(maxD, (int)up(cp.layers[0].c_out, 32));
    add_conv(cp.layers[0], kResHidden, 0, 1, false);
    for (uint32_t b = 0; b < cp.n_blocks; ++b) {
      maxK = std::max(maxK, (int)up(cp.layers[1 + 2 * b].c_out, 32));
      add_conv(cp.layers[1 + 2 * b], kResHidden, 1, 2, true);
      const int j = add_conv(cp.layers[2 + 2 * b], kResBranch, 2, 1, true, cp.layers[0].c_out);
      convs[j].short_m0 = cp.blocks[b].short_m0; convs[j].short_s = cp.blocks[b].short_s;
    }
    add_conv(cp.layers[cp.n_layers - 1], kResOut, 1, 1, true);
  }
  int prior_conv = -1;
  if (lv.has_prior) prior_conv = add_conv(lv.prior_layer, kResPrior, 0, 0, false);

  ResHead H{};
  H.n_couplings = (int)lv.n_couplings; H.n_convs = (int)convs.size(); H.prior_conv = prior_conv;
  H.prior_in_m0 = lv.prior_in_m0; H.prior_in_s = lv.prior_in_s; H.ls_lo = lv.ls_lo; H.ls_hi = lv.ls_hi;
  H.xa_pitch = (int)up(ca, 32); H.x_pitch = maxD; H.mid_pitch = maxK;
  auto place = [&](size_t bytes) { blob.resize(up((uint32_t)blob.size(), kAlign), 0); uint32_t o = (uint32_t)blob.size(); blob.resize(o + bytes, 0); return o; };
  blob.clear();
  place(sizeof(ResHead));
  H.coupling_off = place(sizeof(ResCouplingRec) * cps.size());
  H.conv_off = place(sizeof(ResConv) * convs.size());
  for (uint32_t ki = 0; ki < lv.n_couplings; ++ki) {
    cps[ki].colA_off = place(4 * (size_t)ca);
    std::memcpy(blob.data() + cps[ki].colA_off, cols[ki].data(), 4 * (size_t)ca);
    cps[ki].colB_off = place(4 * (size_t)cb);
    std::memcpy(blob.data() + cps[ki].colB_off, cols[ki].data() + ca, 4 * (size_t)cb);
  }
  // per conv: requantisation constants, index list, nine weight slices
  size_t block_of_branch = 0;
  std::vector<const iodf_resblock_desc*> branch_block;
  for (uint32_t ki = 0; ki < lv.n_couplings; ++ki)
    for (uint32_t b = 0; b < lv.couplings[ki].n_blocks; ++b) branch_block.push_back(&lv.couplings[ki].blocks[b]);
  for (size_t ci = 0; ci < convs.size(); ++ci) {
    ResConv& c = convs[ci];
    const iodf_layer_desc& L = *conv_layer[ci];
    c.rq_off = place(sizeof(OutRq) * (size_t)c.n_pad);
    std::vector<OutRq> rq(c.n_pad, OutRq{1 << 30, 0, 1u << 30, 0u});          // padding: 0 -> 0
    // Scatter add (Sec. 4.5) at pack time: filter j of a block's second conv becomes row idx[j] of a
    // conv as wide as the shortcut. Rows without a filter have zero weights, no bias and requantise 0
    // to 0, so the sum is the same and the kernel adds sixteen adjacent channels at a time.
    const int32_t* row_of = nullptr;
    if (c.kind == kResBranch) row_of = branch_block[block_of_branch++]->idx;
    if (row_of) {
      std::vector<OutRq> compact(L.c_out);
      put_out_rq(compact.data(), L, B);
      for (uint32_t j = 0; j < L.c_out; ++j) rq[row_of[j]] = compact[j];
    } else {
      put_out_rq(rq.data(), L, B);
    }
    std::memcpy(blob.data() + c.rq_off, rq.data(), sizeof(OutRq) * rq.size());
    c.w_off = place(9 * (size_t)c.slice_bytes);
    const int8_t* w = B.w + L.weight_off;
    for (int tap = 0; tap < 9; ++tap) {
      uint8_t* sl = blob.data() + c.w_off + (size_t)tap * c.slice_bytes;
      for (uint32_t n = 0; n < L.c_out; ++n)
        for (uint32_t k = 0; k < L.c_in; ++k)
          sl[wpos(c.n_pad, row_of ? row_of[n] : (int)n, (int)k)] = (uint8_t)w[((size_t)n * 9 + tap) * L.c_in + k];
    }
  }
  // shared memory: flow variable, the three activation buffers in the padded chunk-major layout
  // (cleared together at kernel start), position table, conv tables, weight ring
  // one CTA per image, or per band of hb rows (a cluster of `bands` CTAs per image)
  const int bands = residual_bands((uint32_t)P.h, (uint32_t)P.w);
  if (bands == 0) return IODF_EUNSUPPORTED;
  const int hb = P.h / bands;
  (void)px;
  const int w2 = P.w + 2, guard = w2 + 1;
  // images per CTA: one, or (throughput plan, whole images) as many frames as one tile holds and as
  // leave the weight ring two slots
  int group = 1;
  if (throughput && bands == 1) group = std::max(1, std::min<int>(kTileM / ((hb + 2) * w2), (int)max_batch));
  uint32_t pg = 0, off = 0;
  int ntiles = 0, rows = 0;
  for (;; --group) {
    pg = up((uint32_t)(group * hb * P.w), 32);
    ntiles = (int)(up((uint32_t)(group * (hb + 2) * w2), kTileM) / kTileM);
    rows = guard + ntiles * kTileM + w2 + 1;
    off = 0;
    auto take = [&](uint32_t bytes) { uint32_t o = off; off = up(off + bytes, kAlign); return o; };
    H.s_v = take((uint32_t)P.c * pg * 4);
    H.s_xa = take((uint32_t)(H.xa_pitch / 16) * rows * 16);
    H.s_x = take((uint32_t)(H.x_pitch / 16) * rows * 16);
    H.s_mid = take((uint32_t)(H.mid_pitch / 16) * rows * 16);
    H.s_rowinfo = take((uint32_t)ntiles * kTileM * 8);     // pixel and edge-row tables
    H.s_tab = take((uint32_t)kResMaxWidth * (sizeof(OutRq) + sizeof(int32_t)) + 256);   // + the shortcut table
    // as deep a weight ring as fits (at least two slots)
    H.w_slot_bytes = up((uint32_t)nmax * kmax, kAlign);
    H.n_wslots = kResMaxWSlots;
    while (H.n_wslots > 2 && off + (uint32_t)H.n_wslots * H.w_slot_bytes > smem_limit) --H.n_wslots;
    H.s_wring = take((uint32_t)H.n_wslots * H.w_slot_bytes);
    if (off <= smem_limit || group == 1) break;
  }
  H.w2 = w2; H.guard = guard; H.rows = rows; H.ntiles = ntiles;
  H.bands = bands; H.hb = hb; H.group = group;
  H.s_total = off;
  // one tile: every issuing warp keeps a partial accumulator of its own
  H.tmem_cols = (ntiles > 2 || ntiles == 1) ? 4 * kResMaxWidth : 2 * kResMaxWidth;
  if (off > smem_limit || ntiles > 4 || rows * 16 >= (1 << 18)) return IODF_EUNSUPPORTED;
  std::memcpy(blob.data(), &H, sizeof(H));
  std::memcpy(blob.data() + H.coupling_off, cps.data(), sizeof(ResCouplingRec) * cps.size());
  std::memcpy(blob.data() + H.conv_off, convs.data(), sizeof(ResConv) * convs.size());
  P.residual = 1;
  P.res_bands = bands;
  P.group = group; P.pg = (int)pg; P.tiles = ntiles; P.rep = 1; P.nslots = 1;
  P.s_total = H.s_total;
  return IODF_OK;
}

int build_model(const iodf_model_desc* desc, const Blobs& B, int device, iodf_model* m) {
  if (desc->abi_version != IODF_ABI_VERSION) return IODF_EVERSION;
  if (!desc->levels || desc->n_levels < 1 || desc->n_levels > IODF_MAX_LEVELS || desc->max_batch < 1 ||
      desc->in_c < 1 || desc->in_h < 1 || desc->in_w < 1 || desc->plan > IODF_PLAN_THROUGHPUT)
    return IODF_EINVAL;
  if ((desc->in_h % (1u << desc->n_levels)) || (desc->in_w % (1u << desc->n_levels))) return IODF_EINVAL;
  m->device = device;
  m->max_batch = desc->max_batch;
  m->in_c = desc->in_c; m->in_h = desc->in_h; m->in_w = desc->in_w;

  iodf_layout& lay = m->layout;
  lay = iodf_layout{};
  lay.n_levels = desc->n_levels;
  lay.d = (uint64_t)desc->in_c * desc->in_h * desc->in_w;

  // pass 1: shapes, validation, latent layout
  uint32_t c = desc->in_c, h = desc->in_h, w = desc->in_w;
  uint64_t zo = 0, po = 0;
  for (uint32_t li = 0; li < desc->n_levels; ++li) {
    const iodf_level_desc& lv = desc->levels[li];
    c *= 4; h /= 2; w /= 2;
    if (c % 2 || c > (uint32_t)kMaxC) return c % 2 ? IODF_EINVAL : IODF_EUNSUPPORTED;
    if (lv.n_couplings > (uint32_t)kMaxCouplings) return IODF_EUNSUPPORTED;
    if (lv.n_couplings && !lv.couplings) return IODF_EINVAL;
    if (lv.has_prior && !lv.split) return IODF_EINVAL;
    lay.level_c[li] = c; lay.level_h[li] = h; lay.level_w[li] = w;
    lay.z_off[li] = zo; lay.prior_off[li] = po;
    const uint32_t ca = c / 2, cb = c - ca, px = h * w;
    for (uint32_t ki = 0; ki < lv.n_couplings; ++ki) {
      const iodf_coupling_desc& cp = lv.couplings[ki];
      if (!cp.perm || !cp.layers) return IODF_EINVAL;
      std::vector<char> seen(c, 0);
      for (uint32_t k = 0; k < c; ++k) {
        if (cp.perm[k] < 0 || cp.perm[k] >= (int32_t)c || seen[cp.perm[k]]) return IODF_EINVAL;
        seen[cp.perm[k]] = 1;
      }
      if (cp.in_m0 < (1 << 30) || cp.in_s < 0 || cp.in_s > 31) return IODF_EINVAL;
      if (cp.n_layers < 1) return IODF_EINVAL;
      uint32_t cin = ca;
      for (uint32_t q = 0; q < cp.n_layers; ++q) {
        int rc = check_layer(cp.layers[q], B);
        if (rc) return rc;
        if (cp.n_blocks == 0 && cp.layers[q].c_in != cin) return IODF_EINVAL;
        cin = cp.layers[q].c_out;
      }
      if (cp.n_blocks > 0) {
        int rc = check_residual(cp, B, ca, cb, h, w);
        if (rc) return rc;
        if (ki > 0 && lv.couplings[0].n_blocks == 0) return IODF_EUNSUPPORTED;    // one kind per level
        for (uint32_t q = 0; q < cp.n_layers; ++q)
          lay.macs_per_image += (uint64_t)px * 9 * cp.layers[q].c_in * cp.layers[q].c_out;
        continue;
      }
      if (lv.couplings[0].n_blocks > 0) return IODF_EUNSUPPORTED;
      if (cin != cb) return IODF_EINVAL;
      const iodf_layer_desc& last = cp.layers[cp.n_layers - 1];
      if (last.relu || last.has_clamp) return IODF_EINVAL;
      // the shape this build runs
      if (cp.n_layers != 3 || cp.layers[0].k != 3 || cp.layers[1].k != 1 || cp.layers[2].k != 3)
        return IODF_EUNSUPPORTED;
      if (cp.layers[0].c_out > (uint32_t)kMaxHidden || cp.layers[1].c_out > (uint32_t)kMaxHidden)
        return IODF_EUNSUPPORTED;
      Act a1, a2;
      int rc = hidden_range(cp.layers[0], &a1);
      if (rc) return rc;
      rc = hidden_range(cp.layers[1], &a2);
      if (rc) return rc;
      if ((rc = check_overflow(cp.layers[0], B, 128))) return rc;
      if ((rc = check_overflow(cp.layers[1], B, std::max(std::abs(a1.lo), std::abs(a1.hi))))) return rc;
      if ((rc = check_overflow(cp.layers[2], B, std::max(std::abs(a2.lo), std::abs(a2.hi))))) return rc;
      for (uint32_t q = 0; q < cp.n_layers; ++q)
        lay.macs_per_image += (uint64_t)px * cp.layers[q].k * cp.layers[q].k * cp.layers[q].c_in * cp.layers[q].c_out;
    }
    if (lv.has_prior) {
      const iodf_layer_desc& L = lv.prior_layer;
      int rc = check_layer(L, B);
      if (rc) return rc;
      if (L.c_in != ca || L.c_out != 2 * cb) return IODF_EINVAL;
      if (lv.prior_in_m0 < (1 << 30) || lv.prior_in_s < 0 || lv.prior_in_s > 31 || lv.ls_lo > lv.ls_hi)
        return IODF_EINVAL;
      if (L.k != 3 || L.relu || L.has_clamp) return IODF_EUNSUPPORTED;
      if ((rc = check_overflow(L, B, 128))) return rc;
      lay.macs_per_image += (uint64_t)px * 9 * L.c_in * L.c_out;
    }
    if (lv.split) {
      zo += (uint64_t)cb * px;
      if (lv.has_prior) po += (uint64_t)cb * px;
      c = ca;
    }
  }
  lay.z_final_off = zo;
  lay.d_fact = po;
  if (zo + (uint64_t)c * h * w != lay.d) return IODF_EINVAL;

  // Everything above is host-only, so a malformed descriptor is reported even without a device.
  int smem_limit = 0;
  CU(m, cudaSetDevice(device));
  CU(m, cudaDeviceGetAttribute(&smem_limit, cudaDevAttrMaxSharedMemoryPerBlockOptin, device));
  smem_limit -= 1024;   // static control block and alignment slack
  int num_sms = 1;
  CU(m, cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, device));

  // pass 2: pack and plan
  m->levels.resize(desc->n_levels);
  c = desc->in_c; h = desc->in_h; w = desc->in_w;
  uint32_t max_smem = 0;
  for (uint32_t li = 0; li < desc->n_levels; ++li) {
    const iodf_level_desc& lv = desc->levels[li];
    HostLevel& hl = m->levels[li];
    LevelPlan& P = hl.plan;
    std::memset(&P, 0, sizeof(P));
    c *= 4; h /= 2; w /= 2;
    const int ca = (int)c / 2, cb = (int)c - ca;
    P.c = (int)c; P.h = (int)h; P.w = (int)w; P.px = (int)(h * w); P.ca = ca; P.cb = cb;
    P.n_couplings = (int)lv.n_couplings;
    P.split = lv.split ? 1 : 0; P.has_prior = lv.has_prior ? 1 : 0;
    hl.ls_lo = lv.ls_lo; hl.ls_hi = lv.ls_hi;
    P.is_first = li == 0; P.is_last = li + 1 == desc->n_levels;
    P.keep_c = lv.split ? ca : (int)c;
    P.z_off = lay.z_off[li]; P.prior_off = lay.prior_off[li]; P.z_final_off = lay.z_final_off;
    P.d = lay.d; P.d_fact = lay.d_fact;

    P.cpad = (int)up(ca, 8); P.cbp = (int)up(cb, 8);
    auto magic = [](uint64_t d) -> uint32_t { return d <= 1 ? 0u : (uint32_t)(((1ull << 32) + d - 1) / d); };
    P.mul_per_img = magic((uint64_t)c * h * w); P.mul_4px = magic(4ull * h * w); P.mul_w2 = magic(2ull * w);
    P.mul_px = magic((uint64_t)h * w); P.mul_w = magic(w);
    P.recip_gpa = 65536u / (uint32_t)(P.cpad / 8) + 1u;
    P.recip_gpb = 65536u / (uint32_t)(P.cbp / 8) + 1u;
    std::vector<int> pi(c);
    for (uint32_t k = 0; k < c; ++k) pi[k] = (int)k;
    if (lv.n_couplings > 0 && lv.couplings[0].n_blocks > 0) {
      std::vector<std::vector<int>> cols;
      for (uint32_t ki = 0; ki < lv.n_couplings; ++ki) {
        const iodf_coupling_desc& cp = lv.couplings[ki];
        std::vector<int> nxt(c);
        for (uint32_t k = 0; k < c; ++k) nxt[k] = pi[cp.perm[k]];
        pi.swap(nxt);
        cols.push_back(pi);
      }
      for (int k = 0; k < (int)c; ++k) P.col_out[k] = pi[k];
      int rc = pack_residual_level(lv, B, P, hl.blob, cols, (uint32_t)smem_limit, desc->max_batch,
                                   desc->plan == IODF_PLAN_THROUGHPUT);
      if (rc) return rc;
      if ((uint64_t)P.group * c * h * w * ((uint64_t)c * h * w) >= (1ull << 32)) return IODF_EUNSUPPORTED;
      if (lv.split) c = (uint32_t)ca;
      continue;
    }
    uint32_t a_bytes = 16, meta = 16, wmax[3] = {16, 16, 16};
    uint32_t n_max = 32;
    PipeDims pd;
    pd.eligible = lv.n_couplings > 0;
    std::vector<PackedBlock> blocks;
    for (uint32_t ki = 0; ki < lv.n_couplings; ++ki) {
      const iodf_coupling_desc& cp = lv.couplings[ki];
      std::vector<int> nxt(c);
      for (uint32_t k = 0; k < c; ++k) nxt[k] = pi[cp.perm[k]];
      pi.swap(nxt);
      Act a1, a2r;
      hidden_range(cp.layers[0], &a1);
      hidden_range(cp.layers[1], &a2r);
      Dims d;
      blocks.push_back(pack_coupling(cp, B, ca, cb, pi.data(), pi.data() + ca, a1, a2r, &d));
      a_bytes = std::max<uint32_t>(a_bytes, kTileM * std::max(d.kd1, std::max(d.kd2, d.kd3)));
      n_max = std::max<uint32_t>(n_max, std::max(d.n1, std::max(d.n2, d.n3)));
      const CouplingMeta* cm = reinterpret_cast<const CouplingMeta*>(blocks.back().meta.data());
      if (cm->mode1 != 3 || cm->mode2 != 3 || a1.lo != 0 || a1.hi != 127 || a2r.lo != 0 || a2r.hi != 127) pd.eligible = false;
      pd.n_hidden = std::max<uint32_t>(pd.n_hidden, (uint32_t)std::max(d.n1, d.n2));
      pd.a1_bytes = std::max<uint32_t>(pd.a1_bytes, (uint32_t)kTileM * d.kd1);
      pd.n_taps = std::max<uint32_t>(pd.n_taps, (uint32_t)d.n3);
    }
    for (int k = 0; k < (int)c; ++k) P.col_out[k] = pi[k];
    PackedBlock prior_block;
    if (lv.has_prior) {
      int n, kd;
      prior_block = pack_prior(lv, B, ca, cb, &n, &kd);
      a_bytes = std::max<uint32_t>(a_bytes, kTileM * kd);
      n_max = std::max<uint32_t>(n_max, n);
      pd.n_hidden = std::max<uint32_t>(pd.n_hidden, (uint32_t)n);
      pd.a1_bytes = std::max<uint32_t>(pd.a1_bytes, (uint32_t)kTileM * kd);
    }
    if (n_max > 512) return IODF_EUNSUPPORTED;
    {   // im2col granule table of the level's first convs (couplings and prior head share it)
      const int gpt = P.cpad / 8, ndata = 9 * gpt;
      P.n_gran = (int)up((uint32_t)(ndata + 1), 4);
      if (P.n_gran > kMaxGran) return IODF_EUNSUPPORTED;
      for (int g = 0; g < P.n_gran; ++g) {
        int off = 0, sel = g == ndata ? kGranBias : kGranPad;
        if (g < ndata) {
          const int tap = g / gpt, i = g % gpt, u = tap / 3, v = tap % 3;
          off = ((u - 1) * (int)w + (v - 1)) * P.cpad + 8 * i;
          sel = tap;
        }
        P.gran_tab[2 * g] = off;
        P.gran_tab[2 * g + 1] = sel;
      }
    }
    for (uint32_t ki = 0; ki < lv.n_couplings; ++ki) {
      append_block(hl.blob, blocks[ki], &P.coupling[ki]);
      meta = std::max(meta, P.coupling[ki].meta_bytes);
      for (int i = 0; i < 3; ++i) wmax[i] = std::max(wmax[i], P.coupling[ki].w_bytes[i]);
    }
    if (lv.has_prior) {
      append_block(hl.blob, prior_block, &P.prior);
      meta = std::max(meta, P.prior.meta_bytes);
      wmax[0] = std::max(wmax[0], P.prior.w_bytes[0]);
    }
    if (hl.blob.empty()) hl.blob.resize(kAlign, 0);
    if (!plan_smem(P, a_bytes, meta, wmax, n_max, (uint32_t)smem_limit, desc->max_batch, num_sms, pd,
                   desc->plan == IODF_PLAN_THROUGHPUT))
      return IODF_EUNSUPPORTED;
    // the index maps divide numbers below group * c * px by at most c * px with a 32-bit magic multiplier
    if ((uint64_t)P.group * c * h * w * ((uint64_t)c * h * w) >= (1ull << 32)) return IODF_EUNSUPPORTED;
    max_smem = std::max(max_smem, P.s_total);
    if (lv.split) c = (uint32_t)ca;
  }

  // device objects
  // The attribute belongs to the kernel, not to a model: always raise it to the device maximum so
  // that creating a second, smaller model cannot lower it under a first model's needs.
  (void)max_smem;
  CU(m, configure_level_kernels((uint32_t)smem_limit));
  CU(m, configure_res_kernels((uint32_t)smem_limit));
  CU(m, configure_pipe_kernels((uint32_t)smem_limit));
  const size_t L = desc->n_levels;
  m->d_plan.assign(L, nullptr); m->d_blob.assign(L, nullptr); m->d_keep.assign(L, nullptr);
  for (size_t li = 0; li < L; ++li) {
    HostLevel& hl = m->levels[li];
    CU(m, cudaMalloc(&m->d_plan[li], sizeof(LevelPlan)));
    CU(m, cudaMemcpy(m->d_plan[li], &hl.plan, sizeof(LevelPlan), cudaMemcpyHostToDevice));
    CU(m, cudaMalloc(&m->d_blob[li], hl.blob.size()));
    CU(m, cudaMemcpy(m->d_blob[li], hl.blob.data(), hl.blob.size(), cudaMemcpyHostToDevice));
    if (li + 1 < L)
      CU(m, cudaMalloc(&m->d_keep[li], (size_t)desc->max_batch * hl.plan.keep_c * hl.plan.px * sizeof(int32_t)));
  }
  m->ev.assign(L + 1, nullptr);
  for (size_t i = 0; i <= L; ++i) CU(m, cudaEventCreate(&m->ev[i]));
  CU(m, cudaMalloc(&m->d_status, sizeof(uint32_t)));
  CU(m, cudaMemset(m->d_status, 0, sizeof(uint32_t)));
  CU(m, cudaMalloc(&m->d_x, (size_t)desc->max_batch * lay.d));
  CU(m, cudaMalloc(&m->d_z, (size_t)desc->max_batch * lay.d * sizeof(int32_t)));
  if (lay.d_fact) CU(m, cudaMalloc(&m->d_prior, (size_t)desc->max_batch * 2 * lay.d_fact * sizeof(int32_t)));
  CU(m, cudaDeviceSynchronize());
  return IODF_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The batch as the patch grid of one image (first level's load / last store); img_w = 0: a plain batch.
struct PatchGrid {
  int img_h = 0, img_w = 0, patches_x = 0;
};

void set_patch_grid(LevelArgs& a, const PatchGrid& g) {
  a.img_h = g.img_h; a.img_w = g.img_w; a.patches_x = g.patches_x;
  a.mul_patches_x = g.patches_x > 1 ? (uint32_t)(((1ull << 32) + g.patches_x - 1) / g.patches_x) : 0u;
}

// The kernel that runs a level: residual couplings, the stage pipeline, or the general kernel.
cudaError_t launch_any_level(const LevelPlan& P, const LevelArgs& a, bool inverse, int B, cudaStream_t st) {
  const int grid = (B + P.group - 1) / P.group;
  if (P.residual) return launch_res_level(a, inverse, grid, P.res_bands, P.s_total, st);
  if (P.pipe) return launch_level_pipe(a, inverse, grid, P.s_total, st);
  return launch_level(a, inverse, P.lean != 0, grid, P.s_total, st);
}

int run_forward(iodf_model* m, const uint8_t* x, int B, int32_t* z, int32_t* prior, cudaStream_t st,
                bool timed = false, PatchGrid grid = PatchGrid()) {
  const size_t L = m->levels.size();
  if (timed) CU(m, cudaEventRecord(m->ev[0], st));
  for (size_t li = 0; li < L; ++li) {
    const LevelPlan& P = m->levels[li].plan;
    LevelArgs a{};
    a.plan = m->d_plan[li];
    a.blob = m->d_blob[li];
    a.in = li == 0 ? (const void*)x : (const void*)m->d_keep[li - 1];
    a.in_stride = 0;
    a.z = z;
    a.prior = prior;
    a.out = m->d_keep[li];
    a.oor = nullptr;
    a.status = m->d_status;
    a.batch = B;
    if (li == 0) set_patch_grid(a, grid);
    CU(m, launch_any_level(P, a, false, B, st));
    if (timed) CU(m, cudaEventRecord(m->ev[li + 1], st));
  }
  return IODF_OK;
}

// One decode launch of level li. phase: 0 = whole level, 1 = prior head only, 2 = couplings only.
int launch_inverse_level(iodf_model* m, int li, int phase, const int32_t* z, int B, uint8_t* x, int32_t* prior,
                         uint32_t* oor, cudaStream_t st, const PatchGrid& grid) {
  const int L = (int)m->levels.size();
  const LevelPlan& P = m->levels[li].plan;
  LevelArgs a{};
  a.plan = m->d_plan[li];
  a.blob = m->d_blob[li];
  if (li == L - 1) { a.in = z + m->layout.z_final_off; a.in_stride = (long long)m->layout.d; }
  else { a.in = m->d_keep[li]; a.in_stride = (long long)P.keep_c * P.px; }
  a.z = const_cast<int32_t*>(z);
  a.prior = prior;
  a.out = li == 0 ? (void*)x : (void*)m->d_keep[li - 1];
  a.oor = oor;
  a.status = m->d_status;
  a.batch = B;
  a.phase = phase;
  if (li == 0) set_patch_grid(a, grid);
  CU(m, launch_any_level(P, a, true, B, st));
  return IODF_OK;
}

int run_inverse(iodf_model* m, const int32_t* z, int B, uint8_t* x, int32_t* prior, uint32_t* oor, cudaStream_t st,
                bool timed = false, PatchGrid grid = PatchGrid()) {
  const int L = (int)m->levels.size();
  if (timed) CU(m, cudaEventRecord(m->ev[L], st));
  for (int li = L - 1; li >= 0; --li) {
    int rc = launch_inverse_level(m, li, 0, z, B, x, prior, oor, st, grid);
    if (rc) return rc;
    if (timed) CU(m, cudaEventRecord(m->ev[li], st));
  }
  return IODF_OK;
}

// H x W image as a grid of in_h x in_w patches: the batch size, or an error
int patch_grid(const iodf_model* m, int H, int W, PatchGrid* g, int* B) {
  if (H < 1 || W < 1 || H % (int)m->in_h || W % (int)m->in_w) return IODF_EINVAL;
  const long long n = (long long)(H / (int)m->in_h) * (W / (int)m->in_w);
  if (n < 1 || n > (long long)m->max_batch) return IODF_EINVAL;
  // the patch index is split with a 32-bit magic multiplier: exact while B * patches_x < 2^32
  if ((unsigned long long)n * (unsigned long long)(W / (int)m->in_w) >= (1ull << 32)) return IODF_EUNSUPPORTED;
  g->img_h = H; g->img_w = W; g->patches_x = W / (int)m->in_w;
  *B = (int)n;
  return IODF_OK;
}

// Level li ran between events li and li+1 (encode) or li+1 and li (decode).
int read_level_times(iodf_model* m, cudaStream_t st, bool inverse, float* level_ms) {
  CU(m, cudaStreamSynchronize(st));
  const size_t L = m->levels.size();
  for (size_t li = 0; li < L; ++li) {
    if (inverse) CU(m, cudaEventElapsedTime(&level_ms[li], m->ev[li + 1], m->ev[li]));
    else CU(m, cudaEventElapsedTime(&level_ms[li], m->ev[li], m->ev[li + 1]));
  }
  return IODF_OK;
}

}  // namespace

// ---- allocation-free encode -----------------------------------------------------------------------
// Fixed inter-level scratch for iodf_forward_static. In host code `g_static_scratch` is only a
// handle for the symbol, not a device address: the address is looked up once per device with
// cudaGetSymbolAddress and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[IODF_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
unsigned char* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the static scratch on `device` (looked up on first use, cached afterwards).
int static_scratch_address(iodf_model* m, int device, unsigned char** out) {
  if (device < 0 || device >= kMaxDevices) return IODF_EINVAL;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[device]) {
    int prev = -1;
    CU(m, cudaGetDevice(&prev));
    CU(m, cudaSetDevice(device));
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    cudaError_t e2 = cudaSetDevice(prev);
    if (e != cudaSuccess) return cuda_fail(m, e);
    if (e2 != cudaSuccess) return cuda_fail(m, e2);
    if (!p) return IODF_ECUDA;
    g_scratch_ptr[device] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_ptr[device];
  return IODF_OK;
}

size_t static_bytes_per_image(const iodf_model* m) {
  size_t bytes = 0;
  for (size_t li = 0; li + 1 < m->levels.size(); ++li) {
    const LevelPlan& P = m->levels[li].plan;
    bytes += ((size_t)P.keep_c * P.px * sizeof(int32_t) + 255) / 256 * 256;
  }
  return bytes;
}

}  // namespace

extern "C" {

size_t iodf_static_scratch_bytes_per_image(const iodf_model* m) { return m ? static_bytes_per_image(m) : 0; }

int iodf_forward_static(iodf_model* m, const uint8_t* x_u8, int B, int32_t* z, int32_t* prior, void* cuda_stream) {
  if (!m || !x_u8 || !z || B < 1) return IODF_EINVAL;
  if (!aligned16(x_u8) || !aligned16(z) || !aligned16(prior)) return IODF_EINVAL;
  const size_t per_image = static_bytes_per_image(m);
  if ((size_t)B > (size_t)IODF_STATIC_SCRATCH_BYTES / (per_image ? per_image : 1) && per_image) return IODF_ELIMIT;
  unsigned char* base = nullptr;
  int rc = static_scratch_address(m, m->device, &base);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int32_t* prior_arg = m->layout.d_fact ? prior : nullptr;
  // the kept channels of level l live at keep[l] inside the fixed array, sized for this call's B
  const size_t L = m->levels.size();
  int32_t* keep[IODF_MAX_LEVELS];
  size_t off = 0;
  for (size_t li = 0; li < L; ++li) {
    keep[li] = reinterpret_cast<int32_t*>(base + off);
    if (li + 1 < L) {
      const LevelPlan& P = m->levels[li].plan;
      off += ((size_t)P.keep_c * P.px * sizeof(int32_t) + 255) / 256 * 256 * (size_t)B;
    }
  }
  for (size_t li = 0; li < L; ++li) {
    const LevelPlan& P = m->levels[li].plan;
    LevelArgs a{};
    a.plan = m->d_plan[li];
    a.blob = m->d_blob[li];
    a.in = li == 0 ? (const void*)x_u8 : (const void*)keep[li - 1];
    a.in_stride = 0;
    a.z = z;
    a.prior = prior_arg;
    a.out = keep[li];
    a.oor = nullptr;
    a.status = m->d_status;
    a.batch = B;
    CU(m, launch_any_level(P, a, false, B, st));
  }
  return IODF_OK;
}

}  // extern "C"

extern "C" {

int iodf_create(const iodf_model_desc* desc, const int8_t* weights, size_t weights_count, const int32_t* requant,
                size_t requant_count, int device, iodf_model** out) {
  if (!desc || !weights || !requant || !out) return IODF_EINVAL;
  *out = nullptr;
  iodf_model* m = new (std::nothrow) iodf_model();
  if (!m) return IODF_ENOMEM;
  int rc;
  try {
    Blobs B{weights, weights_count, requant, requant_count};
    rc = build_model(desc, B, device, m);
  } catch (const std::bad_alloc&) {
    rc = IODF_ENOMEM;
  }
  if (rc != IODF_OK) {
    iodf_destroy(m);
    return rc;
  }
  *out = m;
  return IODF_OK;
}

void iodf_destroy(iodf_model* m) {
  if (!m) return;
  cudaSetDevice(m->device);
  for (auto p : m->d_plan) if (p) cudaFree(p);
  for (auto p : m->d_blob) if (p) cudaFree(p);
  for (auto p : m->d_keep) if (p) cudaFree(p);
  for (auto e : m->ev) if (e) cudaEventDestroy(e);
  if (m->d_status) cudaFree(m->d_status);
  if (m->d_x) cudaFree(m->d_x);
  if (m->d_z) cudaFree(m->d_z);
  if (m->d_prior) cudaFree(m->d_prior);
  delete m;
}

int iodf_get_layout(const iodf_model* m, iodf_layout* out) {
  if (!m || !out) return IODF_EINVAL;
  *out = m->layout;
  return IODF_OK;
}

int iodf_forward(iodf_model* m, const uint8_t* x_u8, int B, int32_t* z, int32_t* prior, void* cuda_stream) {
  if (!m || !x_u8 || !z || B < 1 || (uint32_t)B > m->max_batch) return IODF_EINVAL;
  if (!aligned16(x_u8) || !aligned16(z) || !aligned16(prior)) return IODF_EINVAL;
  return run_forward(m, x_u8, B, z, m->layout.d_fact ? prior : nullptr, (cudaStream_t)cuda_stream);
}

int iodf_inverse(iodf_model* m, const int32_t* z, int B, uint8_t* x_u8, int32_t* prior, uint32_t* out_of_range_count,
                 void* cuda_stream) {
  if (!m || !x_u8 || !z || B < 1 || (uint32_t)B > m->max_batch) return IODF_EINVAL;
  if (!aligned16(x_u8) || !aligned16(z) || !aligned16(prior)) return IODF_EINVAL;
  return run_inverse(m, z, B, x_u8, m->layout.d_fact ? prior : nullptr, out_of_range_count,
                     (cudaStream_t)cuda_stream);
}

int iodf_inverse_level(iodf_model* m, int level, int phase, const int32_t* z, int B, uint8_t* x_u8, int32_t* prior,
                       uint32_t* out_of_range_count, void* cuda_stream) {
  if (!m || !z || B < 1 || (uint32_t)B > m->max_batch) return IODF_EINVAL;
  if (level < 0 || level >= (int)m->levels.size()) return IODF_EINVAL;
  if (phase != IODF_LEVEL_PRIOR && phase != IODF_LEVEL_COUPLINGS) return IODF_EINVAL;
  if (!aligned16(z) || !aligned16(prior) || !aligned16(x_u8)) return IODF_EINVAL;
  const LevelPlan& P = m->levels[level].plan;
  if (phase == IODF_LEVEL_PRIOR) {
    if (!P.has_prior || !prior) return IODF_EINVAL;
    return launch_inverse_level(m, level, 1, z, B, nullptr, prior, nullptr, (cudaStream_t)cuda_stream, PatchGrid());
  }
  if (level == 0 && !x_u8) return IODF_EINVAL;
  return launch_inverse_level(m, level, 2, z, B, x_u8, nullptr, out_of_range_count, (cudaStream_t)cuda_stream,
                              PatchGrid());
}

int iodf_forward_patches(iodf_model* m, const uint8_t* image_u8, int H, int W, int32_t* z, int32_t* prior,
                         void* cuda_stream) {
  if (!m || !image_u8 || !z) return IODF_EINVAL;
  if (!aligned16(image_u8) || !aligned16(z) || !aligned16(prior)) return IODF_EINVAL;
  PatchGrid g;
  int B = 0;
  int rc = patch_grid(m, H, W, &g, &B);
  if (rc) return rc;
  return run_forward(m, image_u8, B, z, m->layout.d_fact ? prior : nullptr, (cudaStream_t)cuda_stream, false, g);
}

int iodf_inverse_patches(iodf_model* m, const int32_t* z, int H, int W, uint8_t* image_u8, int32_t* prior,
                         uint32_t* out_of_range_count, void* cuda_stream) {
  if (!m || !image_u8 || !z) return IODF_EINVAL;
  if (!aligned16(image_u8) || !aligned16(z) || !aligned16(prior)) return IODF_EINVAL;
  PatchGrid g;
  int B = 0;
  int rc = patch_grid(m, H, W, &g, &B);
  if (rc) return rc;
  return run_inverse(m, z, B, image_u8, m->layout.d_fact ? prior : nullptr, out_of_range_count,
                     (cudaStream_t)cuda_stream, false, g);
}

// ---- entropy coding ---------------------------------------------------------------------------------
#define CUC(c, x)                                                      \
  do {                                                                 \
    cudaError_t e__ = (x);                                             \
    if (e__ != cudaSuccess) {                                          \
      (c)->last_cuda = (int)e__;                                       \
      return e__ == cudaErrorMemoryAllocation ? IODF_ENOMEM : IODF_ECUDA; \
    }                                                                  \
  } while (0)

int iodf_codec_create(const iodf_model* m, const iodf_codec_desc* desc, iodf_codec** out) {
  if (!m || !desc || !out) return IODF_EINVAL;
  *out = nullptr;
  if (desc->abi_version != IODF_ABI_VERSION) return IODF_EVERSION;
  if (!desc->sigmoid_table || !desc->inv_scale || desc->umax < 1 || desc->umax > 8192 || desc->n_scales < 1 ||
      desc->n_scales > 1024 || desc->elems_per_stream < 1 || desc->elems_per_stream > 65536)
    return IODF_EINVAL;
  if (desc->final_ls < 0 || desc->final_ls >= (int32_t)desc->n_scales) return IODF_EINVAL;
  const uint32_t top = (1u << 16) - (2u * 2048u + 1u);
  for (uint32_t i = 0; i < 2 * desc->umax + 1; ++i) {
    if (desc->sigmoid_table[i] > top) return IODF_EINVAL;
    if (i && desc->sigmoid_table[i] < desc->sigmoid_table[i - 1]) return IODF_EINVAL;   // must not decrease
  }
  for (uint32_t i = 0; i < desc->n_scales; ++i)   // 2^21 / s with s >= 2^-9: the kernels multiply in 32 bits
    if (desc->inv_scale[i] < 1 || desc->inv_scale[i] >= (1u << 30)) return IODF_EINVAL;
  iodf_codec* c = new (std::nothrow) iodf_codec();
  if (!c) return IODF_ENOMEM;
  c->device = m->device;
  c->max_batch = m->max_batch;
  c->elems_per_stream = desc->elems_per_stream;
  RansArgs& a = c->args;
  a.umax = (int)desc->umax; a.n_scales = (int)desc->n_scales; a.final_ls = desc->final_ls;
  a.d = (long long)m->layout.d; a.d_fact = (long long)m->layout.d_fact;
  a.cap = (int)(3 * desc->elems_per_stream + 2);
  // coded blocks: every factored-out block in z order, then the final block
  int nb = 0, first = 0;
  const uint32_t E = desc->elems_per_stream;
  auto add_block = [&](uint64_t z_off, uint64_t n, long long prior_off) {
    RansBlock& b = a.blocks[nb];
    b.z_off = (long long)z_off; b.n = (long long)n; b.prior_off = prior_off;
    b.first_stream = first; b.n_streams = (int)((n + E - 1) / E);
    c->layout.block_z_off[nb] = z_off; c->layout.block_elems[nb] = n;
    c->layout.block_first_stream[nb] = (uint32_t)first; c->layout.block_streams[nb] = (uint32_t)b.n_streams;
    c->layout.block_level[nb] = -1;
    first += b.n_streams;
    ++nb;
  };
  for (size_t li = 0; li < m->levels.size(); ++li) {
    const LevelPlan& P = m->levels[li].plan;
    if (!P.split) continue;
    // every scale index a prior head of this level can emit must be an entry of the scale table
    if (P.has_prior && (m->levels[li].ls_lo < 0 || m->levels[li].ls_hi >= (int32_t)desc->n_scales)) {
      delete c;
      return IODF_EINVAL;
    }
    add_block(P.z_off, (uint64_t)P.cb * P.px, P.has_prior ? (long long)P.prior_off : -1);
    c->layout.block_level[nb - 1] = (int32_t)li;
  }
  add_block(m->layout.z_final_off, m->layout.d - m->layout.z_final_off, -1);
  a.n_blocks = nb; a.n_streams = first;
  c->layout.n_blocks = (uint32_t)nb; c->layout.n_streams = (uint32_t)first; c->layout.words_per_stream = (uint32_t)a.cap;
  int prev = -1;
  const size_t rbytes = 4 * (size_t)desc->n_scales, gbytes = 2 * (size_t)(2 * desc->umax + 1);
  cudaError_t e = cudaGetDevice(&prev);
  if (e == cudaSuccess) e = cudaSetDevice(c->device);
  if (e != cudaSuccess) {
    delete c;
    return IODF_ECUDA;
  }
  e = cudaMalloc(&c->d_tables, rbytes + gbytes);
  if (e == cudaSuccess) e = cudaMemcpy(c->d_tables, desc->inv_scale, rbytes, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(c->d_tables + rbytes, desc->sigmoid_table, gbytes, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMalloc(&c->d_errors, sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMalloc(&c->d_sizes, sizeof(uint32_t) * (size_t)c->max_batch);
  if (e == cudaSuccess) e = cudaMemset(c->d_errors, 0, sizeof(uint32_t));
  cudaSetDevice(prev);
  if (e != cudaSuccess) {
    const int rc = e == cudaErrorMemoryAllocation ? IODF_ENOMEM : IODF_ECUDA;
    iodf_codec_destroy(c);
    return rc;
  }
  a.R = reinterpret_cast<const uint32_t*>(c->d_tables);
  a.G = reinterpret_cast<const uint16_t*>(c->d_tables + rbytes);
  a.errors = c->d_errors;
  *out = c;
  return IODF_OK;
}

void iodf_codec_destroy(iodf_codec* c) {
  if (!c) return;
  cudaSetDevice(c->device);
  if (c->d_tables) cudaFree(c->d_tables);
  if (c->d_errors) cudaFree(c->d_errors);
  if (c->d_sizes) cudaFree(c->d_sizes);
  if (c->d_words) cudaFree(c->d_words);
  if (c->d_counts) cudaFree(c->d_counts);
  if (c->d_packed) cudaFree(c->d_packed);
  delete c;
}

int iodf_codec_get_layout(const iodf_codec* c, iodf_codec_layout* out) {
  if (!c || !out) return IODF_EINVAL;
  *out = c->layout;
  return IODF_OK;
}

int iodf_rans_encode(iodf_codec* c, const int32_t* z, const int32_t* prior, int B, uint16_t* words, uint32_t* counts,
                     void* cuda_stream) {
  if (!c || !z || !words || !counts || B < 1 || (uint32_t)B > c->max_batch) return IODF_EINVAL;
  if (c->args.d_fact && !prior) return IODF_EINVAL;
  RansArgs a = c->args;
  a.batch = B;
  CUC(c, launch_rans_encode(a, z, prior, words, counts, (cudaStream_t)cuda_stream));
  return IODF_OK;
}

int iodf_rans_decode_block(iodf_codec* c, int block, const uint16_t* words, const uint32_t* counts,
                           const int32_t* prior, int B, int32_t* z, void* cuda_stream) {
  if (!c || !z || !words || !counts || B < 1 || (uint32_t)B > c->max_batch) return IODF_EINVAL;
  if (block < 0 || block >= c->args.n_blocks) return IODF_EINVAL;
  if (c->args.blocks[block].prior_off >= 0 && !prior) return IODF_EINVAL;
  RansArgs a = c->args;
  a.batch = B;
  CUC(c, launch_rans_decode(a, block, words, counts, prior, z, (cudaStream_t)cuda_stream));
  return IODF_OK;
}

size_t iodf_rans_packed_capacity(const iodf_codec* c, int B) {
  if (!c || B < 1) return 0;
  const size_t S = (size_t)c->args.n_streams, cap = (size_t)c->args.cap;
  return 4 * ((size_t)B + 1) + (size_t)B * 2 * (S + S * cap);
}

int iodf_rans_pack(iodf_codec* c, const uint16_t* words, const uint32_t* counts, int B, uint8_t* packed,
                   void* cuda_stream) {
  if (!c || !words || !counts || !packed || B < 1 || (uint32_t)B > c->max_batch) return IODF_EINVAL;
  if ((reinterpret_cast<uintptr_t>(packed) & 3u) || c->args.cap > 65535) return IODF_EINVAL;
  // record offsets are 32-bit and the per-stream offsets of an image live in shared memory
  if (iodf_rans_packed_capacity(c, B) >= (1ull << 32) || c->args.n_streams > 8192) return IODF_EUNSUPPORTED;
  RansArgs a = c->args;
  a.batch = B;
  CUC(c, launch_rans_pack(a, words, counts, c->d_sizes, packed, (cudaStream_t)cuda_stream));
  return IODF_OK;
}

int iodf_rans_unpack(iodf_codec* c, const uint8_t* packed, size_t packed_bytes, int B, uint16_t* words,
                     uint32_t* counts, void* cuda_stream) {
  if (!c || !words || !counts || !packed || B < 1 || (uint32_t)B > c->max_batch) return IODF_EINVAL;
  if ((reinterpret_cast<uintptr_t>(packed) & 3u) || c->args.cap > 65535) return IODF_EINVAL;
  if (packed_bytes < 4 * ((size_t)B + 1)) return IODF_EINVAL;
  if (packed_bytes >= (1ull << 32) || c->args.n_streams > 8192) return IODF_EUNSUPPORTED;
  RansArgs a = c->args;
  a.batch = B;
  CUC(c, launch_rans_unpack(a, packed, (unsigned long long)(packed_bytes - 4 * ((size_t)B + 1)), words, counts,
                            (cudaStream_t)cuda_stream));
  return IODF_OK;
}

namespace {
int codec_staging(iodf_codec* c) {
  if (c->d_packed) return IODF_OK;
  int prev = -1;
  CUC(c, cudaGetDevice(&prev));
  CUC(c, cudaSetDevice(c->device));
  const size_t S = (size_t)c->args.n_streams, cap = (size_t)c->args.cap, B = c->max_batch;
  c->packed_capacity = iodf_rans_packed_capacity(c, (int)B);
  cudaError_t e = cudaMalloc(&c->d_words, B * S * cap * sizeof(uint16_t));
  if (e == cudaSuccess) e = cudaMalloc(&c->d_counts, B * S * sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMalloc(&c->d_packed, c->packed_capacity);
  cudaSetDevice(prev);
  if (e != cudaSuccess) {
    c->last_cuda = (int)e;
    return e == cudaErrorMemoryAllocation ? IODF_ENOMEM : IODF_ECUDA;
  }
  return IODF_OK;
}
}  // namespace

int iodf_compress_host(iodf_model* m, iodf_codec* c, const uint8_t* x_u8_host, int B, uint8_t* out_host,
                       size_t out_capacity, size_t* out_bytes, void* cuda_stream) {
  if (!m || !c || !x_u8_host || !out_host || !out_bytes || B < 1 || (uint32_t)B > m->max_batch ||
      (uint32_t)B > c->max_batch || c->args.d != (long long)m->layout.d || c->args.cap > 65535)
    return IODF_EINVAL;
  if (iodf_rans_packed_capacity(c, B) >= (1ull << 32) || c->args.n_streams > 8192) return IODF_EUNSUPPORTED;
  int rc = codec_staging(c);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t d = m->layout.d;
  int32_t* prior = m->layout.d_fact ? m->d_prior : nullptr;
  CU(m, cudaMemcpyAsync(m->d_x, x_u8_host, (size_t)B * d, cudaMemcpyHostToDevice, st));
  rc = run_forward(m, m->d_x, B, m->d_z, prior, st);
  if (rc) return rc;
  RansArgs a = c->args;
  a.batch = B;
  CUC(c, launch_rans_encode(a, m->d_z, prior, c->d_words, c->d_counts, st));
  CUC(c, launch_rans_pack(a, c->d_words, c->d_counts, c->d_sizes, c->d_packed, st));
  // the payload size is only known now: read it, then copy exactly header + payload
  uint32_t payload = 0;
  CUC(c, cudaMemcpyAsync(&payload, c->d_packed + 4 * (size_t)B, sizeof(payload), cudaMemcpyDeviceToHost, st));
  CUC(c, cudaStreamSynchronize(st));
  const size_t total = 4 * ((size_t)B + 1) + payload;
  *out_bytes = total;
  if (total > out_capacity) return IODF_ELIMIT;
  CUC(c, cudaMemcpyAsync(out_host, c->d_packed, total, cudaMemcpyDeviceToHost, st));
  CUC(c, cudaStreamSynchronize(st));
  return IODF_OK;
}

int iodf_decompress_host(iodf_model* m, iodf_codec* c, const uint8_t* in_host, size_t in_bytes, int B,
                         uint8_t* x_u8_host, void* cuda_stream) {
  if (!m || !c || !in_host || !x_u8_host || B < 1 || (uint32_t)B > m->max_batch || (uint32_t)B > c->max_batch ||
      c->args.d != (long long)m->layout.d || c->args.cap > 65535)
    return IODF_EINVAL;
  int rc = codec_staging(c);
  if (rc) return rc;
  if (in_bytes < 4 * ((size_t)B + 1) || in_bytes > c->packed_capacity) return IODF_EINVAL;
  if (in_bytes >= (1ull << 32) || c->args.n_streams > 8192) return IODF_EUNSUPPORTED;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CU(m, cudaMemcpyAsync(c->d_packed, in_host, in_bytes, cudaMemcpyHostToDevice, st));
  RansArgs a = c->args;
  a.batch = B;
  CUC(c, launch_rans_unpack(a, c->d_packed, (unsigned long long)(in_bytes - 4 * ((size_t)B + 1)), c->d_words,
                            c->d_counts, st));
  int32_t* prior = m->layout.d_fact ? m->d_prior : nullptr;
  // decoder order: the final block, then per level: prior parameters, the level's block, inverse couplings
  CUC(c, launch_rans_decode(a, a.n_blocks - 1, c->d_words, c->d_counts, prior, m->d_z, st));
  const int L = (int)m->levels.size();
  for (int li = L - 1; li >= 0; --li) {
    int q = -1;
    for (int k = 0; k + 1 < a.n_blocks; ++k)
      if (c->layout.block_level[k] == li) q = k;
    if (q >= 0) {
      if (m->levels[li].plan.has_prior) {
        rc = launch_inverse_level(m, li, 1, m->d_z, B, nullptr, prior, nullptr, st, PatchGrid());
        if (rc) return rc;
      }
      CUC(c, launch_rans_decode(a, q, c->d_words, c->d_counts, prior, m->d_z, st));
    }
    rc = launch_inverse_level(m, li, 2, m->d_z, B, m->d_x, nullptr, nullptr, st, PatchGrid());
    if (rc) return rc;
  }
  CU(m, cudaMemcpyAsync(x_u8_host, m->d_x, (size_t)B * m->layout.d, cudaMemcpyDeviceToHost, st));
  return IODF_OK;
}

int iodf_codec_check(iodf_codec* c, void* cuda_stream, uint32_t* bad_streams) {
  if (!c) return IODF_EINVAL;
  uint32_t n = 0;
  CUC(c, cudaMemcpyAsync(&n, c->d_errors, sizeof(n), cudaMemcpyDeviceToHost, (cudaStream_t)cuda_stream));
  CUC(c, cudaStreamSynchronize((cudaStream_t)cuda_stream));
  if (n) CUC(c, cudaMemsetAsync(c->d_errors, 0, sizeof(n), (cudaStream_t)cuda_stream));
  if (bad_streams) *bad_streams = n;
  return n ? IODF_EDATA : IODF_OK;
}

int iodf_forward_timed(iodf_model* m, const uint8_t* x_u8, int B, int32_t* z, int32_t* prior, void* cuda_stream,
                       float* level_ms) {
  if (!m || !x_u8 || !z || !level_ms || B < 1 || (uint32_t)B > m->max_batch) return IODF_EINVAL;
  if (!aligned16(x_u8) || !aligned16(z) || !aligned16(prior)) return IODF_EINVAL;
  int rc = run_forward(m, x_u8, B, z, m->layout.d_fact ? prior : nullptr, (cudaStream_t)cuda_stream, true);
  if (rc) return rc;
  return read_level_times(m, (cudaStream_t)cuda_stream, false, level_ms);
}

int iodf_inverse_timed(iodf_model* m, const int32_t* z, int B, uint8_t* x_u8, int32_t* prior,
                       uint32_t* out_of_range_count, void* cuda_stream, float* level_ms) {
  if (!m || !x_u8 || !z || !level_ms || B < 1 || (uint32_t)B > m->max_batch) return IODF_EINVAL;
  if (!aligned16(x_u8) || !aligned16(z) || !aligned16(prior)) return IODF_EINVAL;
  int rc = run_inverse(m, z, B, x_u8, m->layout.d_fact ? prior : nullptr, out_of_range_count,
                       (cudaStream_t)cuda_stream, true);
  if (rc) return rc;
  return read_level_times(m, (cudaStream_t)cuda_stream, true, level_ms);
}

int iodf_forward_host(iodf_model* m, const uint8_t* x_u8_host, int B, int32_t* z_host, int32_t* prior_host,
                      void* cuda_stream) {
  if (!m || !x_u8_host || !z_host || B < 1 || (uint32_t)B > m->max_batch) return IODF_EINVAL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t d = m->layout.d, df = m->layout.d_fact;
  int32_t* prior = (prior_host && df) ? m->d_prior : nullptr;
  CU(m, cudaMemcpyAsync(m->d_x, x_u8_host, (size_t)B * d, cudaMemcpyHostToDevice, st));
  int rc = run_forward(m, m->d_x, B, m->d_z, prior, st);
  if (rc) return rc;
  CU(m, cudaMemcpyAsync(z_host, m->d_z, (size_t)B * d * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  if (prior) CU(m, cudaMemcpyAsync(prior_host, prior, (size_t)B * 2 * df * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  return IODF_OK;
}

int iodf_inverse_host(iodf_model* m, const int32_t* z_host, int B, uint8_t* x_u8_host, void* cuda_stream) {
  if (!m || !x_u8_host || !z_host || B < 1 || (uint32_t)B > m->max_batch) return IODF_EINVAL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t d = m->layout.d;
  CU(m, cudaMemcpyAsync(m->d_z, z_host, (size_t)B * d * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  int rc = run_inverse(m, m->d_z, B, m->d_x, nullptr, nullptr, st);
  if (rc) return rc;
  CU(m, cudaMemcpyAsync(x_u8_host, m->d_x, (size_t)B * d, cudaMemcpyDeviceToHost, st));
  return IODF_OK;
}

int iodf_check(iodf_model* m, void* cuda_stream) {
  if (!m) return IODF_EINVAL;
  uint32_t st = 0;
  CU(m, cudaStreamSynchronize((cudaStream_t)cuda_stream));
  CU(m, cudaMemcpy(&st, m->d_status, sizeof(st), cudaMemcpyDeviceToHost));
  if (st) {
    CU(m, cudaMemset(m->d_status, 0, sizeof(uint32_t)));
    return IODF_ETIMEOUT;
  }
  return IODF_OK;
}

int iodf_selftest_timeout(iodf_model* m, uint32_t tries, void* cuda_stream) {
  if (!m || tries < 1 || tries > 100u) return IODF_EINVAL;
  CU(m, launch_timeout_probe(m->d_status, tries, (cudaStream_t)cuda_stream));
  return IODF_OK;
}

int iodf_int8_mma_peak(iodf_model* m, uint32_t mma_groups, void* cuda_stream, unsigned long long* ops_out) {
  if (!m || mma_groups < 1 || mma_groups > (1u << 22)) return IODF_EINVAL;
  int sms = 0;
  CU(m, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, m->device));
  CU(m, launch_int8_mma_peak(m->d_status, mma_groups, sms, (cudaStream_t)cuda_stream, ops_out));
  return IODF_OK;
}

const char* iodf_level_kernel_name(const iodf_model* m, int level) {
  if (!m || level < 0 || level >= (int)m->levels.size()) return "";
  const LevelPlan& P = m->levels[level].plan;
  return P.residual ? "res_level_kernel" : (P.pipe ? "level_pipe_kernel" : "level_kernel");
}

int iodf_level_images_per_cta(const iodf_model* m, int level) {
  if (!m || level < 0 || level >= (int)m->levels.size()) return IODF_EINVAL;
  return m->levels[level].plan.group;
}

int iodf_launches_per_call(const iodf_model* m, int inverse) {
  (void)inverse;
  return m ? (int)m->levels.size() : 0;
}

const char* iodf_strerror(int status) {
  switch (status) {
    case IODF_OK: return "ok";
    case IODF_EINVAL: return "invalid argument or malformed model descriptor";
    case IODF_ENOMEM: return "out of memory";
    case IODF_ECUDA: return "CUDA call failed";
    case IODF_EVERSION: return "ABI version mismatch";
    case IODF_ETIMEOUT: return "a bounded device-side wait gave up";
    case IODF_EUNSUPPORTED: return "model shape not supported by this build";
    case IODF_EOVERFLOW: return "worst-case accumulator leaves the int32 range";
    case IODF_ELIMIT: return "request exceeds a fixed capacity (static scratch or caller's output buffer)";
    case IODF_EDATA: return "entropy coder: scale index outside the table or malformed stream";
    default: return "unknown status";
  }
}

int iodf_last_cuda_error(const iodf_model* m) { return m ? m->last_cuda : 0; }

}  // extern "C"
