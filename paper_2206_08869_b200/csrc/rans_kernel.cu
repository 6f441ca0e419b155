// Entropy coding of the flow's latents on the GPU: the discrete logistic prior of Sec. 3 in integer
// table form and range-ANS (App. A) with a 32-bit state renormalised in 16-bit words, one thread
// per stream. The streams are independent (an image's coded blocks are cut into streams of about
// `elems_per_stream` interleaved elements), so a batch of 128 ImageNet64-sized latents is 6 144
// streams: the GPU coder that Sec. 5.3 names as future work (the paper codes on the CPU).
//
//   symbol of an element   k = clamp(z - mu, -2048, 2048) + 2048          (0 and 4096: escapes, then
//                                                                          z follows as 2 x 16 raw bits)
//   cumulative counts      Cum(k) = k + G[clamp(floor((2(k-2048)-1) R[ls] / 2^16), -umax, umax) + umax]
//                          Cum(0) = 0, Cum(4097) = M = 2^16
//   encode step            if x >= F * 2^16: move the low 16 bits of x out;  x = (x / F) * M + (x mod F) + C
//   decode step            slot = x mod M; k: Cum(k) <= slot < Cum(k+1);  x = F * (x / M) + slot - C;
//                          if x < 2^16: x = x * 2^16 + next word
//
// The encoder walks a stream's elements last to first and appends words, then the state (low half,
// high half); the decoder starts at the end of the words and walks back, producing the elements
// first to last. Consecutive threads own consecutive streams of a block, whose i-th elements are
// consecutive in memory: the loads of z and of the prior parameters are coalesced.
#include "rans_kernel.h"

namespace iodf {

namespace {

constexpr int kWin = 2048;
constexpr uint32_t kM = 1u << 16;
constexpr int kThreadsPerBlock = 128;

struct Tables {
  const uint16_t* G;       // shared memory
  const uint32_t* R;       // shared memory
  int umax, n_scales;
};

__device__ __forceinline__ uint32_t cum(const Tables& t, int ls, int k) {
  if (k <= 0) return 0u;
  if (k >= 2 * kWin + 1) return kM;
  // floor(edge2 * R / 2^16) in 32-bit pieces: with R = Rh 2^16 + Rl it is edge2 * Rh + floor(edge2 * Rl /
  // 2^16) exactly (|edge2| < 2^13, Rl < 2^16, Rh < 2^15 for the scales a codec accepts)
  const int edge2 = 2 * (k - kWin) - 1;
  const uint32_t R = t.R[ls];
  int u = edge2 * (int)(R >> 16) + ((edge2 * (int)(R & 0xFFFFu)) >> 16);      // arithmetic shift: floor
  u = max(-t.umax, min(t.umax, u));
  return (uint32_t)k + t.G[u + t.umax];
}

__device__ __forceinline__ void load_tables(const RansArgs& a, uint16_t* sG, uint32_t* sR) {
  for (int i = threadIdx.x; i < 2 * a.umax + 1; i += blockDim.x) sG[i] = a.G[i];
  for (int i = threadIdx.x; i < a.n_scales; i += blockDim.x) sR[i] = a.R[i];
  __syncthreads();
}

// the element's prior parameters; a block without a prior head has mu = 0 and the fixed scale index
__device__ __forceinline__ void prior_of(const RansArgs& a, const RansBlock& blk, const int32_t* prior_img, long e,
                                         int32_t* mu, int* ls, uint32_t* bad) {
  if (blk.prior_off < 0) { *mu = 0; *ls = a.final_ls; return; }
  *mu = prior_img[blk.prior_off + e];
  int l = prior_img[a.d_fact + blk.prior_off + e];
  if (l < 0 || l >= a.n_scales) { *bad = 1u; l = l < 0 ? 0 : a.n_scales - 1; }
  *ls = l;
}

__global__ void __launch_bounds__(kThreadsPerBlock) rans_encode_kernel(const RansArgs a, const int32_t* __restrict__ z,
                                                                       const int32_t* __restrict__ prior,
                                                                       uint16_t* __restrict__ words,
                                                                       uint32_t* __restrict__ counts) {
  extern __shared__ __align__(16) uint8_t smem[];
  uint32_t* sR = reinterpret_cast<uint32_t*>(smem);
  uint16_t* sG = reinterpret_cast<uint16_t*>(smem + 4 * a.n_scales);
  load_tables(a, sG, sR);
  const Tables t{sG, sR, a.umax, a.n_scales};
  const long gid = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= (long)a.batch * a.n_streams) return;
  const int b = (int)(gid / a.n_streams), s = (int)(gid - (long)b * a.n_streams);
  int q = 0;
  while (q + 1 < a.n_blocks && s >= a.blocks[q + 1].first_stream) ++q;
  const RansBlock blk = a.blocks[q];
  const int j = s - blk.first_stream, ns = blk.n_streams;
  const long n_el = (blk.n - j + ns - 1) / ns;
  const int32_t* zb = z + (long)b * a.d + blk.z_off;
  const int32_t* pb = prior + (long)b * 2 * a.d_fact;
  uint16_t* out = words + gid * a.cap;
  uint32_t pos = 0, x = 1u << 16, bad = 0;
  auto push = [&](uint32_t F, uint32_t C) {
    if ((unsigned long long)x >= ((unsigned long long)F << 16)) {
      out[pos++] = (uint16_t)(x & 0xFFFFu);
      x >>= 16;
    }
    x = ((x / F) << 16) + (x % F) + C;
  };
  for (long i = n_el - 1; i >= 0; --i) {
    const long e = j + i * ns;
    const int32_t zv = zb[e];
    int32_t mu; int ls;
    prior_of(a, blk, pb, e, &mu, &ls, &bad);
    long long r = (long long)zv - (long long)mu;
    r = r < -kWin ? -kWin : (r > kWin ? kWin : r);
    const int k = (int)r + kWin;
    if (k == 0 || k == 2 * kWin) {
      push(1u, (uint32_t)zv & 0xFFFFu);
      push(1u, ((uint32_t)zv >> 16) & 0xFFFFu);
    }
    const uint32_t C = cum(t, ls, k), F = cum(t, ls, k + 1) - C;
    push(F, C);
  }
  out[pos++] = (uint16_t)(x & 0xFFFFu);
  out[pos++] = (uint16_t)(x >> 16);
  counts[gid] = pos;
  if (bad && a.errors) atomicAdd(a.errors, 1u);
}

// Decode: one WARP per stream. The state, the word pointer and every step are the same in all 32
// lanes; what the lanes share out is everything that would otherwise be a dependent trip to memory
// or a dependent search step on the stream's serial chain (state -> symbol -> state):
//   * the symbol search: instead of 13 bisection steps, three rounds in which lane L tests one
//     candidate k each (steps of 129, 5 and 1) and a ballot picks the largest k with Cum(k) <= slot;
//     the last round's values also give C = Cum(k) and Cum(k + 1) by shuffle;
//   * the prior parameters: the (mu, scale index) of the next 32 elements are loaded by the 32 lanes
//     in one go and handed out by shuffle, so no global-memory latency sits between two symbols;
//   * the coded words: the lanes hold a window of the stream's next 32 words (the decoder reads the
//     stream backwards), refilled when used up; a renormalisation is a shuffle.
// A stream's latency bounds the decompressor (a block's streams are few and long).
__global__ void __launch_bounds__(kThreadsPerBlock) rans_decode_kernel(const RansArgs a, int q,
                                                                       const uint16_t* __restrict__ words,
                                                                       const uint32_t* __restrict__ counts,
                                                                       const int32_t* __restrict__ prior,
                                                                       int32_t* __restrict__ z) {
  extern __shared__ __align__(16) uint8_t smem[];
  uint32_t* sR = reinterpret_cast<uint32_t*>(smem);
  uint16_t* sG = reinterpret_cast<uint16_t*>(smem + 4 * a.n_scales);
  load_tables(a, sG, sR);
  const Tables t{sG, sR, a.umax, a.n_scales};
  const RansBlock blk = a.blocks[q];
  const int lane = threadIdx.x & 31;
  const long wid = ((long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;       // one stream per warp
  if (wid >= (long)a.batch * blk.n_streams) return;
  const int b = (int)(wid / blk.n_streams), j = (int)(wid - (long)b * blk.n_streams), ns = blk.n_streams;
  const long sid = (long)b * a.n_streams + blk.first_stream + j;
  const long n_el = (blk.n - j + ns - 1) / ns;
  const uint16_t* in = words + sid * a.cap;
  long pos = min((long)counts[sid], (long)a.cap);      // words not yet consumed: in[0 .. pos)
  uint32_t bad = 0;
  // window of the next 32 words: lane L holds in[top - 1 - L] (0 before the stream's first word)
  long top = pos;
  uint32_t win = (top - 1 - lane >= 0) ? in[top - 1 - lane] : 0u;
  auto next = [&]() -> uint32_t {               // never reads before the stream's first word
    if (pos <= 0) { bad = 1u; return 0u; }
    int used = (int)(top - pos);
    if (used == 32) {
      top = pos;
      win = (top - 1 - lane >= 0) ? in[top - 1 - lane] : 0u;
      used = 0;
    }
    --pos;
    return __shfl_sync(0xFFFFFFFFu, win, used);
  };
  uint32_t x = next() << 16;
  x |= next();
  int32_t* zb = z + (long)b * a.d + blk.z_off;
  const int32_t* pb = prior + (long)b * 2 * a.d_fact;
  for (long i0 = 0; i0 < n_el; i0 += 32) {
    // this lane's element of the next 32: its prior parameters now, its decoded value at the end
    int32_t mu_l = 0, zv_l = 0;
    int ls_l = a.final_ls;
    if (i0 + lane < n_el) prior_of(a, blk, pb, j + (i0 + lane) * ns, &mu_l, &ls_l, &bad);
    const int n_here = (int)min(32l, n_el - i0);
    for (int ii = 0; ii < n_here; ++ii) {
      const int32_t mu = __shfl_sync(0xFFFFFFFFu, mu_l, ii);
      const int ls = __shfl_sync(0xFFFFFFFFu, ls_l, ii);
      const uint32_t slot = x & 0xFFFFu;
      // largest k in [0, 4096] with Cum(k) <= slot (Cum(0) = 0 <= slot always; Cum(k > 4096) = M > slot)
      int k = 0;
#pragma unroll
      for (int round = 0; round < 2; ++round) {
        const int step = round == 0 ? 129 : 5;
        const unsigned ok = __ballot_sync(0xFFFFFFFFu, cum(t, ls, k + lane * step) <= slot);   // a prefix of the lanes (Cum is monotone)
        k += (31 - __clz((int)ok)) * step;
      }
      const uint32_t cl = cum(t, ls, k + lane);
      const int sel = 31 - __clz((int)__ballot_sync(0xFFFFFFFFu, cl <= slot));
      k += sel;
      const uint32_t C = __shfl_sync(0xFFFFFFFFu, cl, sel);
      const uint32_t Cn = sel < 31 ? __shfl_sync(0xFFFFFFFFu, cl, sel + 1) : cum(t, ls, k + 1);
      const uint32_t F = Cn - C;
      x = F * (x >> 16) + slot - C;
      if (x < (1u << 16)) x = (x << 16) | next();
      int32_t zv;
      if (k == 0 || k == 2 * kWin) {
        const uint32_t h = x & 0xFFFFu;
        x >>= 16;                                  // F = 1, C = slot: x = x / M
        if (x < (1u << 16)) x = (x << 16) | next();
        const uint32_t l = x & 0xFFFFu;
        x >>= 16;
        if (x < (1u << 16)) x = (x << 16) | next();
        zv = (int32_t)((h << 16) | l);
      } else {
        zv = (int32_t)((long long)mu + (k - kWin));
      }
      if (lane == ii) zv_l = zv;
    }
    if (i0 + lane < n_el) zb[j + (i0 + lane) * ns] = zv_l;
  }
  if (pos != 0 || x != (1u << 16)) bad = 1u;     // every word used and the state back at its start
  bad = __any_sync(0xFFFFFFFFu, bad != 0) ? 1u : 0u;
  if (bad && lane == 0 && a.errors) atomicAdd(a.errors, 1u);
}

// ---- compact byte stream -----------------------------------------------------------------------------
// Packed form of a batch's container (little endian):
//   uint32 offset[B + 1]      byte offset of image b's record from the start of the payload; offset[B] =
//                             payload bytes
//   payload, per image:       uint16 count[n_streams], then the words of stream 0, 1, ... back to back
// so an image's record is 2 * (n_streams + sum of its counts) bytes.

// exclusive scan of n values by one warp, 32 at a time; returns the total (in every lane)
template <typename Load, typename Store>
__device__ __forceinline__ uint32_t warp_scan(int n, int lane, Load load, Store store) {
  uint32_t run = 0;
  for (int base = 0; base < n; base += 32) {
    const int i = base + lane;
    const uint32_t v = i < n ? load(i) : 0u;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
      if (lane >= d) inc += o;
    }
    if (i < n) store(i, run + inc - v);
    run += __shfl_sync(0xFFFFFFFFu, inc, 31);
  }
  return run;
}

// record size of every image, in bytes
__global__ void pack_sizes_kernel(const uint32_t* __restrict__ counts, int n_streams, int cap, uint32_t* __restrict__ sizes) {
  __shared__ uint32_t part[8];
  const int b = blockIdx.x;
  uint32_t sum = 0;
  for (int s = threadIdx.x; s < n_streams; s += blockDim.x) sum += min(counts[(long)b * n_streams + s], (uint32_t)cap);
  sum = __reduce_add_sync(0xFFFFFFFFu, sum);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t t = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += part[w];
    sizes[b] = 2u * ((uint32_t)n_streams + t);
  }
}

// offset[0 .. B] from the sizes (one warp)
__global__ void pack_offsets_kernel(const uint32_t* __restrict__ sizes, int B, uint32_t* __restrict__ offset) {
  const int lane = threadIdx.x;
  const uint32_t total = warp_scan(B, lane, [&](int i) { return sizes[i]; }, [&](int i, uint32_t v) { offset[i] = v; });
  if (lane == 0) offset[B] = total;
}

// kPack: container -> records; !kPack: records -> container. One CTA per image.
template <bool kPack>
__global__ void __launch_bounds__(256) pack_copy_kernel(uint16_t* __restrict__ words, uint32_t* __restrict__ counts,
                                                        int n_streams, int cap, uint8_t* __restrict__ packed,
                                                        int B, unsigned long long payload_bytes, uint32_t* errors) {
  extern __shared__ uint32_t start[];       // word offset of every stream inside the record, after the counts
  __shared__ uint32_t bad;
  const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const uint32_t* offset = reinterpret_cast<const uint32_t*>(packed);
  uint8_t* payload = packed + 4 * (size_t)(B + 1);
  if (threadIdx.x == 0) bad = 0;
  __syncthreads();
  const uint32_t off = offset[b], end = offset[b + 1];
  // a record that does not fit the payload, or that cannot even hold its counts, is skipped
  const bool fits = kPack || (off <= end && end <= payload_bytes && (end - off) >= 2u * (uint32_t)n_streams && (off & 1u) == 0);
  uint16_t* rec = reinterpret_cast<uint16_t*>(payload + off);
  uint32_t* cnt = counts + (long)b * n_streams;
  if (!fits) {
    for (int s = threadIdx.x; s < n_streams; s += blockDim.x) cnt[s] = 0;
    if (threadIdx.x == 0 && errors) atomicAdd(errors, 1u);
    return;
  }
  if (warp == 0) {
    const uint32_t total = warp_scan(n_streams, lane,
        [&](int s) { return min(kPack ? cnt[s] : (uint32_t)rec[s], (uint32_t)cap); },
        [&](int s, uint32_t v) { start[s] = v; });
    if (lane == 0) {
      start[n_streams] = total;
      if (!kPack && 2u * ((uint32_t)n_streams + total) != end - off) bad = 1;    // counts disagree with the record size
    }
  }
  __syncthreads();
  if (bad) {
    for (int s = threadIdx.x; s < n_streams; s += blockDim.x) cnt[s] = 0;
    if (threadIdx.x == 0 && errors) atomicAdd(errors, 1u);
    return;
  }
  for (int s = threadIdx.x; s < n_streams; s += blockDim.x) {
    if (kPack) rec[s] = (uint16_t)min(cnt[s], (uint32_t)cap);
    else cnt[s] = min((uint32_t)rec[s], (uint32_t)cap);
  }
  uint16_t* body = rec + n_streams;
  for (int s = warp; s < n_streams; s += nwarps) {
    const uint32_t n = start[s + 1] - start[s];
    uint16_t* w = words + ((long)b * n_streams + s) * cap;
    uint16_t* r = body + start[s];
    for (uint32_t i = lane; i < n; i += 32) {
      if (kPack) r[i] = w[i]; else w[i] = r[i];
    }
  }
}

}  // namespace

cudaError_t launch_rans_pack(const RansArgs& a, const uint16_t* words, const uint32_t* counts, uint32_t* sizes,
                             uint8_t* packed, cudaStream_t stream) {
  pack_sizes_kernel<<<a.batch, 256, 0, stream>>>(counts, a.n_streams, a.cap, sizes);
  pack_offsets_kernel<<<1, 32, 0, stream>>>(sizes, a.batch, reinterpret_cast<uint32_t*>(packed));
  pack_copy_kernel<true><<<a.batch, 256, 4 * (a.n_streams + 1), stream>>>(
      const_cast<uint16_t*>(words), const_cast<uint32_t*>(counts), a.n_streams, a.cap, packed, a.batch, 0ull, a.errors);
  return cudaGetLastError();
}

cudaError_t launch_rans_unpack(const RansArgs& a, const uint8_t* packed, unsigned long long payload_bytes,
                               uint16_t* words, uint32_t* counts, cudaStream_t stream) {
  pack_copy_kernel<false><<<a.batch, 256, 4 * (a.n_streams + 1), stream>>>(
      words, counts, a.n_streams, a.cap, const_cast<uint8_t*>(packed), a.batch, payload_bytes, a.errors);
  return cudaGetLastError();
}

static size_t table_smem(const RansArgs& a) { return 4 * (size_t)a.n_scales + 2 * (size_t)(2 * a.umax + 1) + 16; }

cudaError_t launch_rans_encode(const RansArgs& a, const int32_t* z, const int32_t* prior, uint16_t* words,
                               uint32_t* counts, cudaStream_t stream) {
  const long total = (long)a.batch * a.n_streams;
  const unsigned grid = (unsigned)((total + kThreadsPerBlock - 1) / kThreadsPerBlock);
  rans_encode_kernel<<<grid, kThreadsPerBlock, table_smem(a), stream>>>(a, z, prior, words, counts);
  return cudaGetLastError();
}

cudaError_t launch_rans_decode(const RansArgs& a, int block, const uint16_t* words, const uint32_t* counts,
                               const int32_t* prior, int32_t* z, cudaStream_t stream) {
  const long total = (long)a.batch * a.blocks[block].n_streams * 32;        // a warp per stream
  const unsigned grid = (unsigned)((total + kThreadsPerBlock - 1) / kThreadsPerBlock);
  rans_decode_kernel<<<grid, kThreadsPerBlock, table_smem(a), stream>>>(a, block, words, counts, prior, z);
  return cudaGetLastError();
}

}  // namespace iodf
