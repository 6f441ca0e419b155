// CPU oracle of the entropy-coding side of the integer flow: TEST INFRASTRUCTURE ONLY.
//
// Only tests, the smoke check and the benchmark's CPU-baseline leg may use this file. It shares no
// code with the CUDA path; it is a plain, sequential restatement of
//   * the factorised discrete logistic prior of Sec. 3,
//       p(z | mu, s) = sigma((z + 1/2 - mu) / s) - sigma((z - 1/2 - mu) / s),
//     in the integer form the codec fixes (the paper is silent on it): the sigmoid is a table G of
//     integers over u = x * 64 (a codec parameter, given by the caller), the scale is one of a
//     list of fixed-point reciprocals R[ls] = 2^21 / s (also given), and every symbol of the coded
//     window gets one extra count so that no frequency is zero;
//   * range-ANS coding as in App. A ("Asymmetric Numeral System"):
//       encode  X_t     = floor(X_{t-1} / F) * M + C + (X_{t-1} mod F)
//       decode  s_t     : C_s <= X_t mod M < C_s + F_s
//               X_{t-1} = floor(X_t / M) * F + (X_t mod M) - C
//     with M = 2^16, made streaming in the usual way (the appendix keeps one unbounded integer):
//     the state is kept in [2^16, 2^32) by moving its low 16 bits to the output before a step that
//     would overflow, and by reading 16 bits back after a step that underflows.
//
// Symbols. For an element with prior (mu, ls) the residual r = z - mu is coded as the symbol
// k = clamp(r, -2048, 2048) + 2048 in [0, 4096]; k = 0 and k = 4096 are escapes (r <= -2048,
// r >= 2048) after which the 32 bits of z follow as two uniform 16-bit symbols (high half first
// for the decoder). Cumulative counts, for k in [0, 4097]:
//       Cum(0) = 0,  Cum(4097) = M,
//       Cum(k) = k + G[clamp(floor((2 (k - 2048) - 1) * R[ls] / 2^16), -umax, umax) + umax]
// i.e. the table sigmoid at the lower edge r - 1/2 of symbol k's residual, plus k: strictly
// increasing because G is non-decreasing with G <= M - 4097.
//
// Streams. An image's latent is coded block by block (every factored-out block, then the final
// block), because a decoder learns a block's prior parameters only after the deeper blocks have
// been decoded and inverted. A block of n elements is cut into ceil(n / E) streams; stream j holds
// elements j, j + ns, j + 2 ns, ... The encoder visits a stream's elements last to first (rANS is a
// stack), appends the 16-bit words it moves out, and finally the state (low half, then high half);
// the decoder starts at the end of the stream's words and walks back.
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

constexpr int kWin = 2048;
constexpr uint32_t kM = 1u << 16;

struct Codec {
  const uint16_t* G;
  int umax;
  const uint32_t* R;
  int n_scales;
};

int64_t floor_div(int64_t a, int64_t b) {   // b > 0
  int64_t q = a / b;
  if ((a % b) != 0 && a < 0) --q;
  return q;
}

uint32_t cum(const Codec& c, int ls, int k) {
  if (k <= 0) return 0;
  if (k >= 2 * kWin + 1) return kM;
  const int64_t edge2 = 2 * (int64_t)(k - kWin) - 1;                 // twice the lower edge r - 1/2
  int64_t u = floor_div(edge2 * (int64_t)c.R[ls], (int64_t)1 << 16);
  if (u < -c.umax) u = -c.umax;
  if (u > c.umax) u = c.umax;
  return (uint32_t)k + c.G[u + c.umax];
}

int symbol_of(int64_t r) {
  if (r < -kWin) r = -kWin;
  if (r > kWin) r = kWin;
  return (int)r + kWin;
}

// one rANS step of App. A on the streaming state
void push(uint32_t& x, uint32_t F, uint32_t C, std::vector<uint16_t>& out) {
  if ((uint64_t)x >= ((uint64_t)F << 16)) {
    out.push_back((uint16_t)(x & 0xFFFFu));
    x >>= 16;
  }
  x = ((x / F) << 16) + (x % F) + C;
}

struct Reader {
  const uint16_t* w;
  long pos;      // next word to read is w[pos - 1]
  bool bad = false;
  uint32_t next() {
    if (pos <= 0) { bad = true; return 0; }
    return w[--pos];
  }
};

void pop(uint32_t& x, uint32_t F, uint32_t C, Reader& rd) {
  const uint32_t slot = x & 0xFFFFu;
  x = F * (x >> 16) + slot - C;
  if (x < (1u << 16)) x = (x << 16) | rd.next();
}

void prior_of(const int32_t* prior_img, long d_fact, long poff, long e, int final_ls, int32_t* mu, int* ls) {
  if (poff < 0) { *mu = 0; *ls = final_ls; return; }
  *mu = prior_img[poff + e];
  *ls = prior_img[d_fact + poff + e];
}

}  // namespace

extern "C" {

uint32_t orc_rans_cum(const uint16_t* G, int umax, const uint32_t* R, int n_scales, int ls, int k) {
  Codec c{G, umax, R, n_scales};
  return cum(c, ls, k);
}

// Encode one stream given per-element (z, mu, ls) in forward order. Returns the word count.
long orc_rans_encode_stream(const uint16_t* G, int umax, const uint32_t* R, int n_scales, const int32_t* z,
                            const int32_t* mu, const int32_t* ls, long n, uint16_t* words, long cap) {
  Codec c{G, umax, R, n_scales};
  std::vector<uint16_t> out;
  uint32_t x = 1u << 16;
  for (long i = n - 1; i >= 0; --i) {
    if (ls[i] < 0 || ls[i] >= n_scales) return -2;
    const int k = symbol_of((int64_t)z[i] - (int64_t)mu[i]);
    if (k == 0 || k == 2 * kWin) {
      push(x, 1, (uint32_t)z[i] & 0xFFFFu, out);
      push(x, 1, ((uint32_t)z[i] >> 16) & 0xFFFFu, out);
    }
    const uint32_t C = cum(c, ls[i], k), F = cum(c, ls[i], k + 1) - C;
    push(x, F, C, out);
  }
  out.push_back((uint16_t)(x & 0xFFFFu));
  out.push_back((uint16_t)(x >> 16));
  if ((long)out.size() > cap) return -1;
  std::memcpy(words, out.data(), out.size() * sizeof(uint16_t));
  return (long)out.size();
}

// Decode one stream of `count` words into z (forward order) given per-element (mu, ls). 0 on success.
int orc_rans_decode_stream(const uint16_t* G, int umax, const uint32_t* R, int n_scales, const uint16_t* words,
                           long count, const int32_t* mu, const int32_t* ls, long n, int32_t* z) {
  Codec c{G, umax, R, n_scales};
  Reader rd{words, count};
  uint32_t x = rd.next() << 16;
  x |= rd.next();
  for (long i = 0; i < n; ++i) {
    if (ls[i] < 0 || ls[i] >= n_scales) return -2;
    const uint32_t slot = x & 0xFFFFu;
    int lo = 0, hi = 2 * kWin;                      // largest k with Cum(k) <= slot
    while (lo < hi) {
      const int mid = (lo + hi + 1) / 2;
      if (cum(c, ls[i], mid) <= slot) lo = mid; else hi = mid - 1;
    }
    const int k = lo;
    const uint32_t C = cum(c, ls[i], k), F = cum(c, ls[i], k + 1) - C;
    pop(x, F, C, rd);
    if (k == 0 || k == 2 * kWin) {
      const uint32_t h = x & 0xFFFFu;
      pop(x, 1, h, rd);
      const uint32_t l = x & 0xFFFFu;
      pop(x, 1, l, rd);
      z[i] = (int32_t)((h << 16) | l);
    } else {
      z[i] = (int32_t)((int64_t)mu[i] + (k - kWin));
    }
  }
  if (rd.bad || rd.pos != 0 || x != (1u << 16)) return -1;   // every word used, state back at its start
  return 0;
}

// Whole batch. Blocks: nblocks entries {z offset, element count, prior offset or -1 (fixed prior:
// mu = 0, ls = final_ls)}. Streams of an image are numbered block by block. words is
// [B][n_streams][cap], counts [B][n_streams].
int orc_rans_encode(const uint16_t* G, int umax, const uint32_t* R, int n_scales, int final_ls, long E,
                    const int32_t* z, const int32_t* prior, long B, long d, long d_fact, int nblocks,
                    const long* blk_zoff, const long* blk_n, const long* blk_poff, long n_streams, long cap,
                    uint16_t* words, uint32_t* counts) {
  for (long b = 0; b < B; ++b) {
    long s0 = 0;
    for (int q = 0; q < nblocks; ++q) {
      const long n = blk_n[q], ns = (n + E - 1) / E;
      for (long j = 0; j < ns; ++j) {
        std::vector<int32_t> zz, mu, ls;
        for (long e = j; e < n; e += ns) {
          int32_t m; int l;
          prior_of(prior + b * 2 * d_fact, d_fact, blk_poff[q], e, final_ls, &m, &l);
          zz.push_back(z[b * d + blk_zoff[q] + e]); mu.push_back(m); ls.push_back(l);
        }
        const long cnt = orc_rans_encode_stream(G, umax, R, n_scales, zz.data(), mu.data(), ls.data(),
                                                (long)zz.size(), words + (b * n_streams + s0 + j) * cap, cap);
        if (cnt < 0) return (int)cnt;
        counts[b * n_streams + s0 + j] = (uint32_t)cnt;
      }
      s0 += ns;
    }
    if (s0 != n_streams) return -3;
  }
  return 0;
}

// Decode block q of every image into z (the other blocks of z are left alone).
int orc_rans_decode_block(const uint16_t* G, int umax, const uint32_t* R, int n_scales, int final_ls, long E,
                          const uint16_t* words, const uint32_t* counts, const int32_t* prior, long B, long d,
                          long d_fact, int nblocks, const long* blk_zoff, const long* blk_n, const long* blk_poff,
                          long n_streams, long cap, int q, int32_t* z) {
  long s0 = 0;
  for (int p = 0; p < q; ++p) s0 += (blk_n[p] + E - 1) / E;
  const long n = blk_n[q], ns = (n + E - 1) / E;
  for (long b = 0; b < B; ++b)
    for (long j = 0; j < ns; ++j) {
      std::vector<int32_t> mu, ls;
      std::vector<long> where;
      for (long e = j; e < n; e += ns) {
        int32_t m; int l;
        prior_of(prior + b * 2 * d_fact, d_fact, blk_poff[q], e, final_ls, &m, &l);
        mu.push_back(m); ls.push_back(l); where.push_back(b * d + blk_zoff[q] + e);
      }
      std::vector<int32_t> zz(mu.size());
      const int rc = orc_rans_decode_stream(G, umax, R, n_scales, words + (b * n_streams + s0 + j) * cap,
                                            counts[b * n_streams + s0 + j], mu.data(), ls.data(), (long)mu.size(),
                                            zz.data());
      if (rc) return rc;
      for (size_t i = 0; i < zz.size(); ++i) z[where[i]] = zz[i];
    }
  return 0;
}

}  // extern "C"
