// CPU oracle for integer-only discrete flow inference (IODF, arXiv 2206.08869).
//
// TEST INFRASTRUCTURE ONLY. This file is the slow, literal definition that the CUDA library is
// compared against; nothing on the product path may call it. It shares no code, header, table
// or helper with the CUDA sources.
//
// Every tensor is a dense NCHW array of int32 (or int64 for accumulators); every convolution is
// the seven nested loops of Eq. 5; nothing is tiled, fused, vectorised or reordered.
//
// What each function follows:
//   rq            Eq. "quant_conv" (Sec. 4.1): y = (s_W s_x / s_y) * acc + b / s_y, with the real
//                 multiplier written as M0 * 2^-(31+s) and rounded half up (ties toward +inf).
//   conv_acc      Eq. 5 (Sec. 4.1): y_c = sum_c' W_{c,c'} (*) x_c' + b_c, stride 1, zero padding
//                 (k-1)/2 so the map keeps its shape (App. B.1), int32 accumulator + int32 bias.
//   hidden layers Sec. 4.1 "Integer-Only ReLU": max(0, .) on the integer part, then the 8-bit clip.
//   gate          Eq. 8 (Sec. 4.4): a filter whose binary gate is 0 outputs an all-zero map.
//   residual t    Eq. 3 (Sec. 4.1) and the scatter add of Sec. 4.5: a coupling whose network is
//                 conv -> L x [ ReLU(SAdd(Q(x), GConv(ReLU(GConv(Q(x)))))) ] -> conv (App. B.1: eight
//                 blocks, 3x3 convs, 128 hidden channels). In integers (a reading, the paper
//                 requantises in floating point): the block input x is an 8-bit tensor of D channels
//                 and feeds the first conv as it is; the second conv's requantised outputs (kept
//                 channels only) are added, through their index list, to the requantised shortcut
//                 rq(x; M_r, s_r) of all D channels; then max(0, .) and the block's clip.
//   coupling      Eq. 2 (Sec. 3): z_a = x_a, z_b = x_b + round(t(x_a)); inverse subtracts.
//   levels        Sec. 5 / App. B.1: L levels of D couplings; 2x2 space-to-depth before a level;
//                 half of the channels factored out after it; the prior head gives (mu, log-scale
//                 index) of the factored-out half from the kept half (Sec. 3, factorised
//                 discretised logistic prior).
//
// Readings taken where the paper is silent (the same list is in the design notes):
//   squeeze order out[c*4 + dy*2 + dx][i][j] = in[c][2i+dy][2j+dx]; before a coupling
//   y[k] = x[perm[k]]; x_a = first half (feeds the network), x_b = second half (is updated);
//   kept half = first half of the channels, factored-out half = second half; flow-variable
//   adds/subtracts wrap modulo 2^32; bias is added to the accumulator before requantisation.
//
// Parity against the authors' implementation is UNPINNED: the paper prints no integer
// input/output pair and requantises in floating point. The pins are the invariants and brute-force
// checks under tests/ (exact invertibility, rational rounding, brute-force convolution, closed
// form index maps, masked == compact == zero-padded).
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>
#include <atomic>
#include <algorithm>

namespace {

typedef std::vector<int32_t> T32;  // [C][H][W]

struct Layer {
  int k, c_in, c_out, relu, has_clamp, clamp_lo, clamp_hi, has_gate;
  const int8_t* w;       // [c_out][k][k][c_in]
  const int32_t* bias;   // [c_out]
  const int32_t* m0;     // [c_out]
  const int32_t* s;      // [c_out]
  const int32_t* gate;   // [c_out] or null
};
struct ResBlock {                  // block l uses layers[1 + 2l] and layers[2 + 2l] of its coupling
  int32_t short_m0, short_s;       // shortcut requantisation Q(x), per tensor
  int32_t clamp_lo, clamp_hi;      // clip after the block's ReLU
  std::vector<int32_t> idx;        // channel of the block's D-wide tensor that receives output j of the second conv
};
struct Coupling {
  std::vector<int32_t> perm;
  int32_t in_m0, in_s;
  std::vector<Layer> layers;
  std::vector<ResBlock> blocks;    // empty: plain chain of layers; else [conv_in, (conv_a, conv_b) per block, conv_out]
};
struct Head {
  int32_t in_m0, in_s, ls_lo, ls_hi;
  Layer layer;
};
struct Level {
  int c, h, w, split, has_prior;
  std::vector<Coupling> couplings;
  Head head;
};
struct Model {
  int in_c, in_h, in_w;
  std::vector<Level> levels;
  long d, d_fact;
};

// floor((a * M0 + 2^(30+s)) / 2^(31+s)) in 128-bit integers, floor division written out.
int64_t rq(int64_t a, int32_t m0, int32_t s) {
  __int128 num = (__int128)a * (__int128)m0 + ((__int128)1 << (30 + s));
  __int128 den = (__int128)1 << (31 + s);
  __int128 q = num / den;              // truncates toward zero
  if (num % den != 0 && num < 0) q -= 1;
  return (int64_t)q;
}

int64_t clampi(int64_t v, int64_t lo, int64_t hi) { return v < lo ? lo : (v > hi ? hi : v); }

// acc[co][i][j] = bias[co] + sum_{ci,u,v} W[co][u][v][ci] * in[ci][i+u-p][j+v-p], zero outside.
// Returns false if an accumulator leaves the int32 range.
bool conv_acc(const Layer& L, const int32_t* in, int h, int w, std::vector<int64_t>& acc) {
  const int k = L.k, p = (k - 1) / 2;
  acc.assign((size_t)L.c_out * h * w, 0);
  bool ok = true;
  for (int co = 0; co < L.c_out; ++co)
    for (int i = 0; i < h; ++i)
      for (int j = 0; j < w; ++j) {
        int64_t a = 0;
        for (int ci = 0; ci < L.c_in; ++ci)
          for (int u = 0; u < k; ++u)
            for (int v = 0; v < k; ++v) {
              int ii = i + u - p, jj = j + v - p;
              if (ii < 0 || ii >= h || jj < 0 || jj >= w) continue;
              a += (int64_t)L.w[(((size_t)co * k + u) * k + v) * L.c_in + ci] *
                   (int64_t)in[((size_t)ci * h + ii) * w + jj];
            }
        a += (int64_t)L.bias[co];
        if (a > INT32_MAX || a < INT32_MIN) ok = false;
        acc[((size_t)co * h + i) * w + j] = a;
      }
  return ok;
}

// One conv layer: accumulate, requantise per output channel, optional ReLU, optional clip, gate.
bool run_layer(const Layer& L, const T32& in, int h, int w, std::vector<int64_t>& out) {
  std::vector<int64_t> acc;
  bool ok = conv_acc(L, in.data(), h, w, acc);
  out.resize(acc.size());
  for (int co = 0; co < L.c_out; ++co)
    for (int q = 0; q < h * w; ++q) {
      int64_t y = rq(acc[(size_t)co * h * w + q], L.m0[co], L.s[co]);
      if (L.relu) y = std::max<int64_t>(y, 0);
      if (L.has_clamp) y = clampi(y, L.clamp_lo, L.clamp_hi);
      if (L.has_gate && L.gate[co] == 0) y = 0;
      out[(size_t)co * h * w + q] = y;
    }
  return ok;
}

// t = round(t_theta(x_a)): input requant to int8, then the layer list. x_a is [ca][h][w].
bool translation(const Coupling& cp, const int32_t* xa, int ca, int h, int w, std::vector<int64_t>& t) {
  T32 a((size_t)ca * h * w);
  for (size_t i = 0; i < a.size(); ++i) a[i] = (int32_t)clampi(rq(xa[i], cp.in_m0, cp.in_s), -128, 127);
  bool ok = true;
  std::vector<int64_t> y;
  if (!cp.blocks.empty()) {
    const size_t px = (size_t)h * w;
    ok = run_layer(cp.layers[0], a, h, w, y) && ok;                      // conv_in -> x of the first block
    T32 x(y.begin(), y.end());
    const int D = cp.layers[0].c_out;
    for (size_t b = 0; b < cp.blocks.size(); ++b) {
      const ResBlock& rb = cp.blocks[b];
      std::vector<int64_t> mid, br;
      ok = run_layer(cp.layers[1 + 2 * b], x, h, w, mid) && ok;          // ReLU(GConv(Q(x)))
      T32 m32(mid.begin(), mid.end());
      ok = run_layer(cp.layers[2 + 2 * b], m32, h, w, br) && ok;         // GConv(.), kept channels only
      std::vector<int64_t> sum((size_t)D * px);
      for (size_t i = 0; i < sum.size(); ++i) sum[i] = rq(x[i], rb.short_m0, rb.short_s);   // Q(x), all D channels
      for (size_t j = 0; j < rb.idx.size(); ++j)                          // scatter add
        for (size_t q = 0; q < px; ++q) sum[(size_t)rb.idx[j] * px + q] += br[j * px + q];
      for (size_t i = 0; i < sum.size(); ++i)
        x[i] = (int32_t)clampi(std::max<int64_t>(sum[i], 0), rb.clamp_lo, rb.clamp_hi);
    }
    ok = run_layer(cp.layers.back(), x, h, w, y) && ok;                  // conv_out -> translation
    t.swap(y);
    for (size_t i = 0; i < t.size(); ++i)
      if (t[i] > INT32_MAX || t[i] < INT32_MIN) ok = false;
    return ok;
  }
  for (size_t li = 0; li < cp.layers.size(); ++li) {
    ok = run_layer(cp.layers[li], a, h, w, y) && ok;
    if (li + 1 < cp.layers.size()) {
      a.resize(y.size());
      for (size_t i = 0; i < y.size(); ++i) a[i] = (int32_t)y[i];
    }
  }
  t.swap(y);
  for (size_t i = 0; i < t.size(); ++i)
    if (t[i] > INT32_MAX || t[i] < INT32_MIN) ok = false;
  return ok;
}

T32 squeeze(const T32& x, int c, int h, int w) {
  T32 y((size_t)c * h * w);
  int h2 = h / 2, w2 = w / 2;
  for (int ch = 0; ch < c; ++ch)
    for (int dy = 0; dy < 2; ++dy)
      for (int dx = 0; dx < 2; ++dx)
        for (int i = 0; i < h2; ++i)
          for (int j = 0; j < w2; ++j)
            y[((size_t)(ch * 4 + dy * 2 + dx) * h2 + i) * w2 + j] = x[((size_t)ch * h + 2 * i + dy) * w + 2 * j + dx];
  return y;
}

T32 unsqueeze(const T32& y, int c4, int h2, int w2) {  // inverse of squeeze: c4 = 4c channels at h2 x w2
  int c = c4 / 4, h = h2 * 2, w = w2 * 2;
  T32 x((size_t)c * h * w);
  for (int ch = 0; ch < c; ++ch)
    for (int dy = 0; dy < 2; ++dy)
      for (int dx = 0; dx < 2; ++dx)
        for (int i = 0; i < h2; ++i)
          for (int j = 0; j < w2; ++j)
            x[((size_t)ch * h + 2 * i + dy) * w + 2 * j + dx] = y[((size_t)(ch * 4 + dy * 2 + dx) * h2 + i) * w2 + j];
  return x;
}

// Prior head: (mu, ls) for the factored-out half from the kept half (first c_keep channels of v).
bool prior_params(const Head& hd, const int32_t* keep, int c_keep, int h, int w, int32_t* mu, int32_t* ls) {
  T32 a((size_t)c_keep * h * w);
  for (size_t i = 0; i < a.size(); ++i) a[i] = (int32_t)clampi(rq(keep[i], hd.in_m0, hd.in_s), -128, 127);
  std::vector<int64_t> y;
  bool ok = run_layer(hd.layer, a, h, w, y);
  int c_out = hd.layer.c_out / 2;
  size_t n = (size_t)c_out * h * w;
  for (size_t i = 0; i < n; ++i) {
    if (y[i] > INT32_MAX || y[i] < INT32_MIN) ok = false;
    mu[i] = (int32_t)y[i];
    ls[i] = (int32_t)clampi(y[n + i], hd.ls_lo, hd.ls_hi);
  }
  return ok;
}

// x (u8 CHW) -> z (per-image latent, blocks in level order, final block last) and prior params.
// stop_level >= 0: return the flow variable right after coupling `stop_coupling` of that level
// (channel order as the coupling sees it) in `trace` and stop.
bool forward_one(const Model& M, const uint8_t* x, int32_t* z, int32_t* mu, int32_t* ls,
                 int stop_level, int stop_coupling, int32_t* trace) {
  T32 v((size_t)M.in_c * M.in_h * M.in_w);
  for (size_t i = 0; i < v.size(); ++i) v[i] = (int32_t)x[i];
  int c = M.in_c, h = M.in_h, w = M.in_w;
  size_t zo = 0, po = 0;
  bool ok = true;
  for (size_t li = 0; li < M.levels.size(); ++li) {
    const Level& lv = M.levels[li];
    v = squeeze(v, c, h, w);
    c *= 4; h /= 2; w /= 2;
    const int ca = c / 2, cb = c - ca, px = h * w;
    for (size_t ki = 0; ki < lv.couplings.size(); ++ki) {
      const Coupling& cp = lv.couplings[ki];
      T32 y(v.size());
      for (int k = 0; k < c; ++k)
        std::memcpy(&y[(size_t)k * px], &v[(size_t)cp.perm[k] * px], sizeof(int32_t) * px);
      std::vector<int64_t> t;
      ok = translation(cp, y.data(), ca, h, w, t) && ok;
      for (size_t i = 0; i < (size_t)cb * px; ++i)
        y[(size_t)ca * px + i] = (int32_t)((uint32_t)y[(size_t)ca * px + i] + (uint32_t)(int32_t)t[i]);
      v.swap(y);
      if ((int)li == stop_level && (int)ki == stop_coupling) {
        std::memcpy(trace, v.data(), sizeof(int32_t) * v.size());
        return ok;
      }
    }
    if (lv.split) {
      std::memcpy(z + zo, &v[(size_t)ca * px], sizeof(int32_t) * cb * px);
      zo += (size_t)cb * px;
      if (lv.has_prior) {
        if (mu) ok = prior_params(lv.head, v.data(), ca, h, w, mu + po, ls + po) && ok;
        po += (size_t)cb * px;
      }
      v.resize((size_t)ca * px);
      c = ca;
    }
  }
  std::memcpy(z + zo, v.data(), sizeof(int32_t) * v.size());
  return ok;
}

bool inverse_one(const Model& M, const int32_t* z, int32_t* x_out, int32_t* mu, int32_t* ls) {
  // shapes and offsets of every block
  std::vector<size_t> zoff(M.levels.size()), poff(M.levels.size());
  size_t zo = 0, po = 0;
  int c = M.in_c, h = M.in_h, w = M.in_w;
  for (size_t li = 0; li < M.levels.size(); ++li) {
    const Level& lv = M.levels[li];
    c *= 4; h /= 2; w /= 2;
    zoff[li] = zo; poff[li] = po;
    if (lv.split) {
      int cb = c - c / 2;
      zo += (size_t)cb * h * w;
      if (lv.has_prior) po += (size_t)cb * h * w;
      c = c / 2;
    }
  }
  T32 v(z + zo, z + zo + (size_t)c * h * w);  // final block
  bool ok = true;
  for (int li = (int)M.levels.size() - 1; li >= 0; --li) {
    const Level& lv = M.levels[li];
    const int px = h * w;
    if (lv.split) {
      int ca = c, cb = lv.c - ca;
      if (lv.has_prior && mu) ok = prior_params(lv.head, v.data(), ca, h, w, mu + poff[li], ls + poff[li]) && ok;
      v.resize((size_t)lv.c * px);
      std::memcpy(&v[(size_t)ca * px], z + zoff[li], sizeof(int32_t) * cb * px);
      c = lv.c;
    }
    const int ca = c / 2, cb = c - ca;
    for (int ki = (int)lv.couplings.size() - 1; ki >= 0; --ki) {
      const Coupling& cp = lv.couplings[ki];
      std::vector<int64_t> t;
      ok = translation(cp, v.data(), ca, h, w, t) && ok;
      for (size_t i = 0; i < (size_t)cb * px; ++i)
        v[(size_t)ca * px + i] = (int32_t)((uint32_t)v[(size_t)ca * px + i] - (uint32_t)(int32_t)t[i]);
      T32 y(v.size());
      for (int k = 0; k < c; ++k)
        std::memcpy(&y[(size_t)cp.perm[k] * px], &v[(size_t)k * px], sizeof(int32_t) * px);
      v.swap(y);
    }
    v = unsqueeze(v, c, h, w);
    c /= 4; h *= 2; w *= 2;
  }
  std::memcpy(x_out, v.data(), sizeof(int32_t) * v.size());
  return ok;
}

// ---- descriptor parsing -------------------------------------------------------------------------
struct Cursor {
  const int32_t* p; long n, i;
  bool ok;
  int32_t next() { if (i >= n) { ok = false; return 0; } return p[i++]; }
};

bool parse_layer(Cursor& cu, const int8_t* wts, const int32_t* par, Layer& L) {
  L.k = cu.next(); L.c_in = cu.next(); L.c_out = cu.next(); L.relu = cu.next();
  L.has_clamp = cu.next(); L.clamp_lo = cu.next(); L.clamp_hi = cu.next(); L.has_gate = cu.next();
  long w_off = cu.next(), p_off = cu.next();
  if (!cu.ok || (L.k != 1 && L.k != 3) || L.c_in < 1 || L.c_out < 1) return false;
  L.w = wts + w_off;
  L.bias = par + p_off; L.m0 = L.bias + L.c_out; L.s = L.m0 + L.c_out;
  L.gate = L.has_gate ? L.s + L.c_out : nullptr;
  for (int i = 0; i < L.c_out; ++i)
    if (L.m0[i] < (1 << 30) || L.s[i] < 0 || L.s[i] > 31) return false;
  return true;
}

bool parse(const int32_t* desc, long n, const int8_t* wts, const int32_t* par, Model& M) {
  Cursor cu{desc, n, 0, true};
  if (cu.next() != 0x10DF) return false;
  M.in_c = cu.next(); M.in_h = cu.next(); M.in_w = cu.next();
  int nl = cu.next();
  if (!cu.ok || nl < 1 || nl > 16) return false;
  int c = M.in_c, h = M.in_h, w = M.in_w;
  M.d = 0; M.d_fact = 0;
  for (int li = 0; li < nl; ++li) {
    Level lv;
    if (h % 2 || w % 2) return false;
    c *= 4; h /= 2; w /= 2;
    lv.c = c; lv.h = h; lv.w = w;
    int nk = cu.next(); lv.split = cu.next(); lv.has_prior = cu.next();
    if (!cu.ok || nk < 0 || c % 2) return false;
    for (int ki = 0; ki < nk; ++ki) {
      Coupling cp;
      if (cu.next() != c) return false;
      std::vector<int> seen(c, 0);
      for (int k = 0; k < c; ++k) {
        int pk = cu.next();
        if (pk < 0 || pk >= c || seen[pk]) return false;
        seen[pk] = 1; cp.perm.push_back(pk);
      }
      cp.in_m0 = cu.next(); cp.in_s = cu.next();
      int nlay = cu.next();
      int nblk = cu.next();
      if (!cu.ok || nlay < 1 || nblk < 0 || cp.in_m0 < (1 << 30) || cp.in_s < 0 || cp.in_s > 31) return false;
      if (nblk > 0 && nlay != 2 + 2 * nblk) return false;
      int cin = c / 2, D = 0;
      for (int q = 0; q < nlay; ++q) {
        Layer L;
        if (!parse_layer(cu, wts, par, L) || L.c_in != cin) return false;
        cin = L.c_out;
        if (q == 0) D = L.c_out;
        // after a block's second conv the tensor is D wide again, whatever that conv keeps
        if (nblk > 0 && q >= 2 && q % 2 == 0 && q < nlay - 1) cin = D;
        cp.layers.push_back(L);
      }
      if (cin != c - c / 2) return false;
      for (int b = 0; b < nblk; ++b) {
        ResBlock rb;
        rb.short_m0 = cu.next(); rb.short_s = cu.next(); rb.clamp_lo = cu.next(); rb.clamp_hi = cu.next();
        int nidx = cu.next();
        if (!cu.ok || rb.short_m0 < (1 << 30) || rb.short_s < 0 || rb.short_s > 31 || rb.clamp_lo > rb.clamp_hi)
          return false;
        const Layer& second = cp.layers[2 + 2 * b];
        if (nidx != second.c_out || second.relu || second.has_clamp) return false;
        std::vector<int> used(D, 0);
        for (int j = 0; j < nidx; ++j) {
          int ch = cu.next();
          if (!cu.ok || ch < 0 || ch >= D || used[ch]) return false;
          used[ch] = 1; rb.idx.push_back(ch);
        }
        cp.blocks.push_back(rb);
      }
      lv.couplings.push_back(cp);
    }
    if (lv.has_prior) {
      if (!lv.split) return false;
      lv.head.in_m0 = cu.next(); lv.head.in_s = cu.next();
      if (!parse_layer(cu, wts, par, lv.head.layer)) return false;
      lv.head.ls_lo = cu.next(); lv.head.ls_hi = cu.next();
      if (lv.head.layer.c_in != c / 2 || lv.head.layer.c_out != 2 * (c - c / 2)) return false;
    }
    if (lv.split) {
      M.d += (long)(c - c / 2) * h * w;
      if (lv.has_prior) M.d_fact += (long)(c - c / 2) * h * w;
      c = c / 2;
    }
    M.levels.push_back(lv);
  }
  M.d += (long)c * h * w;
  return cu.ok && cu.i == cu.n;
}

template <class F>
bool for_images(int B, int threads, F fn) {
  std::atomic<int> next(0);
  std::atomic<bool> ok(true);
  threads = std::max(1, std::min(threads, B));
  std::vector<std::thread> pool;
  for (int t = 0; t < threads; ++t)
    pool.emplace_back([&]() {
      for (;;) {
        int b = next.fetch_add(1);
        if (b >= B) break;
        if (!fn(b)) ok = false;
      }
    });
  for (auto& th : pool) th.join();
  return ok;
}

}  // namespace

// ---- C entry points (called from Python tests through ctypes) ------------------------------------
// Return 0 on success, -1 bad descriptor, -2 an accumulator or translation left the int32 range.
extern "C" {

int64_t orc_rq(int64_t a, int32_t m0, int32_t s) { return rq(a, m0, s); }

int orc_layout(const int32_t* desc, long n, const int8_t* wts, const int32_t* par, long* d, long* d_fact) {
  Model M;
  if (!parse(desc, n, wts, par, M)) return -1;
  *d = M.d; *d_fact = M.d_fact;
  return 0;
}

// Plain convolution accumulator (bias included) for one image: in int32 [c_in][h][w] -> int64.
int orc_conv_acc(int k, int c_in, int c_out, const int8_t* w, const int32_t* bias, const int32_t* in,
                 int h, int wd, int64_t* out) {
  Layer L{};
  L.k = k; L.c_in = c_in; L.c_out = c_out; L.w = w; L.bias = bias;
  std::vector<int64_t> acc;
  bool ok = conv_acc(L, in, h, wd, acc);
  std::copy(acc.begin(), acc.end(), out);
  return ok ? 0 : -2;
}

void orc_squeeze(const int32_t* x, int c, int h, int w, int32_t* y) {
  T32 in(x, x + (size_t)c * h * w);
  T32 o = squeeze(in, c, h, w);
  std::copy(o.begin(), o.end(), y);
}

void orc_unsqueeze(const int32_t* y, int c4, int h2, int w2, int32_t* x) {
  T32 in(y, y + (size_t)c4 * h2 * w2);
  T32 o = unsqueeze(in, c4, h2, w2);
  std::copy(o.begin(), o.end(), x);
}

int orc_forward(const int32_t* desc, long n, const int8_t* wts, const int32_t* par, const uint8_t* x,
                int B, int32_t* z, int32_t* prior, int threads) {
  Model M;
  if (!parse(desc, n, wts, par, M)) return -1;
  const size_t xin = (size_t)M.in_c * M.in_h * M.in_w;
  bool ok = for_images(B, threads, [&](int b) {
    int32_t* mu = prior ? prior + (size_t)b * 2 * M.d_fact : nullptr;
    return forward_one(M, x + b * xin, z + (size_t)b * M.d, mu, mu ? mu + M.d_fact : nullptr, -1, -1, nullptr);
  });
  return ok ? 0 : -2;
}

int orc_trace(const int32_t* desc, long n, const int8_t* wts, const int32_t* par, const uint8_t* x,
              int level, int coupling, int32_t* v_out) {
  Model M;
  if (!parse(desc, n, wts, par, M)) return -1;
  if (level < 0 || level >= (int)M.levels.size() || coupling < 0 ||
      coupling >= (int)M.levels[level].couplings.size()) return -1;
  std::vector<int32_t> z(M.d);
  return forward_one(M, x, z.data(), nullptr, nullptr, level, coupling, v_out) ? 0 : -2;
}

int orc_inverse(const int32_t* desc, long n, const int8_t* wts, const int32_t* par, const int32_t* z,
                int B, uint8_t* x_u8, int32_t* x_i32, int32_t* prior, uint32_t* out_of_range, int threads) {
  Model M;
  if (!parse(desc, n, wts, par, M)) return -1;
  const size_t xin = (size_t)M.in_c * M.in_h * M.in_w;
  std::atomic<uint32_t> oor(0);
  bool ok = for_images(B, threads, [&](int b) {
    std::vector<int32_t> xi(xin);
    int32_t* mu = prior ? prior + (size_t)b * 2 * M.d_fact : nullptr;
    bool r = inverse_one(M, z + (size_t)b * M.d, xi.data(), mu, mu ? mu + M.d_fact : nullptr);
    uint32_t cnt = 0;
    for (size_t i = 0; i < xin; ++i) {
      if (xi[i] < 0 || xi[i] > 255) ++cnt;
      x_u8[b * xin + i] = (uint8_t)((uint32_t)xi[i] & 0xFFu);
      if (x_i32) x_i32[b * xin + i] = xi[i];
    }
    oor += cnt;
    return r;
  });
  if (out_of_range) *out_of_range = oor.load();
  return ok ? 0 : -2;
}

}  // extern "C"
