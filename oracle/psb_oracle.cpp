// Reference (oracle) implementation of progressive stochastic binarization (PSB)
// inference layers.  TEST INFRASTRUCTURE ONLY: plain, single-threaded, slow, and
// written to be checked against the paper by eye.  It shares no code with the
// CUDA library and must never be called from the product path.
//
// Everything here follows "Progressive Stochastic Binarization of Deep Networks"
// (arXiv 1904.02205).  Section / equation numbers below refer to that paper:
//   Eq. 1   y = relu(sum_i x_i w_i)                                   (Sec. 3)
//   Eq. 4   w -> s * 2^e * (B_p + 1)                                  (Sec. 3.1)
//   Eq. 5-7 s = sign w, e = floor(log2 |w|), p = |w| / 2^e - 1        (Sec. 3.1)
//   Eq. 8   w -> s * 2^e * (B_{n,p} / n + 1)   ("capacitor", n draws) (Sec. 3.1)
//   Eq. 9   x * w_n = s * (sum_i x << (e + B_p^(i))) >> log2 n        (Sec. 3.1)
//
// Readings taken where the paper is silent (all listed again in the design notes):
//   * w == 0 and sub-normal weights carry nothing (class ZERO); non-finite weights
//     are an error.
//   * exponents live in a window of 2^exp_bits octaves below the largest exponent
//     of the group (whole layer, or one output channel); smaller weights flush to
//     ZERO (Fig. 1 caption: very deep shifts of integers give 0; Sec. 4.4: 4-bit
//     exponents suffice).
//   * one set of draws per weight and per call, shared by every batch element and
//     every output location (Sec. 4.1: the filter itself is sampled).
//   * the number of draws k is a power of two; level k uses draws 0..k-1 of one
//     stream, so larger levels refine smaller ones ("progressive").
//   * the division by k (the ">> n" of Eq. 9) is never applied to integers: the
//     accumulator stays exact and 1/k is folded into the floating-point scale.
//   * optional (Sec. 3.1 "Stochastic multiplication", applied at the floor of the window): a weight
//     below the window, |w| < 2^e_base, is not flushed but replaced per draw by s * 2^e_base * B_q with
//     q = |w| / 2^e_base, the plain Bernoulli gate of Eq. 2-3; unbiased, no "+ 1" term.
//   * optional (Sec. 4.4): probabilities stored with b bits on the regular grid {0, 1/2^b, ...,
//     1 - 1/2^b}; p is rounded to the nearest grid point, and a p that rounds to 1 becomes p = 0 at the
//     next exponent (the grid leaves 1 out because it belongs there).  The comparator then has
//     b bits (supplement, "Stochastic multiplier") and one Philox word serves floor(32 / b) draws.
//     The deterministic variant of Sec. 4.4 uses the upper shift in round(p_q * k) of the k cases.
//   * the random stream is Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11),
//     counter = (draw / 4, layer, lo32(weight index), hi32(weight index)),
//     key = (lo32(seed), hi32(seed)); draw j uses output word j mod 4.
//
// Build:  g++ -O2 -std=c++17 -ffp-contract=off -fPIC -shared psb_oracle.cpp -o libpsb_oracle.so

#include <cmath>
#include <cstdint>
#include <cstring>

namespace {

enum { CLASS_ZERO = 0, CLASS_NORMAL = 1, CLASS_NONFINITE = 2 };

// Eq. 5-7 read off the IEEE-754 binary32 fields: for a normal number
// |w| = 2^(E-127) * (1 + m / 2^23), hence e = E - 127 and p = m / 2^23 exactly.
struct Decoded {
  int cls;
  int s;         // 0 for +, 1 for -
  int e;         // floor(log2 |w|)
  uint32_t m;    // p * 2^23
};

Decoded decode(float w) {
  uint32_t u;
  std::memcpy(&u, &w, 4);
  Decoded d;
  d.s = (int)(u >> 31);
  uint32_t E = (u >> 23) & 0xFFu;
  d.m = u & 0x7FFFFFu;
  d.e = (int)E - 127;
  d.cls = (E == 0) ? CLASS_ZERO : (E == 255 ? CLASS_NONFINITE : CLASS_NORMAL);
  return d;
}

// Philox4x32-10 as published (SC'11, Sec. 4 and Table 2 of that paper): a 4-word
// counter, a 2-word key, ten rounds; the key is bumped by the Weyl constants
// between rounds.
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  const uint64_t M0 = 0xD2511F53ull, M1 = 0xCD9E8D57ull;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = M0 * c0;
    uint64_t p1 = M1 * c2;
    uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// One Bernoulli draw B_p of Eq. 4: compare a uniform 32-bit word with p * 2^32.
// This is the comparator of the paper's stochastic multiplier (supplement,
// "Stochastic multiplier").  Pr[bit = 1] = (m << 9) / 2^32 = p exactly.
int draw_bit_thr(uint64_t seed, uint32_t layer, uint64_t index, uint32_t j, uint32_t T) {
  uint32_t ctr[4] = {j >> 2, layer, (uint32_t)index, (uint32_t)(index >> 32)};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t r[4];
  philox4x32_10(ctr, key, r);
  return r[j & 3] < T ? 1 : 0;      // Pr[1] = T / 2^32
}

int draw_bit(uint64_t seed, uint32_t layer, uint64_t index, uint32_t j, uint32_t m) {
  return draw_bit_thr(seed, layer, index, j, m << 9);
}

inline int64_t ipow2(int n) { return (int64_t)1 << n; }

// Sec. 4.4: the probability on a grid of 2^b points, nearest point, p = 1 carried into the exponent.
// Returns the quantised (e, p * 2^b).  b == 0 leaves the weight as it is (p * 2^23 in *pq).
void quantise(const Decoded& d, uint32_t b, int* e, uint32_t* pq) {
  *e = d.e;
  if (b == 0) { *pq = d.m; return; }
  uint32_t q = (d.m + (1u << (22 - b))) >> (23 - b);     // round half up to b bits
  if (q == (1u << b)) {
    if (d.e < 127) { *e = d.e + 1; q = 0; }              // the next power of two, exactly
    else q = (1u << b) - 1;                              // no exponent above: the last grid point
  }
  *pq = q;
}

// One draw with a b-bit comparator: draw j takes bit field (j mod n) of output word ((j / n) mod 4) of
// Philox call j / (4 n), n = floor(32 / b) fields per word, field f = bits [f b, f b + b).
int draw_bit_packed(uint64_t seed, uint32_t layer, uint64_t index, uint32_t j, uint32_t thr, uint32_t b) {
  const uint32_t n = 32u / b;
  uint32_t ctr[4] = {j / (4u * n), layer, (uint32_t)index, (uint32_t)(index >> 32)};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t r[4];
  philox4x32_10(ctr, key, r);
  const uint32_t field = (r[(j / n) & 3u] >> ((j % n) * b)) & ((1u << b) - 1u);
  return field < thr ? 1 : 0;
}

// What one weight turns into under a given window: W_k = s (base k + c_k) 2^sh, c_k counting draws with
// Pr[1] = thr / 2^32 (b == 0) or thr / 2^b.
struct Sampled {
  int live;        // 0: contributes nothing
  uint32_t base;   // 1: a weight inside the window (Eq. 8); 0: the Bernoulli gate below it
  int sh;
  uint32_t thr;
};

Sampled classify(const Decoded& d, int e_base, uint32_t b, uint32_t underflow) {
  Sampled r = {0, 0, 0, 0};
  if (d.cls != CLASS_NORMAL) return r;
  int e;
  uint32_t pq;
  quantise(d, b, &e, &pq);
  if (e >= e_base) {
    r.live = 1; r.base = 1; r.sh = e - e_base;
    r.thr = b ? pq : (pq << 9);
    return r;
  }
  if (!underflow) return r;
  // q = |w| / 2^e_base = (1 + p) 2^-dist, dist >= 1
  const int dist = e_base - e;
  if (b == 0) {
    const uint64_t mant = ((uint64_t)(1u << 23) + pq) << 9;          // (1 + p) 2^32
    const uint32_t thr = dist < 42 ? (uint32_t)(mant >> dist) : 0u;   // floor(q 2^32)
    if (thr) { r.live = 1; r.thr = thr; }
    return r;
  }
  const uint64_t mant = ((uint64_t)1 << b) + pq;                      // (1 + p_q) 2^b
  const uint64_t q = dist < 40 ? (mant + ((uint64_t)1 << (dist - 1))) >> dist : 0;   // round half up to b bits
  if (q == ((uint64_t)1 << b)) { r.live = 1; r.base = 1; r.sh = 0; r.thr = 0; }      // rounds to 2^e_base exactly
  else if (q) { r.live = 1; r.thr = (uint32_t)q; }
  return r;
}

}  // namespace

extern "C" {

// ---- building blocks exposed for the pins ---------------------------------

void psbo_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  philox4x32_10(ctr, key, out);
}

// Eq. 5-7.  Returns the class; *p_num is p * 2^23.
int psbo_decode(float w, int* s, int* e, uint32_t* p_num) {
  Decoded d = decode(w);
  *s = d.s; *e = d.e; *p_num = d.m;
  return d.cls;
}

int psbo_draw_bit(uint64_t seed, uint32_t layer, uint64_t index, uint32_t j, uint32_t p_num) {
  return draw_bit(seed, layer, index, j, p_num);
}

// Exponent window of one layer.  w is [O][D] (D = weights per output channel).
// norm = 0: one group per layer; norm = 1: one group per output channel.
// e_base[o] = e_max(group of o) - (2^exp_bits - 1); 0 for a group without any
// normal weight.  Returns 0, or -1 if a weight is Inf/NaN.
int psbo_window(const float* w, uint32_t O, uint64_t D, uint32_t exp_bits, uint32_t norm,
                int32_t* e_base) {
  const int span = (1 << exp_bits) - 1;
  bool any_layer = false;
  int emax_layer = 0;
  for (uint32_t o = 0; o < O; ++o) {
    bool any = false;
    int emax = 0;
    for (uint64_t i = 0; i < D; ++i) {
      Decoded d = decode(w[o * D + i]);
      if (d.cls == CLASS_NONFINITE) return -1;
      if (d.cls == CLASS_ZERO) continue;
      if (!any || d.e > emax) { emax = d.e; any = true; }
    }
    if (norm == 1) e_base[o] = any ? emax - span : 0;
    if (any && (!any_layer || emax > emax_layer)) { emax_layer = emax; any_layer = true; }
  }
  if (norm == 0)
    for (uint32_t o = 0; o < O; ++o) e_base[o] = any_layer ? emax_layer - span : 0;
  return 0;
}

// The same with b-bit probabilities: the window is taken over the exponents after quantisation.
int psbo_window_q(const float* w, uint32_t O, uint64_t D, uint32_t exp_bits, uint32_t norm, uint32_t prob_bits,
                  int32_t* e_base) {
  const int span = (1 << exp_bits) - 1;
  bool any_layer = false;
  int emax_layer = 0;
  for (uint32_t o = 0; o < O; ++o) {
    bool any = false;
    int emax = 0;
    for (uint64_t i = 0; i < D; ++i) {
      Decoded d = decode(w[o * D + i]);
      if (d.cls == CLASS_NONFINITE) return -1;
      if (d.cls == CLASS_ZERO) continue;
      int e;
      uint32_t pq;
      quantise(d, prob_bits, &e, &pq);
      if (!any || e > emax) { emax = e; any = true; }
    }
    if (norm == 1) e_base[o] = any ? emax - span : 0;
    if (any && (!any_layer || emax > emax_layer)) { emax_layer = emax; any_layer = true; }
  }
  if (norm == 0)
    for (uint32_t o = 0; o < O; ++o) e_base[o] = any_layer ? emax_layer - span : 0;
  return 0;
}

int psbo_quantise(float w, uint32_t prob_bits, int* e, uint32_t* pq) {
  Decoded d = decode(w);
  if (d.cls == CLASS_NORMAL) quantise(d, prob_bits, e, pq);
  return d.cls;
}

// What a weight becomes under a window with base exponent e_base: out = (live, base, sh, thr), see
// psbo_sample_level_ex.  Exposed for the pins.
void psbo_classify(float w, int32_t e_base, uint32_t prob_bits, uint32_t underflow, uint32_t* out) {
  const Sampled sm = classify(decode(w), e_base, prob_bits, underflow);
  out[0] = (uint32_t)sm.live; out[1] = sm.base; out[2] = (uint32_t)sm.sh; out[3] = sm.thr;
}

int psbo_draw_bit_packed(uint64_t seed, uint32_t layer, uint64_t index, uint32_t j, uint32_t thr, uint32_t prob_bits) {
  return draw_bit_packed(seed, layer, index, j, thr, prob_bits);
}

// Integer weights of one level with the options of Sec. 3.1 / 4.4:
//   opts[0] exp_bits, [1] norm, [2] underflow (0 flush below the window, 1 Bernoulli gate at its floor),
//   [3] prob_bits (0 = the full 23 bits, else 1..8), [4] deterministic (needs prob_bits > 0).
// W_k[i] = s (base k + c_k) 2^sh; inside the window base = 1, sh = e - e_base (Eq. 8 scaled by k / 2^e_base);
// below it (underflow = 1) base = 0, sh = 0, so that W_k 2^e_base / k = s 2^e_base c_k / k with
// c_k ~ Binomial(k, |w| / 2^e_base).  class_out (optional): 0 nothing, 1 window, 2 gate.
int psbo_sample_level_ex(const float* w, uint32_t O, uint64_t D, uint64_t seed, uint32_t layer,
                         const uint32_t* opts, uint32_t log2k, const uint32_t* counts_in, int64_t* W_out,
                         int32_t* e_base, uint32_t* counts_out, uint8_t* class_out) {
  const uint32_t exp_bits = opts[0], norm = opts[1], underflow = opts[2], b = opts[3], deterministic = opts[4];
  if (b > 8 || (deterministic && b == 0)) return -3;
  if (psbo_window_q(w, O, D, exp_bits, norm, b, e_base) != 0) return -1;
  const uint32_t k = 1u << log2k;
  for (uint32_t o = 0; o < O; ++o) {
    for (uint64_t pos = 0; pos < D; ++pos) {
      const uint64_t i = (uint64_t)o * D + pos;
      const Decoded d = decode(w[i]);
      const Sampled sm = classify(d, e_base[o], b, underflow);
      uint32_t c = 0;
      if (class_out) class_out[i] = sm.live ? (sm.base ? 1 : 2) : 0;
      if (!sm.live) {
        W_out[i] = 0;
        if (counts_out) counts_out[i] = 0;
        continue;
      }
      if (counts_in) {
        c = counts_in[i];
      } else if (deterministic) {
        c = (sm.thr * k + (1u << (b - 1))) >> b;            // the upper shift in round(p_q k) of k cases
      } else {
        for (uint32_t j = 0; j < k; ++j)
          c += b ? (uint32_t)draw_bit_packed(seed, layer, i, j, sm.thr, b)
                 : (uint32_t)draw_bit_thr(seed, layer, i, j, sm.thr);
      }
      const int64_t mag = (int64_t)(sm.base * k + c) * ipow2(sm.sh);
      W_out[i] = d.s ? -mag : mag;
      if (counts_out) counts_out[i] = c;
    }
  }
  return 0;
}

// Integer weights of one level k = 2^log2k (Eq. 8 scaled by k / 2^e_base):
//   W_k[i] = (+/-) (k + c_k) * 2^(e - e_base),  c_k = number of upper draws among
//   draws 0..k-1, so that W_k * 2^e_base / k = s * 2^e * (1 + c_k / k).
// w is [O][D] in canonical order (D = (C/groups)*KH*KW, index i = o*D + position);
// counts_in, if not NULL, replaces the Philox draws (brute-force pins inject bits).
// counts_out, if not NULL, receives c_k per weight.
int psbo_sample_level(const float* w, uint32_t O, uint64_t D, uint64_t seed, uint32_t layer,
                      uint32_t exp_bits, uint32_t norm, uint32_t log2k,
                      const uint32_t* counts_in, int64_t* W_out, int32_t* e_base,
                      uint32_t* counts_out) {
  if (psbo_window(w, O, D, exp_bits, norm, e_base) != 0) return -1;
  const uint32_t k = 1u << log2k;
  for (uint32_t o = 0; o < O; ++o) {
    for (uint64_t pos = 0; pos < D; ++pos) {
      const uint64_t i = (uint64_t)o * D + pos;
      Decoded d = decode(w[i]);
      uint32_t c = 0;
      if (d.cls == CLASS_ZERO || d.e < e_base[o]) {
        W_out[i] = 0;
        if (counts_out) counts_out[i] = 0;
        continue;
      }
      if (counts_in) {
        c = counts_in[i];
      } else {
        for (uint32_t j = 0; j < k; ++j) c += (uint32_t)draw_bit(seed, layer, i, j, d.m);
      }
      int64_t mag = (int64_t)(k + c) * ipow2(d.e - e_base[o]);
      W_out[i] = d.s ? -mag : mag;
      if (counts_out) counts_out[i] = c;
    }
  }
  return 0;
}

// ---- the contraction (Eq. 1 with every product replaced by Eq. 9) ---------

// Tensor geometry shared by the functions below.  layout: 0 = NCHW, 1 = NHWC.
// x_dtype: 0 = unsigned 8-bit, 1 = signed 8-bit.
struct psbo_conv_geom {
  uint32_t layout, x_dtype;
  uint32_t N, C, H, W;          // input
  uint32_t O, KH, KW, groups;   // filter [O][C/groups][KH][KW]
  uint32_t stride, pad;
  uint32_t OH, OW;              // output spatial size
};

static inline int64_t load_x(const void* x, const psbo_conv_geom& g, uint32_t n, uint32_t c,
                             uint32_t h, uint32_t w) {
  uint64_t idx = (g.layout == 0)
                     ? (((uint64_t)n * g.C + c) * g.H + h) * g.W + w
                     : (((uint64_t)n * g.H + h) * g.W + w) * g.C + c;
  return g.x_dtype == 0 ? (int64_t)((const uint8_t*)x)[idx] : (int64_t)((const int8_t*)x)[idx];
}

static inline uint64_t out_index(const psbo_conv_geom& g, uint32_t n, uint32_t o, uint32_t oy,
                                 uint32_t ox) {
  return (g.layout == 0) ? (((uint64_t)n * g.O + o) * g.OH + oy) * g.OW + ox
                         : (((uint64_t)n * g.OH + oy) * g.OW + ox) * g.O + o;
}

// One accumulator: sum over (ci, kh, kw) of x * W_k, with k chosen by the output
// location.  W_levels[l] is the level-l integer filter (NULL if not sampled).
static int64_t acc_one(const void* x, const psbo_conv_geom& g, const int64_t* const* W_levels,
                       uint32_t level, uint32_t n, uint32_t o, uint32_t oy, uint32_t ox) {
  const uint32_t Cg = g.C / g.groups;
  const uint32_t Og = g.O / g.groups;
  const uint32_t grp = o / Og;
  const int64_t* Wk = W_levels[level];
  int64_t acc = 0;
  for (uint32_t ci = 0; ci < Cg; ++ci)
    for (uint32_t kh = 0; kh < g.KH; ++kh)
      for (uint32_t kw = 0; kw < g.KW; ++kw) {
        int64_t iy = (int64_t)oy * g.stride + kh - g.pad;
        int64_t ix = (int64_t)ox * g.stride + kw - g.pad;
        if (iy < 0 || iy >= (int64_t)g.H || ix < 0 || ix >= (int64_t)g.W) continue;
        int64_t xv = load_x(x, g, n, grp * Cg + ci, (uint32_t)iy, (uint32_t)ix);
        int64_t wv = Wk[(((uint64_t)o * Cg + ci) * g.KH + kh) * g.KW + kw];
        acc += xv * wv;
      }
  return acc;
}

// Level (log2 k) used by output location (n, oy, ox): from the map if given.
static inline uint32_t level_at(const uint8_t* kmap, uint32_t uniform_log2k,
                                const psbo_conv_geom& g, uint32_t n, uint32_t oy, uint32_t ox) {
  return kmap ? kmap[((uint64_t)n * g.OH + oy) * g.OW + ox] : uniform_log2k;
}

// All accumulators of a layer, written in the layout of g.  Returns -2 if a
// location asks for a level that was not supplied.
int psbo_conv_acc(const void* x, const psbo_conv_geom* gp, const int64_t* const* W_levels,
                  const uint8_t* kmap, uint32_t uniform_log2k, int64_t* acc_out) {
  const psbo_conv_geom& g = *gp;
  for (uint32_t n = 0; n < g.N; ++n)
    for (uint32_t oy = 0; oy < g.OH; ++oy)
      for (uint32_t ox = 0; ox < g.OW; ++ox) {
        uint32_t level = level_at(kmap, uniform_log2k, g, n, oy, ox);
        if (level > 6 || !W_levels[level]) return -2;
        for (uint32_t o = 0; o < g.O; ++o)
          acc_out[out_index(g, n, o, oy, ox)] = acc_one(x, g, W_levels, level, n, o, oy, ox);
      }
  return 0;
}

// Accumulators at chosen output coordinates only: pts is [n_pts][4] = (n, o, oy, ox).
int psbo_conv_acc_points(const void* x, const psbo_conv_geom* gp, const int64_t* const* W_levels,
                         const uint8_t* kmap, uint32_t uniform_log2k, const uint32_t* pts,
                         uint64_t n_pts, int64_t* acc_out) {
  const psbo_conv_geom& g = *gp;
  for (uint64_t t = 0; t < n_pts; ++t) {
    uint32_t n = pts[4 * t], o = pts[4 * t + 1], oy = pts[4 * t + 2], ox = pts[4 * t + 3];
    uint32_t level = level_at(kmap, uniform_log2k, g, n, oy, ox);
    if (level > 6 || !W_levels[level]) return -2;
    acc_out[t] = acc_one(x, g, W_levels, level, n, o, oy, ox);
  }
  return 0;
}

// ---- dequantise, bias, shortcut, ReLU, re-quantise --------------------------

// One output value.  The integer accumulator stands for acc * 2^e_base / k in
// units of the input step; scale[o] carries that step and any folded
// batch-norm factor (Sec. 3: bn(y) = a*y + b folded into the layer).
//   a  = (float) acc                       round to nearest even
//   sc = scale * 2^(e_base - log2k)        exact (power of two)
//   y  = fma(a, sc, bias)
//   y  = fma((float) res_q, res_scale, y)  if a shortcut is added
//   y  = max(y, 0)                         if relu (Eq. 1)
//   q  = clamp(round_half_even(y * inv_step), qmin, qmax)
static inline float dequant_one(int64_t acc, float scale, int32_t e_base, uint32_t log2k,
                                float bias, int has_res, int32_t res_q, float res_scale,
                                int relu) {
  float a = (float)acc;
  float sc = std::ldexp(scale, e_base - (int32_t)log2k);
  float y = std::fmaf(a, sc, bias);
  if (has_res) y = std::fmaf((float)res_q, res_scale, y);
  if (relu) y = std::fmax(y, 0.0f);
  return y;
}

static inline int32_t requant_one(float y, float inv_step, int32_t qmin, int32_t qmax) {
  float t = y * inv_step;
  float r = std::nearbyintf(t);  // default rounding mode: ties to even
  if (r < (float)qmin) r = (float)qmin;
  if (r > (float)qmax) r = (float)qmax;
  return (int32_t)r;
}

float psbo_dequant_one(int64_t acc, float scale, int32_t e_base, uint32_t log2k, float bias,
                       int has_res, int32_t res_q, float res_scale, int relu) {
  return dequant_one(acc, scale, e_base, log2k, bias, has_res, res_q, res_scale, relu);
}

int32_t psbo_requant_one(float y, float inv_step, int32_t qmin, int32_t qmax) {
  return requant_one(y, inv_step, qmin, qmax);
}

struct psbo_epilogue {
  const float* scale;      // [O]
  const float* bias;       // [O]
  const int32_t* e_base;   // [O]
  const void* residual;    // same shape/layout as the output, or NULL
  uint32_t residual_dtype; // 0 = u8, 1 = s8
  float residual_scale;
  uint32_t relu;
  float inv_step;
  int32_t qmin, qmax;
};

// Epilogue over a whole output tensor laid out as g says.  y_out (float) and
// q_out (int32, one per element) may each be NULL.
void psbo_epilogue_apply(const int64_t* acc, const psbo_conv_geom* gp, const psbo_epilogue* ep,
                         const uint8_t* kmap, uint32_t uniform_log2k, float* y_out,
                         int32_t* q_out) {
  const psbo_conv_geom& g = *gp;
  for (uint32_t n = 0; n < g.N; ++n)
    for (uint32_t oy = 0; oy < g.OH; ++oy)
      for (uint32_t ox = 0; ox < g.OW; ++ox) {
        uint32_t level = level_at(kmap, uniform_log2k, g, n, oy, ox);
        for (uint32_t o = 0; o < g.O; ++o) {
          uint64_t idx = out_index(g, n, o, oy, ox);
          int32_t rq = 0;
          if (ep->residual)
            rq = ep->residual_dtype == 0 ? (int32_t)((const uint8_t*)ep->residual)[idx]
                                         : (int32_t)((const int8_t*)ep->residual)[idx];
          float y = dequant_one(acc[idx], ep->scale[o], ep->e_base[o], level, ep->bias[o],
                                ep->residual != nullptr, rq, ep->residual_scale, (int)ep->relu);
          if (y_out) y_out[idx] = y;
          if (q_out) q_out[idx] = requant_one(y, ep->inv_step, ep->qmin, ep->qmax);
        }
      }
}

// ---- glue between layers (supplement, "ReLU, Batch-Norm, and Pooling") ------

// Max-pooling on unsigned 8-bit activations: comparators only.  Padded positions
// never win (they are skipped).  layout as above.
void psbo_maxpool_u8(const uint8_t* x, uint32_t layout, uint32_t N, uint32_t C, uint32_t H,
                     uint32_t W, uint32_t ksize, uint32_t stride, uint32_t pad, uint8_t* out) {
  const uint32_t OH = (H + 2 * pad - ksize) / stride + 1;
  const uint32_t OW = (W + 2 * pad - ksize) / stride + 1;
  for (uint32_t n = 0; n < N; ++n)
    for (uint32_t c = 0; c < C; ++c)
      for (uint32_t oy = 0; oy < OH; ++oy)
        for (uint32_t ox = 0; ox < OW; ++ox) {
          int best = 0;
          for (uint32_t kh = 0; kh < ksize; ++kh)
            for (uint32_t kw = 0; kw < ksize; ++kw) {
              int64_t iy = (int64_t)oy * stride + kh - pad, ix = (int64_t)ox * stride + kw - pad;
              if (iy < 0 || iy >= (int64_t)H || ix < 0 || ix >= (int64_t)W) continue;
              uint64_t idx = layout == 0 ? (((uint64_t)n * C + c) * H + iy) * W + ix
                                         : (((uint64_t)n * H + iy) * W + ix) * C + c;
              if ((int)x[idx] > best) best = x[idx];
            }
          uint64_t od = layout == 0 ? (((uint64_t)n * C + c) * OH + oy) * OW + ox
                                    : (((uint64_t)n * OH + oy) * OW + ox) * C + c;
          out[od] = (uint8_t)best;
        }
}

// Global average pooling: integer sum over H*W, then one re-quantisation with the
// factor in_step / (H*W) * inv_step_out folded into pool_mul by the caller.
void psbo_global_avgpool_u8(const uint8_t* x, uint32_t layout, uint32_t N, uint32_t C, uint32_t H,
                            uint32_t W, float pool_mul, int32_t qmin, int32_t qmax,
                            uint8_t* out /* [N][C] */) {
  for (uint32_t n = 0; n < N; ++n)
    for (uint32_t c = 0; c < C; ++c) {
      int32_t sum = 0;
      for (uint32_t h = 0; h < H; ++h)
        for (uint32_t w = 0; w < W; ++w) {
          uint64_t idx = layout == 0 ? (((uint64_t)n * C + c) * H + h) * W + w
                                     : (((uint64_t)n * H + h) * W + w) * C + c;
          sum += x[idx];
        }
      out[(uint64_t)n * C + c] = (uint8_t)requant_one((float)sum, pool_mul, qmin, qmax);
    }
}

}  // extern "C"
