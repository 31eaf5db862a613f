// Weight sampler: turns an fp32 filter into exact integer filters, one per
// requested draw count k (paper Eq. 4-8).  Per weight:
//   decode (s, e, p) from the IEEE-754 fields          Eq. 5-7
//   window the exponent against the group's maximum    (4-bit exponents, Sec. 4.4)
//   draw k Bernoulli(p) bits from Philox4x32-10         the comparator of the
//                                                       stochastic multiplier
//   count the upper draws among the first k, every k    Eq. 8 (binomial count)
//   emit W_k = s (k + c_k) 2^(e - e_base) as int32 and as signed 7-bit digit
//   planes in the layout the tensor path loads with TMA.
// The random bits never leave registers.
#include <new>

#include "psb_common.cuh"

#include <algorithm>

namespace psb {

namespace {

constexpr int kThreads = 256;
constexpr int kStage = 2048;  // weights staged in shared memory per block
constexpr int kEmaxRows = kThreads / 32;   // output channels per block of the exponent pass (norm == 1, short rows)
constexpr int kEmaxLongRow = 1024;         // rows longer than this get a block each
constexpr int kRowSumRows = 256;   // filter rows per block for which the sampler keeps sums of |W_k|

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and
// xors; the key advances by the two Weyl constants after every round.  The ten round keys
// depend on the seed only: the host computes them once per launch (PhiloxKeys) and hands them to the kernel as a
// parameter, so every round reads its key straight from the constant bank and no register holds one.
struct PhiloxKeys {
  uint32_t k0[10], k1[10];
  __host__ __device__ __forceinline__ PhiloxKeys(uint32_t seed_lo, uint32_t seed_hi) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
      k0[r] = seed_lo + (uint32_t)r * 0x9E3779B9u;
      k1[r] = seed_hi + (uint32_t)r * 0xBB67AE85u;
    }
  }
};

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              const PhiloxKeys& key, uint32_t (&out)[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    // one widening multiply gives both halves
    const unsigned long long p0 = (unsigned long long)M0 * c0, p1 = (unsigned long long)M1 * c2;
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    const uint32_t n0 = hi1 ^ c1 ^ key.k0[r];
    const uint32_t n2 = hi0 ^ c3 ^ key.k1[r];
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t (&out)[4]) {
  const PhiloxKeys key(k0, k1);
  philox4x32_10(c0, c1, c2, c3, key, out);
}

// Counts with a B-bit comparator (Sec. 4.4; supplement, "Stochastic multiplier"): draw j is bit field
// (j mod n) of word ((j / n) mod 4) of Philox call j / (4 n), n = 32 / B; cnt[l] = ones among the first 2^l
// draws.  Every index is a compile-time constant here, so the loops unroll into one extract / compare / add
// per draw.
template <int B>
__device__ __forceinline__ void packed_counts(uint32_t thr, uint32_t max_level, uint32_t layer_id, uint32_t i_lo,
                                              uint32_t i_hi, const PhiloxKeys& keys, uint32_t (&cnt)[kMaxLevels]) {
  constexpr int n = 32 / B, per_call = 4 * n, calls = (64 + per_call - 1) / per_call;
  const uint32_t kmax = 1u << max_level;
  uint32_t c = 0;
#pragma unroll
  for (int q = 0; q < calls; ++q) {
    if ((uint32_t)(q * per_call) < kmax) {
      uint32_t rnd[4];
      philox4x32_10((uint32_t)q, layer_id, i_lo, i_hi, keys, rnd);
#pragma unroll
      for (int wd = 0; wd < 4; ++wd) {
#pragma unroll
        for (int f = 0; f < n; ++f) {
          constexpr uint32_t fmask = (1u << B) - 1u;
          const int j = q * per_call + wd * n + f;
          if (j < 64) {
            c += ((rnd[wd] >> (f * B)) & fmask) < thr ? 1u : 0u;
            if (((j + 1) & j) == 0) {           // j + 1 is a power of two: a level is complete
              const int l = j + 1 == 1 ? 0 : j + 1 == 2 ? 1 : j + 1 == 4 ? 2 : j + 1 == 8 ? 3 : j + 1 == 16 ? 4 : j + 1 == 32 ? 5 : 6;
              cnt[l] = c;
            }
          }
        }
      }
    }
  }
}

// The same for any width 1..8, indices at run time.
__device__ __forceinline__ void packed_counts_any(uint32_t pbits, uint32_t thr, uint32_t max_level, uint32_t layer_id,
                                               uint32_t i_lo, uint32_t i_hi, const PhiloxKeys& keys,
                                               uint32_t (&cnt)[kMaxLevels]) {
  const uint32_t n = 32u / pbits, per_call = 4u * n, fmask = (1u << pbits) - 1u, kmax = 1u << max_level;
  unsigned long long drawn = 0ull;      // bit j = draw j
  for (uint32_t q = 0; q * per_call < kmax && q * per_call < 64u; ++q) {
    uint32_t rnd[4];
    philox4x32_10(q, layer_id, i_lo, i_hi, keys, rnd);
#pragma unroll
    for (int wd = 0; wd < 4; ++wd) {
      uint32_t word = rnd[wd];
      unsigned long long bits = 0ull;
      for (uint32_t f = 0; f < n; ++f, word >>= pbits) bits |= (unsigned long long)((word & fmask) < thr ? 1u : 0u) << f;
      const uint32_t j0 = q * per_call + (uint32_t)wd * n;
      if (j0 < 64u) drawn |= bits << j0;
    }
  }
#pragma unroll
  for (int l = 0; l < kMaxLevels; ++l)
    cnt[l] = (uint32_t)__popcll(l == 6 ? drawn : drawn & ((1ull << (1u << l)) - 1ull));
}

// Division of a small number (< 2^16) by a block-uniform divisor (< 2^16): q = umulhi(t, magic)
// with magic = floor((2^32 - 1) / d) + 1 is exact in that range.
__device__ __forceinline__ uint32_t small_div_magic(uint32_t d) { return 0xFFFFFFFFu / d + 1u; }
__device__ __forceinline__ uint32_t small_div(uint32_t t, uint32_t magic) { return magic ? __umulhi(t, magic) : t; }   // magic wraps to 0 for d = 1

// Largest biased exponent of the finite weights of each exponent group; flags Inf/NaN (which
// contribute nothing: the finite weights of the group keep the window they would have without it).
// norm == 1: one warp (short rows) or one block per output channel.  norm == 0: grid-stride over the layer.
// Biased exponent of a weight after its probability has been rounded to `pbits` bits (Sec. 4.4): a
// probability that rounds to 1 is the next power of two.  pbits == 0: the exponent as it is.
__device__ __forceinline__ uint32_t quantised_exponent(uint32_t u, uint32_t pbits) {
  const uint32_t E = (u >> 23) & 0xFFu;
  if (pbits == 0u || E == 0u || E >= 254u) return E;
  const uint32_t pq = ((u & 0x7FFFFFu) + (1u << (22u - pbits))) >> (23u - pbits);
  return E + (pq >> pbits);
}

__device__ __forceinline__ void emax_block(const float* __restrict__ w, uint32_t O, uint32_t d,
                                           uint32_t norm, uint32_t* __restrict__ e_max,
                                           uint32_t* __restrict__ err, uint32_t block, uint32_t blocks,
                                           uint32_t tag, uint32_t* __restrict__ rowsum, uint32_t pbits) {
  __shared__ uint32_t red[kThreads / 32];
  // the sampling pass that follows adds its row sums of |W_k| into these words: start them at zero
  if (rowsum)
    for (uint32_t i = block * blockDim.x + threadIdx.x; i < (uint32_t)kMaxLevels * O; i += blocks * blockDim.x)
      rowsum[i] = 0u;
  uint32_t best = 0;
  bool bad = false;
  if (norm) {
    // short rows: one warp per output channel, kEmaxRows channels per block; long rows: one block per
    // channel.  16-byte loads where the row allows, several in flight per lane.
    const bool per_warp = d <= (uint32_t)kEmaxLongRow;
    const uint32_t o = per_warp ? block * (uint32_t)kEmaxRows + (threadIdx.x >> 5) : block;
    const uint32_t lane = per_warp ? (threadIdx.x & 31u) : threadIdx.x, lanes = per_warp ? 32u : blockDim.x;
    if (o < O) {
      const float* row = w + (size_t)o * d;
      if ((((uintptr_t)row) & 15u) == 0u && (d & 3u) == 0u) {
#pragma unroll 4
        for (uint32_t i = lane * 4u; i < d; i += lanes * 4u) {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(row + i));
          const uint32_t u4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t E = quantised_exponent(u4[j], pbits);
            bad |= (E == 255u);
            best = max(best, E == 255u ? 0u : E);     // Inf/NaN is flagged and takes no part in the window
          }
        }
      } else {
#pragma unroll 4
        for (uint32_t i = lane; i < d; i += lanes) {
          const uint32_t E = quantised_exponent(__float_as_uint(__ldg(row + i)), pbits);
          bad |= (E == 255u);
          best = max(best, E == 255u ? 0u : E);
        }
      }
    }
    if (per_warp) {
      if (o >= O) return;                                   // warp-uniform; no block-wide barrier on this path
      if (__any_sync(0xFFFFFFFFu, bad) && lane == 0u) atomicOr(err, kDevErrNonFinite);
      best = __reduce_max_sync(0xFFFFFFFFu, best);
      // `tag` (a call number in the bits above the exponent) distinguishes this call's maxima from whatever
      // an earlier call left in the word
      if (lane == 0u) e_max[o] = tag | best;
      return;
    }
  } else {
    const size_t total = (size_t)O * d;
    if ((((uintptr_t)w) & 15u) == 0u && (total & 3u) == 0u) {
#pragma unroll 4
      for (size_t i = ((size_t)block * blockDim.x + threadIdx.x) * 4u; i < total; i += (size_t)blocks * blockDim.x * 4u) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(w + i));
        const uint32_t u4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t E = quantised_exponent(u4[j], pbits);
          bad |= (E == 255u);
          best = max(best, E == 255u ? 0u : E);
        }
      }
    } else {
      for (size_t i = (size_t)block * blockDim.x + threadIdx.x; i < total; i += (size_t)blocks * blockDim.x) {
        const uint32_t E = quantised_exponent(__float_as_uint(__ldg(w + i)), pbits);
        bad |= (E == 255u);
        best = max(best, E == 255u ? 0u : E);
      }
    }
  }
  if (__any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicOr(err, kDevErrNonFinite);
  best = __reduce_max_sync(0xFFFFFFFFu, best);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < kThreads / 32; ++i) best = max(best, red[i]);
    // `tag` (a call number in the bits above the exponent) makes the maxima of this call beat
    // whatever an earlier call left in the word, so the words need no clearing between calls
    if (norm) e_max[block] = tag | best;
    else if (best) atomicMax(&e_max[0], tag | best);
  }
}

__global__ void emax_kernel(const float* __restrict__ w, uint32_t O, uint32_t d, uint32_t norm,
                            uint32_t* __restrict__ e_max, uint32_t* __restrict__ err, uint32_t tag,
                            uint32_t* __restrict__ rowsum, uint32_t pbits) {
  pdl_prologue();
  emax_block(w, O, d, norm, e_max, err, blockIdx.x, gridDim.x, tag, rowsum, pbits);
}

// What one weight becomes at every level: W_k = s (base k + c_k) 2^sh with c_k = cnt[log2 k]; a weight that is
// not live becomes 0.  `u` is the weight's bit pattern, `index` its canonical index (the Philox counter),
// `ebase_biased` the biased exponent of the window's floor.
struct Drawn {
  uint32_t cnt[kMaxLevels];
  uint32_t base, sh;
  bool live;
};

__device__ __forceinline__ void draw_weight(uint32_t u, uint64_t index, int ebase_biased, uint32_t pbits,
                                            uint32_t underflow, uint32_t deterministic, uint32_t max_level,
                                            uint32_t layer_id, const PhiloxKeys& keys, Drawn& out) {
  const uint32_t E = (u >> 23) & 0xFFu;
  const uint32_t m = u & 0x7FFFFFu;
  uint32_t (&cnt)[kMaxLevels] = out.cnt;
#pragma unroll
  for (int l = 0; l < kMaxLevels; ++l) cnt[l] = 0u;
  // probability on the grid of 2^pbits points, a p of 1 carried into the exponent (Sec. 4.4)
  uint32_t Eq = E, pq = m;
  if (pbits) {
    pq = (m + (1u << (22u - pbits))) >> (23u - pbits);
    if (pq == (1u << pbits)) {
      if (E < 254u) { Eq = E + 1u; pq = 0u; } else pq = (1u << pbits) - 1u;
    }
  }
  // what the weight becomes: W_k = s (base k + c_k) 2^sh, c_k counting draws with Pr[1] = thr / 2^32 (or
  // thr / 2^pbits).  Inside the window base = 1 (Eq. 8); below it, if asked for, the Bernoulli gate at the
  // window's floor (Sec. 3.1): base = 0, sh = 0, thr = |w| / 2^e_base
  bool live = (E != 0u) && (E != 255u);
  uint32_t base = 1u, sh = 0u, thr = 0u;
  const int dist = ebase_biased - (int)Eq;
  if (dist <= 0) {
    sh = (uint32_t)(-dist);
    thr = pbits ? pq : pq << 9;
  } else if (underflow) {
    base = 0u;
    if (pbits == 0u) {
      thr = dist < 42 ? (uint32_t)((((unsigned long long)(0x800000u + pq)) << 9) >> dist) : 0u;
      live = live && thr != 0u;
    } else {
      const unsigned long long mant = (1ull << pbits) + pq;
      const unsigned long long qv = dist < 40 ? (mant + (1ull << (dist - 1))) >> dist : 0ull;
      if (qv == (1ull << pbits)) base = 1u;          // rounds to the window's floor itself
      else { thr = (uint32_t)qv; live = live && qv != 0ull; }
    }
  } else {
    live = false;
  }

  // c_k for every level k = 2^l: level l is complete after draw 2^l, i.e. levels 0..2 after the
  // first Philox call, level l >= 2 after call 2^(l-2)
  if (live && thr != 0u) {
    const uint32_t i_lo = (uint32_t)index, i_hi = (uint32_t)(index >> 32);
    uint32_t rnd[4];
    if (pbits == 0u) {
      const uint32_t T = thr;
      philox4x32_10(0u, layer_id, i_lo, i_hi, keys, rnd);
      cnt[0] = rnd[0] < T ? 1u : 0u;
      cnt[1] = cnt[0] + (rnd[1] < T ? 1u : 0u);
      uint32_t c = cnt[1] + (rnd[2] < T ? 1u : 0u) + (rnd[3] < T ? 1u : 0u);
      cnt[2] = c;
#pragma unroll
      for (int l = 3; l < kMaxLevels; ++l) {
        if ((uint32_t)l <= max_level) {
          for (uint32_t q = 1u << (l - 3); q < (1u << (l - 2)); ++q) {
            philox4x32_10(q, layer_id, i_lo, i_hi, keys, rnd);
            c += (rnd[0] < T ? 1u : 0u) + (rnd[1] < T ? 1u : 0u) + (rnd[2] < T ? 1u : 0u) + (rnd[3] < T ? 1u : 0u);
          }
          cnt[l] = c;
        }
      }
    } else if (deterministic) {
#pragma unroll
      for (int l = 0; l < kMaxLevels; ++l) cnt[l] = ((thr << l) + (1u << (pbits - 1u))) >> pbits;
    } else {
      // pbits-bit comparator, n = 32 / pbits draws per random word
      switch (pbits) {
        case 4: packed_counts<4>(thr, max_level, layer_id, i_lo, i_hi, keys, cnt); break;
        case 6: packed_counts<6>(thr, max_level, layer_id, i_lo, i_hi, keys, cnt); break;
        case 8: packed_counts<8>(thr, max_level, layer_id, i_lo, i_hi, keys, cnt); break;
        default: packed_counts_any(pbits, thr, max_level, layer_id, i_lo, i_hi, keys, cnt); break;
      }
    }
  }

  out.base = base;
  out.sh = sh;
  out.live = live;
}

struct SampleParams {
  const float* w;
  uint32_t O, Cg, KHKW, d;
  uint32_t rows_per_block, ch_per_block, ch_chunks;
  uint32_t norm, span, level_mask, max_level;
  uint32_t underflow, pbits, deterministic;   // options of psb_sample_cfg
  uint32_t seed_lo, seed_hi, layer_id;
  uint32_t cpad, kpad, has_planes;
  uint32_t bk, n_cb, n_kb;         // operand tiles of the tensor path: K block bytes, blocks per tap, blocks per row
  uint32_t packed_kw, run_pitch;   // packed K (packed_kw = kw, else 0): plane column = kh * run_pitch + kw * Cg + ci
  const uint32_t* e_max;
  uint32_t e_tag;                  // call number the words of e_max must carry (bits 8 and up)
  int32_t* e_base;
  uint32_t* rowsum;                // [kMaxLevels][O] row sums of |W_k| / 256 (see psb_weights), or null
  int32_t* wint[kMaxLevels];
  int8_t* planes[kMaxLevels];
  int planes_count[kMaxLevels];
};

// kVec: whether the instance contains the four-weights-per-thread loop at all (a launch whose items are all
// small carries only the one-weight loop: with the L2 cold, what a short kernel costs is mostly its code)
template <bool kVec>
__device__ __forceinline__ void sample_block(const SampleParams& p, uint32_t block, const PhiloxKeys& keys,
                                             float* stage) {
  // the parameters may sit in global memory (batched launch): read the scalars once
  const uint32_t norm = p.norm, span = p.span, level_mask = p.level_mask, max_level = p.max_level;
  const uint32_t underflow = p.underflow, pbits = p.pbits, deterministic = p.deterministic;
  const uint32_t layer_id = p.layer_id, KHKW = p.KHKW, Cg = p.Cg;
  const uint32_t packed_kw = p.packed_kw, run_pitch = p.run_pitch, has_planes = p.has_planes;
  const uint32_t bk = p.bk, n_cb = p.n_cb, n_kb = p.n_kb;
  const uint32_t bk_shift = 31u - (uint32_t)__clz((int)bk), bk_mask = bk - 1u;     // bk is a power of two (32, 64, 128)
  // Row sums of |W_k| (in units of 256, each weight rounded up) for the bound that lets the contraction
  // recombine its digit planes in 32 bits: gathered per block in shared memory, then added to the layer's words
  __shared__ uint32_t row_sum[kMaxLevels][kRowSumRows];
  uint32_t* const rowsum = p.rowsum;
  const bool track = rowsum != nullptr && p.rows_per_block <= (uint32_t)kRowSumRows;
  if (track)
    for (uint32_t i = threadIdx.x; i < (uint32_t)(kMaxLevels * kRowSumRows); i += blockDim.x)
      row_sum[i / kRowSumRows][i % kRowSumRows] = 0u;
  const uint32_t row_block = block / p.ch_chunks;
  const uint32_t chunk = block % p.ch_chunks;
  const uint32_t o0 = row_block * p.rows_per_block;
  const uint32_t c0 = chunk * p.ch_per_block;
  const uint32_t rows = min(p.rows_per_block, p.O - o0);
  const uint32_t cc = min(p.ch_per_block, p.Cg - c0);
  const uint32_t per_row = cc * p.KHKW;     // canonical elements of one row in this block
  const uint32_t count = rows * per_row;

  // The slice is one contiguous run of the weight tensor (whole rows, or a channel range of one row): stage it
  // with 16-byte loads where the run allows.
  {
    const float* src = p.w + (size_t)o0 * p.d + (size_t)c0 * p.KHKW;
    if ((((uintptr_t)src) & 15u) == 0u && (count & 3u) == 0u) {
#pragma unroll 2
      for (uint32_t t = threadIdx.x * 4u; t < count; t += blockDim.x * 4u)
        *reinterpret_cast<float4*>(stage + t) = __ldg(reinterpret_cast<const float4*>(src + t));
    } else {
#pragma unroll 4
      for (uint32_t t = threadIdx.x; t < count; t += blockDim.x) stage[t] = __ldg(src + t);
    }
  }
  __syncthreads();

  const uint32_t d = p.d, e_tag = p.e_tag;
  const uint32_t* const e_max = p.e_max;
  int32_t* const e_base_out = p.e_base;
  // count <= kStage and the divisors are block-uniform: divisions by multiply-high.  The slice is walked in
  // output order (row, tap, channel) so that stores coalesce.
  if (kVec && !packed_kw && has_planes && ((cc | Cg | c0) & 3u) == 0u && count >= 4u * blockDim.x) {
    // Items that give every thread at least four weights: four consecutive channels per thread, one 16-byte
    // store of the integer weights and one 4-byte store per digit plane and level.  Between the draws and the stores the four weights' counts travel as the bytes of
    // one word per level (c_k <= 64), and (sh, base, sign) as one byte per weight.
    const uint32_t cc4 = cc >> 2, per_row4 = per_row >> 2;
    const uint32_t per_row4_magic = small_div_magic(per_row4), cc4_magic = small_div_magic(cc4);
    for (uint32_t t = threadIdx.x; t < (count >> 2); t += blockDim.x) {
      const uint32_t r = small_div(t, per_row4_magic), rem = t - r * per_row4;
      const uint32_t tap = small_div(rem, cc4_magic), cl = (rem - tap * cc4) << 2;
      const uint32_t o = o0 + r, ci = c0 + cl;
      // a word written by an earlier call (other tag) means this call found no live weight in the group
      const uint32_t e_word = e_max[norm ? o : 0];
      const uint32_t Emax = (e_word >> 8) == e_tag ? (e_word & 0xFFu) : 0u;
      // biased exponents throughout: e - e_base = E - (Emax - span)
      const int ebase_biased = (int)Emax - (int)span;
      if (tap == 0 && ci == 0) e_base_out[o] = Emax ? ebase_biased - 127 : 0;
      uint32_t cntpk[kMaxLevels] = {0u, 0u, 0u, 0u, 0u, 0u, 0u};
      uint32_t meta = 0u;
#pragma unroll 1       // one copy of the drawing code: unrolled four times it no longer fits the instruction cache
      for (int j = 0; j < 4; ++j) {
        const uint32_t u = __float_as_uint(stage[r * per_row + (cl + (uint32_t)j) * KHKW + tap]);
        const uint64_t index = (uint64_t)o * d + (uint64_t)(ci + (uint32_t)j) * KHKW + tap;  // canonical
        Drawn dw;
        draw_weight(u, index, ebase_biased, pbits, underflow, deterministic, max_level, layer_id, keys, dw);
        if (dw.live) {
#pragma unroll
          for (int l = 0; l < kMaxLevels; ++l) cntpk[l] |= dw.cnt[l] << (8 * j);
          meta |= (dw.sh | (dw.base << 4) | ((u >> 31) << 5)) << (8 * j);
        }
      }
      const size_t wpos = ((size_t)o * KHKW + tap) * Cg + ci;
      const uint32_t kb = tap * n_cb + (ci >> bk_shift), kin = ci & bk_mask;
      const uint32_t jt = o / kTileN, on = o % kTileN;
#pragma unroll
      for (int l = 0; l < kMaxLevels; ++l) {
        if (!((level_mask >> l) & 1u)) continue;
        uint32_t mag[4];
        int wv[4];
        uint32_t part = 0u;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t m8 = meta >> (8 * j), c = (cntpk[l] >> (8 * j)) & 0xFFu;
          mag[j] = ((((m8 >> 4) & 1u) << l) + c) << (m8 & 15u);
          wv[j] = ((m8 >> 5) & 1u) ? -(int32_t)mag[j] : (int32_t)mag[j];
          part += (mag[j] + 255u) >> 8;
        }
        *reinterpret_cast<int4*>(p.wint[l] + wpos) = make_int4(wv[0], wv[1], wv[2], wv[3]);
        if (track) {
          // lanes of a warp mostly share a row: then one reduction and one shared-memory add per warp
          const uint32_t lanes = __activemask();
          const uint32_t r_first = __shfl_sync(lanes, r, (int)__ffs((int)lanes) - 1);
          if (__all_sync(lanes, r == r_first)) {
            const uint32_t sum = __reduce_add_sync(lanes, part);
            if ((threadIdx.x & 31u) == (uint32_t)__ffs((int)lanes) - 1u && sum) atomicAdd(&row_sum[l][r], sum);
          } else if (part) {
            atomicAdd(&row_sum[l][r], part);
          }
        }
        const int P = p.planes_count[l];
        int8_t* tile = p.planes[l] + (((size_t)jt * n_kb + kb) * (size_t)P << (6u + bk_shift));   // P * 64 * bk per tile
        // byte offset of (row, kin) in the swizzled tile (plane_offset), advanced by 64 rows per plane; the four
        // bytes share a 16-byte piece
        const uint32_t lin0 = (on << bk_shift) + kin, sw_mask = (bk >> 4) - 1u;
        for (int pl = 0; pl < P; ++pl) {
          uint32_t word = 0u;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int digit = (int)((mag[j] >> (kDigitBits * pl)) & 0x7Fu);
            word |= (uint32_t)((wv[j] < 0 ? -digit : digit) & 0xFF) << (8 * j);
          }
          const uint32_t lin = lin0 + ((uint32_t)pl << (6u + bk_shift));
          *reinterpret_cast<uint32_t*>(tile + (lin ^ (((lin >> 7) & sw_mask) << 4))) = word;
        }
      }
    }
  } else {
  const uint32_t per_row_magic = small_div_magic(per_row), cc_magic = small_div_magic(cc);
  for (uint32_t t = threadIdx.x; t < count; t += blockDim.x) {
    const uint32_t r = small_div(t, per_row_magic), rem = t - r * per_row;
    const uint32_t tap = small_div(rem, cc_magic), cl = rem - tap * cc;
    const uint32_t o = o0 + r, ci = c0 + cl;
    const uint32_t u = __float_as_uint(stage[r * per_row + cl * KHKW + tap]);
    const uint64_t index = (uint64_t)o * d + (uint64_t)ci * KHKW + tap;  // canonical
    // a word written by an earlier call (other tag) means this call found no live weight in the group
    const uint32_t e_word = e_max[norm ? o : 0];
    const uint32_t Emax = (e_word >> 8) == e_tag ? (e_word & 0xFFu) : 0u;
    // biased exponents throughout: e - e_base = E - (Emax - span)
    const int ebase_biased = (int)Emax - (int)span;
    if (tap == 0 && ci == 0) e_base_out[o] = Emax ? ebase_biased - 127 : 0;
    Drawn dw;
    draw_weight(u, index, ebase_biased, pbits, underflow, deterministic, max_level, layer_id, keys, dw);
    const bool live = dw.live, neg = (u >> 31) != 0u;
    const uint32_t base = dw.base, sh = dw.sh;
    const uint32_t (&cnt)[kMaxLevels] = dw.cnt;

    const size_t wpos = ((size_t)o * KHKW + tap) * Cg + ci;
    // K block and column inside it (bk is a power of two)
    uint32_t kb = tap * n_cb + (ci >> bk_shift), kin = ci & bk_mask;
    if (packed_kw) {
      const uint32_t kh = tap / packed_kw;
      const uint32_t kcol = kh * run_pitch + (tap - kh * packed_kw) * Cg + ci;
      kb = kcol >> bk_shift;
      kin = kcol & bk_mask;
    }
    const uint32_t jt = o / kTileN, on = o % kTileN;
#pragma unroll
    for (int l = 0; l < kMaxLevels; ++l) {
      if (!((level_mask >> l) & 1u)) continue;
      const uint32_t mag = live ? (((base << l) + cnt[l]) << sh) : 0u;
      p.wint[l][wpos] = neg ? -(int32_t)mag : (int32_t)mag;
      if (track) {
        // lanes of a warp mostly share a row: then one reduction and one shared-memory add per warp
        const uint32_t lanes = __activemask();
        const uint32_t r_first = __shfl_sync(lanes, r, (int)__ffs((int)lanes) - 1);
        const uint32_t part = (mag + 255u) >> 8;
        if (__all_sync(lanes, r == r_first)) {
          const uint32_t sum = __reduce_add_sync(lanes, part);
          if ((threadIdx.x & 31u) == (uint32_t)__ffs((int)lanes) - 1u && sum) atomicAdd(&row_sum[l][r], sum);
        } else if (part) {
          atomicAdd(&row_sum[l][r], part);
        }
      }
      if (has_planes) {
        const int P = p.planes_count[l];
        int8_t* tile = p.planes[l] + (((size_t)jt * n_kb + kb) * (size_t)P << (6u + bk_shift));   // P * 64 * bk per tile
        // byte offset of (row, kin) in the swizzled tile (plane_offset), advanced by 64 rows per plane
        const uint32_t lin0 = (on << bk_shift) + kin, sw_mask = (bk >> 4) - 1u;
        for (int pl = 0; pl < P; ++pl) {
          const int digit = (int)((mag >> (kDigitBits * pl)) & 0x7Fu);
          const uint32_t lin = lin0 + ((uint32_t)pl << (6u + bk_shift));
          tile[lin ^ (((lin >> 7) & sw_mask) << 4)] = (int8_t)(neg ? -digit : digit);
        }
      }
    }
  }
  }
  if (rowsum) {
    __syncthreads();
#pragma unroll
    for (int l = 0; l < kMaxLevels; ++l) {
      if (!((level_mask >> l) & 1u)) continue;
      for (uint32_t r = threadIdx.x; r < rows; r += blockDim.x) {
        // a block that could not keep sums (more rows than the table holds) leaves the bound unknown
        if (!track) atomicMax(&rowsum[(uint32_t)l * p.O + o0 + r], 0xFFFFFFFFu);
        else if (row_sum[l][r]) atomicAdd(&rowsum[(uint32_t)l * p.O + o0 + r], row_sum[l][r]);
      }
    }
  }
}

template <bool kVec>
__global__ void __launch_bounds__(kThreads) sample_kernel(const __grid_constant__ SampleParams p,
                                                          const __grid_constant__ PhiloxKeys keys) {
  pdl_prologue();
  __shared__ float stage[kStage];
  sample_block<kVec>(p, blockIdx.x, keys, stage);
}

// All layers of a network in two launches.  Entry i owns blocks [first, first + count) of each
// grid; its parameters sit in device memory (every thread of a block reads the same words).
struct BatchEntry {
  SampleParams p;
  uint32_t emax_first, emax_blocks, sample_first, sample_blocks;
};

__device__ __forceinline__ uint32_t find_entry(const BatchEntry* __restrict__ e, uint32_t n, uint32_t block,
                                               bool emax) {
  uint32_t lo = 0, hi = n - 1;
  while (lo < hi) {
    const uint32_t mid = (lo + hi + 1) >> 1;
    const uint32_t first = emax ? e[mid].emax_first : e[mid].sample_first;
    if (first <= block) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__global__ void __launch_bounds__(kThreads) emax_batch_kernel(const BatchEntry* __restrict__ entries, uint32_t n,
                                                              uint32_t* __restrict__ err) {
  pdl_prologue();
  const BatchEntry& e = entries[find_entry(entries, n, blockIdx.x, true)];
  emax_block(e.p.w, e.p.O, e.p.d, e.p.norm, const_cast<uint32_t*>(e.p.e_max), err,
             blockIdx.x - e.emax_first, e.emax_blocks, 0u, e.p.rowsum, e.p.pbits);
}

__global__ void __launch_bounds__(kThreads) sample_batch_kernel(const BatchEntry* __restrict__ entries, uint32_t n,
                                                                const __grid_constant__ PhiloxKeys keys) {
  pdl_prologue();
  __shared__ float stage[kStage];
  const BatchEntry& e = entries[find_entry(entries, n, blockIdx.x, false)];
  sample_block<true>(e.p, blockIdx.x - e.sample_first, keys, stage);
}

// 128 * (sum of each filter row): the constant that restores sum x*W from sum (x-128)*W when
// unsigned activations are fed to the signed MMA with an offset of 128.  One warp per row.
__global__ void corr128_kernel(const int32_t* wint, uint32_t O, uint32_t d,
                               long long* __restrict__ corr) {
  pdl_prologue();
  const uint32_t row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31u;
  if (row >= O) return;
  long long sum = 0;
  for (uint32_t i = lane; i < d; i += 32u) sum += wint[(size_t)row * d + i];
  for (int off = 16; off; off >>= 1) sum += __shfl_down_sync(0xFFFFFFFFu, sum, off);
  if (lane == 0) corr[row] = sum * 128;
}

// Canonical-order copy of one level for the test hook.
__global__ void export_kernel(const int32_t* __restrict__ wint, int32_t* __restrict__ out, uint32_t O,
                              uint32_t Cg, uint32_t KHKW) {
  pdl_prologue();
  size_t total = (size_t)O * Cg * KHKW;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (size_t)gridDim.x * blockDim.x) {
    uint32_t tap = (uint32_t)(i % KHKW);
    size_t t = i / KHKW;
    uint32_t ci = (uint32_t)(t % Cg);
    size_t o = t / Cg;
    out[i] = wint[(o * KHKW + tap) * Cg + ci];
  }
}

}  // namespace

namespace {

uint32_t emax_blocks_for(uint32_t O, uint32_t d, uint32_t norm) {
  if (norm) return d <= (uint32_t)kEmaxLongRow ? (O + (uint32_t)kEmaxRows - 1u) / (uint32_t)kEmaxRows : O;
  size_t total = (size_t)O * d;
  // sixteen weights per thread (four 16-byte loads in flight) once that still fills the machine, four otherwise
  uint32_t blocks = (uint32_t)((total + kThreads * 16 - 1) / (kThreads * 16));
  if (blocks < 296u) blocks = (uint32_t)std::min<size_t>(296u, (total + kThreads * 4 - 1) / (kThreads * 4));
  return blocks < 1 ? 1 : (blocks > 1184 ? 1184 : blocks);
}

// Parameters of one layer's sampling pass; returns the number of blocks it needs.
uint32_t fill_sample_params(const float* w_dev, const psb_weights* wt, uint32_t* e_max, SampleParams& p,
                            bool batched) {
  const psb_wshape& sh = wt->shape;
  const uint32_t O = sh.out_ch, Cg = sh.in_ch_per_group, KHKW = sh.kh * sh.kw, d = wt->d;
  p.w = w_dev;
  p.O = O; p.Cg = Cg; p.KHKW = KHKW; p.d = d;
  // weights per block: the whole staging buffer for large layers; a layer sampled by a launch of its own
  // gets less if it is small, so that it still spreads over a few hundred blocks (in a batched launch the
  // other layers' blocks fill the machine)
  const uint64_t total = (uint64_t)O * d;
  uint32_t budget = batched ? (uint32_t)kStage
                            : (uint32_t)std::min<uint64_t>((uint64_t)kStage, std::max<uint64_t>(256u, total / 296u));
  if (budget < KHKW) budget = KHKW;   // at least one channel (host validation keeps kh*kw <= kStage)
  if (d <= budget) {
    p.rows_per_block = std::min<uint32_t>(budget / d, (uint32_t)kRowSumRows);   // the rows a block keeps sums for
    p.ch_per_block = Cg;
    p.ch_chunks = 1;
  } else {
    p.rows_per_block = 1;
    p.ch_per_block = budget / KHKW;
    if (p.ch_per_block > 16u) p.ch_per_block &= ~15u;   // whole 16-byte pieces of the plane rows
    p.ch_chunks = (Cg + p.ch_per_block - 1) / p.ch_per_block;
  }
  p.norm = wt->cfg.norm;
  p.span = (1u << wt->cfg.exp_bits) - 1u;
  p.level_mask = wt->cfg.level_mask;
  p.underflow = wt->cfg.underflow;
  p.pbits = wt->cfg.prob_bits;
  p.deterministic = wt->cfg.deterministic;
  p.max_level = 0;
  for (uint32_t l = 0; l < (uint32_t)kMaxLevels; ++l)
    if ((p.level_mask >> l) & 1u) p.max_level = l;
  p.seed_lo = (uint32_t)wt->cfg.seed;
  p.seed_hi = (uint32_t)(wt->cfg.seed >> 32);
  p.layer_id = wt->cfg.layer_id;
  p.cpad = wt->cpad; p.kpad = wt->kpad; p.has_planes = wt->has_planes ? 1u : 0u;
  p.bk = wt->bk; p.n_cb = wt->n_cb; p.n_kb = wt->n_kb;
  p.packed_kw = wt->packed_k ? wt->shape.kw : 0u;
  p.run_pitch = wt->run_pitch;
  p.e_max = e_max;
  p.e_tag = 0;
  p.e_base = wt->e_base;
  p.rowsum = wt->rowsum256;
  for (int l = 0; l < kMaxLevels; ++l) {
    p.wint[l] = wt->level[l].wint;
    p.planes[l] = wt->level[l].planes;
    p.planes_count[l] = wt->level[l].planes_count;
  }
  const uint32_t row_blocks = (O + p.rows_per_block - 1) / p.rows_per_block;
  return row_blocks * p.ch_chunks;
}

}  // namespace

cudaError_t launch_corr128(const psb_weights* wt, uint32_t level, cudaStream_t s) {
  const uint32_t O = wt->shape.out_ch;
  launch_pdl(corr128_kernel, (O * 32 + kThreads - 1) / kThreads, kThreads, 0, s, (const int32_t*)wt->level[level].wint, O,
             wt->d, wt->level[level].corr128); note_launch();
  return cudaGetLastError();
}

cudaError_t launch_sampler(const float* w_dev, psb_weights* wt, uint32_t* err_dev, cudaStream_t s) {
  const uint32_t O = wt->shape.out_ch;
  // the exponent maxima carry the number of the call that wrote them; the words were cleared when
  // the handle was made and are cleared again only when the 24-bit call number wraps
  wt->e_calls = (wt->e_calls + 1u) & 0xFFFFFFu;
  if (wt->e_calls == 0u) {
    cudaError_t e = cudaMemsetAsync(wt->e_max, 0, sizeof(uint32_t) * O, s);
    if (e != cudaSuccess) return e;
    wt->e_calls = 1u;
  }
  launch_pdl(emax_kernel, emax_blocks_for(O, wt->d, wt->cfg.norm), kThreads, 0, s, w_dev, O, wt->d, wt->cfg.norm,
             wt->e_max, err_dev, wt->e_calls << 8, wt->rowsum256, wt->cfg.prob_bits); note_launch();
  SampleParams p;
  const uint32_t blocks = fill_sample_params(w_dev, wt, wt->e_max, p, false);
  p.e_tag = wt->e_calls;
  // items of fewer than four weights per thread never take the four-weights loop: launch the instance without it
  const uint64_t item_weights = (uint64_t)p.rows_per_block * std::min<uint64_t>(p.ch_per_block, p.Cg) * p.KHKW;
  if (item_weights >= 4u * (uint64_t)kThreads)
    launch_pdl(sample_kernel<true>, blocks, kThreads, 0, s, p, PhiloxKeys(p.seed_lo, p.seed_hi));
  else
    launch_pdl(sample_kernel<false>, blocks, kThreads, 0, s, p, PhiloxKeys(p.seed_lo, p.seed_hi));
  note_launch();
  return cudaGetLastError();
}

}  // namespace psb

// ---- batched sampling: every layer of a network in two launches ---------------------------
struct psb_sample_batch {
  uint32_t n = 0;
  psb::BatchEntry* entries_dev = nullptr;
  uint32_t* e_max_pool = nullptr;     // one word per output channel of every layer
  size_t e_max_words = 0;
  uint32_t emax_grid = 0, sample_grid = 0;
  int device = 0;
};

namespace psb {

psb_status sample_batch_create(psb_ctx* ctx, uint32_t n, const float* const* w_dev,
                               psb_weights* const* weights, psb_sample_batch** out) {
  psb_sample_batch* b = new (std::nothrow) psb_sample_batch();
  BatchEntry* host = new (std::nothrow) BatchEntry[n];
  if (!b || !host) { delete b; delete[] host; return PSB_ERR_ALLOC; }
  size_t words = 0;
  for (uint32_t i = 0; i < n; ++i) words += weights[i]->shape.out_ch;
  bool ok = cudaMalloc(&b->e_max_pool, sizeof(uint32_t) * words) == cudaSuccess &&
            cudaMalloc(&b->entries_dev, sizeof(BatchEntry) * n) == cudaSuccess;
  if (ok) {
    size_t off = 0;
    uint32_t eb = 0, sb = 0;
    for (uint32_t i = 0; i < n; ++i) {
      const psb_weights* wt = weights[i];
      BatchEntry& e = host[i];
      e.sample_blocks = fill_sample_params(w_dev[i], wt, b->e_max_pool + off, e.p, true);
      e.emax_blocks = emax_blocks_for(wt->shape.out_ch, wt->d, wt->cfg.norm);
      e.emax_first = eb;
      e.sample_first = sb;
      eb += e.emax_blocks;
      sb += e.sample_blocks;
      off += wt->shape.out_ch;
    }
    b->emax_grid = eb;
    b->sample_grid = sb;
    ok = cudaMemcpy(b->entries_dev, host, sizeof(BatchEntry) * n, cudaMemcpyHostToDevice) == cudaSuccess;
  }
  delete[] host;
  if (!ok) {
    cudaGetLastError();
    if (b->e_max_pool) cudaFree(b->e_max_pool);
    if (b->entries_dev) cudaFree(b->entries_dev);
    delete b;
    return PSB_ERR_ALLOC;
  }
  b->n = n;
  b->e_max_words = words;
  b->device = ctx->device;
  *out = b;
  return PSB_OK;
}

psb_status sample_batch_run(psb_ctx* ctx, psb_sample_batch* b, uint64_t seed, cudaStream_t s) {
  if (cudaMemsetAsync(b->e_max_pool, 0, sizeof(uint32_t) * b->e_max_words, s) != cudaSuccess)
    return PSB_ERR_CUDA;
  launch_pdl(emax_batch_kernel, b->emax_grid, kThreads, 0, s, (const BatchEntry*)b->entries_dev, b->n, ctx->err_dev);
  note_launch();
  launch_pdl(sample_batch_kernel, b->sample_grid, kThreads, 0, s, (const BatchEntry*)b->entries_dev, b->n,
             PhiloxKeys((uint32_t)seed, (uint32_t)(seed >> 32)));
  note_launch();
  return cudaGetLastError() == cudaSuccess ? PSB_OK : PSB_ERR_CUDA;
}

void sample_batch_free(psb_sample_batch* b) {
  if (b->e_max_pool) cudaFree(b->e_max_pool);
  if (b->entries_dev) cudaFree(b->entries_dev);
  delete b;
}

cudaError_t launch_export(const psb_weights* wt, uint32_t level, int32_t* wint_out,
                          int32_t* e_base_out, cudaStream_t s) {
  const psb_wshape& sh = wt->shape;
  if (wint_out) {
    size_t total = (size_t)sh.out_ch * wt->d;
    uint32_t blocks = (uint32_t)((total + 255) / 256);
    blocks = blocks > 4096 ? 4096 : (blocks < 1 ? 1 : blocks);
    export_kernel<<<blocks, 256, 0, s>>>(wt->level[level].wint, wint_out, sh.out_ch,
                                        sh.in_ch_per_group, sh.kh * sh.kw); note_launch();
  }
  if (e_base_out) {
    cudaError_t e = cudaMemcpyAsync(e_base_out, wt->e_base, sizeof(int32_t) * sh.out_ch,
                                    cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

}  // namespace psb

// ---------------------------------------------------------------------------
// Allocation-free sampling of one level (psb_sample_level_static in psb.h).
//
// Some hosts may not allocate device memory when they need fresh weights: a
// real-time loop that must not block on the allocator, code running while a CUDA
// graph is being captured elsewhere in the process, or a process whose memory
// budget was handed out at start-up.  For them the window reduction's scratch
// (one biased exponent per output channel, plus a device error word nobody reads)
// lives in this file-scope device array instead of a cudaMalloc'ed buffer.  Every
// GPU that loads the library holds these 16 KB + 256 B until the process exits.
namespace psb {
namespace {

constexpr uint32_t kStaticMaxOutCh = 4096;   // PSB_STATIC_MAX_OUT_CH in psb.h
static __device__ __align__(256) uint32_t g_static_scratch[kStaticMaxOutCh + 64];

constexpr int kMaxDevices = 64;
uint32_t* g_static_scratch_addr[kMaxDevices] = {};   // device address per device ordinal

// One thread per weight, canonical order in and out (both coalesce).  e_max is
// the device address of the static scratch, filled by emax_kernel just before.
__global__ void __launch_bounds__(kThreads)
sample_level_canonical_kernel(const float* __restrict__ w, uint32_t O, uint32_t d, uint32_t norm,
                              uint32_t span, uint32_t log2k, uint32_t seed_lo, uint32_t seed_hi,
                              uint32_t layer_id, const uint32_t* __restrict__ e_max,
                              int32_t* __restrict__ wint_out, int32_t* __restrict__ e_base_out) {
  pdl_prologue();
  const size_t total = (size_t)O * d;
  for (size_t index = (size_t)blockIdx.x * blockDim.x + threadIdx.x; index < total;
       index += (size_t)gridDim.x * blockDim.x) {
    const uint32_t o = (uint32_t)(index / d);
    const uint32_t u = __float_as_uint(w[index]);
    const uint32_t E = (u >> 23) & 0xFFu, m = u & 0x7FFFFFu;
    const uint32_t Emax = e_max[norm ? o : 0];
    const int ebase_biased = (int)Emax - (int)span;
    if (index % d == 0 && e_base_out) e_base_out[o] = Emax ? ebase_biased - 127 : 0;
    if (!wint_out) continue;
    const bool live = (E != 0u) && (E != 255u) && ((int)E >= ebase_biased);
    uint32_t c = 0;
    if (live && m != 0u) {
      const uint32_t T = m << 9, k = 1u << log2k;
      for (uint32_t q = 0; q * 4u < k; ++q) {
        uint32_t rnd[4];
        philox4x32_10(q, layer_id, (uint32_t)index, (uint32_t)(index >> 32), seed_lo, seed_hi, rnd);
#pragma unroll
        for (int v = 0; v < 4; ++v)
          if (q * 4u + v < k) c += (rnd[v] < T) ? 1u : 0u;
      }
    }
    const uint32_t mag = live ? (((1u << log2k) + c) << (uint32_t)((int)E - ebase_biased)) : 0u;
    wint_out[index] = (u >> 31) ? -(int32_t)mag : (int32_t)mag;
  }
}

}  // namespace
}  // namespace psb

extern "C" psb_status psb_sample_level_static(const float* w_dev, const psb_wshape* shape,
                                              const psb_sample_cfg* cfg, uint32_t log2k,
                                              int32_t* wint_out_dev, int32_t* e_base_out_dev,
                                              void* stream) {
  using namespace psb;
  if (!w_dev || !shape || !cfg || (!wint_out_dev && !e_base_out_dev)) return PSB_ERR_INVALID_ARG;
  if (((uintptr_t)w_dev | (uintptr_t)wint_out_dev | (uintptr_t)e_base_out_dev) & 3u)
    return PSB_ERR_INVALID_ARG;
  if (!shape->out_ch || !shape->in_ch_per_group || !shape->kh || !shape->kw || !shape->groups)
    return PSB_ERR_INVALID_ARG;
  if (log2k >= (uint32_t)kMaxLevels) return PSB_ERR_BAD_K;
  const uint32_t exp_bits = cfg->exp_bits ? cfg->exp_bits : 4u;
  if (exp_bits > 4 || cfg->norm > 1) return PSB_ERR_INVALID_ARG;
  if (cfg->underflow || cfg->prob_bits || cfg->deterministic) return PSB_ERR_UNSUPPORTED;
  // the static scratch holds one word per output channel: larger filters are refused
  if (shape->out_ch > kStaticMaxOutCh) return PSB_ERR_UNSUPPORTED;
  const uint64_t d64 = (uint64_t)shape->in_ch_per_group * shape->kh * shape->kw;
  if (d64 > (1u << 24) || d64 * shape->out_ch > (1ull << 31)) return PSB_ERR_UNSUPPORTED;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PSB_ERR_CUDA;
  if (!g_static_scratch_addr[dev]) {
    // first call on this device: the symbol's name is only a host-side stand-in, so ask the
    // runtime for the array's address on the current device
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || !addr) {
      cudaGetLastError();
      return PSB_ERR_CUDA;
    }
    g_static_scratch_addr[dev] = (uint32_t*)addr;
  }
  uint32_t* scratch = g_static_scratch_addr[dev];
  uint32_t* e_max = scratch;                        // [out_ch]
  uint32_t* err_sink = scratch + kStaticMaxOutCh;   // written on Inf/NaN, never read
  cudaStream_t s = (cudaStream_t)stream;
  const uint32_t O = shape->out_ch, d = (uint32_t)d64;
  // the array keeps the previous call's maxima: the reduction must start from zero
  if (cudaMemsetAsync(e_max, 0, sizeof(uint32_t) * O, s) != cudaSuccess) return PSB_ERR_CUDA;
  if (cfg->norm) {
    emax_kernel<<<emax_blocks_for(O, d, 1), kThreads, 0, s>>>(w_dev, O, d, 1, e_max, err_sink, 0u, nullptr, 0u); note_launch();
  } else {
    size_t total = (size_t)O * d;
    uint32_t blocks = (uint32_t)((total + kThreads * 8 - 1) / (kThreads * 8));
    blocks = blocks < 1 ? 1 : (blocks > 1184 ? 1184 : blocks);
    emax_kernel<<<blocks, kThreads, 0, s>>>(w_dev, O, d, 0, e_max, err_sink, 0u, nullptr, 0u); note_launch();
  }
  size_t total = (size_t)O * d;
  uint32_t blocks = (uint32_t)((total + kThreads - 1) / kThreads);
  blocks = blocks > 148u * 16u ? 148u * 16u : blocks;
  sample_level_canonical_kernel<<<blocks, kThreads, 0, s>>>(
      w_dev, O, d, cfg->norm, (1u << exp_bits) - 1u, log2k, (uint32_t)cfg->seed,
      (uint32_t)(cfg->seed >> 32), cfg->layer_id, e_max, wint_out_dev, e_base_out_dev); note_launch();
  return cudaGetLastError() == cudaSuccess ? PSB_OK : PSB_ERR_CUDA;
}
