// CUDA-core contraction ("shift-add" path) and the glue kernels.
//
// The paper's capacitor unit adds x << (e + B) over the draws (Eq. 9); summed over
// the k draws that is x * (k + c_k) << (e - e_base), an integer product with the
// sampled integer weight.  On the GPU one 64-bit integer multiply-add per
// (activation, weight) pair realises exactly that sum.  This path serves layers
// that are not dense matrix products for the tensor cores: depthwise filters,
// fully connected layers at small batch, very few input channels, 8-bit unsigned
// activations, and it honours per-location draw counts directly.
#include "psb_common.cuh"

namespace psb {

namespace {

// True when one of the four bytes of `v` exceeds `limit` in magnitude (signed bytes: |b| > limit).
__device__ __forceinline__ bool bytes_beyond(uint32_t v, uint32_t is_signed, uint32_t limit) {
  const uint32_t mag = is_signed ? __vabs4(v) : v;        // |-128| = 128 as an unsigned byte
  return __vcmpgtu4(mag, limit * 0x01010101u) != 0u;
}

__device__ __forceinline__ int load_act(const void* x, uint32_t dtype, size_t idx) {
  return dtype == PSB_DT_U8 ? (int)((const uint8_t*)x)[idx] : (int)((const int8_t*)x)[idx];
}

__device__ __forceinline__ void store_outputs(const ConvArgs& a, size_t oidx, uint32_t o,
                                              uint32_t level, long long acc) {
  if (a.acc_out) a.acc_out[oidx] = acc;
  if (a.q_out || a.f32_out) {
    float sc = ldexpf(a.scale[o], a.e_base[o] - (int)level);
    int rq = a.residual ? load_act(a.residual, a.residual_dtype, oidx) : 0;
    float y = dequant(acc, sc, a.bias[o], a.residual != nullptr, rq, a.residual_scale, a.relu != 0);
    if (a.f32_out) a.f32_out[oidx] = y;
    if (a.q_out) {
      int q = requant(y, a.inv_step, a.qmin, a.qmax);
      if (a.out_dtype == PSB_DT_U8) ((uint8_t*)a.q_out)[oidx] = (uint8_t)q;
      else ((int8_t*)a.q_out)[oidx] = (int8_t)q;
    }
  }
}

// One thread per output element, output channel fastest.  For depthwise filters
// (one input channel per group) neighbouring threads read neighbouring bytes.
__global__ void __launch_bounds__(256) conv_direct_kernel(const ConvArgs a, const WintTable wt) {
  pdl_prologue();
  const size_t total = (size_t)a.N * a.OH * a.OW * a.O;
  const uint32_t Cg = a.C / a.groups, Og = a.O / a.groups;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    const uint32_t o = (uint32_t)(idx % a.O);
    const size_t pix = idx / a.O;
    const uint32_t ox = (uint32_t)(pix % a.OW);
    const uint32_t oy = (uint32_t)((pix / a.OW) % a.OH);
    const uint32_t n = (uint32_t)(pix / ((size_t)a.OW * a.OH));
    const uint32_t level = a.kmap ? a.kmap[pix] : a.uniform_log2k;
    if (level >= (uint32_t)kMaxLevels || !((a.level_mask >> level) & 1u)) {
      atomicOr(a.err, kDevErrBadLevel);
      continue;
    }
    const int32_t* w = wt.w[level] + (size_t)o * a.KH * a.KW * Cg;
    const uint32_t cbase = (o / Og) * Cg;
    long long acc = 0;
    for (uint32_t kh = 0; kh < a.KH; ++kh) {
      const int iy = (int)(oy * a.stride + kh) - (int)a.pad;
      if (iy < 0 || iy >= (int)a.H) continue;
      for (uint32_t kw = 0; kw < a.KW; ++kw) {
        const int ix = (int)(ox * a.stride + kw) - (int)a.pad;
        if (ix < 0 || ix >= (int)a.W) continue;
        const size_t xoff = (((size_t)n * a.H + iy) * a.W + ix) * a.C + cbase;
        const int32_t* wr = w + (size_t)(kh * a.KW + kw) * Cg;
        for (uint32_t ci = 0; ci < Cg; ++ci) {
          int xv = load_act(a.x, a.in_dtype, xoff + ci);
          acc += (long long)xv * (long long)__ldca(wr + ci);
        }
      }
    }
    const size_t oidx = a.out_nchw ? (((size_t)n * a.O + o) * a.OH + oy) * a.OW + ox : idx;
    store_outputs(a, oidx, o, level, acc);
  }
}

// Fully connected layers at small batch (1x1 filter on a 1x1 image, one group): a warp per output
// element, the lanes stride over the input features (coalesced runs of the filter row and of the
// activation row) and the 64-bit partial sums meet in a shuffle tree.  With one thread per output the
// 256 dependent loads of a 256-feature row made the layer ten times longer than its launch.
__global__ void __launch_bounds__(256) gemv_warp_kernel(const ConvArgs a, const WintTable wt) {
  pdl_prologue();
  const size_t total = (size_t)a.N * a.O;
  const uint32_t lane = threadIdx.x & 31u;
  for (size_t idx = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; idx < total;
       idx += ((size_t)gridDim.x * blockDim.x) >> 5) {
    const uint32_t o = (uint32_t)(idx % a.O);
    const uint32_t n = (uint32_t)(idx / a.O);
    const uint32_t level = a.kmap ? a.kmap[n] : a.uniform_log2k;
    if (level >= (uint32_t)kMaxLevels || !((a.level_mask >> level) & 1u)) {
      if (lane == 0) atomicOr(a.err, kDevErrBadLevel);
      continue;
    }
    const int32_t* w = wt.w[level] + (size_t)o * a.C;
    const size_t xoff = (size_t)n * a.C;
    long long acc = 0;
    for (uint32_t ci = lane; ci < a.C; ci += 32u)
      acc += (long long)load_act(a.x, a.in_dtype, xoff + ci) * (long long)__ldca(w + ci);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(0xFFFFFFFFu, acc, d);
    if (lane == 0) store_outputs(a, idx, o, level, acc);
  }
}

// Depthwise filters (one input channel per output channel), channels-last, one draw count for
// the layer: a thread owns 8 consecutive channels of one output location.  The block keeps the
// layer's integer filter in shared memory as [tap][channel]; activations come in 8-byte loads;
// the integer sum x * W_k over the taps is Eq. 9 summed over the draws.  Writes 8 codes at once.
__global__ void __launch_bounds__(256) dwconv_nhwc8_kernel(const ConvArgs a, const int32_t* wint) {
  pdl_prologue();
  extern __shared__ int32_t dw_w[];   // [KH*KW][C]
  const uint32_t taps = a.KH * a.KW, C = a.C;
  for (uint32_t i = threadIdx.x; i < taps * C; i += blockDim.x) dw_w[(i % taps) * C + i / taps] = wint[i];
  __syncthreads();
  const uint32_t level = a.uniform_log2k;
  const uint32_t groups = C / 8u;
  const size_t total = (size_t)a.N * a.OH * a.OW * groups;
  const bool has_res = a.residual != nullptr;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    const uint32_t g = (uint32_t)(idx % groups);
    const size_t pix = idx / groups;
    const uint32_t ox = (uint32_t)(pix % a.OW), oy = (uint32_t)((pix / a.OW) % a.OH);
    const uint32_t n = (uint32_t)(pix / ((size_t)a.OW * a.OH));
    const uint32_t c0 = g * 8u;
    long long acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (uint32_t kh = 0; kh < a.KH; ++kh) {
      const int iy = (int)(oy * a.stride + kh) - (int)a.pad;
      if (iy < 0 || iy >= (int)a.H) continue;
      for (uint32_t kw = 0; kw < a.KW; ++kw) {
        const int ix = (int)(ox * a.stride + kw) - (int)a.pad;
        if (ix < 0 || ix >= (int)a.W) continue;
        const uint2 xv = __ldcg(reinterpret_cast<const uint2*>(
            (const uint8_t*)a.x + (((size_t)n * a.H + iy) * a.W + ix) * C + c0));
        const int32_t* wr = dw_w + (kh * a.KW + kw) * C + c0;
        const int4 w0 = *reinterpret_cast<const int4*>(wr), w1 = *reinterpret_cast<const int4*>(wr + 4);
        const int ws[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
        const uint32_t xw[2] = {xv.x, xv.y};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t b = (xw[j >> 2] >> (8 * (j & 3))) & 0xFFu;
          const int xi = a.in_dtype == PSB_DT_U8 ? (int)b : (int)(int8_t)b;
          acc[j] += (long long)xi * (long long)ws[j];
        }
      }
    }
    const size_t oidx = pix * C + c0;
    uint32_t rw[2] = {0, 0};
    if (has_res) {
      const uint2 rv = __ldcg(reinterpret_cast<const uint2*>((const uint8_t*)a.residual + oidx));
      rw[0] = rv.x; rw[1] = rv.y;
    }
    uint32_t qw[2] = {0, 0};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint32_t o = c0 + j;
      const float sc = ldexpf(a.scale[o], a.e_base[o] - (int)level);
      int rb = (int)((rw[j >> 2] >> (8 * (j & 3))) & 0xFFu);
      if (a.residual_dtype == PSB_DT_S8) rb = (int)(int8_t)rb;
      const float y = dequant(acc[j], sc, a.bias[o], has_res, rb, a.residual_scale, a.relu != 0);
      const int q = requant(y, a.inv_step, a.qmin, a.qmax);
      qw[j >> 2] |= ((uint32_t)q & 0xFFu) << (8 * (j & 3));
    }
    *reinterpret_cast<uint2*>((uint8_t*)a.q_out + oidx) = make_uint2(qw[0], qw[1]);
  }
}

// Depthwise 3x3, channels-last, one draw count, only codes wanted.  A thread owns 4 channels
// and kDwSeg consecutive output columns of one output row: its 36 filter values and 8 output
// constants stay in registers, every input column of the 3-row band is loaded once (one 32-bit
// load per row) and serves up to three outputs.  All loads of the band are issued before the
// arithmetic; positions outside the image read as zero through a predicate.  The output stage
// is dequant()/requant() written without the conversion unit (exponent arithmetic, see
// acc_to_float_small).  Adjacent threads take adjacent channel quads, so a warp's loads and
// stores are contiguous runs of the channels-last rows.
template <int S>
struct DwSeg { static constexpr int kOut = S == 1 ? 8 : 4; static constexpr int kCols = (kOut - 1) * S + 3; };

template <int S, bool kSignedIn>
__global__ void __launch_bounds__(256, 2) dwconv3x3_row_kernel(const ConvArgs a, const int32_t* wint) {
  pdl_prologue();
  constexpr int L = DwSeg<S>::kOut, NC = DwSeg<S>::kCols;
  const uint32_t C = a.C, G = C / 4u;
  const uint32_t segs = (a.OW + L - 1) / L;
  const uint32_t total = a.N * a.OH * segs * G;   // the launcher keeps this below 2^32
  const uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  uint32_t t = idx / G;
  const uint32_t c0 = (idx - t * G) * 4u;
  const uint32_t seg = t % segs; t /= segs;
  const uint32_t oy = t % a.OH, n = t / a.OH;
  const uint32_t ox0 = seg * L;

  // band of input: rows iy0..iy0+2, columns ix0..ix0+NC-1
  const int iy0 = (int)(oy * S) - (int)a.pad, ix0 = (int)(ox0 * S) - (int)a.pad;
  const uint32_t last_ox = min(ox0 + (uint32_t)L, a.OW) - 1u;
  const int ix_end = (int)(last_ox * S) - (int)a.pad + 2;     // last column any output of the segment reads
  uint32_t raw[3][NC];
#pragma unroll
  for (int r = 0; r < 3; ++r) {
    const int iy = iy0 + r;
    const bool row_in = (unsigned)iy < a.H;
    const uint8_t* rp = (const uint8_t*)a.x + ((size_t)(n * a.H + (row_in ? iy : 0)) * a.W) * C + c0;
#pragma unroll
    for (int cidx = 0; cidx < NC; ++cidx) {
      const int ix = ix0 + cidx;
      raw[r][cidx] = 0u;
      if (row_in && (unsigned)ix < a.W && ix <= ix_end)
        raw[r][cidx] = __ldcg(reinterpret_cast<const uint32_t*>(rp + (size_t)ix * C));
    }
  }
  // filter [channel][tap] and output constants of the 4 channels
  int w[36];
  {
    const int4* wp = reinterpret_cast<const int4*>(wint + (size_t)c0 * 9u);
#pragma unroll
    for (int i = 0; i < 9; ++i) {
      const int4 v = __ldca(wp + i);
      w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
    }
  }
  float sc[4], bi[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    sc[j] = ldexpf(a.scale[c0 + j], a.e_base[c0 + j] - (int)a.uniform_log2k);
    bi[j] = a.bias[c0 + j];
  }
  const bool has_res = a.residual != nullptr;
  const uint32_t res_sign = a.residual_dtype == PSB_DT_S8 ? 0x80u : 0u;
  const float res_bias = 8388608.0f + (float)res_sign;
  const float relu_floor = (a.relu && a.qmin < 0) ? 0.0f : __int_as_float(0xFF800000);
  const float qmin_f = (float)a.qmin, qmax_f = (float)a.qmax;
  const size_t obase = ((size_t)(n * a.OH + oy) * a.OW + ox0) * C + c0;

#pragma unroll
  for (int i = 0; i < L; ++i) {
    if (ox0 + i > last_ox) break;
    const size_t oidx = obase + (size_t)i * C;
    uint32_t rv = 0u;
    if (has_res) rv = __ldcg(reinterpret_cast<const uint32_t*>((const uint8_t*)a.residual + oidx));
    long long acc[4] = {0, 0, 0, 0};
#pragma unroll
    for (int r = 0; r < 3; ++r) {
#pragma unroll
      for (int kw = 0; kw < 3; ++kw) {
        const uint32_t v = raw[r][i * S + kw];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t b = (v >> (8 * j)) & 0xFFu;
          const int xi = kSignedIn ? (int)(int8_t)b : (int)b;
          acc[j] += (long long)xi * (long long)w[j * 9 + r * 3 + kw];
        }
      }
    }
    uint32_t q[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float y = __fmaf_rn(acc_to_float_small(acc[j]), sc[j], bi[j]);
      if (has_res) {
        const uint32_t rb = ((rv >> (8 * j)) & 0xFFu) ^ res_sign;   // byte + 128 if signed
        y = __fmaf_rn(__uint_as_float(0x4B000000u | rb) - res_bias, a.residual_scale, y);
      }
      y = fmaxf(y, relu_floor);
      // clamp, then round half to even by adding 1.5 * 2^23: the low byte of the sum is the code
      const float tq = fminf(fmaxf(__fmul_rn(y, a.inv_step), qmin_f), qmax_f);
      q[j] = __float_as_uint(tq + 12582912.0f);
    }
    *reinterpret_cast<uint32_t*>((uint8_t*)a.q_out + oidx) =
        __byte_perm(__byte_perm(q[0], q[1], 0x0040), __byte_perm(q[2], q[3], 0x0040), 0x5410);
  }
}

// The same layer class with the arithmetic cut down to what the bytes need.  The integer sum x * W_k over the
// nine taps (Eq. 9 summed over the draws) fits 32 bits whenever (largest activation) x (sum of |W_k| of the
// channel) stays below 2^31; the sampler keeps those sums, so a thread knows per channel whether 32-bit
// multiply-adds are exact and falls back to 64-bit ones where they are not.  A thread owns 4 channels and kOut
// consecutive outputs of one row and works channel by channel: the bytes of the 3 x kCols input words are
// extracted once per row and channel and serve up to three outputs each, one multiply-add per tap; the output
// stage is dequant()/requant() with conversion-unit instructions (one int -> float, one float -> int, both
// round to nearest even as the definitions ask).  About 25 instructions per output where the 64-bit kernel
// above needs about 70.
template <typename Acc>
__device__ __forceinline__ float dw_acc_to_float(Acc acc);
template <>
__device__ __forceinline__ float dw_acc_to_float<int>(int acc) { return __int2float_rn(acc); }
template <>
__device__ __forceinline__ float dw_acc_to_float<long long>(long long acc) { return acc_to_float(acc); }

template <int S, bool kSignedIn, typename Acc>
__device__ __forceinline__ void dw_channel(const uint32_t (&raw)[3][DwSeg<S>::kCols], int j, const int32_t* wch,
                                           float sc, float bi, bool has_res, const uint32_t (&rv)[DwSeg<S>::kOut],
                                           bool res_signed, float res_scale, float relu_floor, float inv_step,
                                           float lo_f, float hi_f, uint32_t n_out, uint32_t (&qw)[DwSeg<S>::kOut]) {
  constexpr int L = DwSeg<S>::kOut, NC = DwSeg<S>::kCols;
  Acc acc[L];
#pragma unroll
  for (int i = 0; i < L; ++i) acc[i] = 0;
#pragma unroll
  for (int r = 0; r < 3; ++r) {
    const int w0 = __ldca(wch + r * 3), w1 = __ldca(wch + r * 3 + 1), w2 = __ldca(wch + r * 3 + 2);
    int xb[NC];
#pragma unroll
    for (int cidx = 0; cidx < NC; ++cidx) {
      const uint32_t b = (raw[r][cidx] >> (8 * j)) & 0xFFu;
      xb[cidx] = kSignedIn ? (int)(signed char)b : (int)b;
    }
#pragma unroll
    for (int i = 0; i < L; ++i) {
      acc[i] += (Acc)xb[i * S] * (Acc)w0;
      acc[i] += (Acc)xb[i * S + 1] * (Acc)w1;
      acc[i] += (Acc)xb[i * S + 2] * (Acc)w2;
    }
  }
#pragma unroll
  for (int i = 0; i < L; ++i) {
    if ((uint32_t)i >= n_out) break;
    float y = __fmaf_rn(dw_acc_to_float<Acc>(acc[i]), sc, bi);
    if (has_res) {
      const uint32_t rb = (rv[i] >> (8 * j)) & 0xFFu;
      y = __fmaf_rn(res_signed ? (float)(int)(signed char)rb : (float)rb, res_scale, y);
    }
    y = fmaxf(y, relu_floor);
    const float t = fminf(fmaxf(__fmul_rn(y, inv_step), lo_f), hi_f);
    const uint32_t q = (uint32_t)__float2int_rn(t) & 0xFFu;
    qw[i] |= q << (8 * j);
  }
}

template <int S, bool kSignedIn>
__global__ void __launch_bounds__(256, 3) dwconv3x3_row32_kernel(const ConvArgs a, const int32_t* wint,
                                                                 const uint32_t* rowsum256,
                                                                 uint32_t amax) {
  pdl_prologue();
  constexpr int L = DwSeg<S>::kOut, NC = DwSeg<S>::kCols;
  const uint32_t C = a.C, G = C / 4u;
  const uint32_t segs = (a.OW + L - 1) / L;
  const uint32_t total = a.N * a.OH * segs * G;   // the launcher keeps this below 2^32
  const uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  uint32_t t = idx / G;
  const uint32_t c0 = (idx - t * G) * 4u;
  const uint32_t seg = t % segs; t /= segs;
  const uint32_t oy = t % a.OH, n = t / a.OH;
  const uint32_t ox0 = seg * L;

  // band of input: rows iy0..iy0+2, columns ix0..ix0+NC-1, every word = 4 channels of one position
  const int iy0 = (int)(oy * S) - (int)a.pad, ix0 = (int)(ox0 * S) - (int)a.pad;
  const uint32_t last_ox = min(ox0 + (uint32_t)L, a.OW) - 1u;
  const int ix_end = (int)(last_ox * S) - (int)a.pad + 2;     // last column any output of the segment reads
  uint32_t raw[3][NC];
#pragma unroll
  for (int r = 0; r < 3; ++r) {
    const int iy = iy0 + r;
    const bool row_in = (unsigned)iy < a.H;
    const uint8_t* rp = (const uint8_t*)a.x + ((size_t)(n * a.H + (row_in ? iy : 0)) * a.W) * C + c0;
#pragma unroll
    for (int cidx = 0; cidx < NC; ++cidx) {
      const int ix = ix0 + cidx;
      raw[r][cidx] = 0u;
      if (row_in && (unsigned)ix < a.W && ix <= ix_end)
        raw[r][cidx] = __ldcg(reinterpret_cast<const uint32_t*>(rp + (size_t)ix * C));
    }
  }
  const bool has_res = a.residual != nullptr;
  const size_t obase = ((size_t)(n * a.OH + oy) * a.OW + ox0) * C + c0;
  const uint32_t n_out = last_ox - ox0 + 1u;
  uint32_t rv[L], qw[L];
#pragma unroll
  for (int i = 0; i < L; ++i) {
    qw[i] = 0u;
    rv[i] = 0u;
    if (has_res && (uint32_t)i < n_out)
      rv[i] = __ldcg(reinterpret_cast<const uint32_t*>((const uint8_t*)a.residual + obase + (size_t)i * C));
  }
  const float relu_floor = a.relu ? 0.0f : __int_as_float(0xFF800000);
  const float lo_f = (float)a.qmin, hi_f = (float)a.qmax;
  const bool res_signed = a.residual_dtype == PSB_DT_S8;
  const uint32_t level = a.uniform_log2k;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t o = c0 + j;
    const float sc = ldexpf(a.scale[o], a.e_base[o] - (int)level), bi = a.bias[o];
    const int32_t* wch = wint + (size_t)o * 9u;
    // (a sum marked unknown, 0xFFFFFFFF, fails the test like a large one)
    const unsigned long long bound = (unsigned long long)__ldca(rowsum256 + (size_t)level * a.O + o) * 256ull * amax;
    if (bound < (1ull << 31))
      dw_channel<S, kSignedIn, int>(raw, j, wch, sc, bi, has_res, rv, res_signed, a.residual_scale, relu_floor,
                                    a.inv_step, lo_f, hi_f, n_out, qw);
    else
      dw_channel<S, kSignedIn, long long>(raw, j, wch, sc, bi, has_res, rv, res_signed, a.residual_scale, relu_floor,
                                          a.inv_step, lo_f, hi_f, n_out, qw);
  }
#pragma unroll
  for (int i = 0; i < L; ++i)
    if ((uint32_t)i < n_out) *reinterpret_cast<uint32_t*>((uint8_t*)a.q_out + obase + (size_t)i * C) = qw[i];
}

// x ^ 0x80 over a whole tensor: unsigned bytes become (x - 128) as signed bytes, 16 per thread.
__global__ void offset128_kernel(const uint4* src, uint4* dst, size_t n16, uint32_t limit,
                                 uint32_t* __restrict__ err) {
  pdl_prologue();
  bool bad = false;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (size_t)gridDim.x * blockDim.x) {
    uint4 v = __ldcg(src + i);
    if (limit < 255u)
      bad |= bytes_beyond(v.x, 0u, limit) | bytes_beyond(v.y, 0u, limit) | bytes_beyond(v.z, 0u, limit) |
             bytes_beyond(v.w, 0u, limit);
    v.x ^= 0x80808080u; v.y ^= 0x80808080u; v.z ^= 0x80808080u; v.w ^= 0x80808080u;
    dst[i] = v;
  }
  if (bad) atomicOr(err, kDevErrRange);
}

// Largest byte magnitude of a tensor against the bound the caller gave (PSB_CHECK_RANGE): 16 bytes per
// thread and iteration, the ragged tail byte by byte.
__global__ void range_check_kernel(const uint8_t* x, size_t bytes, uint32_t is_signed, uint32_t limit,
                                   uint32_t* __restrict__ err) {
  pdl_prologue();
  bool bad = false;
  const size_t head = min(bytes, (size_t)((16u - ((uintptr_t)x & 15u)) & 15u));   // bytes before 16-byte alignment
  const size_t n16 = (bytes - head) / 16u;
  const uint4* x16 = reinterpret_cast<const uint4*>(x + head);
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (size_t)gridDim.x * blockDim.x) {
    const uint4 v = __ldcg(x16 + i);
    bad |= bytes_beyond(v.x, is_signed, limit) | bytes_beyond(v.y, is_signed, limit) |
           bytes_beyond(v.z, is_signed, limit) | bytes_beyond(v.w, is_signed, limit);
  }
  if (blockIdx.x == 0) {
    const size_t tail0 = head + n16 * 16u;
    for (size_t i = threadIdx.x; i < head; i += blockDim.x) bad |= bytes_beyond((uint32_t)x[i], is_signed, limit);
    for (size_t i = tail0 + threadIdx.x; i < bytes; i += blockDim.x) bad |= bytes_beyond((uint32_t)x[i], is_signed, limit);
  }
  if (bad) atomicOr(err, kDevErrRange);
}

// Explicit gather of the activation matrix for filters with few input channels (e.g. a 7x7
// stem on 3 channels): row m = output location; filter row kh occupies bytes
// [kh * run_pitch, kh * run_pitch + KW * C) of it, which in a channels-last image is one
// contiguous run of the input row iy0 + kh; the rest of the matrix row is zero.  Values are
// stored minus `offset` (0 or 128) as signed bytes; a padded input position is the value 0, i.e.
// -offset.  A block handles a strip of up to kIm2colPix consecutive output locations of
// kIm2colRows consecutive output rows: the input-row spans they touch are staged in shared
// memory, each at the byte offset that keeps its 16-byte pieces aligned with global memory
// (whole-piece copies; single bytes only at the image's edges), then each thread copies whole
// runs: aligned shared-memory words, a funnel shift by the byte misalignment, 8-byte stores.
constexpr uint32_t kIm2colPix = 128;
constexpr uint32_t kIm2colRows = 2;

__host__ __device__ __forceinline__ uint32_t im2col_span_pitch(uint32_t stride, uint32_t C, uint32_t run_pitch) {
  // alignment shift (< 16) + the last pixel's run, read up to run_pitch + 7 bytes past its start in whole words
  return (15u + (kIm2colPix - 1u) * stride * C + run_pitch + 12u + 15u) & ~15u;
}

__global__ void __launch_bounds__(256) im2col_s8_kernel(const ConvArgs a, uint32_t kpad, uint32_t run_pitch,
                                                       uint32_t offset, uint32_t limit, int8_t* __restrict__ dst) {
  pdl_prologue();
  bool bad = false;
  extern __shared__ __align__(16) uint32_t im2col_smem[];     // [staged rows][span_pitch / 4] words
  __shared__ uint32_t row_adj[(kIm2colRows - 1u) * 8u + 128u];   // per staged row: byte offset of the span's start
  const uint32_t span_pitch = im2col_span_pitch(a.stride, a.C, run_pitch);
  const uint32_t strips = (a.OW + kIm2colPix - 1) / kIm2colPix;
  const uint32_t row_groups = (a.OH + kIm2colRows - 1) / kIm2colRows;
  const uint32_t strip = blockIdx.x % strips;
  const uint32_t oy0 = ((blockIdx.x / strips) % row_groups) * kIm2colRows;
  const uint32_t n = blockIdx.x / (strips * row_groups);
  const uint32_t nrows = min(kIm2colRows, a.OH - oy0);
  const uint32_t ox0 = strip * kIm2colPix;
  const uint32_t npix = min(kIm2colPix, a.OW - ox0);
  const int ix0 = (int)(ox0 * a.stride) - (int)a.pad;         // leftmost input column of the strip
  const int iy0 = (int)(oy0 * a.stride) - (int)a.pad;         // topmost input row
  const uint32_t staged = (nrows - 1u) * a.stride + a.KH;     // input rows the block touches
  const uint32_t span_bytes = ((npix - 1u) * a.stride + a.KW) * a.C;
  const uint8_t* x = (const uint8_t*)a.x;
  const uint32_t flip = offset ? 0x80808080u : 0u;            // v - 128 == v ^ 0x80 as a byte
  const uint32_t fill = (0u - offset) & 0xFFu;
  const uint32_t fill4 = fill * 0x01010101u;
  const uint32_t is_signed = a.in_dtype == PSB_DT_S8 ? 1u : 0u;
  // bytes [lo_b, hi_b) of a span lie inside the image row
  const int lo_b = ix0 < 0 ? -ix0 * (int)a.C : 0;
  const int hi_b = min((int)span_bytes, ((int)a.W - ix0) * (int)a.C);
  const uint32_t pieces = span_pitch / 16u;
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  for (uint32_t sr = warp; sr < staged; sr += 8u) {
    const int iy = iy0 + (int)sr;
    const bool row_in = iy >= 0 && iy < (int)a.H;
    const uint8_t* src = x + (((size_t)n * a.H + (row_in ? iy : 0)) * a.W) * a.C + (ptrdiff_t)ix0 * (int)a.C;
    const uint32_t adj = (uint32_t)((uintptr_t)src & 15u);    // span byte b sits at shared byte adj + b
    if (lane == 0) row_adj[sr] = adj;
    const uint8_t* src16 = src - adj;                          // 16-byte aligned
    uint32_t* out_row = im2col_smem + sr * (span_pitch / 4u);
    for (uint32_t pc = lane; pc < pieces; pc += 32u) {
      const int b0 = (int)(pc * 16u) - (int)adj;               // span byte of the piece's first byte
      uint4 v;
      if (row_in && b0 >= lo_b && b0 + 16 <= hi_b) {
        v = __ldcg(reinterpret_cast<const uint4*>(src16 + pc * 16u));
        bad |= bytes_beyond(v.x, is_signed, limit) | bytes_beyond(v.y, is_signed, limit) |
               bytes_beyond(v.z, is_signed, limit) | bytes_beyond(v.w, is_signed, limit);
        v.x ^= flip; v.y ^= flip; v.z ^= flip; v.w ^= flip;
      } else {
        uint32_t wv[4] = {fill4, fill4, fill4, fill4};
        if (row_in && b0 + 16 > lo_b && b0 < hi_b) {
          for (int j = 0; j < 16; ++j) {
            const int b = b0 + j;
            if (b >= lo_b && b < hi_b) {
              const uint32_t raw = src[b];
              bad |= bytes_beyond(raw, is_signed, limit);
              wv[j >> 2] = (wv[j >> 2] & ~(0xFFu << (8 * (j & 3)))) | (((raw ^ offset) & 0xFFu) << (8 * (j & 3)));
            }
          }
        }
        v = make_uint4(wv[0], wv[1], wv[2], wv[3]);
      }
      *reinterpret_cast<uint4*>(out_row + pc * 4u) = v;
    }
  }
  if (bad) atomicOr(a.err, kDevErrRange);
  __syncthreads();
  const uint32_t run = a.KW * a.C;                            // bytes of one filter row
  const uint32_t words = run_pitch / 4u;
  const uint32_t tail0 = a.KH * run_pitch;                    // zero bytes [tail0, kpad)
  const uint32_t items = a.KH + (kpad > tail0 ? 1u : 0u);
  const uint32_t per_row = npix * items;
  for (uint32_t t = threadIdx.x; t < nrows * per_row; t += blockDim.x) {
    const uint32_t ry = t / per_row, t1 = t - ry * per_row;
    const uint32_t px = t1 / items, kh = t1 - px * items;
    const size_t m = ((size_t)n * a.OH + oy0 + ry) * a.OW + ox0 + px;
    int8_t* out = dst + m * kpad + kh * run_pitch;
    if (kh == a.KH) {
      for (uint32_t b = 0; b < kpad - tail0; b += 8u) *reinterpret_cast<uint2*>(out + b) = make_uint2(0u, 0u);
      continue;
    }
    const uint32_t sr = ry * a.stride + kh;
    const uint32_t o = row_adj[sr] + px * a.stride * a.C;     // byte offset of the run in the staged row
    const uint32_t* wsrc = im2col_smem + sr * (span_pitch / 4u) + (o >> 2);
    const uint32_t sh = (o & 3u) * 8u;
    uint32_t lo = wsrc[0];
    for (uint32_t w = 0; w < words; w += 2u) {
      const uint32_t mid = wsrc[w + 1], hi = wsrc[w + 2];
      uint32_t v0 = __funnelshift_r(lo, mid, sh), v1 = __funnelshift_r(mid, hi, sh);
      // bytes at or beyond the run are K padding: zero
      const uint32_t b0 = w * 4u;
      if (b0 + 4u > run) v0 = b0 >= run ? 0u : (v0 & (0xFFFFFFFFu >> (8u * (b0 + 4u - run))));
      if (b0 + 8u > run) v1 = b0 + 4u >= run ? 0u : (v1 & (0xFFFFFFFFu >> (8u * (b0 + 8u - run))));
      *reinterpret_cast<uint2*>(out + b0) = make_uint2(v0, v1);
      lo = hi;
    }
  }
}

// [N][C][HW] -> [N][HW][C], elements of 1 byte, through a 32x33 tile.
__global__ void nchw_to_nhwc_u8_kernel(const uint8_t* src, uint8_t* dst,
                                       uint32_t C, uint32_t HW, uint32_t is_signed, uint32_t limit,
                                       uint32_t* __restrict__ err) {
  pdl_prologue();
  __shared__ uint8_t tile[32][33];
  const size_t base = (size_t)blockIdx.z * C * HW;
  const uint32_t p0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
  bool bad = false;
  for (uint32_t r = threadIdx.y; r < 32; r += blockDim.y) {
    uint32_t c = c0 + r, p = p0 + threadIdx.x;
    if (c < C && p < HW) {
      const uint8_t v = src[base + (size_t)c * HW + p];
      bad |= bytes_beyond((uint32_t)v, is_signed, limit);
      tile[r][threadIdx.x] = v;
    }
  }
  if (bad) atomicOr(err, kDevErrRange);
  __syncthreads();
  for (uint32_t r = threadIdx.y; r < 32; r += blockDim.y) {
    uint32_t p = p0 + r, c = c0 + threadIdx.x;
    if (c < C && p < HW) dst[base + (size_t)p * C + c] = tile[threadIdx.x][r];
  }
}

// The same for C and HW multiples of 4, four bytes at a time.  A block moves 32 channels x 128
// locations.  Warp i takes channels 4i..4i+3: each lane loads 4 locations of each of them (four
// 128-byte runs per warp), transposes the 4x4 bytes in registers and parks the four words (one
// per location, 4 channels each) in shared memory with one 16-byte store.  Then 8 consecutive
// lanes write the 32 channel bytes of one location: whole 32-byte sectors, no bank conflicts
// (row pitch 132 words: bank = 4 * quad + location).
__global__ void __launch_bounds__(256) nchw_to_nhwc_u8x4_kernel(const uint8_t* src,
                                                               uint8_t* __restrict__ dst, uint32_t C,
                                                               uint32_t HW, uint32_t is_signed, uint32_t limit,
                                                               uint32_t* __restrict__ err) {
  pdl_prologue();
  __shared__ __align__(16) uint32_t tile[8][132];
  const size_t base = (size_t)blockIdx.z * C * HW;
  const uint32_t p0 = blockIdx.x * 128u, c0 = blockIdx.y * 32u;
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  {
    const uint32_t c = c0 + 4u * warp, p = p0 + 4u * lane;
    uint32_t r[4] = {0u, 0u, 0u, 0u};
    if (c < C && p < HW) {
#pragma unroll
      for (int k = 0; k < 4; ++k)
        r[k] = __ldcg(reinterpret_cast<const uint32_t*>(src + base + (size_t)(c + k) * HW + p));
      if (bytes_beyond(r[0], is_signed, limit) | bytes_beyond(r[1], is_signed, limit) |
          bytes_beyond(r[2], is_signed, limit) | bytes_beyond(r[3], is_signed, limit))
        atomicOr(err, kDevErrRange);
    }
    const uint32_t a = __byte_perm(r[0], r[1], 0x5140), b = __byte_perm(r[2], r[3], 0x5140);
    const uint32_t cc = __byte_perm(r[0], r[1], 0x7362), d = __byte_perm(r[2], r[3], 0x7362);
    *reinterpret_cast<uint4*>(&tile[warp][4u * lane]) =
        make_uint4(__byte_perm(a, b, 0x5410), __byte_perm(a, b, 0x7632), __byte_perm(cc, d, 0x5410),
                   __byte_perm(cc, d, 0x7632));
  }
  __syncthreads();
  const uint32_t q = threadIdx.x & 7u;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const uint32_t pl = (threadIdx.x >> 3) + 32u * r;
    const uint32_t p = p0 + pl, c = c0 + 4u * q;
    if (p < HW && c < C) *reinterpret_cast<uint32_t*>(dst + base + (size_t)p * C + c) = tile[q][pl];
  }
}

__global__ void maxpool_kernel(const uint8_t* x, uint32_t nchw, uint32_t N, uint32_t C,
                               uint32_t H, uint32_t W, uint32_t k, uint32_t stride, uint32_t pad,
                               uint32_t OH, uint32_t OW, uint8_t* __restrict__ out) {
  pdl_prologue();
  const size_t total = (size_t)N * OH * OW * C;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    uint32_t c, ox, oy, n;
    if (nchw) {
      ox = idx % OW; oy = (idx / OW) % OH; c = (idx / ((size_t)OW * OH)) % C;
      n = idx / ((size_t)OW * OH * C);
    } else {
      c = idx % C; ox = (idx / C) % OW; oy = (idx / ((size_t)C * OW)) % OH;
      n = idx / ((size_t)C * OW * OH);
    }
    int best = 0;
    for (uint32_t kh = 0; kh < k; ++kh) {
      int iy = (int)(oy * stride + kh) - (int)pad;
      if (iy < 0 || iy >= (int)H) continue;
      for (uint32_t kw = 0; kw < k; ++kw) {
        int ix = (int)(ox * stride + kw) - (int)pad;
        if (ix < 0 || ix >= (int)W) continue;
        size_t xi = nchw ? (((size_t)n * C + c) * H + iy) * W + ix
                         : (((size_t)n * H + iy) * W + ix) * C + c;
        best = max(best, (int)x[xi]);
      }
    }
    out[idx] = (uint8_t)best;
  }
}

// Channels-last max-pooling, 16 channels per thread: 16-byte loads, byte-wise maxima.
__global__ void __launch_bounds__(256) maxpool_nhwc16_kernel(const uint8_t* x, uint32_t N, uint32_t C,
                                                            uint32_t H, uint32_t W, uint32_t k, uint32_t stride,
                                                            uint32_t pad, uint32_t OH, uint32_t OW,
                                                            uint8_t* __restrict__ out) {
  pdl_prologue();
  const uint32_t groups = C / 16u;
  const size_t total = (size_t)N * OH * OW * groups;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    const uint32_t g = (uint32_t)(idx % groups);
    const size_t pix = idx / groups;
    const uint32_t ox = (uint32_t)(pix % OW), oy = (uint32_t)((pix / OW) % OH);
    const uint32_t n = (uint32_t)(pix / ((size_t)OW * OH));
    uint4 best = make_uint4(0, 0, 0, 0);
    for (uint32_t kh = 0; kh < k; ++kh) {
      const int iy = (int)(oy * stride + kh) - (int)pad;
      if (iy < 0 || iy >= (int)H) continue;
      for (uint32_t kw = 0; kw < k; ++kw) {
        const int ix = (int)(ox * stride + kw) - (int)pad;
        if (ix < 0 || ix >= (int)W) continue;
        const uint4 v = __ldcg(reinterpret_cast<const uint4*>(x + (((size_t)n * H + iy) * W + ix) * C + g * 16u));
        best.x = __vmaxu4(best.x, v.x); best.y = __vmaxu4(best.y, v.y);
        best.z = __vmaxu4(best.z, v.z); best.w = __vmaxu4(best.w, v.w);
      }
    }
    *reinterpret_cast<uint4*>(out + pix * C + g * 16u) = best;
  }
}

// One warp per (n, c): integer sum over H*W, then one re-quantisation.
// Channels-last, 16 channels per thread: every load is 16 bytes, neighbouring threads read neighbouring
// channel groups of the same position.
__global__ void __launch_bounds__(128) avgpool_nhwc16_kernel(const uint8_t* x, uint32_t N, uint32_t C, uint32_t HW,
                                                             float pool_mul, int qmin, int qmax, uint8_t* __restrict__ out) {
  pdl_prologue();
  const uint32_t groups = C / 16u;
  const uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= N * groups) return;
  const uint32_t n = idx / groups, g = idx - n * groups;
  const uint8_t* src = x + (size_t)n * HW * C + g * 16u;
  int sum[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) sum[j] = 0;
#pragma unroll 4
  for (uint32_t p = 0; p < HW; ++p) {
    const uint4 v = __ldcg(reinterpret_cast<const uint4*>(src + (size_t)p * C));
    const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 16; ++j) sum[j] += (int)((w4[j >> 2] >> (8 * (j & 3))) & 0xFFu);
  }
  uint32_t q[4] = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int j = 0; j < 16; ++j)
    q[j >> 2] |= ((uint32_t)requant((float)sum[j], pool_mul, qmin, qmax) & 0xFFu) << (8 * (j & 3));
  *reinterpret_cast<uint4*>(out + (size_t)n * C + g * 16u) = make_uint4(q[0], q[1], q[2], q[3]);
}

__global__ void avgpool_kernel(const uint8_t* x, uint32_t nchw, uint32_t N, uint32_t C,
                               uint32_t HW, float pool_mul, int qmin, int qmax,
                               uint8_t* __restrict__ out) {
  pdl_prologue();
  const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= N * C) return;
  const uint32_t n = warp / C, c = warp % C;
  int sum = 0;
  for (uint32_t p = lane; p < HW; p += 32) {
    size_t xi = nchw ? ((size_t)n * C + c) * HW + p : ((size_t)n * HW + p) * C + c;
    sum += x[xi];
  }
  sum = __reduce_add_sync(0xFFFFFFFFu, sum);
  if (lane == 0) out[warp] = (uint8_t)requant((float)sum, pool_mul, qmin, qmax);
}

uint32_t grid_for(size_t total, uint32_t threads) {
  size_t b = (total + threads - 1) / threads;
  if (b < 1) b = 1;
  if (b > 148u * 32u) b = 148u * 32u;
  return (uint32_t)b;
}

}  // namespace

cudaError_t launch_offset128(const void* src, void* dst, size_t bytes, uint32_t limit, uint32_t* err, cudaStream_t s) {
  const size_t n16 = bytes / 16;
  launch_pdl(offset128_kernel, grid_for(n16, 256), 256, 0, s, (const uint4*)src, (uint4*)dst, n16, limit, err);
  note_launch();
  return cudaGetLastError();
}

cudaError_t launch_range_check(const void* x, size_t bytes, uint32_t is_signed, uint32_t limit, uint32_t* err,
                               cudaStream_t s) {
  uint32_t blocks = grid_for(bytes / 16 + 1, 256);
  if (blocks > 148u * 8u) blocks = 148u * 8u;
  launch_pdl(range_check_kernel, blocks, 256, 0, s, (const uint8_t*)x, bytes, is_signed, limit, err);
  note_launch();
  return cudaGetLastError();
}

cudaError_t launch_shift_add(const ConvArgs& a, const WintTable& wt, const uint32_t* rowsum256, uint32_t amax,
                             cudaStream_t s) {
  size_t total = (size_t)a.N * a.OH * a.OW * a.O;
  // depthwise, channels-last, one draw count, only codes wanted: the vectorised kernel
  const size_t dw_smem = (size_t)a.KH * a.KW * a.C * sizeof(int32_t);
  if (a.groups == a.C && a.O == a.C && a.C % 8u == 0 && !a.kmap && a.q_out && !a.f32_out && !a.acc_out &&
      !a.out_nchw && dw_smem <= 64 * 1024 &&
      !(((uintptr_t)a.x | (uintptr_t)a.q_out | (uintptr_t)a.residual) & 7u)) {
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
      cudaFuncSetAttribute(dwconv_nhwc8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
      attr_set[dev] = true;
    }
    if (a.KH == 3 && a.KW == 3 && (a.stride == 1 || a.stride == 2)) {
      const uint32_t seg_out = a.stride == 1 ? DwSeg<1>::kOut : DwSeg<2>::kOut;
      const uint64_t threads = (uint64_t)a.N * a.OH * ((a.OW + seg_out - 1) / seg_out) * (a.C / 4u);
      if (threads < (1ull << 32) - 256u) {
        const uint32_t blocks = (uint32_t)((threads + 255u) / 256u);
        const int32_t* wl = wt.w[a.uniform_log2k];
        const bool sg = a.in_dtype == PSB_DT_S8;
        if (rowsum256) {
          if (a.stride == 1) {
            if (sg) launch_pdl(dwconv3x3_row32_kernel<1, true>, blocks, 256, 0, s, a, wl, rowsum256, amax);
            else launch_pdl(dwconv3x3_row32_kernel<1, false>, blocks, 256, 0, s, a, wl, rowsum256, amax);
          } else {
            if (sg) launch_pdl(dwconv3x3_row32_kernel<2, true>, blocks, 256, 0, s, a, wl, rowsum256, amax);
            else launch_pdl(dwconv3x3_row32_kernel<2, false>, blocks, 256, 0, s, a, wl, rowsum256, amax);
          }
        } else if (a.stride == 1) {
          if (sg) launch_pdl(dwconv3x3_row_kernel<1, true>, blocks, 256, 0, s, a, wl);
          else launch_pdl(dwconv3x3_row_kernel<1, false>, blocks, 256, 0, s, a, wl);
        } else {
          if (sg) launch_pdl(dwconv3x3_row_kernel<2, true>, blocks, 256, 0, s, a, wl);
          else launch_pdl(dwconv3x3_row_kernel<2, false>, blocks, 256, 0, s, a, wl);
        }
        note_launch();
        return cudaGetLastError();
      }
    }
    uint32_t blocks = grid_for(total / 8, 256);
    if (blocks > 148u * 4u) blocks = 148u * 4u;
    launch_pdl(dwconv_nhwc8_kernel, blocks, 256, dw_smem, s, a, wt.w[a.uniform_log2k]); note_launch();
    return cudaGetLastError();
  }
  if (a.KH == 1 && a.KW == 1 && a.H == 1 && a.W == 1 && a.groups == 1 && a.C >= 64u && !a.out_nchw &&
      total < (1u << 24)) {
    launch_pdl(gemv_warp_kernel, grid_for(total * 32u, 256), 256, 0, s, a, wt); note_launch();
    return cudaGetLastError();
  }
  launch_pdl(conv_direct_kernel, grid_for(total, 256), 256, 0, s, a, wt); note_launch();
  return cudaGetLastError();
}

size_t im2col_s8_smem(const ConvArgs& a, uint32_t run_pitch) {
  return (size_t)((kIm2colRows - 1u) * a.stride + a.KH) * im2col_span_pitch(a.stride, a.C, run_pitch);
}

cudaError_t launch_im2col_s8(const ConvArgs& a, uint32_t kpad, uint32_t run_pitch, uint32_t offset, int8_t* dst,
                             uint32_t limit, cudaStream_t s) {
  const uint32_t strips = (a.OW + kIm2colPix - 1) / kIm2colPix;
  const uint32_t row_groups = (a.OH + kIm2colRows - 1) / kIm2colRows;
  const size_t smem = im2col_s8_smem(a, run_pitch);
  if (smem > 48 * 1024 || (uint64_t)a.N * row_groups * strips >= (1ull << 31) || run_pitch % 8u || kpad % 16u ||
      (offset != 0u && offset != 128u) || a.KH * run_pitch > kpad || (kIm2colRows - 1u) * a.stride + a.KH > 128u)
    return cudaErrorInvalidValue;
  launch_pdl(im2col_s8_kernel, a.N * row_groups * strips, 256, smem, s, a, kpad, run_pitch, offset, limit, dst);
  note_launch();
  return cudaGetLastError();
}

cudaError_t launch_nchw_to_nhwc(const void* src, void* dst, uint32_t N, uint32_t C, uint32_t HW,
                                uint32_t elem_bytes, uint32_t is_signed, uint32_t limit, uint32_t* err,
                                cudaStream_t s) {
  if (elem_bytes != 1) return cudaErrorInvalidValue;
  if (C % 4u == 0 && HW % 4u == 0 && !(((uintptr_t)src | (uintptr_t)dst) & 3u)) {
    dim3 grid4((HW + 127) / 128, (C + 31) / 32, N);
    launch_pdl(nchw_to_nhwc_u8x4_kernel, grid4, 256, 0, s, (const uint8_t*)src, (uint8_t*)dst, C, HW, is_signed, limit,
               err);
  } else {
    dim3 grid((HW + 31) / 32, (C + 31) / 32, N), block(32, 8);
    launch_pdl(nchw_to_nhwc_u8_kernel, grid, block, 0, s, (const uint8_t*)src, (uint8_t*)dst, C, HW, is_signed, limit,
               err);
  }
  note_launch();
  return cudaGetLastError();
}

cudaError_t launch_maxpool(const uint8_t* x, uint32_t nchw, uint32_t N, uint32_t C, uint32_t H,
                           uint32_t W, uint32_t k, uint32_t stride, uint32_t pad, uint8_t* out,
                           cudaStream_t s) {
  uint32_t OH = (H + 2 * pad - k) / stride + 1, OW = (W + 2 * pad - k) / stride + 1;
  size_t total = (size_t)N * OH * OW * C;
  if (!nchw && C % 16u == 0 && !(((uintptr_t)x | (uintptr_t)out) & 15u))
    launch_pdl(maxpool_nhwc16_kernel, grid_for(total / 16, 256), 256, 0, s, x, N, C, H, W, k, stride, pad, OH, OW, out);
  else
    launch_pdl(maxpool_kernel, grid_for(total, 256), 256, 0, s, x, nchw, N, C, H, W, k, stride, pad, OH, OW, out);
  note_launch();
  return cudaGetLastError();
}

cudaError_t launch_avgpool(const uint8_t* x, uint32_t nchw, uint32_t N, uint32_t C, uint32_t H,
                           uint32_t W, float pool_mul, int32_t qmin, int32_t qmax, uint8_t* out,
                           cudaStream_t s) {
  if (!nchw && C % 16u == 0 && !(((uintptr_t)x | (uintptr_t)out) & 15u) && (uint64_t)N * (C / 16u) < (1ull << 31)) {
    const uint32_t threads = N * (C / 16u);
    launch_pdl(avgpool_nhwc16_kernel, (threads + 127u) / 128u, 128, 0, s, x, N, C, H * W, pool_mul, qmin, qmax, out);
    note_launch();
    return cudaGetLastError();
  }
  size_t warps = (size_t)N * C;
  uint32_t blocks = (uint32_t)((warps * 32 + 255) / 256);
  launch_pdl(avgpool_kernel, blocks, 256, 0, s, x, nchw, N, C, H * W, pool_mul, qmin, qmax, out); note_launch();
  return cudaGetLastError();
}

}  // namespace psb
