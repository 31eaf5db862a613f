// Internal declarations shared by the translation units of the PSB library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "psb.h"

namespace psb {

constexpr int kMaxLevels = 7;        // k = 1, 2, 4, ..., 64
constexpr int kDigitBits = 7;        // magnitude bits per signed digit plane
constexpr int kTileN = 64;           // output channels per tensor-path tile
constexpr int kMaxPlanes = 4;

// Bits of the device error word.
constexpr uint32_t kDevErrNonFinite = 1u;
constexpr uint32_t kDevErrTimeout = 2u;
constexpr uint32_t kDevErrBadLevel = 4u;
constexpr uint32_t kDevErrRange = 8u;      // an activation byte exceeds the magnitude the caller vouched for

// Bound of every device-side wait, in SM clocks, unless the context says otherwise (about 2 s).
constexpr unsigned long long kDefaultWaitLimitCycles = 4000000000ull;

// Number of 7-bit digit planes that hold |W_k| = (k + c) * 2^(e - e_base) for
// every weight of a window of 2^exp_bits octaves: the top value is 2k * 2^span.
inline int planes_for(uint32_t exp_bits, uint32_t log2k) {
  int span = (1 << exp_bits) - 1;
  int bits = span + (int)log2k + 2;  // bit length of 2k << span
  return (bits + kDigitBits - 1) / kDigitBits;
}

// Reduction-axis block (bytes of activations per MMA stage row) for the tensor path.
inline uint32_t tensor_bk(uint32_t cg) { return cg >= 128 ? 128u : (cg >= 64 ? 64u : 32u); }
inline uint32_t round_up(uint32_t a, uint32_t b) { return (a + b - 1) / b * b; }

// Byte offset, inside one operand tile of P * kTileN rows by bk bytes, of column `kin` of row
// `row`: rows are bk bytes apart and the 16-byte chunks of a row are permuted by the row number
// the way the 32/64/128-byte swizzle modes of TMA and of the MMA descriptors do (address bits 4..
// XOR address bits 7..).  A tile copied as it is to a 1024-byte aligned shared-memory address is
// a valid K-major swizzled operand.
__host__ __device__ inline uint32_t plane_offset(uint32_t row, uint32_t kin, uint32_t bk) {
  const uint32_t lin = row * bk + kin;
  return lin ^ (((lin >> 7) & (bk / 16u - 1u)) << 4);
}

struct LevelStore {
  int32_t* wint = nullptr;  // [O][KH][KW][Cg]  signed integer filter, channels innermost
  int8_t* planes = nullptr; // [O_tiles][K blocks][P * kTileN rows][bk bytes]  signed 7-bit digits: every
                            // (channel tile, K block) operand tile is contiguous and already in the
                            // swizzled order the MMA reads from shared memory (plane_offset below)
  int planes_count = 0;
  long long* corr128 = nullptr;  // [O] 128 * sum of the filter row, refreshed by the calls that need it
};

}  // namespace psb

struct psb_weights {
  psb_wshape shape;
  psb_sample_cfg cfg;
  uint32_t d;        // in_ch_per_group * kh * kw
  uint32_t cpad;     // channels per tap in the plane layout (multiple of the K block)
  uint32_t kpad;     // kh * kw * cpad; packed K: kh * run_pitch rounded up to 16
  uint32_t run_pitch; // packed K: bytes reserved per filter row (kw * cin rounded up to 8); else kw * cpad
  uint32_t o_tiles;  // ceil(out_ch / kTileN)
  uint32_t bk;       // K block of the tensor path
  uint32_t n_cb;     // K blocks per tap (packed K: K blocks in all)
  uint32_t n_kb;     // K blocks of a filter row: kh * kw * n_cb (packed K: n_cb)
  bool has_planes;   // digit planes are produced (groups == 1)
  bool packed_k;     // few input channels: the K axis is the flat (kh, kw, ci) index, padded to 16;
                     // such a layer runs as a plain GEMM on an explicitly gathered activation matrix
  psb::LevelStore level[psb::kMaxLevels];
  int32_t* e_base = nullptr;   // [O]
  uint32_t* e_max = nullptr;   // [O] scratch of the window reduction: (call number << 8) | biased exponent
  uint32_t e_calls = 0;        // sampling calls made on this handle, modulo 2^24
  uint32_t* rowsum256 = nullptr;  // [kMaxLevels][O] row sums of |W_k| of the last sampling, in units of 256 (each
                                  // weight rounded up): the contraction derives from them whether its accumulators
                                  // fit 32 bits
  int device;
};

struct psb_ctx {
  int device;
  uint32_t* err_dev = nullptr;      // device error word
  const uint8_t* kmap = nullptr;    // borrowed
  uint32_t map_n = 0, map_oh = 0, map_ow = 0;
  uint32_t uniform_log2k = 0;
  // scratch: [0] layout conversion, [1] gathered / offset activation matrix, [2] level-sorted order of the
  // current draw-count map (control block, permutation, tile levels), [3] activation rows in that order
  void* scratch[4] = {nullptr, nullptr, nullptr, nullptr};
  size_t scratch_bytes[4] = {0, 0, 0, 0};
  // the sorted order in scratch[2] belongs to this map (pointer and dimensions); 0 rows = none
  const uint8_t* sorted_map = nullptr;
  uint32_t sorted_rows = 0;
  int32_t last_path = 0;
  int sm_count = 0;
  unsigned long long wait_limit_cycles = psb::kDefaultWaitLimitCycles;   // bound of every device-side wait
  uint32_t checks = 0;              // PSB_CHECK_* bits: extra device-side validation of the inputs
  void* encode_tiled = nullptr;     // cuTensorMapEncodeTiled
  void* encode_im2col = nullptr;    // cuTensorMapEncodeIm2col
  // measurement aid: event pairs around the contraction launches made since timing was switched on
  static constexpr int kTimedLaunches = 256;
  bool time_contraction = false;
  int timed_launches = 0;           // pairs recorded since timing was switched on (at most kTimedLaunches)
  cudaEvent_t t_begin[kTimedLaunches] = {}, t_end[kTimedLaunches] = {};
};

namespace psb {

// Everything a contraction kernel needs besides the filter.
struct ConvArgs {
  const void* x;         // NHWC activations
  uint32_t in_dtype;
  uint32_t N, C, H, W, O, KH, KW, groups, stride, pad, OH, OW;
  const uint8_t* kmap;   // [N][OH][OW] or null
  uint32_t uniform_log2k;
  uint32_t level_mask;
  // epilogue
  const float* scale;
  const float* bias;
  const int32_t* e_base;
  const void* residual;
  uint32_t residual_dtype;
  float residual_scale;
  uint32_t relu;
  float inv_step;
  int32_t qmin, qmax;
  uint32_t out_dtype;
  void* q_out;
  float* f32_out;
  int64_t* acc_out;
  uint32_t out_nchw;     // outputs (and residual) are laid out [n][o][oy][ox]
  uint32_t* err;
};

struct WintTable {
  const int32_t* w[kMaxLevels];
};
struct PlaneTable {
  const int8_t* p[kMaxLevels];
  int count[kMaxLevels];
};

// ---- fused output stage, identical in every kernel ---------------------------
// sc = scale[o] * 2^(e_base[o] - log2k) is exact; the rest is one fma, an
// optional fma for the shortcut, a max, one multiply and a round-half-even.
__device__ __forceinline__ float dequant(long long acc, float sc, float bias, bool has_res,
                                         int res_q, float res_scale, bool relu) {
  float a = __ll2float_rn(acc);
  float y = __fmaf_rn(a, sc, bias);
  if (has_res) y = __fmaf_rn((float)res_q, res_scale, y);
  if (relu) y = fmaxf(y, 0.0f);
  return y;
}

__device__ __forceinline__ int requant(float y, float inv_step, int qmin, int qmax) {
  float t = __fmul_rn(y, inv_step);
  float r = rintf(t);
  r = fmaxf(r, (float)qmin);
  r = fminf(r, (float)qmax);
  return (int)r;
}

// Exact round-to-nearest conversion of a 64-bit accumulator, |acc| < 2^55: split into a high
// part (multiple of 2^24) and a 24-bit low part, both exact in fp32; one fma rounds their sum once.
__device__ __forceinline__ float acc_to_float(long long acc) {
  const int hi = (int)(acc >> 24);
  const int lo = (int)((unsigned int)acc & 0xFFFFFFu);
  return __fmaf_rn((float)hi, 16777216.0f, (float)lo);
}

// The same for |acc| < 2^45, without the conversion unit: the parts get their float form by
// exponent arithmetic,
//   float(n) = as_float(0x4B400000 + n) - 1.5 * 2^23   for |n| < 2^22,
//   float(n) = as_float(0x4B000000 | n) - 2^23         for 0 <= n < 2^23.
__device__ __forceinline__ float acc_to_float_small(long long acc) {
  const int hi = (int)(acc >> 23);
  const unsigned int lo = (unsigned int)acc & 0x7FFFFFu;
  const float hi_f = __int_as_float(0x4B400000 + hi) - 12582912.0f;
  const float lo_f = __uint_as_float(0x4B000000u | lo) - 8388608.0f;
  return __fmaf_rn(hi_f, 8388608.0f, lo_f);
}

// Programmatic dependent launch: a kernel launched through launch_pdl may be scheduled while the
// kernel before it in the stream is still running; it must call pdl_prologue() before it touches
// global memory, which waits for the earlier grids to complete (and lets the kernel after it be
// scheduled in turn).  What is saved is the launch latency between the many short kernels of a step.
//
// Rule for such kernels: whatever an earlier kernel of the stream may have written (activations, integer
// filters and their row sums, the sorted order of a draw-count map, scratch matrices) is read with ordinary
// loads (plain, __ldca, __ldcg), never through the read-only path (__ldg, or a const __restrict__ kernel
// parameter, which the compiler turns into the same instruction).  That path promises data that does not
// change during the kernel's lifetime, which here begins before the earlier kernel has finished: the compiler
// may move such a load above the wait in pdl_prologue().  (Seen once: a gather that read the number of sorted
// tiles before the sorting kernel had written it.)
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_prologue() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
template <typename K, typename... Args>
inline cudaError_t launch_pdl(K kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}
#endif

// every kernel launch of the library is counted (process-wide), for throughput reports
void note_launch();
unsigned long long launches_so_far();

// host-side launchers (defined in the .cu files)
cudaError_t launch_sampler(const float* w_dev, psb_weights* wt, uint32_t* err_dev, cudaStream_t s);
psb_status sample_batch_create(psb_ctx* ctx, uint32_t n, const float* const* w_dev,
                               psb_weights* const* weights, psb_sample_batch** out);
psb_status sample_batch_run(psb_ctx* ctx, psb_sample_batch* b, uint64_t seed, cudaStream_t s);
void sample_batch_free(psb_sample_batch* b);
cudaError_t launch_export(const psb_weights* wt, uint32_t level, int32_t* wint_out,
                          int32_t* e_base_out, cudaStream_t s);
// rowsum256: [level][O] row sums of |W_k| / 256 kept by the sampler; amax: largest activation magnitude
cudaError_t launch_shift_add(const ConvArgs& a, const WintTable& wt, const uint32_t* rowsum256, uint32_t amax,
                             cudaStream_t s);
// gathers [M][kpad] signed bytes (x - offset; zero padding becomes -offset, K padding 0); row kh of the
// filter window occupies bytes [kh * run_pitch, kh * run_pitch + kw * c) of a matrix row
size_t im2col_s8_smem(const ConvArgs& a, uint32_t run_pitch);   // shared memory the gather kernel needs
cudaError_t launch_im2col_s8(const ConvArgs& a, uint32_t kpad, uint32_t run_pitch, uint32_t offset, int8_t* dst,
                             uint32_t limit, cudaStream_t s);
cudaError_t launch_corr128(const psb_weights* wt, uint32_t level, cudaStream_t s);
// `limit`: largest byte magnitude allowed (255 for unsigned / 128 for signed data = no check); a byte beyond
// it raises kDevErrRange in *err
cudaError_t launch_offset128(const void* src, void* dst, size_t bytes, uint32_t limit, uint32_t* err, cudaStream_t s);
cudaError_t launch_nchw_to_nhwc(const void* src, void* dst, uint32_t N, uint32_t C, uint32_t HW,
                                uint32_t elem_bytes, uint32_t is_signed, uint32_t limit, uint32_t* err,
                                cudaStream_t s);
cudaError_t launch_range_check(const void* x, size_t bytes, uint32_t is_signed, uint32_t limit, uint32_t* err,
                               cudaStream_t s);
// one tiny CTA waits, with the context's bound, on a barrier that nobody arrives at (psb_tensor.cu)
cudaError_t launch_wait_selftest(psb_ctx* ctx, cudaStream_t s);
cudaError_t launch_maxpool(const uint8_t* x, uint32_t nchw, uint32_t N, uint32_t C, uint32_t H,
                           uint32_t W, uint32_t k, uint32_t stride, uint32_t pad, uint8_t* out,
                           cudaStream_t s);
cudaError_t launch_avgpool(const uint8_t* x, uint32_t nchw, uint32_t N, uint32_t C, uint32_t H,
                           uint32_t W, float pool_mul, int32_t qmin, int32_t qmax, uint8_t* out,
                           cudaStream_t s);
// tensor path: returns PSB_ERR_UNSUPPORTED if the shape does not fit it
psb_status tensor_supported(const psb_ctx* ctx, const psb_weights* wt, const ConvArgs& a);
// sorted != null: the activation matrix is in level-sorted row order (psb_sort.cu)
struct SortedRows {
  const uint32_t* perm;       // [tiles * 128] location of every sorted row, 0xFFFFFFFF = padding
  const uint8_t* tile_mask;   // [tiles] the level of every tile as a one-bit mask (0 = unused tile)
  uint32_t tiles;             // upper bound of the tiles in use
};
psb_status launch_tensor(psb_ctx* ctx, const psb_weights* wt, const ConvArgs& a, uint32_t amax,
                         bool add_corr128, const SortedRows* sorted, cudaStream_t s);

// level-sorted rows for draw-count maps (psb_sort.cu)
size_t sort_ctl_bytes();
uint32_t sorted_tiles_bound(uint64_t M);
cudaError_t launch_level_sort(const uint8_t* kmap, uint32_t M, void* ctl, uint32_t* perm, uint8_t* tile_mask,
                              cudaStream_t s);
cudaError_t launch_gather_sorted(const ConvArgs& a, const uint32_t* perm, const void* ctl, uint32_t cpad, uint8_t* dst,
                                 cudaStream_t s);

// attention proposal (psb_attention.cu)
cudaError_t launch_entropy(const void* act, uint32_t is_signed, uint32_t locations, uint32_t C, float step,
                           float* entropy, cudaStream_t s);
cudaError_t launch_attention_maps(const float* entropy, uint32_t N, uint32_t H, uint32_t W, uint32_t lo_log2k,
                                  uint32_t hi_log2k, uint32_t n_res, const uint32_t* res, uint8_t* const* maps,
                                  float* mean_out, cudaStream_t s);

// int8 tensor-core issue-rate probe (psb_probe.cu)
psb_status int8_mma_probe(psb_ctx* ctx, uint32_t n_cols, uint32_t groups, double* mac_per_clk_per_sm,
                          double* tera_ops_per_s, cudaStream_t s);

}  // namespace psb
