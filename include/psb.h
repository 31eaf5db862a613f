/*
 * psb.h - C ABI of the B200 (sm_100a) library for progressive stochastic
 * binarization (PSB) inference layers, after "Progressive Stochastic
 * Binarization of Deep Networks" (arXiv 1904.02205).
 *
 * What a layer computes (paper Sec. 3 and 3.1):
 *   Eq. 1    y = relu(sum_i x_i * w_i)                      the layer
 *   Eq. 4-7  w -> s * 2^e * (B_p + 1),  s = sign w, e = floor(log2 |w|),
 *            p = |w| / 2^e - 1, B_p a Bernoulli(p) bit      the number system
 *   Eq. 8    w -> s * 2^e * (B_{k,p} / k + 1)               k accumulated draws
 *   Eq. 9    x * w_k = s * (sum_j x << (e + B_p^(j))) >> log2 k
 * Activations x are small integers (one byte each); every weight is replaced by
 * k random picks between its two neighbouring powers of two; the sum over the k
 * picks and over i is an exact integer; k may differ per output location
 * (Sec. 4.5).  The library keeps the integer accumulator exact (64-bit) and folds
 * 1/k and the group's base exponent into the fp32 dequantisation scale.
 *
 * Conventions
 *   - Every pointer named *_dev is DEVICE memory owned by the caller unless said
 *     otherwise; everything else is host memory.  Sizes are in elements.
 *   - `stream` is a cudaStream_t passed as void*.  All compute calls are
 *     asynchronous on that stream and do not synchronise the device, with one
 *     exception: a call that needs a larger internal scratch buffer than any
 *     call before it on this context (layout conversion, gathered matrices,
 *     the sorted order of a draw-count map) frees and allocates device
 *     memory, which waits for the device; after one pass over a network's
 *     shapes no call grows anything.  Otherwise only psb_create, psb_destroy,
 *     the first psb_sample_weights for a handle, psb_weights_free and
 *     psb_device_status may block.
 *   - Every function returns a psb_status: 0 on success, negative on error.
 *     Arguments are validated on the host before anything is launched; a call
 *     that returns an error has launched nothing.  There is no CPU fallback: if
 *     no CUDA device is usable, psb_create fails.
 *   - Filters are given as fp32 in canonical [out_ch][in_ch/groups][kh][kw]
 *     order.  The canonical linear index of a weight in that order keys its
 *     random stream, so results do not depend on any internal tiling.
 *   - Activation tensors are [n][c][h][w] (PSB_LAYOUT_NCHW) or [n][h][w][c]
 *     (PSB_LAYOUT_NHWC), one byte per element.  NHWC is the native layout; NCHW
 *     inputs and outputs are converted inside the call.
 */
#ifndef PSB_H_
#define PSB_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t psb_status;

enum {
  PSB_OK = 0,
  PSB_ERR_INVALID_ARG = -1,      /* null / misaligned pointer, zero dimension, shape mismatch   */
  PSB_ERR_BAD_K = -2,            /* level not sampled, or k not a power of two in 1..64          */
  PSB_ERR_UNSUPPORTED = -3,      /* valid request that no kernel of this library covers          */
  PSB_ERR_ALLOC = -4,            /* device or host allocation failed                             */
  PSB_ERR_CUDA = -5,             /* a CUDA runtime / driver call failed                          */
  PSB_ERR_TIMEOUT = -6,          /* a bounded device-side wait ran out (reported by the device)  */
  PSB_ERR_NONFINITE_WEIGHT = -7, /* a filter holds Inf or NaN (reported by the device)           */
  PSB_ERR_RANGE = -8             /* an activation exceeds the in_max the caller vouched for
                                    (reported by the device)                                     */
};

enum { PSB_LAYOUT_NCHW = 0, PSB_LAYOUT_NHWC = 1 };
enum { PSB_DT_U8 = 0, PSB_DT_S8 = 1 };

/* Which contraction kernel a conv / gemm call uses. */
enum {
  PSB_PATH_AUTO = 0,       /* library chooses                                                     */
  PSB_PATH_SHIFT_ADD = 1,  /* CUDA-core integer path (depthwise, tiny batch, few input channels)  */
  PSB_PATH_TENSOR = 2      /* tcgen05 int8 MMA on signed digit planes, accumulators in TMEM       */
};

typedef struct psb_ctx psb_ctx;         /* per-device state: error word, scratch, current draw-count map */
typedef struct psb_weights psb_weights; /* library-owned sampled integer filters of one layer            */

/* Create / destroy the per-device context.  `device` is a CUDA ordinal.  The
 * context owns a small device error word and scratch buffers that grow on
 * demand (growth allocates, so it blocks).  Not thread-safe: use one context per
 * host thread. */
psb_status psb_create(psb_ctx** ctx, int device);
psb_status psb_destroy(psb_ctx* ctx);

/* Static, human-readable name of a status code. */
const char* psb_status_string(psb_status st);

/* Synchronise `stream`, then return and clear the sticky device-side error
 * (PSB_ERR_TIMEOUT, PSB_ERR_NONFINITE_WEIGHT, PSB_ERR_BAD_K from a draw-count
 * map naming a level that was not sampled, PSB_ERR_RANGE), or PSB_OK. */
psb_status psb_device_status(psb_ctx* ctx, void* stream);

/* Extra device-side validation, sticky until changed (no counterpart in the paper).
 *   PSB_CHECK_RANGE  every conv / gemm call verifies that no input byte exceeds its in_max
 *                    (see psb_conv_desc) and raises PSB_ERR_RANGE through psb_device_status
 *                    otherwise.  Calls that convert or gather their input (NCHW tensors, filters
 *                    with few input channels, unsigned bytes above 127) verify it in that pass
 *                    whether the flag is set or not; the flag adds one read-only pass over the
 *                    input to the calls that hand the tensor straight to the copy engine. */
enum { PSB_CHECK_RANGE = 1 };
psb_status psb_set_checks(psb_ctx* ctx, uint32_t flags);

/* Every wait inside a kernel (on a copy, on the tensor pipe, on another warp) is bounded; a wait
 * that runs out makes the kernel return and raises PSB_ERR_TIMEOUT (see psb_device_status); the
 * context stays usable.  psb_set_wait_limit sets the bound in SM clocks for the following
 * launches of this context (0 restores the default, 4e9 clocks, about 2 s).
 * psb_wait_selftest launches one small thread block that waits, with that bound, on a barrier
 * nobody arrives at: the one way to see the time-out path work without a fault.  Set a short
 * bound (1e5 clocks) before calling it. */
psb_status psb_set_wait_limit(psb_ctx* ctx, uint64_t sm_clocks);
psb_status psb_wait_selftest(psb_ctx* ctx, void* stream);

/* Shape of a filter in canonical order [out_ch][in_ch_per_group][kh][kw]. */
typedef struct {
  uint32_t out_ch, in_ch_per_group, kh, kw, groups;
} psb_wshape;

/* How to sample a filter.
 *   seed, layer_id  key of the random stream: draw j of the weight with canonical
 *                   index i is word (j mod 4) of Philox4x32-10 with counter
 *                   (j / 4, layer_id, lo32(i), hi32(i)) and key (lo32(seed),
 *                   hi32(seed)); the bit is 1 ("upper shift", Eq. 4) when that
 *                   word is below p * 2^32.
 *   level_mask      bit l set => produce the filter for k = 2^l draws, l = 0..6.
 *                   All levels share draws: level k uses draws 0..k-1
 *                   (progressive refinement, Sec. 1.1).
 *   exp_bits        1..4: exponents are kept in a window of 2^exp_bits octaves
 *                   below the group's largest exponent; smaller weights, zeros
 *                   and sub-normals contribute nothing (Sec. 4.4: 4-bit
 *                   exponents suffice).  0 selects 4.
 *   norm            0: one exponent window per layer; 1: one per output channel.
 *   underflow       0: weights below the window contribute nothing.  1: a weight below the
 *                   window, |w| < 2^e_base, is replaced per draw by s * 2^e_base * B_q with
 *                   q = |w| / 2^e_base (the plain Bernoulli gate of Sec. 3.1, "Stochastic
 *                   multiplication"): W_k = s * c_k with c_k ~ Binomial(k, q), unbiased, which is
 *                   what makes windows of fewer octaves (exp_bits 3, 2: fewer digit planes)
 *                   usable.  Draw j uses the same random word as above, compared with
 *                   floor(q * 2^32).
 *   prob_bits       0: probabilities keep their 23 bits.  b = 1..8 (Sec. 4.4): p is rounded to the
 *                   nearest point of the grid {0, 1/2^b, .., 1 - 1/2^b}; a p that rounds to 1
 *                   becomes p = 0 at the next exponent (before the window is taken); the
 *                   comparator has b bits and one random word serves n = floor(32 / b) draws:
 *                   draw j compares bits [f*b, f*b + b), f = j mod n, of word (j / n) mod 4 of
 *                   Philox4x32-10 with counter (j / (4n), layer_id, lo32(i), hi32(i)) with p * 2^b.
 *                   With underflow = 1, q is rounded to the same grid (q = 1: the weight 2^e_base).
 *   deterministic   1 (needs prob_bits > 0): no draws; the upper shift is taken in
 *                   round(p * k) of the k cases (Sec. 4.4, the variant for bounded precision).
 *   reserved        0. */
typedef struct {
  uint64_t seed;
  uint32_t layer_id;
  uint32_t level_mask;
  uint32_t exp_bits;
  uint32_t norm;
  uint32_t underflow;
  uint32_t prob_bits;
  uint32_t deterministic;
  uint32_t reserved;
} psb_sample_cfg;

/* Draw the random bits and build the integer filters (Eq. 8 scaled by
 * k / 2^e_base):  W_k[i] = s_i * (k + c_k[i]) * 2^(e_i - e_base),  c_k = number of
 * upper draws among the first k.  Nothing random is stored: the bits live in
 * registers only.
 *   w_dev     fp32 filter, canonical order, device memory, 4-byte aligned.
 *   *weights  NULL: a handle is created (allocates, blocks).  Non-NULL: must
 *             come from an earlier call with the same shape, level_mask,
 *             exp_bits; it is re-sampled in place without allocating.
 * A filter with Inf/NaN sets the device error word (see psb_device_status). */
psb_status psb_sample_weights(psb_ctx* ctx, const float* w_dev, const psb_wshape* shape,
                              const psb_sample_cfg* cfg, psb_weights** weights, void* stream);

/* Test hook: copy the level-2^log2k integer filter (int32, canonical order,
 * out_ch*in_ch_per_group*kh*kw elements) and e_base (int32 [out_ch]) to caller
 * device buffers.  Either pointer may be NULL. */
psb_status psb_weights_export(psb_ctx* ctx, const psb_weights* weights, uint32_t log2k,
                              int32_t* wint_dev, int32_t* e_base_dev, void* stream);

psb_status psb_weights_free(psb_ctx* ctx, psb_weights* weights);

/* Localised accuracy control (Sec. 4.5): the number of draws used by output
 * location (n, oy, ox) of the following conv / gemm calls.
 *   log2k_dev      u8 [n][oh][ow] holding log2 k per location, or NULL for a
 *                  uniform k = 2^uniform_log2k.  The pointer is borrowed: it must
 *                  stay valid until the calls that use it have finished.  Its
 *                  dimensions must equal the output dimensions of those calls.
 * The setting is sticky until changed.  A new context starts uniform, k = 1. */
psb_status psb_set_sample_map(psb_ctx* ctx, const uint8_t* log2k_dev, uint32_t n, uint32_t oh,
                              uint32_t ow, uint32_t uniform_log2k);

/* Fused output stage (Eq. 1's relu, the folded batch-norm a*y+b of Sec. 3, and
 * the fixed-point intermediates of Sec. 4.1), per output element:
 *   a  = (float) acc                              round to nearest even
 *   y  = fma(a, scale[o] * 2^(e_base[o] - log2 k), bias[o])
 *   y  = fma((float) residual, residual_scale, y)  if residual_dev != NULL
 *   y  = max(y, 0)                                 if relu
 *   q  = clamp(rint(y * inv_step), qmin, qmax)     ties to even
 * Outputs, each optional (NULL) but at least one present, all in the layout of
 * the call: q_out_dev (one byte, out_dtype), f32_out_dev (y), acc_out_dev (the
 * raw 64-bit accumulator, a test hook).  residual_dev has the output's shape and
 * layout, one byte per element of residual_dtype. */
typedef struct {
  const float* scale_dev;    /* [out_ch] */
  const float* bias_dev;     /* [out_ch] */
  const void* residual_dev;  /* nullable */
  float residual_scale;
  uint32_t residual_dtype;
  uint32_t relu;
  float inv_step;
  int32_t qmin, qmax;
  uint32_t out_dtype;        /* PSB_DT_U8 | PSB_DT_S8 */
  void* q_out_dev;           /* nullable */
  float* f32_out_dev;        /* nullable */
  int64_t* acc_out_dev;      /* nullable */
} psb_epilogue;

/* 2-D convolution, zero padding, square stride.  Output size
 * oh = (h + 2*pad - kh) / stride + 1 (same for ow).
 *   in_max   largest activation magnitude the caller guarantees (e.g. 15 for
 *            4-bit data); 0 means "full range of in_dtype".  The tensor path
 *            feeds activations to the MMA as signed bytes.  Unsigned data
 *            above 127 reaches it as x - 128 with 128 * sum(W) added back
 *            (filters gathered explicitly, or any filter without padding);
 *            with padding it takes the shift-add path.  A smaller in_max also
 *            lets the output stage recombine the digit planes in 32 bits.
 *            It is a promise the kernels rely on: a byte beyond it gives a
 *            wrong result.  Passes that read every byte anyway verify it; the
 *            other routes verify it on request (psb_set_checks); a violation
 *            is reported as PSB_ERR_RANGE by psb_device_status.
 *   path    PSB_PATH_AUTO, or force one path (PSB_ERR_UNSUPPORTED if the forced
 *            path cannot run this shape). */
typedef struct {
  uint32_t layout;
  uint32_t in_dtype;
  uint32_t in_max;
  uint32_t n, c, h, w;
  uint32_t stride, pad;
  uint32_t path;
  psb_epilogue ep;
} psb_conv_desc;

psb_status psb_conv2d(psb_ctx* ctx, const psb_weights* weights, const void* x_dev,
                      const psb_conv_desc* desc, void* stream);

/* Fully connected layer: x [batch][in_features] (one byte each), filter shape
 * [out][in][1][1], outputs [batch][out].  The draw-count map, if set, is
 * [batch][1][1]. */
typedef struct {
  uint32_t in_dtype;
  uint32_t in_max;
  uint32_t batch, in_features;
  uint32_t path;
  psb_epilogue ep;
} psb_gemm_desc;

psb_status psb_gemm(psb_ctx* ctx, const psb_weights* weights, const void* x_dev,
                    const psb_gemm_desc* desc, void* stream);

/* Which path the last successful psb_conv2d / psb_gemm call on this context took
 * (PSB_PATH_SHIFT_ADD or PSB_PATH_TENSOR); 0 before any call. */
int32_t psb_last_path(const psb_ctx* ctx);

/* Number of GPU kernels this library has launched in this process so far (all
 * contexts, all entry points).  A reporting aid: throughput figures state how
 * many launches a timed region took.  Never fails. */
uint64_t psb_launch_count(void);

/* Measurement aid, no counterpart in the paper: device time of the tensor-core
 * contraction kernel inside a larger step.  With `enable` != 0 every launch of
 * that kernel by this context is bracketed by a pair of CUDA events on its
 * stream (which also keeps it from starting under its predecessor's tail, so a
 * step runs a little slower while this is on); psb_contraction_time waits for
 * those launches and returns the sum of their durations in milliseconds, over
 * the launches made since timing was last switched on (switching it on again
 * starts a new sum; at most 256 launches are kept, later ones go untimed).
 * PSB_ERR_INVALID_ARG for null arguments or when no launch has been timed yet,
 * PSB_ERR_CUDA if the events cannot be created or read. */
psb_status psb_contraction_timing(psb_ctx* ctx, uint32_t enable);
psb_status psb_contraction_time(psb_ctx* ctx, float* milliseconds);
/* The same launches one by one, in launch order: *count receives how many have been timed since timing
 * was switched on, milliseconds[0 .. min(*count, capacity)) their durations. */
psb_status psb_contraction_times(psb_ctx* ctx, float* milliseconds, uint32_t capacity, uint32_t* count);

/* Measurement aid, no counterpart in the paper: the ceiling of the dense path.
 * Every SM issues `groups` groups of four back-to-back tcgen05.mma kind::i8
 * instructions (M = 128, N = n_cols, K = 32, s8 x s8 -> s32 in TMEM) on zero
 * operand tiles resident in shared memory; nothing is copied or stored.
 *   n_cols: 16..256, multiple of 16.  groups: 1..2^20.
 *   mac_per_clk_per_sm (host, out): int8 multiply-accumulates per SM clock of
 *     the slowest SM, from the SM cycle counter.
 *   tera_ops_per_s (host, out): 2 * MACs of all SMs / elapsed time of the
 *     launch (CUDA events on `stream`), in 10^12 operations per second.
 * Synchronises `stream` and allocates one small device buffer for the duration
 * of the call.  A wait that runs out sets the device error word (see
 * psb_device_status).  Errors: PSB_ERR_INVALID_ARG, PSB_ERR_ALLOC, PSB_ERR_CUDA. */
psb_status psb_int8_mma_probe(psb_ctx* ctx, uint32_t n_cols, uint32_t groups, double* mac_per_clk_per_sm,
                              double* tera_ops_per_s, void* stream);

/* Glue between layers (supplement, "ReLU, Batch-Norm, and Pooling"): max-pooling
 * is comparators only; the 1/(h*w) of average pooling is folded into one
 * re-quantisation factor.
 * psb_maxpool2d_u8: u8 activations, window k, given stride and padding; padded
 *   positions never win.  Output [n][oh][ow][c] / [n][c][oh][ow].
 * psb_global_avgpool_u8: integer sum over h*w, then
 *   q = clamp(rint((float) sum * pool_mul), qmin, qmax), output u8 [n][c]. */
psb_status psb_maxpool2d_u8(psb_ctx* ctx, const uint8_t* x_dev, uint32_t layout, uint32_t n,
                            uint32_t c, uint32_t h, uint32_t w, uint32_t k, uint32_t stride,
                            uint32_t pad, uint8_t* out_dev, void* stream);
psb_status psb_global_avgpool_u8(psb_ctx* ctx, const uint8_t* x_dev, uint32_t layout, uint32_t n,
                                 uint32_t c, uint32_t h, uint32_t w, float pool_mul, int32_t qmin,
                                 int32_t qmax, uint8_t* out_dev, void* stream);

/* Attention proposal (Sec. 4.5, "Computational Attention"): from a cheap pass with few draws everywhere,
 * find the regions that deserve more.
 * psb_attention_entropy: pixelwise entropy of the softmax over the channels of a layer's activations
 *   a = code * step (the paper uses the last convolutional layer):
 *   h[n][y][x] = - sum_c softmax(a[n][y][x][.])_c * log softmax(a[n][y][x][.])_c,  fp32.
 *   act_dev: channels-last codes [n][h][w][c] of in_dtype; entropy_dev: float [n][h][w].
 * psb_attention_maps: hard threshold at the mean entropy of each image; locations above it get
 *   hi_log2k, the others lo_log2k.  The mask serves every layer resolution by nearest-neighbour
 *   sampling: location (y, x) of map i reads the mask at (floor(y * h / res[i]), floor(x * w / res[i])).
 *   res (host): n_res <= 8 resolutions; maps_dev (host array of device pointers): u8 [n][res[i]][res[i]],
 *   ready for psb_set_sample_map; mean_dev: float [n], the thresholds, may be NULL. */
psb_status psb_attention_entropy(psb_ctx* ctx, const void* act_dev, uint32_t in_dtype, uint32_t n, uint32_t h,
                                 uint32_t w, uint32_t c, float step, float* entropy_dev, void* stream);
psb_status psb_attention_maps(psb_ctx* ctx, const float* entropy_dev, uint32_t n, uint32_t h, uint32_t w,
                              uint32_t lo_log2k, uint32_t hi_log2k, uint32_t n_res, const uint32_t* res,
                              uint8_t* const* maps_dev, float* mean_dev, void* stream);

/* Whole networks with few host calls.
 *
 * psb_sample_batch_*: re-sample many layers at once.  The handles must exist already (created
 * by psb_sample_weights, which also fixes each layer's layer_id, level_mask, exp_bits and norm);
 * w_dev[i] is the fp32 filter of weights[i].  psb_sample_batch_run draws every layer under one
 * new `seed` in two kernel launches and gives exactly the filters that psb_sample_weights would
 * give layer by layer with that seed.  Create and free allocate / block; run does not.  The
 * filters, handles and the batch must stay alive while a run is in flight.
 *
 * psb_run: executes a list of layer operations in order on `stream`, each exactly as the
 * corresponding single call would (psb_set_sample_map with the op's draw-count fields, then
 * psb_conv2d / psb_gemm / psb_maxpool2d_u8 / psb_global_avgpool_u8).  It stops at the first
 * error and returns it; operations before it stay launched. */
typedef struct psb_sample_batch psb_sample_batch;
psb_status psb_sample_batch_create(psb_ctx* ctx, uint32_t n, const float* const* w_dev,
                                   psb_weights* const* weights, psb_sample_batch** batch);
psb_status psb_sample_batch_run(psb_ctx* ctx, psb_sample_batch* batch, uint64_t seed, void* stream);
psb_status psb_sample_batch_free(psb_ctx* ctx, psb_sample_batch* batch);

enum { PSB_OP_CONV2D = 0, PSB_OP_GEMM = 1, PSB_OP_MAXPOOL = 2, PSB_OP_AVGPOOL = 3 };
typedef struct {
  uint32_t kind;
  const psb_weights* weights;   /* conv2d, gemm */
  const void* x_dev;            /* input activations of the op */
  const uint8_t* map_dev;       /* draw counts per output location, or NULL for uniform_log2k */
  uint32_t map_n, map_oh, map_ow, uniform_log2k;
  psb_conv_desc conv;           /* conv2d; pooling reads layout, n, c, h, w, stride, pad from it */
  psb_gemm_desc gemm;           /* gemm */
  uint32_t pool_k;              /* max-pool window */
  float pool_mul;               /* average pool: see psb_global_avgpool_u8 */
  int32_t pool_qmin, pool_qmax;
  uint8_t* pool_out_dev;
} psb_op;
psb_status psb_run(psb_ctx* ctx, const psb_op* ops, uint32_t n_ops, void* stream);

/* Sampling of one level without any allocation.  (The paper has no counterpart:
 * this entry point exists for hosts, not for the method.)
 *
 * psb_sample_weights creates a handle with cudaMalloc on first use.  Some callers
 * cannot do that at the moment they need fresh draws: a real-time loop that must
 * never block on the device allocator, a thread working while another part of the
 * process captures a CUDA graph (allocation is illegal during capture), or a
 * process whose device memory was fully handed out at start-up.  This variant
 * allocates nothing, on the device or through any library: its only scratch, the
 * per-output-channel exponent maxima of the window reduction, lives in a fixed
 * array inside the library's device image (PSB_STATIC_MAX_OUT_CH words + 256 B,
 * held by every GPU that loads the library until the process exits).
 *
 *   w_dev, shape, cfg   as for psb_sample_weights; cfg->level_mask is ignored; the options underflow,
 *                       prob_bits and deterministic must be 0 (PSB_ERR_UNSUPPORTED otherwise).
 *   log2k               the one level to produce, k = 2^log2k, 0..6.
 *   wint_out_dev        int32, canonical [out_ch][in_ch_per_group][kh][kw] order,
 *                       caller-owned device memory; receives the same integers that
 *                       psb_weights_export returns for that level.  May be NULL.
 *   e_base_out_dev      int32 [out_ch], caller-owned; may be NULL (not both).
 * Works on the current device, asynchronously on `stream`.
 * Errors: PSB_ERR_UNSUPPORTED if shape->out_ch > PSB_STATIC_MAX_OUT_CH (the fixed
 * array cannot hold the reduction) or the filter exceeds the sizes
 * psb_sample_weights accepts; PSB_ERR_INVALID_ARG / PSB_ERR_BAD_K as usual.  Inf/NaN
 * weights are not reported here; they contribute nothing.
 * The first call on each device looks up the array's device address (a runtime
 * query, no allocation); make that first call outside any stream capture.
 * All calls on a device share the one array, which still holds the previous
 * call's contents; every call clears the part it uses on `stream` first.  Two
 * calls that can overlap on the GPU (different streams, no dependency) race on
 * it: serialise them. */
#define PSB_STATIC_MAX_OUT_CH 4096
psb_status psb_sample_level_static(const float* w_dev, const psb_wshape* shape,
                                   const psb_sample_cfg* cfg, uint32_t log2k, int32_t* wint_out_dev,
                                   int32_t* e_base_out_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PSB_H_ */
