// Host side of the C ABI declared in psb.h: argument validation, handle
// management, path selection and kernel launches.  No arithmetic of the method
// happens on the host.
#include <new>

#include "psb_common.cuh"

#include <atomic>

using namespace psb;

namespace {

bool pow2_level_ok(uint32_t log2k) { return log2k < (uint32_t)kMaxLevels; }

psb_status ensure_scratch(psb_ctx* ctx, int slot, size_t bytes) {
  if (ctx->scratch_bytes[slot] >= bytes) return PSB_OK;
  if (ctx->scratch[slot]) cudaFree(ctx->scratch[slot]);
  ctx->scratch[slot] = nullptr;
  ctx->scratch_bytes[slot] = 0;
  size_t want = bytes + bytes / 4;
  if (cudaMalloc(&ctx->scratch[slot], want) != cudaSuccess) {
    cudaGetLastError();
    return PSB_ERR_ALLOC;
  }
  ctx->scratch_bytes[slot] = want;
  return PSB_OK;
}

void free_weights_storage(psb_weights* w) {
  for (int l = 0; l < kMaxLevels; ++l) {
    if (w->level[l].wint) cudaFree(w->level[l].wint);
    if (w->level[l].planes) cudaFree(w->level[l].planes);
    if (w->level[l].corr128) cudaFree(w->level[l].corr128);
    w->level[l] = LevelStore();
  }
  if (w->e_base) cudaFree(w->e_base);
  if (w->e_max) cudaFree(w->e_max);
  if (w->rowsum256) cudaFree(w->rowsum256);
  w->e_base = nullptr;
  w->e_max = nullptr;
  w->rowsum256 = nullptr;
}

psb_status check_epilogue(const psb_epilogue& ep) {
  if (!ep.scale_dev || !ep.bias_dev) return PSB_ERR_INVALID_ARG;
  if (!ep.q_out_dev && !ep.f32_out_dev && !ep.acc_out_dev) return PSB_ERR_INVALID_ARG;
  if (ep.out_dtype != PSB_DT_U8 && ep.out_dtype != PSB_DT_S8) return PSB_ERR_INVALID_ARG;
  if (ep.residual_dev && ep.residual_dtype != PSB_DT_U8 && ep.residual_dtype != PSB_DT_S8)
    return PSB_ERR_INVALID_ARG;
  if (ep.qmin > ep.qmax) return PSB_ERR_INVALID_ARG;
  if (ep.q_out_dev) {
    int lo = ep.out_dtype == PSB_DT_U8 ? 0 : -128, hi = ep.out_dtype == PSB_DT_U8 ? 255 : 127;
    if (ep.qmin < lo || ep.qmax > hi) return PSB_ERR_INVALID_ARG;
  }
  if (((uintptr_t)ep.scale_dev | (uintptr_t)ep.bias_dev | (uintptr_t)ep.f32_out_dev) & 3u)
    return PSB_ERR_INVALID_ARG;
  if ((uintptr_t)ep.acc_out_dev & 7u) return PSB_ERR_INVALID_ARG;
  return PSB_OK;
}

// Shared body of psb_conv2d and psb_gemm.
psb_status run_layer(psb_ctx* ctx, const psb_weights* wt, const void* x_dev, uint32_t layout,
                     uint32_t in_dtype, uint32_t in_max, uint32_t n, uint32_t c, uint32_t h,
                     uint32_t w, uint32_t stride, uint32_t pad, uint32_t path,
                     const psb_epilogue& ep, void* stream) {
  if (!ctx || !wt || !x_dev) return PSB_ERR_INVALID_ARG;
  if (wt->device != ctx->device) return PSB_ERR_INVALID_ARG;
  if (layout != PSB_LAYOUT_NCHW && layout != PSB_LAYOUT_NHWC) return PSB_ERR_INVALID_ARG;
  if (in_dtype != PSB_DT_U8 && in_dtype != PSB_DT_S8) return PSB_ERR_INVALID_ARG;
  if (path > PSB_PATH_TENSOR) return PSB_ERR_INVALID_ARG;
  const psb_wshape& sh = wt->shape;
  if (n == 0 || c == 0 || h == 0 || w == 0 || stride == 0) return PSB_ERR_INVALID_ARG;
  if (c != sh.in_ch_per_group * sh.groups) return PSB_ERR_INVALID_ARG;
  if (h + 2 * pad < sh.kh || w + 2 * pad < sh.kw) return PSB_ERR_INVALID_ARG;
  if (pad > 0 && (pad >= sh.kh || pad >= sh.kw)) return PSB_ERR_INVALID_ARG;
  psb_status st = check_epilogue(ep);
  if (st != PSB_OK) return st;
  const uint32_t oh = (h + 2 * pad - sh.kh) / stride + 1, ow = (w + 2 * pad - sh.kw) / stride + 1;
  if ((uint64_t)n * oh * ow >= (1ull << 31)) return PSB_ERR_UNSUPPORTED;
  if (ctx->kmap) {
    if (ctx->map_n != n || ctx->map_oh != oh || ctx->map_ow != ow) return PSB_ERR_INVALID_ARG;
  } else {
    if (!pow2_level_ok(ctx->uniform_log2k) || !((wt->cfg.level_mask >> ctx->uniform_log2k) & 1u))
      return PSB_ERR_BAD_K;
  }
  cudaStream_t s = (cudaStream_t)stream;

  ConvArgs a;
  a.x = x_dev;
  a.in_dtype = in_dtype;
  a.N = n; a.C = c; a.H = h; a.W = w;
  a.O = sh.out_ch; a.KH = sh.kh; a.KW = sh.kw; a.groups = sh.groups;
  a.stride = stride; a.pad = pad; a.OH = oh; a.OW = ow;
  a.kmap = ctx->kmap;
  a.uniform_log2k = ctx->uniform_log2k;
  a.level_mask = wt->cfg.level_mask;
  a.scale = ep.scale_dev; a.bias = ep.bias_dev; a.e_base = wt->e_base;
  a.residual = ep.residual_dev; a.residual_dtype = ep.residual_dtype;
  a.residual_scale = ep.residual_scale;
  a.relu = ep.relu; a.inv_step = ep.inv_step; a.qmin = ep.qmin; a.qmax = ep.qmax;
  a.out_dtype = ep.out_dtype;
  a.q_out = ep.q_out_dev; a.f32_out = ep.f32_out_dev; a.acc_out = ep.acc_out_dev;
  a.err = ctx->err_dev;
  // NCHW differs from NHWC only when both the channel and the spatial extent exceed one.
  const bool in_conv = layout == PSB_LAYOUT_NCHW && c > 1 && (uint64_t)h * w > 1;
  a.out_nchw = (layout == PSB_LAYOUT_NCHW && sh.out_ch > 1 && (uint64_t)oh * ow > 1) ? 1u : 0u;

  // largest activation magnitude the caller vouches for
  uint32_t amax = in_max ? in_max : (in_dtype == PSB_DT_U8 ? 255u : 128u);
  const uint64_t M = (uint64_t)n * oh * ow;
  bool tensor_ok = false, range_checked = false;
  if (path != PSB_PATH_SHIFT_ADD) {
    // the MMA takes signed bytes: unsigned data above 127 qualifies only where the activation
    // matrix is gathered explicitly (packed-K filters), which stores x - 128
    // the MMA takes signed bytes.  Unsigned data above 127 still qualifies where it can be fed as
    // x - 128 and corrected by 128 * sum(W): packed-K filters (the gathered matrix is built with
    // the offset) and layers without padding (one pass flips the top bit of the whole input)
    const bool needs_offset = in_dtype == PSB_DT_U8 && amax > 127u;
    tensor_ok = (!needs_offset || wt->packed_k || pad == 0) && tensor_supported(ctx, wt, a) == PSB_OK;
    if (path == PSB_PATH_TENSOR && !tensor_ok) return PSB_ERR_UNSUPPORTED;
    if (path == PSB_PATH_AUTO && M < (wt->packed_k ? 128u : 32u)) tensor_ok = false;
  }

  if (in_conv) {
    size_t bytes = (size_t)n * c * h * w;
    st = ensure_scratch(ctx, 0, bytes);
    if (st != PSB_OK) return st;
    if (launch_nchw_to_nhwc(x_dev, ctx->scratch[0], n, c, h * w, 1, in_dtype == PSB_DT_S8, amax, ctx->err_dev, s) !=
        cudaSuccess)
      return PSB_ERR_CUDA;
    a.x = ctx->scratch[0];
    range_checked = true;     // the conversion pass has looked at every byte
  }
  // in_max is a promise the kernels rely on (bytes above 127 would read as negative on the tensor path):
  // passes that touch every input byte anyway verify it for free; the routes that hand the tensor
  // straight to the copy engine verify it only on request (PSB_CHECK_RANGE)
  const uint32_t no_limit = in_dtype == PSB_DT_U8 ? 255u : 128u;
  const bool gathers = tensor_ok && (wt->packed_k || (in_dtype == PSB_DT_U8 && amax > 127u));
  if (!range_checked && !gathers && (ctx->checks & PSB_CHECK_RANGE) && amax < no_limit) {
    if (launch_range_check(a.x, (size_t)n * c * h * w, in_dtype == PSB_DT_S8, amax, ctx->err_dev, s) != cudaSuccess)
      return PSB_ERR_CUDA;
    range_checked = true;
  }
  const uint32_t gather_limit = range_checked ? no_limit : amax;

  if (tensor_ok) {
    bool add_corr = false;
    if (wt->packed_k) {
      // gather the activation matrix [M][kpad] once, then run the layer as a plain GEMM
      st = ensure_scratch(ctx, 1, (size_t)M * wt->kpad);
      if (st != PSB_OK) return st;
      const uint32_t offset = in_dtype == PSB_DT_U8 ? 128u : 0u;
      if (launch_im2col_s8(a, wt->kpad, wt->run_pitch, offset, (int8_t*)ctx->scratch[1], gather_limit, s) != cudaSuccess)
        return PSB_ERR_CUDA;
      a.x = ctx->scratch[1];
      a.in_dtype = PSB_DT_S8;
      a.C = wt->kpad;
      a.H = oh; a.W = ow;
      a.KH = 1; a.KW = 1; a.stride = 1; a.pad = 0;
      add_corr = offset != 0;
      amax = 128;
    } else if (in_dtype == PSB_DT_U8 && amax > 127u) {
      const size_t bytes = (size_t)n * c * h * w;   // a multiple of 16: c is
      st = ensure_scratch(ctx, 1, bytes);
      if (st != PSB_OK) return st;
      if (launch_offset128(a.x, ctx->scratch[1], bytes, gather_limit, ctx->err_dev, s) != cudaSuccess) return PSB_ERR_CUDA;
      a.x = ctx->scratch[1];
      a.in_dtype = PSB_DT_S8;
      add_corr = true;
      amax = 128;
    }
    if (add_corr) {
      // 128 * (row sums of the integer filter) for every level this call may use
      for (uint32_t l = 0; l < (uint32_t)kMaxLevels; ++l)
        if (wt->level[l].corr128 && (ctx->kmap || l == ctx->uniform_log2k))
          if (launch_corr128(wt, l, s) != cudaSuccess) return PSB_ERR_CUDA;
    }
    SortedRows sorted;
    if (a.kmap) {
      // per-location draw counts: sort the locations by level (once per map), gather the activation rows in
      // that order, contract the matrix with one level per tile, scatter the rows back in the output stage
      const uint32_t tiles = sorted_tiles_bound(M);
      const size_t ctl_bytes = (sort_ctl_bytes() + 255u) & ~(size_t)255u;
      const size_t perm_bytes = (size_t)tiles * 128u * sizeof(uint32_t);
      if (ctx->scratch_bytes[2] < ctl_bytes + perm_bytes + tiles) ctx->sorted_rows = 0;    // the buffer moves
      st = ensure_scratch(ctx, 2, ctl_bytes + perm_bytes + tiles);
      if (st != PSB_OK) return st;
      uint8_t* base = (uint8_t*)ctx->scratch[2];
      uint32_t* perm = (uint32_t*)(base + ctl_bytes);
      uint8_t* tile_mask = base + ctl_bytes + perm_bytes;
      if (ctx->sorted_map != a.kmap || ctx->sorted_rows != (uint32_t)M) {
        if (launch_level_sort(a.kmap, (uint32_t)M, base, perm, tile_mask, s) != cudaSuccess) return PSB_ERR_CUDA;
        ctx->sorted_map = a.kmap;
        ctx->sorted_rows = (uint32_t)M;
      }
      // the matrix: K index (kh * KW + kw) * cpad + ci, cpad = channel blocks of the filter's plane layout
      const uint32_t cpad = wt->packed_k ? wt->n_cb * wt->bk : ((a.C + wt->bk - 1) / wt->bk) * wt->bk;
      const size_t row_bytes = (size_t)a.KH * a.KW * cpad;
      st = ensure_scratch(ctx, 3, (size_t)tiles * 128u * row_bytes);
      if (st != PSB_OK) return st;
      if (launch_gather_sorted(a, perm, base, cpad, (uint8_t*)ctx->scratch[3], s) != cudaSuccess) return PSB_ERR_CUDA;
      a.x = ctx->scratch[3];
      a.C = (uint32_t)row_bytes;
      a.H = oh; a.W = ow;
      a.KH = 1; a.KW = 1; a.stride = 1; a.pad = 0;
      sorted.perm = perm;
      sorted.tile_mask = tile_mask;
      sorted.tiles = tiles;
    }
    st = launch_tensor(ctx, wt, a, amax, add_corr, a.kmap ? &sorted : nullptr, s);
    if (st != PSB_OK) return st;
    ctx->last_path = PSB_PATH_TENSOR;
    return PSB_OK;
  }
  WintTable tab;
  for (int l = 0; l < kMaxLevels; ++l) tab.w[l] = wt->level[l].wint;
  if (launch_shift_add(a, tab, wt->rowsum256, amax, s) != cudaSuccess) return PSB_ERR_CUDA;
  ctx->last_path = PSB_PATH_SHIFT_ADD;
  return PSB_OK;
}

}  // namespace

namespace psb {
static std::atomic<unsigned long long> g_launches{0};
void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
unsigned long long launches_so_far() { return g_launches.load(std::memory_order_relaxed); }
}  // namespace psb

extern "C" {

psb_status psb_create(psb_ctx** out, int device) {
  if (!out) return PSB_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
    cudaGetLastError();
    return PSB_ERR_CUDA;
  }
  if (cudaSetDevice(device) != cudaSuccess) return PSB_ERR_CUDA;
  int major = 0;
  cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
  if (major != 10) return PSB_ERR_UNSUPPORTED;  // kernels are built for sm_100a only
  psb_ctx* ctx = new (std::nothrow) psb_ctx();
  if (!ctx) return PSB_ERR_ALLOC;
  ctx->device = device;
  cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
  if (cudaMalloc(&ctx->err_dev, sizeof(uint32_t)) != cudaSuccess ||
      cudaMemset(ctx->err_dev, 0, sizeof(uint32_t)) != cudaSuccess) {
    delete ctx;
    return PSB_ERR_ALLOC;
  }
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ctx->encode_tiled, cudaEnableDefault, &q) !=
          cudaSuccess || q != cudaDriverEntryPointSuccess)
    ctx->encode_tiled = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &ctx->encode_im2col, cudaEnableDefault, &q) !=
          cudaSuccess || q != cudaDriverEntryPointSuccess)
    ctx->encode_im2col = nullptr;
  cudaGetLastError();
  *out = ctx;
  return PSB_OK;
}

psb_status psb_destroy(psb_ctx* ctx) {
  if (!ctx) return PSB_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  cudaDeviceSynchronize();
  for (int i = 0; i < 4; ++i)
    if (ctx->scratch[i]) cudaFree(ctx->scratch[i]);
  if (ctx->err_dev) cudaFree(ctx->err_dev);
  for (int i = 0; i < psb_ctx::kTimedLaunches; ++i) {
    if (ctx->t_begin[i]) cudaEventDestroy(ctx->t_begin[i]);
    if (ctx->t_end[i]) cudaEventDestroy(ctx->t_end[i]);
  }
  delete ctx;
  return PSB_OK;
}

const char* psb_status_string(psb_status st) {
  switch (st) {
    case PSB_OK: return "PSB_OK";
    case PSB_ERR_INVALID_ARG: return "PSB_ERR_INVALID_ARG";
    case PSB_ERR_BAD_K: return "PSB_ERR_BAD_K";
    case PSB_ERR_UNSUPPORTED: return "PSB_ERR_UNSUPPORTED";
    case PSB_ERR_ALLOC: return "PSB_ERR_ALLOC";
    case PSB_ERR_CUDA: return "PSB_ERR_CUDA";
    case PSB_ERR_TIMEOUT: return "PSB_ERR_TIMEOUT";
    case PSB_ERR_NONFINITE_WEIGHT: return "PSB_ERR_NONFINITE_WEIGHT";
    case PSB_ERR_RANGE: return "PSB_ERR_RANGE";
    default: return "PSB_ERR_UNKNOWN";
  }
}

psb_status psb_device_status(psb_ctx* ctx, void* stream) {
  if (!ctx) return PSB_ERR_INVALID_ARG;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return PSB_ERR_CUDA;
  uint32_t word = 0;
  if (cudaMemcpy(&word, ctx->err_dev, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess)
    return PSB_ERR_CUDA;
  if (word) cudaMemset(ctx->err_dev, 0, sizeof(word));
  if (word & kDevErrTimeout) return PSB_ERR_TIMEOUT;
  if (word & kDevErrNonFinite) return PSB_ERR_NONFINITE_WEIGHT;
  if (word & kDevErrBadLevel) return PSB_ERR_BAD_K;
  if (word & kDevErrRange) return PSB_ERR_RANGE;
  return PSB_OK;
}

psb_status psb_set_checks(psb_ctx* ctx, uint32_t flags) {
  if (!ctx || (flags & ~(uint32_t)PSB_CHECK_RANGE)) return PSB_ERR_INVALID_ARG;
  ctx->checks = flags;
  return PSB_OK;
}

psb_status psb_set_wait_limit(psb_ctx* ctx, uint64_t sm_clocks) {
  if (!ctx) return PSB_ERR_INVALID_ARG;
  ctx->wait_limit_cycles = sm_clocks ? sm_clocks : kDefaultWaitLimitCycles;
  return PSB_OK;
}

psb_status psb_wait_selftest(psb_ctx* ctx, void* stream) {
  if (!ctx) return PSB_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  return launch_wait_selftest(ctx, (cudaStream_t)stream) == cudaSuccess ? PSB_OK : PSB_ERR_CUDA;
}

psb_status psb_sample_weights(psb_ctx* ctx, const float* w_dev, const psb_wshape* shape,
                              const psb_sample_cfg* cfg_in, psb_weights** weights, void* stream) {
  if (!ctx || !w_dev || !shape || !cfg_in || !weights) return PSB_ERR_INVALID_ARG;
  if ((uintptr_t)w_dev & 3u) return PSB_ERR_INVALID_ARG;
  psb_sample_cfg cfg = *cfg_in;
  if (cfg.exp_bits == 0) cfg.exp_bits = 4;
  if (cfg.exp_bits > 4 || cfg.norm > 1) return PSB_ERR_INVALID_ARG;
  if (cfg.underflow > 1 || cfg.prob_bits > 8 || cfg.deterministic > 1 || cfg.reserved != 0 ||
      (cfg.deterministic && cfg.prob_bits == 0))
    return PSB_ERR_INVALID_ARG;
  if (cfg.level_mask == 0 || cfg.level_mask >= (1u << kMaxLevels)) return PSB_ERR_BAD_K;
  if (!shape->out_ch || !shape->in_ch_per_group || !shape->kh || !shape->kw || !shape->groups)
    return PSB_ERR_INVALID_ARG;
  if (shape->out_ch % shape->groups) return PSB_ERR_INVALID_ARG;
  if ((uint64_t)shape->kh * shape->kw > 2048) return PSB_ERR_UNSUPPORTED;
  uint64_t d64 = (uint64_t)shape->in_ch_per_group * shape->kh * shape->kw;
  if (d64 > (1u << 24) || d64 * shape->out_ch > (1ull << 31)) return PSB_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)stream;

  psb_weights* w = *weights;
  if (w) {
    const psb_wshape& a = w->shape;
    if (a.out_ch != shape->out_ch || a.in_ch_per_group != shape->in_ch_per_group ||
        a.kh != shape->kh || a.kw != shape->kw || a.groups != shape->groups ||
        w->cfg.level_mask != cfg.level_mask || w->cfg.exp_bits != cfg.exp_bits ||
        w->device != ctx->device)
      return PSB_ERR_INVALID_ARG;
    w->cfg = cfg;
  } else {
    w = new (std::nothrow) psb_weights();
    if (!w) return PSB_ERR_ALLOC;
    w->shape = *shape;
    w->cfg = cfg;
    w->device = ctx->device;
    w->d = (uint32_t)d64;
    const bool wide = shape->in_ch_per_group % 16 == 0 && shape->in_ch_per_group >= 32;
    w->packed_k = shape->groups == 1 && !wide && d64 >= 16;
    w->has_planes = shape->groups == 1 && (wide || w->packed_k);
    w->cpad = shape->in_ch_per_group;
    w->run_pitch = shape->kw * w->cpad;
    if (w->packed_k) w->run_pitch = round_up(w->run_pitch, 8);
    w->kpad = round_up(shape->kh * w->run_pitch, 16);
    w->o_tiles = (shape->out_ch + kTileN - 1) / kTileN;
    w->bk = tensor_bk(w->packed_k ? w->kpad : shape->in_ch_per_group);
    w->n_cb = ((w->packed_k ? w->kpad : shape->in_ch_per_group) + w->bk - 1) / w->bk;
    w->n_kb = w->packed_k ? w->n_cb : shape->kh * shape->kw * w->n_cb;
    bool ok = cudaMalloc(&w->e_base, sizeof(int32_t) * shape->out_ch) == cudaSuccess &&
              cudaMalloc(&w->e_max, sizeof(uint32_t) * shape->out_ch) == cudaSuccess &&
              cudaMalloc(&w->rowsum256, sizeof(uint32_t) * kMaxLevels * shape->out_ch) == cudaSuccess &&
              cudaMemsetAsync(w->e_max, 0, sizeof(uint32_t) * shape->out_ch, s) == cudaSuccess;
    for (uint32_t l = 0; ok && l < (uint32_t)kMaxLevels; ++l) {
      if (!((cfg.level_mask >> l) & 1u)) continue;
      ok = cudaMalloc(&w->level[l].wint, sizeof(int32_t) * d64 * shape->out_ch) == cudaSuccess;
      if (ok && w->has_planes) {
        int P = planes_for(cfg.exp_bits, l);
        size_t bytes = (size_t)w->o_tiles * w->n_kb * P * kTileN * w->bk;
        w->level[l].planes_count = P;
        ok = cudaMalloc(&w->level[l].planes, bytes) == cudaSuccess &&
             cudaMemsetAsync(w->level[l].planes, 0, bytes, s) == cudaSuccess;
        if (ok)
          ok = cudaMalloc(&w->level[l].corr128, sizeof(long long) * shape->out_ch) == cudaSuccess;
      }
    }
    if (!ok) {
      cudaGetLastError();
      free_weights_storage(w);
      delete w;
      return PSB_ERR_ALLOC;
    }
  }
  if (launch_sampler(w_dev, w, ctx->err_dev, s) != cudaSuccess) {
    if (!*weights) { free_weights_storage(w); delete w; }
    return PSB_ERR_CUDA;
  }
  *weights = w;
  return PSB_OK;
}

psb_status psb_weights_export(psb_ctx* ctx, const psb_weights* weights, uint32_t log2k,
                              int32_t* wint_dev, int32_t* e_base_dev, void* stream) {
  if (!ctx || !weights) return PSB_ERR_INVALID_ARG;
  if (!pow2_level_ok(log2k) || !((weights->cfg.level_mask >> log2k) & 1u)) return PSB_ERR_BAD_K;
  if (((uintptr_t)wint_dev | (uintptr_t)e_base_dev) & 3u) return PSB_ERR_INVALID_ARG;
  if (launch_export(weights, log2k, wint_dev, e_base_dev, (cudaStream_t)stream) != cudaSuccess)
    return PSB_ERR_CUDA;
  return PSB_OK;
}

psb_status psb_weights_free(psb_ctx* ctx, psb_weights* weights) {
  if (!ctx || !weights) return PSB_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  cudaDeviceSynchronize();
  free_weights_storage(weights);
  delete weights;
  return PSB_OK;
}

psb_status psb_set_sample_map(psb_ctx* ctx, const uint8_t* log2k_dev, uint32_t n, uint32_t oh,
                              uint32_t ow, uint32_t uniform_log2k) {
  if (!ctx) return PSB_ERR_INVALID_ARG;
  ctx->sorted_rows = 0;      // whatever was derived from an earlier map is dropped
  if (log2k_dev) {
    if (!n || !oh || !ow) return PSB_ERR_INVALID_ARG;
    ctx->kmap = log2k_dev;
    ctx->map_n = n; ctx->map_oh = oh; ctx->map_ow = ow;
  } else {
    if (!pow2_level_ok(uniform_log2k)) return PSB_ERR_BAD_K;
    ctx->kmap = nullptr;
    ctx->map_n = ctx->map_oh = ctx->map_ow = 0;
    ctx->uniform_log2k = uniform_log2k;
  }
  return PSB_OK;
}

psb_status psb_conv2d(psb_ctx* ctx, const psb_weights* weights, const void* x_dev,
                      const psb_conv_desc* d, void* stream) {
  if (!d) return PSB_ERR_INVALID_ARG;
  return run_layer(ctx, weights, x_dev, d->layout, d->in_dtype, d->in_max, d->n, d->c, d->h, d->w,
                   d->stride, d->pad, d->path, d->ep, stream);
}

psb_status psb_gemm(psb_ctx* ctx, const psb_weights* weights, const void* x_dev,
                    const psb_gemm_desc* d, void* stream) {
  if (!d) return PSB_ERR_INVALID_ARG;
  if (weights && (weights->shape.kh != 1 || weights->shape.kw != 1 || weights->shape.groups != 1))
    return PSB_ERR_INVALID_ARG;
  return run_layer(ctx, weights, x_dev, PSB_LAYOUT_NHWC, d->in_dtype, d->in_max, d->batch,
                   d->in_features, 1, 1, 1, 0, d->path, d->ep, stream);
}

int32_t psb_last_path(const psb_ctx* ctx) { return ctx ? ctx->last_path : 0; }

uint64_t psb_launch_count(void) { return (uint64_t)psb::launches_so_far(); }

psb_status psb_contraction_timing(psb_ctx* ctx, uint32_t enable) {
  if (!ctx) return PSB_ERR_INVALID_ARG;
  if (enable && !ctx->t_begin[0]) {
    cudaSetDevice(ctx->device);
    for (int i = 0; i < psb_ctx::kTimedLaunches; ++i)
      if (cudaEventCreate(&ctx->t_begin[i]) != cudaSuccess || cudaEventCreate(&ctx->t_end[i]) != cudaSuccess) {
        cudaGetLastError();
        return PSB_ERR_CUDA;
      }
  }
  ctx->time_contraction = enable != 0;
  if (enable) ctx->timed_launches = 0;     // switching it on starts a new sum
  return PSB_OK;
}

psb_status psb_contraction_time(psb_ctx* ctx, float* milliseconds) {
  if (!ctx || !milliseconds || ctx->timed_launches == 0) return PSB_ERR_INVALID_ARG;
  float total = 0.0f;
  for (int i = 0; i < ctx->timed_launches; ++i) {
    float ms = 0.0f;
    if (cudaEventSynchronize(ctx->t_end[i]) != cudaSuccess ||
        cudaEventElapsedTime(&ms, ctx->t_begin[i], ctx->t_end[i]) != cudaSuccess) {
      cudaGetLastError();
      return PSB_ERR_CUDA;
    }
    total += ms;
  }
  *milliseconds = total;
  return PSB_OK;
}

psb_status psb_contraction_times(psb_ctx* ctx, float* milliseconds, uint32_t capacity, uint32_t* count) {
  if (!ctx || !milliseconds || !count) return PSB_ERR_INVALID_ARG;
  *count = (uint32_t)ctx->timed_launches;
  for (int i = 0; i < ctx->timed_launches && (uint32_t)i < capacity; ++i) {
    if (cudaEventSynchronize(ctx->t_end[i]) != cudaSuccess ||
        cudaEventElapsedTime(&milliseconds[i], ctx->t_begin[i], ctx->t_end[i]) != cudaSuccess) {
      cudaGetLastError();
      return PSB_ERR_CUDA;
    }
  }
  return PSB_OK;
}

psb_status psb_int8_mma_probe(psb_ctx* ctx, uint32_t n_cols, uint32_t groups, double* mac_per_clk_per_sm,
                              double* tera_ops_per_s, void* stream) {
  if (!ctx) return PSB_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  return psb::int8_mma_probe(ctx, n_cols, groups, mac_per_clk_per_sm, tera_ops_per_s, (cudaStream_t)stream);
}

psb_status psb_sample_batch_create(psb_ctx* ctx, uint32_t n, const float* const* w_dev,
                                   psb_weights* const* weights, psb_sample_batch** batch) {
  if (!ctx || !n || !w_dev || !weights || !batch) return PSB_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < n; ++i) {
    if (!w_dev[i] || !weights[i] || ((uintptr_t)w_dev[i] & 3u)) return PSB_ERR_INVALID_ARG;
    if (weights[i]->device != ctx->device) return PSB_ERR_INVALID_ARG;
  }
  return sample_batch_create(ctx, n, w_dev, weights, batch);
}

psb_status psb_sample_batch_run(psb_ctx* ctx, psb_sample_batch* batch, uint64_t seed, void* stream) {
  if (!ctx || !batch) return PSB_ERR_INVALID_ARG;
  return sample_batch_run(ctx, batch, seed, (cudaStream_t)stream);
}

psb_status psb_sample_batch_free(psb_ctx* ctx, psb_sample_batch* batch) {
  if (!ctx || !batch) return PSB_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  cudaDeviceSynchronize();
  sample_batch_free(batch);
  return PSB_OK;
}

psb_status psb_run(psb_ctx* ctx, const psb_op* ops, uint32_t n_ops, void* stream) {
  if (!ctx || (!ops && n_ops)) return PSB_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < n_ops; ++i) {
    const psb_op& op = ops[i];
    psb_status st;
    switch (op.kind) {
      case PSB_OP_CONV2D:
      case PSB_OP_GEMM: {
        // within one list a map that several operations name is sorted by level once (the maps must not
        // change while the list runs); psb_set_sample_map drops the sorted order, so it is kept across it
        const uint8_t* kept_map = ctx->sorted_map;
        const uint32_t kept_rows = i ? ctx->sorted_rows : 0u;
        st = psb_set_sample_map(ctx, op.map_dev, op.map_n, op.map_oh, op.map_ow, op.uniform_log2k);
        if (st != PSB_OK) return st;
        ctx->sorted_map = kept_map;
        ctx->sorted_rows = kept_rows;
        st = op.kind == PSB_OP_CONV2D ? psb_conv2d(ctx, op.weights, op.x_dev, &op.conv, stream)
                                      : psb_gemm(ctx, op.weights, op.x_dev, &op.gemm, stream);
        break;
      }
      case PSB_OP_MAXPOOL:
        st = psb_maxpool2d_u8(ctx, (const uint8_t*)op.x_dev, op.conv.layout, op.conv.n, op.conv.c, op.conv.h,
                              op.conv.w, op.pool_k, op.conv.stride, op.conv.pad, op.pool_out_dev, stream);
        break;
      case PSB_OP_AVGPOOL:
        st = psb_global_avgpool_u8(ctx, (const uint8_t*)op.x_dev, op.conv.layout, op.conv.n, op.conv.c,
                                   op.conv.h, op.conv.w, op.pool_mul, op.pool_qmin, op.pool_qmax,
                                   op.pool_out_dev, stream);
        break;
      default:
        st = PSB_ERR_INVALID_ARG;
    }
    if (st != PSB_OK) return st;
  }
  return PSB_OK;
}

psb_status psb_attention_entropy(psb_ctx* ctx, const void* act_dev, uint32_t in_dtype, uint32_t n, uint32_t h,
                                 uint32_t w, uint32_t c, float step, float* entropy_dev, void* stream) {
  if (!ctx || !act_dev || !entropy_dev || !n || !h || !w || !c) return PSB_ERR_INVALID_ARG;
  if (in_dtype != PSB_DT_U8 && in_dtype != PSB_DT_S8) return PSB_ERR_INVALID_ARG;
  if (!(step > 0.0f) || ((uintptr_t)entropy_dev & 3u)) return PSB_ERR_INVALID_ARG;
  if ((uint64_t)n * h * w >= (1ull << 31)) return PSB_ERR_UNSUPPORTED;
  if (launch_entropy(act_dev, in_dtype == PSB_DT_S8, n * h * w, c, step, entropy_dev, (cudaStream_t)stream) != cudaSuccess)
    return PSB_ERR_CUDA;
  return PSB_OK;
}

psb_status psb_attention_maps(psb_ctx* ctx, const float* entropy_dev, uint32_t n, uint32_t h, uint32_t w,
                              uint32_t lo_log2k, uint32_t hi_log2k, uint32_t n_res, const uint32_t* res,
                              uint8_t* const* maps_dev, float* mean_dev, void* stream) {
  if (!ctx || !entropy_dev || !n || !h || !w || !n_res || n_res > 8u || !res || !maps_dev) return PSB_ERR_INVALID_ARG;
  if (!pow2_level_ok(lo_log2k) || !pow2_level_ok(hi_log2k)) return PSB_ERR_BAD_K;
  for (uint32_t i = 0; i < n_res; ++i)
    if (!res[i] || !maps_dev[i] || (uint64_t)res[i] * res[i] >= (1ull << 31)) return PSB_ERR_INVALID_ARG;
  if (launch_attention_maps(entropy_dev, n, h, w, lo_log2k, hi_log2k, n_res, res, maps_dev, mean_dev,
                            (cudaStream_t)stream) != cudaSuccess)
    return PSB_ERR_CUDA;
  return PSB_OK;
}

psb_status psb_maxpool2d_u8(psb_ctx* ctx, const uint8_t* x_dev, uint32_t layout, uint32_t n,
                            uint32_t c, uint32_t h, uint32_t w, uint32_t k, uint32_t stride,
                            uint32_t pad, uint8_t* out_dev, void* stream) {
  if (!ctx || !x_dev || !out_dev || !n || !c || !h || !w || !k || !stride) return PSB_ERR_INVALID_ARG;
  if (layout > PSB_LAYOUT_NHWC || h + 2 * pad < k || w + 2 * pad < k || pad >= k)
    return PSB_ERR_INVALID_ARG;
  if (launch_maxpool(x_dev, layout == PSB_LAYOUT_NCHW, n, c, h, w, k, stride, pad, out_dev,
                     (cudaStream_t)stream) != cudaSuccess)
    return PSB_ERR_CUDA;
  return PSB_OK;
}

psb_status psb_global_avgpool_u8(psb_ctx* ctx, const uint8_t* x_dev, uint32_t layout, uint32_t n,
                                 uint32_t c, uint32_t h, uint32_t w, float pool_mul, int32_t qmin,
                                 int32_t qmax, uint8_t* out_dev, void* stream) {
  if (!ctx || !x_dev || !out_dev || !n || !c || !h || !w) return PSB_ERR_INVALID_ARG;
  if (layout > PSB_LAYOUT_NHWC || qmin < 0 || qmax > 255 || qmin > qmax) return PSB_ERR_INVALID_ARG;
  if ((uint64_t)h * w * 255 >= (1ull << 31)) return PSB_ERR_UNSUPPORTED;
  if (launch_avgpool(x_dev, layout == PSB_LAYOUT_NCHW, n, c, h, w, pool_mul, qmin, qmax, out_dev,
                     (cudaStream_t)stream) != cudaSuccess)
    return PSB_ERR_CUDA;
  return PSB_OK;
}

}  // extern "C"
