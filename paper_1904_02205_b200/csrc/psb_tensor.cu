// Dense contraction on the 5th-generation tensor cores (tcgen05, sm_100a).
//
// acc[m, o] = sum_i X[m, i] * W_k[o, i]  (paper Eq. 1 with Eq. 9 summed over the
// draws) is an integer matrix product: M = output locations, N = output channels,
// K = taps x input channels.  |W_k| needs up to 22 bits, an MMA operand holds 8, so
// W_k is split into P signed 7-bit digit planes, W_k = sum_p D_p * 2^(7p).  One
// tcgen05.mma (kind::i8, s8 x s8 -> s32) of shape 128 x (P*64) x 32 multiplies an
// activation tile with all planes of 64 output channels at once; each plane owns
// 64 accumulator columns in tensor memory (TMEM) and the epilogue recombines them
// in 64-bit integers, which makes the result exact.
//
// Structure of one CTA (one per SM, persistent over tiles):
//   warp 0   producer: TMA loads of the activation tile (im2col mode for
//            filters with taps, stride or padding; plain 2-D tiles otherwise) and
//            of the digit-plane tile into a ring of shared-memory stages
//   warp 1   allocates TMEM; one thread issues the MMAs and commits them to the
//            stage-free and accumulator-ready barriers
//   warps 2-5  epilogue: TMEM -> registers, recombine planes, dequantise, bias,
//            shortcut, ReLU, re-quantise, vectorised stores; overlaps the next
//            tile's MMAs through two TMEM accumulator buffers
// Per-location draw counts (Sec. 4.5): a tile is contracted once per level present
// among its 128 rows; the epilogue of each pass stores only the rows of that level.
// Every wait is bounded; on a timeout the kernel raises the device error word and
// leaves through the common exit that frees TMEM.
#include <cuda.h>

#include <cstring>

#include "psb_common.cuh"

namespace psb {

namespace {

constexpr int kTileM = 128;
constexpr int kThreadsTensor = 192;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemBufStride = 256;
constexpr int kMaxStages = 8;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s per wait

struct TmapSet {
  CUtensorMap a;
  CUtensorMap b[kMaxLevels];
};

struct TensorParams {
  ConvArgs a;
  uint32_t M;           // N * OH * OW
  uint32_t m_tiles, o_tiles;
  uint32_t n_cb;        // channel blocks per tap
  uint32_t cpad;
  uint32_t im2col;      // 1: activation tile through the im2col tensor map
  uint32_t stages;
  uint32_t stage_bytes_a, stage_bytes_b_max;
  uint32_t planes[kMaxLevels];
  uint32_t vec_ok;      // 16-byte stores are legal for every output pointer
};

// ---- thin PTX wrappers -------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  Returns false after kWaitLimitNs without completion, or as soon
// as another thread of the CTA has given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0u) {
      if (*abort) return false;
      if (global_ns() - t0 > kWaitLimitNs) return false;
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x,
                                            int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                                   int c, int w, int h, int n, uint16_t off_w,
                                                   uint16_t off_h) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}

__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t desc_a, uint64_t desc_b,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major tile whose rows are `bk` bytes wide
// and swizzled with the matching TMA mode; groups of 8 rows are 8*bk bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t bk) {
  const uint64_t layout = bk == 128 ? 2ull : (bk == 64 ? 4ull : 6ull);
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                       // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)((8u * bk) >> 4) << 32;        // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                       // descriptor version of this architecture
  d |= layout << 61;
  return d;
}

// Levels (log2 k) present among the 128 rows of a tile, as a bit mask.  Warp-collective.
__device__ __forceinline__ uint32_t tile_levels(const TensorParams& p, uint32_t m0) {
  if (!p.a.kmap) return 1u << p.a.uniform_log2k;
  const uint32_t lane = threadIdx.x & 31u;
  uint32_t mask = 0;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    uint32_t m = m0 + r * 32u + lane;
    if (m < p.M) mask |= 1u << (p.a.kmap[m] & 31u);
  }
  return __reduce_or_sync(0xFFFFFFFFu, mask);
}

struct SharedCtl {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long acc_full[2];
  unsigned long long acc_empty[2];
  uint32_t tmem_base;
  volatile uint32_t abort;
  float sc[4][kTileN];      // per epilogue warp: scale[o] * 2^(e_base[o] - log2 k)
  float bias[4][kTileN];
};

template <int P>
__device__ __forceinline__ void epilogue_chunk(const TensorParams& p, uint32_t tmem_row_base,
                                               uint32_t chunk, uint32_t o_base, uint32_t m, bool valid,
                                               uint32_t n, uint32_t pix, const float* sc_s,
                                               const float* bias_s) {
  uint32_t v[P][16];
#pragma unroll
  for (int pl = 0; pl < P; ++pl) tc_ld16(tmem_row_base + pl * kTileN + chunk * 16u, v[pl]);
  tc_wait_ld();
  if (!valid) return;
  const ConvArgs& a = p.a;
  const uint32_t ohow = a.OH * a.OW;
  long long acc[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    long long s = (long long)(int)v[0][j];
#pragma unroll
    for (int pl = 1; pl < P; ++pl) s += (long long)(int)v[pl][j] << (kDigitBits * pl);
    acc[j] = s;
  }
  const bool full16 = o_base + 16u <= a.O;
  if (p.vec_ok && full16 && !a.out_nchw) {
    const size_t oidx = (size_t)m * a.O + o_base;
    if (a.acc_out) {
      longlong2* dst = reinterpret_cast<longlong2*>(a.acc_out + oidx);
#pragma unroll
      for (int j = 0; j < 8; ++j) dst[j] = make_longlong2(acc[2 * j], acc[2 * j + 1]);
    }
    if (a.q_out || a.f32_out) {
      uint32_t rw[4] = {0, 0, 0, 0};
      if (a.residual) {
        uint4 r4 = *reinterpret_cast<const uint4*>((const uint8_t*)a.residual + oidx);
        rw[0] = r4.x; rw[1] = r4.y; rw[2] = r4.z; rw[3] = r4.w;
      }
      float y[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        int rb = (int)((rw[j >> 2] >> (8 * (j & 3))) & 0xFFu);
        if (a.residual_dtype == PSB_DT_S8) rb = (int)(int8_t)rb;
        y[j] = dequant(acc[j], sc_s[chunk * 16 + j], bias_s[chunk * 16 + j], a.residual != nullptr, rb,
                       a.residual_scale, a.relu != 0);
      }
      if (a.f32_out) {
        float4* dst = reinterpret_cast<float4*>(a.f32_out + oidx);
#pragma unroll
        for (int j = 0; j < 4; ++j) dst[j] = make_float4(y[4 * j], y[4 * j + 1], y[4 * j + 2], y[4 * j + 3]);
      }
      if (a.q_out) {
        uint32_t qw[4] = {0, 0, 0, 0};
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          int q = requant(y[j], a.inv_step, a.qmin, a.qmax);
          qw[j >> 2] |= ((uint32_t)q & 0xFFu) << (8 * (j & 3));
        }
        *reinterpret_cast<uint4*>((uint8_t*)a.q_out + oidx) = make_uint4(qw[0], qw[1], qw[2], qw[3]);
      }
    }
    return;
  }
  // element-wise stores: channel-major outputs, ragged channel counts, odd alignment
#pragma unroll 1
  for (int j = 0; j < 16; ++j) {
    const uint32_t o = o_base + j;
    if (o >= a.O) break;
    const size_t oidx = a.out_nchw ? ((size_t)n * a.O + o) * ohow + pix : (size_t)m * a.O + o;
    if (a.acc_out) a.acc_out[oidx] = acc[j];
    if (a.q_out || a.f32_out) {
      int rb = 0;
      if (a.residual)
        rb = a.residual_dtype == PSB_DT_U8 ? (int)((const uint8_t*)a.residual)[oidx]
                                           : (int)((const int8_t*)a.residual)[oidx];
      float y = dequant(acc[j], sc_s[chunk * 16 + j], bias_s[chunk * 16 + j], a.residual != nullptr, rb,
                        a.residual_scale, a.relu != 0);
      if (a.f32_out) a.f32_out[oidx] = y;
      if (a.q_out) {
        int q = requant(y, a.inv_step, a.qmin, a.qmax);
        if (a.out_dtype == PSB_DT_U8) ((uint8_t*)a.q_out)[oidx] = (uint8_t)q;
        else ((int8_t*)a.q_out)[oidx] = (int8_t)q;
      }
    }
  }
}

template <int BK>
__global__ void __launch_bounds__(kThreadsTensor, 1)
psb_mma_kernel(const __grid_constant__ TmapSet maps, const TensorParams p) {
  extern __shared__ uint8_t smem_raw[];
  // stage buffers need 1024-byte alignment for the 128-byte swizzle pattern
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023u) & ~(uintptr_t)1023u);
  const uint32_t stage_bytes = p.stage_bytes_a + p.stage_bytes_b_max;
  SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + (size_t)p.stages * stage_bytes);

  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  const uint32_t n_tiles = p.m_tiles * p.o_tiles;
  const uint32_t k_iters = p.a.KH * p.a.KW * p.n_cb;

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctl->acc_full[b]), 1);
      mbar_init(smem_u32(&ctl->acc_empty[b]), 4);
    }
    ctl->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&ctl->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  volatile uint32_t* abort = &ctl->abort;
  bool failed = false;

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    uint32_t g = 0;  // stage use counter
    for (uint32_t tile = blockIdx.x; tile < n_tiles && !failed; tile += gridDim.x) {
      const uint32_t m_tile = tile / p.o_tiles, o_tile = tile % p.o_tiles;
      const uint32_t m0 = m_tile * kTileM;
      const uint32_t levels = tile_levels(p, m0);
      const uint32_t ohow = p.a.OH * p.a.OW;
      const uint32_t n0 = m0 / ohow, rem = m0 % ohow;
      const int h0 = (int)((rem / p.a.OW) * p.a.stride) - (int)p.a.pad;
      const int w0 = (int)((rem % p.a.OW) * p.a.stride) - (int)p.a.pad;
      for (uint32_t l = 0; l < (uint32_t)kMaxLevels && !failed; ++l) {
        if (!((levels >> l) & 1u)) continue;
        if (!((p.a.level_mask >> l) & 1u)) continue;   // flagged by the epilogue
        const uint32_t P = p.planes[l];
        const uint32_t bytes = p.stage_bytes_a + P * kTileN * BK;
        for (uint32_t it = 0; it < k_iters; ++it, ++g) {
          const uint32_t s = g % p.stages, ph = (g / p.stages) & 1u;
          if (lane == 0) {
            if (!mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1u, abort)) failed = true;
            if (!failed) {
              const uint32_t tap = it / p.n_cb, cb = it % p.n_cb;
              const uint32_t bar = smem_u32(&ctl->full[s]);
              const uint32_t dst_a = smem_u32(smem + (size_t)s * stage_bytes);
              const uint32_t dst_b = dst_a + p.stage_bytes_a;
              mbar_expect_tx(bar, bytes);
              if (p.im2col)
                tma_load_im2col_4d(dst_a, &maps.a, bar, (int)(cb * BK), w0, h0, (int)n0,
                                   (uint16_t)(tap % p.a.KW), (uint16_t)(tap / p.a.KW));
              else
                tma_load_2d(dst_a, &maps.a, bar, (int)(cb * BK), (int)m0);
              tma_load_2d(dst_b, &maps.b[l], bar, (int)(tap * p.cpad + cb * BK),
                          (int)(o_tile * P * kTileN));
            }
          }
          failed = __shfl_sync(0xFFFFFFFFu, failed ? 1 : 0, 0) != 0;
          if (failed) break;
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA
    uint32_t g = 0, pass = 0;
    for (uint32_t tile = blockIdx.x; tile < n_tiles && !failed; tile += gridDim.x) {
      const uint32_t m0 = (tile / p.o_tiles) * kTileM;
      const uint32_t levels = tile_levels(p, m0);
      for (uint32_t l = 0; l < (uint32_t)kMaxLevels && !failed; ++l) {
        if (!((levels >> l) & 1u)) continue;
        if (!((p.a.level_mask >> l) & 1u)) continue;
        const uint32_t P = p.planes[l];
        const uint32_t buf = pass & 1u, aph = (pass >> 1) & 1u;
        // instruction descriptor: s32 accumulators, s8 x s8, both K-major, M = 128, N = P * 64
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | (((P * kTileN) >> 3) << 17) |
                               ((kTileM >> 4) << 24);
        const uint32_t d_tmem = tmem_base + buf * kTmemBufStride;
        if (lane == 0) {
          if (!mbar_wait(smem_u32(&ctl->acc_empty[buf]), aph ^ 1u, abort)) failed = true;
        }
        failed = __shfl_sync(0xFFFFFFFFu, failed ? 1 : 0, 0) != 0;
        if (failed) break;
        tc_fence_after();
        for (uint32_t it = 0; it < k_iters; ++it, ++g) {
          const uint32_t s = g % p.stages, ph = (g / p.stages) & 1u;
          if (lane == 0) {
            if (!mbar_wait(smem_u32(&ctl->full[s]), ph, abort)) failed = true;
            if (!failed) {
              tc_fence_after();
              const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
              const uint32_t b_addr = a_addr + p.stage_bytes_a;
#pragma unroll
              for (int ks = 0; ks < BK / 32; ++ks)
                tc_mma_i8(d_tmem, smem_desc(a_addr + ks * 32, BK), smem_desc(b_addr + ks * 32, BK),
                          idesc, (it | ks) != 0 ? 1u : 0u);
              tc_commit(smem_u32(&ctl->empty[s]));
              if (it + 1 == k_iters) tc_commit(smem_u32(&ctl->acc_full[buf]));
            }
          }
          failed = __shfl_sync(0xFFFFFFFFu, failed ? 1 : 0, 0) != 0;
          if (failed) break;
        }
        ++pass;
      }
    }
  } else {
    // ----------------------------------------------------------- epilogue
    const uint32_t quarter = warp & 3u;              // TMEM lanes this warp may touch
    const uint32_t row = quarter * 32u + lane;
    uint32_t pass = 0;
    for (uint32_t tile = blockIdx.x; tile < n_tiles && !failed; tile += gridDim.x) {
      const uint32_t m_tile = tile / p.o_tiles, o_tile = tile % p.o_tiles;
      const uint32_t m0 = m_tile * kTileM;
      const uint32_t levels = tile_levels(p, m0);
      const uint32_t m = m0 + row;
      const bool in_range = m < p.M;
      const uint32_t my_level = in_range ? (p.a.kmap ? (uint32_t)p.a.kmap[m] : p.a.uniform_log2k) : 0xFFu;
      const uint32_t ohow = p.a.OH * p.a.OW;
      const uint32_t n = in_range ? m / ohow : 0u, pix = in_range ? m % ohow : 0u;
      if (in_range && (my_level >= (uint32_t)kMaxLevels || !((p.a.level_mask >> my_level) & 1u)))
        atomicOr(p.a.err, kDevErrBadLevel);
      for (uint32_t l = 0; l < (uint32_t)kMaxLevels && !failed; ++l) {
        if (!((levels >> l) & 1u)) continue;
        if (!((p.a.level_mask >> l) & 1u)) continue;
        const uint32_t P = p.planes[l];
        const uint32_t buf = pass & 1u, aph = (pass >> 1) & 1u;
        // per-channel constants of this pass (exact power-of-two rescale of the scale);
        // every warp keeps its own copy so that no CTA-wide barrier is needed
#pragma unroll
        for (uint32_t e = lane; e < (uint32_t)kTileN; e += 32u) {
          const uint32_t o = o_tile * kTileN + e;
          float sc = 0.f, bi = 0.f;
          if (o < p.a.O) {
            sc = ldexpf(p.a.scale[o], p.a.e_base[o] - (int)l);
            bi = p.a.bias[o];
          }
          ctl->sc[quarter][e] = sc;
          ctl->bias[quarter][e] = bi;
        }
        __syncwarp();
        if (lane == 0) {
          if (!mbar_wait(smem_u32(&ctl->acc_full[buf]), aph, abort)) failed = true;
        }
        failed = __shfl_sync(0xFFFFFFFFu, failed ? 1 : 0, 0) != 0;
        if (failed) break;
        tc_fence_after();
        const uint32_t trow = tmem_base + buf * kTmemBufStride + ((quarter * 32u) << 16);
        const bool valid = in_range && my_level == l;
        for (uint32_t chunk = 0; chunk < (uint32_t)kTileN / 16u; ++chunk) {
          const uint32_t o_base = o_tile * kTileN + chunk * 16u;
          if (o_base >= p.a.O) break;
          switch (P) {
            case 1: epilogue_chunk<1>(p, trow, chunk, o_base, m, valid, n, pix, ctl->sc[quarter], ctl->bias[quarter]); break;
            case 2: epilogue_chunk<2>(p, trow, chunk, o_base, m, valid, n, pix, ctl->sc[quarter], ctl->bias[quarter]); break;
            case 3: epilogue_chunk<3>(p, trow, chunk, o_base, m, valid, n, pix, ctl->sc[quarter], ctl->bias[quarter]); break;
            default: epilogue_chunk<4>(p, trow, chunk, o_base, m, valid, n, pix, ctl->sc[quarter], ctl->bias[quarter]); break;
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[buf]));
        ++pass;
      }
    }
  }

  // ------------------------------------------------------------- common exit
  if (failed) {
    if (lane == 0) {
      *abort = 1u;
      atomicOr(p.a.err, kDevErrTimeout);
    }
    // give copies and MMAs already in flight time to land before the CTA retires
    for (int i = 0; i < 64; ++i) __nanosleep(2000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(kTmemCols)
                 : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const int*, const int*,
                                   cuuint32_t, cuuint32_t, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

CUtensorMapSwizzle swizzle_for(uint32_t bk) {
  return bk == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                   : (bk == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}

bool is_plain_gemm(const ConvArgs& a) {
  return a.KH == 1 && a.KW == 1 && a.stride == 1 && a.pad == 0;
}

constexpr size_t kSmemBudget = 227 * 1024;

}  // namespace

psb_status tensor_supported(const psb_ctx* ctx, const psb_weights* wt, const ConvArgs& a) {
  if (!ctx->encode_tiled || !ctx->encode_im2col) return PSB_ERR_UNSUPPORTED;
  if (!wt->has_planes || a.groups != 1) return PSB_ERR_UNSUPPORTED;
  if (a.C % 16u || a.C < 32u) return PSB_ERR_UNSUPPORTED;
  if ((uintptr_t)a.x & 15u) return PSB_ERR_UNSUPPORTED;
  if (a.stride > 8 || a.pad > 127 || a.KH > 128 || a.KW > 128) return PSB_ERR_UNSUPPORTED;
  // each plane accumulates in 32 bits: |digit| <= 127, |x| <= 128
  if ((uint64_t)wt->d * 127ull * 128ull >= (1ull << 31)) return PSB_ERR_UNSUPPORTED;
  return PSB_OK;
}

psb_status launch_tensor(psb_ctx* ctx, const psb_weights* wt, const ConvArgs& a, cudaStream_t s) {
  TmapSet maps;
  TensorParams p;
  p.a = a;
  p.M = a.N * a.OH * a.OW;
  p.m_tiles = (p.M + kTileM - 1) / kTileM;
  p.o_tiles = wt->o_tiles;
  const uint32_t bk = wt->bk;
  p.n_cb = (a.C + bk - 1) / bk;
  p.cpad = wt->cpad;
  p.im2col = is_plain_gemm(a) ? 0u : 1u;
  uint32_t pmax = 1;
  for (int l = 0; l < kMaxLevels; ++l) {
    p.planes[l] = (uint32_t)wt->level[l].planes_count;
    if (p.planes[l] > pmax) pmax = p.planes[l];
  }
  p.stage_bytes_a = kTileM * bk;
  p.stage_bytes_b_max = pmax * kTileN * bk;
  const size_t ctl_bytes = sizeof(SharedCtl) + 1024;
  uint32_t stages = (uint32_t)((kSmemBudget - ctl_bytes) / (p.stage_bytes_a + p.stage_bytes_b_max));
  if (stages > (uint32_t)kMaxStages) stages = kMaxStages;
  if (stages < 2) return PSB_ERR_UNSUPPORTED;
  p.stages = stages;
  const size_t smem_bytes = (size_t)stages * (p.stage_bytes_a + p.stage_bytes_b_max) + ctl_bytes;
  bool vec = !a.out_nchw && a.O % 16u == 0;
  vec = vec && !(((uintptr_t)a.q_out | (uintptr_t)a.residual | (uintptr_t)a.f32_out |
                  (uintptr_t)a.acc_out) & 15u);
  p.vec_ok = vec ? 1u : 0u;

  const CUtensorMapSwizzle swz = swizzle_for(bk);
  EncodeTiledFn enc_tiled = (EncodeTiledFn)ctx->encode_tiled;
  EncodeIm2colFn enc_im2col = (EncodeIm2colFn)ctx->encode_im2col;
  if (p.im2col) {
    cuuint64_t dims[4] = {a.C, a.W, a.H, a.N};
    cuuint64_t strides[3] = {(cuuint64_t)a.C, (cuuint64_t)a.C * a.W, (cuuint64_t)a.C * a.W * a.H};
    int lower[2] = {-(int)a.pad, -(int)a.pad};
    int upper[2] = {(int)a.pad - (int)(a.KW - 1), (int)a.pad - (int)(a.KH - 1)};
    cuuint32_t estr[4] = {1, a.stride, a.stride, 1};
    if (enc_im2col(&maps.a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(a.x), dims, strides,
                   lower, upper, bk, kTileM, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return PSB_ERR_CUDA;
  } else {
    cuuint64_t dims[2] = {a.C, p.M};
    cuuint64_t strides[1] = {(cuuint64_t)a.C};
    cuuint32_t box[2] = {bk, kTileM};
    cuuint32_t estr[2] = {1, 1};
    if (enc_tiled(&maps.a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(a.x), dims, strides, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return PSB_ERR_CUDA;
  }
  for (int l = 0; l < kMaxLevels; ++l) {
    if (!wt->level[l].planes) { memset(&maps.b[l], 0, sizeof(CUtensorMap)); continue; }
    const uint32_t P = (uint32_t)wt->level[l].planes_count;
    cuuint64_t dims[2] = {wt->kpad, (cuuint64_t)wt->o_tiles * P * kTileN};
    cuuint64_t strides[1] = {(cuuint64_t)wt->kpad};
    cuuint32_t box[2] = {bk, P * kTileN};
    cuuint32_t estr[2] = {1, 1};
    if (enc_tiled(&maps.b[l], CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, wt->level[l].planes, dims, strides, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return PSB_ERR_CUDA;
  }

  const uint32_t n_tiles = p.m_tiles * p.o_tiles;
  const uint32_t grid = n_tiles < (uint32_t)ctx->sm_count ? n_tiles : (uint32_t)ctx->sm_count;
  cudaError_t e;
#define PSB_LAUNCH(BKV)                                                                              \
  e = cudaFuncSetAttribute(psb_mma_kernel<BKV>, cudaFuncAttributeMaxDynamicSharedMemorySize,         \
                           (int)smem_bytes);                                                         \
  if (e == cudaSuccess) psb_mma_kernel<BKV><<<grid, kThreadsTensor, smem_bytes, s>>>(maps, p);
  if (bk == 128) { PSB_LAUNCH(128) } else if (bk == 64) { PSB_LAUNCH(64) } else { PSB_LAUNCH(32) }
#undef PSB_LAUNCH
  if (e != cudaSuccess || cudaGetLastError() != cudaSuccess) return PSB_ERR_CUDA;
  return PSB_OK;
}

}  // namespace psb
