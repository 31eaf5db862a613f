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
//   warps 0-1 producers (one thread each, taking the stages in turns): TMA loads of the activation tile (im2col mode for
//            filters with taps, stride or padding; plain 2-D tiles otherwise) and
//            of the digit-plane tile into a ring of shared-memory stages
//   warps 2-3 MMA issuers (one thread each; warp 3 also allocates TMEM): the pipeline stages
//            alternate between them.  The tensor pipe takes only a few MMAs ahead of the one it
//            executes, so whatever else an issuing thread does (barrier waits, commits, tile
//            bookkeeping: a few hundred clocks per stage) would leave the pipe idle; with two
//            issuers one thread's bookkeeping runs under the other's MMAs
//   warps 4-19 epilogue: TMEM -> registers, recombine planes, dequantise, bias,
//            shortcut, ReLU, re-quantise, vectorised stores; overlaps the next
//            tile's MMAs through two TMEM accumulator buffers
// Per-location draw counts (Sec. 4.5): the caller sorts the output locations by level and
// gathers the activation rows in that order (psb_sort.cu); every tile then has one level, and
// the epilogue scatters each row back to its location.
// Every wait is bounded; on a timeout the kernel raises the device error word and
// leaves through the common exit that frees TMEM.
#include <cuda.h>

#include <cstring>

#include "psb_common.cuh"

namespace psb {

namespace {

constexpr int kTileM = 128;
constexpr int kProducerWarps = 2;    // one issuing thread each: their barrier waits overlap
constexpr int kMmaWarp0 = kProducerWarps;          // issues the even passes
constexpr int kMmaWarp1 = kMmaWarp0 + 1;           // issues the odd passes; owns the TMEM allocation
constexpr int kFirstEpilogueWarp = kMmaWarp1 + 1;  // a multiple of 4: warp & 3 = TMEM lane quarter
constexpr int kPlaneBars = 4;        // resident digit planes arrive in this many parts, each with its barrier
constexpr int kEpilogueWarps = 16;
constexpr int kThreadsTensor = 32 * (kFirstEpilogueWarp + kEpilogueWarps);
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemBufStride = 256;
constexpr int kMaxStages = 12;
constexpr uint32_t kResidentMaxBytes = 112 * 1024;          // digit planes kept in shared memory
constexpr int kTapBatch = 6;                                // descriptor offsets fetched ahead of their MMAs
constexpr int kMaxBandMmas = 128;                           // MMAs per tile (taps x K steps) that band mode handles

struct TmapSet {
  CUtensorMap a;     // activations; the digit planes need none: their tiles are contiguous
};

struct TensorParams {
  ConvArgs a;
  uint32_t M;           // N * OH * OW
  uint32_t m_tiles, o_tiles;
  uint32_t n_cb;        // channel blocks per tap
  uint32_t im2col;      // 1: activation tile through the im2col tensor map
  uint32_t stages;
  uint32_t group;       // K blocks per pipeline stage (one barrier hand-over per group)
  uint32_t stage_bytes_a, stage_bytes_b_max;
  uint32_t planes[kMaxLevels];
  const uint8_t* tile_mask;   // per row tile: levels present (bit l = level l), or null without a map
  uint32_t vec_ok;      // output rows (and pointers) are multiples of 16 bytes (2), of 8 bytes (1), or neither
  uint32_t resident;    // 1: the CTA keeps the digit planes of its channel tile in shared memory
  uint32_t ctas_per_otile;
  uint32_t resident_bytes;
  const uint32_t* rowsum256;   // [level][O] row sums of |W_k| in units of 256 (rounded up), or null
  uint32_t amax;        // largest activation magnitude the caller vouches for
  const long long* corr[kMaxLevels];  // per-channel integer addend, or null
  const int8_t* planes_ptr[kMaxLevels];  // digit planes: [o_tile][K block][P * 64 rows][BK], pre-swizzled tiles
  // Band mode (stride-1 filters with taps, one channel block, resident planes): a tile is 128
  // consecutive positions of one image's output in "padded-linear" order t = oy * Wp + ox with
  // Wp = W + 2 * pad (positions with ox >= OW are computed and dropped).  In that order the
  // input pixel of tap (kh, kw) for position t is pixel t + kh * Wp + kw of the zero-padded
  // image, so one copy of a band of padded input rows serves every tap: the activation operand
  // of a tap is the same shared-memory band read from a start address moved by
  // (kh * Wp + kw) pixels.  (The swizzle of a K-major operand is a function of the
  // shared-memory address bits, so a start address moved by whole rows reads correctly.)
  uint32_t band;        // 1: band mode
  uint32_t Wp;          // padded row length
  uint32_t tpi;         // tiles per image: ceil(OH * Wp / 128)
  uint32_t band_rows;   // padded input rows per band
  uint32_t band_bytes;  // stage size (band_rows * Wp * C rounded up to 1024)
  // Per-location draw counts: the rows of the activation matrix are sorted by level (psb_sort.cu), every tile
  // has one level (tile_mask holds one bit), and row r of the matrix is output location perm[r]
  const uint32_t* perm;  // or null
  uint32_t Wp_magic, tpi_magic;   // ceil(2^32 / Wp), ceil(2^32 / tpi): quotients by multiply-high (exact in the
                                  // ranges band mode is restricted to)
  unsigned long long wait_limit;  // bound of every wait in SM clocks
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

// What a bounded wait consults on its slow path: the CTA-wide give-up flag and the bound in SM clocks.
struct WaitCtl {
  volatile uint32_t abort;
  uint32_t pad;
  volatile unsigned long long limit;
};

constexpr uint32_t kNoSleep = 0xFFFFFFFFu;   // backoff value of a wait that is about to end: poll without sleeping

// Bounded wait.  Returns false after wc->limit SM clocks without completion, or as soon
// as another thread of the CTA has given up.  (The SM cycle counter is cheap to read.)
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, WaitCtl* wc,
                                          uint32_t backoff_ns = 0) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    // a thread that has to wait long should not eat the issue slots of the warps doing the
    // arithmetic: poll a few times at full speed, then sleep between polls
    ++spins;
    if (backoff_ns != kNoSleep && (backoff_ns || spins > 4u))
      __nanosleep(backoff_ns ? backoff_ns : (spins > 32u ? 256u : 64u));
    if ((spins & 15u) == 0u) {
      if (wc->abort) return false;
      if ((unsigned long long)(clock64() - t0) > wc->limit) return false;
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

// Plain bulk copy of a contiguous, 16-byte aligned run of global memory.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c, int w, int h,
                                            int n) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n)
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

// The same instruction for the issue loops: accumulate always, descriptors given as (low word, high word),
// no memory clobber (the loop's own loads of descriptor offsets may then be scheduled ahead of it; the
// operands are written by the copy engine and ordered by the barrier waits, which keep their clobbers).
template <bool ACC>
__device__ __forceinline__ void tc_mma_i8_lohi(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                               uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(ACC ? 1u : 0u));
}
__device__ __forceinline__ void tc_mma_i8_acc(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                              uint32_t idesc) {
  tc_mma_i8_lohi<true>(d_tmem, a_lo, b_lo, desc_hi, idesc);
}
__device__ __forceinline__ void tc_mma_i8_zero(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                               uint32_t idesc) {
  tc_mma_i8_lohi<false>(d_tmem, a_lo, b_lo, desc_hi, idesc);
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

// The two words of that descriptor.  Only the low word depends on the address (bits 0..13 = address / 16;
// shared memory ends below 2^18, so adding a byte offset / 16 to the low word moves the start address and
// touches nothing else).
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | (1u << 16); }
__device__ __forceinline__ uint32_t smem_desc_hi(uint32_t bk) {
  const uint32_t layout = bk == 128 ? 2u : (bk == 64 ? 4u : 6u);
  return ((8u * bk) >> 4) | (1u << 14) | (layout << 29);
}

// Levels (log2 k) of a tile as a bit mask: one byte per row tile, written by the level sort just before the
// contraction kernel (rows are sorted by level, so exactly one bit is set).
__device__ __forceinline__ uint32_t tile_levels(const TensorParams& p, uint32_t m_tile) {
  if (!p.tile_mask) return 1u << p.a.uniform_log2k;
  return (uint32_t)p.tile_mask[m_tile];
}

// Walks the tiles of this CTA without divisions in the loop.  Resident mode: the CTA owns one
// channel tile and strides over the row tiles; streaming mode: tiles are dealt round-robin with
// the channel tile fastest.
struct TileIter {
  uint32_t m_tile, o_tile, step_m, step_o, o_tiles, m_tiles;
  __device__ __forceinline__ void init(const TensorParams& p) {
    o_tiles = p.o_tiles;
    m_tiles = p.m_tiles;
    if (p.resident) {
      o_tile = blockIdx.x / p.ctas_per_otile;
      m_tile = blockIdx.x % p.ctas_per_otile;
      step_m = p.ctas_per_otile;
      step_o = 0;
    } else {
      m_tile = blockIdx.x / p.o_tiles;
      o_tile = blockIdx.x % p.o_tiles;
      step_m = gridDim.x / p.o_tiles;
      step_o = gridDim.x % p.o_tiles;
    }
  }
  __device__ __forceinline__ bool valid() const { return m_tile < m_tiles; }
  __device__ __forceinline__ void next() {
    m_tile += step_m;
    o_tile += step_o;
    if (o_tile >= o_tiles) { o_tile -= o_tiles; ++m_tile; }
  }
};

struct SharedCtl {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long acc_full[2];
  unsigned long long acc_empty[2];
  unsigned long long planes_full[kPlaneBars];
  unsigned long long started[2];        // per accumulator buffer: the zeroing MMA of the pass has been issued
  unsigned long long pass_issued;       // all but the last K block of a pass have been issued (phase = pass number)
  uint2 tap_tab[2][kMaxBandMmas];       // band mode, per issuing thread: (activation, plane) descriptor offsets of the
                                        // tile's MMAs, in units of 16 bytes
  uint32_t tmem_base;
  WaitCtl wait;
  alignas(16) float2 scb[kEpilogueWarps][16];   // per epilogue warp: (scale * 2^(e_base - log2 k), bias), read two
                                                // channels (16 bytes) at a time
  long long corr[kEpilogueWarps][16];   // per epilogue warp: integer addend per channel
};

// Output arithmetic of one 16-channel chunk held in registers (v[plane][channel]), common case:
// only re-quantised bytes are wanted.  Same arithmetic as dequant()/requant(), with as few issued
// instructions per output as the definition allows (the output stage of a layer with few input
// channels is bound by instruction issue, and every slot it takes is one the MMA-issuing thread of
// the same scheduler does not get):
//   W32: the accumulator itself is known to stay below 2^31 in magnitude (the sampler keeps the
//        largest row sum of |W_k|, the caller vouches for the largest activation): the planes are
//        recombined in 32 bits (wrap-around in the partial sums is harmless) and one conversion
//        instruction rounds to nearest even, as the 64-bit conversion would.  Otherwise 64-bit
//        recombination plus the per-channel integer addend, converted in two exact halves.
//   y = fma(a, sc, bias); optional shortcut fma on a byte converted by the conversion unit.
//   t = y * inv_step, clamped above in fp32; cvt.rni (round half to even, saturating) gives the
//   integer; cvt.pack.sat packs two integers at a time into bytes, saturating to the byte's range.
//   FAST_U8: unsigned codes whose lower bound is 0 (the ReLU, if any, folded into it): the byte
//   saturation is the lower clamp.  Otherwise both clamps are applied in fp32 first.
struct EpiConst {
  float res_scale, inv_step, lo_f, hi_f;   // lo_f already holds the relu (see the epilogue set-up)
  uint32_t out_signed;
};

// d = bytes (sat(b), sat(a), c.b0, c.b1), saturation to the unsigned / signed byte range
__device__ __forceinline__ uint32_t pack_sat_u8(int a, int b, uint32_t c) {
  uint32_t d;
  asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t pack_sat_s8(int a, int b, uint32_t c) {
  uint32_t d;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// RES: 0 no shortcut, 1 unsigned shortcut bytes, 2 signed ones.
template <int P, bool W32, int RES, bool FAST_U8>
__device__ __forceinline__ uint4 chunk_math(const uint32_t (&v)[P][16], const uint4& r4, const float2* scb,
                                            const long long* corr, const EpiConst& c) {
  const uint32_t rw[4] = {r4.x, r4.y, r4.z, r4.w};
  const float4* scb2 = reinterpret_cast<const float4*>(scb);   // two channels' (scale, bias) per load
  uint32_t qw[4];
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    int q[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int j = 4 * g + e;
      float af;
      if (W32) {
        int acc = (int)v[0][j];
#pragma unroll
        for (int pl = 1; pl < P; ++pl) acc += (int)v[pl][j] << (kDigitBits * pl);
        af = __int2float_rn(acc);
      } else {
        long long acc = (long long)(int)v[0][j];
#pragma unroll
        for (int pl = 1; pl < P; ++pl) acc += (long long)(int)v[pl][j] * (long long)(1 << (kDigitBits * pl));
        acc += corr[j];
        af = acc_to_float(acc);
      }
      const float4 sb2 = scb2[j >> 1];
      float y = (j & 1) ? __fmaf_rn(af, sb2.z, sb2.w) : __fmaf_rn(af, sb2.x, sb2.y);
      if (RES == 1) y = __fmaf_rn((float)((rw[g] >> (8 * e)) & 0xFFu), c.res_scale, y);
      if (RES == 2) y = __fmaf_rn((float)(int)(signed char)(rw[g] >> (8 * e)), c.res_scale, y);
      float t = fminf(__fmul_rn(y, c.inv_step), c.hi_f);
      if (!FAST_U8) t = fmaxf(t, c.lo_f);
      q[e] = __float2int_rn(t);
    }
    if (FAST_U8) {
      qw[g] = pack_sat_u8(q[1], q[0], pack_sat_u8(q[3], q[2], 0u));
    } else {
      const uint32_t u = pack_sat_u8(q[1], q[0], pack_sat_u8(q[3], q[2], 0u));
      const uint32_t sg = pack_sat_s8(q[1], q[0], pack_sat_s8(q[3], q[2], 0u));
      qw[g] = c.out_signed ? sg : u;
    }
  }
  return make_uint4(qw[0], qw[1], qw[2], qw[3]);
}

// 16 bytes of a channels-last row.  Rows that are only 8-byte aligned (channel counts that are odd
// multiples of 8) move as two halves; `both` is false for the last 8 channels of such a row.
// The loads are volatile asm so that they stay where they are written (a tile ahead of their use, before
// the wait for the accumulator) instead of being sunk to the first use of the value.
__device__ __forceinline__ uint4 load_row16(const uint8_t* src, bool vec16, bool both) {
  uint4 r = make_uint4(0u, 0u, 0u, 0u);
  if (vec16) {
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(src));
    return r;
  }
  asm volatile("ld.global.nc.v2.u32 {%0, %1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(src));
  if (both) asm volatile("ld.global.nc.v2.u32 {%0, %1}, [%2];" : "=r"(r.z), "=r"(r.w) : "l"(src + 8));
  return r;
}
__device__ __forceinline__ void store_row16(uint8_t* dst, uint4 v, bool vec16, bool both) {
  if (vec16) {
    *reinterpret_cast<uint4*>(dst) = v;
  } else {
    *reinterpret_cast<uint2*>(dst) = make_uint2(v.x, v.y);
    if (both) *reinterpret_cast<uint2*>(dst + 8) = make_uint2(v.z, v.w);
  }
}

// The same 16 channels of one output location in a planar ([n][o][oy][ox]) tensor: byte j sits
// j * plane further on.  Lanes of a warp hold consecutive locations, so each of the 16 accesses
// is a contiguous run of 32 bytes per warp.
// (Out of line to keep the callers' loops small.  The registers such a function may use are what all
// of its callers can spare, so each caller family gets its own instance, selected by TAG: when the
// plain output-stage loop, which holds more live values, shared one instance with the band-mode loop,
// the byte loop of the store spilled and band mode with planar output lost a third of its speed.)
template <int TAG>
__device__ __noinline__ uint4 load_planar16(const uint8_t* src, size_t plane, uint32_t count) {
  uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int j = 0; j < 16; ++j)
    if ((uint32_t)j < count) w[j >> 2] |= (uint32_t)__ldcg(src + (size_t)j * plane) << (8 * (j & 3));
  return make_uint4(w[0], w[1], w[2], w[3]);
}
template <int TAG>
__device__ __noinline__ void store_planar16(uint8_t* dst, size_t plane, uint32_t count, uint4 v) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 16; ++j)
    if ((uint32_t)j < count) dst[(size_t)j * plane] = (uint8_t)(w[j >> 2] >> (8 * (j & 3)));
}

// The P plane sums of a 16-channel chunk, TMEM -> registers.  With 32-bit recombination the planes are
// folded as they arrive (v0 + 2^7 v1 + ..., what chunk_math computes first anyway): 32 registers at the
// peak instead of 16 P, which is what the loop around it was spilling.  The folded planes are left as
// literal zeros, so the arithmetic after them drops out.
template <int P, bool W32>
__device__ __forceinline__ void load_chunk(uint32_t taddr, uint32_t (&v)[P][16]) {
  if (P >= 3 && W32) {
    tc_ld16(taddr, v[0]);
    tc_ld16(taddr + kTileN, v[1]);
    tc_wait_ld();
#pragma unroll
    for (int pl = 2; pl < P; ++pl) {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        v[0][j] = (uint32_t)((int)v[0][j] + ((int)v[pl - 1][j] << (kDigitBits * (pl - 1))));
        v[pl - 1][j] = 0u;
      }
      tc_ld16(taddr + pl * kTileN, v[pl]);
      tc_wait_ld();
    }
  } else {
#pragma unroll
    for (int pl = 0; pl < P; ++pl) tc_ld16(taddr + pl * kTileN, v[pl]);
    tc_wait_ld();
  }
}

template <int P, bool W32, int RES>
__device__ __noinline__ void epilogue_chunk_q(uint32_t taddr, bool valid, uint8_t* q_dst, uint4 r4, bool vec16,
                                              bool both, const float2* scb, const long long* corr, EpiConst c) {
  uint32_t v[P][16];
  load_chunk<P, W32>(taddr, v);
  if (!valid) return;
  store_row16(q_dst, chunk_math<P, W32, RES, false>(v, r4, scb, corr, c), vec16, both);
}

// General output stage: any combination of outputs, layouts, ragged channel counts.
template <int P>
__device__ __noinline__ void epilogue_chunk(const TensorParams& p, uint32_t taddr, uint32_t o_base,
                                            uint32_t m, bool valid, uint32_t n, uint32_t pix,
                                            const float2* scb, const long long* corr, bool use_corr) {
  uint32_t v[P][16];
#pragma unroll
  for (int pl = 0; pl < P; ++pl) tc_ld16(taddr + pl * kTileN, v[pl]);
  tc_wait_ld();
  if (!valid) return;
  const ConvArgs& a = p.a;
  const uint32_t ohow = a.OH * a.OW;
  const bool vec = p.vec_ok == 2u && o_base + 16u <= a.O && !a.out_nchw;
  uint32_t rw[4] = {0, 0, 0, 0};
  if (vec && a.residual) {
    uint4 r4 = *reinterpret_cast<const uint4*>((const uint8_t*)a.residual + (size_t)m * a.O + o_base);
    rw[0] = r4.x; rw[1] = r4.y; rw[2] = r4.z; rw[3] = r4.w;
  }
  uint32_t qw[4] = {0, 0, 0, 0};
#pragma unroll 1
  for (int j = 0; j < 16; ++j) {
    const uint32_t o = o_base + j;
    if (o >= a.O) break;
    long long acc = (long long)(int)v[0][j];
#pragma unroll
    for (int pl = 1; pl < P; ++pl) acc += (long long)(int)v[pl][j] * (long long)(1 << (kDigitBits * pl));
    if (use_corr) acc += corr[j];
    const size_t oidx = a.out_nchw ? ((size_t)n * a.O + o) * ohow + pix : (size_t)m * a.O + o;
    if (a.acc_out) a.acc_out[oidx] = acc;
    if (a.q_out || a.f32_out) {
      int rb = 0;
      if (a.residual) {
        if (vec) rb = (int)((rw[j >> 2] >> (8 * (j & 3))) & 0xFFu);
        else rb = (int)((const uint8_t*)a.residual)[oidx];
        if (a.residual_dtype == PSB_DT_S8) rb = (int)(int8_t)rb;
      }
      const float y = dequant(acc, scb[j].x, scb[j].y, a.residual != nullptr, rb, a.residual_scale, a.relu != 0);
      if (a.f32_out) a.f32_out[oidx] = y;
      if (a.q_out) {
        const int q = requant(y, a.inv_step, a.qmin, a.qmax);
        if (vec) qw[j >> 2] |= ((uint32_t)q & 0xFFu) << (8 * (j & 3));
        else ((uint8_t*)a.q_out)[oidx] = (uint8_t)q;
      }
    }
  }
  if (vec && a.q_out)
    *reinterpret_cast<uint4*>((uint8_t*)a.q_out + (size_t)m * a.O + o_base) = make_uint4(qw[0], qw[1], qw[2], qw[3]);
}

// True when the layer takes the specialised epilogue loop below.
__host__ __device__ __forceinline__ bool uniform_epilogue(const TensorParams& p) {
  const ConvArgs& a = p.a;
  const bool q_only = a.q_out && !a.f32_out && !a.acc_out && (p.vec_ok || a.out_nchw) && a.inv_step > 0.0f;
  if (a.kmap) {
    // rows sorted by level: the same loop serves if every sampled level has the same number of digit planes
    uint32_t P0 = 0;
    for (uint32_t lv = 0; lv < (uint32_t)kMaxLevels; ++lv)
      if ((a.level_mask >> lv) & 1u) {
        if (P0 && p.planes[lv] != P0) return false;
        P0 = p.planes[lv];
      }
    return p.perm && q_only && P0 >= 2u && P0 <= 4u;
  }
  const uint32_t P0 = p.planes[a.uniform_log2k < (uint32_t)kMaxLevels ? a.uniform_log2k : 0u];
  return q_only && P0 >= 2u && P0 <= 4u;
}

// The same two functions on register copies of the few parameters they need.  Inside an out-of-line
// function the kernel's parameter block is reached through a generic pointer, and every asm statement
// with a memory clobber (barrier waits, TMEM loads) makes the compiler fetch such fields again: a
// dozen dependent loads per tile in the output-stage loop before the copies were made.  (Plain mode.)
struct RowMap {
  static constexpr int kTag = 1;     // distinguishes the row maps in template tags
  uint32_t M, O, ohow, planar;
  __device__ __forceinline__ void init(const TensorParams& p) {
    M = p.M; O = p.a.O; ohow = p.a.OH * p.a.OW; planar = p.a.out_nchw;
  }
  __device__ __forceinline__ uint32_t row_index(uint32_t m_tile, uint32_t row, bool* valid) const {
    const uint32_t m = m_tile * kTileM + row;
    *valid = m < M;
    return m;
  }
  __device__ __forceinline__ size_t offset(uint32_t m, uint32_t o_base) const {
    if (!planar) return (size_t)m * O + o_base;
    const uint32_t n = m / ohow;
    return ((size_t)n * O + o_base) * ohow + (m - n * ohow);
  }
};

// Band mode: rows of a tile are padded-linear positions of one image (tile_row_index above).
struct RowMapBand {
  static constexpr int kTag = 0;
  uint32_t tpi, tpi_magic, Wp, Wp_magic, OH, OW, O, ohow, planar;
  __device__ __forceinline__ void init(const TensorParams& p) {
    tpi = p.tpi; tpi_magic = p.tpi_magic; Wp = p.Wp; Wp_magic = p.Wp_magic;
    OH = p.a.OH; OW = p.a.OW; O = p.a.O; ohow = p.a.OH * p.a.OW; planar = p.a.out_nchw;
  }
  __device__ __forceinline__ uint32_t row_index(uint32_t m_tile, uint32_t row, bool* valid) const {
    const uint32_t n = __umulhi(m_tile, tpi_magic);
    const uint32_t t = (m_tile - n * tpi) * kTileM + row;
    const uint32_t oy = __umulhi(t, Wp_magic), ox = t - oy * Wp;
    *valid = oy < OH && ox < OW;
    return (n * OH + oy) * OW + ox;
  }
  __device__ __forceinline__ size_t offset(uint32_t m, uint32_t o_base) const {
    if (!planar) return (size_t)m * O + o_base;
    const uint32_t n = m / ohow;
    return ((size_t)n * O + o_base) * ohow + (m - n * ohow);
  }
};

// Whether the accumulators of level l stay below 2^31 in magnitude: (largest row sum of |W_k|, kept by the
// sampler in units of 256, each weight rounded up) x (largest activation magnitude).  Not used when an
// integer addend follows.  Warp-collective: the lanes share the scan over the rows.
__device__ __forceinline__ bool fits_32_bits(const TensorParams& p, uint32_t l) {
  if (!p.rowsum256 || p.corr[l] != nullptr) return false;
  const uint32_t* sums = p.rowsum256 + (size_t)l * p.a.O;
  uint32_t best = 0;
  for (uint32_t o = threadIdx.x & 31u; o < p.a.O; o += 32u) best = max(best, sums[o]);
  best = __reduce_max_sync(0xFFFFFFFFu, best);
  // (a sum that wrapped or was marked unknown reads as huge either way)
  return (unsigned long long)best * 256ull * (unsigned long long)p.amax < (1ull << 31) && best < (1u << 24);
}

// Rows sorted by level (per-location draw counts): row r of the matrix is location perm[r].
struct RowMapSorted {
  static constexpr int kTag = 2;
  const uint32_t* perm;
  uint32_t O, ohow, planar;
  __device__ __forceinline__ void init(const TensorParams& p) {
    perm = p.perm; O = p.a.O; ohow = p.a.OH * p.a.OW; planar = p.a.out_nchw;
  }
  __device__ __forceinline__ uint32_t row_index(uint32_t m_tile, uint32_t row, bool* valid) const {
    const uint32_t m = __ldcg(perm + (size_t)m_tile * kTileM + row);
    *valid = m != 0xFFFFFFFFu;
    return m;
  }
  __device__ __forceinline__ size_t offset(uint32_t m, uint32_t o_base) const {
    if (!planar) return (size_t)m * O + o_base;
    const uint32_t n = m / ohow;
    return ((size_t)n * O + o_base) * ohow + (m - n * ohow);
  }
};

// Epilogue loop of one warp for the common case: one draw count for the whole layer, only
// re-quantised bytes wanted.  The warp owns 32 rows (its TMEM lane quarter) x 16 channels of
// every tile.  Per tile: wait for the accumulator, pull the chunk into registers, hand the TMEM
// buffer back at once (the MMA of the tile after next can start), then do the arithmetic and
// the store.  Shortcut bytes are fetched one tile ahead.  RM maps the rows of a tile to output
// locations (plain tiles or band mode).  Returns true if a wait timed out.
template <int P, bool W32, int RES, bool FAST_U8, typename RM>
__device__ __noinline__ bool epilogue_uniform(const TensorParams& p, SharedCtl* ctl, uint32_t tmem_base,
                                              uint32_t ew, uint32_t lane, EpiConst c) {
  constexpr bool HAS_RES = RES != 0;
  // every instance of this loop gets its own instance of the out-of-line planar helpers (see load_planar16)
  constexpr int TAG = (((P * 2 + (W32 ? 1 : 0)) * 3 + RES) * 2 + (FAST_U8 ? 1 : 0)) * 2 + RM::kTag;
  const ConvArgs& a = p.a;
  const uint32_t quarter = ew & 3u, sub = ew >> 2;
  const uint32_t row = quarter * 32u + lane;
  constexpr bool kSorted = RM::kTag == 2;      // one level per tile, taken from the tile's mask
  uint32_t l = a.uniform_log2k;
  const bool use_corr = p.corr[kSorted ? (uint32_t)__ffs((int)(a.level_mask & 0x7Fu)) - 1u : l] != nullptr;
  WaitCtl* abort = &ctl->wait;
  const uint8_t* const res_base = (const uint8_t*)a.residual;
  uint8_t* const q_base = (uint8_t*)a.q_out;
  RM rm;
  rm.init(p);
  const float2* scb = ctl->scb[ew];
  const long long* corr = ctl->corr[ew];
  const bool vec16 = p.vec_ok == 2u, planar = rm.planar != 0u;
  const uint32_t ohow = rm.ohow;
  TileIter ti;
  ti.init(p);
  uint32_t pass = 0, cur_o_tile = 0xFFFFFFFFu;
  uint4 r_next = make_uint4(0, 0, 0, 0);
  // Sorted rows: the location of this thread's row and the tile's level are lookups in global memory.  They are
  // made one tile ahead (nx_*) and the shortcut fetch of the next tile, whose address depends on them, is issued
  // after the accumulator wait instead of before it, so that no address waits for a lookup.
  // (Without a shortcut nothing but the final store depends on the row's location, and looking ahead only
  // costs registers: measured slower.)
  constexpr bool kAhead = kSorted && HAS_RES;
  uint32_t nx_m = 0, nx_levels = 0;
  bool nx_ok = false;
  if (kSorted && ti.valid()) {
    if (kAhead) nx_m = rm.row_index(ti.m_tile, row, &nx_ok);
    nx_levels = tile_levels(p, ti.m_tile);
  }
  if (HAS_RES && ti.valid()) {
    bool ok_row;
    uint32_t m = nx_m;
    if (kAhead) ok_row = nx_ok; else m = rm.row_index(ti.m_tile, row, &ok_row);
    const uint32_t ob = ti.o_tile * kTileN + sub * 16u;
    if (ok_row && ob < rm.O) {
      const uint8_t* src = res_base + rm.offset(m, ob);
      r_next = planar ? load_planar16<TAG>(src, ohow, rm.O - ob) : load_row16(src, vec16, ob + 16u <= rm.O);
    }
  }
  while (ti.valid()) {
    bool row_valid = nx_ok;
    uint32_t m = nx_m;
    if (!kAhead) m = rm.row_index(ti.m_tile, row, &row_valid);
    const uint32_t o_tile = ti.o_tile;
    const uint32_t o_base = o_tile * kTileN + sub * 16u;
    const bool active = o_base < rm.O;          // warp-uniform
    if (kSorted) {
      // the tile's level; a tile without a sampled level gets no pass from the other roles either
      const uint32_t levels = nx_levels;
      if (!(levels & a.level_mask & 0x7Fu)) {
        if (row_valid) atomicOr(a.err, kDevErrBadLevel);     // a location asks for a level that was not sampled
        ti.next();
        if (ti.valid()) {
          if (kAhead) nx_m = rm.row_index(ti.m_tile, row, &nx_ok);
          nx_levels = tile_levels(p, ti.m_tile);
        }
        if (HAS_RES && ti.valid()) {
          const bool ok_row = nx_ok;
          const uint32_t mn = nx_m, ob = ti.o_tile * kTileN + sub * 16u;
          r_next = make_uint4(0, 0, 0, 0);
          if (ok_row && ob < rm.O) {
            const uint8_t* src = res_base + rm.offset(mn, ob);
            r_next = planar ? load_planar16<TAG>(src, ohow, rm.O - ob) : load_row16(src, vec16, ob + 16u <= rm.O);
          }
        }
        continue;
      }
      l = (uint32_t)__ffs((int)(levels & a.level_mask & 0x7Fu)) - 1u;
    }
    ti.next();
    if (kSorted && ti.valid()) {
      if (kAhead) nx_m = rm.row_index(ti.m_tile, row, &nx_ok);
      nx_levels = tile_levels(p, ti.m_tile);
    }
    if ((kSorted ? o_tile * 8u + l : o_tile) != cur_o_tile) {
      // per-channel constants of this channel tile: the warp keeps its own copy of its 16 channels
      __syncwarp();
      if (lane < 16u) {
        const uint32_t o = o_base + lane;
        float2 sb = make_float2(0.f, 0.f);
        long long cr = 0;
        if (o < a.O) {
          sb.x = ldexpf(a.scale[o], a.e_base[o] - (int)l);
          sb.y = a.bias[o];
          if (use_corr) cr = p.corr[l][o];
        }
        ctl->scb[ew][lane] = sb;
        ctl->corr[ew][lane] = cr;
      }
      cur_o_tile = kSorted ? o_tile * 8u + l : o_tile;
      __syncwarp();
    }
    const uint4 r_cur = r_next;
    if (HAS_RES && !kAhead && ti.valid()) {
      bool ok_row;
      const uint32_t mn = rm.row_index(ti.m_tile, row, &ok_row), ob = ti.o_tile * kTileN + sub * 16u;
      r_next = make_uint4(0, 0, 0, 0);
      if (ok_row && ob < rm.O) {
        const uint8_t* src = res_base + rm.offset(mn, ob);
        r_next = planar ? load_planar16<TAG>(src, ohow, rm.O - ob) : load_row16(src, vec16, ob + 16u <= rm.O);
      }
    }
    const uint32_t buf = pass & 1u, aph = (pass >> 1) & 1u;
    const bool ok = mbar_wait(smem_u32(&ctl->acc_full[buf]), aph, abort, 32);
    if (__any_sync(0xFFFFFFFFu, !ok)) return true;
    tc_fence_after();
    uint32_t v[P][16];
    if (active) {
      const uint32_t taddr = tmem_base + buf * kTmemBufStride + ((quarter * 32u) << 16) + sub * 16u;
      load_chunk<P, W32>(taddr, v);
    }
    // the chunk is in registers: give the accumulator buffer back before doing the arithmetic
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[buf]));
    if (kAhead && ti.valid()) {
      const uint32_t ob = ti.o_tile * kTileN + sub * 16u;
      r_next = make_uint4(0, 0, 0, 0);
      if (nx_ok && ob < rm.O) {
        const uint8_t* src = res_base + rm.offset(nx_m, ob);
        r_next = planar ? load_planar16<TAG>(src, ohow, rm.O - ob) : load_row16(src, vec16, ob + 16u <= rm.O);
      }
    }
    if (active && row_valid) {
      const uint4 q16 = chunk_math<P, W32, RES, FAST_U8>(v, r_cur, scb, corr, c);
      uint8_t* dst = q_base + rm.offset(m, o_base);
      if (planar) store_planar16<TAG>(dst, ohow, rm.O - o_base, q16);
      else store_row16(dst, q16, vec16, o_base + 16u <= rm.O);
    }
    ++pass;
  }
  return false;
}

// Run-time options of the uniform output stage -> template instance.
template <int P, bool W32, int RES>
__device__ __forceinline__ bool uniform_dispatch_tail(const TensorParams& p, SharedCtl* ctl, uint32_t tmem_base,
                                                      uint32_t ew, uint32_t lane, const EpiConst& c, bool fast_u8) {
  if (p.band)
    return fast_u8 ? epilogue_uniform<P, W32, RES, true, RowMapBand>(p, ctl, tmem_base, ew, lane, c)
                   : epilogue_uniform<P, W32, RES, false, RowMapBand>(p, ctl, tmem_base, ew, lane, c);
  if (p.perm)
    return fast_u8 ? epilogue_uniform<P, W32, RES, true, RowMapSorted>(p, ctl, tmem_base, ew, lane, c)
                   : epilogue_uniform<P, W32, RES, false, RowMapSorted>(p, ctl, tmem_base, ew, lane, c);
  return fast_u8 ? epilogue_uniform<P, W32, RES, true, RowMap>(p, ctl, tmem_base, ew, lane, c)
                 : epilogue_uniform<P, W32, RES, false, RowMap>(p, ctl, tmem_base, ew, lane, c);
}
template <int P>
__device__ __forceinline__ bool uniform_dispatch(const TensorParams& p, SharedCtl* ctl, uint32_t tmem_base,
                                                 uint32_t ew, uint32_t lane, const EpiConst& c, bool fast_u8,
                                                 bool w32, uint32_t res) {
  if (w32) {
    if (res == 0u) return uniform_dispatch_tail<P, true, 0>(p, ctl, tmem_base, ew, lane, c, fast_u8);
    if (res == 1u) return uniform_dispatch_tail<P, true, 1>(p, ctl, tmem_base, ew, lane, c, fast_u8);
    return uniform_dispatch_tail<P, true, 2>(p, ctl, tmem_base, ew, lane, c, fast_u8);
  }
  if (res == 0u) return uniform_dispatch_tail<P, false, 0>(p, ctl, tmem_base, ew, lane, c, fast_u8);
  if (res == 1u) return uniform_dispatch_tail<P, false, 1>(p, ctl, tmem_base, ew, lane, c, fast_u8);
  return uniform_dispatch_tail<P, false, 2>(p, ctl, tmem_base, ew, lane, c, fast_u8);
}

// The MMA issuing role, one thread of warp kMmaWarp0 (mine = 0) and one of kMmaWarp1 (mine = 1).
// Both walk the same sequence of passes and ring stages; stage uses are numbered through the
// whole kernel and the number's parity selects the thread.  The thread that owns the first
// stage of a pass waits for the accumulator buffer and issues the zeroing MMA; the other one
// joins the pass after that (`started`).  Integer accumulation is exact, so the order in
// which the two threads' MMAs reach the accumulator is immaterial.  A parity wait on a stage
// barrier is meaningful while the waiter is less than two uses of that stage ahead of it; the
// ring has an even number of stages, so a thread always meets the same slots and its wait for
// a slot follows its own previous use of that slot.  Kept out of line and fed from local copies of
// the parameters so that its loop state lives in registers: the pipe idles for every clock this
// thread spends between two MMAs beyond what the other thread covers.  Returns true on a timeout.
//
// Passes of a single stage are issued in their order: the first MMA of a pass follows the last but one K block
// of the pass before it (`pass_issued`; the waits for the stage and the accumulator buffer are done by then).  Without
// the rule both threads issue at once whenever both have a stage ready, the MMAs of two tiles interleave in
// the pipe, both tiles complete late and together, and the pipe then idles until the output stage has
// emptied an accumulator buffer.
template <int BK>
__device__ __noinline__ bool mma_role(const TensorParams& p, SharedCtl* ctl, uint32_t tmem_base, uint32_t ring_addr,
                                      uint32_t planes_addr, uint32_t stage_bytes, uint32_t sub_bytes,
                                      uint32_t k_iters, uint32_t mine) {
  WaitCtl* abort = &ctl->wait;
  const uint32_t group = p.group, stages = p.stages, resident = p.resident, stage_bytes_a = p.stage_bytes_a;
  const uint32_t level_mask = p.a.level_mask;
  const uint32_t n_groups = (k_iters + group - 1) / group;
  const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
  const uint32_t acc_full0 = smem_u32(&ctl->acc_full[0]), acc_empty0 = smem_u32(&ctl->acc_empty[0]);
  const uint32_t started0 = smem_u32(&ctl->started[0]);
  const uint32_t pass_issued = smem_u32(&ctl->pass_issued);
  // (passes of several stages already have both threads at work on the same pass in turns; there the rule
  // only took the overlap at the pass boundaries away and cost a few per cent)
  const bool ordered = n_groups == 1u;
  const uint32_t desc_hi = smem_desc_hi(BK);
  // resident digit planes: K blocks below planes_upto are known to have landed
  const uint32_t plane_part = (k_iters + kPlaneBars - 1) / kPlaneBars;
  uint32_t planes_ready = 0, planes_upto = resident ? 0u : 0xFFFFFFFFu;
  uint32_t s = 0, ph = 0, pass = 0, use = 0;
  TileIter ti;
  for (ti.init(p); ti.valid(); ti.next()) {
    const uint32_t levels = tile_levels(p, ti.m_tile) & level_mask;
    for (uint32_t todo = levels & 0x7Fu; todo; todo &= todo - 1u) {
      const uint32_t l = (uint32_t)__ffs((int)todo) - 1u;
      const uint32_t P = p.planes[l];
      const uint32_t buf = pass & 1u, aph = (pass >> 1) & 1u;
      // instruction descriptor: s32 accumulators, s8 x s8, both K-major, M = 128, N = P * 64
      const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | (((P * kTileN) >> 3) << 17) |
                             ((kTileM >> 4) << 24);
      const uint32_t d_tmem = tmem_base + buf * kTmemBufStride;
      const uint32_t blk = P * kTileN * BK;
      bool joined = (use & 1u) == mine;
      if (joined) {
        if (!mbar_wait(acc_empty0 + 8u * buf, aph ^ 1u, abort)) return true;
        tc_fence_after();
      }
      uint32_t b_res = planes_addr, g = 0;
      for (uint32_t it = 0; it < k_iters; ++g, ++use) {
        const uint32_t cnt = min(group, k_iters - it);
        if ((use & 1u) == mine) {
          if (!joined) {
            if (!mbar_wait(started0 + 8u * buf, aph, abort)) return true;
            joined = true;
          }
          if (!mbar_wait(full0 + 8u * s, ph, abort)) return true;
          while (it + cnt > planes_upto) {
            if (!mbar_wait(smem_u32(&ctl->planes_full[planes_ready]), 0u, abort)) return true;
            ++planes_ready;
            planes_upto = planes_ready == (uint32_t)kPlaneBars ? 0xFFFFFFFFu : planes_upto + plane_part;
          }
          if (ordered && pass != 0u) {
            if (!mbar_wait(pass_issued, (pass - 1u) & 1u, abort, kNoSleep)) return true;
          }
          tc_fence_after();
          // K blocks of the stage: activation tiles sub_bytes apart, planes beside them or resident; only the
          // low words of the descriptors move (by bytes / 16)
          uint32_t a_lo = smem_desc_lo(ring_addr + s * stage_bytes);
          uint32_t b_lo = resident ? smem_desc_lo(b_res) : a_lo + (stage_bytes_a >> 4);
          const uint32_t a_step = sub_bytes >> 4, b_step = resident ? blk >> 4 : sub_bytes >> 4;
          for (uint32_t j = 0; j < cnt; ++j, a_lo += a_step, b_lo += b_step) {
            // the pass after this one may start under this pass's last K block
            if (ordered && j + 1u == cnt) mbar_arrive(pass_issued);
            if (it == 0 && j == 0) {
              tc_mma_i8_zero(d_tmem, a_lo, b_lo, desc_hi, idesc);
#pragma unroll
              for (int ks = 1; ks < BK / 32; ++ks) tc_mma_i8_acc(d_tmem, a_lo + 2 * ks, b_lo + 2 * ks, desc_hi, idesc);
            } else {
#pragma unroll
              for (int ks = 0; ks < BK / 32; ++ks) tc_mma_i8_acc(d_tmem, a_lo + 2 * ks, b_lo + 2 * ks, desc_hi, idesc);
            }
          }
          if (it == 0 && n_groups > 1u) {
            tc_fence_before();
            mbar_arrive(started0 + 8u * buf);
          }
          tc_commit(empty0 + 8u * s);
          // this thread's last stage of the pass: the last or the last but one
          if (g + 2u >= n_groups) tc_commit(acc_full0 + 8u * buf);
        }
        b_res += cnt * blk;
        it += cnt;
        if (++s == stages) { s = 0; ph ^= 1u; }
      }
      ++pass;
    }
  }
  return false;
}

// The same role in band mode, where a ring stage holds the band of a whole tile: both threads work on every
// tile, thread 0 on the first half of its MMAs (taps x K steps), thread 1 on the second half, both into the
// one accumulator (the order of integer additions is immaterial).  One thread alone needs about 115 clocks
// per MMA where the pipe needs 96, and a hand-over between tiles costs a few hundred more; two threads on
// the same tile keep the pipe fed and the tiles in order.  Thread 0 issues the zeroing MMA first (`started`);
// both commit to the stage's and the accumulator's barriers (count 2 in this mode).  The descriptor offsets of
// a thread's MMAs are computed once (a table in shared memory, read a few entries ahead of the MMAs); the
// issue loop then spends two additions per MMA.
template <int BK>
__device__ __noinline__ bool mma_role_band(const TensorParams& p, SharedCtl* ctl, uint32_t tmem_base,
                                           uint32_t ring_addr, uint32_t planes_addr, uint32_t stage_bytes,
                                           uint32_t mine) {
  WaitCtl* abort = &ctl->wait;
  const uint32_t stages = p.stages, row_bytes = p.Wp * p.a.C, KH = p.a.KH, KW = p.a.KW;
  const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
  const uint32_t acc_full0 = smem_u32(&ctl->acc_full[0]), acc_empty0 = smem_u32(&ctl->acc_empty[0]);
  const uint32_t started0 = smem_u32(&ctl->started[0]);
  const uint32_t desc_hi = smem_desc_hi(BK);
  const uint32_t P = p.planes[p.a.uniform_log2k];
  const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | (((P * kTileN) >> 3) << 17) | ((kTileM >> 4) << 24);
  const uint32_t blk = P * kTileN * BK;
  constexpr uint32_t kSteps = BK / 32;
  const uint32_t n_mmas = KH * KW * kSteps, half = (n_mmas + 1u) / 2u;
  const uint32_t j_begin = mine ? half : 0u, cnt = mine ? n_mmas - half : half;
  uint2* const tab = ctl->tap_tab[mine];
  for (uint32_t i = 0; i < (cnt + kTapBatch - 1) / kTapBatch * kTapBatch; ++i) {
    const uint32_t j = j_begin + i, tap = j / kSteps, ks = j - tap * kSteps, kh = tap / KW, kw = tap - kh * KW;
    tab[i] = i < cnt ? make_uint2((kh * row_bytes + kw * (uint32_t)BK + ks * 32u) >> 4, (tap * blk + ks * 32u) >> 4)
                     : make_uint2(0u, 0u);
  }
  // resident digit planes arrive in kPlaneBars parts of `plane_part` K blocks (= taps): this thread needs the
  // parts up to the one that holds its last tap
  const uint32_t k_iters = KH * KW, plane_part = (k_iters + kPlaneBars - 1) / kPlaneBars;
  const uint32_t parts_needed = min((uint32_t)kPlaneBars, (j_begin + cnt - 1u) / kSteps / plane_part + 1u);
  const uint32_t planes_lo = smem_desc_lo(planes_addr);
  uint32_t s = 0, ph = 0, pass = 0;
  TileIter ti;
  for (ti.init(p); ti.valid(); ti.next(), ++pass) {
    const uint32_t buf = pass & 1u, aph = (pass >> 1) & 1u;
    const uint32_t d_tmem = tmem_base + buf * kTmemBufStride;
    // byte offset of the tile's first position in its band
    const uint32_t t0 = (ti.m_tile - __umulhi(ti.m_tile, p.tpi_magic) * p.tpi) * kTileM;
    const uint32_t band_off = (t0 - __umulhi(t0, p.Wp_magic) * p.Wp) * (uint32_t)BK;
    if (!mbar_wait(acc_empty0 + 8u * buf, aph ^ 1u, abort)) return true;
    if (mine && !mbar_wait(started0 + 8u * buf, aph, abort, kNoSleep)) return true;
    if (!mbar_wait(full0 + 8u * s, ph, abort)) return true;
    if (pass == 0u)
      for (uint32_t b = 0; b < parts_needed; ++b)
        if (!mbar_wait(smem_u32(&ctl->planes_full[b]), 0u, abort)) return true;
    tc_fence_after();
    const uint32_t a0 = smem_desc_lo(ring_addr + s * stage_bytes + band_off);
    for (uint32_t i0 = 0; i0 < cnt; i0 += kTapBatch) {
      uint2 t[kTapBatch];
#pragma unroll
      for (int j = 0; j < kTapBatch; ++j) t[j] = tab[i0 + j];
#pragma unroll
      for (int j = 0; j < kTapBatch; ++j) {
        if (i0 + (uint32_t)j >= cnt) break;
        if (j == 0 && i0 == 0u && !mine) {
          tc_mma_i8_zero(d_tmem, a0 + t[0].x, planes_lo + t[0].y, desc_hi, idesc);
          tc_fence_before();
          mbar_arrive(started0 + 8u * buf);
        } else {
          tc_mma_i8_acc(d_tmem, a0 + t[j].x, planes_lo + t[j].y, desc_hi, idesc);
        }
      }
    }
    tc_commit(empty0 + 8u * s);
    tc_commit(acc_full0 + 8u * buf);
    if (++s == stages) { s = 0; ph ^= 1u; }
  }
  return false;
}

// kGeneral: which output stage the instance carries, the loop for the common case (uniform_epilogue) or the
// general one; the host picks the instance, so neither drags the other's code and registers along.
template <int BK, bool kGeneral>
__global__ void __launch_bounds__(kThreadsTensor, 1)
psb_mma_kernel(const __grid_constant__ TmapSet maps, const __grid_constant__ TensorParams p) {
  extern __shared__ uint8_t smem_raw[];
  // stage buffers need 1024-byte alignment for the 128-byte swizzle pattern
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023u) & ~(uintptr_t)1023u);
  // resident mode: [digit planes of all K blocks][ring of activation stages][control]
  // streaming mode: [ring of (activation, planes) stages][control]
  uint8_t* ring = smem + (p.resident ? p.resident_bytes : 0u);
  // a stage holds `group` K blocks, each an activation tile followed (streaming mode) by planes
  const uint32_t sub_bytes = p.stage_bytes_a + (p.resident ? 0u : p.stage_bytes_b_max);
  const uint32_t stage_bytes = p.band ? p.band_bytes : sub_bytes * p.group;
  SharedCtl* ctl = reinterpret_cast<SharedCtl*>(ring + (size_t)p.stages * stage_bytes);

  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  const uint32_t k_iters = p.a.KH * p.a.KW * p.n_cb;

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), p.band ? 2u : 1u);     // band mode: both issuing threads use every stage
    }
    for (int b = 0; b < 2; ++b) {
      // both issuing threads commit to it when a pass has more than one stage, and in band mode
      mbar_init(smem_u32(&ctl->acc_full[b]), (p.band || (k_iters + p.group - 1) / p.group > 1u) ? 2u : 1u);
      mbar_init(smem_u32(&ctl->acc_empty[b]), kEpilogueWarps);
    }
    {  // part b of the resident planes holds K blocks [b * part, (b + 1) * part): one arrival per block
      const uint32_t part = (k_iters + kPlaneBars - 1) / kPlaneBars;
      for (uint32_t b = 0; b < (uint32_t)kPlaneBars; ++b) {
        const uint32_t lo = b * part, hi = min(lo + part, k_iters);
        mbar_init(smem_u32(&ctl->planes_full[b]), hi > lo ? hi - lo : 1u);
      }
    }
    for (int b = 0; b < 2; ++b) mbar_init(smem_u32(&ctl->started[b]), 1);
    mbar_init(smem_u32(&ctl->pass_issued), 1);
    ctl->wait.abort = 0;
    ctl->wait.limit = p.wait_limit;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x == 32) {
    // descriptor fetches of the first copies would otherwise sit on the critical path of the first tile
    asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.a) : "memory");
  }
  if (warp == kMmaWarp1) {
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
  WaitCtl* abort = &ctl->wait;
  bool failed = false;
  // The kernel is launched with programmatic stream serialisation: a CTA may get here while the
  // kernel before it in the stream is still draining.  Nothing above touches global memory; from
  // here on everything does (activations, planes, constants, outputs), so every thread waits for
  // the earlier grids to complete and their writes to be visible.  The kernel after this one may
  // be scheduled as soon as SMs free up (it waits at the same point).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp < (uint32_t)kProducerWarps) {
    // ----------------------------------------------------------- producers
    // A copy instruction holds its thread for a few hundred clocks, whatever its size, while the
    // copy engine takes several at a time: the K blocks of a stage are therefore issued by as
    // many lanes of the warp in one go (lane j copies block j), after lane 0 has waited for the
    // stage and posted the byte count; and the producer warps take the stages in turns (all of
    // them walk the same sequence of stages, each issues every second one).
    uint32_t s = 0, ph = 0;   // ring position and phase of the current stage use
    uint32_t turn = 0;        // whose turn it is among the producer warps
    const uint32_t ring_addr = smem_u32(ring);
    TileIter ti;
    for (ti.init(p); ti.valid() && !failed; ti.next()) {
      const uint32_t m_tile = ti.m_tile, o_tile = ti.o_tile;
      const uint32_t m0 = m_tile * kTileM;
      const uint32_t levels = tile_levels(p, ti.m_tile) & p.a.level_mask;
      // image coordinates of the tile's first row: divisions, so only the warp that is about to
      // issue a copy of this tile computes them
      uint32_t n0 = 0;
      int h0 = 0, w0 = 0;
      bool have_coords = !p.im2col || p.band;
      // one pass per level present in the tile (levels that were not sampled are flagged by the
      // epilogue and skipped by every role)
      for (uint32_t todo = levels & 0x7Fu; todo && !failed; todo &= todo - 1u) {
        const uint32_t l = (uint32_t)__ffs((int)todo) - 1u;
        const uint32_t P = p.planes[l];
        const uint32_t bytes = p.stage_bytes_a + (p.resident ? 0u : P * kTileN * BK);
        const uint32_t blk = P * kTileN * BK;
        const int8_t* b_tiles = p.planes_ptr[l] + (size_t)o_tile * k_iters * blk;   // this channel tile's K blocks
        for (uint32_t it = 0; it < k_iters;) {
          const uint32_t cnt = min(p.group, k_iters - it);
          if (turn == warp) {
            if (!have_coords) {
              const uint32_t ohow = p.a.OH * p.a.OW;
              n0 = m0 / ohow;
              const uint32_t rem = m0 - n0 * ohow, oy = rem / p.a.OW;
              h0 = (int)(oy * p.a.stride) - (int)p.a.pad;
              w0 = (int)((rem - oy * p.a.OW) * p.a.stride) - (int)p.a.pad;
              have_coords = true;
            }
            const uint32_t bar = smem_u32(&ctl->full[s]);
            bool ok = true;
            if (lane == 0) {
              ok = mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1u, abort);
              if (ok) mbar_expect_tx(bar, p.band ? p.band_rows * p.Wp * p.a.C : bytes * cnt);
            }
            if (!__shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0)) { failed = true; break; }
            if (p.band) {
              // one copy per tile: the band of padded input rows that holds every tap of the tile;
              // rows and columns outside the image read as zeros
              if (lane == 0) {
                const uint32_t n = __umulhi(m_tile, p.tpi_magic);
                const uint32_t r0 = __umulhi((m_tile - n * p.tpi) * kTileM, p.Wp_magic);
                tma_load_4d(ring_addr + s * stage_bytes, &maps.a, bar, 0, -(int)p.a.pad, (int)r0 - (int)p.a.pad, (int)n);
              }
            } else if (lane < cnt) {
              // K block it + lane: tap (kh, kw), channel block cb, column kcol of the plane matrix
              const uint32_t kb = it + lane;
              const uint32_t tap = kb / p.n_cb, cb = kb - tap * p.n_cb;
              const uint32_t kh = tap / p.a.KW, kw = tap - kh * p.a.KW;
              const uint32_t dst = ring_addr + s * stage_bytes + lane * sub_bytes;
              if (p.im2col)
                tma_load_im2col_4d(dst, &maps.a, bar, (int)(cb * BK), w0, h0, (int)n0, (uint16_t)kw, (uint16_t)kh);
              else
                tma_load_2d(dst, &maps.a, bar, (int)(cb * BK), (int)m0);
              if (!p.resident) bulk_load(dst + p.stage_bytes_a, b_tiles + (size_t)kb * blk, blk, bar);
            }
          }
          it += cnt;
          if (++s == p.stages) { s = 0; ph ^= 1u; }
          if (++turn == (uint32_t)kProducerWarps) turn = 0;
        }
      }
    }
  } else if (warp == (uint32_t)kMmaWarp0 || warp == (uint32_t)kMmaWarp1) {
    // ---------------------------------------------------------------- MMA
    if (lane == 0)
      failed = p.band ? mma_role_band<BK>(p, ctl, tmem_base, smem_u32(ring), smem_u32(smem), stage_bytes,
                                          warp - (uint32_t)kMmaWarp0)
                      : mma_role<BK>(p, ctl, tmem_base, smem_u32(ring), smem_u32(smem), stage_bytes, sub_bytes, k_iters,
                                     warp - (uint32_t)kMmaWarp0);
    failed = __shfl_sync(0xFFFFFFFFu, failed ? 1 : 0, 0) != 0;
  } else {
    // ----------------------------------------------------------- epilogue
    // 16 warps: warp & 3 selects the TMEM lane quarter (32 rows), ew >> 2 the 16 of the tile's 64
    // channels.
    const uint32_t ew = warp - (uint32_t)kFirstEpilogueWarp;   // 0..15
    const uint32_t quarter = ew & 3u;
    const uint32_t sub = ew >> 2;
    const uint32_t row = quarter * 32u + lane;
    const ConvArgs& a = p.a;
    const bool q_only = a.q_out && !a.f32_out && !a.acc_out && (p.vec_ok || a.out_nchw) && a.inv_step > 0.0f;
    EpiConst ec;
    ec.res_scale = a.residual_scale;
    // With inv_step > 0 (a condition of the fast paths) max(y, 0) * inv_step == max(y * inv_step, 0):
    // the relu is folded into the lower clamp bound.
    ec.inv_step = a.inv_step;
    ec.lo_f = (a.relu && a.qmin < 0) ? 0.0f : (float)a.qmin;
    ec.hi_f = (float)a.qmax;
    ec.out_signed = a.out_dtype == PSB_DT_S8 ? 1u : 0u;
    // unsigned codes from 0 up: the byte saturation of the packing instruction is the lower clamp
    const bool fast_u8 = a.out_dtype == PSB_DT_U8 && a.qmin == 0;
    const uint32_t res_kind = !a.residual ? 0u : (a.residual_dtype == PSB_DT_S8 ? 2u : 1u);
    uint32_t P0 = p.planes[a.uniform_log2k < (uint32_t)kMaxLevels ? a.uniform_log2k : 0u];
    if (a.kmap) P0 = p.planes[(uint32_t)__ffs((int)(a.level_mask & 0x7Fu)) - 1u];
    if (p.resident && lane == 0) {
      // the digit planes of this CTA's channel tile, all K blocks, once: the epilogue warps have
      // nothing else to do yet, and sixteen threads get the copies under way sooner than one
      const uint32_t o_tile = blockIdx.x / p.ctas_per_otile;
      const uint32_t blk = P0 * kTileN * BK;
      const uint32_t part = (k_iters + kPlaneBars - 1) / kPlaneBars;
      for (uint32_t it = ew; it < k_iters; it += (uint32_t)kEpilogueWarps) {
        const uint32_t bar = smem_u32(&ctl->planes_full[it / part]);
        mbar_expect_tx(bar, blk);
        bulk_load(smem_u32(smem) + it * blk, p.planes_ptr[a.uniform_log2k] + ((size_t)o_tile * k_iters + it) * blk, blk,
                  bar);
      }
    }
    if (!kGeneral) {
      bool w32 = true;
      if (a.kmap) {          // every level a tile may have must fit
        for (uint32_t lv = 0; lv < (uint32_t)kMaxLevels; ++lv)
          if ((a.level_mask >> lv) & 1u) w32 = fits_32_bits(p, lv) && w32;
      } else {
        w32 = fits_32_bits(p, a.uniform_log2k);
      }
      if (P0 == 4u) failed = uniform_dispatch<4>(p, ctl, tmem_base, ew, lane, ec, fast_u8, w32, res_kind);
      else if (P0 == 3u) failed = uniform_dispatch<3>(p, ctl, tmem_base, ew, lane, ec, fast_u8, w32, res_kind);
      else failed = uniform_dispatch<2>(p, ctl, tmem_base, ew, lane, ec, fast_u8, w32, res_kind);
    } else {
      // general loop: per-location draw counts, any outputs and layouts, ragged channel counts
      const float2* scb = ctl->scb[ew];
      const long long* corr = ctl->corr[ew];
      uint32_t pass = 0, cur_key = 0xFFFFFFFFu;
      uint32_t w32_levels = 0;      // levels whose accumulators are known to fit 32 bits
      if (q_only)
        for (uint32_t l = 0; l < (uint32_t)kMaxLevels; ++l)
          if (((a.level_mask >> l) & 1u) && fits_32_bits(p, l)) w32_levels |= 1u << l;
      TileIter ti;
      for (ti.init(p); !failed && ti.valid(); ti.next()) {
        const uint32_t m0 = ti.m_tile * kTileM, o_tile = ti.o_tile;
        const uint32_t levels = tile_levels(p, ti.m_tile) & a.level_mask;
        uint32_t m = m0 + row;
        bool in_range = m < p.M;
        if (p.perm) {           // rows sorted by level: the location of this row
          m = p.perm[m0 + row];
          in_range = m != 0xFFFFFFFFu;
        }
        const uint32_t my_level = in_range ? (a.kmap ? (uint32_t)a.kmap[m] : a.uniform_log2k) : 0xFFu;
        if (in_range && (my_level >= (uint32_t)kMaxLevels || !((a.level_mask >> my_level) & 1u)))
          atomicOr(a.err, kDevErrBadLevel);
        const uint32_t o_base = o_tile * kTileN + sub * 16u;
        const size_t oidx = (size_t)m * a.O + o_base;
        const bool vec16 = p.vec_ok == 2u, both = o_base + 16u <= a.O;
        const bool fast = q_only && !a.out_nchw && o_base < a.O;
        uint4 r4 = make_uint4(0, 0, 0, 0);
        if (fast && a.residual && in_range) r4 = load_row16((const uint8_t*)a.residual + oidx, vec16, both);
        for (uint32_t todo = levels & 0x7Fu; todo && !failed; todo &= todo - 1u) {
          const uint32_t l = (uint32_t)__ffs((int)todo) - 1u;
          const uint32_t P = p.planes[l];
          const uint32_t buf = pass & 1u, aph = (pass >> 1) & 1u;
          const bool use_corr = p.corr[l] != nullptr;
          // per-channel constants of this (channel tile, level), refreshed only when the pair changes
          const uint32_t key = o_tile * 8u + l;
          if (key != cur_key) {
            __syncwarp();
            if (lane < 16u) {
              const uint32_t o = o_base + lane;
              float2 sb = make_float2(0.f, 0.f);
              long long cr = 0;
              if (o < a.O) {
                sb.x = ldexpf(a.scale[o], a.e_base[o] - (int)l);
                sb.y = a.bias[o];
                if (use_corr) cr = p.corr[l][o];
              }
              ctl->scb[ew][lane] = sb;
              ctl->corr[ew][lane] = cr;
            }
            cur_key = key;
            __syncwarp();
          }
          const bool ok = mbar_wait(smem_u32(&ctl->acc_full[buf]), aph, abort, 32);
          failed = __any_sync(0xFFFFFFFFu, !ok) != 0;
          if (failed) break;
          tc_fence_after();
          const uint32_t taddr = tmem_base + buf * kTmemBufStride + ((quarter * 32u) << 16) + sub * 16u;
          const bool valid = in_range && my_level == l;
          if (o_base < a.O) {
            if (fast) {
              uint8_t* q_dst = (uint8_t*)a.q_out + oidx;
              const bool w32 = ((w32_levels >> l) & 1u) != 0u;
#define PSB_EPI(PV, WV, RV) epilogue_chunk_q<PV, WV, RV>(taddr, valid, q_dst, r4, vec16, both, scb, corr, ec)
#define PSB_EPI_P(WV, RV)                                                                          \
  do {                                                                                             \
    if (P == 4) PSB_EPI(4, WV, RV); else if (P == 3) PSB_EPI(3, WV, RV);                           \
    else if (P == 2) PSB_EPI(2, WV, RV); else PSB_EPI(1, WV, RV);                                  \
  } while (0)
              if (w32) {
                if (res_kind == 0u) PSB_EPI_P(true, 0); else if (res_kind == 1u) PSB_EPI_P(true, 1); else PSB_EPI_P(true, 2);
              } else {
                if (res_kind == 0u) PSB_EPI_P(false, 0); else if (res_kind == 1u) PSB_EPI_P(false, 1); else PSB_EPI_P(false, 2);
              }
#undef PSB_EPI_P
#undef PSB_EPI
            } else {
              const uint32_t ohow = a.OH * a.OW;
              const uint32_t n = in_range ? m / ohow : 0u, pix = in_range ? m % ohow : 0u;
              switch (P) {
                case 1: epilogue_chunk<1>(p, taddr, o_base, m, valid, n, pix, scb, corr, use_corr); break;
                case 2: epilogue_chunk<2>(p, taddr, o_base, m, valid, n, pix, scb, corr, use_corr); break;
                case 3: epilogue_chunk<3>(p, taddr, o_base, m, valid, n, pix, scb, corr, use_corr); break;
                default: epilogue_chunk<4>(p, taddr, o_base, m, valid, n, pix, scb, corr, use_corr); break;
              }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[buf]));
          ++pass;
        }
      }
    }
  }

  // ------------------------------------------------------------- common exit
  if (failed) {
    if (lane == 0) {
      abort->abort = 1u;
      atomicOr(p.a.err, kDevErrTimeout);
    }
    // give copies and MMAs already in flight time to land before the CTA retires
    for (int i = 0; i < 64; ++i) __nanosleep(2000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(kTmemCols)
                 : "memory");
  }
}

// One warp waits, with the given bound, on a barrier that has no other party: the wait runs out,
// the kernel raises the error word and returns.  Exercises mbar_wait's give-up path as the contraction
// kernel would take it, with nothing in flight.
__global__ void wait_selftest_kernel(unsigned long long limit, uint32_t* __restrict__ err) {
  __shared__ unsigned long long bar;
  __shared__ WaitCtl wc;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    wc.abort = 0;
    wc.limit = limit;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) ok = mbar_wait(smem_u32(&bar), 0u, &wc);
  if (!ok) {
    wc.abort = 1u;
    atomicOr(err, kDevErrTimeout);
  }
  __syncthreads();
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
constexpr int kMaxDevicesForAttr = 64;

}  // namespace

cudaError_t launch_wait_selftest(psb_ctx* ctx, cudaStream_t s) {
  wait_selftest_kernel<<<1, 32, 0, s>>>(ctx->wait_limit_cycles, ctx->err_dev);
  note_launch();
  return cudaGetLastError();
}

psb_status tensor_supported(const psb_ctx* ctx, const psb_weights* wt, const ConvArgs& a) {
  if (!ctx->encode_tiled || !ctx->encode_im2col) return PSB_ERR_UNSUPPORTED;
  if (!wt->has_planes || a.groups != 1) return PSB_ERR_UNSUPPORTED;
  // each plane accumulates in 32 bits: |digit| <= 127, |x| <= 128
  if ((uint64_t)wt->d * 127ull * 128ull >= (1ull << 31)) return PSB_ERR_UNSUPPORTED;
  if (wt->packed_k) {
    // the gather kernel stages the input-row segments of a strip of output locations in 48 KB of shared memory
    return (a.KH > 120u || im2col_s8_smem(a, wt->run_pitch) > 48u * 1024u) ? PSB_ERR_UNSUPPORTED : PSB_OK;
  }
  if (a.C % 16u || a.C < 32u) return PSB_ERR_UNSUPPORTED;
  if ((uintptr_t)a.x & 15u) return PSB_ERR_UNSUPPORTED;
  if (a.stride > 8 || a.pad > 127 || a.KH > 128 || a.KW > 128) return PSB_ERR_UNSUPPORTED;
  return PSB_OK;
}

psb_status launch_tensor(psb_ctx* ctx, const psb_weights* wt, const ConvArgs& a, uint32_t amax,
                         bool add_corr128, const SortedRows* sorted, cudaStream_t s) {
  TmapSet maps;
  TensorParams p;
  p.a = a;
  p.wait_limit = ctx->wait_limit_cycles;
  p.M = a.N * a.OH * a.OW;
  p.m_tiles = (p.M + kTileM - 1) / kTileM;
  p.o_tiles = wt->o_tiles;
  const uint32_t bk = wt->bk;
  p.n_cb = (a.C + bk - 1) / bk;
  p.im2col = is_plain_gemm(a) ? 0u : 1u;
  uint32_t pmax = 1;
  for (int l = 0; l < kMaxLevels; ++l) {
    p.planes[l] = (uint32_t)wt->level[l].planes_count;
    if (p.planes[l] > pmax) pmax = p.planes[l];
  }
  p.stage_bytes_a = kTileM * bk;
  p.stage_bytes_b_max = pmax * kTileN * bk;
  const size_t ctl_bytes = sizeof(SharedCtl) + 1024;
  const uint32_t k_iters = a.KH * a.KW * p.n_cb;
  // Resident mode: with one draw count for the whole layer, a CTA that owns a single tile of 64
  // output channels keeps that tile's digit planes in shared memory for all its row tiles.
  p.resident = 0;
  p.ctas_per_otile = 1;
  p.resident_bytes = 0;
  p.band = 0;
  p.Wp = p.tpi = p.band_rows = p.band_bytes = p.Wp_magic = p.tpi_magic = 0;
  const uintptr_t out_ptrs = (uintptr_t)a.q_out | (uintptr_t)a.residual | (uintptr_t)a.f32_out | (uintptr_t)a.acc_out;
  p.vec_ok = 0u;
  if (!a.out_nchw && a.O % 16u == 0u && !(out_ptrs & 15u)) p.vec_ok = 2u;
  else if (!a.out_nchw && a.O % 8u == 0u && !(out_ptrs & 7u)) p.vec_ok = 1u;
  p.perm = nullptr;
  if (a.kmap) {
    // the caller has sorted the rows by level and gathered the matrix in that order
    if (!sorted || p.im2col) return PSB_ERR_INVALID_ARG;
    p.perm = sorted->perm;
    p.m_tiles = sorted->tiles;
  }
  if (!a.kmap) {
    const uint32_t P = p.planes[a.uniform_log2k];
    const uint32_t need = k_iters * P * kTileN * bk;
    const uint32_t cpo = (uint32_t)ctx->sm_count / p.o_tiles;
    if (need <= kResidentMaxBytes && cpo >= 1 && p.o_tiles * cpo * 10u >= (uint32_t)ctx->sm_count * 9u) {
      p.resident = 1;
      p.resident_bytes = need;
      // band mode: see TensorParams; needs the specialised output stage (codes only)
      const bool codes_only = a.q_out && !a.f32_out && !a.acc_out && (p.vec_ok || a.out_nchw) && a.inv_step > 0.0f &&
                              P >= 2u && P <= 4u;
      const uint32_t Wp = a.W + 2u * a.pad;
      const uint32_t span = kTileM + (a.KH - 1u) * Wp + (a.KW - 1u);   // band pixels a tile touches
      const uint32_t rows = (Wp - 1u + span + Wp - 1u) / Wp;           // whatever the tile's offset in its first row
      const uint32_t bytes = round_up(rows * Wp * a.C, 1024u);
      // x / d == mulhi(x, ceil(2^32 / d)) while x * d < 2^32 (d >= 2): positions t < tpi * 128 against Wp,
      // tile numbers < N * tpi against tpi
      const uint64_t tpi = ((uint64_t)a.OH * Wp + kTileM - 1) / kTileM;
      const bool quotients_ok = Wp >= 2u && tpi >= 2u && tpi * kTileM * Wp < (1ull << 32) &&
                                (uint64_t)a.N * tpi * tpi < (1ull << 32);
      if (codes_only && p.im2col && a.stride == 1 && a.KH * a.KW > 1u && a.C == bk && (bk == 64u || bk == 128u) &&
          Wp <= 256u && rows <= 256u && a.KH * a.KW * (bk / 32u) <= (uint32_t)(kMaxBandMmas - kTapBatch) && (kSmemBudget - ctl_bytes - need) / bytes >= 2u && quotients_ok) {
        p.band = 1;
        p.Wp = Wp;
        p.tpi = (uint32_t)tpi;
        p.Wp_magic = (uint32_t)(((1ull << 32) + Wp - 1) / Wp);
        p.tpi_magic = (uint32_t)(((1ull << 32) + tpi - 1) / tpi);
        p.band_rows = rows;
        p.band_bytes = bytes;
        p.m_tiles = a.N * p.tpi;
      }
      p.ctas_per_otile = cpo < p.m_tiles ? cpo : p.m_tiles;
    }
  }
  // K blocks are handed over in groups: every barrier round trip costs the issuing thread a
  // few hundred cycles, so a stage should carry about eight MMAs (M=128, N=P*64, K=32 each)
  const uint32_t sub_bytes = p.stage_bytes_a + (p.resident ? 0u : p.stage_bytes_b_max);
  const size_t avail = kSmemBudget - ctl_bytes - p.resident_bytes;
  uint32_t group = 8u / (bk / 32u);
  if (group < 1) group = 1;
  if (group > k_iters) group = k_iters;
  while (group > 1 && avail / ((size_t)group * sub_bytes) < 4) --group;
  {  // balance the groups of one tile: same number of groups, as even as possible
    const uint32_t n_groups = (k_iters + group - 1) / group;
    group = (k_iters + n_groups - 1) / n_groups;
  }
  if (p.band) group = k_iters;   // one stage = one band = every tap of a tile
  p.group = group;
  uint32_t stages = (uint32_t)(p.band ? avail / p.band_bytes : avail / ((size_t)group * sub_bytes));
  if (stages > (uint32_t)kMaxStages) stages = kMaxStages;
  // An even number of stages: the two producer warps and the two MMA issuing threads each take
  // every second stage use, so with an even ring each of them keeps to its own slots and every
  // parity wait on a slot's barriers follows that same thread's previous use of the slot.  (With
  // an odd ring a thread could wait on a slot whose previous use, the other thread's, has not
  // happened yet, and a parity wait cannot tell two phases apart.)
  stages &= ~1u;
  if (stages < 2) return PSB_ERR_UNSUPPORTED;
  p.stages = stages;
  const size_t smem_bytes = (p.band ? (size_t)stages * p.band_bytes : (size_t)stages * group * sub_bytes) +
                            p.resident_bytes + ctl_bytes;
  for (int l = 0; l < kMaxLevels; ++l) p.corr[l] = add_corr128 ? wt->level[l].corr128 : nullptr;
  p.rowsum256 = wt->rowsum256;
  p.amax = amax;
  const CUtensorMapSwizzle swz = swizzle_for(bk);
  EncodeTiledFn enc_tiled = (EncodeTiledFn)ctx->encode_tiled;
  EncodeIm2colFn enc_im2col = (EncodeIm2colFn)ctx->encode_im2col;
  if (p.band) {
    cuuint64_t dims[4] = {a.C, a.W, a.H, a.N};
    cuuint64_t strides[3] = {(cuuint64_t)a.C, (cuuint64_t)a.C * a.W, (cuuint64_t)a.C * a.W * a.H};
    cuuint32_t box[4] = {a.C, p.Wp, p.band_rows, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    if (enc_tiled(&maps.a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(a.x), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return PSB_ERR_CUDA;
  } else if (p.im2col) {
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
    cuuint64_t dims[2] = {a.C, a.kmap ? (cuuint64_t)p.m_tiles * kTileM : (cuuint64_t)p.M};
    cuuint64_t strides[1] = {(cuuint64_t)a.C};
    cuuint32_t box[2] = {bk, kTileM};
    cuuint32_t estr[2] = {1, 1};
    if (enc_tiled(&maps.a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(a.x), dims, strides, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return PSB_ERR_CUDA;
  }
  for (int l = 0; l < kMaxLevels; ++l) p.planes_ptr[l] = wt->level[l].planes;

  p.tile_mask = a.kmap ? sorted->tile_mask : nullptr;
  const uint32_t n_tiles = p.m_tiles * p.o_tiles;
  const uint32_t grid = p.resident ? p.o_tiles * p.ctas_per_otile
                                   : (n_tiles < (uint32_t)ctx->sm_count ? n_tiles : (uint32_t)ctx->sm_count);
  cudaError_t e;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreadsTensor);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // the shared-memory limit of an instance is raised once per device, to the most a launch can ask for
#define PSB_LAUNCH_INST(BKV, GEN, SLOT)                                                              \
  {                                                                                                  \
    static bool raised[kMaxDevicesForAttr][6];                                                       \
    const int dv = ctx->device;                                                                      \
    e = cudaSuccess;                                                                                 \
    if (dv < 0 || dv >= kMaxDevicesForAttr || !raised[dv][SLOT]) {                                   \
      e = cudaFuncSetAttribute(psb_mma_kernel<BKV, GEN>, cudaFuncAttributeMaxDynamicSharedMemorySize,\
                               (int)kSmemBudget);                                                    \
      if (e == cudaSuccess && dv >= 0 && dv < kMaxDevicesForAttr) raised[dv][SLOT] = true;           \
    }                                                                                                \
    if (e == cudaSuccess) e = cudaLaunchKernelEx(&cfg, psb_mma_kernel<BKV, GEN>, maps, p);           \
  }
#define PSB_LAUNCH(BKV, SLOT)                                                                        \
  if (general) PSB_LAUNCH_INST(BKV, true, SLOT) else PSB_LAUNCH_INST(BKV, false, SLOT + 1)           \
  note_launch();
  const bool general = !uniform_epilogue(p);
  const bool timed = ctx->time_contraction && ctx->t_begin[0] && ctx->timed_launches < psb_ctx::kTimedLaunches;
  if (timed) cudaEventRecord(ctx->t_begin[ctx->timed_launches], s);
  if (bk == 128) { PSB_LAUNCH(128, 0) } else if (bk == 64) { PSB_LAUNCH(64, 2) } else { PSB_LAUNCH(32, 4) }
#undef PSB_LAUNCH
#undef PSB_LAUNCH_INST
  if (timed) {
    cudaEventRecord(ctx->t_end[ctx->timed_launches], s);
    ++ctx->timed_launches;
  }
  if (e != cudaSuccess || cudaGetLastError() != cudaSuccess) return PSB_ERR_CUDA;
  return PSB_OK;
}

}  // namespace psb
