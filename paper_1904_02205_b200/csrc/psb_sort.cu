// Per-location draw counts (paper Sec. 4.5) on the tensor path: rows sorted by level.
//
// A contraction tile is 128 output locations and one integer filter; under a draw-count map the
// locations of a tile would need different filters W_k.  So the locations are first sorted by their
// level (a counting sort over the seven levels; every level's run is padded to whole tiles), the
// activation rows are gathered in that order into one matrix (an explicit patch matrix for filters with
// taps), the contraction runs over it as a plain matrix product with one level per tile, and the output
// stage scatters every row back to its location through the same permutation.  Every location is
// contracted exactly once, with the filter of its own level: the cost no longer depends on how the levels
// are mixed in space.
#include "psb_common.cuh"

namespace psb {

namespace {

constexpr uint32_t kBins = 8;        // levels 0..6 and one bin for invalid entries (flagged by the output stage)
constexpr uint32_t kTileRows = 128;

}  // namespace

struct SortCtl {
  uint32_t count[kBins];      // locations per level
  uint32_t cursor[kBins];     // next free slot per level while scattering
  uint32_t start[kBins + 1];  // first sorted row of each level (multiples of the tile height)
  uint32_t ticket;
  uint32_t tiles;             // tiles in use
};

namespace {

// Histogram of the map; the last block to finish turns it into the padded run starts.  Also marks the whole
// permutation as padding, which the scatter pass then overwrites where a location lands.
__global__ void __launch_bounds__(256) level_count_kernel(const uint8_t* kmap, uint32_t M,
                                                          SortCtl* __restrict__ ctl, uint32_t* __restrict__ perm,
                                                          uint32_t perm_words) {
  pdl_prologue();
  __shared__ uint32_t hist[kBins];
  if (threadIdx.x < kBins) hist[threadIdx.x] = 0u;
  __syncthreads();
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < perm_words; i += gridDim.x * blockDim.x)
    perm[i] = 0xFFFFFFFFu;
  for (uint32_t m = blockIdx.x * blockDim.x + threadIdx.x; m < M; m += gridDim.x * blockDim.x) {
    const uint32_t l = min((uint32_t)kmap[m], kBins - 1u);
    const uint32_t peers = __match_any_sync(__activemask(), l);
    if ((threadIdx.x & 31u) == (uint32_t)__ffs((int)peers) - 1u) atomicAdd(&hist[l], (uint32_t)__popc(peers));
  }
  __syncthreads();
  if (threadIdx.x < kBins && hist[threadIdx.x]) atomicAdd(&ctl->count[threadIdx.x], hist[threadIdx.x]);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    if (atomicAdd(&ctl->ticket, 1u) == gridDim.x - 1u) {
      __threadfence();
      uint32_t at = 0;
      for (uint32_t l = 0; l < kBins; ++l) {
        ctl->start[l] = at;
        at += (atomicAdd(&ctl->count[l], 0u) + kTileRows - 1u) / kTileRows * kTileRows;
      }
      ctl->start[kBins] = at;
      ctl->tiles = at / kTileRows;
    }
  }
}

// perm[sorted row] = location.  Lanes of a warp that share a level take consecutive slots, so the order of
// the locations is kept within a warp (neighbouring locations stay neighbours in memory).  Also writes the
// level of every tile as a one-bit mask (0 for tiles beyond the last run).
__global__ void __launch_bounds__(256) level_scatter_kernel(const uint8_t* kmap, uint32_t M,
                                                            SortCtl* __restrict__ ctl, uint32_t* __restrict__ perm,
                                                            uint8_t* __restrict__ tile_mask, uint32_t max_tiles) {
  pdl_prologue();
  const uint32_t gid = blockIdx.x * blockDim.x + threadIdx.x, lane = threadIdx.x & 31u;
  for (uint32_t t = gid; t < max_tiles; t += gridDim.x * blockDim.x) {
    uint32_t mask = 0u;
    const uint32_t row = t * kTileRows;
    for (uint32_t l = 0; l < kBins; ++l)
      if (row >= ctl->start[l] && row < ctl->start[l + 1u]) mask = 1u << l;
    tile_mask[t] = (uint8_t)mask;
  }
  for (uint32_t m0 = (gid - lane); m0 < M; m0 += gridDim.x * blockDim.x) {
    const uint32_t m = m0 + lane;
    const bool ok = m < M;
    const uint32_t l = ok ? min((uint32_t)kmap[m], kBins - 1u) : 0xFFu;
    const uint32_t peers = __match_any_sync(0xFFFFFFFFu, l);
    uint32_t base = 0;
    const uint32_t leader = (uint32_t)__ffs((int)peers) - 1u;
    if (ok && lane == leader) base = atomicAdd(&ctl->cursor[l], (uint32_t)__popc(peers));
    base = __shfl_sync(0xFFFFFFFFu, base, (int)leader);
    if (ok) perm[ctl->start[l] + base + (uint32_t)__popc(peers & ((1u << lane) - 1u))] = m;
  }
}

// Activation rows in sorted order: row r of the matrix is the patch of location perm[r], K index
// (kh * KW + kw) * cpad + ci (cpad >= C bytes per tap, the rest zero); positions outside the image are zero.
// A group of `lanes_per_row` lanes copies the patches of kGatherRows rows at a time, tap by tap, in 16-byte
// pieces: the loads of the rows are issued together, then their stores (a copy with one load in flight per
// thread, behind the lookup of its row, reached a third of the memory bandwidth).
constexpr int kGatherRows = 4;

__global__ void __launch_bounds__(256) gather_sorted_kernel(const ConvArgs a, const uint32_t* perm,
                                                            const SortCtl* ctl, uint32_t cpad,
                                                            uint32_t lanes_per_row, uint8_t* __restrict__ dst) {
  pdl_prologue();
  const uint32_t taps = a.KH * a.KW, pitch = taps * cpad;
  const uint32_t rows = __ldcg(&ctl->tiles) * kTileRows;
  const uint32_t slots = blockDim.x / lanes_per_row;
  const uint32_t sub = threadIdx.x % lanes_per_row, slot = threadIdx.x / lanes_per_row;
  const uint32_t ohow = a.OH * a.OW;
  const uint8_t* x = (const uint8_t*)a.x;
  const uint32_t step = gridDim.x * slots;              // rows between the rows of one thread
  for (uint32_t r0 = blockIdx.x * slots + slot; r0 < rows; r0 += step * (uint32_t)kGatherRows) {
    // the rows of this round: image base, input coordinates of the filter's first tap, whether the row is real
    const uint8_t* img[kGatherRows];
    uint8_t* out[kGatherRows];
    int y0[kGatherRows], x0[kGatherRows];
    bool live[kGatherRows];
#pragma unroll
    for (int u = 0; u < kGatherRows; ++u) {
      const uint32_t r = r0 + (uint32_t)u * step;
      const uint32_t m = r < rows ? __ldcg(perm + r) : 0xFFFFFFFFu;
      live[u] = m != 0xFFFFFFFFu;                       // padding rows are never stored by the output stage
      const uint32_t mm = live[u] ? m : 0u;
      const uint32_t n = mm / ohow, pix = mm - n * ohow, oy = pix / a.OW, ox = pix - oy * a.OW;
      img[u] = x + (size_t)n * a.H * a.W * a.C;
      y0[u] = (int)(oy * a.stride) - (int)a.pad;
      x0[u] = (int)(ox * a.stride) - (int)a.pad;
      out[u] = dst + (size_t)(live[u] ? r : 0u) * pitch;
    }
    uint32_t kh = 0, kw = 0;
    for (uint32_t tap = 0; tap < taps; ++tap) {
      for (uint32_t b = sub * 16u; b < cpad; b += lanes_per_row * 16u) {
        uint4 v[kGatherRows];
#pragma unroll
        for (int u = 0; u < kGatherRows; ++u) {
          const int iy = y0[u] + (int)kh, ix = x0[u] + (int)kw;
          const bool inside = live[u] && (unsigned)iy < a.H && (unsigned)ix < a.W && b < a.C;
          v[u] = make_uint4(0u, 0u, 0u, 0u);
          if (inside) v[u] = __ldcg(reinterpret_cast<const uint4*>(img[u] + ((size_t)iy * a.W + (uint32_t)ix) * a.C + b));
        }
#pragma unroll
        for (int u = 0; u < kGatherRows; ++u)
          if (live[u]) *reinterpret_cast<uint4*>(out[u] + (size_t)tap * cpad + b) = v[u];
      }
      if (++kw == a.KW) { kw = 0; ++kh; }
    }
  }
}

}  // namespace

size_t sort_ctl_bytes() { return sizeof(SortCtl); }
uint32_t sorted_tiles_bound(uint64_t M) { return (uint32_t)((M + kTileRows - 1) / kTileRows + kBins); }

cudaError_t launch_level_sort(const uint8_t* kmap, uint32_t M, void* ctl, uint32_t* perm, uint8_t* tile_mask,
                              cudaStream_t s) {
  const uint32_t max_tiles = sorted_tiles_bound(M);
  cudaError_t e = cudaMemsetAsync(ctl, 0, sizeof(SortCtl), s);
  if (e != cudaSuccess) return e;
  uint32_t blocks = (M + 255u) / 256u;
  if (blocks > 148u * 8u) blocks = 148u * 8u;
  if (blocks < 1u) blocks = 1u;
  launch_pdl(level_count_kernel, blocks, 256, 0, s, kmap, M, (SortCtl*)ctl, perm, max_tiles * kTileRows);
  note_launch();
  launch_pdl(level_scatter_kernel, blocks, 256, 0, s, kmap, M, (SortCtl*)ctl, perm, tile_mask, max_tiles);
  note_launch();
  return cudaGetLastError();
}

cudaError_t launch_gather_sorted(const ConvArgs& a, const uint32_t* perm, const void* ctl, uint32_t cpad, uint8_t* dst,
                                 cudaStream_t s) {
  uint32_t lanes = 1;
  while (lanes < 32u && lanes * 16u < cpad) lanes *= 2u;
  const uint64_t rows = (uint64_t)sorted_tiles_bound((uint64_t)a.N * a.OH * a.OW) * kTileRows;
  const uint32_t rows_per_block = (256u / lanes) * (uint32_t)kGatherRows;
  uint64_t blocks = (rows + rows_per_block - 1) / rows_per_block;
  if (blocks > 148u * 16u) blocks = 148u * 16u;
  if (blocks < 1u) blocks = 1u;
  launch_pdl(gather_sorted_kernel, (uint32_t)blocks, 256, 0, s, a, perm, (const SortCtl*)ctl, cpad, lanes, dst);
  note_launch();
  return cudaGetLastError();
}

}  // namespace psb
