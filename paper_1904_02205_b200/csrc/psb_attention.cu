// Attention proposal (paper Sec. 4.5, "Computational Attention"): where to spend more draws.
//
// From a cheap pass of the network (few draws everywhere), the pixelwise entropy of the softmax over the
// channels of the last convolutional layer,  h_xy = - sum_c softmax(a_xy)_c log softmax(a_xy)_c,  marks the
// regions whose classification is least settled; a hard threshold at the image's mean entropy splits the
// locations into two classes, and the resulting mask, sampled by nearest neighbour at every layer resolution,
// becomes the per-location draw-count map (psb_set_sample_map) of the second pass.
#include "psb_common.cuh"

namespace psb {

namespace {

// One warp per location.  Activations are integer codes times a step, so softmax needs exp at no more than
// 256 (u8) / 511 (s8 differences) arguments: a table in shared memory, exp(-j * step) for j = 0.., filled
// once per block; the two sums of a location are then table look-ups and multiply-adds:
//   z_c = (q_c - q_max) * step <= 0,  S = sum exp(z_c),  T = sum z_c exp(z_c),  h = log S - T / S.
__global__ void __launch_bounds__(256) entropy_kernel(const uint8_t* act, uint32_t is_signed,
                                                      uint32_t locations, uint32_t C, float step,
                                                      float* __restrict__ entropy) {
  pdl_prologue();
  __shared__ float table[512];
  for (uint32_t j = threadIdx.x; j < 512u; j += blockDim.x) table[j] = expf(-(float)j * step);
  __syncthreads();
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t warps = (gridDim.x * blockDim.x) >> 5;
  for (uint32_t loc = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; loc < locations; loc += warps) {
    const uint8_t* row = act + (size_t)loc * C;
    int best = -1000;
    for (uint32_t c = lane; c < C; c += 32u) {
      const int q = is_signed ? (int)(signed char)row[c] : (int)row[c];
      best = max(best, q);
    }
    best = __reduce_max_sync(0xFFFFFFFFu, best);
    float S = 0.0f, T = 0.0f;
    for (uint32_t c = lane; c < C; c += 32u) {
      const int q = is_signed ? (int)(signed char)row[c] : (int)row[c];
      const int j = best - q;                       // 0 .. 510
      const float e = table[j];
      S += e;
      T = __fmaf_rn(-(float)j * step, e, T);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      S += __shfl_xor_sync(0xFFFFFFFFu, S, d);
      T += __shfl_xor_sync(0xFFFFFFFFu, T, d);
    }
    if (lane == 0) entropy[loc] = logf(S) - T / S;
  }
}

struct MapTable {
  uint8_t* map[8];
  uint32_t res[8];
};

// One block per image: mean entropy (fixed summation order), threshold, maps of every resolution.
__global__ void __launch_bounds__(256) attention_maps_kernel(const float* entropy, uint32_t H, uint32_t W,
                                                             uint32_t lo_log2k, uint32_t hi_log2k, uint32_t n_res,
                                                             const MapTable maps, float* __restrict__ mean_out) {
  pdl_prologue();
  __shared__ float part[256];
  __shared__ float mean_s;
  const uint32_t n = blockIdx.x, pixels = H * W;
  const float* h = entropy + (size_t)n * pixels;
  float s = 0.0f;
  for (uint32_t i = threadIdx.x; i < pixels; i += blockDim.x) s += h[i];
  part[threadIdx.x] = s;
  __syncthreads();
  for (uint32_t d = 128; d > 0; d >>= 1) {
    if (threadIdx.x < d) part[threadIdx.x] += part[threadIdx.x + d];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    mean_s = part[0] / (float)pixels;
    if (mean_out) mean_out[n] = mean_s;
  }
  __syncthreads();
  const float mean = mean_s;
  for (uint32_t r = 0; r < n_res; ++r) {
    const uint32_t R = maps.res[r];
    uint8_t* out = maps.map[r] + (size_t)n * R * R;
    for (uint32_t i = threadIdx.x; i < R * R; i += blockDim.x) {
      const uint32_t y = i / R, x = i - y * R;
      const uint32_t sy = (uint32_t)(((unsigned long long)y * H) / R), sx = (uint32_t)(((unsigned long long)x * W) / R);
      out[i] = (uint8_t)(h[sy * W + sx] > mean ? hi_log2k : lo_log2k);
    }
  }
}

}  // namespace

cudaError_t launch_entropy(const void* act, uint32_t is_signed, uint32_t locations, uint32_t C, float step,
                           float* entropy, cudaStream_t s) {
  uint32_t blocks = (locations + 7u) / 8u;
  if (blocks > 148u * 8u) blocks = 148u * 8u;
  if (blocks < 1u) blocks = 1u;
  launch_pdl(entropy_kernel, blocks, 256, 0, s, (const uint8_t*)act, is_signed, locations, C, step, entropy);
  note_launch();
  return cudaGetLastError();
}

cudaError_t launch_attention_maps(const float* entropy, uint32_t N, uint32_t H, uint32_t W, uint32_t lo_log2k,
                                  uint32_t hi_log2k, uint32_t n_res, const uint32_t* res, uint8_t* const* maps,
                                  float* mean_out, cudaStream_t s) {
  MapTable t;
  for (uint32_t i = 0; i < 8u; ++i) { t.map[i] = i < n_res ? maps[i] : nullptr; t.res[i] = i < n_res ? res[i] : 0u; }
  launch_pdl(attention_maps_kernel, N, 256, 0, s, entropy, H, W, lo_log2k, hi_log2k, n_res, t, mean_out);
  note_launch();
  return cudaGetLastError();
}

}  // namespace psb
