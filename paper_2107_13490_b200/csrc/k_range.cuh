// K1: per-layer range scan (min, max, non-finite / out-of-range flags) over all
// layers in one launch, and the small finalisation kernel that turns the
// result into the bin origin and scale shared by all histograms of the layer
// (Sec. 3.3: binning at resolution r on the float tensor's own range).
#pragma once

#include "common.cuh"

namespace adapt {

constexpr int kTile = 4096;          // elements per tile (in aligned indexing)
constexpr int kRangeThreads = 128;   // 8 quads per thread per tile: loads first, then arithmetic

constexpr unsigned kFlagDegenerate = 2u;
constexpr unsigned kFlagNonfinite = 4u;
constexpr unsigned kFlagRange = 8u;

__global__ void __launch_bounds__(kRangeThreads)
range_scan_kernel(const LayerDesc* __restrict__ layers, int n_layers, long long n_tiles,
                  LayerState* __restrict__ state) {
  // contiguous slice of the global tile list for this CTA
  const long long per = (n_tiles + gridDim.x - 1) / gridDim.x;
  long long t = per * blockIdx.x;
  const long long t_end = min(n_tiles, t + per);
  if (t >= t_end) return;

  __shared__ unsigned s_min[kRangeThreads / 32], s_max[kRangeThreads / 32], s_flag[kRangeThreads / 32];
  __shared__ float s_abs[kRangeThreads / 32];
  __shared__ unsigned s_zero[kRangeThreads / 32], s_lsb[kRangeThreads / 32];
  int l = layer_of_tile(layers, n_layers, t);

  while (t < t_end) {
    const LayerDesc L = layers[l];
    const long long layer_tiles_end = min(t_end, layers[l + 1].tile_begin);
    const float* base = L.ptr - L.mis;
    const long long jbeg = L.mis, jend = L.mis + L.n;

    float vmin = __int_as_float(0x7f800000), vmax = __int_as_float(0xff800000);
    unsigned flags = 0;
    float asum = 0.0f;
    unsigned nzero = 0, lsb = 0xFFFFFFFFu;
    for (; t < layer_tiles_end; ++t) {
      const long long j_tile = (t - L.tile_begin) * kTile;
      constexpr int kQ = kTile / 4 / kRangeThreads;
      float v[kQ][4];
      unsigned m[kQ];
      if (j_tile >= jbeg && j_tile + kTile <= jend) {
        // full tile: all loads first, then the arithmetic
#pragma unroll
        for (int q = 0; q < kQ; ++q) {
          const float4 w4 = __ldg(reinterpret_cast<const float4*>(base + j_tile) + q * kRangeThreads + threadIdx.x);
          v[q][0] = w4.x; v[q][1] = w4.y; v[q][2] = w4.z; v[q][3] = w4.w;
          m[q] = 0xFu;
        }
      } else {
#pragma unroll
        for (int q = 0; q < kQ; ++q) {
          const long long j0 = j_tile + 4ll * (q * kRangeThreads + threadIdx.x);
          m[q] = 0;
          v[q][0] = v[q][1] = v[q][2] = v[q][3] = 0.0f;
          if (j0 < jend) m[q] = load_quad(base, j0, jbeg, jend, v[q]);
        }
      }
#pragma unroll
      for (int q = 0; q < kQ; ++q) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (m[q] & (1u << k)) {
            float a = fabsf(v[q][k]);
            // NaN fails both compares; Inf is caught by the first
            if (!(a <= 3.402823466e38f)) flags |= kFlagNonfinite;
            else if (a >= 18446744073709551616.0f) flags |= kFlagRange;
            vmin = fminf(vmin, v[q][k]);
            vmax = fmaxf(vmax, v[q][k]);
            asum += a;
            if (q == 0) {                                  // one quad in kQ: a sample is enough
              nzero += (a == 0.0f) ? 1u : 0u;
              // position of the element's lowest set significand bit (hidden bit included)
              const unsigned bits = __float_as_uint(v[q][k]);
              const unsigned at = ((bits >> 23) & 0xFFu) + static_cast<unsigned>(__ffs(bits | 0x00800000u) - 1);
              if (a != 0.0f) lsb = min(lsb, at);
            }
          }
        }
      }
    }
    // -0.0 and +0.0 are the same value: canonicalise before taking keys
    unsigned kmin = float_key(__fadd_rn(vmin, 0.0f));
    unsigned kmax = float_key(__fadd_rn(vmax, 0.0f));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
      kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
      flags |= __shfl_xor_sync(0xffffffffu, flags, o);
      asum += __shfl_xor_sync(0xffffffffu, asum, o);
      nzero += __shfl_xor_sync(0xffffffffu, nzero, o);
      lsb = min(lsb, __shfl_xor_sync(0xffffffffu, lsb, o));
    }
    const int w = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) { s_min[w] = kmin; s_max[w] = kmax; s_flag[w] = flags; s_abs[w] = asum; s_zero[w] = nzero; s_lsb[w] = lsb; }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int i = 1; i < kRangeThreads / 32; ++i) {
        kmin = min(kmin, s_min[i]); kmax = max(kmax, s_max[i]); flags |= s_flag[i];
        asum += s_abs[i]; nzero += s_zero[i]; lsb = min(lsb, s_lsb[i]);
      }
      atomicMin(&state[L.index].min_key, kmin);
      atomicMax(&state[L.index].max_key, kmax);
      if (flags) atomicOr(&state[L.index].flags, flags);
      if (asum == asum && asum < 3.0e38f) atomicAdd(&state[L.index].abs_sum, asum);
      if (nzero) atomicAdd(&state[L.index].zero_count, nzero * static_cast<unsigned>(kTile / 4 / kRangeThreads));
      if (lsb != 0xFFFFFFFFu) atomicMin(&state[L.index].min_lsb, lsb);
    }
    __syncthreads();
    ++l;
    while (l < n_layers && layers[l + 1].tile_begin <= t) ++l;  // skip empty layers
  }
}

// One thread per layer: decode min/max, derive the bin scale and flags.
__global__ void range_finalize_kernel(const LayerDesc* __restrict__ layers, int n_layers,
                                      LayerState* __restrict__ state,
                                      float* __restrict__ range_out) {
  int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l >= n_layers) return;
  LayerState s = state[l];
  const int n_bins = layers[l].n_bins;
  float lo = 0.0f, hi = 0.0f;
  if (layers[l].n > 0 && !(s.flags & kFlagNonfinite)) {
    lo = key_float(s.min_key);
    hi = key_float(s.max_key);
  }
  float w = __fsub_rn(hi, lo);
  float scale = (w == 0.0f) ? 0.0f : __fdiv_rn(static_cast<float>(n_bins), w);
  if (layers[l].n == 0 || hi == lo) s.flags |= kFlagDegenerate;
  s.lo = lo; s.hi = hi; s.scale = scale; s.bmax = static_cast<float>(n_bins - 1);
  state[l] = s;
  if (range_out) { range_out[2 * l] = lo; range_out[2 * l + 1] = hi; }
}

}  // namespace adapt
