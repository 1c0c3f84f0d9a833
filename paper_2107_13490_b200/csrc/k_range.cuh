// K1: per-layer range scan (min, max, non-finite / out-of-range flags) over all
// layers in one launch.  The CTA that adds the last part of a layer (a ticket per
// layer, no waiting) turns the result into the bin origin and scale shared by all
// histograms of the layer (Sec. 3.3: binning at resolution r on the float tensor's
// own range).
#pragma once

#include "common.cuh"

namespace adapt {

constexpr int kRangeThreads = 128;   // 8 quads per thread per tile: loads first, then arithmetic

struct RangeParams {
  const LayerDesc* layers;   // all layers (+ sentinel), tiles of kTile elements
  int n_layers;
  long long n_tiles;
  LayerState* state;         // by LayerDesc::index; keys, flags and tickets start as the host set them
  float* range_out;          // optional [n_layers][2] = {min, max}
};

// Decodes the extremes of layer l into the bin origin, scale and flags.
__device__ __forceinline__ void range_finalize_layer(const RangeParams& p, const LayerDesc* layer) {
  const LayerDesc L = *layer;
  LayerState* st = p.state + L.index;
  const unsigned min_key = *reinterpret_cast<volatile unsigned*>(&st->min_key);
  const unsigned max_key = *reinterpret_cast<volatile unsigned*>(&st->max_key);
  unsigned flags = *reinterpret_cast<volatile unsigned*>(&st->flags);
  float lo = 0.0f, hi = 0.0f;
  if (L.n > 0 && !(flags & kFlagNonfinite)) {
    lo = key_float(min_key);
    hi = key_float(max_key);
  }
  const float w = __fsub_rn(hi, lo);
  const float scale = (w == 0.0f) ? 0.0f : __fdiv_rn(static_cast<float>(L.n_bins), w);
  if (L.n == 0 || hi == lo) flags |= kFlagDegenerate;
  st->flags = flags; st->lo = lo; st->hi = hi; st->scale = scale;
  st->bmax = static_cast<float>(L.n_bins - 1);
  if (p.range_out) { p.range_out[2 * L.index] = lo; p.range_out[2 * L.index + 1] = hi; }
}

// One CTA's part of a layer (already reduced over the CTA) is added to the layer's state; returns
// whether it was the last part, in which case the layer's bin origin and scale have been derived.
__device__ __forceinline__ bool range_layer_commit(const RangeParams& p, const LayerDesc* layer,
                                                unsigned kmin, unsigned kmax, unsigned flags,
                                                unsigned nzero) {
  LayerState* st = p.state + layer->index;
  atomicMin(&st->min_key, kmin);
  atomicMax(&st->max_key, kmax);
  if (flags) atomicOr(&st->flags, flags);
  if (nzero) atomicAdd(&st->zero_count, nzero * static_cast<unsigned>(kTile / 4 / kRangeThreads));
  __threadfence();
  const unsigned done = atomicAdd(&st->ticket, 1u);
  if (done + 1u != static_cast<unsigned>(layer->range_ctas)) return false;
  __threadfence();
  range_finalize_layer(p, layer);
  return true;
}

// What a CTA does with its part of a layer once its tiles are read: reduce the threads' values
// and add them to the layer's state.  Called by the whole CTA.
__device__ __forceinline__ void range_layer_tail(const RangeParams& p, const LayerDesc* layer,
                                                 float vmin, float vmax, unsigned amax,
                                                 unsigned nzero) {
  __shared__ unsigned s_min[kRangeThreads / 32], s_max[kRangeThreads / 32], s_flag[kRangeThreads / 32];
  __shared__ unsigned s_zero[kRangeThreads / 32];
  // -0.0 and +0.0 are the same value: canonicalise before taking keys
  unsigned kmin = float_key(__fadd_rn(vmin, 0.0f));
  unsigned kmax = float_key(__fadd_rn(vmax, 0.0f));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    nzero += __shfl_xor_sync(0xffffffffu, nzero, o);
  }
  // amax = the largest magnitude as a bit pattern (sign cleared): NaN and Inf are the patterns
  // from 0x7F800000 up, 2^64 is 0x5F800000.  (An out-of-range magnitude is reported only for
  // layers without NaN/Inf.)
  unsigned flags = amax >= 0x7F800000u ? kFlagNonfinite : (amax >= 0x5F800000u ? kFlagRange : 0u);
  const int w = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) { s_min[w] = kmin; s_max[w] = kmax; s_flag[w] = flags; s_zero[w] = nzero; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < kRangeThreads / 32; ++i) {
      kmin = min(kmin, s_min[i]); kmax = max(kmax, s_max[i]); flags |= s_flag[i];
      nzero += s_zero[i];
    }
    // the CTA that brings the last part of the layer finishes it
    range_layer_commit(p, layer, kmin, kmax, flags, nzero);
  }
  __syncthreads();
}

// Layers without elements have no tile and no last CTA: the first CTA settles them.
__device__ __forceinline__ void range_prologue(const RangeParams& p) {
  if (blockIdx.x == 0)
    for (int l = threadIdx.x; l < p.n_layers; l += kRangeThreads)
      if (p.layers[l].n == 0) range_finalize_layer(p, p.layers + l);
}

__global__ void __launch_bounds__(kRangeThreads, 8) range_scan_kernel(const __grid_constant__ RangeParams p) {
  const LayerDesc* __restrict__ layers = p.layers;
  const int n_layers = p.n_layers;
  const long long n_tiles = p.n_tiles;
  range_prologue(p);

  // contiguous slice of the global tile list for this CTA
  const long long per = (n_tiles + gridDim.x - 1) / gridDim.x;
  long long t = per * blockIdx.x;
  const long long t_end = min(n_tiles, t + per);
  if (t >= t_end) return;

  int l = layer_of_tile(layers, n_layers, t);

  while (t < t_end) {
    const LayerDesc L = layers[l];
    const long long layer_tiles_end = min(t_end, layers[l + 1].tile_begin);
    const float* base = L.ptr - L.mis;
    const long long jbeg = L.mis, jend = L.mis + L.n;

    float vmin = __int_as_float(0x7f800000), vmax = __int_as_float(0xff800000);
    unsigned amax = 0;
    unsigned nzero = 0;
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
            const unsigned a = __float_as_uint(v[q][k]) & 0x7FFFFFFFu;
            amax = max(amax, a);                  // NaN, Inf and |x| >= 2^64 show in the pattern
            vmin = fminf(vmin, v[q][k]);          // (a NaN operand is ignored)
            vmax = fmaxf(vmax, v[q][k]);
            if (q == 0) nzero += (a == 0u) ? 1u : 0u;   // one quad in kQ: a sample is enough
          }
        }
      }
    }
    range_layer_tail(p, layers + l, vmin, vmax, amax, nzero);
    ++l;
    while (l < n_layers && layers[l + 1].tile_begin <= t) ++l;  // skip empty layers
  }
}

}  // namespace adapt
