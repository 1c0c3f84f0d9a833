// Gradient diversity of each layer over its last K gradient tensors (Sec. 3.3, the PushUp
// heuristic):  delta_s = sum_k ||g_k||_2 / || sum_k g_k ||_2 , log form = log(delta_s) if
// 0 < delta_s < inf else 1.  A streaming reduction: every gradient element is read once
// (4 B per element and tensor), squares and the element-wise sum are accumulated in double.
#pragma once

#include <math.h>

#include "common.cuh"

namespace adapt {

constexpr int kDivThreads = 128;
constexpr int kDivPerThread = 16;                       // elements per thread per tile (4 quads)
constexpr int kDivTile = kDivThreads * kDivPerThread;   // 2048 elements
constexpr int kDivMaxGrads = 256;                       // gradient tensors per layer

struct DivLayer {
  long long n;            // elements per gradient tensor
  long long tile_begin;   // first tile of the layer in the launch's tile list
  int vec;                // every gradient pointer of the layer is 16-byte aligned
  int pad_;
};

struct DivParams {
  const DivLayer* layers;        // [n_layers + 1] (sentinel holds the tile total)
  const float* const* grads;     // [n_layers][n_grads] device pointers
  double* sumsq;                 // [n_layers][n_grads + 1]: per-gradient sums of squares, then
                                 // the sum of squares of the element-wise sum
  int n_layers, n_grads;
  long long n_tiles;
};

__global__ void __launch_bounds__(kDivThreads) diversity_kernel(const DivParams p) {
  __shared__ double s_sq[kDivMaxGrads + 1];
  const long long per = (p.n_tiles + gridDim.x - 1) / gridDim.x;
  long long t = per * blockIdx.x;
  const long long t_end = min(p.n_tiles, t + per);
  if (t >= t_end) return;
  const int K = p.n_grads;
  const int lane = threadIdx.x & 31;

  int lo = 0, hi = p.n_layers - 1;          // layer that owns tile t
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (p.layers[mid].tile_begin <= t) lo = mid; else hi = mid - 1;
  }
  int l = lo;
  while (t < t_end) {
    const DivLayer L = p.layers[l];
    const long long layer_end = min(t_end, p.layers[l + 1].tile_begin);
    const float* const* G = p.grads + static_cast<size_t>(l) * K;
    for (int k = threadIdx.x; k <= K; k += kDivThreads) s_sq[k] = 0.0;
    __syncthreads();
    double sq_of_sum = 0.0;
    for (; t < layer_end; ++t) {
      const long long tile_first = (t - L.tile_begin) * kDivTile;
      const long long i0 = tile_first + threadIdx.x;
      double s[kDivPerThread];
#pragma unroll
      for (int j = 0; j < kDivPerThread; ++j) s[j] = 0.0;
      // four gradients per trip: their loads are issued together (measured: 5.4 against 5.0 TB/s)
#pragma unroll 4
      for (int k = 0; k < K; ++k) {
        const float* g = G[k];
        float x[kDivPerThread];
        // which elements a thread takes only has to be the same for every k of the tile
        if (L.vec && tile_first + kDivTile <= L.n) {       // full tile, aligned: 128-bit loads
#pragma unroll
          for (int q = 0; q < kDivPerThread / 4; ++q) {
            const float4 v4 = __ldcs(reinterpret_cast<const float4*>(g + tile_first) +
                                     q * kDivThreads + threadIdx.x);
            x[4 * q] = v4.x; x[4 * q + 1] = v4.y; x[4 * q + 2] = v4.z; x[4 * q + 3] = v4.w;
          }
        } else {
#pragma unroll
          for (int j = 0; j < kDivPerThread; ++j) {
            const long long i = i0 + static_cast<long long>(j) * kDivThreads;
            x[j] = (i < L.n) ? __ldcs(g + i) : 0.0f;
          }
        }
        double sq = 0.0;
#pragma unroll
        for (int j = 0; j < kDivPerThread; ++j) {
          const double d = static_cast<double>(x[j]);
          sq = fma(d, d, sq);
          s[j] += d;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
        if (lane == 0) atomicAdd(&s_sq[k], sq);
      }
#pragma unroll
      for (int j = 0; j < kDivPerThread; ++j) sq_of_sum = fma(s[j], s[j], sq_of_sum);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq_of_sum += __shfl_xor_sync(0xffffffffu, sq_of_sum, o);
    if (lane == 0) atomicAdd(&s_sq[K], sq_of_sum);
    __syncthreads();
    double* out = p.sumsq + static_cast<size_t>(l) * (K + 1);
    for (int k = threadIdx.x; k <= K; k += kDivThreads)
      if (s_sq[k] != 0.0) atomicAdd(&out[k], s_sq[k]);
    __syncthreads();
    ++l;
    while (l < p.n_layers && p.layers[l + 1].tile_begin <= t) ++l;
  }
}

// Gradient normalisation (Sec. 3.3, "Dealing with Fixed-Points Limited Range"):
// out = g / ||g||_2 per layer, the norm taken from the sums of squares the reduction above left
// in sumsq (one gradient per layer: sumsq[2 l]).  The quotient is formed in double, as a product
// with the reciprocal of the norm (a double division per element would make the kernel
// FP64-bound), and rounded to float: like the norm's summation order this can move a result by
// one fp32 ulp where the quotient sits on a rounding boundary, never more.  A layer whose norm
// is 0 is copied.  out may be g itself.  8 B per element.
__global__ void __launch_bounds__(kDivThreads)
normalize_kernel(const DivLayer* __restrict__ layers, const float* const* __restrict__ grads,
                 float* const* __restrict__ outs, const double* __restrict__ sumsq, int n_layers,
                 long long n_tiles) {
  for (long long t = blockIdx.x; t < n_tiles; t += gridDim.x) {
    int lo = 0, hi = n_layers - 1;          // layer that owns tile t
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (layers[mid].tile_begin <= t) lo = mid; else hi = mid - 1;
    }
    const DivLayer L = layers[lo];
    const float* g = grads[lo];
    float* out = outs[lo];
    const double norm = sqrt(sumsq[2 * lo]);
    const bool scale = norm > 0.0;
    const double inv = scale ? 1.0 / norm : 0.0;
    const long long i0 = (t - L.tile_begin) * kDivTile;
    const long long i1 = min(L.n, i0 + kDivTile);
    if (L.vec && i1 - i0 == kDivTile) {
      const float4* g4 = reinterpret_cast<const float4*>(g + i0);
      float4* o4 = reinterpret_cast<float4*>(out + i0);
#pragma unroll
      for (int q = 0; q < kDivPerThread / 4; ++q) {
        float4 v = __ldcs(g4 + q * kDivThreads + threadIdx.x);
        if (scale) {
          v.x = __double2float_rn(__dmul_rn(static_cast<double>(v.x), inv));
          v.y = __double2float_rn(__dmul_rn(static_cast<double>(v.y), inv));
          v.z = __double2float_rn(__dmul_rn(static_cast<double>(v.z), inv));
          v.w = __double2float_rn(__dmul_rn(static_cast<double>(v.w), inv));
        }
        __stcs(o4 + q * kDivThreads + threadIdx.x, v);
      }
    } else {
      for (long long i = i0 + threadIdx.x; i < i1; i += kDivThreads) {
        const float x = __ldcs(g + i);
        out[i] = scale ? __double2float_rn(__dmul_rn(static_cast<double>(x), inv)) : x;
      }
    }
  }
}

// One thread per layer: norms from the sums of squares, then the two forms of the diversity.
__global__ void diversity_finalize_kernel(const double* __restrict__ sumsq, int n_layers,
                                          int n_grads, double* __restrict__ out) {
  const int l = blockIdx.x * blockDim.x + threadIdx.x;
  if (l >= n_layers) return;
  const double* q = sumsq + static_cast<size_t>(l) * (n_grads + 1);
  double sum_norms = 0.0;
  for (int k = 0; k < n_grads; ++k) sum_norms += sqrt(q[k]);
  const double norm_sum = sqrt(q[n_grads]);
  const double ds = sum_norms / norm_sum;
  out[4 * l + 0] = sum_norms;
  out[4 * l + 1] = norm_sum;
  out[4 * l + 2] = ds;
  out[4 * l + 3] = (ds > 0.0 && ds < __longlong_as_double(0x7ff0000000000000ll)) ? log(ds) : 1.0;
}

}  // namespace adapt
