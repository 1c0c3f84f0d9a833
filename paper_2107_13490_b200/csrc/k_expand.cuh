// Expansion of the keyed kernel's cell counts into the per-level histograms.
//
// expand_cells_kernel: one thread per (cell, layer).  A cell's count feeds
//   * the "stable" histogram (interior cells only): these elements fall in the
//     cell's bin in the float histogram and at every fine level f >= G;
//   * every coarse level f < G: the rounded value rint(x * 2^f) of any element
//     of the cell is a + (rem >= half), with c = a * 2^d + rem, d = G - f
//     (ties that go down were fixed up element by element in the keyed kernel).
// combine_kernel: one thread per (bin, level, layer) adds the base terms to
// the correction counts already sitting in U: stable + edge-element histogram
// for fine levels, the exact zeros at the bin of 0, and builds Q and the zero
// counts of the fine levels from the zero classes.  The exact zeros are the
// elements no cell counted.
#pragma once

#include "common.cuh"
#include "k_plan.cuh"
#include "k_search_keyed.cuh"

namespace adapt {

struct ExpandParams {
  const LayerDesc* layers;     // keyed layer list
  int n_layers;
  const LayerState* state;
  const LayerPlan* plan;
  const unsigned* cell_init;   // [layer][cell_cap]
  const unsigned* cell_count;  // [layer][cell_cap]
  const unsigned* qe_hist;     // [layer][n_bins]
  unsigned* stable_hist;       // [layer][n_bins]
  unsigned* q_hist;            // [layer][n_bins]
  unsigned* u_hist;            // [layer][n_levels][n_bins]
  unsigned long long* zeros;   // [layer][n_levels]
  const unsigned long long* zero_class;  // [layer][kZeroClasses]
  unsigned long long* cell_total;        // [layer] sum of the cell counts = non-zero elements
  int n_bins, n_levels, cell_cap;
};

__global__ void __launch_bounds__(256) expand_cells_kernel(const ExpandParams p) {
  const LayerDesc L = p.layers[blockIdx.y];
  const int l = L.index;
  const LayerPlan P = p.plan[l];
  if (!P.keyed) return;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  const unsigned m = (c < P.cells) ? p.cell_count[static_cast<size_t>(l) * p.cell_cap + c] : 0u;
  // the layer's non-zero elements = sum of all its cell counts
  unsigned long long wsum = m;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
  if ((threadIdx.x & 31) == 0 && wsum) atomicAdd(&p.cell_total[l], wsum);
  if (m == 0) return;
  const LayerState S = p.state[l];
  const int B = p.n_bins;
  const long long cc = P.c0 + c;
  if (!(p.cell_init[static_cast<size_t>(l) * p.cell_cap + c] & kCellEdge)) {
    const float lf = __double2float_rd(ldexp(static_cast<double>(cc), -P.g));
    atomicAdd(&p.stable_hist[static_cast<size_t>(l) * B + bin_of(lf, S.lo, S.scale, S.bmax)], m);
  }
  unsigned* U = p.u_hist + static_cast<size_t>(l) * p.n_levels * B;
  const int coarse_end = min(P.g, p.n_levels);
  for (int f = 0; f < coarse_end; ++f) {
    const int d = P.g - f;                       // 1..32
    const long long a = cc >> d;                 // floor(c / 2^d)
    const long long rem = cc - (a << d);
    const long long r = a + ((rem >= (1ll << (d - 1))) ? 1 : 0);
    const float v = __fmul_rn(__ll2float_rn(r), pow2f(-f));
    atomicAdd(&U[static_cast<size_t>(f) * B + bin_of(v, S.lo, S.scale, S.bmax)], m);
    if (r == 0) atomicAdd(&p.zeros[static_cast<size_t>(l) * p.n_levels + f],
                          static_cast<unsigned long long>(m));
  }
}

__global__ void __launch_bounds__(256) combine_kernel(const ExpandParams p) {
  const LayerDesc L = p.layers[blockIdx.z];
  const int l = L.index;
  const LayerPlan P = p.plan[l];
  if (!P.keyed) return;
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  const int f = blockIdx.y;                      // level, or n_levels for the float histogram
  const int B = p.n_bins;
  if (b >= B) return;
  const LayerState S = p.state[l];
  const unsigned nz = static_cast<unsigned>(static_cast<unsigned long long>(L.n) - p.cell_total[l]);
  const int bz = bin_of(0.0f, S.lo, S.scale, S.bmax);
  const unsigned base = p.stable_hist[static_cast<size_t>(l) * B + b] +
                        p.qe_hist[static_cast<size_t>(l) * B + b];
  const unsigned zero_here = (b == bz) ? nz : 0u;
  if (f == p.n_levels) {
    p.q_hist[static_cast<size_t>(l) * B + b] = base + zero_here;
    return;
  }
  unsigned* u = p.u_hist + (static_cast<size_t>(l) * p.n_levels + f) * B + b;
  *u = *u + (f >= P.fs ? base : 0u) + zero_here;
  if (b == 0) {
    unsigned long long z = nz;
    if (f >= P.fs) {
      const unsigned long long* zc = p.zero_class + static_cast<size_t>(l) * kZeroClasses;
      for (int k = f; k <= 32; ++k) z += zc[k + 1];   // classes whose highest zero level >= f
    }
    p.zeros[static_cast<size_t>(l) * p.n_levels + f] += z;
  }
}

}  // namespace adapt
