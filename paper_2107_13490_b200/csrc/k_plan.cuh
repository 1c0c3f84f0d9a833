// Per-layer plan of the keyed search kernel (round-to-nearest-even only).
//
// Idea.  Cut the value axis into cells of width 2^-G (G per layer, as fine as
// the cell table that fits in shared memory allows).  An element x lies in
// cell c = floor(x * 2^G).  Then, exactly:
//  * for every coarser level f < G the rounded value rint(x * 2^f) is a
//    function of c alone (unless x sits exactly on the level-G grid AND on a
//    rounding tie of level f - at most one level per element, fixed up
//    separately), so one count per cell yields the histograms of all coarse
//    levels afterwards;
//  * for every finer level f >= G the rounded value stays inside the closed
//    cell, so if the whole closed cell lies in one bin ("interior cell") the
//    element falls in that bin at every fine level and in the float histogram;
//  * only elements of cells that contain a bin edge ("edge cells") need their
//    fine levels looked at one by one, and among those only the levels whose
//    half quantum 2^-(f+1) exceeds the element's distance to its bin's edges;
//  * for f >= G an element rounds to zero only if it lies in cell -1 or 0.
// This kernel chooses G, computes the exact bin edges (smallest float of each
// bin, by bisection over the float order with the bin function itself), and
// marks each cell: bit 31 = edge cell, bit 30 = cell -1 or 0.
#pragma once

#include "common.cuh"
#include "k_range.cuh"

namespace adapt {

constexpr unsigned kCellEdge = 0x80000000u;
constexpr unsigned kCellNearZero = 0x40000000u;
constexpr unsigned kCellCountMask = 0x3FFFFFFFu;
constexpr int kPlanThreads = 256;

struct LayerPlan {
  long long c0;   // cell index of the first cell: floor(lo * 2^G)
  int g;          // cell level G (cells are 2^-G wide); may be negative
  int cells;      // number of cells covering [lo, hi]
  int fs;         // first fine level: max(G, 0)
  float c0f;      // (float)c0 when it is exact, else unused
  float two_g;    // 2^G
  int keyed;      // 1 if the layer goes through the keyed kernel
};

struct PlanParams {
  const LayerDesc* layers;   // keyed layer list
  int n_layers;              // entries in that list
  const LayerState* state;   // indexed by LayerDesc::index
  LayerPlan* plan;           // indexed by LayerDesc::index
  float* edges;              // [all layers][n_bins + 1]
  unsigned* cell_init;       // [all layers][cell_cap]
  int n_bins;
  int cell_cap;              // table entries per layer (memory stride)
  int cell_target;           // most cells a layer may use (<= cell_cap)
};

__device__ __forceinline__ long long floor_scaled(float v, int g) {
  // floor(v * 2^g) exactly: |v| < 2^64 and |g| <= 64 keep the product inside double
  return static_cast<long long>(floor(ldexp(static_cast<double>(v), g)));
}

__global__ void __launch_bounds__(kPlanThreads) plan_kernel(const PlanParams p) {
  const LayerDesc L = p.layers[blockIdx.x];
  const int l = L.index;
  const LayerState S = p.state[l];
  __shared__ LayerPlan s_plan;
  const int B = p.n_bins;

  if (threadIdx.x == 0) {
    LayerPlan P;
    P.keyed = !(S.flags & (kFlagNonfinite | kFlagRange)) && L.n > 0;
    int g = 32;
    long long c0 = 0, c1 = 0;
    // largest G <= 32 whose cells fit the table; the width shrinks by 2 per step
    for (; g > -100; --g) {
      // products up to 2^64 * 2^32 overflow long long: skip levels that cannot fit anyway
      double span = ldexp(static_cast<double>(S.hi) - static_cast<double>(S.lo), g);
      if (span >= static_cast<double>(p.cell_target)) continue;
      if (fabs(ldexp(static_cast<double>(S.hi), g)) > 9.0e18 ||
          fabs(ldexp(static_cast<double>(S.lo), g)) > 9.0e18) continue;
      c0 = floor_scaled(S.lo, g);
      c1 = floor_scaled(S.hi, g);
      if (c1 - c0 + 1 <= p.cell_target) break;
    }
    P.g = g; P.c0 = c0; P.cells = static_cast<int>(c1 - c0 + 1);
    P.fs = g > 0 ? g : 0;
    P.c0f = static_cast<float>(c0);
    P.two_g = pow2f(g);
    s_plan = P;
    p.plan[l] = P;
  }
  __syncthreads();
  const LayerPlan P = s_plan;
  if (!P.keyed) return;

  // exact lower edge of every bin: smallest float v with bin_of(v) >= b
  float* E = p.edges + static_cast<size_t>(l) * (B + 1);
  const unsigned klo = float_key(S.lo), khi = float_key(S.hi);
  for (int b = threadIdx.x; b <= B; b += kPlanThreads) {
    float e;
    if (b == 0) e = __int_as_float(0xff800000);          // -inf: bin 0 takes everything below
    else if (b == B) e = __int_as_float(0x7f800000);     // +inf
    else if (bin_of(S.hi, S.lo, S.scale, S.bmax) < b) e = __int_as_float(0x7f800000);
    else {
      unsigned a = klo, z = khi;   // bin(a) < b (bin(lo) = 0), bin(z) >= b
      while (z - a > 1) {
        unsigned m = a + ((z - a) >> 1);
        if (bin_of(key_float(m), S.lo, S.scale, S.bmax) >= b) z = m; else a = m;
      }
      e = key_float(z);
    }
    E[b] = e;
  }

  // cell marks
  unsigned* init = p.cell_init + static_cast<size_t>(l) * p.cell_cap;
  for (int c = threadIdx.x; c < P.cells; c += kPlanThreads) {
    const long long cc = P.c0 + c;
    const double left = ldexp(static_cast<double>(cc), -P.g);
    const double right = ldexp(static_cast<double>(cc + 1), -P.g);
    const float lf = __double2float_rd(left), rf = __double2float_ru(right);
    unsigned mark = 0;
    if (bin_of(lf, S.lo, S.scale, S.bmax) != bin_of(rf, S.lo, S.scale, S.bmax)) mark |= kCellEdge;
    if (cc == 0 || cc == -1) mark |= kCellNearZero;
    init[c] = mark;
  }
}

}  // namespace adapt
