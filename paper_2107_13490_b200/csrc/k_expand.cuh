// Expansion of the keyed kernel's cell counts into the per-level histograms.
//
// One CTA (or a few, each with a slice of the cells) per (level, layer); level n_levels
// stands for the float histogram Q.  The CTA walks its cells and adds each cell's count to
// a shared-memory histogram of its level:
//   * float histogram and fine levels (f >= the segment's G), interior cells
//     only: the cell's own bin (elements of edge cells were binned one by one
//     by the keyed kernel into the segment's edge-element histogram, which is
//     added here, and their level-by-level moves already sit in U);
//   * coarse levels (f < G), every cell: the rounded value rint(x * 2^f) of any
//     element of the cell is a + (rem >= half), with c = a * 2^d + rem,
//     d = G - f (grid points whose tie goes down were counted in the cell to their left);
// then the exact zeros (layer size minus all cell counts) at the bin of 0, and
// for the zero counts the cells that round to 0 plus, at fine levels of the
// main segment, the zero classes.  The result is added to the corrections
// already in U.  When there are few (level, layer) pairs the cells are split over several
// CTAs, each adding its part with one global atomic per non-empty bin.
#pragma once

#include "common.cuh"
#include "k_plan.cuh"
#include "k_search_keyed.cuh"

namespace adapt {

constexpr int kExpandThreads = 512;

struct ExpandParams {
  const LayerDesc* layers;     // keyed layer list
  int n_layers;
  const LayerState* state;
  const LayerPlan* plan;
  const unsigned* cell_count;  // [layer][cell_stride]
  const unsigned* qe_hist;     // [layer][2][n_bins]
  const unsigned* sub_count;   // [layer][2][n_bins][kSubCells]  sub-cell counts of the edge cells
  const float* edges;          // [layer][n_bins + 1]  exact bin edges
  unsigned* q_hist;            // [layer][n_bins]
  unsigned* u_hist;            // [layer][n_levels][n_bins]
  unsigned long long* zeros;   // [layer][n_levels]
  const unsigned long long* zero_class;  // [layer][kZeroClasses]
  const unsigned long long* cell_total;  // [layer] non-zero elements (sum of all cell counts)
  int n_bins, n_levels, cell_stride;
};

__global__ void __launch_bounds__(kExpandThreads) expand_kernel(const ExpandParams p) {
  extern __shared__ unsigned s_hist[];          // [n_bins]
  __shared__ unsigned long long s_zero;
  const LayerDesc L = p.layers[blockIdx.y];
  const int l = L.index;
  const LayerPlan P = p.plan[l];
  if (!P.keyed) return;
  const LayerState S = p.state[l];
  const int B = p.n_bins;
  const int f = blockIdx.x;                     // level, or n_levels for the float histogram
  const bool is_q = (f == p.n_levels);

  for (int b = threadIdx.x; b < B; b += kExpandThreads) s_hist[b] = 0;
  if (threadIdx.x == 0) s_zero = 0;
  __syncthreads();

  const unsigned* count = p.cell_count + static_cast<size_t>(l) * p.cell_stride;
  unsigned long long zero = 0;
  // the cells are shared by the gridDim.z CTAs of this (level, layer), a contiguous slice each
  const int per_slice = ((P.total_cells + gridDim.z - 1) / gridDim.z + 3) & ~3;
  const int i_end = min(P.total_cells, static_cast<int>(blockIdx.z + 1) * per_slice);
  // four cells per thread and trip, counts and marks fetched as 128-bit words (slices start on
  // multiples of four cells; the rows are 16-byte aligned and a multiple of four cells long)
  const uint4* count4 = reinterpret_cast<const uint4*>(count);
#pragma unroll 2
  for (int i0 = blockIdx.z * per_slice + 4 * threadIdx.x; i0 < i_end; i0 += 4 * kExpandThreads) {
    const uint4 m4 = __ldg(count4 + (i0 >> 2));
    const unsigned ms[4] = {m4.x, m4.y, m4.z, m4.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int i = i0 + e;
      const unsigned m = ms[e];
      if (m == 0 || i >= i_end) continue;
      const int s = (P.seg[1].cells > 0 && i >= P.seg[1].offset) ? 1 : 0;
      const SegPlan& sp = P.seg[s];
      const long long cc = sp.c0 + (i - sp.offset);
      if (P.value) {
        // value-keyed layer: the cell is the single value cc * 2^-g (exact: |cc| < 2^22)
        const float x = __fmul_rn(__ll2float_rn(cc), pow2f(-sp.g));
        float v = x;
        if (!is_q) {
          const float r = rintf(__fmul_rn(x, pow2f(f)));
          v = __fmul_rn(r, pow2f(-f));
          if (r == 0.0f) zero += m;
        }
        if (ADAPT_IN_BOUNDS(bin_of(v, S.lo, S.scale, S.bmax), B, 30)) atomicAdd(&s_hist[bin_of(v, S.lo, S.scale, S.bmax)], m);
      } else if (is_q || f >= sp.g) {
        // interior cells only (the marks are recomputed: a cell whose closed interval meets two bins)
        float lf, rf;
        cell_ends(cc, sp.g, P.fast != 0, &lf, &rf);
        const int bl = bin_of(lf, S.lo, S.scale, S.bmax);
        if (bl == bin_of(rf, S.lo, S.scale, S.bmax) && ADAPT_IN_BOUNDS(bl, B, 31)) atomicAdd(&s_hist[bl], m);
      } else {
        const int d = sp.g - f;                      // 1..32
        const long long a = cc >> d;                 // floor(c / 2^d)
        const long long rem = cc - (a << d);
        const long long r = a + ((rem >= (1ll << (d - 1))) ? 1 : 0);
        const float v = __fmul_rn(__ll2float_rn(r), pow2f(-f));
        if (ADAPT_IN_BOUNDS(bin_of(v, S.lo, S.scale, S.bmax), B, 32)) atomicAdd(&s_hist[bin_of(v, S.lo, S.scale, S.bmax)], m);
        if (r == 0) zero += m;
      }
    }
  }
  // sub-cells of the edge cells (refined layers).  Entry (segment, id, j): sub-cell j of the edge
  // cell whose left end lies in bin id, i.e. the cell that holds the bin edge E[id + 1] (the
  // cell to its left when that edge sits exactly on the cell grid).  Levels below the
  // segment's G are served by the cell itself; for G <= f < G + kSubBits the sub-cell index
  // fixes the rounded value; for finer levels and the float histogram an interior sub-cell
  // puts its elements into its bin (those of a sub-cell with a bin edge inside were binned one
  // by one).  Sub-cells never add to the zero counts: next to zero the zero classes do.
  if (P.refined) {
    const float* E = p.edges + static_cast<size_t>(l) * (B + 1);
    const unsigned* sub = p.sub_count + static_cast<size_t>(l) * 2 * B * kSubCells;
    for (int s = 0; s < 2; ++s) {
      const SegPlan& sp = P.seg[s];
      if (sp.cells == 0) continue;
      if (!is_q && f < sp.fs) continue;
      const int gs = sp.g + kSubBits;
      // the main segment's counts, when they were kept in shared memory, lie in a short range of ids
      const bool narrow = (s == 0 && P.sub_base >= 0);
      const int k_lo = narrow ? P.sub_base * kSubCells : 0;
      const int k_hi = narrow ? min(L.n_bins, P.sub_base + kSubSharedIds) * kSubCells : L.n_bins * kSubCells;
      const int per_z = ((k_hi - k_lo + gridDim.z - 1) / gridDim.z + 3) & ~3;
      const int k_end = min(k_hi, k_lo + static_cast<int>(blockIdx.z + 1) * per_z);
      const uint4* sub4 = reinterpret_cast<const uint4*>(sub + static_cast<size_t>(s) * B * kSubCells);
      for (int k0 = k_lo + blockIdx.z * per_z + 4 * threadIdx.x; k0 < k_end; k0 += 4 * kExpandThreads) {
        const uint4 m4 = __ldg(sub4 + (k0 >> 2));
        const unsigned ms[4] = {m4.x, m4.y, m4.z, m4.w};
        if ((m4.x | m4.y | m4.z | m4.w) == 0u) continue;
        const int id = k0 / kSubCells;                      // the four share their edge cell
        if (!ADAPT_IN_BOUNDS(id + 1, B + 1, 35)) continue;
        const long long cc = static_cast<long long>(ceil(ldexp(static_cast<double>(E[id + 1]), sp.g))) - 1;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const unsigned m = ms[e];
          if (m == 0) continue;
          const long long jj = cc * kSubCells + ((k0 + e) & (kSubCells - 1));
          if (is_q || f >= gs) {
            const float l2 = __double2float_rd(ldexp(static_cast<double>(jj), -gs));
            const float r2 = __double2float_ru(ldexp(static_cast<double>(jj + 1), -gs));
            const int bl = bin_of(l2, S.lo, S.scale, S.bmax);
            if (bl == bin_of(r2, S.lo, S.scale, S.bmax) && ADAPT_IN_BOUNDS(bl, B, 33)) atomicAdd(&s_hist[bl], m);
          } else {
            const int d = gs - f;                        // 1..kSubBits
            const long long a = jj >> d;
            const long long rem = jj - (a << d);
            const long long r = a + ((rem >= (1ll << (d - 1))) ? 1 : 0);
            const float v = __fmul_rn(__ll2float_rn(r), pow2f(-f));
            if (ADAPT_IN_BOUNDS(bin_of(v, S.lo, S.scale, S.bmax), B, 34)) atomicAdd(&s_hist[bin_of(v, S.lo, S.scale, S.bmax)], m);
          }
        }
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) zero += __shfl_xor_sync(0xffffffffu, zero, o);
  if ((threadIdx.x & 31) == 0 && zero) atomicAdd(&s_zero, zero);
  __syncthreads();

  // the first slice also adds what does not come from cells: exact zeros, edge elements, classes
  const bool lead = (blockIdx.z == 0);
  const unsigned n_zero =
      lead ? static_cast<unsigned>(static_cast<unsigned long long>(L.n) - p.cell_total[l]) : 0u;
  const int bz = bin_of(0.0f, S.lo, S.scale, S.bmax);
  const unsigned* qe0 = p.qe_hist + static_cast<size_t>(l) * 2 * B;
  const unsigned* qe1 = qe0 + B;
  // the edge-element histograms hold what the level loop looked at: from the sub-cells' level on
  const int fe0 = P.refined ? max(P.seg[0].g + kSubBits, 0) : P.seg[0].fs;
  const int fe1 = P.refined ? max(P.seg[1].g + kSubBits, 0) : P.seg[1].fs;
  const bool fine0 = lead && (is_q || f >= fe0);
  const bool fine1 = lead && P.seg[1].cells > 0 && (is_q || f >= fe1);
  unsigned* out = is_q ? p.q_hist + static_cast<size_t>(l) * B
                       : p.u_hist + (static_cast<size_t>(l) * p.n_levels + f) * B;
  for (int b = threadIdx.x; b < B; b += kExpandThreads) {
    unsigned h = s_hist[b] + (b == bz ? n_zero : 0u);
    if (fine0) h += qe0[b];
    if (fine1) h += qe1[b];
    if (h) atomicAdd(&out[b], h);     // U holds the corrections, Q starts at zero
  }
  if (!is_q && threadIdx.x == 0) {
    unsigned long long z = s_zero + n_zero;
    if (lead && f >= P.seg[0].fs) {
      const unsigned long long* zc = p.zero_class + static_cast<size_t>(l) * kZeroClasses;
      for (int k = f; k <= 32; ++k) z += zc[k + 1];   // classes whose highest zero level >= f
    }
    if (z) atomicAdd(&p.zeros[static_cast<size_t>(l) * p.n_levels + f], z);
  }
}

}  // namespace adapt
