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
// already in U.
//
// Two forms.  Layers in the magic-constant forms (cell indices below 2^22, sub-cells under the
// edge cells) take the pyramid form: a CTA per (slice of the cells, layer) does all levels.  The
// counts of the cells of level G summed in pairs are the counts of the cells of level G - 1, and
// the rounded value at level f is a function of the cell of level f + 1 alone (r = (c + 1) >> 1), so
// the CTA halves its slice level by level and bins, per level, only the entries of that level:
// about two entries per cell in all, instead of one per cell and level.  The sub-cells of an
// edge cell go through the same halving inside a warp.  What the cells and sub-cells add to the
// fine levels does not depend on the level (each interior one into its own bin): it is
// gathered once in a shared histogram and added to every level it belongs to.  The other
// layers (keyed by value, or far from zero) keep the level form: a CTA per (level, layer).
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
  int slices;                  // pyramid form: CTAs per layer
  int slice_cap;               // ... and the cells one of them may hold (a multiple of 4)
};

// Level form: this CTA serves slice `slice` of n_slices of the cells at level f (n_levels: the
// float histogram) of the layer.
__device__ __forceinline__ void expand_by_level(const ExpandParams& p, const LayerDesc& L, const LayerPlan& P,
                                                const LayerState& S, int f, int slice, int n_slices,
                                                unsigned* s_hist) {
  __shared__ unsigned long long s_zero;
  const int l = L.index;
  const int B = p.n_bins;
  const bool is_q = (f == p.n_levels);
  // From level f_same on, what the cells and sub-cells add is the same at every level and in the
  // float histogram (interior cells and interior sub-cells, each into its own bin): the float
  // histogram's CTAs compute it once and add it to all of those levels, whose own CTAs only add
  // what differs from level to level (zero counts, edge elements).
  int f_same = p.n_levels;
  if (!P.value) {
    f_same = max(P.seg[0].g, 0);
    if (P.seg[1].cells > 0) f_same = max(f_same, P.seg[1].g);
    f_same = min(f_same, p.n_levels);
  }
  const bool shared_walk = !is_q && f >= f_same;   // this level's cells are served by the Q CTAs

  for (int b = threadIdx.x; b < B; b += kExpandThreads) s_hist[b] = 0;
  if (threadIdx.x == 0) s_zero = 0;
  __syncthreads();

  const unsigned* count = p.cell_count + static_cast<size_t>(l) * p.cell_stride;
  unsigned long long zero = 0;
  // the cells are shared by the n_slices CTAs of this (level, layer), a contiguous slice each
  const int per_slice = ((P.total_cells + n_slices - 1) / n_slices + 3) & ~3;
  const int i_end = min(P.total_cells, (slice + 1) * per_slice);
  // four cells per thread and trip, counts and marks fetched as 128-bit words (slices start on
  // multiples of four cells; the rows are 16-byte aligned and a multiple of four cells long)
  const uint4* count4 = reinterpret_cast<const uint4*>(count);
#pragma unroll 2
  for (int i0 = slice * per_slice + 4 * threadIdx.x; i0 < i_end && !shared_walk; i0 += 4 * kExpandThreads) {
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
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) zero += __shfl_xor_sync(0xffffffffu, zero, o);
  if ((threadIdx.x & 31) == 0 && zero) atomicAdd(&s_zero, zero);
  __syncthreads();

  // the first slice also adds what does not come from cells: exact zeros, edge elements, classes
  const bool lead = (slice == 0);
  const unsigned n_zero =
      lead ? static_cast<unsigned>(static_cast<unsigned long long>(L.n) - p.cell_total[l]) : 0u;
  const int bz = bin_of(0.0f, S.lo, S.scale, S.bmax);
  const unsigned* qe0 = p.qe_hist + static_cast<size_t>(l) * 2 * B;
  const unsigned* qe1 = qe0 + B;
  // the edge-element histograms hold what the level loop looked at: the fine levels
  const int fe0 = P.seg[0].fs;
  const int fe1 = P.seg[1].fs;
  const bool fine0 = lead && (is_q || f >= fe0);
  const bool fine1 = lead && P.seg[1].cells > 0 && (is_q || f >= fe1);
  unsigned* out = is_q ? p.q_hist + static_cast<size_t>(l) * B
                       : p.u_hist + (static_cast<size_t>(l) * p.n_levels + f) * B;
  for (int b = threadIdx.x; b < B; b += kExpandThreads) {
    const unsigned walked = s_hist[b];
    unsigned h = walked + (b == bz ? n_zero : 0u);
    if (fine0) h += qe0[b];
    if (fine1) h += qe1[b];
    if (h) atomicAdd(&out[b], h);     // U holds the corrections, Q starts at zero
    if (is_q && walked)
      for (int g = f_same; g < p.n_levels; ++g)
        atomicAdd(&p.u_hist[(static_cast<size_t>(l) * p.n_levels + g) * B + b], walked);
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

// Pyramid form: this CTA serves slice `slice` of the layer's cells and sub-cells at all levels,
// in one of six roles (segment x part), so that the parts - each a short chain of dependent
// steps - run side by side on different SMs instead of one after the other:
constexpr int kExpandRoles = 6;
constexpr int kRoleCells = 0;     // interior cells into the fine levels and the float histogram
constexpr int kRoleSub = 1;       // sub-cells of the edge cells, edge-element histogram
constexpr int kRoleCoarse = 2;    // the coarse levels by halving
// s_mem: [n_bins] fine histogram, then two buffers for the halving ([slice_cap] and
// [slice_cap / 2 + 2]).
__device__ __forceinline__ void expand_pyramid(const ExpandParams& p, const LayerDesc& L, const LayerPlan& P,
                                               const LayerState& S, int slice, int role, unsigned* s_mem) {
  const int l = L.index;
  const int B = p.n_bins;
  const int F = p.n_levels;
  unsigned* s_fine = s_mem;
  unsigned* buf0 = s_mem + B;
  unsigned* buf1 = buf0 + p.slice_cap;
  const bool lead = (slice == 0 && role == 0);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kWarps = kExpandThreads / 32;
  const int s = role / 3, part = role % 3;
  unsigned* Q = p.q_hist + static_cast<size_t>(l) * B;
  unsigned* U = p.u_hist + static_cast<size_t>(l) * F * B;
  unsigned long long* Z = p.zeros + static_cast<size_t>(l) * F;
  const unsigned* count = p.cell_count + static_cast<size_t>(l) * p.cell_stride;
  const float* E = p.edges + static_cast<size_t>(l) * (B + 1);
  const unsigned* qe = p.qe_hist + static_cast<size_t>(l) * 2 * B;

  // the layer's table is cut into equal slices (multiples of four cells)
  const int per_slice = ((P.total_cells + p.slices - 1) / p.slices + 3) & ~3;
  if (per_slice > p.slice_cap) return;   // cannot happen: the host sized the buffers from the plan's own cap
  const int t_lo = min(P.total_cells, slice * per_slice);
  const int t_hi = min(P.total_cells, t_lo + per_slice);

  if (P.seg[s].cells > 0) {
    const SegPlan& sp = P.seg[s];
    const int g = sp.g;
    const int fs = min(max(g, 0), F);               // first level the interior cells serve
    const int fe = min(max(g + kSubBits, 0), F);    // ... and the interior sub-cells, the edge elements
    if (part != kRoleCoarse) {
      for (int b = threadIdx.x; b < B; b += kExpandThreads) s_fine[b] = 0;
      __syncthreads();
    }

    // this slice's cells of the segment: table positions [a, z)
    const int a = max(t_lo, sp.offset), z = min(t_hi, sp.offset + sp.cells);
    const int n = max(z - a, 0);
    const int c_first = static_cast<int>(sp.c0) + (a - sp.offset);   // |cell index| < 2^22
    if (part == kRoleCells) {
      for (int j = threadIdx.x; j < n; j += kExpandThreads) {
        const unsigned m = __ldg(count + a + j);
        if (m) {
          float lf, rf;
          cell_ends(c_first + j, g, true, &lf, &rf);
          const int bl = bin_of(lf, S.lo, S.scale, S.bmax);
          if (bl == bin_of(rf, S.lo, S.scale, S.bmax) && ADAPT_IN_BOUNDS(bl, B, 31)) atomicAdd(&s_fine[bl], m);
        }
      }
      __syncthreads();
      // levels [fs, F) and the float histogram
      for (int b = threadIdx.x; b < B; b += kExpandThreads) {
        const unsigned h = s_fine[b];
        if (h) {
          atomicAdd(&Q[b], h);
          for (int f = fs; f < F; ++f) atomicAdd(&U[static_cast<size_t>(f) * B + b], h);
        }
      }
    }

    // sub-cells of the segment's edge cells: one warp per edge cell (entry id = the bin in which
    // the cell's left end lies; the cell is the one that holds the bin edge E[id + 1])
    if (part == kRoleSub) {
      const bool narrow = (s == 0 && P.sub_base >= 0);
      const int id_lo = narrow ? P.sub_base : 0;
      const int id_hi = narrow ? min(L.n_bins, P.sub_base + kSubSharedIds) : L.n_bins;
      const int per_ids = (id_hi - id_lo + p.slices - 1) / p.slices;
      const int my_lo = id_lo + slice * per_ids, my_hi = min(id_hi, my_lo + per_ids);
      const unsigned* sub = p.sub_count + (static_cast<size_t>(l) * 2 + s) * B * kSubCells;
      const int gs = g + kSubBits;
      // (the counts and edges of four of the warp's cells are fetched together: the loads are
      // what a warp would otherwise wait for, cell after cell)
      constexpr int kAhead = 4;
      for (int id0 = my_lo + warp; id0 < my_hi; id0 += kWarps * kAhead) {
        unsigned m_in[kAhead];
        float e_in[kAhead];
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
          const int idu = id0 + u * kWarps;
          m_in[u] = idu < my_hi ? __ldg(sub + static_cast<size_t>(idu) * kSubCells + lane) : 0u;
          e_in[u] = (idu < my_hi && ADAPT_IN_BOUNDS(idu + 1, B + 1, 35)) ? __ldg(E + idu + 1) : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
        const unsigned m = m_in[u];
        if (__ballot_sync(0xffffffffu, m != 0u) == 0u) continue;
        const int cc = static_cast<int>(ceil(scale_pow2(static_cast<double>(e_in[u]), g))) - 1;
        const int jj = cc * kSubCells + lane;           // sub-cell index, below 2^27 in magnitude
        // interior sub-cells serve the levels from fe on and the float histogram.  The two ends
        // of the sub-cell, rounded outwards: the cell's left end and the offsets are exact floats
        if (m) {
          const float cl = __fmul_rn(__int2float_rn(cc), pow2f(-g));
          const float l2 = __fadd_rd(cl, __fmul_rn(__int2float_rn(lane), pow2f(-gs)));
          const float r2 = __fadd_ru(cl, __fmul_rn(__int2float_rn(lane + 1), pow2f(-gs)));
          const int bl = bin_of(l2, S.lo, S.scale, S.bmax);
          if (bl == bin_of(r2, S.lo, S.scale, S.bmax) && ADAPT_IN_BOUNDS(bl, B, 33)) atomicAdd(&s_fine[bl], m);
        }
        // levels gs - 1 .. g: the rounded value at level f is a function of the entry of level
        // f + 1, and the entries of level gs - t are sums of 2^t neighbouring sub-cells.  First
        // pass: level gs - 1 from the sub-cells themselves.  Second pass: the entries of the four
        // levels above (16 + 8 + 4 + 2 of them), one per lane, from a prefix sum over the lanes.
        static_assert(kSubBits == 5, "the lane map below is written for 32 sub-cells");
        unsigned pre = m;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned up = __shfl_up_sync(0xffffffffu, pre, o);
          if (lane >= o) pre += up;
        }
        const int t = lane < 16 ? 1 : (lane < 24 ? 2 : (lane < 28 ? 3 : (lane < 30 ? 4 : 0)));
        const int q = lane - (lane < 16 ? 0 : (lane < 24 ? 16 : (lane < 28 ? 24 : 28)));
        const unsigned hi_sum = __shfl_sync(0xffffffffu, pre, (((q + 1) << t) - 1) & 31);
        const unsigned lo_sum = __shfl_sync(0xffffffffu, pre, ((q << t) - 1) & 31);
        const unsigned m2 = (t == 0) ? 0u : hi_sum - (q > 0 ? lo_sum : 0u);
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
          const unsigned mm = pass == 0 ? m : m2;
          const int tt = pass == 0 ? 0 : t;
          const int f = gs - 1 - tt;
          const int entry = pass == 0 ? jj : ((cc * kSubCells) >> tt) + q;
          if (mm != 0u && f >= 0 && f < F) {
            const int r = (entry + 1) >> 1;
            const float v = __fmul_rn(__int2float_rn(r), pow2f(-f));
            const int bv = bin_of(v, S.lo, S.scale, S.bmax);
            if (ADAPT_IN_BOUNDS(bv, B, 34)) atomicAdd(&U[static_cast<size_t>(f) * B + bv], mm);
          }
        }
        }
      }
    }
    if (part == kRoleSub) {
    __syncthreads();
    // levels [fe, F) and the float histogram: interior sub-cells and the elements that the
    // counting kernel binned one by one (their histogram is dealt to the slices by bins)
    const int qe_per = (B + p.slices - 1) / p.slices;
    const int qe_lo = slice * qe_per, qe_hi = min(B, qe_lo + qe_per);
    for (int b = threadIdx.x; b < B; b += kExpandThreads) {
      unsigned h = s_fine[b];
      if (b >= qe_lo && b < qe_hi) h += qe[static_cast<size_t>(s) * B + b];
      if (h) {
        atomicAdd(&Q[b], h);
        for (int f = fe; f < F; ++f) atomicAdd(&U[static_cast<size_t>(f) * B + b], h);
      }
    }
    }

    // coarse levels g - 1 .. 0: bin the entries of level f + 1, then halve.  The whole CTA works
    // while a level has more than 64 entries; the short levels that follow are left to one warp,
    // which needs no CTA-wide barrier between them.
    if (part == kRoleCoarse) {
    for (int j = threadIdx.x; j < n; j += kExpandThreads)
      if (ADAPT_IN_BOUNDS(j, p.slice_cap, 36)) buf0[j] = __ldg(count + a + j);
    __syncthreads();
    unsigned* cur = buf0;
    unsigned* nxt = buf1;
    int cur_first = c_first, cur_n = n;
    int f = g - 1;
    auto level = [&](int tid, int stride) {
      // one pass: entries 2q and 2q + 1 (by absolute index) of the level above are binned at
      // level f and summed into entry q of the next level
      const bool wanted = f < F;
      const float w = pow2f(-f);
      const int nxt_first = cur_first >> 1;
      const int nxt_n = ((cur_first + cur_n - 1) >> 1) - nxt_first + 1;
      for (int j = tid; j < nxt_n; j += stride) {
        const int i0 = 2 * (nxt_first + j) - cur_first;
        unsigned sum = 0;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int i = i0 + e;
          if (i < 0 || i >= cur_n) continue;
          const unsigned m = cur[i];
          if (m == 0u) continue;
          sum += m;
          if (wanted) {
            const int r = (cur_first + i + 1) >> 1;
            const float v = __fmul_rn(__int2float_rn(r), w);
            const int bv = bin_of(v, S.lo, S.scale, S.bmax);
            if (ADAPT_IN_BOUNDS(bv, B, 32)) atomicAdd(&U[static_cast<size_t>(f) * B + bv], m);
            if (r == 0) atomicAdd(&Z[f], static_cast<unsigned long long>(m));
          }
        }
        if (ADAPT_IN_BOUNDS(j, p.slice_cap / 2 + 2, 37)) nxt[j] = sum;
      }
      unsigned* sw = cur; cur = nxt; nxt = sw;
      cur_first = nxt_first; cur_n = nxt_n;
    };
    for (; f >= 0 && cur_n > 64; --f) {
      level(threadIdx.x, kExpandThreads);
      __syncthreads();
    }
    if (warp == 0) {
      for (; f >= 0 && cur_n > 0; --f) {
        level(lane, 32);
        __syncwarp();
      }
    }
    }
  }

  // once per layer: the exact zeros (layer size minus all cell counts) at the bin of 0 in every
  // histogram and in every zero count, and the zero classes at the main segment's fine levels
  if (lead) {
    const unsigned n_zero = static_cast<unsigned>(static_cast<unsigned long long>(L.n) - p.cell_total[l]);
    const int bz = bin_of(0.0f, S.lo, S.scale, S.bmax);
    const unsigned long long* zc = p.zero_class + static_cast<size_t>(l) * kZeroClasses;
    for (int f = threadIdx.x; f <= F; f += kExpandThreads) {
      if (f == F) {
        if (n_zero) atomicAdd(&Q[bz], n_zero);
      } else {
        if (n_zero) atomicAdd(&U[static_cast<size_t>(f) * B + bz], n_zero);
        unsigned long long zsum = n_zero;
        if (f >= P.seg[0].fs)
          for (int k = f; k <= 32; ++k) zsum += zc[k + 1];   // classes whose highest zero level >= f
        if (zsum) atomicAdd(&Z[f], zsum);
      }
    }
  }
}

// blockIdx.y: the layer.  Pyramid form: blockIdx.x = slice and role (the first 6 p.slices CTAs work);
// level form: the levels (and the float histogram) are dealt to the gridDim.x CTAs of the layer.
__global__ void __launch_bounds__(kExpandThreads) expand_kernel(const ExpandParams p) {
  grid_dependency_wait();
  extern __shared__ unsigned s_expand[];
  const LayerDesc L = p.layers[blockIdx.y];
  const LayerPlan P = p.plan[L.index];
  if (!P.keyed) return;
  const LayerState S = p.state[L.index];
  if (P.refined && P.fast && !P.value) {
    if (static_cast<int>(blockIdx.x) < p.slices * kExpandRoles)
      expand_pyramid(p, L, P, S, blockIdx.x / kExpandRoles, blockIdx.x % kExpandRoles, s_expand);
  } else {
    // enough CTAs: each level's cells are cut into slices; too few: a CTA takes several levels
    const int per_level = static_cast<int>(gridDim.x) / (p.n_levels + 1);
    if (per_level >= 1) {
      const int slice = blockIdx.x / (p.n_levels + 1);
      if (slice < per_level) expand_by_level(p, L, P, S, blockIdx.x % (p.n_levels + 1), slice, per_level, s_expand);
    } else {
      for (int f = blockIdx.x; f <= p.n_levels; f += gridDim.x) {
        expand_by_level(p, L, P, S, f, 0, 1, s_expand);
        __syncthreads();
      }
    }
  }
}

}  // namespace adapt
