// Per-layer plan of the keyed search kernel (round-to-nearest-even only).
//
// Idea.  Cut the value axis into cells of width 2^-G.  An element x lies in
// cell c = floor(x * 2^G).  Then, exactly:
//  * for every coarser level f < G the rounded value rint(x * 2^f) is a
//    function of c alone (an x exactly on the level-G grid is a rounding tie at
//    one coarser level; it is counted in the cell to its left when that tie
//    rounds down, which settles it), so one count per cell yields the
//    histograms of all coarse levels afterwards;
//  * for every finer level f >= G the rounded value stays inside the closed
//    cell, so if the whole closed cell lies in one bin ("interior cell") the
//    element falls in that bin at every fine level and in the float histogram;
//  * only elements of cells that contain a bin edge ("edge cells") need their
//    fine levels looked at one by one, and among those only the levels whose
//    half quantum 2^-(f+1) exceeds the element's distance to its bin's edges;
//  * for f >= G an element rounds to zero only if it lies in cell -1 or 0.
// The finer the cells, the fewer elements fall in edge cells or next to zero.
// The table that holds the counts lives in shared memory, so its size is
// fixed; to spend it where the elements are, a layer whose range contains
// zero and whose mass sits in a small part of the range gets TWO segments:
// a main segment of fine cells on [-R, R) (R a power of two, a multiple of the
// mean magnitude found by the range scan) and an auxiliary segment of coarse
// cells over the whole range for the few elements outside.  R only steers
// speed: any R gives the same results.
//
// plan_kernel: make_layer_plan chooses the segments; bin_lower_edge gives the exact bin edges (smallest float of each bin, found with
// the bin function itself); cell_mark gives each cell its marks: bit 31 = edge cell,
// bit 30 = cell -1 or 0 of the main segment.  (Bit 29 is left to the counting kernel, which adds it to the word an
// atomic returns when the element sits exactly on the cell grid.)
#pragma once

#include "common.cuh"

namespace adapt {

constexpr unsigned kCellEdge = 0x80000000u;
constexpr unsigned kCellNearZero = 0x40000000u;
constexpr unsigned kCellOnGrid = 0x20000000u;     // added to a returned word, never stored
constexpr unsigned kCellCountMask = 0x1FFFFFFFu;

// Second level under the edge cells.  An element of an edge cell is counted again in one of
// kSubCells sub-cells (2^-(G + kSubBits) wide) of a table in global memory, indexed by segment,
// by the bin of the edge cell's left end (no two edge cells of a segment share it) and by the
// sub-cell.  Towards the levels G .. G + kSubBits - 1 a sub-cell is what a cell is towards the
// coarse levels, towards the finer levels and the float histogram an interior sub-cell is what
// an interior cell is; only the elements of sub-cells that themselves hold a bin edge still go
// through the level loop.  Used for layers in the magic-constant forms (cell indices below 2^22).
#ifndef ADAPT_SUB_BITS
#define ADAPT_SUB_BITS 5
#endif
constexpr int kSubBits = ADAPT_SUB_BITS;
constexpr int kSubCells = 1 << kSubBits;
// The main segment's edge cells sit where the mass is: a few cells can take a large share of all
// sub-cell counts, so they are kept per CTA in shared memory when the segment's cells start in at
// most this many bins (reductions of all SMs into one line of global memory would serialise).
constexpr int kSubSharedIds = 128;

// Tunables of the table shape (performance only).
#ifndef ADAPT_CELL_BALANCE
#define ADAPT_CELL_BALANCE 4    // cells ~ sqrt(balance * n_bins * elements one CTA sees of the layer)
#endif
#ifndef ADAPT_TWO_SEGMENT_GAIN
#define ADAPT_TWO_SEGMENT_GAIN 0.8   // two segments must promise this much of one segment's edge-cell share, or less
#endif
#ifndef ADAPT_FINE_RATIO
#define ADAPT_FINE_RATIO 512    // stop refining once a bin holds this many cells
#endif

struct SegPlan {
  long long c0;   // cell index of the segment's first cell: floor(left end * 2^G)
  int g;          // cell level G (cells are 2^-G wide); may be negative
  int cells;      // number of cells
  int fs;         // first fine level: max(G, 0)
  int offset;     // position of the segment's first cell in the layer's table
  float two_g;    // 2^G
  float c0f;      // (float)(c0 + 1) = floor(left end * 2^G), exact; c0 itself counts the spare cell
  float magic;    // 1.5 * 2^23 - c0 + offset: x * 2^G + magic, rounded down, has the
                  // table position in its low mantissa bits (fast layers only)
  int pad_;
};

struct LayerPlan {
  SegPlan seg[2];   // [0] main, [1] auxiliary (cells == 0 when unused)
  float radius;     // elements with |x| < radius use the main segment (+inf: all of them)
  int keyed;        // 1 if the layer goes through the keyed kernel
  int fast;         // 1 if every cell index is below 2^22 in magnitude
  int total_cells;  // seg[0].cells + seg[1].cells
  unsigned grid_mask;  // low mantissa bits that are zero in every element on its segment's grid
  int masked;       // 1 if the counting kernel may take "those bits are zero" as its grid-point flag
  int dense;        // 1 if, besides, exact zeros are so rare that they may go through the handler
  int refined;      // 1 if the elements of edge cells are counted once more, in sub-cells
  int sub_base;     // main segment: bin of its first cell's left end, or -1 if the bins its cells
                    // start in number more than kSubSharedIds (its sub-cell counts then go
                    // straight to global memory like the auxiliary segment's)
  unsigned grid_mul;   // 2^(32 - bits of grid_mask): x's bit pattern times this is 0 exactly when those bits are
  int value;        // 1 if the table is keyed by the element's value itself: the layer (as sampled by
                    // the range scan) lies on a grid 2^-g whose points between its extremes fit
                    // the table, so seg[0] has one cell per grid point and no cell has marks
};

// A float x = M 2^(E-23) (M its 24-bit significand) lies on the grid of level G exactly when
// M 2^(E-23+G) is an integer, i.e. when M ends in at least 23 - E - G zero bits.  Over a
// segment whose largest magnitude has exponent E_max, every grid point therefore ends in at
// least T = 23 - E_max - G zero bits: "the low T bits are zero" flags a superset of the grid
// points (about one element in 2^T besides them), which the element handler then tests
// exactly.  Below this many bits the superset is too large to be worth it.
#ifndef ADAPT_MIN_GRID_MASK_BITS
#define ADAPT_MIN_GRID_MASK_BITS 8
#endif
constexpr int kMinGridMaskBits = ADAPT_MIN_GRID_MASK_BITS;
#ifndef ADAPT_DENSE_ZERO_RATIO
#define ADAPT_DENSE_ZERO_RATIO 2048
#endif
constexpr long long kDenseZeroRatio = ADAPT_DENSE_ZERO_RATIO;   // <= 0 switches the dense form off

struct PlanParams {
  const LayerDesc* layers;   // keyed layer list
  const LayerState* state;   // indexed by LayerDesc::index
  LayerPlan* plan;           // indexed by LayerDesc::index
  float* edges;              // [all layers][n_bins + 1] (n_bins = the stride below)
  int n_bins;                // stride of the per-bin arrays (the largest layer's bins)
  int cell_cap;              // table entries a layer may use
  int value_cap;             // ... when it is keyed by value (its table may run over the others)
  int stochastic;            // 1: plans for the stochastic-rounding kernel (one segment, cell indices
                             // exact in float, room for the coarse levels' tables)
  int fine_ratio;            // stop refining once a bin holds this many cells
  long long elems_per_cta;   // elements one CTA of the keyed kernel processes
};

// v * 2^g by one multiplication with a constructed power of two: exact while |g| <= 1000 and the
// product is a normal double (floats times 2^g with |g| <= 200 always are), and far cheaper
// than the library's ldexp for the single thread that plans a layer.
__device__ __forceinline__ double scale_pow2(double v, int g) {
  return v * __hiloint2double((1023 + g) << 20, 0);
}

// Binary exponent of a positive normal double (floor of its base-2 logarithm); 1024 for +inf.
__device__ __forceinline__ int exponent_of(double v) {
  return ((__double2hiint(v) >> 20) & 0x7FF) - 1023;
}

__device__ __forceinline__ long long floor_scaled(float v, int g) {
  // floor(v * 2^g) exactly: the product stays inside double
  return static_cast<long long>(floor(scale_pow2(static_cast<double>(v), g)));
}

// Largest level G <= g_max such that the cells covering [lo, hi] number at most max_cells.
__device__ inline void fit_segment(float lo, float hi, int max_cells, int g_max, SegPlan* s) {
  // the answer is near log2(max_cells / (hi - lo)): start just above it instead of at g_max
  int g = g_max;
  {
    const double span0 = static_cast<double>(hi) - static_cast<double>(lo);
    if (span0 > 1.0e-300 && span0 < 1.0e300) g = min(g_max, exponent_of(static_cast<double>(max_cells)) - exponent_of(span0) + 2);
  }
  long long c0 = 0, c1 = 0;
  for (; g > -100; --g) {
    const double span = scale_pow2(static_cast<double>(hi) - static_cast<double>(lo), g);
    if (span + 1.0 >= static_cast<double>(max_cells)) continue;
    if (fabs(scale_pow2(static_cast<double>(hi), g)) > 9.0e18 ||
        fabs(scale_pow2(static_cast<double>(lo), g)) > 9.0e18) continue;
    c0 = floor_scaled(lo, g) - 1;   // one spare cell on the left (grid points that go left)
    c1 = floor_scaled(hi, g);
    if (c1 - c0 + 1 <= max_cells) break;
  }
  s->g = g; s->c0 = c0; s->cells = static_cast<int>(c1 - c0 + 1);
  s->fs = g > 0 ? g : 0;
  s->two_g = pow2f(g);
  s->c0f = static_cast<float>(c0 + 1);   // floor(lo * 2^G): exactly representable
}

// Level at which a bin of width bw holds about `ratio` cells (no need to go finer).
__device__ inline int level_for_ratio(float lo, float hi, int n_bins, int ratio) {
  const double bw = (static_cast<double>(hi) - static_cast<double>(lo)) / n_bins;
  if (!(bw > 0.0)) return 32;
  const double y = static_cast<double>(ratio) / bw;
  if (!(y < 1.0e300)) return 32;
  if (!(y > 1.0e-300)) return -100;
  // ceil(log2(y)): the exponent, one more unless y is a power of two
  const bool pow2 = (__double2hiint(y) & 0xFFFFF) == 0 && __double2loint(y) == 0;
  const int g = exponent_of(y) + (pow2 ? 0 : 1);
  return max(-100, min(g, 32));
}

// The two ends of cell cc of level g as floats, rounded outwards.  Magic-constant layers keep
// |cc| below 2^22 and g within the normal exponents, so both products are exact in float.
__device__ __forceinline__ void cell_ends(long long cc, int g, bool exact_in_float, float* lf, float* rf) {
  if (exact_in_float && g >= -100 && g <= 100) {
    const float w = pow2f(-g);
    *lf = __fmul_rn(__ll2float_rn(cc), w);
    *rf = __fmul_rn(__ll2float_rn(cc + 1), w);
  } else {
    *lf = __double2float_rd(scale_pow2(static_cast<double>(cc), -g));
    *rf = __double2float_ru(scale_pow2(static_cast<double>(cc + 1), -g));
  }
}

// Marks of table position i of a layer: edge cell (its closed interval meets two bins), cell -1
// or 0 of the main segment.  A value-keyed layer has no marks.
__device__ __forceinline__ unsigned cell_mark(const LayerPlan& P, const LayerState& S, int i) {
  if (P.value) return 0u;
  const int s = (i >= P.seg[1].offset && P.seg[1].cells > 0) ? 1 : 0;
  const SegPlan& sp = P.seg[s];
  const long long cc = sp.c0 + (i - sp.offset);
  float lf, rf;
  cell_ends(cc, sp.g, P.fast != 0, &lf, &rf);
  unsigned mark = 0;
  if (bin_of(lf, S.lo, S.scale, S.bmax) != bin_of(rf, S.lo, S.scale, S.bmax)) mark |= kCellEdge;
  if (s == 0 && (cc == 0 || cc == -1)) mark |= kCellNearZero;
  return mark;
}

// The plan of one layer from its final state: called by all 32 lanes of one warp together (they
// compute the same plan; the candidate radii of the two-segment choice are dealt to the lanes).
__device__ inline void make_layer_plan(const PlanParams& p, const LayerDesc& L, const LayerState& S,
                                       unsigned min_lsb, const int* exp_below, int n_samples,
                                       LayerPlan* out) {
  const int B = L.n_bins;      // this layer's own number of bins
  {
    LayerPlan P;
    P.keyed = !(S.flags & (kFlagNonfinite | kFlagRange)) && L.n > 0;
    P.radius = __int_as_float(0x7f800000);
    P.seg[1].c0 = 0; P.seg[1].g = 0; P.seg[1].cells = 0; P.seg[1].fs = 0; P.seg[1].offset = 0;
    P.seg[1].two_g = 1.0f; P.seg[1].c0f = 0.0f; P.seg[1].magic = 0.0f; P.seg[1].pad_ = 0;
    P.seg[0].pad_ = 0;
    if (p.stochastic) {
      // Stochastic rounding: every level below the cells' costs each element an evaluation, every
      // element of an edge cell a walk over the levels above; about 16 cells per bin balances
      // the two.  The tables of the coarse levels (about as many words as there are cells) must
      // fit beside the cells, and every cell index must be exact in a float.
      const int want_g = level_for_ratio(S.lo, S.hi, B, 16);
      fit_segment(S.lo, S.hi, p.cell_cap, want_g, &P.seg[0]);
      for (;;) {
        long long words = 0;
        for (int f = 0; f < P.seg[0].g && f < kMaxFl; ++f)
          words += floor_scaled(S.hi, f) - floor_scaled(S.lo, f) + 3;
        if (words <= p.cell_cap || P.seg[0].g <= -100) break;
        fit_segment(S.lo, S.hi, p.cell_cap, P.seg[0].g - 1, &P.seg[0]);
      }
      P.seg[0].offset = 0;
      P.seg[1].offset = P.seg[0].cells;
      P.total_cells = P.seg[0].cells;
      const float top = fmaxf(fabsf(S.lo), fabsf(S.hi));
      P.fast = (scale_pow2(static_cast<double>(top), max(P.seg[0].g, 0)) < 4.0e6 && P.seg[0].g >= -100 &&
                P.seg[0].g <= 100) ? 1 : 0;
      if (!P.fast) P.keyed = 0;           // left to the direct kernel
      P.seg[0].magic = 0.0f;
      P.grid_mask = 0u; P.grid_mul = 0u; P.masked = 0; P.dense = 0; P.refined = 0; P.sub_base = -1;
      P.value = 0;
      *out = P;
      return;
    }
    const int g_want = level_for_ratio(S.lo, S.hi, B, p.fine_ratio);
    // every CTA that meets the layer sets up and flushes its private table once (cost ~ cells),
    // while the share of elements that need the slow path falls as n_bins / cells: the sum is
    // least near cells = sqrt(k * n_bins * elements the CTA sees of the layer)
    const double seen = static_cast<double>(min(L.n, p.elems_per_cta));
    const long long want = static_cast<long long>(sqrt(ADAPT_CELL_BALANCE * static_cast<double>(B) * seen));
    const int cap = static_cast<int>(min(static_cast<long long>(p.cell_cap), max(2048ll, want)));
    fit_segment(S.lo, S.hi, cap, g_want, &P.seg[0]);
    // Two segments pay off when zero is inside the range, the single segment cannot reach the
    // wanted fineness, and the mass sits within a small radius.  The radius is the power of two
    // for which the sampled magnitudes promise the fewest elements in edge cells: a segment whose
    // bins hold k cells each leaves about 1/k of its elements there.  (Exact zeros are left out
    // of the estimate: they never sit in an edge cell.)
    const float amax = fmaxf(fabsf(S.lo), fabsf(S.hi));
    if (P.keyed && S.lo <= 0.0f && S.hi >= 0.0f && P.seg[0].g < g_want && n_samples > 0 &&
        amax > 0.0f && amax < 3.0e38f) {
      const double span = static_cast<double>(S.hi) - static_cast<double>(S.lo);
      const double bw = span / B;
      const double share_one = fmin(1.0, scale_pow2(1.0, -P.seg[0].g) / bw);
      const int top_e = static_cast<int>((__float_as_uint(amax) >> 23) & 0xFFu) - 127;   // 2^top_e <= amax
      const int main_cap = cap - cap / 4;
      // one candidate radius 2^e per lane, the largest first
      const int lane = threadIdx.x & 31;
      const int e = top_e - lane;
      double share = 2.0;                           // "not a candidate"
      if (e > -100) {
        const double r = scale_pow2(1.0, e);
        const double span_m = fmin(static_cast<double>(S.hi), r) - fmax(static_cast<double>(S.lo), -r);
        const int g_m = min(g_want, exponent_of((main_cap - 3) / span_m));
        const double cells_m = scale_pow2(span_m, g_m) + 3.0;
        const int g_a = min(g_want, exponent_of((cap - cells_m - 3.0) / span));
        // finer main cells than one segment's, and the auxiliary cells next to zero stay empty
        if (g_m > P.seg[0].g && r > scale_pow2(1.0, -g_a)) {
          // sampled share of the elements below 2^e in magnitude (biased exponent below e + 127)
          const int below = exp_below[max(0, min(e + 127, 255))];
          const double in = static_cast<double>(below) / n_samples;
          share = in * fmin(1.0, scale_pow2(1.0, -g_m) / bw) +
                  (1.0 - in) * fmin(1.0, scale_pow2(1.0, -g_a) / bw);
        }
      }
      // the smallest share wins, the larger radius among equals
      int best_e = e;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const double s2 = __shfl_xor_sync(0xffffffffu, share, o);
        const int e2 = __shfl_xor_sync(0xffffffffu, best_e, o);
        if (s2 < share || (s2 == share && e2 > best_e)) { share = s2; best_e = e2; }
      }
      if (!(share < share_one * ADAPT_TWO_SEGMENT_GAIN)) best_e = -1000;
      if (best_e > -1000) {
        const float r = pow2f(best_e);
        {
          SegPlan aux, main;
          // the main segment takes what it needs (up to three quarters), the rest is auxiliary
          const float mlo = fmaxf(S.lo, -r), mhi = fminf(S.hi, r);
          fit_segment(mlo, mhi, main_cap, g_want, &main);
          fit_segment(S.lo, S.hi, cap - main.cells, g_want, &aux);
          // the auxiliary cells next to zero must stay empty: R at least two of them wide
          if (main.g > P.seg[0].g && r > pow2f(-aux.g)) {
            P.seg[0] = main; P.seg[1] = aux; P.radius = r;
            P.seg[0].pad_ = 0; P.seg[1].pad_ = 0;
          }
        }
      }
    }
    P.seg[0].offset = 0;
    P.seg[1].offset = P.seg[0].cells;
    P.total_cells = P.seg[0].cells + P.seg[1].cells;
    P.fast = 1;
    for (int s = 0; s < 2; ++s) {
      const SegPlan& sp = P.seg[s];
      if (sp.c0 <= -(1ll << 22) || sp.c0 + sp.cells >= (1ll << 22)) P.fast = 0;
    }
    if (P.seg[1].cells > 0 && !P.fast) {   // cannot happen (zero is inside); stay safe
      fit_segment(S.lo, S.hi, cap, g_want, &P.seg[0]);
      P.seg[1].cells = 0; P.radius = __int_as_float(0x7f800000);
      P.total_cells = P.seg[0].cells;
    }
    for (int s = 0; s < 2; ++s)
      P.seg[s].magic = 12582912.0f - static_cast<float>(P.seg[s].c0) +
                       static_cast<float>(P.seg[s].offset);
    int zero_bits = 23;
    for (int s = 0; s < 2; ++s) {
      if (s == 1 && P.seg[1].cells == 0) break;
      // largest magnitude the segment sees: the main segment of two stops below the radius
      float top = amax;
      if (s == 0 && P.seg[1].cells > 0) top = __uint_as_float(__float_as_uint(P.radius) - 1u);
      const int biased = max(1, static_cast<int>((__float_as_uint(top) >> 23) & 0xFFu));
      zero_bits = min(zero_bits, 23 - (biased - 127) - P.seg[s].g);
    }
    P.refined = (P.keyed && P.fast) ? 1 : 0;
    P.sub_base = -1;
    if (P.refined) {
      const SegPlan& m0 = P.seg[0];
      const float first = __double2float_rd(scale_pow2(static_cast<double>(m0.c0), -m0.g));
      const float last = __double2float_rd(scale_pow2(static_cast<double>(m0.c0 + m0.cells - 1), -m0.g));
      const int b_first = bin_of(first, S.lo, S.scale, S.bmax);
      if (bin_of(last, S.lo, S.scale, S.bmax) - b_first < kSubSharedIds) P.sub_base = b_first;
    }
    P.grid_mask = zero_bits >= 1 ? (1u << zero_bits) - 1u : 0u;
    P.masked = (P.fast && zero_bits >= kMinGridMaskBits) ? 1 : 0;
    P.grid_mul = zero_bits >= 1 ? 1u << (32 - zero_bits) : 0u;
    // zeros handled one by one cost about as much as edge elements: fine below one in 2048
    P.dense = (kDenseZeroRatio > 0 && P.masked && S.lo <= 0.0f && S.hi >= 0.0f &&
               static_cast<long long>(S.zero_count) * kDenseZeroRatio <= L.n) ? 1 : 0;
    // A layer that already lies on a fixed-point grid (a layer after its re-quantisation: the
    // float32 simulation of Sec. 4.1 keeps such tensors) is keyed by value when its grid points
    // fit the table: cell i is the single value (c0 + i) 2^-g, every level's rounded value, bin
    // and zero count is an exact function of the cell, and no element is ever on a boundary.
    // The grid comes from a sample; the counting loop checks every element against it.
    P.value = 0;
    if (P.keyed && min_lsb != 0xFFFFFFFFu) {
      const int g = 150 - static_cast<int>(min_lsb);
      if (g >= -100 && g <= 100) {
        const double span = scale_pow2(static_cast<double>(S.hi) - static_cast<double>(S.lo), g);
        const double far = scale_pow2(static_cast<double>(amax), g);
        if (span + 3.0 <= static_cast<double>(p.value_cap) && far < 4.0e6) {
          SegPlan v;
          v.g = g;
          v.c0 = floor_scaled(S.lo, g) - 1;
          v.cells = static_cast<int>(floor_scaled(S.hi, g) - v.c0 + 1);
          v.fs = g > 0 ? g : 0;
          v.offset = 0;
          v.two_g = pow2f(g);
          v.c0f = static_cast<float>(v.c0 + 1);
          v.magic = 12582912.0f - static_cast<float>(v.c0);
          v.pad_ = 0;
          P.seg[0] = v;
          P.seg[1].cells = 0; P.seg[1].offset = v.cells;
          P.radius = __int_as_float(0x7f800000);
          P.total_cells = v.cells;
          P.fast = 1; P.masked = 0; P.dense = 0; P.refined = 0; P.sub_base = -1;
          P.value = 1;
        }
      }
    }
    *out = P;
  }
}

// Exact lower edge of bin b (1 <= b < n_bins) of a layer: the smallest float v with
// bin_of(v) >= b, or +inf if no value up to the layer's maximum reaches the bin.  The bin
// function is monotone, so the edge is found by bisection over the float order.  The bracket
// starts around the estimate lo + b / scale: the bin function rounds v - lo and its product with
// the scale, so the edge lies within a few units in the last place OF THAT DIFFERENCE from the
// estimate (which near zero can be thousands of floats); [lo, hi] is the fallback bracket.
__device__ inline float bin_lower_edge(int b, const LayerState& S) {
  if (bin_of(S.hi, S.lo, S.scale, S.bmax) < b) return __int_as_float(0x7f800000);
  unsigned a = float_key(S.lo), z = float_key(S.hi);   // bin(a) = 0 < b <= bin(z)
  const float t = __fdiv_rn(static_cast<float>(b), S.scale);
  const float guess = __fadd_rn(S.lo, t);
  const float d = __fmul_rn(fmaxf(t, fabsf(guess)), 4.76837158203125e-7f);   // 2^-21 of the larger
  const float ga = __fsub_rn(guess, d), gz = __fadd_rn(guess, d);
  if (ga == ga && gz == gz && d > 0.0f && fabsf(gz) < 3.0e38f && fabsf(ga) < 3.0e38f) {
    const unsigned ka = float_key(ga), kz = float_key(gz);
    if (ka > a && ka < z && bin_of(ga, S.lo, S.scale, S.bmax) < b) a = ka;
    if (kz < z && kz > a && bin_of(gz, S.lo, S.scale, S.bmax) >= b) z = kz;
  }
  while (z - a > 1) {
    const unsigned m = a + ((z - a) >> 1);
    if (bin_of(key_float(m), S.lo, S.scale, S.bmax) >= b) z = m; else a = m;
  }
  return key_float(z);
}

constexpr int kPlanThreads = 256;
constexpr int kPlanSamples = 1024;   // elements of a layer looked at for the grid it lies on
static_assert(kPlanThreads == 256, "the exponent classes are scanned one per thread");

// One layer per blockIdx.x; the gridDim.y CTAs of a layer all derive its plan (one thread each)
// and share its bin edges.
__global__ void __launch_bounds__(kPlanThreads) plan_kernel(const PlanParams p) {
  grid_dependency_wait();
  __shared__ LayerPlan s_plan;
  __shared__ unsigned s_lsb;
  __shared__ int s_exp[256];     // sampled elements by biased exponent, then "below this exponent"
  __shared__ int s_warp[kPlanThreads / 32];
  __shared__ int s_total;
  const LayerDesc L = p.layers[blockIdx.x];
  const int l = L.index;
  const LayerState S = p.state[l];
  // The grid the layer lies on, from a sample of kPlanSamples elements spread over the layer:
  // 150 + the binary exponent of the coarsest grid 2^e that all sampled non-zero elements lie on
  // (biased exponent + trailing zero bits of the 24-bit significand).  It only decides whether
  // the layer is keyed by value; the counting loop checks every element against the grid.
  if (threadIdx.x == 0) s_lsb = 0xFFFFFFFFu;
  for (int i = threadIdx.x; i < 256; i += kPlanThreads) s_exp[i] = 0;
  __syncthreads();
  const long long n_s = min(L.n, static_cast<long long>(kPlanSamples));
  {
    const long long step = n_s > 0 ? L.n / n_s : 1;
    unsigned lsb = 0xFFFFFFFFu;
    for (long long i = threadIdx.x; i < n_s; i += kPlanThreads) {
      const unsigned bits = __float_as_uint(__ldg(L.ptr + i * step));
      const unsigned at = ((bits >> 23) & 0xFFu) + static_cast<unsigned>(__ffs(bits | 0x00800000u) - 1);
      if ((bits & 0x7FFFFFFFu) != 0u) lsb = min(lsb, at);
      if ((bits & 0x7FFFFFFFu) != 0u) atomicAdd(&s_exp[(bits >> 23) & 0xFFu], 1);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lsb = min(lsb, __shfl_xor_sync(0xffffffffu, lsb, o));
    if ((threadIdx.x & 31) == 0 && lsb != 0xFFFFFFFFu) atomicMin(&s_lsb, lsb);
  }
  __syncthreads();
  // the same sample by magnitude: s_exp[k] becomes the number of sampled non-zero elements whose
  // biased exponent is below k (it steers the choice of segments only); kPlanThreads == 256
  {
    const int own = s_exp[threadIdx.x];
    int incl = own;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, incl, o);
      if ((threadIdx.x & 31) >= o) incl += up;
    }
    if ((threadIdx.x & 31) == 31) s_warp[threadIdx.x >> 5] = incl;
    __syncthreads();
    int before = 0;
    for (int w = 0; w < (threadIdx.x >> 5); ++w) before += s_warp[w];
    s_exp[threadIdx.x] = before + incl - own;
    if (threadIdx.x == kPlanThreads - 1) s_total = before + incl;
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    LayerPlan P;
    make_layer_plan(p, L, S, s_lsb, s_exp, s_total, &P);
    if (threadIdx.x == 0) {
      s_plan = P;
      if (blockIdx.y == 0) p.plan[l] = P;
    }
  }
  __syncthreads();
  if (!s_plan.keyed || s_plan.value) return;     // a value-keyed layer needs no bin edges
  // exact lower edge of every bin (bin 0 takes everything below, nothing lies above the last)
  float* E = p.edges + static_cast<size_t>(l) * (p.n_bins + 1);
  for (int b = blockIdx.y * kPlanThreads + threadIdx.x; b <= L.n_bins; b += kPlanThreads * gridDim.y) {
    float e;
    if (b == 0) e = __int_as_float(0xff800000);
    else if (b == L.n_bins) e = __int_as_float(0x7f800000);
    else e = bin_lower_edge(b, S);
    E[b] = e;
  }
}

}  // namespace adapt
