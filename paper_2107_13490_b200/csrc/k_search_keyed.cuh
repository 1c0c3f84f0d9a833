// K2 (keyed form, round-to-nearest-even): fused multi-candidate quantize +
// zero count + histograms with ONE shared-memory atomic per element on the
// common path.  See k_plan.cuh for the cell decomposition this relies on.
//
// Per element x != 0:   pos = table position of x's cell;  old = atomicAdd(cell[pos], 1)
// The returned word carries the cell's marks in its top bits, and bit 29 is added to it when
// the element sits exactly on the cell grid:
//   bit 30 (cell -1 / 0 of the main segment), bit 31 (edge cell) or bit 29: the element goes
//          to a per-warp queue that the warp drains 32 entries at a time:
//            cell -1 / 0: the element is added to the class counter "highest level at
//              which it still rounds to zero";
//            edge entry: b0 = bin(x) into the segment's edge-element histogram,
//              then only the fine levels f whose half quantum can reach one of
//              the bin's edges are evaluated; a level is recorded only if its
//              bin differs from b0 (-1 at b0, +1 at the new bin).
// An element exactly on the cell grid is counted in the cell to its left or right according to
// the parity rule of grid_point_goes_left (its handler moves the count when it belongs left),
// which makes every coarse rounding tie come out even.
// Exact zeros are sent to per-lane dummy slots (their number is the layer size
// minus the sum of the cell counts).  A dummy slot starts with all three top bits set; zero is
// on every grid, so the added bit 29 wraps the returned word around to a plain small count.
// Everything else about an element - the float histogram, all coarse levels, all fine levels
// of interior cells - is derived from the cell counts by the expand kernel.
//
// Four forms of the counting loop, chosen per layer by the plan (same results, different cost):
//   general  range far from zero (cell indices of 2^22 and more): difference to the first cell first;
//   fast     magic-constant index, grid point = "round-down equals round-up" (two more FMAs);
//   masked   magic-constant index, grid-point flag = "the low significand bits that every grid
//            point of the layer has zero are zero" (a superset, settled exactly by the handler);
//   dense    as masked, for layers with (almost) no exact zeros: no zero test, no flag arithmetic
//            on the returned word; a zero lands in the marked cell [0, 2^-G) and its handler
//            takes it out again.
//
// One CTA of 1024 threads per SM owns (almost) all of the SM's shared memory
// for its tables; each thread handles 16 elements (four 128-bit loads, issued
// together) per tile, and one thread asks for the CTA's next tile to be brought into L2
// by a bulk prefetch while the current one is counted.
#pragma once

#include "common.cuh"
#include "k_plan.cuh"

namespace adapt {

#ifndef ADAPT_KEYED_PF_DIST
#define ADAPT_KEYED_PF_DIST 1    // tiles between the one being counted and the one asked into L2
#endif

constexpr int kKeyedThreads = 1024;
constexpr int kKeyedWarps = kKeyedThreads / 32;
constexpr int kKeyedQuads = 4;                                  // 128-bit loads per thread per tile
constexpr int kKeyedTile = kKeyedThreads * kKeyedQuads * 4;     // 16384 elements
constexpr int kQueueCap = 160;      // per-warp queue entries: under 32 left over + at most 128 from one quad
constexpr int kZeroClasses = 34;    // class k+1, k = highest zero level in -1..32
constexpr int kDummySlots = 32;     // where the atomics of exact zeros land (one per lane)
constexpr int kKeyedPrefetchTiles = ADAPT_KEYED_PF_DIST;   // L2 prefetch distance in tiles (0: none)

struct KeyedParams {
  const LayerDesc* layers;     // keyed layer list (+ sentinel), tiles of kKeyedTile elements
  int n_layers;
  long long n_tiles;
  const LayerState* state;     // by LayerDesc::index
  const LayerPlan* plan;       // by LayerDesc::index
  const float* edges;          // [layer][n_bins + 1]
  unsigned* cell_count;        // [layer][cell_stride]   global cell counts
  unsigned* qe_hist;           // [layer][2][n_bins]     float histogram of the edge elements, per segment
  unsigned* u_hist;            // [layer][n_levels][n_bins]  receives the per-level corrections
  unsigned* q_hist;            // [layer][n_bins]  float histogram (value-keyed layers: stray elements)
  unsigned* sub_count;         // [layer][2][n_bins][kSubCells]  sub-cell counts of the edge cells
  unsigned long long* zeros;   // [layer][n_levels]
  unsigned long long* zero_class;  // [layer][kZeroClasses]
  unsigned long long* cell_total;  // [layer] sum of all cell counts = non-zero elements
  int n_bins;
  int n_levels;                // levels 0..n_levels-1 are wanted
  int cell_cap;                // table entries a layer may use (the other tables follow them)
  int cell_stride;             // row length of the global cell arrays: the largest table any
                               // layer may use, keyed_value_cap() of a value-keyed one
  int d_levels;                // fine levels of the main segment whose corrections stay in shared memory
  const long long* cta_begin;  // [gridDim.x + 1] first tile of every CTA (a CTA's tiles are contiguous);
                               // NULL: equal shares
};

__host__ __device__ inline size_t keyed_smem_bytes(int cell_cap, int n_bins, int d_levels) {
  return sizeof(unsigned) * (static_cast<size_t>(cell_cap) + kDummySlots + n_bins +
                             static_cast<size_t>(d_levels) * n_bins) +
         sizeof(float) * (static_cast<size_t>(n_bins) + 4) +      // the layer's bin edges
         sizeof(unsigned) * kSubSharedIds * kSubCells +          // main segment's sub-cell counts
         sizeof(float) * kKeyedWarps * kQueueCap;
}

// A value-keyed layer needs none of the other tables, so its cells may run over them, up to the
// queues (its dummy slots come last).
__host__ __device__ inline int keyed_value_cap(int cell_cap, int n_bins, int d_levels) {
  const size_t words = static_cast<size_t>(cell_cap) + kDummySlots + n_bins +
                       static_cast<size_t>(d_levels) * n_bins + (static_cast<size_t>(n_bins) + 4) +
                       static_cast<size_t>(kSubSharedIds) * kSubCells;
  return static_cast<int>((words - kDummySlots) & ~static_cast<size_t>(3));
}

// Everything the special-element handler needs about the current layer (in shared memory).
struct LayerCtx {
  float lo, scale, bmax;       // bin function
  float radius;
  float two_g[2], c0f[2];      // cell function per segment (general form)
  long long c0[2];
  int g[2], fs[2], offset[2];
  const float* E;              // shared copy of the layer's exact bin edges [n_bins + 1]
  unsigned* cells;             // shared cell table (marks in the two top bits)
  unsigned* qe;                // shared [n_bins]: main segment's edge-element histogram
  int* d;                      // shared [d_levels][n_bins]
  unsigned* qe_aux;            // global [n_bins]: auxiliary segment's edge-element histogram
  unsigned* u_hist;            // global, this layer's [n_levels][n_bins]
  unsigned long long* zeros;   // global, this layer's [n_levels]
  unsigned* zclass;            // shared [kZeroClasses]
  int n_bins, n_levels, d_levels;
  float magic[2];
  int keyed, fast, total_cells;
  unsigned grid_mask;
  int masked, dense;
  unsigned grid_mul;
  int zero_pos;                // table position of the main segment's cell [0, 2^-G)
  int refined;                 // edge cells have sub-cells
  int fs_edge[2];              // first level the level loop looks at: fs, or the sub-cells' level
  float sub_two[2];            // 2^(G + kSubBits) per segment
  unsigned* sub;               // global, this layer's [2][n_bins][kSubCells]
  unsigned* sub_s;             // shared [kSubSharedIds][kSubCells]: main segment's, when sub_base >= 0
  int sub_base;
  unsigned cells_at, zclass_at, sub_s_at, qe_at, d_at;   // shared addresses of the tables the handler adds to
  int table_words;             // words of the cell table this layer may touch (cells + dummy slots)
  int value;                   // value-keyed layer
  unsigned* q_hist;            // global, this layer's [n_bins]
  unsigned* stray;             // shared: elements of a value-keyed layer that are off its grid
};

// An element that sits exactly on its segment's grid (x * 2^G = p, an integer) is a rounding
// tie at exactly one coarser level (the one whose half quantum is p's lowest set bit), where
// it must go to the even neighbour a or a + 1, a = p >> (lowest set bit + 1).  The cell table
// derives coarse levels from the cell index alone, and cell p rounds such a tie up while cell
// p - 1 rounds it down; at every other level, and as closed intervals for the fine levels, both
// cells serve p equally.  So the element is counted in cell p - 1 when a is even, in cell p
// when a is odd: no correction is ever needed.  (Each segment has one spare cell on its left.)
__device__ __forceinline__ int grid_point_goes_left(long long p) {
  const long long low = p & -p;
  return (p & (low << 1)) == 0 ? 1 : 0;
}

// Handles one queued element (finite).  No warp-level primitive inside:
// any subset of lanes may call it.
__device__ __noinline__ void handle_special(const LayerCtx& c, float x) {
  const int B = c.n_bins;
  if (x == 0.0f) {
    // only the dense form lets an exact zero through: it was counted in the cell [0, 2^-G),
    // where no zero belongs (zeros are the layer size minus all cell counts)
    if (ADAPT_IN_BOUNDS(c.zero_pos, c.table_words, 10)) smem_red_add(c.cells_at + 4u * c.zero_pos, 0xFFFFFFFFu);
    return;
  }
  const int s = (fabsf(x) < c.radius) ? 0 : 1;
  const float z = __fmul_rn(x, c.two_g[s]);
  const float cf = floorf(z);
  int ci = __float2int_rz(__fsub_rn(cf, c.c0f[s])) + 1;     // cell index inside the segment
  if (!ADAPT_IN_BOUNDS(c.offset[s] + ci - 1, c.total_cells, 11) ||
      !ADAPT_IN_BOUNDS(c.offset[s] + ci, c.total_cells, 12)) return;
  if (z == cf && grid_point_goes_left(c.c0[s] + ci)) {
    // on the grid and belonging to the left cell: move its count there
    smem_red_add(c.cells_at + 4u * (c.offset[s] + ci), 0xFFFFFFFFu);
    ci -= 1;
    smem_red_add(c.cells_at + 4u * (c.offset[s] + ci), 1u);
  }
  const long long cc = c.c0[s] + ci;
  // ---- cells -1 / 0 of the main segment: the zero class of x --------------------------
  if (s == 0 && (cc == 0 || cc == -1)) {
    // highest level k at which x still rounds to zero: |x| <= 2^-(k+1)
    const unsigned ax = __float_as_uint(x) & 0x7FFFFFFFu;
    int kz = 125 - static_cast<int>((ax - 1u) >> 23);
    kz = max(-1, min(kz, 32));
    smem_red_add(c.zclass_at + 4u * (kz + 1), 1u);
  }
  // ---- edge cell: its sub-cell, float bin, then the fine levels that can still move ---------
  if (!(c.cells[c.offset[s] + ci] & kCellEdge)) return;
  if (c.refined) {
    // sub-cell index: x * 2^(G + kSubBits) is exact, the cell's first sub-cell index c * 2^kSubBits
    // is a float (c < 2^22), and the two lie within 2^kSubBits of each other.  A point of the
    // sub-grid goes left or right by the same parity rule as a point of the cell grid (for a
    // point of both grids the two decisions agree: the rule does not depend on the scale).
    const float zs = __fmul_rn(x, c.sub_two[s]);
    const float cfs = floorf(zs);
    int j = __float2int_rz(__fsub_rn(cfs, __ll2float_rn(cc * kSubCells)));
    if (zs == cfs && grid_point_goes_left(cc * kSubCells + j)) j -= 1;
    j = max(0, min(j, kSubCells - 1));      // always true by construction; keeps the address in the table
    const long long jj = cc * kSubCells + j;
    const int g = c.g[s];
    // left end of the cell (exact: c < 2^22), then the ends of the sub-cell's closed interval,
    // rounded outwards (c * 2^kSubBits + j can need 27 bits); in float when the powers of two
    // involved are normal numbers - the same real numbers rounded the same way as in double
    float lf, l2, r2;
    if (g >= -120 && g + kSubBits <= 120) {
      const float w2 = pow2f(-(g + kSubBits));
      lf = __fmul_rn(__ll2float_rn(cc), pow2f(-g));
      l2 = __fadd_rd(lf, __fmul_rn(__int2float_rn(j), w2));
      r2 = __fadd_ru(lf, __fmul_rn(__int2float_rn(j + 1), w2));
    } else {
      lf = __double2float_rd(ldexp(static_cast<double>(cc), -g));
      l2 = __double2float_rd(ldexp(static_cast<double>(jj), -(g + kSubBits)));
      r2 = __double2float_ru(ldexp(static_cast<double>(jj + 1), -(g + kSubBits)));
    }
    const int id = bin_of(lf, c.lo, c.scale, c.bmax);
    if (s == 0 && c.sub_base >= 0) {
      if (ADAPT_IN_BOUNDS((id - c.sub_base) * kSubCells + j, kSubSharedIds * kSubCells, 13))
        smem_red_add(c.sub_s_at + 4u * ((id - c.sub_base) * kSubCells + j), 1u);
    } else if (ADAPT_IN_BOUNDS(id, B, 14)) {
      atomicAdd(&c.sub[(static_cast<size_t>(s) * B + id) * kSubCells + j], 1u);
    }
    // an interior sub-cell (its closed interval in one bin) settles the element
    if (bin_of(l2, c.lo, c.scale, c.bmax) == bin_of(r2, c.lo, c.scale, c.bmax)) return;
  }
  const int b0 = bin_of(x, c.lo, c.scale, c.bmax);
  if (!ADAPT_IN_BOUNDS(b0, B, 15)) return;
  if (s == 0) smem_red_add(c.qe_at + 4u * b0, 1u); else atomicAdd(&c.qe_aux[b0], 1u);
  const float e_lo = c.E[b0], e_hi = c.E[b0 + 1];
  // distance to the bin's two edges, rounded down: a level is safe once 2^-(f+1) < margin
  const float m = fminf(__fsub_rd(x, e_lo), __fsub_rd(e_hi, x));
  int f_end = 32;
  if (m > 0.0f) f_end = 126 - static_cast<int>((__float_as_uint(m) - 1u) >> 23);
  f_end = min(f_end, c.n_levels);
  const int fs = c.fs_edge[s];
  for (int f = fs; f < f_end; ++f) {
    const float r = rintf(__fmul_rn(x, pow2f(f)));
    const float v = __fmul_rn(r, pow2f(-f));
    if (v >= e_lo && v < e_hi) continue;       // still in b0 (edges are exact)
    const int b = bin_of(v, c.lo, c.scale, c.bmax);
    if (!ADAPT_IN_BOUNDS(b, B, 16)) continue;
    const int j = f - fs;
    if (s == 0 && j < c.d_levels) {
      smem_red_add(c.d_at + 4u * (j * B + b), 1u);
      smem_red_add(c.d_at + 4u * (j * B + b0), 0xFFFFFFFFu);
    } else {
      unsigned* U = c.u_hist + static_cast<size_t>(f) * B;
      atomicAdd(&U[b], 1u);
      atomicAdd(&U[b0], 0xFFFFFFFFu);
    }
  }
}

// A value-keyed layer's element that is NOT on the layer's grid (the grid was taken from a
// sample): evaluated by itself, every level, straight into the layer's global histograms and
// zero counts, as the direct form of the kernel would.  No warp-level primitive inside.
__device__ __noinline__ void handle_stray(const LayerCtx& c, float x) {
  const int B = c.n_bins;
  atomicAdd(c.stray, 1u);
  if (ADAPT_IN_BOUNDS(bin_of(x, c.lo, c.scale, c.bmax), B, 17)) atomicAdd(&c.q_hist[bin_of(x, c.lo, c.scale, c.bmax)], 1u);
  for (int f = 0; f < c.n_levels; ++f) {
    const float r = rintf(__fmul_rn(x, pow2f(f)));
    const float v = __fmul_rn(r, pow2f(-f));
    if (ADAPT_IN_BOUNDS(bin_of(v, c.lo, c.scale, c.bmax), B, 18))
      atomicAdd(&c.u_hist[static_cast<size_t>(f) * B + bin_of(v, c.lo, c.scale, c.bmax)], 1u);
    if (r == 0.0f) atomicAdd(&c.zeros[f], 1ull);
  }
}

// The constants one tile needs to place an element in the table.
struct CellFn {
  float radius;
  float two_g0, magic0, c0f0;   // main segment
  float two_g1, magic1;         // auxiliary segment (fast layers only)
  unsigned grid_mask;           // masked form: low significand bits every grid point has zero
  unsigned grid_mul;            // dense form: 2^(32 - those bits)
  unsigned cell_base;           // dense form: shared-memory byte address of position 0, minus 4 * 0x4B400000
  unsigned cells_at;            // shared-memory byte address of position 0
#ifdef ADAPT_CHECK_BOUNDS
  int table_words;              // words of the cell table this layer may touch
#endif
};

// How the counting loop finds an element's table position and its grid-point flag.
constexpr int kCellGeneral = 0;   // range far from zero: difference to the first cell formed first
constexpr int kCellFast = 1;      // magic-constant index, grid point = round-down equals round-up
constexpr int kCellMasked = 2;    // magic-constant index, grid-point flag = low significand bits zero
constexpr int kCellDense = 3;     // as masked, for layers with (almost) no exact zeros: a zero is
                                  // not steered to a dummy slot but counted in the cell [0, 2^-G),
                                  // which is marked, and taken out again by the element handler
constexpr int kCellValue = 4;     // value-keyed layer: one cell per grid point, no marks; an element
                                  // that is off the grid (round-down differs from round-up) is not
                                  // counted in the table but handled by itself

// Table position of x, and in *grid_bit kCellOnGrid if x lies exactly on the cell grid, else 0.
// Fast form (all cell indices below 2^22 in magnitude): adding the segment's magic constant
// 1.5 * 2^23 - c0 + offset to x * 2^G with round-down leaves the position in the low mantissa
// bits; x is on the grid exactly when round-up gives the same.  General form (range far from
// zero, one segment): x * 2^G - c0 is formed first - exact, both are close - and the same
// constant trick is applied to the difference.
//
// Masked form: the flag is a cheap superset instead - every grid point of the layer has its
// low significand bits zero (LayerPlan::grid_mask), so those bits being zero sends the element
// to its handler, which tests exactly; a zero passes the test too, as it must.
template <int kMode>
__device__ __forceinline__ int cell_position(float x, const CellFn& f, unsigned* grid_bit) {
  constexpr bool kFast = kMode != kCellGeneral;
  float rd, ru;
  if (kMode == kCellMasked) {
    const bool inner = fabsf(x) < f.radius;
    rd = inner ? __fmaf_rd(x, f.two_g0, f.magic0) : __fmaf_rd(x, f.two_g1, f.magic1);
    *grid_bit = (__float_as_uint(x) & f.grid_mask) == 0u ? kCellOnGrid : 0u;
    return __float_as_int(rd) - 0x4B400000;
  }
  if (kFast) {
    // both segments' products are written out and one is kept: measured faster than selecting
    // the scale and the constant first, by compare-and-select or arithmetically
    const bool inner = fabsf(x) < f.radius;
    rd = inner ? __fmaf_rd(x, f.two_g0, f.magic0) : __fmaf_rd(x, f.two_g1, f.magic1);
    ru = inner ? __fmaf_ru(x, f.two_g0, f.magic0) : __fmaf_ru(x, f.two_g1, f.magic1);
  } else {
    const float t = __fmaf_rn(x, f.two_g0, -f.c0f0);     // x * 2^G - (c0 + 1), exact
    rd = __fadd_rd(t, 12582913.0f);
    ru = __fadd_ru(t, 12582913.0f);
  }
  // A zero is on every grid: in the fast form rd == ru holds for it by itself; in the general
  // form (where only padding can be zero) it lies far outside the table and is named here.
  *grid_bit = (rd == ru || (!kFast && x == 0.0f)) ? kCellOnGrid : 0u;
  return __float_as_int(rd) - 0x4B400000;
}

// Phase A of one quad (four consecutive elements held by this thread), no branches: the four
// atomics are issued together.  Returns whether one of the four must be looked at in phase B.
template <int kMode>
__device__ __forceinline__ bool keyed_count(unsigned* cells, int dummy_pos, const CellFn& fn,
                                            const float (&v)[4], unsigned (&old)[4]) {
  if (kMode == kCellValue) {
    // x * 2^g is an integer for every element on the grid: round-down and round-up of the sum
    // with the magic constant agree, and its low mantissa bits are the table position.  Zeros
    // and stray elements go to the dummy slots; old[k] only says whether element k is a stray.
    unsigned any = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float x = v[k];
      const float rd = __fmaf_rd(x, fn.two_g0, fn.magic0);
      const bool stray = __fmaf_ru(x, fn.two_g0, fn.magic0) != rd;
      const int pos = (x != 0.0f && !stray) ? __float_as_int(rd) - 0x4B400000 : dummy_pos;
      if (ADAPT_IN_BOUNDS(pos, fn.table_words, 1)) smem_red_add(fn.cells_at + 4u * pos, 1u);
      old[k] = stray ? kCellOnGrid : 0u;
      any |= old[k];
    }
    return any != 0u;
  }
  if (kMode == kCellDense) {
    // dense form: no zero test and no flag arithmetic.  The grid-point test is kept apart
    // from the returned words: x's bit pattern times grid_mul is 0 exactly when the low
    // significand bits that every grid point has zero are zero (a zero included, which lands
    // in the marked cell [0, 2^-G) and is queued anyway).
    unsigned any = 0, tmin = 0xFFFFFFFFu;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float x = v[k];
      const bool inner = fabsf(x) < fn.radius;
      const float rd = inner ? __fmaf_rd(x, fn.two_g0, fn.magic0) : __fmaf_rd(x, fn.two_g1, fn.magic1);
      const unsigned addr = __float_as_uint(rd) * 4u + fn.cell_base;
      unsigned o = 0u;
      if (ADAPT_IN_BOUNDS(static_cast<int>(__float_as_uint(rd)) - 0x4B400000, fn.table_words, 2))
        asm volatile("atom.shared.add.u32 %0, [%1], 1;" : "=r"(o) : "r"(addr) : "memory");
      old[k] = o;
      any |= o;
      tmin = min(tmin, __float_as_uint(x) * fn.grid_mul);
    }
    return any >= kCellOnGrid || tmin == 0u;
  }
  // exact zeros go to a dummy slot.  An element on the cell grid gets bit 29 added to its
  // word and is queued too: its handler may move it one cell to the left.  (Slots that are
  // not loaded hold zeros.)
  unsigned any = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float x = v[k];
    unsigned grid_bit;
    int pos = cell_position<kMode>(x, fn, &grid_bit);
    pos = (x != 0.0f) ? pos : dummy_pos;
    const unsigned o = (ADAPT_IN_BOUNDS(pos, fn.table_words, 3) ? smem_atom_add(fn.cells_at + 4u * pos, 1u) : 0u) + grid_bit;
    old[k] = o;
    any |= o;
  }
  return any >= kCellOnGrid;
}

// Phase B of one quad (rare): elements of marked cells and on-grid elements join the warp's
// queue, which is drained when 32 entries have gathered; the whole warp enters so that the
// queue position can stay in a register.
template <int kMode>
__device__ __forceinline__ void keyed_queue(const LayerCtx& c, float* queue, unsigned& qn,
                                            const CellFn& fn, const float (&v)[4],
                                            const unsigned (&old)[4], bool enter) {
  if (__any_sync(0xffffffffu, enter)) {
    const unsigned lt = (1u << (threadIdx.x & 31)) - 1u;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      bool push = old[k] >= kCellOnGrid;
      if (kMode == kCellDense) push = push || __float_as_uint(v[k]) * fn.grid_mul == 0u;
      const unsigned pm = __ballot_sync(0xffffffffu, push);
      if (pm) {
        if (push && ADAPT_IN_BOUNDS(qn + __popc(pm & lt), kQueueCap, 4)) queue[qn + __popc(pm & lt)] = v[k];
        qn += __popc(pm);
      }
    }
    if (qn >= 32u) {           // drain full groups of 32 (dense lanes)
      __syncwarp();
      do {
        qn -= 32u;
        if (kMode == kCellValue) handle_stray(c, queue[qn + (threadIdx.x & 31)]);
        else handle_special(c, queue[qn + (threadIdx.x & 31)]);
      } while (qn >= 32u);
      __syncwarp();
    }
  }
}

template <int kMode>
__device__ __forceinline__ void keyed_quad(const LayerCtx& c, unsigned* cells, int dummy_pos,
                                           float* queue, unsigned& qn, const CellFn& fn,
                                           const float (&v)[4]) {
  unsigned old[4];
  const bool enter = keyed_count<kMode>(cells, dummy_pos, fn, v, old);
  keyed_queue<kMode>(c, queue, qn, fn, v, old, enter);
}

// A ragged tile (the layer's first one when the tensor does not start on a 16-byte boundary, or
// its last): guarded loads, slots outside the layer hold zeros.
template <int kMode>
__device__ __forceinline__ void keyed_tile_ragged(const LayerCtx& c, unsigned* cells, int dummy_pos,
                                                  float* queue, unsigned& qn, const CellFn& fn,
                                                  const float* base, long long j_tile,
                                                  long long jbeg, long long jend) {
  float v[kKeyedQuads][4];
#pragma unroll
  for (int q = 0; q < kKeyedQuads; ++q) {
    const long long j0 = j_tile + 4ll * (q * kKeyedThreads + threadIdx.x);
    v[q][0] = v[q][1] = v[q][2] = v[q][3] = 0.0f;
    if (j0 < jend) load_quad(base, j0, jbeg, jend, v[q]);
  }
#pragma unroll
  for (int q = 0; q < kKeyedQuads; ++q) keyed_quad<kMode>(c, cells, dummy_pos, queue, qn, fn, v[q]);
}

__device__ __forceinline__ void load_full_quad(const float4* src, float (&v)[4]) {
  const float4 t = __ldcs(src);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}

// All tiles [k0, k1) of one layer that this CTA owns (k counts the layer's own tiles).  Only
// the layer's first tile (when the tensor does not start on a 16-byte boundary) and its last
// tile can be ragged; every tile between runs through a loop that carries one running pointer.
// Not inlined: each form then gets its own register allocation under the 64-register cap
// (inlined side by side the four forms spill inside their loops).
template <int kMode>
__device__ __noinline__ void keyed_segment(const LayerCtx& c, unsigned* cells, int dummy_pos,
                                           float* queue, const float* base, long long jbeg,
                                           long long jend, int k0, int k1) {
  // only the constants this form uses are taken into registers
  CellFn fn;
  fn.radius = c.radius;
  fn.two_g0 = c.two_g[0]; fn.magic0 = c.magic[0]; fn.c0f0 = c.c0f[0];
  fn.two_g1 = c.two_g[1]; fn.magic1 = c.magic[1];
  fn.grid_mask = c.grid_mask;
  fn.grid_mul = c.grid_mul;
  fn.cells_at = smem_addr(cells);
  fn.cell_base = fn.cells_at - 4u * 0x4B400000u;
#ifdef ADAPT_CHECK_BOUNDS
  fn.table_words = c.table_words;
#endif
  unsigned qn = 0;             // entries in this warp's queue (same in every lane)
  // a ragged tile pads with zeros, which the dense form must not see
  constexpr int kRagged = kMode == kCellDense ? kCellMasked : kMode;
  const int kf0 = max(k0, jbeg > 0 ? 1 : 0);
  const int kf1 = min(k1, static_cast<int>(jend / kKeyedTile));
  if (k0 < kf0)
    keyed_tile_ragged<kRagged>(c, cells, dummy_pos, queue, qn, fn, base,
                               static_cast<long long>(k0) * kKeyedTile, jbeg, jend);
  if (kf0 < kf1) {
    const float4* src = reinterpret_cast<const float4*>(base + static_cast<long long>(kf0) * kKeyedTile) +
                        threadIdx.x;
    for (int k = kf0; k < kf1; ++k, src += kKeyedTile / 4) {
      // ask for the next tile to be brought into L2 while this one is counted: one bulk
      // request from one thread (requests cut into per-warp pieces, or reaching further
      // ahead, were measured to gain less or to lose)
      if (kKeyedPrefetchTiles > 0 && threadIdx.x == 0 && k + kKeyedPrefetchTiles < kf1)
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::
                     "l"(base + static_cast<long long>(k + kKeyedPrefetchTiles) * kKeyedTile),
                     "r"(kKeyedTile * 4) : "memory");
      // the thread's four quads are loaded first, then counted quad by quad.  (Fetching ahead
      // into registers - the next tile, or half tiles in turn - was measured and lost.)
      float v[kKeyedQuads][4];
#pragma unroll
      for (int q = 0; q < kKeyedQuads; ++q) load_full_quad(src + q * kKeyedThreads, v[q]);
#pragma unroll
      for (int q = 0; q < kKeyedQuads; ++q) keyed_quad<kMode>(c, cells, dummy_pos, queue, qn, fn, v[q]);
    }
  }
  for (int k = max(kf1, kf0); k < k1; ++k)
    keyed_tile_ragged<kRagged>(c, cells, dummy_pos, queue, qn, fn, base,
                               static_cast<long long>(k) * kKeyedTile, jbeg, jend);
  // what is left in the queue
  __syncwarp();
  if ((threadIdx.x & 31) < qn) {
    if (kMode == kCellValue) handle_stray(c, queue[threadIdx.x & 31]);
    else handle_special(c, queue[threadIdx.x & 31]);
  }
}

__global__ void __launch_bounds__(kKeyedThreads, 1) search_keyed_kernel(const KeyedParams p) {
  grid_dependency_wait();
  extern __shared__ __align__(16) unsigned char s_raw[];
  __shared__ unsigned s_zclass[kZeroClasses];
  __shared__ unsigned s_stray;
  __shared__ LayerCtx s_ctx;

  unsigned* cells = reinterpret_cast<unsigned*>(s_raw);          // [cell_cap + kDummySlots]
  unsigned* qe = cells + p.cell_cap + kDummySlots;
  int* dtab = reinterpret_cast<int*>(qe + p.n_bins);
  float* edges = reinterpret_cast<float*>(dtab + static_cast<size_t>(p.d_levels) * p.n_bins);   // [n_bins + 4]
  unsigned* sub_s = reinterpret_cast<unsigned*>(edges + p.n_bins + 4);   // [kSubSharedIds][kSubCells]
  float* queues = reinterpret_cast<float*>(sub_s + kSubSharedIds * kSubCells);

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* queue = queues + warp * kQueueCap;
  const int value_cap = keyed_value_cap(p.cell_cap, p.n_bins, p.d_levels);

  const long long per = (p.n_tiles + gridDim.x - 1) / gridDim.x;
  long long t = p.cta_begin ? p.cta_begin[blockIdx.x] : per * blockIdx.x;
  const long long t_end = p.cta_begin ? min(p.n_tiles, p.cta_begin[blockIdx.x + 1]) : min(p.n_tiles, t + per);
  if (t >= t_end) return;
  int li = layer_of_tile(p.layers, p.n_layers, t);

  while (t < t_end) {
    const LayerDesc L = p.layers[li];
    const int l = L.index;
    unsigned* const layer_u = p.u_hist + static_cast<size_t>(l) * p.n_levels * p.n_bins;
    __syncthreads();             // the previous layer's users of s_ctx are done
    if (threadIdx.x == 0) {
      const LayerState S = p.state[l];
      const LayerPlan* P = p.plan + l;
      LayerCtx c;
      c.lo = S.lo; c.scale = S.scale; c.bmax = S.bmax; c.radius = P->radius;
      c.two_g[0] = P->seg[0].two_g; c.c0f[0] = P->seg[0].c0f; c.c0[0] = P->seg[0].c0;
      c.g[0] = P->seg[0].g; c.fs[0] = P->seg[0].fs; c.offset[0] = P->seg[0].offset;
      c.two_g[1] = P->seg[1].two_g; c.c0f[1] = P->seg[1].c0f; c.c0[1] = P->seg[1].c0;
      c.g[1] = P->seg[1].g; c.fs[1] = P->seg[1].fs; c.offset[1] = P->seg[1].offset;
      c.magic[0] = P->seg[0].magic; c.magic[1] = P->seg[1].magic;
      c.keyed = P->keyed; c.fast = P->fast; c.total_cells = P->total_cells;
      c.grid_mask = P->grid_mask; c.masked = P->masked; c.dense = P->dense;
      c.refined = P->refined;
      for (int sg = 0; sg < 2; ++sg) {
        const int gs = P->seg[sg].g + kSubBits;
        c.fs_edge[sg] = P->refined ? max(gs, 0) : P->seg[sg].fs;
        c.sub_two[sg] = P->refined ? pow2f(max(-126, min(gs, 127))) : 1.0f;
      }
      c.sub = p.sub_count + static_cast<size_t>(l) * 2 * p.n_bins * kSubCells;
      c.sub_s = sub_s; c.sub_base = P->refined ? P->sub_base : -1;
      c.grid_mul = P->grid_mul;
      c.value = P->value;
      c.table_words = (P->value ? keyed_value_cap(p.cell_cap, p.n_bins, p.d_levels) : p.cell_cap) + kDummySlots;
      c.q_hist = p.q_hist + static_cast<size_t>(l) * p.n_bins;
      c.stray = &s_stray;
      c.zero_pos = P->seg[0].offset + static_cast<int>(-P->seg[0].c0);
      c.E = edges;
      c.cells = cells; c.qe = qe; c.d = dtab; c.zclass = s_zclass;
      c.cells_at = smem_addr(cells); c.qe_at = smem_addr(qe); c.d_at = smem_addr(dtab);
      c.zclass_at = smem_addr(s_zclass); c.sub_s_at = smem_addr(sub_s);
      c.qe_aux = p.qe_hist + (static_cast<size_t>(l) * 2 + 1) * p.n_bins;
      c.u_hist = layer_u;
      c.zeros = p.zeros + static_cast<size_t>(l) * p.n_levels;
      c.n_bins = p.n_bins; c.n_levels = p.n_levels; c.d_levels = p.d_levels;
      s_ctx = c;
    }
    __syncthreads();
    const LayerCtx& c = s_ctx;
    const long long layer_tiles_end = min(t_end, p.layers[li + 1].tile_begin);
    const float* base = L.ptr - L.mis;
    const long long jbeg = L.mis, jend = L.mis + L.n;
    const bool ok = c.keyed != 0;
    const bool fast = c.fast != 0;
    const int total_cells = c.total_cells;
    const bool masked = c.masked != 0;
    const bool dense = c.dense != 0;
    const bool by_value = c.value != 0;
    // where the atomics of exact zeros (and of a value-keyed layer's strays) land: one slot per lane
    const int dummy_pos = (by_value ? value_cap : p.cell_cap) + lane;

    // ---- per-layer set-up of the private tables ----------------------------------
    if (ok) {
      if (by_value) {
        // no marks, and the cells may run over the other tables, which this layer does not use
        uint4* cells4 = reinterpret_cast<uint4*>(cells);
        const int n4 = (total_cells + 3) >> 2;
        for (int i = threadIdx.x; i < n4; i += kKeyedThreads) cells4[i] = make_uint4(0u, 0u, 0u, 0u);
      } else {
        // every count starts at zero; the marks follow below
        if (fast) {
          uint4* cells4 = reinterpret_cast<uint4*>(cells);
          const int n4 = (total_cells + 3) >> 2;
          for (int i = threadIdx.x; i < n4; i += kKeyedThreads) cells4[i] = make_uint4(0u, 0u, 0u, 0u);
        } else {
          const LayerState S = p.state[l];
          const LayerPlan P = p.plan[l];
          for (int i = threadIdx.x; i < total_cells; i += kKeyedThreads) cells[i] = cell_mark(P, S, i);
        }
        for (int i = threadIdx.x; i < p.n_bins * (1 + p.d_levels); i += kKeyedThreads) qe[i] = 0;
        const float* layer_edges = p.edges + static_cast<size_t>(l) * (p.n_bins + 1);
        for (int i = threadIdx.x; i <= L.n_bins; i += kKeyedThreads) edges[i] = __ldg(layer_edges + i);
        for (int i = threadIdx.x; i < kSubSharedIds * kSubCells; i += kKeyedThreads) sub_s[i] = 0;
      }
      if (threadIdx.x < kZeroClasses) s_zclass[threadIdx.x] = 0;
      if (threadIdx.x == 0) s_stray = 0;
      if (threadIdx.x < kDummySlots)
        cells[dummy_pos - lane + threadIdx.x] = kCellEdge | kCellNearZero | kCellOnGrid;
    }
    __syncthreads();
    if (ok && fast && !by_value) {
      // Marks of a magic-constant layer, from the bin edges instead of cell by cell: the cell
      // whose closed interval holds the exact edge E[b] (lf < E[b] <= rf, both ends exact here)
      // is cell ceil(E[b] 2^G) - 1 - the same cells the cell-by-cell test marks.
      for (int b = 1 + threadIdx.x; b < L.n_bins; b += kKeyedThreads) {
        const float e = edges[b];
        if (!(fabsf(e) <= 3.402823466e38f)) continue;
#pragma unroll
        for (int sg = 0; sg < 2; ++sg) {
          if (sg == 1 && c.offset[1] >= total_cells) break;      // no auxiliary segment
          const float t = ceilf(__fmul_rn(e, c.two_g[sg]));      // exact product
          if (!(fabsf(t) < 8388608.0f)) continue;
          const int n_seg = (sg == 0) ? (c.offset[1] - c.offset[0]) : (total_cells - c.offset[1]);
          const int ci = __float2int_rz(t) - 1 - static_cast<int>(c.c0[sg]);
          if (ci >= 0 && ci < n_seg) atomicOr(&cells[c.offset[sg] + ci], kCellEdge);
        }
      }
      if (threadIdx.x < 2) {
        const int ci = -static_cast<int>(threadIdx.x) - static_cast<int>(c.c0[0]);   // cells 0 and -1
        if (ci >= 0 && ci < c.offset[1] - c.offset[0]) atomicOr(&cells[c.offset[0] + ci], kCellNearZero);
      }
      __syncthreads();
    }

    if (ok) {
      const int k0 = static_cast<int>(t - L.tile_begin), k1 = static_cast<int>(layer_tiles_end - L.tile_begin);
      if (by_value) keyed_segment<kCellValue>(c, cells, dummy_pos, queue, base, jbeg, jend, k0, k1);
      else if (dense) keyed_segment<kCellDense>(c, cells, dummy_pos, queue, base, jbeg, jend, k0, k1);
      else if (masked) keyed_segment<kCellMasked>(c, cells, dummy_pos, queue, base, jbeg, jend, k0, k1);
      else if (fast) keyed_segment<kCellFast>(c, cells, dummy_pos, queue, base, jbeg, jend, k0, k1);
      else keyed_segment<kCellGeneral>(c, cells, dummy_pos, queue, base, jbeg, jend, k0, k1);
    }
    t = layer_tiles_end;
    __syncthreads();

    // ---- flush the private tables into the layer's global ones -----------------------
    if (ok) {
      unsigned* gc = p.cell_count + static_cast<size_t>(l) * p.cell_stride;
      unsigned long long counted = 0;
      // Cell counts (and the main segment's sub-cell counts below) go through the bulk-copy
      // engine as whole arrays: the marks are taken out of the words first.  Tables of the
      // magic-constant and value-keyed forms are zero-filled in whole quads, so the last quad's
      // spare words add nothing.  (The general form's table is flushed word by word.)
      const bool bulk = fast || by_value;
      // (the sub-cell table follows arrays of n_bins words: 16-byte aligned only for some n_bins)
      const bool bulk_sub = bulk && (smem_addr(sub_s) & 15u) == 0u;
      if (bulk) {
        uint4* cells4 = reinterpret_cast<uint4*>(cells);
        const int n4 = (total_cells + 3) >> 2;
        for (int i = threadIdx.x; i < n4; i += kKeyedThreads) {
          uint4 w = cells4[i];
          w.x &= kCellCountMask; w.y &= kCellCountMask; w.z &= kCellCountMask; w.w &= kCellCountMask;
          cells4[i] = w;
          counted += static_cast<unsigned long long>(w.x) + w.y + w.z + w.w;
        }
      } else {
        for (int i = threadIdx.x; i < total_cells; i += kKeyedThreads) {
          const unsigned n = cells[i] & kCellCountMask;
          if (n) atomicAdd(&gc[i], n);
          counted += n;
        }
      }
      __syncthreads();
      if (threadIdx.x == 0 && bulk) {
        bulk_reduce_add_u32(gc, smem_addr(cells), 16u * static_cast<unsigned>((total_cells + 3) >> 2));
        if (c.sub_base >= 0 && !by_value && bulk_sub) {
          const int room = (p.n_bins - c.sub_base) * kSubCells;
          bulk_reduce_add_u32(c.sub + static_cast<size_t>(c.sub_base) * kSubCells, smem_addr(sub_s),
                              4u * static_cast<unsigned>(min(kSubSharedIds * kSubCells, room)));
        }
        bulk_reduce_commit();
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) counted += __shfl_xor_sync(0xffffffffu, counted, o);
      if (lane == 0 && counted) atomicAdd(&p.cell_total[l], counted);
      if (threadIdx.x == 0 && s_stray) atomicAdd(&p.cell_total[l], static_cast<unsigned long long>(s_stray));
      unsigned* gq = p.qe_hist + static_cast<size_t>(l) * 2 * p.n_bins;
      for (int i = threadIdx.x; i < (by_value ? 0 : p.n_bins); i += kKeyedThreads) {
        const unsigned n = qe[i];
        if (n) atomicAdd(&gq[i], n);
      }
      if (c.sub_base >= 0 && !by_value && !bulk_sub) {
        unsigned* gs = c.sub + static_cast<size_t>(c.sub_base) * kSubCells;     // segment 0, id sub_base
        const int room = (p.n_bins - c.sub_base) * kSubCells;
        for (int i = threadIdx.x; i < min(kSubSharedIds * kSubCells, room); i += kKeyedThreads) {
          const unsigned n = sub_s[i];
          if (n) atomicAdd(&gs[i], n);
        }
      }
      for (int i = threadIdx.x; i < (by_value ? 0 : p.n_bins * p.d_levels); i += kKeyedThreads) {
        const int dv = dtab[i];
        if (dv) {
          const int j = i / p.n_bins, b = i - j * p.n_bins;
          const int f = c.fs_edge[0] + j;
          if (f < p.n_levels)
            atomicAdd(&layer_u[static_cast<size_t>(f) * p.n_bins + b], static_cast<unsigned>(dv));
        }
      }
      if (threadIdx.x < kZeroClasses) {
        const unsigned n = s_zclass[threadIdx.x];
        if (n) atomicAdd(&p.zero_class[static_cast<size_t>(l) * kZeroClasses + threadIdx.x],
                         static_cast<unsigned long long>(n));
      }
      // the engine must have read the tables before the next layer's set-up writes them
      if (threadIdx.x == 0 && bulk) bulk_reduce_wait_read();
    }
    __syncthreads();
    ++li;
    while (li < p.n_layers && p.layers[li + 1].tile_begin <= t) ++li;
  }
  if (threadIdx.x == 0) bulk_reduce_wait_all();
}

}  // namespace adapt
