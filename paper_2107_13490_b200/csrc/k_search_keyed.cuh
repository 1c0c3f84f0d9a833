// K2 (keyed form, round-to-nearest-even): fused multi-candidate quantize +
// zero count + histograms with ONE shared-memory atomic per element on the
// common path.  See k_plan.cuh for the cell decomposition this relies on.
//
// Per element x != 0:   pos = table position of x's cell;  old = atomicAdd(cell[pos], 1)
// An element that sits exactly on the cell grid is settled BEFORE its atomic: it is counted in
// the cell to its left or right according to the parity rule of grid_point_goes_left, which
// makes every coarse rounding tie come out even.  (Tensors that already lie on a fixed-point
// grid - a layer after its re-quantisation - consist of such elements only.)
// The returned word carries the cell's marks in its top bits:
//   bit 30 (cell -1 / 0 of the main segment) or bit 31 (edge cell): the element goes to a
//          per-warp queue that the warp drains 32 entries at a time:
//            cell -1 / 0: the element is added to the class counter "highest level at
//              which it still rounds to zero";
//            edge cell: the element is counted once more in a sub-cell of its cell; only when
//              the sub-cell itself holds a bin edge does it join a second per-warp queue, whose
//              full groups of 32 run the level loop: b0 = bin(x) into the segment's
//              edge-element histogram, then only the fine levels f whose half quantum can
//              reach one of the bin's edges are evaluated; a level is recorded only if its
//              bin differs from b0 (-1 at b0, +1 at the new bin).
// Exact zeros are sent to per-lane dummy slots (their number is the layer size
// minus the sum of the cell counts).
// Everything else about an element - the float histogram, all coarse levels, all fine levels
// of interior cells - is derived from the cell counts by the expand kernel.
//
// Four forms of the counting loop, chosen per layer by the plan (same results, different cost):
//   general  range far from zero (cell indices of 2^22 and more): difference to the first cell first;
//   fast     magic-constant index, grid point = "round-down equals round-up" (two more FMAs);
//   masked   magic-constant index, grid-point candidates = "the low significand bits that every
//            grid point of the layer has zero are zero" (a superset, tested exactly only then);
//   dense    as masked, for layers with (almost) no exact zeros: no zero test; a zero lands in
//            the marked cell [0, 2^-G) and its handler takes it out again.
//
// One CTA of 1024 threads per SM owns (almost) all of the SM's shared memory
// for its tables; each thread handles 16 elements (four 128-bit loads, issued
// together) per tile, and one thread asks for the CTA's next tile to be brought into L2
// by a bulk prefetch while the current one is counted.
#pragma once

#include "common.cuh"
#include "k_plan.cuh"
#include "k_range.cuh"

namespace adapt {

#ifndef ADAPT_KEYED_PF_DIST
#define ADAPT_KEYED_PF_DIST 1    // tiles between the one being counted and the one asked into L2
#endif

constexpr int kKeyedThreads = 1024;
constexpr int kKeyedWarps = kKeyedThreads / 32;
constexpr int kKeyedQuads = 4;                                  // 128-bit loads per thread per tile
constexpr int kKeyedTile = kKeyedThreads * kKeyedQuads * 4;     // 16384 elements
constexpr int kQueueCap = 160;      // per-warp queue entries: under 32 left over + at most 128 from one quad
constexpr int kQueue2Cap = 64;      // second per-warp queue (level loop): under 32 left over + one group of 32
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
  const unsigned* cell_init;   // [layer][cell_cap]
  unsigned* cell_count;        // [layer][cell_cap]      global cell counts
  unsigned* qe_hist;           // [layer][2][n_bins]     float histogram of the edge elements, per segment
  unsigned* u_hist;            // [layer][n_levels][n_bins]  receives the per-level corrections
  unsigned* sub_count;         // [layer][2][n_bins][kSubCells]  sub-cell counts of the edge cells
  unsigned long long* zeros;   // [layer][n_levels]
  unsigned long long* zero_class;  // [layer][kZeroClasses]
  unsigned long long* cell_total;  // [layer] sum of all cell counts = non-zero elements
  int n_bins;
  int n_levels;                // levels 0..n_levels-1 are wanted
  int cell_cap;
  int d_levels;                // fine levels of the main segment whose corrections stay in shared memory
};

__host__ __device__ inline size_t keyed_smem_bytes(int cell_cap, int n_bins, int d_levels) {
  return sizeof(unsigned) * (static_cast<size_t>(cell_cap) + kDummySlots + n_bins +
                             static_cast<size_t>(d_levels) * n_bins) +
         sizeof(float) * (static_cast<size_t>(n_bins) + 4) +      // the layer's bin edges
         sizeof(unsigned) * kSubSharedIds * kSubCells +          // main segment's sub-cell counts
         sizeof(float) * kKeyedWarps * (kQueueCap + kQueue2Cap);
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
  int pbias[2];                // fast layers: cell index on the value axis = table position + pbias
  int zero_pos;                // table position of the main segment's cell [0, 2^-G)
  int refined;                 // edge cells have sub-cells
  int fs_edge[2];              // first level the level loop looks at: fs, or the sub-cells' level
  float inv_two_g[2];          // 2^-G per segment (refined layers: a normal float)
  float sub_w[2];              // 2^-(G + kSubBits) per segment: width of a sub-cell
  unsigned* sub;               // global, this layer's [2][n_bins][kSubCells]
  unsigned* sub_s;             // shared [kSubSharedIds][kSubCells]: main segment's, when sub_base >= 0
  int sub_base;
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
// The same rule on the low 32 bits of p (it looks at the lowest set bit and the bit above it;
// callers keep |p| below 2^30).
__device__ __forceinline__ int grid_point_goes_left32(int p) {
  const int low = p & -p;
  return (p & (low << 1)) == 0 ? 1 : 0;
}

// First stage for a queued element (its cell is marked): the zero class of an element next to
// zero, and for an element of an edge cell its sub-cell count.  Returns whether the element
// still has to run the level loop (its sub-cell holds a bin edge, or the layer has no
// sub-cells).  No warp-level primitive inside: any subset of lanes may call it.
__device__ __noinline__ bool handle_queued(const LayerCtx& c, float x) {
  if (x == 0.0f) {
    // only the dense form lets an exact zero through: it was counted in the cell [0, 2^-G),
    // where no zero belongs (zeros are the layer size minus all cell counts)
    atomicSub(&c.cells[c.zero_pos], 1u);
    return false;
  }
  const int s = (fabsf(x) < c.radius) ? 0 : 1;
  const float z = __fmul_rn(x, c.two_g[s]);
  const float cf = floorf(z);
  int ci = __float2int_rz(__fsub_rn(cf, c.c0f[s])) + 1;     // cell index inside the segment
  // a point of the cell grid was counted in the cell the parity rule gives it
  const bool moved = (z == cf) && grid_point_goes_left(c.c0[s] + ci);
  if (moved) ci -= 1;
  const long long cc = c.c0[s] + ci;
  // ---- cells -1 / 0 of the main segment: the zero class of x --------------------------
  if (s == 0 && (cc == 0 || cc == -1)) {
    // highest level k at which x still rounds to zero: |x| <= 2^-(k+1)
    const unsigned ax = __float_as_uint(x) & 0x7FFFFFFFu;
    int kz = 125 - static_cast<int>((ax - 1u) >> 23);
    kz = max(-1, min(kz, 32));
    atomicAdd(&c.zclass[kz + 1], 1u);
  }
  if (!(c.cells[c.offset[s] + ci] & kCellEdge)) return false;
  if (!c.refined) return true;
  // ---- edge cell: its sub-cell ----------------------------------------------------------
  // Refined layers keep every cell index below 2^22 in magnitude, so the cell index is the
  // float cf (less one if the point moved left), its left end cf * 2^-G is exact, and the
  // position inside the cell, (z - cf) * 2^kSubBits, is exact too.  A point of the sub-grid goes
  // left or right by the same parity rule as a point of the cell grid (for a point of both
  // grids the two decisions agree: the rule does not depend on the scale).
  const float cfl = moved ? __fsub_rn(cf, 1.0f) : cf;
  int j = kSubCells - 1;                                    // a point that moved left: last sub-cell
  if (!moved) {
    const float fj = __fmul_rn(__fsub_rn(z, cf), static_cast<float>(kSubCells));
    const float mj = floorf(fj);
    j = __float2int_rz(mj);
    if (fj == mj && j != 0) j -= grid_point_goes_left32(static_cast<int>(cc) * kSubCells + j);
  }
  j = max(0, min(j, kSubCells - 1));      // always true by construction; keeps the address in the table
  const float lf = __fmul_rn(cfl, c.inv_two_g[s]);          // left end of the cell
  const int id = bin_of(lf, c.lo, c.scale, c.bmax);
  if (s == 0 && c.sub_base >= 0) atomicAdd(&c.sub_s[(id - c.sub_base) * kSubCells + j], 1u);
  else atomicAdd(&c.sub[(static_cast<size_t>(s) * c.n_bins + id) * kSubCells + j], 1u);
  // the ends of the sub-cell's closed interval, rounded outwards (cell index * 2^kSubBits + j can
  // need 27 bits); an interior sub-cell (its closed interval in one bin) settles the element
  const float w2 = c.sub_w[s];
  const float l2 = __fadd_rd(lf, __fmul_rn(__int2float_rn(j), w2));
  const float r2 = __fadd_ru(lf, __fmul_rn(__int2float_rn(j + 1), w2));
  return bin_of(l2, c.lo, c.scale, c.bmax) != bin_of(r2, c.lo, c.scale, c.bmax);
}

// Second stage, for the few elements whose (sub-)cell holds a bin edge: the float bin, then the
// fine levels that can still move the element across an edge.  No warp-level primitive inside.
__device__ __noinline__ void level_loop(const LayerCtx& c, float x) {
  const int B = c.n_bins;
  const int s = (fabsf(x) < c.radius) ? 0 : 1;
  const int b0 = bin_of(x, c.lo, c.scale, c.bmax);
  if (s == 0) atomicAdd(&c.qe[b0], 1u); else atomicAdd(&c.qe_aux[b0], 1u);
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
    const int j = f - fs;
    if (s == 0 && j < c.d_levels) {
      atomicAdd(&c.d[j * B + b], 1);
      atomicAdd(&c.d[j * B + b0], -1);
    } else {
      unsigned* U = c.u_hist + static_cast<size_t>(f) * B;
      atomicAdd(&U[b], 1u);
      atomicAdd(&U[b0], 0xFFFFFFFFu);
    }
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
};

// How the counting loop finds an element's table position and its grid points.
constexpr int kCellGeneral = 0;   // range far from zero: difference to the first cell formed first
constexpr int kCellFast = 1;      // magic-constant index, grid point = round-down equals round-up
constexpr int kCellMasked = 2;    // magic-constant index, grid-point candidates = low significand bits zero
constexpr int kCellDense = 3;     // as masked, for layers with (almost) no exact zeros: a zero is
                                  // not steered to a dummy slot but counted in the cell [0, 2^-G),
                                  // which is marked, and taken out again by the element handler

// Magic-constant forms (all cell indices below 2^22 in magnitude): adding the segment's constant
// 1.5 * 2^23 - c0 + offset to x * 2^G with round-down leaves the table position in the low
// mantissa bits of the sum; x is on the cell grid exactly when round-up gives the same sum.
__device__ __forceinline__ float magic_sum_rd(float x, const CellFn& f) {
  // both segments' products are written out and one is kept: measured faster than selecting
  // the scale and the constant first, by compare-and-select or arithmetically
  return fabsf(x) < f.radius ? __fmaf_rd(x, f.two_g0, f.magic0) : __fmaf_rd(x, f.two_g1, f.magic1);
}
__device__ __forceinline__ float magic_sum_ru(float x, const CellFn& f) {
  return fabsf(x) < f.radius ? __fmaf_ru(x, f.two_g0, f.magic0) : __fmaf_ru(x, f.two_g1, f.magic1);
}

// Settles the grid points among four elements of a magic-constant form: rd[k] holds the
// round-down sum of element k; an element exactly on its segment's grid whose parity rule sends
// it left gets the sum of the cell before (one less in the last place).  Zeros are left alone:
// they never count in a cell of their own.  c.c0 - c.offset turns a table position into the
// cell's index on the value axis.
__device__ __forceinline__ void settle_grid_points(const LayerCtx& c, const CellFn& fn,
                                                   const float (&v)[4], float (&rd)[4]) {
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float x = v[k];
    if (x != 0.0f && magic_sum_ru(x, fn) == rd[k]) {
      const int s = fabsf(x) < fn.radius ? 0 : 1;
      const int p = (__float_as_int(rd[k]) - 0x4B400000) + c.pbias[s];
      if (grid_point_goes_left32(p)) rd[k] = __int_as_float(__float_as_int(rd[k]) - 1);
    }
  }
}

// Phase A of one quad (four consecutive elements held by this thread): the four positions, the
// rare settling of grid points, then the four atomics issued together.  Returns whether one of
// the four must be looked at in phase B.
template <int kMode>
__device__ __forceinline__ bool keyed_count(const LayerCtx& c, unsigned* cells, int dummy_pos,
                                            const CellFn& fn, const float (&v)[4],
                                            unsigned (&old)[4]) {
  unsigned any = 0;
  if constexpr (kMode == kCellDense) {
    // dense form: no zero test.  x's bit pattern times grid_mul is 0 exactly when the low
    // significand bits that every grid point has zero are zero (a zero included, which lands
    // in the marked cell [0, 2^-G) and is queued)
    float rd[4];
    unsigned tmin = 0xFFFFFFFFu;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      rd[k] = magic_sum_rd(v[k], fn);
      tmin = min(tmin, __float_as_uint(v[k]) * fn.grid_mul);
    }
    if (tmin == 0u) settle_grid_points(c, fn, v, rd);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const unsigned addr = __float_as_uint(rd[k]) * 4u + fn.cell_base;
      unsigned o;
      asm volatile("atom.shared.add.u32 %0, [%1], 1;" : "=r"(o) : "r"(addr) : "memory");
      old[k] = o;
      any |= o;
    }
    return any >= kCellNearZero;
  } else if constexpr (kMode == kCellMasked) {
    float rd[4];
    bool cand = false;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      rd[k] = magic_sum_rd(v[k], fn);
      cand = cand || (__float_as_uint(v[k]) & fn.grid_mask) == 0u;
    }
    if (cand) settle_grid_points(c, fn, v, rd);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      // exact zeros go to a dummy slot (slots that are not loaded hold zeros)
      const int pos = (v[k] != 0.0f) ? __float_as_int(rd[k]) - 0x4B400000 : dummy_pos;
      const unsigned o = atomicAdd(&cells[pos], 1u);
      old[k] = o;
      any |= o;
    }
    return any >= kCellNearZero;
  } else {
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float x = v[k];
    int pos;
    if (kMode == kCellFast) {
      const float rd = magic_sum_rd(x, fn);
      pos = __float_as_int(rd) - 0x4B400000;
      if (x != 0.0f && magic_sum_ru(x, fn) == rd)
        pos -= grid_point_goes_left32(pos + c.pbias[fabsf(x) < fn.radius ? 0 : 1]);
    } else {
      // general form (range far from zero, one segment at offset 0): x * 2^G - (c0 + 1) is
      // formed first - exact, both are close - and the constant trick applied to the difference
      const float t = __fmaf_rn(x, fn.two_g0, -fn.c0f0);
      const float rd = __fadd_rd(t, 12582913.0f);
      pos = __float_as_int(rd) - 0x4B400000;
      if (x != 0.0f && __fadd_ru(t, 12582913.0f) == rd) pos -= grid_point_goes_left(c.c0[0] + pos);
    }
    pos = (x != 0.0f) ? pos : dummy_pos;
    const unsigned o = atomicAdd(&cells[pos], 1u);
    old[k] = o;
    any |= o;
  }
  return any >= kCellNearZero;
  }
}

// One group of the first queue: the first stage for every lane's entry, then the entries that
// still need the level loop are compacted into the warp's second queue, whose full groups run it.
// Called by the whole warp (lanes without an entry pass valid = false).
__device__ __forceinline__ void keyed_drain(const LayerCtx& c, float x, bool valid, float* queue2,
                                            unsigned* qn2_slot) {
  const bool again = valid && handle_queued(c, x);
  const unsigned pm = __ballot_sync(0xffffffffu, again);
  if (pm) {
    const unsigned lane = threadIdx.x & 31;
    unsigned n2 = *qn2_slot;                   // the same in every lane
    if (again) queue2[n2 + __popc(pm & ((1u << lane) - 1u))] = x;
    n2 += __popc(pm);
    __syncwarp();
    if (n2 >= 32u) {
      n2 -= 32u;
      level_loop(c, queue2[n2 + lane]);
      __syncwarp();
    }
    if (lane == 0) *qn2_slot = n2;
    __syncwarp();
  }
}

// Phase B of one quad (rare): elements of marked cells join the warp's queue, which is drained
// when 32 entries have gathered; the whole warp enters so that the queue position can stay in
// a register.
__device__ __forceinline__ void keyed_queue(const LayerCtx& c, float* queue, unsigned& qn,
                                            float* queue2, unsigned* qn2_slot, const float (&v)[4],
                                            const unsigned (&old)[4], bool enter) {
  if (__any_sync(0xffffffffu, enter)) {
    const unsigned lt = (1u << (threadIdx.x & 31)) - 1u;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const bool push = old[k] >= kCellNearZero;
      const unsigned pm = __ballot_sync(0xffffffffu, push);
      if (pm) {
        if (push) queue[qn + __popc(pm & lt)] = v[k];
        qn += __popc(pm);
      }
    }
    if (qn >= 32u) {           // drain full groups of 32 (dense lanes)
      __syncwarp();
      do {
        qn -= 32u;
        keyed_drain(c, queue[qn + (threadIdx.x & 31)], true, queue2, qn2_slot);
      } while (qn >= 32u);
      __syncwarp();
    }
  }
}

template <int kMode>
__device__ __forceinline__ void keyed_quad(const LayerCtx& c, unsigned* cells, int dummy_pos,
                                           float* queue, unsigned& qn, float* queue2,
                                           unsigned* qn2_slot, const CellFn& fn, const float (&v)[4]) {
  unsigned old[4];
  const bool enter = keyed_count<kMode>(c, cells, dummy_pos, fn, v, old);
  keyed_queue(c, queue, qn, queue2, qn2_slot, v, old, enter);
}

// A ragged tile (the layer's first one when the tensor does not start on a 16-byte boundary, or
// its last): guarded loads, slots outside the layer hold zeros.
template <int kMode>
__device__ __forceinline__ void keyed_tile_ragged(const LayerCtx& c, unsigned* cells, int dummy_pos,
                                                  float* queue, unsigned& qn, float* queue2,
                                                  unsigned* qn2_slot, const CellFn& fn,
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
  for (int q = 0; q < kKeyedQuads; ++q)
    keyed_quad<kMode>(c, cells, dummy_pos, queue, qn, queue2, qn2_slot, fn, v[q]);
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
                                           float* queue, float* queue2, unsigned* qn2_slot,
                                           const float* base, long long jbeg,
                                           long long jend, int k0, int k1) {
  // only the constants this form uses are taken into registers
  CellFn fn;
  fn.radius = c.radius;
  fn.two_g0 = c.two_g[0]; fn.magic0 = c.magic[0]; fn.c0f0 = c.c0f[0];
  fn.two_g1 = c.two_g[1]; fn.magic1 = c.magic[1];
  fn.grid_mask = c.grid_mask;
  fn.grid_mul = c.grid_mul;
  fn.cell_base = static_cast<unsigned>(__cvta_generic_to_shared(cells)) - 4u * 0x4B400000u;
  unsigned qn = 0;             // entries in this warp's queue (same in every lane)
  if ((threadIdx.x & 31) == 0) *qn2_slot = 0;
  __syncwarp();
  // a ragged tile pads with zeros, which the dense form must not see
  constexpr int kRagged = kMode == kCellDense ? kCellMasked : kMode;
  const int kf0 = max(k0, jbeg > 0 ? 1 : 0);
  const int kf1 = min(k1, static_cast<int>(jend / kKeyedTile));
  if (k0 < kf0)
    keyed_tile_ragged<kRagged>(c, cells, dummy_pos, queue, qn, queue2, qn2_slot, fn, base,
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
      for (int q = 0; q < kKeyedQuads; ++q)
        keyed_quad<kMode>(c, cells, dummy_pos, queue, qn, queue2, qn2_slot, fn, v[q]);
    }
  }
  for (int k = max(kf1, kf0); k < k1; ++k)
    keyed_tile_ragged<kRagged>(c, cells, dummy_pos, queue, qn, queue2, qn2_slot, fn, base,
                               static_cast<long long>(k) * kKeyedTile, jbeg, jend);
  // what is left in the two queues
  __syncwarp();
  const unsigned lane = threadIdx.x & 31;
  keyed_drain(c, queue[lane], lane < qn, queue2, qn2_slot);
  __syncwarp();
  if (lane < *qn2_slot) level_loop(c, queue2[lane]);
  __syncwarp();
  if (lane == 0) *qn2_slot = 0;
}

__global__ void __launch_bounds__(kKeyedThreads, 1) search_keyed_kernel(const KeyedParams p) {
  extern __shared__ __align__(16) unsigned char s_raw[];
  __shared__ unsigned s_zclass[kZeroClasses];
  __shared__ unsigned s_qn2[kKeyedWarps];      // entries in each warp's second queue
  __shared__ LayerCtx s_ctx;

  unsigned* cells = reinterpret_cast<unsigned*>(s_raw);          // [cell_cap + kDummySlots]
  unsigned* qe = cells + p.cell_cap + kDummySlots;
  int* dtab = reinterpret_cast<int*>(qe + p.n_bins);
  float* edges = reinterpret_cast<float*>(dtab + static_cast<size_t>(p.d_levels) * p.n_bins);   // [n_bins + 4]
  unsigned* sub_s = reinterpret_cast<unsigned*>(edges + p.n_bins + 4);   // [kSubSharedIds][kSubCells]
  float* queues = reinterpret_cast<float*>(sub_s + kSubSharedIds * kSubCells);

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* queue = queues + warp * kQueueCap;
  float* queue2 = queues + kKeyedWarps * kQueueCap + warp * kQueue2Cap;
  const int dummy_pos = p.cell_cap + lane;

  const long long per = (p.n_tiles + gridDim.x - 1) / gridDim.x;
  long long t = per * blockIdx.x;
  const long long t_end = min(p.n_tiles, t + per);
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
        c.inv_two_g[sg] = P->refined ? pow2f(-P->seg[sg].g) : 1.0f;
        c.sub_w[sg] = P->refined ? pow2f(-gs) : 1.0f;
        c.pbias[sg] = static_cast<int>(P->seg[sg].c0) - P->seg[sg].offset;   // used by fast layers only
      }
      c.sub = p.sub_count + static_cast<size_t>(l) * 2 * p.n_bins * kSubCells;
      c.sub_s = sub_s; c.sub_base = P->refined ? P->sub_base : -1;
      c.grid_mul = P->grid_mul;
      c.zero_pos = P->seg[0].offset + static_cast<int>(-P->seg[0].c0);
      c.E = edges;
      c.cells = cells; c.qe = qe; c.d = dtab; c.zclass = s_zclass;
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

    // ---- per-layer set-up of the private tables ----------------------------------
    if (ok) {
      const unsigned* init = p.cell_init + static_cast<size_t>(l) * p.cell_cap;
      // 128-bit copies, several in flight per thread (the table and its rows are 16-byte aligned,
      // the row has room for the last quad: the table size is a multiple of four)
      const uint4* init4 = reinterpret_cast<const uint4*>(init);
      uint4* cells4 = reinterpret_cast<uint4*>(cells);
      const int n4 = (total_cells + 3) >> 2;
#pragma unroll 4
      for (int i = threadIdx.x; i < n4; i += kKeyedThreads) cells4[i] = __ldg(init4 + i);
      for (int i = threadIdx.x; i < p.n_bins * (1 + p.d_levels); i += kKeyedThreads) qe[i] = 0;
      const float* layer_edges = p.edges + static_cast<size_t>(l) * (p.n_bins + 1);
      for (int i = threadIdx.x; i <= L.n_bins; i += kKeyedThreads) edges[i] = __ldg(layer_edges + i);
      if (threadIdx.x < kZeroClasses) s_zclass[threadIdx.x] = 0;
      for (int i = threadIdx.x; i < kSubSharedIds * kSubCells; i += kKeyedThreads) sub_s[i] = 0;
      if (threadIdx.x < kDummySlots) cells[p.cell_cap + threadIdx.x] = 0;
    }
    __syncthreads();

    if (ok) {
      const int k0 = static_cast<int>(t - L.tile_begin), k1 = static_cast<int>(layer_tiles_end - L.tile_begin);
      if (dense) keyed_segment<kCellDense>(c, cells, dummy_pos, queue, queue2, &s_qn2[warp], base, jbeg, jend, k0, k1);
      else if (masked) keyed_segment<kCellMasked>(c, cells, dummy_pos, queue, queue2, &s_qn2[warp], base, jbeg, jend, k0, k1);
      else if (fast) keyed_segment<kCellFast>(c, cells, dummy_pos, queue, queue2, &s_qn2[warp], base, jbeg, jend, k0, k1);
      else keyed_segment<kCellGeneral>(c, cells, dummy_pos, queue, queue2, &s_qn2[warp], base, jbeg, jend, k0, k1);
    }
    t = layer_tiles_end;
    __syncthreads();

    // ---- flush the private tables into the layer's global ones -----------------------
    if (ok) {
      unsigned* gc = p.cell_count + static_cast<size_t>(l) * p.cell_cap;
      unsigned long long counted = 0;
      for (int i = threadIdx.x; i < total_cells; i += kKeyedThreads) {
        const unsigned n = cells[i] & kCellCountMask;
        if (n) atomicAdd(&gc[i], n);
        counted += n;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) counted += __shfl_xor_sync(0xffffffffu, counted, o);
      if (lane == 0 && counted) atomicAdd(&p.cell_total[l], counted);
      unsigned* gq = p.qe_hist + static_cast<size_t>(l) * 2 * p.n_bins;
      for (int i = threadIdx.x; i < p.n_bins; i += kKeyedThreads) {
        const unsigned n = qe[i];
        if (n) atomicAdd(&gq[i], n);
      }
      if (c.sub_base >= 0) {
        unsigned* gs = c.sub + static_cast<size_t>(c.sub_base) * kSubCells;     // segment 0, id sub_base
        const int room = (p.n_bins - c.sub_base) * kSubCells;
        for (int i = threadIdx.x; i < min(kSubSharedIds * kSubCells, room); i += kKeyedThreads) {
          const unsigned n = sub_s[i];
          if (n) atomicAdd(&gs[i], n);
        }
      }
      for (int i = threadIdx.x; i < p.n_bins * p.d_levels; i += kKeyedThreads) {
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
    }
    __syncthreads();
    ++li;
    while (li < p.n_layers && p.layers[li + 1].tile_begin <= t) ++li;
  }
}

}  // namespace adapt
