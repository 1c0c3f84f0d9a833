// K2 (keyed form, stochastic rounding - the rounding AdaPT trains with, Sec. 3.2):
// fused multi-candidate quantize + zero count + histograms for large layers.
//
// SR(x) at fraction length f is r_f = floor(y) + (P < y - floor(y)), y = x 2^f, with one P per
// element.  Unlike round-to-nearest, r_f is not a function of a cell of x alone, so the levels
// are split at the cell level G (cells [c, c+1) 2^-G on the value axis, G as fine as the
// shared-memory table allows):
//  * coarse levels f < G are evaluated for every element, but only down to the integer r_f:
//    one count in a table of the level's rounded values (their number is (max-min) 2^f, so all
//    coarse tables together are about as large as the cell table).  Bins and zero counts of a
//    coarse level follow from its table afterwards (r_f 2^-f is exact, r_f = 0 is an entry).
//    At the coarsest levels nearly every element rounds to -1, 0 or 1; atomics of a whole warp
//    on three words would serialise, so those three values of every coarse level are counted
//    in lane-private words (one column per lane: no two lanes of a warp meet) and added to the
//    level's table when the CTA leaves the layer; other values take the table's atomics directly.
//  * fine levels f >= G: floor and floor + 1 of such a level both lie inside the element's
//    closed cell, so an element of an interior cell (closed cell inside one bin) falls in the
//    cell's bin at every fine level and in the float histogram, whatever P is: one count per
//    element in the cell table serves them all.  Elements of cells that hold a bin edge, and of
//    cells -1 / 0 (where a fine level can still round to zero), are queued per warp and handled
//    32 at a time: float bin, then only the fine levels whose quantum reaches one of the bin's
//    edges, recorded as differences to the float bin; zero counts of the fine levels one by one.
// Exact zeros touch no table: they are the layer size minus all cell counts.
// Layers whose cell indices would not fit the exact integer range of a float (ranges far from
// zero) are left to the direct kernel; the plan decides (LayerPlan::keyed).
#pragma once

#include "common.cuh"
#include "k_plan.cuh"

namespace adapt {

constexpr int kSrThreads = 1024;
constexpr int kSrWarps = kSrThreads / 32;
constexpr int kSrQuads = 2;                               // 128-bit loads per thread per tile
constexpr int kSrTile = kSrThreads * kSrQuads * 4;        // 8192 elements
constexpr int kSrQueueCap = 96;    // per-warp queue entries: under 32 left over + at most 64 from two quads... see push

struct SrParams {
  const LayerDesc* layers;     // keyed layer list (+ sentinel), tiles of kSrTile elements
  int n_layers;
  long long n_tiles;
  const LayerState* state;     // by LayerDesc::index
  const LayerPlan* plan;       // by LayerDesc::index (seg[0]: the cells; keyed == 0: not served here)
  const float* edges;          // [layer][n_bins + 1]
  unsigned* cell_count;        // [layer][cell_stride]
  unsigned* coarse_count;      // [layer][cell_stride]   tables of the coarse levels, level after level
  unsigned* qe_hist;           // [layer][2][n_bins]     float histogram of the edge-cell elements ([0] used)
  unsigned* u_hist;            // [layer][n_levels][n_bins]  receives the fine levels' differences
  unsigned long long* zeros;   // [layer][n_levels]      receives the fine levels' zero counts
  unsigned long long* cell_total;  // [layer] sum of all cell counts = non-zero elements
  unsigned long long seed;
  int n_bins, n_levels;
  int table_cap;               // words of shared memory for each of the two tables
  int cell_stride;             // row length of the global arrays
  int d_levels;                // fine levels whose differences stay in shared memory
};

__host__ __device__ inline size_t sr_smem_bytes(int table_cap, int n_bins, int d_levels) {
  return sizeof(unsigned) * (2 * static_cast<size_t>(table_cap) + n_bins + static_cast<size_t>(d_levels) * n_bins) +
         sizeof(float) * (static_cast<size_t>(n_bins) + 4) +
         sizeof(float) * 2 * kSrWarps * kSrQueueCap;
}

// The coarse levels of a layer: level f (0 <= f < n_coarse) holds the rounded values
// r in [rmin_f, rmin_f + size_f), rmin_f = floor(lo 2^f) - 1, at table words
// [offset_f, offset_f + size_f).  Both kernels derive the same numbers from the layer's state.
struct SrLevels {
  int n_coarse;                // min(G, n_levels), at least 0
  int fs;                      // first fine level: max(G, 0)
  int bias[kMaxFl];            // table word of value r at level f: r + bias[f]
  int size[kMaxFl];
  int offset[kMaxFl];
  int total;                   // words of all coarse tables
};

__device__ inline void sr_levels(const LayerPlan& P, const LayerState& S, int n_levels, SrLevels* out) {
  const int g = P.seg[0].g;
  out->n_coarse = max(0, min(g, n_levels));
  out->fs = max(g, 0);
  int at = 0;
  for (int f = 0; f < out->n_coarse; ++f) {
    // |x| 2^G < 2^22 for a layer served here, so these products are exact and small
    const int rmin = __float2int_rd(__fmul_rn(S.lo, pow2f(f))) - 1;
    const int rmax = __float2int_rd(__fmul_rn(S.hi, pow2f(f))) + 1;
    out->size[f] = rmax - rmin + 1;
    out->offset[f] = at;
    out->bias[f] = at - rmin;
    at += out->size[f];
  }
  out->total = at;
}

// Everything the kernel needs about the current layer (in shared memory).
struct SrCtx {
  float lo, scale, bmax;
  float two_g, c0f;            // cell index: floor of x 2^G - c0f formed with round-down; c0f = c0 (the spare cell counts)
  int cells;
  int n_coarse, fs;
  int bias[kMaxFl];
  int n_bins, n_levels, d_levels;
  const float* E;              // shared copy of the layer's exact bin edges
  unsigned* cell_tab;          // shared (read in the handler)
  unsigned cell_at, coarse_at, hot_at, qe_at, d_at, zfine_at;   // shared addresses of the tables
  unsigned* u_hist;            // global, this layer's [n_levels][n_bins]
  // hot: shared [kMaxFl][3][32]: values -1, 0, 1 of each coarse level, per lane
  // zfine: shared [kMaxFl + 1]: elements of cells -1 / 0 by the number of fine
                               // levels (from the first one on) at which they round to zero
};

// One queued element: cells -1 / 0 (zero counts of the fine levels) and edge cells (float bin,
// then the fine levels that can move it across a bin edge).  No warp-level primitive inside.
__device__ __noinline__ void sr_handle(const SrCtx& c, float x, float pr) {
  const int B = c.n_bins;
  const float cf = floorf(__fmaf_rd(x, c.two_g, -c.c0f));   // rounded down: never past the next integer
  const int ci = __float2int_rz(cf);
  if (!ADAPT_IN_BOUNDS(ci, c.cells, 50)) return;
  const unsigned w = c.cell_tab[ci];
  const int b0 = bin_of(x, c.lo, c.scale, c.bmax);
  int f_end = c.fs;                                  // levels below f_end are looked at
  float e_lo = 0.0f, e_hi = 0.0f;
  if ((w & kCellEdge) && ADAPT_IN_BOUNDS(b0, B, 51)) {
    smem_red_add(c.qe_at + 4u * b0, 1u);
    e_lo = c.E[b0]; e_hi = c.E[b0 + 1];
    // distance to the bin's two edges, rounded down: a level is safe once 2^-f <= margin
    // (the rounded value lies strictly within 2^-f of x)
    const float m = fminf(__fsub_rd(x, e_lo), __fsub_rd(e_hi, x));
    f_end = c.n_levels;
    if (m > 0.0f) f_end = min(c.n_levels, max(c.fs, 127 - static_cast<int>(__float_as_uint(m) >> 23)));
  }
  if (w & kCellNearZero) {
    // Zero counts of the fine levels.  r_f = 0 holds for a prefix of the levels: for x > 0 as
    // long as x 2^f <= P, for x < 0 as long as floor is -1 and P < 1 - |x| 2^f as rounded, and
    // both sides only move one way as f grows.  The end of the prefix is found by bisection
    // with the level's own arithmetic.
    int lo_f = c.fs, hi_f = c.n_levels;            // zero at every level in [fs, lo_f), none from hi_f on
    while (lo_f < hi_f) {
      const int mid = (lo_f + hi_f) >> 1;
      if (round_scaled<true>(x, pow2f(mid), pr) == 0.0f) lo_f = mid + 1; else hi_f = mid;
    }
    smem_red_add(c.zfine_at + 4u * (lo_f - c.fs), 1u);
  }
  for (int f = c.fs; f < f_end; ++f) {
    const float r = round_scaled<true>(x, pow2f(f), pr);
    const float v = __fmul_rn(r, pow2f(-f));
    if (v >= e_lo && v < e_hi) continue;             // still in b0 (edges are exact)
    const int b = bin_of(v, c.lo, c.scale, c.bmax);
    if (!ADAPT_IN_BOUNDS(b, B, 52)) continue;
    const int j = f - c.fs;
    if (j < c.d_levels) {
      smem_red_add(c.d_at + 4u * (j * B + b), 1u);
      smem_red_add(c.d_at + 4u * (j * B + b0), 0xFFFFFFFFu);
    } else {
      unsigned* U = c.u_hist + static_cast<size_t>(f) * B;
      atomicAdd(&U[b], 1u);
      atomicAdd(&U[b0], 0xFFFFFFFFu);
    }
  }
}

// Four consecutive elements of one thread (index0 = position of v[0] inside the layer; bit k of
// `valid` = element k belongs to the layer).
__device__ __forceinline__ void sr_quad(const SrCtx& c, const SrParams& p, int layer_id, const float (&v)[4],
                                        unsigned valid, long long index0, float* queue, unsigned& qn) {
  float pr[4], y[4];
  unsigned old[4];
  bool live[4];
  unsigned any = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float x = v[k];
    live[k] = ((valid >> k) & 1u) && x != 0.0f;      // zeros touch no table
    const unsigned h = hash24(p.seed, static_cast<unsigned long long>(layer_id),
                              static_cast<unsigned long long>(index0 + k));
    pr[k] = __fmul_rn(__uint2float_rn(h), 5.9604644775390625e-8f);   // h * 2^-24, exact
    y[k] = x;
    // x 2^G - c0 rounded down never passes the next integer: its floor is the cell
    const int ci = __float2int_rz(floorf(__fmaf_rd(x, c.two_g, -c.c0f)));
    old[k] = 0u;
    if (live[k] && ADAPT_IN_BOUNDS(ci, c.cells, 53)) old[k] = smem_atom_add(c.cell_at + 4u * ci, 1u);
    any |= old[k];
  }
  // coarse levels: the rounded value itself is counted; y doubles from level to level (exact).
  // floor(y) without a conversion: y + 1.5 * 2^23 rounded down has it in its low mantissa bits
  // (|y| < 2^22 for every layer served here), and taking the constant off again gives it as a float
  const int lane_word = threadIdx.x & 31;
#pragma unroll 1
  for (int f = 0; f < c.n_coarse; ++f) {
    const int bias = c.bias[f];
    const unsigned hot = c.hot_at + 4u * (f * 96 + lane_word);   // [3][32] words of this level, this lane's column
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float t = __fadd_rd(y[k], 12582912.0f);
      const float fl = __fsub_rn(t, 12582912.0f);               // exact
      const float frac = __fsub_rn(y[k], fl);
      const int r = __float_as_int(t) - 0x4B400000 + ((pr[k] < frac) ? 1 : 0);
      y[k] = __fadd_rn(y[k], y[k]);
      const unsigned d = static_cast<unsigned>(r + 1);
      const unsigned at = (d < 3u) ? hot + 128u * d : c.coarse_at + 4u * static_cast<unsigned>(r + bias);
      if (live[k] && (d < 3u || ADAPT_IN_BOUNDS(r + bias, p.table_cap, 54))) smem_red_add(at, 1u);
    }
  }
  // elements of marked cells join the warp's queue (value and P), drained 32 at a time
  if (__any_sync(0xffffffffu, any >= kCellNearZero)) {
    const unsigned lt = (1u << (threadIdx.x & 31)) - 1u;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const bool push = old[k] >= kCellNearZero;
      const unsigned pm = __ballot_sync(0xffffffffu, push);
      if (pm) {
        const unsigned at = qn + __popc(pm & lt);
        if (push && ADAPT_IN_BOUNDS(at, kSrQueueCap, 56)) { queue[2 * at] = v[k]; queue[2 * at + 1] = pr[k]; }
        qn += __popc(pm);
      }
      if (qn >= 32u) {
        __syncwarp();
        qn -= 32u;
        const unsigned e = qn + (threadIdx.x & 31);
        sr_handle(c, queue[2 * e], queue[2 * e + 1]);
        __syncwarp();
      }
    }
  }
}

__global__ void __launch_bounds__(kSrThreads, 1) search_sr_kernel(const SrParams p) {
  grid_dependency_wait();
  extern __shared__ __align__(16) unsigned char s_raw[];
  __shared__ SrCtx s_ctx;
  __shared__ SrLevels s_lv;
  __shared__ unsigned s_zfine[kMaxFl + 1];
  __shared__ unsigned s_hot[kMaxFl * 96];

  unsigned* cell_tab = reinterpret_cast<unsigned*>(s_raw);                 // [table_cap]
  unsigned* coarse_tab = cell_tab + p.table_cap;                           // [table_cap]
  unsigned* qe = coarse_tab + p.table_cap;                                 // [n_bins]
  int* dtab = reinterpret_cast<int*>(qe + p.n_bins);                       // [d_levels][n_bins]
  float* edges = reinterpret_cast<float*>(dtab + static_cast<size_t>(p.d_levels) * p.n_bins);   // [n_bins + 4]
  float* queues = edges + p.n_bins + 4;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* queue = queues + 2 * warp * kSrQueueCap;

  const long long per = (p.n_tiles + gridDim.x - 1) / gridDim.x;
  long long t = per * blockIdx.x;
  const long long t_end = min(p.n_tiles, t + per);
  if (t >= t_end) return;
  int li = layer_of_tile(p.layers, p.n_layers, t);

  while (t < t_end) {
    const LayerDesc L = p.layers[li];
    const int l = L.index;
    const long long layer_tiles_end = min(t_end, p.layers[li + 1].tile_begin);
    __syncthreads();             // the previous layer's users of the shared context are done
    if (threadIdx.x == 0) {
      const LayerState S = p.state[l];
      const LayerPlan P = p.plan[l];
      sr_levels(P, S, p.n_levels, &s_lv);
      SrCtx c;
      c.lo = S.lo; c.scale = S.scale; c.bmax = S.bmax;
      c.two_g = P.seg[0].two_g; c.c0f = static_cast<float>(P.seg[0].c0);
      c.cells = P.keyed ? P.seg[0].cells : 0;
      c.n_coarse = s_lv.n_coarse; c.fs = s_lv.fs;
      for (int f = 0; f < kMaxFl; ++f) c.bias[f] = f < s_lv.n_coarse ? s_lv.bias[f] : 0;
      c.n_bins = p.n_bins; c.n_levels = p.n_levels; c.d_levels = p.d_levels;
      c.E = edges; c.cell_tab = cell_tab;
      c.cell_at = smem_addr(cell_tab); c.coarse_at = smem_addr(coarse_tab); c.qe_at = smem_addr(qe);
      c.d_at = smem_addr(dtab);
      c.u_hist = p.u_hist + static_cast<size_t>(l) * p.n_levels * p.n_bins;
      c.zfine_at = smem_addr(s_zfine); c.hot_at = smem_addr(s_hot);
      s_ctx = c;
    }
    __syncthreads();
    const SrCtx& c = s_ctx;
    const bool ok = c.cells > 0 && s_lv.total <= p.table_cap && c.cells <= p.table_cap;
    const int coarse_words = s_lv.total;

    if (ok) {
      for (int i = threadIdx.x; i < c.cells; i += kSrThreads) cell_tab[i] = 0;
      for (int i = threadIdx.x; i < coarse_words; i += kSrThreads) coarse_tab[i] = 0;
      for (int i = threadIdx.x; i < p.n_bins * (1 + p.d_levels); i += kSrThreads) qe[i] = 0;
      const float* layer_edges = p.edges + static_cast<size_t>(l) * (p.n_bins + 1);
      for (int i = threadIdx.x; i <= L.n_bins; i += kSrThreads) edges[i] = __ldg(layer_edges + i);
      if (threadIdx.x <= kMaxFl) s_zfine[threadIdx.x] = 0;
      for (int i = threadIdx.x; i < kMaxFl * 96; i += kSrThreads) s_hot[i] = 0;
    }
    __syncthreads();
    if (ok) {
      // marks: the cell whose closed interval holds the exact edge E[b] is cell ceil(E[b] 2^G) - 1
      for (int b = 1 + threadIdx.x; b < L.n_bins; b += kSrThreads) {
        const float e = edges[b];
        if (!(fabsf(e) <= 3.402823466e38f)) continue;
        const float tt = ceilf(__fmul_rn(e, c.two_g));
        if (!(fabsf(tt) < 8388608.0f)) continue;
        const int ci = __float2int_rz(tt) - 1 - __float2int_rz(c.c0f);
        if (ci >= 0 && ci < c.cells) atomicOr(&cell_tab[ci], kCellEdge);
      }
      if (threadIdx.x < 2) {
        const int ci = -static_cast<int>(threadIdx.x) - __float2int_rz(c.c0f);     // cells 0 and -1
        if (ci >= 0 && ci < c.cells) atomicOr(&cell_tab[ci], kCellNearZero);
      }
    }
    __syncthreads();

    if (ok) {
      const float* base = L.ptr - L.mis;
      const long long jbeg = L.mis, jend = L.mis + L.n;
      unsigned qn = 0;
      for (; t < layer_tiles_end; ++t) {
        const long long j_tile = (t - L.tile_begin) * kSrTile;
        float v[kSrQuads][4];
        unsigned m[kSrQuads];
#pragma unroll
        for (int q = 0; q < kSrQuads; ++q) {
          const long long j0 = j_tile + 4ll * (q * kSrThreads + threadIdx.x);
          m[q] = 0u;
          v[q][0] = v[q][1] = v[q][2] = v[q][3] = 0.0f;
          if (j0 < jend) m[q] = load_quad(base, j0, jbeg, jend, v[q]);
        }
#pragma unroll
        for (int q = 0; q < kSrQuads; ++q) {
          const long long j0 = j_tile + 4ll * (q * kSrThreads + threadIdx.x);
          sr_quad(c, p, L.layer_id, v[q], m[q], j0 - jbeg, queue, qn);
        }
      }
      // what is left in the queue
      __syncwarp();
      if (static_cast<unsigned>(lane) < qn) sr_handle(c, queue[2 * lane], queue[2 * lane + 1]);
    }
    t = layer_tiles_end;
    __syncthreads();

    // ---- flush the private tables into the layer's global ones -----------------------
    if (ok) {
      unsigned* gc = p.cell_count + static_cast<size_t>(l) * p.cell_stride;
      unsigned long long counted = 0;
      for (int i = threadIdx.x; i < c.cells; i += kSrThreads) {
        const unsigned n = cell_tab[i] & kCellCountMask;
        if (n) atomicAdd(&gc[i], n);
        counted += n;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) counted += __shfl_xor_sync(0xffffffffu, counted, o);
      if (lane == 0 && counted) atomicAdd(&p.cell_total[l], counted);
      unsigned* gr = p.coarse_count + static_cast<size_t>(l) * p.cell_stride;
      for (int i = threadIdx.x; i < coarse_words; i += kSrThreads) {
        const unsigned n = coarse_tab[i];
        if (n) atomicAdd(&gr[i], n);
      }
      // the lane-private counts of the values -1, 0, 1: one warp per (level, value)
      for (int k = warp; k < 3 * c.n_coarse; k += kSrWarps) {
        const int f = k / 3, d = k - 3 * f;
        const unsigned n = __reduce_add_sync(0xffffffffu, s_hot[f * 96 + d * 32 + lane]);
        if (lane == 0 && n) atomicAdd(&gr[d - 1 + c.bias[f]], n);
      }
      unsigned* gq = p.qe_hist + static_cast<size_t>(l) * 2 * p.n_bins;
      for (int i = threadIdx.x; i < p.n_bins; i += kSrThreads) {
        const unsigned n = qe[i];
        if (n) atomicAdd(&gq[i], n);
      }
      for (int i = threadIdx.x; i < p.n_bins * p.d_levels; i += kSrThreads) {
        const int dv = dtab[i];
        if (dv) {
          const int j = i / p.n_bins, b = i - j * p.n_bins;
          const int f = c.fs + j;
          if (f < p.n_levels)
            atomicAdd(&c.u_hist[static_cast<size_t>(f) * p.n_bins + b], static_cast<unsigned>(dv));
        }
      }
      if (static_cast<int>(threadIdx.x) >= c.fs && static_cast<int>(threadIdx.x) < p.n_levels) {
        // zero at fine level f: the elements that round to zero at more than f - fs fine levels
        unsigned long long n = 0;
        for (int k = static_cast<int>(threadIdx.x) - c.fs + 1; k <= p.n_levels - c.fs; ++k) n += s_zfine[k];
        if (n) atomicAdd(&p.zeros[static_cast<size_t>(l) * p.n_levels + threadIdx.x], n);
      }
    }
    __syncthreads();
    ++li;
    while (li < p.n_layers && p.layers[li + 1].tile_begin <= t) ++li;
  }
}

// Expansion of the stochastic-rounding tables: one CTA per (level, layer); level n_levels is the
// float histogram Q.  Fine levels and Q: interior cells put their count into their bin, the
// edge-cell elements' float bins are added (their differences already sit in U), exact zeros go
// to the bin of 0.  Coarse levels: every rounded value r of the level's table goes to the bin
// of r 2^-f, the entry r = 0 (plus the exact zeros) is the level's zero count.
struct SrExpandParams {
  const LayerDesc* layers;
  const LayerState* state;
  const LayerPlan* plan;
  const unsigned* cell_count;
  const unsigned* coarse_count;
  const unsigned* qe_hist;
  const unsigned long long* cell_total;
  unsigned* q_hist;
  unsigned* u_hist;
  unsigned long long* zeros;
  int n_bins, n_levels, cell_stride;
};

constexpr int kSrExpandThreads = 512;

__global__ void __launch_bounds__(kSrExpandThreads) expand_sr_kernel(const SrExpandParams p) {
  grid_dependency_wait();
  extern __shared__ unsigned s_hist[];          // [n_bins]
  __shared__ SrLevels s_lv;
  __shared__ unsigned long long s_zero;
  const LayerDesc L = p.layers[blockIdx.y];
  const int l = L.index;
  const LayerPlan P = p.plan[l];
  if (!P.keyed) return;
  const LayerState S = p.state[l];
  const int B = p.n_bins;
  const int f = blockIdx.x;                     // level, or n_levels for the float histogram
  const bool is_q = (f == p.n_levels);
  if (threadIdx.x == 0) { sr_levels(P, S, p.n_levels, &s_lv); s_zero = 0; }
  for (int b = threadIdx.x; b < B; b += kSrExpandThreads) s_hist[b] = 0;
  __syncthreads();
  const bool fine = is_q || f >= s_lv.fs;
  unsigned long long zero = 0;
  if (fine) {
    const unsigned* count = p.cell_count + static_cast<size_t>(l) * p.cell_stride;
    const SegPlan& sp = P.seg[0];
    for (int i = threadIdx.x; i < sp.cells; i += kSrExpandThreads) {
      const unsigned m = count[i];
      if (m == 0) continue;
      float lf, rf;
      cell_ends(sp.c0 + i, sp.g, true, &lf, &rf);
      const int bl = bin_of(lf, S.lo, S.scale, S.bmax);
      if (bl == bin_of(rf, S.lo, S.scale, S.bmax) && ADAPT_IN_BOUNDS(bl, B, 57)) atomicAdd(&s_hist[bl], m);
    }
  } else {
    const unsigned* tab = p.coarse_count + static_cast<size_t>(l) * p.cell_stride + s_lv.offset[f];
    const int rmin = s_lv.offset[f] - s_lv.bias[f];
    const float inv = pow2f(-f);
    for (int i = threadIdx.x; i < s_lv.size[f]; i += kSrExpandThreads) {
      const unsigned m = tab[i];
      if (m == 0) continue;
      const int r = rmin + i;
      const int b = bin_of(__fmul_rn(__int2float_rn(r), inv), S.lo, S.scale, S.bmax);
      if (ADAPT_IN_BOUNDS(b, B, 58)) atomicAdd(&s_hist[b], m);
      if (r == 0) zero += m;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) zero += __shfl_xor_sync(0xffffffffu, zero, o);
  if ((threadIdx.x & 31) == 0 && zero) atomicAdd(&s_zero, zero);
  __syncthreads();
  const unsigned n_zero = static_cast<unsigned>(static_cast<unsigned long long>(L.n) - p.cell_total[l]);
  const int bz = bin_of(0.0f, S.lo, S.scale, S.bmax);
  const unsigned* qe = p.qe_hist + static_cast<size_t>(l) * 2 * B;
  unsigned* out = is_q ? p.q_hist + static_cast<size_t>(l) * B
                       : p.u_hist + (static_cast<size_t>(l) * p.n_levels + f) * B;
  for (int b = threadIdx.x; b < B; b += kSrExpandThreads) {
    unsigned h = s_hist[b] + (b == bz ? n_zero : 0u);
    if (fine) h += qe[b];
    if (h) atomicAdd(&out[b], h);     // U holds the differences, Q starts at zero
  }
  if (!is_q && threadIdx.x == 0) {
    const unsigned long long z = s_zero + n_zero;     // fine levels: the counting kernel added the rest
    if (z) atomicAdd(&p.zeros[static_cast<size_t>(l) * p.n_levels + f], z);
  }
}

}  // namespace adapt
