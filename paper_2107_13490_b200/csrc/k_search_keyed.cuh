// K2 (keyed form, round-to-nearest-even): fused multi-candidate quantize +
// zero count + histograms with ONE shared-memory atomic per element on the
// common path.  See k_plan.cuh for the cell decomposition this relies on.
//
// Per element x != 0:   c = floor(x * 2^G) - c0;  old = atomicAdd(cell[c], 1)
// The returned word carries the cell's marks in its two top bits:
//   bit 30 (cell -1 / 0): add the element to the class counter "highest level
//          at which it still rounds to zero";
//   bit 31 (edge cell), or x exactly on the level-G grid: the element is pushed
//          to a per-warp queue; queues are drained 32 entries at a time by the
//          whole warp (dense lanes):
//            edge entry: b0 = bin(x) into the edge-element histogram Qe, then
//              only the fine levels f whose half quantum can reach one of the
//              bin's edges are evaluated; a level is recorded only if its bin
//              differs from b0 (-1 at b0, +1 at the new bin);
//            on-grid entry: the one coarse level at which x is a rounding tie
//              that goes down is corrected (the cell table assumes "up").
// Exact zeros are only counted (warp ballot).  Everything else about the
// element - the float histogram, all coarse levels, all fine levels of
// interior cells - is derived from the cell counts by the expand kernels.
#pragma once

#include "common.cuh"
#include "k_plan.cuh"
#include "k_range.cuh"

namespace adapt {

constexpr int kKeyedThreads = 512;
constexpr int kKeyedWarps = kKeyedThreads / 32;
constexpr int kQueueCap = 64;       // per-warp queue entries (drained at >= 32)
constexpr int kZeroClasses = 34;    // class k+1, k = highest zero level in -1..31 (32 = all)

struct KeyedParams {
  const LayerDesc* layers;     // keyed layer list (+ sentinel)
  int n_layers;
  long long n_tiles;
  const LayerState* state;     // by LayerDesc::index
  const LayerPlan* plan;       // by LayerDesc::index
  const float* edges;          // [layer][n_bins + 1]
  const unsigned* cell_init;   // [layer][cell_cap]
  unsigned* cell_count;        // [layer][cell_cap]      global cell counts
  unsigned* qe_hist;           // [layer][n_bins]        float histogram of queue "edge" elements
  unsigned* u_hist;            // [layer][n_levels][n_bins]  receives the per-level corrections
  unsigned long long* zeros;   // [layer][n_levels]      receives tie corrections
  unsigned long long* zero_class;  // [layer][kZeroClasses]
  unsigned long long* n_zero;  // [layer]                exact zeros
  int n_bins;
  int n_levels;                // levels 0..n_levels-1 are wanted
  int cell_cap;
  int d_levels;                // fine levels whose corrections are kept in shared memory
};

// shared memory carve-up (dynamic): cells | qe | d | queue_x | queue_tag
struct KeyedSmem {
  unsigned* cells;   // [cell_cap]
  unsigned* qe;      // [n_bins]
  int* d;            // [d_levels][n_bins]
  float* qx;         // [warps][kQueueCap]
  unsigned* qtag;    // [warps][kQueueCap]   bit 31 edge, bit 30 on-grid, low bits cell index
};

__host__ __device__ inline size_t keyed_smem_bytes(int cell_cap, int n_bins, int d_levels) {
  return sizeof(unsigned) * (static_cast<size_t>(cell_cap) + n_bins +
                             static_cast<size_t>(d_levels) * n_bins) +
         (sizeof(float) + sizeof(unsigned)) * kKeyedWarps * kQueueCap;
}

struct LayerCtx {
  LayerState S;
  LayerPlan P;
  const float* E;
  unsigned* u_hist;            // this layer's [n_levels][n_bins]
  unsigned long long* zeros;   // this layer's [n_levels]
  int n_bins, n_levels, d_levels;
};

// Processes one queue entry (all 32 lanes call this; `live` masks real entries).
__device__ __forceinline__ void drain_entry(const LayerCtx& c, const KeyedSmem& sm, bool live,
                                            float x, unsigned tag) {
  const int B = c.n_bins;
  // ---- on-grid entry: fix the single coarse tie level ----------------------
  if (live && (tag & 0x40000000u)) {
    const long long cc = c.P.c0 + static_cast<long long>(tag & 0x3FFFFFFFu);
    if (cc != 0) {
      const int tz = __ffsll(cc) - 1;          // lowest set bit
      const int ft = c.P.g - 1 - tz;           // the level at which x is a tie
      if (ft >= 0 && ft < c.n_levels) {
        const long long a = cc >> (tz + 1);    // floor(x * 2^ft)
        if ((a & 1ll) == 0) {                  // tie goes down to a; the table counted a + 1
          const float s = pow2f(-ft);
          const int b_up = bin_of(__fmul_rn(__ll2float_rn(a + 1), s), c.S.lo, c.S.scale, c.S.bmax);
          const int b_dn = bin_of(__fmul_rn(__ll2float_rn(a), s), c.S.lo, c.S.scale, c.S.bmax);
          unsigned* U = c.u_hist + static_cast<size_t>(ft) * B;
          if (b_up != b_dn) { atomicAdd(&U[b_up], 0xFFFFFFFFu); atomicAdd(&U[b_dn], 1u); }
          if (a + 1 == 0) atomicAdd(&c.zeros[ft], 0xFFFFFFFFFFFFFFFFull);
          if (a == 0) atomicAdd(&c.zeros[ft], 1ull);
        }
      }
    }
  }
  // ---- edge entry: float bin, then the fine levels that can still move ------
  const bool edge = live && (tag & 0x80000000u);
  int b0 = 0, f_end = 0;
  if (edge) {
    b0 = bin_of(x, c.S.lo, c.S.scale, c.S.bmax);
    atomicAdd(&sm.qe[b0], 1u);
    // distance to the bin's two edges, rounded down: safe once 2^-(f+1) < margin
    const float dl = __fsub_rd(x, __ldg(c.E + b0));
    const float dh = __fsub_rd(__ldg(c.E + b0 + 1), x);
    const float m = fminf(dl, dh);
    int f_safe = 32;
    if (m > 0.0f) f_safe = 126 - static_cast<int>((__float_as_uint(m) - 1u) >> 23);
    f_end = min(f_safe, c.n_levels);
  }
  for (int f = c.P.fs;; ++f) {
    const bool act = edge && f < f_end;
    if (!__any_sync(0xffffffffu, act)) break;
    if (act) {
      const float r = rintf(__fmul_rn(x, pow2f(f)));
      const int b = bin_of(__fmul_rn(r, pow2f(-f)), c.S.lo, c.S.scale, c.S.bmax);
      if (b != b0) {
        const int j = f - c.P.fs;
        if (j < c.d_levels) {
          atomicAdd(&sm.d[j * B + b], 1);
          atomicAdd(&sm.d[j * B + b0], -1);
        } else {
          unsigned* U = c.u_hist + static_cast<size_t>(f) * B;
          atomicAdd(&U[b], 1u);
          atomicAdd(&U[b0], 0xFFFFFFFFu);
        }
      }
    }
  }
}

__global__ void __launch_bounds__(kKeyedThreads, 2) search_keyed_kernel(const KeyedParams p) {
  extern __shared__ __align__(16) unsigned char s_raw[];
  __shared__ unsigned s_zclass[kZeroClasses];
  __shared__ unsigned s_nzero;

  KeyedSmem sm;
  sm.cells = reinterpret_cast<unsigned*>(s_raw);
  sm.qe = sm.cells + p.cell_cap;
  sm.d = reinterpret_cast<int*>(sm.qe + p.n_bins);
  sm.qx = reinterpret_cast<float*>(sm.d + static_cast<size_t>(p.d_levels) * p.n_bins);
  sm.qtag = reinterpret_cast<unsigned*>(sm.qx + kKeyedWarps * kQueueCap);

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned lt_mask = (1u << lane) - 1u;
  float* qx = sm.qx + warp * kQueueCap;
  unsigned* qtag = sm.qtag + warp * kQueueCap;

  const long long per = (p.n_tiles + gridDim.x - 1) / gridDim.x;
  long long t = per * blockIdx.x;
  const long long t_end = min(p.n_tiles, t + per);
  if (t >= t_end) return;
  int li = layer_of_tile(p.layers, p.n_layers, t);

  while (t < t_end) {
    const LayerDesc L = p.layers[li];
    const int l = L.index;
    LayerCtx c;
    c.S = p.state[l];
    c.P = p.plan[l];
    c.E = p.edges + static_cast<size_t>(l) * (p.n_bins + 1);
    c.u_hist = p.u_hist + static_cast<size_t>(l) * p.n_levels * p.n_bins;
    c.zeros = p.zeros + static_cast<size_t>(l) * p.n_levels;
    c.n_bins = p.n_bins; c.n_levels = p.n_levels; c.d_levels = p.d_levels;
    const long long layer_tiles_end = min(t_end, p.layers[li + 1].tile_begin);
    const float* base = L.ptr - L.mis;
    const long long jbeg = L.mis, jend = L.mis + L.n;
    const bool ok = c.P.keyed != 0;

    // ---- per-layer set-up of the private tables --------------------------------
    if (ok) {
      const unsigned* init = p.cell_init + static_cast<size_t>(l) * p.cell_cap;
      for (int i = threadIdx.x; i < c.P.cells; i += kKeyedThreads) sm.cells[i] = __ldg(init + i);
      for (int i = threadIdx.x; i < p.n_bins * (1 + p.d_levels); i += kKeyedThreads) sm.qe[i] = 0;
      if (threadIdx.x < kZeroClasses) s_zclass[threadIdx.x] = 0;
      if (threadIdx.x == 0) s_nzero = 0;
    }
    __syncthreads();
    int qn = 0;             // this warp's queue fill (uniform across the warp)
    unsigned n_zero = 0;    // exact zeros seen by this warp (lane 0's copy is used)

    for (; t < layer_tiles_end; ++t) {
      if (!ok) continue;
      const long long j_tile = (t - L.tile_begin) * kTile;
      float v[kTile / 4 / kKeyedThreads][4];
      unsigned vm[kTile / 4 / kKeyedThreads];
#pragma unroll
      for (int q = 0; q < kTile / 4 / kKeyedThreads; ++q) {
        const long long j0 = j_tile + 4ll * (q * kKeyedThreads + threadIdx.x);
        vm[q] = 0;
        v[q][0] = v[q][1] = v[q][2] = v[q][3] = 0.0f;
        if (j0 < jend) vm[q] = load_quad(base, j0, jbeg, jend, v[q]);
      }
#pragma unroll
      for (int q = 0; q < kTile / 4 / kKeyedThreads; ++q) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float x = v[q][k];
          const bool valid = (vm[q] >> k) & 1u;
          const bool nz = valid && (x != 0.0f);
          n_zero += __popc(__ballot_sync(0xffffffffu, valid && !nz));
          const float z = __fmul_rn(x, c.P.two_g);
          const float cf = floorf(z);
          const int idx = __float2int_rz(__fsub_rn(cf, c.P.c0f));
          unsigned old = 0;
          if (nz) old = atomicAdd(&sm.cells[idx], 1u);
          if (old & kCellNearZero) {
            // highest level at which x still rounds to zero: |x| <= 2^-(k+1)
            const unsigned ax = __float_as_uint(x) & 0x7FFFFFFFu;
            int kz = 125 - static_cast<int>((ax - 1u) >> 23);
            kz = max(-1, min(kz, 32));
            atomicAdd(&s_zclass[kz + 1], 1u);
          }
          const bool on_grid = nz && (z == cf);
          const bool push = nz && ((old & kCellEdge) || on_grid);
          const unsigned pm = __ballot_sync(0xffffffffu, push);
          if (pm) {
            if (push) {
              const int pos = qn + __popc(pm & lt_mask);
              qx[pos] = x;
              qtag[pos] = (old & kCellEdge) | (on_grid ? 0x40000000u : 0u) |
                          static_cast<unsigned>(idx);
            }
            qn += __popc(pm);
            __syncwarp();
            if (qn >= 32) {
              qn -= 32;
              drain_entry(c, sm, true, qx[qn + lane], qtag[qn + lane]);
              __syncwarp();
            }
          }
        }
      }
    }
    // ---- drain what is left in the queue ------------------------------------------
    if (ok) {
      __syncwarp();
      if (qn > 0) {
        const bool live = lane < qn;
        drain_entry(c, sm, live, live ? qx[lane] : 0.0f, live ? qtag[lane] : 0u);
      }
      if (lane == 0 && n_zero) atomicAdd(&s_nzero, n_zero);
    }
    __syncthreads();

    // ---- flush the private tables into the layer's global ones -----------------------
    if (ok) {
      unsigned* gc = p.cell_count + static_cast<size_t>(l) * p.cell_cap;
      for (int i = threadIdx.x; i < c.P.cells; i += kKeyedThreads) {
        const unsigned n = sm.cells[i] & kCellCountMask;
        if (n) atomicAdd(&gc[i], n);
      }
      unsigned* gq = p.qe_hist + static_cast<size_t>(l) * p.n_bins;
      for (int i = threadIdx.x; i < p.n_bins; i += kKeyedThreads) {
        const unsigned n = sm.qe[i];
        if (n) atomicAdd(&gq[i], n);
      }
      for (int i = threadIdx.x; i < p.n_bins * p.d_levels; i += kKeyedThreads) {
        const int dv = sm.d[i];
        if (dv) {
          const int j = i / p.n_bins, b = i - j * p.n_bins;
          const int f = c.P.fs + j;
          if (f < p.n_levels)
            atomicAdd(&c.u_hist[static_cast<size_t>(f) * p.n_bins + b], static_cast<unsigned>(dv));
        }
      }
      if (threadIdx.x < kZeroClasses) {
        const unsigned n = s_zclass[threadIdx.x];
        if (n) atomicAdd(&p.zero_class[static_cast<size_t>(l) * kZeroClasses + threadIdx.x],
                         static_cast<unsigned long long>(n));
      }
      if (threadIdx.x == 0 && s_nzero) atomicAdd(&p.n_zero[l], static_cast<unsigned long long>(s_nzero));
    }
    __syncthreads();
    ++li;
    while (li < p.n_layers && p.layers[li + 1].tile_begin <= t) ++li;
  }
}

}  // namespace adapt
