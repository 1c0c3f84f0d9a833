// K2 (direct form): fused multi-candidate quantize + zero count + privatised
// shared-memory histograms, every fraction length evaluated explicitly.
//
// For one FL the rounded value round(x * 2^FL) is the same for every WL of the
// grid - WL only clamps - and the bin function is monotone, so a candidate's
// histogram is the unsaturated per-FL histogram with both tails folded into
// the bins of the two saturation values.  This kernel therefore builds, per
// layer, one unsaturated histogram U[FL] and one zero count Z[FL] for each
// FL from 0 to the grid's largest, plus the float histogram Q; the fold happens
// in the divergence kernel.  (Quantize / EDF steps of Algorithm 3; Sec. 3.2, 3.3.)
//
// Handles both rounding modes; it serves stochastic rounding, small layers and
// very large bin counts, the keyed kernel the rest.  When (FLs + 1) * n_bins counters do
// not fit in shared memory the FL list is cut into groups (blockIdx.y), each
// group re-reading the tensor.
#pragma once

#include "common.cuh"
#include "k_plan.cuh"
#include "k_range.cuh"

namespace adapt {

constexpr int kSearchThreads = 256;       // threads per CTA when several CTAs share an SM
constexpr int kSearchThreadsWide = 1024;  // one CTA per SM owning all of its shared memory

struct SearchParams {
  const LayerDesc* layers;
  const LayerState* state;
  int n_layers;
  int n_fl;                    // fraction lengths 0..n_fl-1 are evaluated
  int fl_per_group;            // FLs handled by one blockIdx.y
  int n_bins;
  long long n_tiles;
  unsigned* q_hist;            // [n_layers][n_bins]
  unsigned* u_hist;            // [n_layers][n_fl][n_bins]
  unsigned long long* zeros;   // [n_layers][n_fl]
  unsigned long long seed;
  const LayerPlan* plan;       // by LayerDesc::index; read only for layers with via_plan set
};

// Bin index by one convert-with-floor and two integer clamps; equal to bin_of for every input
// (a NaN converts to 0, out-of-range values saturate and are clamped).
__device__ __forceinline__ int bin_index_fast(float v, float lo, float scale, int bmax) {
  const int b = __float2int_rd(__fmul_rn(__fsub_rn(v, lo), scale));
  return min(max(b, 0), bmax);
}

// Under round-to-nearest-even an element rounds to zero at fraction length f exactly when
// |x| <= 2^-(f+1).  kz = the largest such f (capped to -1..32), from the exponent field alone.
__device__ __forceinline__ int highest_zero_level(float x) {
  const unsigned ax = __float_as_uint(x) & 0x7FFFFFFFu;
  if (ax == 0u) return 32;
  const int kz = 125 - static_cast<int>((ax - 1u) >> 23);
  return max(-1, min(kz, 32));
}

// The bin function without a float-to-int conversion: floor(clamp(u, 0, top)), top the largest
// float below n_bins, equals clamp(floor(u), 0, n_bins - 1) for every u (a NaN clamps to 0 as
// fmaxf returns its other operand), and adding 1.5 * 2^23 with round-down leaves that floor in
// the low mantissa bits.  Returned: the byte offset 4 * bin + 4 * 0x4B400000 (mod 2^32), which
// the caller adds to a histogram base that has the constant subtracted.
__device__ __forceinline__ unsigned bin_offset_magic(float v, float lo, float scale, float top) {
  const float u = __fmul_rn(__fsub_rn(v, lo), scale);
  const float c = fminf(fmaxf(u, 0.0f), top);
  return __float_as_uint(__fadd_rd(c, 12582912.0f)) * 4u;
}

__device__ __forceinline__ void shared_inc(unsigned byte_addr) {
  asm volatile("red.shared.add.u32 [%0], 1;" :: "r"(byte_addr) : "memory");
}

// Four elements of one thread through the float histogram, the zero bookkeeping and every
// fraction length of the group.  kMasked: some of the four lie outside the layer (mask m).
template <bool kStochastic, bool kMasked>
__device__ __forceinline__ void direct_quad(const float (&v)[4], unsigned m, long long index0,
                                            const SearchParams& p, int layer_id, float lo,
                                            float scale, float top, int nf, bool do_q,
                                            unsigned hist_base, unsigned hist_stride,
                                            const float* s_two, const float* s_inv,
                                            unsigned* s_zero, unsigned* s_zlevel) {
  float pr[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const bool valid = !kMasked || ((m >> k) & 1u);
    pr[k] = 0.0f;
    if (valid && do_q) {
      const unsigned off = bin_offset_magic(v[k], lo, scale, top);
      if (ADAPT_IN_BOUNDS(static_cast<int>(off >> 2) - 0x0B400000, hist_stride >> 2, 20)) shared_inc(hist_base + off);
    }
    if (kStochastic) {
      const unsigned h = hash24(p.seed, static_cast<unsigned long long>(layer_id),
                                static_cast<unsigned long long>(index0 + k));
      pr[k] = __fmul_rn(__uint2float_rn(h), 5.9604644775390625e-8f);  // k * 2^-24, exact
    } else if (valid) {
      if (ADAPT_IN_BOUNDS(highest_zero_level(v[k]) + 1, kMaxFl + 2, 21))
        atomicAdd(&s_zlevel[highest_zero_level(v[k]) + 1], 1u);
    }
  }
  // the thread walks the fraction lengths with its four elements in registers
  unsigned hb = hist_base + hist_stride;
  for (int f = 0; f < nf; ++f, hb += hist_stride) {
    const float two_f = s_two[f], inv_f = s_inv[f];
    unsigned nz = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float r = round_scaled<kStochastic>(v[k], two_f, pr[k]);
      const unsigned off = bin_offset_magic(__fmul_rn(r, inv_f), lo, scale, top);
      if ((!kMasked || ((m >> k) & 1u)) && ADAPT_IN_BOUNDS(static_cast<int>(off >> 2) - 0x0B400000, hist_stride >> 2, 22)) {
        shared_inc(hb + off);
        if (kStochastic) nz += (r == 0.0f) ? 1u : 0u;
      }
    }
    if (kStochastic) {
      nz = __reduce_add_sync(0xffffffffu, nz);
      if ((threadIdx.x & 31) == 0 && nz) atomicAdd(&s_zero[f], nz);
    }
  }
}

template <bool kStochastic>
__global__ void __launch_bounds__(kSearchThreadsWide)
search_direct_kernel(const SearchParams p) {
  grid_dependency_wait();
  extern __shared__ unsigned s_hist[];  // [(fl_per_group + 1)][n_bins]
  __shared__ float s_two[kMaxFl], s_inv[kMaxFl];
  __shared__ unsigned s_zero[kMaxFl];
  __shared__ unsigned s_zlevel[kMaxFl + 2];   // RNE: elements by highest zero level (-1..32)

  const int B = p.n_bins;
  const int f0 = blockIdx.y * p.fl_per_group;
  const int nf = min(p.fl_per_group, p.n_fl - f0);
  const bool do_q = (blockIdx.y == 0);

  const long long per = (p.n_tiles + gridDim.x - 1) / gridDim.x;
  long long t = per * blockIdx.x;
  const long long t_end = min(p.n_tiles, t + per);
  if (t >= t_end) return;

  for (int i = threadIdx.x; i < (nf + 1) * B; i += blockDim.x) s_hist[i] = 0;
  if (threadIdx.x < kMaxFl) {
    s_zero[threadIdx.x] = 0;
    if (threadIdx.x < nf) {
      int fl = f0 + threadIdx.x;
      s_two[threadIdx.x] = pow2f(fl);
      s_inv[threadIdx.x] = pow2f(-fl);
    }
  }
  if (threadIdx.x < kMaxFl + 2) s_zlevel[threadIdx.x] = 0;
  __syncthreads();
  // byte address of the float histogram's bin 0, less the constant bin_offset_magic carries
  const unsigned hist_base = static_cast<unsigned>(__cvta_generic_to_shared(s_hist)) - 4u * 0x4B400000u;
  const unsigned hist_stride = 4u * static_cast<unsigned>(B);

  int l = layer_of_tile(p.layers, p.n_layers, t);
  while (t < t_end) {
    const LayerDesc L = p.layers[l];
    const int gl = L.index;
    const LayerState S = p.state[gl];
    const long long layer_tiles_end = min(t_end, p.layers[l + 1].tile_begin);
    const float* base = L.ptr - L.mis;
    const long long jbeg = L.mis, jend = L.mis + L.n;
    // (a layer that the stochastic-rounding kernel serves is skipped here)
    const bool layer_ok = !(S.flags & (kFlagNonfinite | kFlagRange)) &&
                          !(L.via_plan && p.plan[gl].keyed);
    // largest float below the number of bins: floor of anything clamped to it is the last bin
    const float top = __uint_as_float(__float_as_uint(__fadd_rn(S.bmax, 1.0f)) - 1u);

    for (; t < layer_tiles_end; ++t) {
      if (!layer_ok) continue;
      const long long j_tile = (t - L.tile_begin) * kTile;
      for (int q = 0; q < kTile / 4 / static_cast<int>(blockDim.x); ++q) {
        const long long j0 = j_tile + 4ll * (q * static_cast<int>(blockDim.x) + threadIdx.x);
        float v[4];
        unsigned m = 0;
        if (j0 < jend) m = load_quad(base, j0, jbeg, jend, v);
        else { v[0] = v[1] = v[2] = v[3] = 0.0f; }
        // a warp's quads are all inside the layer except at its two ends
        if (__all_sync(0xffffffffu, m == 0xFu))
          direct_quad<kStochastic, false>(v, m, j0 - jbeg, p, L.layer_id, S.lo, S.scale, top, nf,
                                          do_q, hist_base, hist_stride, s_two, s_inv, s_zero, s_zlevel);
        else
          direct_quad<kStochastic, true>(v, m, j0 - jbeg, p, L.layer_id, S.lo, S.scale, top, nf,
                                         do_q, hist_base, hist_stride, s_two, s_inv, s_zero, s_zlevel);
      }
    }
    __syncthreads();
    // flush this layer's private counts and clear them for the next layer
    if (layer_ok) {
      for (int i = threadIdx.x; i < (nf + 1) * B; i += blockDim.x) {
        unsigned c = s_hist[i];
        if (c) {
          int slot = i / B, b = i - slot * B;
          if (slot == 0) {
            if (do_q) atomicAdd(&p.q_hist[static_cast<size_t>(gl) * B + b], c);
          } else {
            atomicAdd(&p.u_hist[(static_cast<size_t>(gl) * p.n_fl + f0 + slot - 1) * B + b], c);
          }
          s_hist[i] = 0;
        }
      }
      if (threadIdx.x < nf) {
        unsigned long long c = s_zero[threadIdx.x];
        if (!kStochastic) {
          // zero at fraction length f: every element whose highest zero level is >= f
          const int f = f0 + threadIdx.x;
          c = 0;
          for (int kz = f; kz <= 32; ++kz) c += s_zlevel[kz + 1];
        }
        if (c) atomicAdd(&p.zeros[static_cast<size_t>(gl) * p.n_fl + f0 + threadIdx.x], c);
        s_zero[threadIdx.x] = 0;
      }
    }
    __syncthreads();
    if (threadIdx.x < kMaxFl + 2) s_zlevel[threadIdx.x] = 0;
    __syncthreads();             // the next layer's first atomics must find the cleared classes
    ++l;
    while (l < p.n_layers && p.layers[l + 1].tile_begin <= t) ++l;
  }
}

}  // namespace adapt
