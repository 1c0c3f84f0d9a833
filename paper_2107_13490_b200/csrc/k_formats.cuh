// The precision-switch search over other number formats: block floating point (Sec. 2.1
// "Block-Floating-Point Quantization"; the layer scale of Sec. 2.2) and floating point <E,M>
// (Sec. 7 names it as the planned extension), next to fixed point, through the same steps:
// Quantize -> zero count -> histogram over the layer's shared bins -> KL(P||Q) -> choice.
//
// Every format rounds an element on a power-of-two grid and then clamps it to the format's
// range.  The grid is the same for all elements (fixed point: 2^-FL; block floating point:
// 2^-s with the scale s of the layer) or follows the element's own binade (floating point:
// 2^(e-M), e >= emin).  Clamping commutes with the monotone bin function, so the kernels build
// one UNCLAMPED histogram per distinct rounding rule and the divergence kernel folds the two
// tails into the bins of the clamp values; formats that share a rule share a histogram.
#pragma once

#include "common.cuh"
#include "k_kld_select.cuh"
#include "k_range.cuh"

namespace adapt {

constexpr int kFmtFixed = 0, kFmtBfp = 1, kFmtFloat = 2;
constexpr int kRuleIdentity = 3;     // the float tensor itself (histogram Q)
constexpr int kBfpScaleLimit = 100;  // |s| <= 100: 2^s and 2^-s stay normal floats
constexpr int kFormatThreads = 1024;   // one or two CTAs per SM own its shared memory
constexpr int kMaxRulesPerGroup = 64;

struct FormatCand { int kind, a, b, rule; };   // rule: index of the candidate's rounding rule
struct FormatRule { int kind, p0, p1, pad; };  // fixed: p0 = FL; bfp: p0 = WL; float: p0 = E, p1 = M

struct FormatParams {
  const LayerDesc* layers;
  const LayerState* state;
  const FormatCand* cands;      // [n_cand]
  const FormatRule* rules;      // [n_rules]; rule 0 is the identity
  int n_layers, n_cand, n_rules, n_bins;
  int rules_per_group;          // rules handled by one blockIdx.y
  long long n_tiles;
  int* level;                   // [n_layers][n_rules] grid level of fixed / bfp rules, per layer
  float2* clamp;                // [n_layers][n_cand] lowest and highest representable value
  int* b_used;                  // [n_layers][n_cand] b as used (bfp: the layer's scale)
  unsigned* hist;               // [n_layers][n_rules][n_bins]
  unsigned long long* zeros;    // [n_layers][n_rules]
  unsigned long long seed;
  double alpha, inv_ln_base, eps;
  double* kld_out;              // [n_layers][n_cand]
  long long* zeros_out;         // [n_layers][n_cand]
  int* b_out;                   // optional [n_layers][n_cand]
  int* best_out;                // [n_layers][4]
  unsigned* hist_out;           // optional [n_layers][n_cand + 1][n_bins]; slot 0 = float tensor
  int* status_out;              // optional [n_layers]: 0, or the status code of the layer's data error
};

// x * 2^k for -149 <= k <= 149 in two exact steps (a single 2^k may not be a normal float).
__device__ __forceinline__ float scale_pow2(float x, int k) {
  const int k1 = max(-100, min(100, k));
  return __fmul_rn(__fmul_rn(x, pow2f(k1)), pow2f(k - k1));
}

// Largest finite value of <E,M>: (2 - 2^-M) * 2^emax, emax = 2^(E-1) - 1.
__device__ __forceinline__ float float_format_top(int e_bits, int m_bits) {
  const int emax = (1 << (e_bits - 1)) - 1;
  return __fmul_rn(__fsub_rn(2.0f, pow2f(-m_bits)), pow2f(emax));
}

// Scale of a block with extremes lo <= hi (Sec. 2.2): the largest s with
// hi * 2^s <= UB + 0.5 and -lo * 2^s <= -LB + 0.5; products of a float and a power of two are
// exact in double.  An extreme of the wrong sign sets no limit; no limit at all gives 0.
__device__ inline int bfp_scale(float lo, float hi, int wl) {
  const double ub = ldexp(1.0, wl - 1) - 0.5;
  const double lb = ldexp(1.0, wl - 1) + 0.5;
  const bool lim_hi = hi > 0.0f, lim_lo = lo < 0.0f;
  if (!lim_hi && !lim_lo) return 0;
  for (int s = kBfpScaleLimit; s > -kBfpScaleLimit; --s) {
    const bool ok_hi = !lim_hi || ldexp(static_cast<double>(hi), s) <= ub;
    const bool ok_lo = !lim_lo || ldexp(-static_cast<double>(lo), s) <= lb;
    if (ok_hi && ok_lo) return s;
  }
  return -kBfpScaleLimit;
}

// Rounds y to an integer: RNE, or SR(x) of Sec. 3.2 with P = pr.
template <bool kStochastic>
__device__ __forceinline__ float round_to_grid(float y, float pr) {
  if (!kStochastic) return rintf(y);
  const float f = floorf(y);
  const float frac = __fsub_rn(y, f);
  return (pr < frac) ? __fadd_rn(f, 1.0f) : f;
}

// Unclamped value of x on the grid 2^-level.
template <bool kStochastic>
__device__ __forceinline__ float level_value(float x, float two_l, float inv_l, float pr) {
  return __fmul_rn(round_to_grid<kStochastic>(__fmul_rn(x, two_l), pr), inv_l);
}

// Unclamped value of x in <E,M>: M fraction bits of its own binade, of binade emin below it.
template <bool kStochastic>
__device__ __forceinline__ float float_value(float x, int emin, int m_bits, float pr) {
  const int e = static_cast<int>((__float_as_uint(x) >> 23) & 0xffu) - 127;  // subnormal: -127
  const int k = m_bits - max(e, emin);
  const float y = scale_pow2(x, k);                   // |y| < 2^(M+1): exact
  return scale_pow2(round_to_grid<kStochastic>(y, pr), -k);
}

// One CTA per layer: grid level of every rule, clamp values and b-as-used of every candidate.
__global__ void format_resolve_kernel(const FormatParams p) {
  grid_dependency_wait();
  const int l = blockIdx.x;
  const LayerState S = p.state[l];
  for (int r = threadIdx.x; r < p.n_rules; r += blockDim.x) {
    const FormatRule R = p.rules[r];
    int lev = 0;
    if (R.kind == kFmtFixed) lev = R.p0;
    else if (R.kind == kFmtBfp) lev = bfp_scale(S.lo, S.hi, R.p0);
    p.level[static_cast<size_t>(l) * p.n_rules + r] = lev;
  }
  __syncthreads();
  for (int c = threadIdx.x; c < p.n_cand; c += blockDim.x) {
    const FormatCand K = p.cands[c];
    const size_t at = static_cast<size_t>(l) * p.n_cand + c;
    float2 cl;
    int b = K.b;
    if (K.kind == kFmtFloat) {
      const float top = float_format_top(K.a, K.b);
      cl = make_float2(-top, top);
    } else {
      const int lev = p.level[static_cast<size_t>(l) * p.n_rules + K.rule];
      b = lev;
      const float inv = pow2f(-lev);
      const int hi_code = static_cast<int>((1ll << (K.a - 1)) - 1);
      const int lo_code = static_cast<int>(-(1ll << (K.a - 1)));
      cl = make_float2(__fmul_rn(__int2float_rn(lo_code), inv), __fmul_rn(__int2float_rn(hi_code), inv));
    }
    p.clamp[at] = cl;
    p.b_used[at] = b;
    if (p.b_out) p.b_out[at] = b;
  }
}

// Exponent classes for the zero counts under round-to-nearest-even: an element rounds to zero
// exactly when |x| <= 2^t, t = -(level + 1) for a grid rule, emin - M - 1 for a float rule, and
// that only depends on floor(log2 |x|) and on whether |x| is a power of two.  Class 0 holds the
// exact zeros, class e + 150 the elements with floor(log2 |x|) = e (-149 <= e <= 127).
constexpr int kExpClasses = 288;

// The bin function without a float-to-int conversion: floor(clamp(u, 0, top)), top the largest
// float below n_bins, equals clamp(floor(u), 0, n_bins - 1) for every u (a NaN clamps to 0 as
// fmaxf returns its other operand), and adding 1.5 * 2^23 with round-down leaves that floor in
// the low mantissa bits.  Returned: the byte offset 4 * bin + 4 * 0x4B400000 (mod 2^32), which
// the caller adds to a histogram base that has the constant subtracted.
__device__ __forceinline__ unsigned format_bin_offset(float v, float lo, float scale, float top) {
  const float u = __fmul_rn(__fsub_rn(v, lo), scale);
  const float c = fminf(fmaxf(u, 0.0f), top);
  return __float_as_uint(__fadd_rd(c, 12582912.0f)) * 4u;
}

__device__ __forceinline__ void format_shared_inc(unsigned byte_addr) {
  asm volatile("red.shared.add.u32 [%0], 1;" :: "r"(byte_addr) : "memory");
}

// Float rule with the scaling by 2^k as single multiplications when 2^k and 2^-k are normal.
template <bool kStochastic>
__device__ __forceinline__ float float_value_fast(float x, int emin, int m_bits, float pr) {
  const int e = static_cast<int>((__float_as_uint(x) >> 23) & 0xffu) - 127;
  const int k = m_bits - max(e, emin);
  if (k > 126) return float_value<kStochastic>(x, emin, m_bits, pr);   // only |x| < 2^(M-126)
  return __fmul_rn(round_to_grid<kStochastic>(__fmul_rn(x, pow2f(k)), pr), pow2f(-k));
}

// Four elements of one thread through every rule of the group.  kMasked: some of the four lie
// outside the layer (mask m).
template <bool kStochastic, bool kMasked>
__device__ __forceinline__ void format_quad(const float (&v)[4], unsigned m, long long index0,
                                            unsigned long long seed, int layer_id, float lo,
                                            float scale, float top, int nr, unsigned hist_base,
                                            unsigned hist_stride, const int* s_kind,
                                            const int* s_i0, const int* s_i1, const float* s_f0,
                                            const float* s_f1, unsigned* s_zero,
                                            unsigned (*s_cls)[kExpClasses]) {
  float pr[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    pr[k] = 0.0f;
    if (kStochastic) {
      const unsigned h = hash24(seed, static_cast<unsigned long long>(layer_id),
                                static_cast<unsigned long long>(index0 + k));
      pr[k] = __fmul_rn(__uint2float_rn(h), 5.9604644775390625e-8f);  // k * 2^-24, exact
    } else if (!kMasked || ((m >> k) & 1u)) {
      // exponent class of the element (zero counts of all rules come from these)
      const unsigned ax = __float_as_uint(v[k]) & 0x7fffffffu;
      int cls = 0;
      bool p2 = false;
      if (ax) {
        const unsigned eb = ax >> 23, mant = ax & 0x7fffffu;
        cls = eb ? static_cast<int>(eb) + 23 : 32 - __clz(mant);   // e + 150
        p2 = eb ? (mant == 0u) : ((mant & (mant - 1u)) == 0u);
      }
      if (ADAPT_IN_BOUNDS(cls, kExpClasses, 40)) {
        atomicAdd(&s_cls[0][cls], 1u);
        if (p2) atomicAdd(&s_cls[1][cls], 1u);
      }
    }
  }
  unsigned hb = hist_base;
  for (int r = 0; r < nr; ++r, hb += hist_stride) {
    const int kind = s_kind[r];
    if (kind == kRuleIdentity) {
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if ((!kMasked || ((m >> k) & 1u)) &&
            ADAPT_IN_BOUNDS(static_cast<int>(format_bin_offset(v[k], lo, scale, top) >> 2) - 0x0B400000, hist_stride >> 2, 41))
          format_shared_inc(hb + format_bin_offset(v[k], lo, scale, top));
      continue;
    }
    float xq[4];
    if (kind == kFmtFloat) {
      const int emin = s_i0[r], mb = s_i1[r];
#pragma unroll
      for (int k = 0; k < 4; ++k) xq[k] = float_value_fast<kStochastic>(v[k], emin, mb, pr[k]);
    } else {
      const float two_l = s_f0[r], inv_l = s_f1[r];
#pragma unroll
      for (int k = 0; k < 4; ++k) xq[k] = level_value<kStochastic>(v[k], two_l, inv_l, pr[k]);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if ((!kMasked || ((m >> k) & 1u)) &&
          ADAPT_IN_BOUNDS(static_cast<int>(format_bin_offset(xq[k], lo, scale, top) >> 2) - 0x0B400000, hist_stride >> 2, 42))
        format_shared_inc(hb + format_bin_offset(xq[k], lo, scale, top));
    if (kStochastic) {
      // zero count by a warp reduction (the stochastic threshold is per element)
      unsigned nz = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) nz += ((!kMasked || ((m >> k) & 1u)) && xq[k] == 0.0f) ? 1u : 0u;
      nz = __reduce_add_sync(0xffffffffu, nz);
      if ((threadIdx.x & 31) == 0 && nz) atomicAdd(&s_zero[r], nz);
    }
  }
}

// Builds the unclamped histogram and the zero count of every rule, every layer.  The rules are
// cut into groups of rules_per_group (blockIdx.y) so that a group's histograms fit in shared
// memory; each group reads the tensors once.  A thread holds four elements and walks the
// group's rules with them, so a rule's constants are fetched once per four evaluations.
template <bool kStochastic>
__global__ void __launch_bounds__(kFormatThreads) format_search_kernel(const FormatParams p) {
  grid_dependency_wait();
  extern __shared__ unsigned s_fhist[];   // [rules in the group][n_bins]
  __shared__ int s_kind[kMaxRulesPerGroup], s_i0[kMaxRulesPerGroup], s_i1[kMaxRulesPerGroup];
  __shared__ float s_f0[kMaxRulesPerGroup], s_f1[kMaxRulesPerGroup];
  __shared__ unsigned s_zero[kMaxRulesPerGroup];
  __shared__ unsigned s_cls[2][kExpClasses];   // [0] all elements, [1] powers of two

  const int B = p.n_bins;
  const int r0 = blockIdx.y * p.rules_per_group;
  const int nr = min(p.rules_per_group, p.n_rules - r0);

  const long long per = (p.n_tiles + gridDim.x - 1) / gridDim.x;
  long long t = per * blockIdx.x;
  const long long t_end = min(p.n_tiles, t + per);
  if (t >= t_end) return;

  for (int i = threadIdx.x; i < nr * B; i += blockDim.x) s_fhist[i] = 0;
  if (threadIdx.x < kMaxRulesPerGroup) s_zero[threadIdx.x] = 0;
  if (threadIdx.x < 2 * kExpClasses) (&s_cls[0][0])[threadIdx.x] = 0;
  // byte address of the first rule's bin 0, less the constant format_bin_offset carries
  const unsigned hist_base = static_cast<unsigned>(__cvta_generic_to_shared(s_fhist)) - 4u * 0x4B400000u;
  const unsigned hist_stride = 4u * static_cast<unsigned>(B);

  int l = layer_of_tile(p.layers, p.n_layers, t);
  while (t < t_end) {
    const LayerDesc L = p.layers[l];
    const int gl = L.index;
    const LayerState S = p.state[gl];
    const long long layer_tiles_end = min(t_end, p.layers[l + 1].tile_begin);
    const float* base = L.ptr - L.mis;
    const long long jbeg = L.mis, jend = L.mis + L.n;
    const bool layer_ok = !(S.flags & (kFlagNonfinite | kFlagRange));
    // largest float below the number of bins: floor of anything clamped to it is the last bin
    const float top = __uint_as_float(__float_as_uint(__fadd_rn(S.bmax, 1.0f)) - 1u);

    // this layer's form of the group's rules; s_i0 of a grid rule = its level
    if (threadIdx.x < nr) {
      const FormatRule R = p.rules[r0 + threadIdx.x];
      s_kind[threadIdx.x] = R.kind;
      if (R.kind == kFmtFloat) {
        s_i0[threadIdx.x] = 2 - (1 << (R.p0 - 1));   // emin = 1 - bias
        s_i1[threadIdx.x] = R.p1;
      } else if (R.kind != kRuleIdentity) {
        const int lev = p.level[static_cast<size_t>(gl) * p.n_rules + r0 + threadIdx.x];
        s_i0[threadIdx.x] = lev;
        s_f0[threadIdx.x] = pow2f(lev);
        s_f1[threadIdx.x] = pow2f(-lev);
      }
    }
    __syncthreads();

    for (; t < layer_tiles_end; ++t) {
      if (!layer_ok) continue;
      const long long j_tile = (t - L.tile_begin) * kTile;
      for (int q = 0; q < kTile / 4 / kFormatThreads; ++q) {
        const long long j0 = j_tile + 4ll * (q * kFormatThreads + threadIdx.x);
        float v[4];
        unsigned m = 0;
        if (j0 < jend) m = load_quad(base, j0, jbeg, jend, v);
        else { v[0] = v[1] = v[2] = v[3] = 0.0f; }
        // a warp's quads are all inside the layer except at its two ends
        if (__all_sync(0xffffffffu, m == 0xFu))
          format_quad<kStochastic, false>(v, m, j0 - jbeg, p.seed, L.layer_id, S.lo, S.scale, top, nr,
                                          hist_base, hist_stride, s_kind, s_i0, s_i1, s_f0, s_f1,
                                          s_zero, s_cls);
        else
          format_quad<kStochastic, true>(v, m, j0 - jbeg, p.seed, L.layer_id, S.lo, S.scale, top, nr,
                                         hist_base, hist_stride, s_kind, s_i0, s_i1, s_f0, s_f1,
                                         s_zero, s_cls);
      }
    }
    __syncthreads();
    if (layer_ok) {
      for (int i = threadIdx.x; i < nr * B; i += blockDim.x) {
        const unsigned c = s_fhist[i];
        if (c) {
          const int r = i / B, b = i - r * B;
          atomicAdd(&p.hist[(static_cast<size_t>(gl) * p.n_rules + r0 + r) * B + b], c);
          s_fhist[i] = 0;
        }
      }
      if (threadIdx.x < nr) {
        unsigned long long c = s_zero[threadIdx.x];
        if (!kStochastic && s_kind[threadIdx.x] != kRuleIdentity) {
          // |x| <= 2^t rounds to zero: everything below binade t, the value 2^t itself, zeros
          const int tz = (s_kind[threadIdx.x] == kFmtFloat)
                             ? s_i0[threadIdx.x] - s_i1[threadIdx.x] - 1 : -(s_i0[threadIdx.x] + 1);
          const int ct = tz + 150;           // class of binade t
          c = s_cls[0][0];
          for (int i = 1; i < kExpClasses; ++i)
            if (i < ct) c += s_cls[0][i];
          if (ct >= 1 && ct < kExpClasses) c += s_cls[1][ct];
        }
        if (c) atomicAdd(&p.zeros[static_cast<size_t>(gl) * p.n_rules + r0 + threadIdx.x], c);
        s_zero[threadIdx.x] = 0;
      }
    }
    __syncthreads();
    if (threadIdx.x < 2 * kExpClasses) (&s_cls[0][0])[threadIdx.x] = 0;
    ++l;
    while (l < p.n_layers && p.layers[l + 1].tile_begin <= t) ++l;
  }
}

// One CTA per (candidate, layer): the rule's histogram with both tails folded into the bins
// of the candidate's clamp values, then KL(P||Q) against the identity rule's histogram.
__global__ void __launch_bounds__(kKldThreads) format_kld_kernel(const FormatParams p) {
  grid_dependency_wait();
  __shared__ double s_buf[kKldThreads / 32];
  __shared__ int s_inf;
  const int c = blockIdx.x, l = blockIdx.y;
  const int B = p.n_bins;
  const LayerState S = p.state[l];
  const long long n = p.layers[l].n;
  const size_t out = static_cast<size_t>(l) * p.n_cand + c;
  if (S.flags & (kFlagNonfinite | kFlagRange)) {
    if (threadIdx.x == 0) {
      p.kld_out[out] = __longlong_as_double(0x7ff8000000000000ll);  // NaN: unspecified output
      p.zeros_out[out] = 0;
    }
    return;
  }
  const int rule = p.cands[c].rule;
  const unsigned* U = p.hist + (static_cast<size_t>(l) * p.n_rules + rule) * B;
  const unsigned* Q = p.hist + static_cast<size_t>(l) * p.n_rules * B;
  const float2 cl = p.clamp[out];
  const int bl = bin_of(cl.x, S.lo, S.scale, S.bmax);
  const int bh = bin_of(cl.y, S.lo, S.scale, S.bmax);
  const double n_eff = static_cast<double>(n) + p.alpha * B;

  double lo_mass = 0.0, hi_mass = 0.0;
  for (int b = threadIdx.x; b < B; b += kKldThreads) {
    const unsigned u = U[b];
    if (b <= bl) lo_mass += u;
    if (b >= bh) hi_mass += u;
  }
  lo_mass = block_sum(lo_mass, s_buf);
  hi_mass = block_sum(hi_mass, s_buf);
  if (threadIdx.x == 0) s_inf = 0;
  __syncthreads();
  double sum = 0.0;
  bool inf = false;
  unsigned* H = p.hist_out ? p.hist_out + (static_cast<size_t>(l) * (p.n_cand + 1) + c + 1) * B : nullptr;
  unsigned* H0 = (p.hist_out && c == 0) ? p.hist_out + static_cast<size_t>(l) * (p.n_cand + 1) * B : nullptr;
  for (int b = threadIdx.x; b < B; b += kKldThreads) {
    long long pc;
    if (bl == bh) pc = (b == bl) ? n : 0;
    else if (b < bl || b > bh) pc = 0;
    else if (b == bl) pc = static_cast<long long>(lo_mass);
    else if (b == bh) pc = static_cast<long long>(hi_mass);
    else pc = U[b];
    if (H) H[b] = static_cast<unsigned>(pc);
    if (H0) H0[b] = Q[b];
    sum += kld_term(pc, Q[b], p.alpha, &inf);
  }
  if (inf) s_inf = 1;
  sum = block_sum(sum, s_buf);
  if (threadIdx.x == 0) {
    double k;
    if (n_eff <= 0.0) k = 0.0;
    else if (s_inf) k = __longlong_as_double(0x7ff0000000000000ll);
    else { k = sum * p.inv_ln_base / n_eff; if (!(k > 0.0)) k = 0.0; }
    p.kld_out[out] = k;
    p.zeros_out[out] = static_cast<long long>(p.zeros[static_cast<size_t>(l) * p.n_rules + rule]);
  }
}

// One warp per layer: the first format of the caller's list with KLD <= eps, else the one of
// least divergence (first among ties; the last one if every divergence is +inf).
__global__ void format_select_kernel(const FormatParams p) {
  grid_dependency_wait();
  const int l = blockIdx.x, lane = threadIdx.x;
  const double* kld = p.kld_out + static_cast<size_t>(l) * p.n_cand;
  int first_ok = 0x7fffffff, min_pos = -1;
  double min_k = 0.0;
  for (int c = lane; c < p.n_cand; c += 32) {
    const double k = kld[c];
    if (k <= p.eps) first_ok = min(first_ok, c);
    if (k < __longlong_as_double(0x7ff0000000000000ll)) arg_min_merge(min_k, min_pos, k, c);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    first_ok = min(first_ok, __shfl_xor_sync(0xffffffffu, first_ok, o));
    const double k2 = __shfl_xor_sync(0xffffffffu, min_k, o);
    const int pos2 = __shfl_xor_sync(0xffffffffu, min_pos, o);
    arg_min_merge(min_k, min_pos, k2, pos2);
  }
  if (lane == 0) {
    unsigned flags = p.state[l].flags & (kFlagDegenerate | kFlagNonfinite | kFlagRange);
    if (p.status_out) p.status_out[l] = (flags & kFlagNonfinite) ? 2 : ((flags & kFlagRange) ? 3 : 0);
    int c;
    if (first_ok != 0x7fffffff) { c = first_ok; flags |= 1u; }
    else if (min_pos >= 0) c = min_pos;
    else c = p.n_cand - 1;
    int* o = p.best_out + 4 * l;
    o[0] = p.cands[c].a;
    o[1] = p.b_used[static_cast<size_t>(l) * p.n_cand + c];
    o[2] = c;
    o[3] = static_cast<int>(flags);
  }
}

// Quantize(L, format): the tensor mapped to the format's representable values (fp32 out).
struct FormatQuantParams {
  const float* x;
  float* out;
  long long n;
  int kind, a, b, layer_id;
  unsigned long long seed;
};

template <bool kStochastic>
__global__ void __launch_bounds__(256) format_quantize_kernel(const FormatQuantParams p) {
  float lo_v, hi_v, two_l = 1.0f, inv_l = 1.0f;
  int emin = 0;
  if (p.kind == kFmtFloat) {
    hi_v = float_format_top(p.a, p.b);
    lo_v = -hi_v;
    emin = 2 - (1 << (p.a - 1));
  } else {
    two_l = pow2f(p.b);
    inv_l = pow2f(-p.b);
    hi_v = __fmul_rn(__int2float_rn(static_cast<int>((1ll << (p.a - 1)) - 1)), inv_l);
    lo_v = __fmul_rn(__int2float_rn(static_cast<int>(-(1ll << (p.a - 1)))), inv_l);
  }
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < p.n; i += stride) {
    const float x = __ldg(p.x + i);
    float pr = 0.0f;
    if (kStochastic)
      pr = __fmul_rn(__uint2float_rn(hash24(p.seed, static_cast<unsigned long long>(p.layer_id),
                                            static_cast<unsigned long long>(i))),
                     5.9604644775390625e-8f);
    float v = (p.kind == kFmtFloat) ? float_value<kStochastic>(x, emin, p.b, pr)
                                    : level_value<kStochastic>(x, two_l, inv_l, pr);
    v = fminf(fmaxf(v, lo_v), hi_v);
    p.out[i] = __fadd_rn(v, 0.0f);   // -0 becomes +0, as a code of zero would
  }
}

}  // namespace adapt
