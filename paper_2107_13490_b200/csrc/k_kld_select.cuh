// K3: batched divergence and selection over all (layer, candidate) pairs, one launch.
//
// kld_kernel: one CTA per (fraction length, layer).  Folds the layer's unsaturated
// per-FL histogram into each candidate's histogram (both tails collapse into
// the bins of the two saturation values), then sums the discrete
// Kullback-Leibler divergence KL(P||Q) (Sec. 3.3), P = candidate, Q = float
// tensor, in double precision.  With integer counts p, q that share the total
// N, the term (p/N) log((p/N)/(q/N)) is evaluated as p * log1p((p - q)/q) / N:
// the difference is exact in integers, so histograms that differ by a few
// counts in well-filled bins do not lose their divergence to cancellation.
// The unsaturated divergence is summed by the whole CTA; the candidates that
// saturate inside the range are dealt to the CTA's warps, one warp each.
//
// The CTA that writes the last divergences of a layer (a ticket per layer, no
// waiting) selects the layer's format: the lowest <WL,FL> (WL first, then FL)
// with KLD <= eps, else the candidate of least divergence (Algorithm 3).
#pragma once

#include <math.h>

#include "common.cuh"
#include "k_range.cuh"

namespace adapt {

#ifndef ADAPT_KLD_THREADS
#define ADAPT_KLD_THREADS 256
#endif
#ifndef ADAPT_KLD_WARP_BINS
#define ADAPT_KLD_WARP_BINS 128
#endif
constexpr int kKldThreads = ADAPT_KLD_THREADS;

struct KldParams {
  const LayerDesc* layers;
  LayerState* state;           // read, and its kld_ticket counted up
  const int* cand_wl;          // [n_cand]
  const int* cand_fl;          // [n_cand]
  const int* cand_slot;        // [n_cand] index of the candidate's FL in the distinct-FL list
  const int* cand_order;       // [n_cand] candidate indices sorted by (WL, FL, index)
  const int* cand_by_fl;       // [n_cand] candidate indices grouped by FL
  const int* fl_begin;         // [n_fl + 1] start of each FL's group in cand_by_fl
  int n_layers, n_cand, n_fl, n_bins;
  const unsigned* q_hist;      // [n_layers][n_bins]
  const unsigned* u_hist;      // [n_layers][n_fl][n_bins]
  const unsigned long long* zeros;  // [n_layers][n_fl]
  double alpha;                // pseudo-count
  double inv_ln_base;          // 1 / ln(log base)
  double eps;
  double* kld_out;             // [n_layers][n_cand]
  long long* zeros_out;        // [n_layers][n_cand]
  int* best_out;               // [n_layers][4]
  unsigned* hist_out;          // optional [n_layers][n_cand + 1][n_bins]
  const int* start;            // optional [n_layers][2]: descent from this <WL,FL> per layer
  int* status_out;             // optional [n_layers]: 0, or the status code of the layer's data error
};

__device__ __forceinline__ double block_sum(double v, double* s_buf) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int w = threadIdx.x >> 5;
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_buf[w] = v;
  __syncthreads();
  double t = 0.0;
  for (int i = 0; i < kKldThreads / 32; ++i) t += s_buf[i];
  return t;
}

// One term of the divergence sum and whether it is infinite (a filled P bin over an empty Q bin).
__device__ __forceinline__ double kld_term(long long pc, long long qc, double alpha, bool* inf) {
  if (pc == qc) return 0.0;      // log1p(0) = 0 exactly: the term vanishes whatever the pseudo-count
  const double pa = static_cast<double>(pc) + alpha;
  const double qa = static_cast<double>(qc) + alpha;
  if (!(pa > 0.0)) return 0.0;
  if (qa <= 0.0) { *inf = true; return 0.0; }
  return pa * log1p(static_cast<double>(pc - qc) / qa);
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ unsigned long long warp_sum(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// One CTA per (fraction length, layer).  The candidates of one FL differ only in where they
// saturate; those whose two saturation values fall in the first and the last bin have exactly
// the unsaturated histogram U[FL], so their divergence is computed once.  The others fold the
// two tails of U[FL] into the bins of their saturation values and are summed one by one.
struct SelectScratch;
__device__ void select_layer(const KldParams& p, int l, SelectScratch* sh);

__global__ void __launch_bounds__(kKldThreads) kld_kernel(const KldParams p) {
  grid_dependency_wait();
  __shared__ double s_buf[kKldThreads / 32];
  __shared__ int s_inf, s_last, s_nfold;
  __shared__ int s_fold[kKldThreads];       // positions (in FL order) of the candidates that fold
  __shared__ double s_select[(kKldThreads / 32) * 2 + 2];   // a SelectScratch
  const int f = blockIdx.x, l = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c_begin = p.fl_begin[f], c_end = p.fl_begin[f + 1];
  const int stride = p.n_bins;
  const LayerState S = p.state[l];
  const int B = p.layers[l].n_bins;        // this layer's bins; arrays are laid out with `stride`
  const long long n = p.layers[l].n;

  if (c_begin == c_end) {
    // no candidate has this fraction length: nothing to write
  } else if (S.flags & (kFlagNonfinite | kFlagRange)) {
    for (int i = c_begin + blockIdx.z * kKldThreads + threadIdx.x; i < c_end;
         i += kKldThreads * gridDim.z) {
      const size_t out = static_cast<size_t>(l) * p.n_cand + p.cand_by_fl[i];
      p.kld_out[out] = __longlong_as_double(0x7ff8000000000000ll);  // NaN: unspecified output
      p.zeros_out[out] = 0;
    }
  } else {
    const unsigned* U = p.u_hist + (static_cast<size_t>(l) * p.n_fl + f) * stride;
    const unsigned* Q = p.q_hist + static_cast<size_t>(l) * stride;
    const double n_eff = static_cast<double>(n) + p.alpha * B;
    const double inf_value = __longlong_as_double(0x7ff0000000000000ll);
    const long long zero_count = static_cast<long long>(p.zeros[static_cast<size_t>(l) * p.n_fl + f]);

    // divergence of the unsaturated histogram, by the whole CTA
    if (threadIdx.x == 0) s_inf = 0;
    __syncthreads();
    double sum = 0.0;
    bool inf = false;
    for (int b = threadIdx.x; b < B; b += kKldThreads) sum += kld_term(U[b], Q[b], p.alpha, &inf);
    if (inf) s_inf = 1;
    sum = block_sum(sum, s_buf);
    double unsat;
    if (n_eff <= 0.0) unsat = 0.0;
    else if (s_inf) unsat = inf_value;
    else { unsat = sum * p.inv_ln_base / n_eff; if (!(unsat > 0.0)) unsat = 0.0; }

    // The candidates of this FL are dealt to the gridDim.z CTAs that share this (FL, layer).  A
    // candidate whose two saturation values fall in the first and the last bin has the
    // unsaturated histogram itself: those are settled one per thread.  The others fold the tails
    // of U[FL] into the bins of their saturation values and are summed one by one: by the whole
    // CTA (by one warp each when the histogram is short), in rounds of kKldThreads candidates.
    constexpr int kWarps = kKldThreads / 32;
    const bool by_warp = B <= ADAPT_KLD_WARP_BINS;
    const int me = by_warp ? lane : threadIdx.x, team = by_warp ? 32 : kKldThreads;
    const int n_mine = (c_end - c_begin - static_cast<int>(blockIdx.z) + static_cast<int>(gridDim.z) - 1) /
                       static_cast<int>(gridDim.z);          // candidates c_begin + z, + gridDim.z, ...
    for (int round0 = 0; round0 < n_mine; round0 += kKldThreads) {
      if (threadIdx.x == 0) s_nfold = 0;
      __syncthreads();
      {
        const int kk = round0 + threadIdx.x;
        if (kk < n_mine) {
          const int i = c_begin + blockIdx.z + kk * gridDim.z;
          const int c = p.cand_by_fl[i];
          const int wl = p.cand_wl[c];
          const int hi_code = static_cast<int>((1ll << (wl - 1)) - 1);
          const int lo_code = static_cast<int>(-(1ll << (wl - 1)));
          const int bh = bin_of(dequantize(hi_code, f), S.lo, S.scale, S.bmax);
          const int bl = bin_of(dequantize(lo_code, f), S.lo, S.scale, S.bmax);
          if (bl == 0 && bh == B - 1 && B > 1 && !p.hist_out) {
            // nothing folds: the candidate's histogram is U[FL] itself
            const size_t out = static_cast<size_t>(l) * p.n_cand + c;
            p.kld_out[out] = unsat;
            p.zeros_out[out] = zero_count;
          } else {
            s_fold[atomicAdd(&s_nfold, 1)] = i;
          }
        }
      }
      __syncthreads();
      const int n_fold = s_nfold;
      for (int j = by_warp ? warp : 0; j < n_fold; j += by_warp ? kWarps : 1) {
      const int i = s_fold[j];
      const int c = p.cand_by_fl[i];
      const int wl = p.cand_wl[c];
      const size_t out = static_cast<size_t>(l) * p.n_cand + c;
      // bins of the two saturation values of <WL,FL>
      const int hi_code = static_cast<int>((1ll << (wl - 1)) - 1);
      const int lo_code = static_cast<int>(-(1ll << (wl - 1)));
      const int bh = bin_of(dequantize(hi_code, f), S.lo, S.scale, S.bmax);
      const int bl = bin_of(dequantize(lo_code, f), S.lo, S.scale, S.bmax);
      unsigned* H = p.hist_out ? p.hist_out + (static_cast<size_t>(l) * (p.n_cand + 1) + c + 1) * stride
                               : nullptr;
      unsigned* H0 = (p.hist_out && c == 0)
                         ? p.hist_out + static_cast<size_t>(l) * (p.n_cand + 1) * stride : nullptr;
      double k;
      {
        // tail masses that fold into bl and bh (exact: sums of counts)
        unsigned long long lo_mass = 0, hi_mass = 0;
        for (int b = me; b < B; b += team) {
          const unsigned u = U[b];
          if (b <= bl) lo_mass += u;
          if (b >= bh) hi_mass += u;
        }
        if (by_warp) {
          lo_mass = warp_sum(lo_mass);
          hi_mass = warp_sum(hi_mass);
        } else {
          lo_mass = static_cast<unsigned long long>(block_sum(static_cast<double>(lo_mass), s_buf));
          hi_mass = static_cast<unsigned long long>(block_sum(static_cast<double>(hi_mass), s_buf));
          if (threadIdx.x == 0) s_inf = 0;
          __syncthreads();
        }
        double part = 0.0;
        bool part_inf = false;
        for (int b = me; b < B; b += team) {
          long long pc;
          if (bl == bh) pc = (b == bl) ? n : 0;
          else if (b < bl || b > bh) pc = 0;
          else if (b == bl) pc = static_cast<long long>(lo_mass);
          else if (b == bh) pc = static_cast<long long>(hi_mass);
          else pc = U[b];
          const long long qc = Q[b];
          if (H) H[b] = static_cast<unsigned>(pc);
          if (H0) H0[b] = static_cast<unsigned>(qc);
          part += kld_term(pc, qc, p.alpha, &part_inf);
        }
        bool any_inf;
        if (by_warp) {
          part = warp_sum(part);
          any_inf = __any_sync(0xffffffffu, part_inf);
        } else {
          if (part_inf) s_inf = 1;
          part = block_sum(part, s_buf);
          any_inf = s_inf != 0;
          __syncthreads();             // s_inf is rewritten by the next candidate
        }
        if (n_eff <= 0.0) k = 0.0;
        else if (any_inf) k = inf_value;
        else { k = part * p.inv_ln_base / n_eff; if (!(k > 0.0)) k = 0.0; }
      }
      if (me == 0) {
        p.kld_out[out] = k;
        p.zeros_out[out] = zero_count;
      }
      }
      __syncthreads();                 // the list is rewritten by the next round
    }
  }

  // the CTA that completes the layer's divergences selects its format
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned done = atomicAdd(&p.state[l].kld_ticket, 1u);
    s_last = (done == gridDim.x * gridDim.z - 1u) ? 1 : 0;
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    select_layer(p, l, reinterpret_cast<SelectScratch*>(s_select));
  }
}

// lexicographic minimum over (key, position): smaller key wins, then earlier position
__device__ __forceinline__ void arg_min_merge(double& k, int& pos, double k2, int pos2) {
  if (pos2 >= 0 && (pos < 0 || k2 < k || (k2 == k && pos2 < pos))) { k = k2; pos = pos2; }
}

// The whole CTA: the layer's choice from its divergences (written by other CTAs of this
// launch: read past the L1 cache).  Every thread looks at the candidates tid, tid + 256, ...;
// warps reduce by shuffles, the CTA through a few words of shared memory.
struct SelectScratch {
  int first[kKldThreads / 32];
  int pos[kKldThreads / 32];
  double key[kKldThreads / 32];
  int spos, last_bad;
};

__device__ void select_layer(const KldParams& p, int l, SelectScratch* sh) {
  constexpr int kWarps = kKldThreads / 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const LayerState S = p.state[l];
  if (p.status_out && tid == 0)        // 2 / 3: the interface's codes for NaN/Inf and |x| >= 2^64
    p.status_out[l] = (S.flags & kFlagNonfinite) ? 2 : ((S.flags & kFlagRange) ? 3 : 0);
  const double* kld = p.kld_out + static_cast<size_t>(l) * p.n_cand;

  if (p.start) {
    // PushDown as a descent (Algorithm 3): from the layer's current format walk down the
    // (WL, FL) order while the divergence stays <= eps; stop before the first violation
    const int swl = p.start[2 * l], sfl = p.start[2 * l + 1];
    if (tid == 0) { sh->spos = 0x7fffffff; sh->last_bad = -1; }
    __syncthreads();
    int spos = 0x7fffffff;     // position of the start format in candidate order
    for (int pos = tid; pos < p.n_cand; pos += kKldThreads) {
      const int c = p.cand_order[pos];
      if (p.cand_wl[c] == swl && p.cand_fl[c] == sfl) spos = min(spos, pos);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) spos = min(spos, __shfl_xor_sync(0xffffffffu, spos, o));
    if (lane == 0 && spos != 0x7fffffff) atomicMin(&sh->spos, spos);
    __syncthreads();
    spos = sh->spos;
    int last_bad = -1;         // highest position below the start whose divergence exceeds eps
    if (spos != 0x7fffffff)
      for (int pos = tid; pos < spos; pos += kKldThreads)
        if (!(__ldcg(kld + p.cand_order[pos]) <= p.eps)) last_bad = max(last_bad, pos);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) last_bad = max(last_bad, __shfl_xor_sync(0xffffffffu, last_bad, o));
    if (lane == 0 && last_bad >= 0) atomicMax(&sh->last_bad, last_bad);
    __syncthreads();
    if (tid == 0) {
      last_bad = sh->last_bad;
      unsigned flags = S.flags & (kFlagDegenerate | kFlagNonfinite | kFlagRange);
      int* o = p.best_out + 4 * l;
      if (spos == 0x7fffffff) { o[0] = swl; o[1] = sfl; o[2] = -1; o[3] = static_cast<int>(flags); return; }
      const bool ok = __ldcg(kld + p.cand_order[spos]) <= p.eps;
      const int pos = ok ? last_bad + 1 : spos;
      const int c = p.cand_order[pos];
      if (ok) flags |= 1u;
      o[0] = p.cand_wl[c]; o[1] = p.cand_fl[c]; o[2] = c; o[3] = static_cast<int>(flags);
    }
    return;
  }

  int first_ok = 0x7fffffff;  // position (in candidate order) of the first KLD <= eps
  double min_k = 0.0;
  int min_pos = -1;           // position of the least finite divergence
  for (int pos = tid; pos < p.n_cand; pos += kKldThreads) {
    const double k = __ldcg(kld + p.cand_order[pos]);
    if (k <= p.eps) first_ok = min(first_ok, pos);
    if (k < __longlong_as_double(0x7ff0000000000000ll)) arg_min_merge(min_k, min_pos, k, pos);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    first_ok = min(first_ok, __shfl_xor_sync(0xffffffffu, first_ok, o));
    double k2 = __shfl_xor_sync(0xffffffffu, min_k, o);
    int pos2 = __shfl_xor_sync(0xffffffffu, min_pos, o);
    arg_min_merge(min_k, min_pos, k2, pos2);
  }
  if (lane == 0) { sh->first[warp] = first_ok; sh->pos[warp] = min_pos; sh->key[warp] = min_k; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kWarps; ++w) {
      first_ok = min(first_ok, sh->first[w]);
      arg_min_merge(min_k, min_pos, sh->key[w], sh->pos[w]);
    }
    unsigned flags = S.flags & (kFlagDegenerate | kFlagNonfinite | kFlagRange);
    int pos;
    if (first_ok != 0x7fffffff) { pos = first_ok; flags |= 1u; }
    else if (min_pos >= 0) pos = min_pos;
    else pos = p.n_cand - 1;
    const int c = p.cand_order[pos];
    int* o = p.best_out + 4 * l;
    o[0] = p.cand_wl[c]; o[1] = p.cand_fl[c]; o[2] = c; o[3] = static_cast<int>(flags);
  }
}

}  // namespace adapt
