// CPU oracle for the AdaPT precision-switch search (PushDown inner body).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, single-threaded
// restatement of the paper's definitions that the GPU library is checked
// against.  It shares no source, header, table or helper with the CUDA path
// and must never be reached from a product call.
//
// What each function follows:
//   quantize    - signed fixed-point <WL,FL> (Sec. 2.1 "Fixed-Point
//                 Quantization"; Sec. 3.2 "Precision Levels", the SR(x) rule)
//   range/bins  - discretisation "via binning" at resolution r (Sec. 3.3,
//                 the EDF equation), read as r equal-width bins on [min,max]
//   normalize   - gradient normalisation g / ||g||_2 (Sec. 3.3, the paragraph on the
//                 limited range of fixed point)
//   kld         - discrete Kullback-Leibler divergence KL(P||Q), P the
//                 quantized tensor, Q the float tensor (Sec. 3.3, Eq. dkld)
//   select      - "smallest quantization s.t. KL = 0" (Sec. 3.3; Algorithm 3)
//   sparsity    - share of non-zero elements (Sec. 3.4 "Inducing Sparsity")
//   diversity   - gradient diversity of a layer's recent gradients (Sec. 3.3, PushUp)
//   pushup      - the suggestions s_1, s_2, the strategy and the new <WL,FL> (Sec. 3.3, PushUp;
//                 the buffer bits of "Dealing with Fixed-Points Limited Range")
//   formats     - block floating point (Sec. 2.1, 2.2) and floating point (Sec. 7) candidates
//                 through the same EDF / KL steps
//
// The paper gives no bit-level rules; the readings taken (saturation,
// ties-to-even, the stochastic-rounding hash, bin arithmetic, the KLD
// summation form, candidate order) are listed in the design notes of the
// repository.  All of them are pinned only by the tests of this oracle
// against hand-worked values, exact rational brute force, closed forms and
// library routines; the counter hash has no outside definition at all
// (parity unpinned beyond its stored vectors and statistics).
//
// Build: g++ -std=c++17 -O2 -ffp-contract=off -fno-fast-math -shared -fPIC

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

namespace {

constexpr int kRoundNearestEven = 0;
constexpr int kRoundStochastic = 1;

// Counter hash (seed, layer, element index) -> 24 uniform bits.
// The paper only says "a random number P" (Sec. 3.2); this mixer is the
// build's own definition: golden-ratio / sqrt(2) / sqrt(3) odd constants,
// three xor-shift-multiply rounds, top 24 bits.
inline uint32_t hash24(uint64_t seed, uint64_t layer, uint64_t index) {
  const uint64_t c1 = 0x9E3779B97F4A7C15ull;
  const uint64_t c2 = 0x6A09E667F3BCC909ull;
  const uint64_t c3 = 0xBB67AE8584CAA73Bull;
  uint64_t z = seed ^ ((layer + 1ull) * c1);
  z += index * c2;
  z ^= z >> 32;
  z *= c1;
  z ^= z >> 29;
  z *= c3;
  z ^= z >> 32;
  return static_cast<uint32_t>(z >> 40);
}

// Rounded, unsaturated integer value of x * 2^FL, kept as a float.
// RNE: nearest, ties to even.  Stochastic (Sec. 3.2, SR(x)): floor, plus one
// when P < (distance above the floor, in quanta); P = k24 * 2^-24 in [0,1).
inline float round_scaled(float x, int fl, int round_mode, uint32_t k24) {
  const float y = x * std::ldexp(1.0f, fl);  // exact power-of-two scaling
  if (round_mode == kRoundNearestEven) {
    return std::nearbyintf(y);  // default rounding mode: ties to even
  }
  const float f = std::floor(y);
  const float frac = y - f;  // one fp32 subtraction
  const float p = static_cast<float>(k24) * std::ldexp(1.0f, -24);  // exact
  return (p < frac) ? f + 1.0f : f;
}

// Two's-complement saturation to WL bits (Sec. 2.1: results must lie within
// the representable boundaries).
inline int32_t saturate(float r, int wl) {
  const float top = std::ldexp(1.0f, wl - 1);  // 2^(WL-1)
  if (r >= top) return static_cast<int32_t>((int64_t(1) << (wl - 1)) - 1);
  if (r <= -top) return static_cast<int32_t>(-(int64_t(1) << (wl - 1)));
  return static_cast<int32_t>(r);  // integral and in range: exact
}

inline float dequantize(int32_t code, int fl) {
  return static_cast<float>(code) * std::ldexp(1.0f, -fl);
}

// Shared-bin index of value v for bins on [lo,hi] (Sec. 3.3, EDF at
// resolution r = n_bins).  Every operation is one IEEE fp32 operation.
inline int bin_index(float v, float lo, float hi, int n_bins) {
  const float w = hi - lo;
  const float scale = (w == 0.0f) ? 0.0f : static_cast<float>(n_bins) / w;
  const float t = v - lo;
  const float u = t * scale;
  float bf = std::floor(u);
  bf = std::fmax(bf, 0.0f);  // fmax returns the non-NaN operand
  bf = std::fmin(bf, static_cast<float>(n_bins - 1));
  return static_cast<int>(bf);
}

}  // namespace

extern "C" {

// ---- element-level entry points (used by the pins) -------------------------

uint32_t adapt_oracle_hash24(uint64_t seed, uint64_t layer, uint64_t index) {
  return hash24(seed, layer, index);
}

int32_t adapt_oracle_quantize_one(float x, int wl, int fl, int round_mode,
                                  uint32_t k24) {
  return saturate(round_scaled(x, fl, round_mode, k24), wl);
}

float adapt_oracle_dequantize_one(int32_t code, int fl) {
  return dequantize(code, fl);
}

int adapt_oracle_bin_index(float v, float lo, float hi, int n_bins) {
  return bin_index(v, lo, hi, n_bins);
}

// ---- tensor-level steps -----------------------------------------------------

// Quantize(L, <WL,FL>) (Algorithm 1, the re-quantisation step; Algorithm 3,
// the Quantize call).  codes_out / xhat_out may be null.
void adapt_oracle_quantize(const float* x, int64_t n, int wl, int fl,
                           int round_mode, uint64_t seed, uint64_t layer,
                           int32_t* codes_out, float* xhat_out) {
  for (int64_t i = 0; i < n; ++i) {
    const uint32_t k =
        (round_mode == kRoundStochastic) ? hash24(seed, layer, uint64_t(i)) : 0u;
    const int32_t c = saturate(round_scaled(x[i], fl, round_mode, k), wl);
    if (codes_out) codes_out[i] = c;
    if (xhat_out) xhat_out[i] = dequantize(c, fl);
  }
}

// min / max of the float tensor; returns 1 if any element is NaN or Inf.
int adapt_oracle_range(const float* x, int64_t n, float* lo_out, float* hi_out) {
  float lo = std::numeric_limits<float>::infinity();
  float hi = -std::numeric_limits<float>::infinity();
  int nonfinite = 0;
  for (int64_t i = 0; i < n; ++i) {
    if (!std::isfinite(x[i])) nonfinite = 1;
    if (x[i] < lo) lo = x[i];
    if (x[i] > hi) hi = x[i];
  }
  if (n == 0) { lo = 0.0f; hi = 0.0f; }
  *lo_out = lo;
  *hi_out = hi;
  return nonfinite;
}

// Histogram of v[0..n) over n_bins shared bins on [lo,hi]; hist is zeroed here.
void adapt_oracle_histogram(const float* v, int64_t n, float lo, float hi,
                            int n_bins, uint64_t* hist) {
  for (int b = 0; b < n_bins; ++b) hist[b] = 0;
  for (int64_t i = 0; i < n; ++i) hist[bin_index(v[i], lo, hi, n_bins)] += 1;
}

// KL(P||Q) from integer bin counts (Eq. dkld), P = quantized, Q = float.
// Both histograms count the same N elements (equal totals are a precondition).
// With p_b/N and q_b/N the bin masses, p*log(p/q) = p*log1p((p-q)/q); the
// count difference is formed exactly in integers so that histograms that
// differ by a few counts in well-filled bins keep their accuracy.  alpha is
// an optional pseudo-count added to every bin of both histograms.  A bin with
// p_b + alpha > 0 and q_b + alpha = 0 makes the divergence +infinity.
// log_base = 2 gives bits (the paper's "number of bits lost").
double adapt_oracle_kld(const uint64_t* p_hist, const uint64_t* q_hist,
                        int n_bins, double alpha, double log_base) {
  double total = 0.0;
  for (int b = 0; b < n_bins; ++b) total += static_cast<double>(p_hist[b]);
  const double n_eff = total + alpha * n_bins;
  if (n_eff <= 0.0) return 0.0;
  double sum = 0.0;
  for (int b = 0; b < n_bins; ++b) {
    const double p = static_cast<double>(p_hist[b]) + alpha;
    const double q = static_cast<double>(q_hist[b]) + alpha;
    if (p <= 0.0) continue;
    if (q <= 0.0) return std::numeric_limits<double>::infinity();
    const int64_t diff =
        static_cast<int64_t>(p_hist[b]) - static_cast<int64_t>(q_hist[b]);
    sum += p * std::log1p(static_cast<double>(diff) / q);
  }
  const double kld = sum / (n_eff * std::log(log_base));
  return kld > 0.0 ? kld : 0.0;
}

// Lowest <WL,FL> whose divergence is <= eps (Sec. 3.3; Algorithm 3).
// Candidates are compared in (WL, FL) lexicographic order whatever their
// order in the arrays.  If none meets eps the candidate of minimal divergence
// is returned (first in that order among ties; if every divergence is +inf,
// the last in that order).  out = {wl, fl, grid index, flags}; flag bit 0 =
// "met eps".
void adapt_oracle_select(const double* kld, const int32_t* wl, const int32_t* fl,
                         int n_cand, double eps, int32_t* out) {
  auto before = [&](int a, int b) {  // a strictly before b in (WL,FL) order
    if (wl[a] != wl[b]) return wl[a] < wl[b];
    if (fl[a] != fl[b]) return fl[a] < fl[b];
    return a < b;
  };
  int best_ok = -1, best_min = -1, last = -1;
  for (int c = 0; c < n_cand; ++c) {
    if (last < 0 || before(last, c)) last = c;
    if (kld[c] <= eps && (best_ok < 0 || before(c, best_ok))) best_ok = c;
    if (std::isfinite(kld[c])) {
      if (best_min < 0 || kld[c] < kld[best_min] ||
          (kld[c] == kld[best_min] && before(c, best_min)))
        best_min = c;
    }
  }
  int pick = best_ok >= 0 ? best_ok : (best_min >= 0 ? best_min : last);
  out[0] = pick >= 0 ? wl[pick] : 0;
  out[1] = pick >= 0 ? fl[pick] : 0;
  out[2] = pick;
  out[3] = best_ok >= 0 ? 1 : 0;
}

// PushDown as a descent from the layer's current format (Algorithm 3: starting at the
// current <WL,FL>, Decrease and re-test until the divergence tells that a coarser format would
// lose information).  Candidates are ordered by (WL, FL); Decrease steps to the previous
// candidate in that order.  The walk starts at the candidate equal to <start_wl, start_fl> and
// stops before the first candidate whose divergence exceeds eps; it returns the lowest format
// reached.  If the start itself exceeds eps it is returned with the "met eps" flag cleared;
// a start that is not in the grid gives grid index -1.
void adapt_oracle_select_descent(const double* kld, const int32_t* wl, const int32_t* fl,
                                 int n_cand, double eps, int start_wl, int start_fl,
                                 int32_t* out) {
  std::vector<int> order(n_cand);
  for (int c = 0; c < n_cand; ++c) order[c] = c;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
    if (wl[a] != wl[b]) return wl[a] < wl[b];
    return fl[a] < fl[b];
  });
  int pos = -1;
  for (int i = 0; i < n_cand; ++i)
    if (wl[order[i]] == start_wl && fl[order[i]] == start_fl) { pos = i; break; }
  if (pos < 0) { out[0] = start_wl; out[1] = start_fl; out[2] = -1; out[3] = 0; return; }
  const bool ok = kld[order[pos]] <= eps;
  if (ok) while (pos > 0 && kld[order[pos - 1]] <= eps) --pos;
  out[0] = wl[order[pos]];
  out[1] = fl[order[pos]];
  out[2] = order[pos];
  out[3] = ok ? 1 : 0;
}

// The whole search for one layer, one candidate at a time, in the order the
// paper's PushDown body takes them: Quantize -> (zero count) -> EDF of both
// tensors over shared bins -> KL -> choice.  No shortcut of any kind.
//   kld_out   double[n_cand]
//   zeros_out int64[n_cand]   count of zero codes (sparsity = 1 - zeros/n)
//   best_out  int32[4]        {wl, fl, grid index, flags}; flag bit 1 = the
//                             tensor's range is degenerate (max == min or n==0)
//   hist_out  uint64[(n_cand+1)*n_bins] or null; slot 0 = float histogram
//   range_out float[2] or null
// Returns 1 if the tensor holds a NaN or Inf (outputs then unspecified).
int adapt_oracle_precision_search(const float* x, int64_t n, uint64_t layer,
                                  const int32_t* wl, const int32_t* fl,
                                  int n_cand, int n_bins, int round_mode,
                                  uint64_t seed, double eps, double alpha,
                                  double log_base, double* kld_out,
                                  int64_t* zeros_out, int32_t* best_out,
                                  uint64_t* hist_out, float* range_out) {
  float lo, hi;
  const int nonfinite = adapt_oracle_range(x, n, &lo, &hi);
  if (range_out) { range_out[0] = lo; range_out[1] = hi; }
  if (nonfinite) return 1;

  std::vector<uint64_t> q_hist(n_bins), p_hist(n_bins);
  std::vector<int32_t> codes(static_cast<size_t>(n));
  std::vector<float> xhat(static_cast<size_t>(n));

  adapt_oracle_histogram(x, n, lo, hi, n_bins, q_hist.data());
  if (hist_out) std::memcpy(hist_out, q_hist.data(), sizeof(uint64_t) * n_bins);

  for (int c = 0; c < n_cand; ++c) {
    adapt_oracle_quantize(x, n, wl[c], fl[c], round_mode, seed, layer,
                          codes.data(), xhat.data());
    int64_t zeros = 0;
    for (int64_t i = 0; i < n; ++i) zeros += (codes[i] == 0);
    zeros_out[c] = zeros;
    adapt_oracle_histogram(xhat.data(), n, lo, hi, n_bins, p_hist.data());
    if (hist_out)
      std::memcpy(hist_out + size_t(c + 1) * n_bins, p_hist.data(),
                  sizeof(uint64_t) * n_bins);
    kld_out[c] = adapt_oracle_kld(p_hist.data(), q_hist.data(), n_bins, alpha,
                                  log_base);
  }
  adapt_oracle_select(kld_out, wl, fl, n_cand, eps, best_out);
  if (n == 0 || hi == lo) best_out[3] |= 2;
  return 0;
}

// ---- gradient diversity (PushUp's input) ---------------------------------------------

// Gradient normalisation of Sec. 3.3 ("Dealing with Fixed-Points Limited Range"):
// g <- g / ||g||_2.  The norm is the square root of the sum of squares taken in double,
// elements in order; each quotient is formed in double and rounded to float.  A gradient
// whose norm is 0 (all zeros) is returned unchanged (the paper does not say; 0/0 has no value).
void adapt_oracle_normalize_gradient(const float* g, int64_t n, float* out) {
  double sq = 0.0;
  for (int64_t i = 0; i < n; ++i) sq += static_cast<double>(g[i]) * g[i];
  const double norm = std::sqrt(sq);
  for (int64_t i = 0; i < n; ++i)
    out[i] = norm > 0.0 ? static_cast<float>(static_cast<double>(g[i]) / norm) : g[i];
}

// Gradient diversity of one layer over its last n_grads gradient tensors (Sec. 3.3, the
// PushUp heuristic, Eq. ourgd / its log form):
//   delta_s = sum_k ||g_k||_2 / || sum_k g_k ||_2 ,
//   log form = log(delta_s) if 0 < delta_s < inf, else 1.
// grads[k] points to n fp32 values; everything is accumulated in double, in index order.
// out = {sum of norms, norm of the sum, delta_s, log form}.  0/0 gives NaN for delta_s
// (log form 1); x/0 gives +inf (log form 1).
void adapt_oracle_gradient_diversity(const float* const* grads, int n_grads, int64_t n,
                                     double* out) {
  double sum_norms = 0.0;
  for (int k = 0; k < n_grads; ++k) {
    double sq = 0.0;
    for (int64_t i = 0; i < n; ++i) sq += static_cast<double>(grads[k][i]) * grads[k][i];
    sum_norms += std::sqrt(sq);
  }
  double sq_sum = 0.0;
  for (int64_t i = 0; i < n; ++i) {
    double s = 0.0;
    for (int k = 0; k < n_grads; ++k) s += grads[k][i];
    sq_sum += s * s;
  }
  const double norm_sum = std::sqrt(sq_sum);
  const double ds = sum_norms / norm_sum;
  out[0] = sum_norms;
  out[1] = norm_sum;
  out[2] = ds;
  out[3] = (ds > 0.0 && std::isfinite(ds)) ? std::log(ds) : 1.0;
}

// ---- PushUp: the new <WL,FL> of a layer from its gradient diversity ------------------------
//
// Sec. 3.3 "The PushUp Operation" and "Dealing with Fixed-Points Limited Range", in the
// paper's order and notation.  Inputs: d = the log form of the gradient diversity (above),
// <WL_min, FL_min> = what PushDown returned, st = the global strategy (0 min, 1 mean, 2 max),
// buff = the buffer bits.  Steps:
//   if d > 0:  s_1 = max(ceil(1 / (d - 1)), 1)
//              s_2 = max(ceil(min(32 d^2 - 1, 32)) - FL_min, 1)
//              s   = min(s_1, s_2) | ceil(0.5 (s_1 + s_2)) | max(s_1, s_2)      by st
//   else       s   = 1
//   FL = min(FL_min + s, 32);   WL = min(max(WL_min, FL) + 1, 32)
//   FL = min(FL, 32 - buff);    WL = max(min(FL + buff, 32), WL)
//   FL = min(FL, WL - 1)        (a word keeps at least its sign bit)
// Readings where the text leaves a choice: the quotient of s_1 is 1 / (d - 1) as printed (its
// denominator 0 gives the largest suggestion, and every suggestion is capped at 32, beyond
// which FL cannot move anyway); the real number inside s_2 is rounded up like every other
// rounding of the paragraph; the second "if" of the text, printed with the same condition as
// the first, is its complement; d stands for "log delta_s" also where delta_s is 0 or not
// finite (d = 1 then); the FL inside WL's max is the new one, since with the old one the word
// could come out shorter than its fraction; the buffer step works on the values just computed.
// out = {WL, FL, s_1, s_2, s} (s_1 = s_2 = 0 when d <= 0).  All real arithmetic in double.
void adapt_oracle_pushup(double d, int wl_min, int fl_min, int st, int buff, int32_t* out) {
  int s1 = 0, s2 = 0, s = 1;
  if (d > 0.0) {
    const double q = 1.0 / (d - 1.0);                 // +inf when d == 1
    s1 = (q >= 32.0) ? 32 : static_cast<int>(std::fmax(std::ceil(q), 1.0));
    const double w = std::fmin(32.0 * (d * d) - 1.0, 32.0);
    s2 = std::max(static_cast<int>(std::ceil(w)) - fl_min, 1);
    s2 = std::min(s2, 32);
    if (st == 0) s = std::min(s1, s2);
    else if (st == 1) s = (s1 + s2 + 1) / 2;          // ceil(0.5 (s_1 + s_2)) for integers
    else s = std::max(s1, s2);
  }
  int fl = std::min(fl_min + s, 32);
  int wl = std::min(std::max(wl_min, fl) + 1, 32);
  fl = std::min(fl, 32 - buff);
  wl = std::max(std::min(fl + buff, 32), wl);
  fl = std::min(fl, wl - 1);
  out[0] = wl; out[1] = fl; out[2] = s1; out[3] = s2; out[4] = s;
}

// ---- other number formats through the same EDF / KL machinery ---------------------------
//
// The paper names two formats besides fixed point: block floating point (Sec. 2.1
// "Block-Floating-Point Quantization"; Sec. 2.2, MuPPET's per-layer scale) and, as future work
// (Sec. 7), floating-point quantization.  A candidate format is a triple (kind, a, b):
//   kind 0  fixed point      a = WL, b = FL                   (as above)
//   kind 1  block floating   a = WL, b unused on input: the block is the layer and its scale s
//                            follows from the layer's extremes; value = code * 2^-s
//   kind 2  floating point   a = E exponent bits (2..8), b = M mantissa bits (1..23), IEEE-like:
//                            bias 2^(E-1)-1, the all-ones exponent reserved, gradual underflow
// The floating-point rules are this build's reading (the paper gives none): parity unpinned by
// the paper, pinned by the tests against IEEE half precision (numpy) and bfloat16 (torch).

namespace {
constexpr int kFmtFixed = 0, kFmtBfp = 1, kFmtFloat = 2;
constexpr int kBfpScaleLimit = 100;  // |s| <= 100 keeps 2^s and 2^-s normal floats
}  // namespace

// Scale of a block whose extremes are lo <= hi (Sec. 2.2):
//   s = floor(log2(min((UB + 0.5) / X_max, (LB - 0.5) / X_min))), UB = 2^(WL-1)-1, LB = -2^(WL-1),
// i.e. the largest integer s with X_max * 2^s <= UB + 0.5 and |X_min| * 2^s <= |LB| + 0.5.
// A ratio whose extreme has the wrong sign or is zero sets no limit (X_max <= 0, X_min >= 0);
// with no limit at all (every element zero) s = 0.  s is kept within [-100, 100].
// The products are exact in double (a float times a power of two), so no logarithm is rounded.
int adapt_oracle_bfp_scale(float lo, float hi, int wl) {
  const double ub = std::ldexp(1.0, wl - 1) - 1.0 + 0.5;
  const double lb = std::ldexp(1.0, wl - 1) + 0.5;
  const bool lim_hi = hi > 0.0f, lim_lo = lo < 0.0f;
  if (!lim_hi && !lim_lo) return 0;
  for (int s = kBfpScaleLimit; s > -kBfpScaleLimit; --s) {
    const bool ok_hi = !lim_hi || std::ldexp(static_cast<double>(hi), s) <= ub;
    const bool ok_lo = !lim_lo || std::ldexp(-static_cast<double>(lo), s) <= lb;
    if (ok_hi && ok_lo) return s;
  }
  return -kBfpScaleLimit;
}

// Value of x in the floating-point format <E,M>: round x to M fraction bits of its own binade
// (of the lowest normal binade 2^emin when |x| is below it: gradual underflow), then clamp to
// the largest finite value (2 - 2^-M) * 2^emax (saturation, as for fixed point; no infinities).
// Rounding is RNE or the SR(x) rule of Sec. 3.2 on the local grid: y = x / quantum is exact,
// the rest is the fixed-point rule applied to y.
static float float_format_value(float x, int e_bits, int m_bits, int round_mode, uint32_t k24) {
  if (x == 0.0f) return 0.0f;
  const int bias = (1 << (e_bits - 1)) - 1;
  const int emin = 1 - bias, emax = bias;
  const int e = std::ilogb(x);                 // floor(log2 |x|), subnormal x included
  const int ee = std::max(e, emin);
  const float y = std::ldexp(x, m_bits - ee);  // |y| < 2^(M+1): exact
  float r;
  if (round_mode == kRoundNearestEven) {
    r = std::nearbyintf(y);
  } else {
    const float f = std::floor(y);
    const float frac = y - f;
    const float p = static_cast<float>(k24) * std::ldexp(1.0f, -24);
    r = (p < frac) ? f + 1.0f : f;
  }
  float v = std::ldexp(r, ee - m_bits);        // integer times a power of two >= 2^-149: exact
  const float top = std::ldexp(2.0f - std::ldexp(1.0f, -m_bits), emax);
  if (v > top) v = top;
  if (v < -top) v = -top;
  return v;
}

// One element in one format; for kinds 0 and 1, b is the fraction length / block scale.
float adapt_oracle_format_value_one(float x, int kind, int a, int b, int round_mode,
                                    uint32_t k24) {
  if (kind == kFmtFloat) return float_format_value(x, a, b, round_mode, k24);
  return dequantize(saturate(round_scaled(x, b, round_mode, k24), a), b);
}

// A tensor in one format: values_out[i] = the representable value x_i maps to.
void adapt_oracle_format_quantize(const float* x, int64_t n, int kind, int a, int b,
                                  int round_mode, uint64_t seed, uint64_t layer,
                                  float* values_out) {
  for (int64_t i = 0; i < n; ++i) {
    const uint32_t k =
        (round_mode == kRoundStochastic) ? hash24(seed, layer, uint64_t(i)) : 0u;
    values_out[i] = adapt_oracle_format_value_one(x[i], kind, a, b, round_mode, k);
  }
}

// The PushDown body over a list of formats of any kind, one candidate at a time: Quantize ->
// zero count -> EDF over the shared bins -> KL -> choice.  The candidates are taken in the
// caller's order (the caller lists them from cheapest to most expensive): the first one whose
// divergence is <= eps is chosen, else the one of least divergence (first among ties; the last
// candidate if every divergence is +inf).
//   kld_out double[n_cand], zeros_out int64[n_cand] (values equal to zero)
//   b_out   int32[n_cand]: b as used (the derived scale for kind 1, the given b otherwise)
//   best_out int32[4] = {a, b as used, index, flags}; flags as in adapt_oracle_precision_search
int adapt_oracle_format_search(const float* x, int64_t n, uint64_t layer, const int32_t* kind,
                               const int32_t* a, const int32_t* b, int n_cand, int n_bins,
                               int round_mode, uint64_t seed, double eps, double alpha,
                               double log_base, double* kld_out, int64_t* zeros_out,
                               int32_t* b_out, int32_t* best_out, float* range_out) {
  float lo, hi;
  const int nonfinite = adapt_oracle_range(x, n, &lo, &hi);
  if (range_out) { range_out[0] = lo; range_out[1] = hi; }
  if (nonfinite) return 1;
  std::vector<uint64_t> q_hist(n_bins), p_hist(n_bins);
  std::vector<float> values(static_cast<size_t>(n));
  adapt_oracle_histogram(x, n, lo, hi, n_bins, q_hist.data());
  for (int c = 0; c < n_cand; ++c) {
    const int bc = (kind[c] == kFmtBfp) ? adapt_oracle_bfp_scale(lo, hi, a[c]) : b[c];
    b_out[c] = bc;
    adapt_oracle_format_quantize(x, n, kind[c], a[c], bc, round_mode, seed, layer, values.data());
    int64_t zeros = 0;
    for (int64_t i = 0; i < n; ++i) zeros += (values[i] == 0.0f);
    zeros_out[c] = zeros;
    adapt_oracle_histogram(values.data(), n, lo, hi, n_bins, p_hist.data());
    kld_out[c] = adapt_oracle_kld(p_hist.data(), q_hist.data(), n_bins, alpha, log_base);
  }
  int first_ok = -1, least = -1;
  for (int c = 0; c < n_cand; ++c) {
    if (first_ok < 0 && kld_out[c] <= eps) first_ok = c;
    if (std::isfinite(kld_out[c]) && (least < 0 || kld_out[c] < kld_out[least])) least = c;
  }
  const int pick = first_ok >= 0 ? first_ok : (least >= 0 ? least : n_cand - 1);
  best_out[0] = pick >= 0 ? a[pick] : 0;
  best_out[1] = pick >= 0 ? b_out[pick] : 0;
  best_out[2] = pick;
  best_out[3] = (first_ok >= 0 ? 1 : 0) | ((n == 0 || hi == lo) ? 2 : 0);
  return 0;
}

}  // extern "C"
