/* adapt.h - C ABI of the B200 precision-switch search library (libadapt_b200.so).
 *
 * The library implements the data-parallel body of AdaPT's PushDown operation
 * (Sec. 3.3 "The PushDown Operation"; Algorithm 3), evaluated for a whole grid
 * of candidate fixed-point formats at once, plus the stand-alone Quantize step
 * (Algorithm 1, the per-layer re-quantisation loop).
 *
 * Conventions that hold for every entry point unless its comment says otherwise
 *  - Pointers marked DEVICE are CUDA device pointers on the current device and
 *    stay owned by the caller; pointers marked HOST are ordinary host memory,
 *    read (or written) before the call returns.
 *  - Calls enqueue their kernels on a CUDA stream (the legacy default stream
 *    for the entry points without a stream argument) and return without
 *    waiting; outputs are valid once that stream has been synchronised.  A
 *    search may run one of its kernels on a stream of the library's own; that
 *    stream branches off the caller's stream and joins it again inside the
 *    call (events), so to the caller the call still is work on one stream,
 *    and it may be captured into a CUDA graph.
 *  - The return value is an adapt_status.  Errors that the host can see (null
 *    pointers, sizes or formats out of range, workspace too small) return
 *    before anything is launched and write nothing.  Errors in the data
 *    (NaN/Inf elements, |x| >= 2^64) cannot be seen by the host without a
 *    device round trip: they are reported per layer in best_out's flag word
 *    (and, when asked for, as a status word per layer in opts->status_out);
 *    the other outputs of that layer are then unspecified (but in bounds).
 *    Nothing traps on the device and no C++ exception crosses this boundary.
 *  - Formats: 2 <= WL <= 32, 0 <= FL <= WL-1 (Sec. 2.1: a WL-bit signed word
 *    with FL fractional bits; value = code * 2^-FL, code in
 *    [-2^(WL-1), 2^(WL-1)-1]).  Values outside the range saturate.
 *  - Limits: fewer than 2^32 elements per layer; 1 <= n_bins <= 16384;
 *    1 <= n_cand <= 65535; 1 <= n_layers <= 65535.
 */
#ifndef ADAPT_B200_H_
#define ADAPT_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ADAPT_OK = 0,
  ADAPT_ERR_INVALID_ARG = 1, /* null pointer, bad size, bad <WL,FL>, bad mode   */
  ADAPT_ERR_NONFINITE = 2,   /* (host-side entry points only) NaN/Inf in input  */
  ADAPT_ERR_RANGE = 3,       /* (host-side entry points only) |x| >= 2^64       */
  ADAPT_ERR_CUDA = 4,        /* a CUDA runtime call failed                      */
  ADAPT_ERR_WORKSPACE = 5    /* caller-supplied workspace is too small          */
} adapt_status;

/* Rounding of x * 2^FL to an integer (Sec. 3.2 "Precision Levels").
 * RNE: round to nearest, ties to even.
 * STOCHASTIC: the SR(x) rule - floor, plus one when P < fractional position,
 * with P = k / 2^24 drawn per element from a counter hash of
 * (seed, layer, element index); all candidates of one element share its P. */
enum { ADAPT_ROUND_RNE = 0, ADAPT_ROUND_STOCHASTIC = 1 };

/* Flag bits of best_out[l*4 + 3]. */
enum {
  ADAPT_FLAG_MET_EPS = 1,    /* the returned candidate has KLD <= eps           */
  ADAPT_FLAG_DEGENERATE = 2, /* max == min (or empty layer): one bin, KLD == 0  */
  ADAPT_FLAG_NONFINITE = 4,  /* layer holds NaN/Inf: its outputs are unspecified */
  ADAPT_FLAG_RANGE = 8       /* layer holds |x| >= 2^64 (and no NaN/Inf): outputs unspecified */
};

/* Candidate formats. HOST arrays of n_cand entries each, in any order. */
typedef struct adapt_grid {
  int32_t n_cand;
  const int32_t* wl;
  const int32_t* fl;
} adapt_grid;

/* Options of the _ex / _host search calls.  Zero-initialise, then set fields;
 * log_base == 0 means 2 (bits). */
typedef struct adapt_search_opts {
  int32_t round_mode;     /* ADAPT_ROUND_*                                      */
  int32_t layer_base;     /* hash layer id of tensors[l] is layer_base + l      */
  uint64_t seed;          /* stochastic rounding seed                           */
  double eps;             /* accept a candidate when KLD <= eps (default 0)     */
  double pseudo_count;    /* added to every bin of both histograms (default 0)  */
  double log_base;        /* base of the logarithm; 0 -> 2                      */
  void* stream;           /* cudaStream_t; NULL = legacy default stream         */
  void* workspace;        /* DEVICE scratch, 256-byte aligned, or NULL to use a
                             library-owned buffer that grows on demand          */
  size_t workspace_bytes; /* size of workspace                                  */
  uint32_t* hist_out;     /* DEVICE, optional: uint32[n_layers][n_cand+1][n_bins],
                             slot 0 = histogram of the float tensor, slot c+1 =
                             histogram of candidate c's dequantized tensor      */
  float* range_out;       /* DEVICE, optional: float[n_layers][2] = {min, max}  */
  int32_t algorithm;      /* ADAPT_ALGO_*: which form of the fused kernel runs  */
  const int32_t* n_bins_per_layer; /* HOST, optional: int32[n_layers], the resolution
                             r^l of each layer (Sec. 3.3: bins are a per-layer
                             quantity).  When set, the n_bins argument is ignored
                             for the bin arithmetic; hist_out and the workspace
                             are laid out for the largest value, which is also
                             what adapt_search_workspace_bytes must be asked for;
                             bins of hist_out beyond a layer's own count are not
                             written                                             */
  const int32_t* start_wl_fl; /* HOST, optional: int32[n_layers][2], each layer's
                             current <WL,FL>.  When set, best_out is PushDown as
                             Algorithm 3 walks it: from that format step down the
                             (WL, FL) order of the grid while KLD <= eps and
                             return the lowest format reached before the first
                             violation (flag "met eps" cleared and the start
                             returned if the start itself violates; grid index
                             -1 if the start is not in the grid).  When NULL,
                             best_out is the lowest admissible format of the
                             whole grid                                          */
  int32_t* status_out;    /* DEVICE, optional: int32[n_layers], the adapt_status of
                             each layer's data - ADAPT_OK, ADAPT_ERR_NONFINITE
                             (NaN/Inf in the layer) or ADAPT_ERR_RANGE
                             (|x| >= 2^64) - the same facts as the flag bits of
                             best_out, as one status word per layer              */
} adapt_search_opts;

/* Forms of the fused quantize / zero-count / histogram kernel.  Both give the
 * same results bit for bit.  AUTO: the keyed form for layers of at least 32768
 * elements under round-to-nearest-even, and under stochastic rounding for
 * layers of at least 2^20 elements when the call holds 2^22 of them, in both
 * cases with n_bins <= 8192; the direct form for the rest.  KEYED: the keyed
 * form for every layer it can serve (n_bins <= 8192; under stochastic rounding
 * a layer whose range lies too far from zero for exact cell indices stays with
 * the direct form).  DIRECT: the direct form everywhere. */
enum { ADAPT_ALGO_AUTO = 0, ADAPT_ALGO_KEYED = 1, ADAPT_ALGO_DIRECT = 2 };

/* Library version string: "adapt-b200 <major>.<minor>". Never NULL. */
const char* adapt_version(void);

/* Static English text for an adapt_status value. Never NULL. */
const char* adapt_status_string(int status);

/* Detail text of the calling thread's most recent failing call: the CUDA error
 * string, or the limit that was exceeded ("" if none).  The buffer belongs to the
 * calling thread and stays valid until that thread's next failing call. */
const char* adapt_last_error(void);

/* Quantize(L, <WL,FL>) - Algorithm 1 (re-quantisation of each layer after the
 * update) and Algorithm 3 (the Quantize call inside PushDown); format and
 * rounding as in Sec. 2.1 / Sec. 3.2.
 *   x         DEVICE fp32[n], any 4-byte alignment
 *   codes_out DEVICE int32[n]: saturated two's-complement codes
 *   seed      used only by ADAPT_ROUND_STOCHASTIC; hash layer id is 0
 * n == 0 is legal and launches nothing. */
int adapt_quantize(const float* x, int64_t n, int wl, int fl, int round_mode,
                   uint64_t seed, int32_t* codes_out);

/* As adapt_quantize with a hash layer id, an output width and a stream.
 *   code_bits 8, 16 or 32: codes_out is int8/int16/int32[n]; WL must fit.
 *   stream    cudaStream_t or NULL */
int adapt_quantize_ex(const float* x, int64_t n, int wl, int fl, int round_mode,
                      uint64_t seed, int32_t layer, int code_bits,
                      void* codes_out, void* stream);

/* Quantize at a format that is still on the device: `selected` is DEVICE
 * int32[4] as written by a search into best_out + 4*l ({wl, fl, index, flags}).
 * This is Algorithm 1's Quantize(L[l], Q[l].quant) directly after the switch,
 * without a host round trip.  codes_out is DEVICE int32[n]. */
int adapt_quantize_selected(const float* x, int64_t n, const int32_t* selected,
                            int round_mode, uint64_t seed, int32_t layer,
                            int32_t* codes_out, void* stream);

/* Batched form of adapt_quantize_selected: the whole re-quantisation loop of
 * Algorithm 1 (for each layer l: Quantize(L[l], Q[l].quant)) in one launch,
 * every layer at the <WL,FL> the search left for it on the device.
 *   tensors   HOST array of n_layers DEVICE pointers (fp32, 4-byte aligned)
 *   lens      HOST array of element counts (0 allowed)
 *   best      DEVICE int32[n_layers][4], as written by a search
 *   codes_out HOST array of n_layers DEVICE pointers, int32[lens[l]] each
 *   hash layer id of tensors[l] is layer_base + l
 * A layer whose selection is not a valid format is left untouched.  The layer
 * table travels through a library-owned device buffer that is allocated (and
 * grown) inside the call; calls that use it must not overlap on the device. */
int adapt_quantize_selected_batch(const float* const* tensors, const int64_t* lens,
                                  int n_layers, const int32_t* best, int round_mode,
                                  uint64_t seed, int32_t layer_base,
                                  int32_t* const* codes_out, void* stream);

/* adapt_quantize_selected_batch with packed codes: codes_out[l] is DEVICE
 * int8[lens[l]] (code_bits 8), int16[...] (16) or int32[...] (32), aligned to
 * its element size.  The word length of a layer is only known on the device: a
 * layer whose selected WL exceeds code_bits is left untouched and, when
 * unfit_out is given (DEVICE int32[n_layers], cleared by the call), reported
 * there as unfit_out[l] = WL; all other entries stay 0.  (Algorithm 1, the
 * Quantize of every layer after the switch; the packed forms pay once the
 * search has settled on short word lengths: 1 or 2 bytes written per element
 * instead of 4.) */
int adapt_quantize_selected_batch_packed(const float* const* tensors, const int64_t* lens,
                                         int n_layers, const int32_t* best, int round_mode,
                                         uint64_t seed, int32_t layer_base, int code_bits,
                                         void* const* codes_out, int32_t* unfit_out,
                                         void* stream);

/* The same loop with the dequantized values as output: values_out[l][i] =
 * code * 2^-FL as fp32, code as adapt_quantize_selected_batch would write it.
 * This is the layer as a float32 simulation of fixed-point training continues
 * with it (Sec. 4.1: the quantized network is simulated in float32; Algorithm 1,
 * Quantize of every layer after the precision switch).
 *   values_out HOST array of n_layers DEVICE pointers, fp32[lens[l]] each;
 *              values_out[l] may be tensors[l] itself (in place), but must not
 *              overlap it otherwise
 * Other arguments, the untouched layers and the library-owned layer table as
 * for adapt_quantize_selected_batch. */
int adapt_requantize_selected_batch(const float* const* tensors, const int64_t* lens,
                                    int n_layers, const int32_t* best, int round_mode,
                                    uint64_t seed, int32_t layer_base,
                                    float* const* values_out, void* stream);

/* Gradient diversity of each layer over its last n_grads gradient tensors -
 * the quantity PushUp reads (Sec. 3.3, the gradient-diversity equation and its
 * log form):  delta_s = sum_k ||g_k||_2 / || sum_k g_k ||_2, and
 * log(delta_s) when 0 < delta_s < inf, else 1 (natural logarithm).
 *   grads   HOST array of n_layers * n_grads DEVICE pointers, grads[l*n_grads+k]
 *           = gradient k of layer l: fp32[lens[l]], 4-byte aligned
 *   lens    HOST array of n_layers element counts
 *   n_grads 1..256 gradient tensors per layer (the lookback)
 *   out     DEVICE double[n_layers][4] = {sum of norms, norm of the sum,
 *           delta_s, log form}; squares and sums are accumulated in double
 * Pointer table and partial sums live in a library-owned device buffer that is
 * allocated (and grown) inside the call; calls that use it must not overlap on
 * the device. */
int adapt_gradient_diversity(const float* const* grads, const int64_t* lens, int n_layers,
                             int n_grads, double* out, void* stream);

/* Strategies of PushUp (Sec. 3.3, the strategy equation). */
enum { ADAPT_STRATEGY_MIN = 0, ADAPT_STRATEGY_MEAN = 1, ADAPT_STRATEGY_MAX = 2 };

/* PushUp's scalar step (Sec. 3.3 "The PushUp Operation"; buffer bits of "Dealing with
 * Fixed-Points Limited Range"): from each layer's gradient diversity and the format that
 * PushDown found, the format the layer trains on next.  Host arithmetic only - a handful of
 * scalar operations per layer; nothing is launched and no device is touched.
 * With d = diversity[l][3] (the log form adapt_gradient_diversity writes) and
 * <WL_min, FL_min> = best[l][0..1] (as a search writes it):
 *   d > 0:  s1 = max(ceil(1 / (d - 1)), 1), s2 = max(ceil(min(32 d^2 - 1, 32)) - FL_min, 1),
 *           s = min(s1, s2) | ceil((s1 + s2) / 2) | max(s1, s2) by strategy;   else s = 1
 *   FL = min(FL_min + s, 32),   WL = min(max(WL_min, FL) + 1, 32)
 *   FL = min(FL, 32 - buff),    WL = max(min(FL + buff, 32), WL),   FL = min(FL, WL - 1)
 * Readings of the printed text: the quotient's denominator is d - 1 as printed (0 gives the
 * largest suggestion; suggestions are capped at 32, beyond which FL cannot move); the real
 * number in s2 is rounded up like the paragraph's other roundings; the text's second case,
 * printed with the first one's condition, is its complement; the FL inside WL's max is the
 * new one (with the old one the word could come out shorter than its fraction); the buffer
 * step works on the values just computed; the last step keeps the sign bit when buff is 0.
 *   diversity      HOST double[n_layers][4], rows as adapt_gradient_diversity writes them
 *   best           HOST int32[n_layers][4], rows as a search writes them ({wl, fl, ...})
 *   strategy       ADAPT_STRATEGY_*
 *   buff           buffer bits, 0..31 (the paper trains with 4 and 8)
 *   wl_fl_out      HOST int32[n_layers][2] = {WL, FL}: a valid format, WL >= WL_min
 *   suggestion_out HOST int32[n_layers][3] = {s1, s2, s} or NULL (s1 = s2 = 0 when d <= 0)
 * ADAPT_ERR_INVALID_ARG (nothing written) for null pointers, n_layers < 1, an unknown strategy,
 * buff outside 0..31, or a row of best that is not a format (2 <= WL <= 32, 0 <= FL < WL). */
int adapt_pushup(const double* diversity, const int32_t* best, int n_layers, int strategy,
                 int buff, int32_t* wl_fl_out, int32_t* suggestion_out);

/* Gradient normalisation of Sec. 3.3 ("Dealing with Fixed-Points Limited
 * Range"): every layer's gradient is divided by its own L2 norm,
 * out[l][i] = grads[l][i] / ||grads[l]||_2, so that an update step cannot move
 * weights out of the representable range.  The norm is the square root of the
 * sum of squares accumulated in double, each quotient is formed in double (as a
 * product with the norm's reciprocal) and rounded to fp32: within one fp32 ulp
 * of the correctly rounded quotient; a layer whose norm is 0 is copied unchanged.
 *   grads     HOST array of n_layers DEVICE pointers (fp32, 4-byte aligned)
 *   lens      HOST array of element counts (0 allowed)
 *   out       HOST array of n_layers DEVICE pointers, fp32[lens[l]] each;
 *             out[l] may be grads[l] itself (in place), no other overlap
 *   norms_out optional DEVICE double[n_layers]: the SUMS OF SQUARES ||g||_2^2
 * Two launches (reduction, scaling): 4 + 8 bytes per element.  Uses the same
 * library-owned device buffer as adapt_gradient_diversity (allocated and grown
 * inside the call); calls that use it must not overlap on the device. */
int adapt_normalize_gradients(const float* const* grads, const int64_t* lens, int n_layers,
                              float* const* out, double* norms_out, void* stream);

/* Bytes of DEVICE workspace the search needs for these sizes (0 on invalid
 * arguments).  lens is a HOST array. */
size_t adapt_search_workspace_bytes(const int64_t* lens, int n_layers,
                                    const adapt_grid* wl_fl_grid, int n_bins);

/* The precision-switch search - the body of PushDown (Sec. 3.3; Algorithm 3)
 * for every candidate of the grid and every layer in one batched pass:
 * quantize each element to each <WL,FL>, count zero codes (the sparsity of
 * Sec. 3.4), histogram the float tensor and every candidate's dequantized
 * tensor over n_bins shared equal-width bins on the float tensor's [min,max]
 * (the EDF of Sec. 3.3 at resolution n_bins), take KL(P||Q) in bits with P the
 * candidate and Q the float histogram (the discrete KL equation), and pick the
 * lowest <WL,FL> (by WL, then FL) whose divergence is 0; if none is, the
 * candidate of least divergence.  Round-to-nearest-even, eps = 0.
 *   tensors   HOST array of n_layers DEVICE pointers, fp32, 4-byte aligned
 *   lens      HOST array of n_layers element counts (0 allowed)
 *   kld_out   DEVICE double[n_layers][n_cand]   (+inf where a filled P bin
 *             meets an empty Q bin)
 *   zeros_out DEVICE int64[n_layers][n_cand]    zero codes per candidate
 *   best_out  DEVICE int32[n_layers][4]         {wl, fl, grid index, flags}
 * Scratch comes from a library-owned device buffer that is allocated (and
 * grown) inside the call when needed and is shared by every call that does
 * not bring its own: such calls must not overlap on the device (issue them on
 * one stream).  Use the _ex call to supply your own workspace. */
int adapt_precision_search(const float* const* tensors, const int64_t* lens,
                           int n_layers, const adapt_grid* wl_fl_grid, int n_bins,
                           double* kld_out, int64_t* zeros_out, int32_t* best_out);

/* As adapt_precision_search, with options (rounding mode and seed, eps,
 * pseudo-count, log base, stream, caller workspace, optional histogram and
 * range outputs).  opts may be NULL (= all defaults). */
int adapt_precision_search_ex(const float* const* tensors, const int64_t* lens,
                              int n_layers, const adapt_grid* wl_fl_grid, int n_bins,
                              double* kld_out, int64_t* zeros_out, int32_t* best_out,
                              const adapt_search_opts* opts);

/* Host-buffer form of the search: tensors[l] and the three outputs are HOST
 * memory (pinned memory makes the copies asynchronous and fast).  The call
 * copies the layers to a library-owned device buffer, runs the search,
 * copies the results back and synchronises the stream before returning, so
 * data errors are returned as ADAPT_ERR_NONFINITE / ADAPT_ERR_RANGE.
 * opts->workspace, hist_out, range_out and status_out must be NULL/0 here. */
int adapt_precision_search_host(const float* const* tensors, const int64_t* lens,
                                int n_layers, const adapt_grid* wl_fl_grid, int n_bins,
                                double* kld_out, int64_t* zeros_out, int32_t* best_out,
                                const adapt_search_opts* opts);

/* Host-buffer form of the whole switch step: the search as in
 * adapt_precision_search_host, then Algorithm 1's re-quantisation of every
 * layer at its selected <WL,FL>, from the same device copy of the layers (one
 * upload serves both).
 *   codes_out HOST array of n_layers HOST pointers, int32[lens[l]] each
 * Everything else as adapt_precision_search_host; synchronous. */
int adapt_precision_switch_host(const float* const* tensors, const int64_t* lens,
                                int n_layers, const adapt_grid* wl_fl_grid, int n_bins,
                                double* kld_out, int64_t* zeros_out, int32_t* best_out,
                                int32_t* const* codes_out, const adapt_search_opts* opts);

/* adapt_precision_switch_host with packed codes: codes_out[l] is HOST int8[lens[l]]
 * (code_bits 8), int16[...] (16) or int32[...] (32).  The codes leave the device slice
 * by slice (about 64 MB of input each), every slice's download overlapping the next
 * slice's kernel, so the narrower the codes the shorter the call.  A layer whose
 * selected WL exceeds code_bits gets no codes (its buffer is left as it was) and, when
 * unfit_out is given (HOST int32[n_layers]), unfit_out[l] = WL; the other entries are 0.
 * (Algorithm 1: the Quantize of every layer after the switch.)  Synchronous. */
int adapt_precision_switch_host_packed(const float* const* tensors, const int64_t* lens,
                                       int n_layers, const adapt_grid* wl_fl_grid, int n_bins,
                                       double* kld_out, int64_t* zeros_out, int32_t* best_out,
                                       int code_bits, void* const* codes_out, int32_t* unfit_out,
                                       const adapt_search_opts* opts);

/* Host-buffer form of adapt_quantize_ex: x and codes_out are HOST memory;
 * synchronous. */
int adapt_quantize_host(const float* x, int64_t n, int wl, int fl, int round_mode,
                        uint64_t seed, int32_t layer, int code_bits, void* codes_out);

/* Number of kernels the library has launched since it was loaded (all
 * devices, all entry points). */
uint64_t adapt_kernel_launch_count(void);

/* Kernel kinds for the timing calls below. */
enum {
  ADAPT_KERNEL_RANGE = 0,          /* range scan                               */
  ADAPT_KERNEL_RANGE_FINALIZE = 1, /* per-layer bin origin / scale             */
  ADAPT_KERNEL_SEARCH = 2,         /* fused quantize / zero count / histograms,
                                      keyed form (one pass, one atomic/element) */
  ADAPT_KERNEL_KLD = 3,            /* divergence per (layer, candidate)        */
  ADAPT_KERNEL_SELECT = 4,         /* lowest <WL,FL> per layer                 */
  ADAPT_KERNEL_QUANTIZE = 5,       /* stand-alone quantize                     */
  ADAPT_KERNEL_PLAN = 6,           /* per-layer cell plan of the keyed form    */
  ADAPT_KERNEL_EXPAND = 7,         /* cell counts -> per-level histograms      */
  ADAPT_KERNEL_SEARCH_DIRECT = 8,  /* fused kernel, direct form (every FL
                                      evaluated per element)                   */
  ADAPT_KERNEL_DIVERSITY = 9,      /* gradient-diversity reduction              */
  ADAPT_KERNEL_FORMAT_RESOLVE = 10,/* format search: per-layer scales and clamps */
  ADAPT_KERNEL_FORMAT_SEARCH = 11, /* format search: fused round / count / histograms */
  ADAPT_KERNEL_FORMAT_KLD = 12,    /* format search: divergence per (layer, format) */
  ADAPT_KERNEL_FORMAT_QUANTIZE = 13, /* stand-alone quantize to a format         */
  ADAPT_KERNEL_KINDS = 14
};

/* Switches per-kernel device timing on (non-zero) or off.  While on, every
 * launch is bracketed by two CUDA events on the stream it is launched on. */
int adapt_kernel_timing(int enable);

/* Waits for the timed launches recorded so far and returns, per kernel kind,
 * the accumulated device time in milliseconds and the number of launches.
 *   ms_out, launches_out  HOST arrays of ADAPT_KERNEL_KINDS entries (or NULL)
 *   reset                 non-zero clears the accumulators after reading */
int adapt_kernel_times(double* ms_out, uint64_t* launches_out, int reset);

/* Limits of adapt_precision_search_static. */
#define ADAPT_STATIC_MAX_LAYERS 8
#define ADAPT_STATIC_MAX_BINS 512
#define ADAPT_STATIC_MAX_CAND 1024

/* The search for callers that must not allocate.  (The paper has no
 * counterpart: this entry point exists for the way the library is embedded,
 * not for the method.)
 *
 * Some hosts of this library cannot let it call cudaMalloc: a training process
 * that has handed all device memory to its own pool, so that a late cudaMalloc
 * fails or eats into that pool's head-room; a service with a fixed memory
 * budget that is audited at start-up; a step loop in which the implicit
 * device-wide synchronisation of cudaMalloc / cudaFree would stall every other
 * stream.  The other search calls either grow a library-owned buffer or need a
 * caller workspace sized by a query; this one needs neither.
 *
 * It computes exactly what adapt_precision_search computes (round-to-nearest-
 * even, eps 0, bits; same argument meaning, same outputs, same flags), using
 * the direct form of the fused kernel, with all scratch in one fixed array
 * that is part of the library image: about 0.6 MB of device memory on every
 * GPU that loads the library, held until the process exits.  It calls no
 * cudaMalloc, cudaMallocHost, cudaFree or other allocating routine and creates
 * no events or streams.
 *
 *   stream  cudaStream_t or NULL (legacy default stream); kernels and the two
 *           small copies are enqueued there, results are valid after it syncs.
 * Sizes beyond the fixed scratch - more than ADAPT_STATIC_MAX_LAYERS layers,
 * ADAPT_STATIC_MAX_CAND candidates or ADAPT_STATIC_MAX_BINS bins - return
 * ADAPT_ERR_WORKSPACE before anything is launched, with the limits spelled out
 * in adapt_last_error().  Layer lengths are not limited (below 2^32 each).
 *
 * The first call on a device looks up the scratch array's device address
 * (cudaGetSymbolAddress, with that device current) and keeps it; make that
 * first call before any stream capture begins.  Every call copies a small
 * descriptor block from ordinary (pageable) host memory of the library, so the
 * host may wait inside the call for earlier work of that stream, and the call
 * must not be issued on a stream that is being captured: it then returns
 * ADAPT_ERR_INVALID_ARG without enqueuing anything.
 * Every call uses the same array and clears the parts that must start at zero,
 * so calls that can overlap on the GPU (different streams, different host
 * threads) race with each other: issue them on one stream or order them with
 * events. */
int adapt_precision_search_static(const float* const* tensors, const int64_t* lens,
                                  int n_layers, const adapt_grid* wl_fl_grid, int n_bins,
                                  double* kld_out, int64_t* zeros_out, int32_t* best_out,
                                  void* stream);

/* ---- other number formats ---------------------------------------------------
 *
 * The same search (Quantize -> zero count -> histogram over the layer's shared
 * bins -> KL(P||Q) -> choice; Sec. 3.3, Algorithm 3) over candidate formats of
 * three kinds, which may be mixed in one list:
 *   ADAPT_FMT_FIXED  a = WL, b = FL: fixed point as everywhere else in this file.
 *   ADAPT_FMT_BFP    a = WL (2..32), b ignored: block floating point (Sec. 2.1
 *       "Block-Floating-Point Quantization") with the layer as the block.  A WL-bit
 *       signed integer code and a scale s shared by the layer, value = code * 2^-s,
 *       s from the layer's extremes by the rule of Sec. 2.2:
 *       s = floor(log2(min((UB+0.5)/X_max, (LB-0.5)/X_min))), UB = 2^(WL-1)-1,
 *       LB = -2^(WL-1); evaluated exactly as the largest s with X_max*2^s <= UB+0.5
 *       and |X_min|*2^s <= |LB|+0.5.  An extreme that is zero or of the other sign
 *       sets no limit; an all-zero layer gets s = 0; s is kept within [-100, 100].
 *   ADAPT_FMT_FLOAT  a = E exponent bits (2..8), b = M fraction bits (1..23):
 *       floating point (Sec. 7 names it as the extension of the method), IEEE-like:
 *       bias 2^(E-1)-1, all-ones exponent reserved, gradual underflow; a value
 *       beyond the largest finite one, (2-2^-M)*2^bias, saturates to it.  <5,10> is
 *       half precision, <8,7> bfloat16, <8,23> the identity.
 * Rounding is opts->round_mode: to nearest even, or the SR(x) rule applied on the
 * element's local grid, with the same per-element P as everywhere else. */
enum { ADAPT_FMT_FIXED = 0, ADAPT_FMT_BFP = 1, ADAPT_FMT_FLOAT = 2 };
typedef struct { int32_t kind, a, b; } adapt_format;

#define ADAPT_MAX_FORMATS 1024

/* Bytes of workspace adapt_format_search needs for these sizes (0 if invalid). */
size_t adapt_format_search_workspace_bytes(const int64_t* lens, int n_layers,
                                           const adapt_format* formats, int n_formats,
                                           int n_bins);

/* Evaluates every format of the list on every layer and chooses one per layer.
 *   tensors, lens, n_layers   as adapt_precision_search (HOST array of DEVICE pointers)
 *   formats      HOST array of n_formats (1..ADAPT_MAX_FORMATS) candidates, listed
 *                from cheapest to most expensive: the choice is the FIRST format
 *                with KLD <= eps, else the format of least divergence (first among
 *                ties; the last one if every divergence is +inf)
 *   n_bins       1..16384, the same for every layer
 *   kld_out      DEVICE double[n_layers * n_formats]
 *   zeros_out    DEVICE int64[n_layers * n_formats]: elements whose value in the
 *                format is zero
 *   b_out        DEVICE int32[n_layers * n_formats] or NULL: b as used - the layer's
 *                scale s for ADAPT_FMT_BFP, the given b otherwise
 *   best_out     DEVICE int32[n_layers * 4] = {a, b as used, index in formats, flags}
 *   opts         HOST, may be NULL (round to nearest even, eps 0, bits).  Used:
 *                round_mode, layer_base, seed, eps, pseudo_count, log_base, stream,
 *                workspace, workspace_bytes, range_out, status_out, hist_out (DEVICE, optional:
 *                uint32[n_layers][n_formats+1][n_bins], slot 0 = histogram of the float
 *                tensor, slot c+1 = histogram of format c's values).  n_bins_per_layer
 *                and start_wl_fl must be NULL and algorithm 0: ADAPT_ERR_INVALID_ARG
 *                otherwise.
 * Errors as for adapt_precision_search. */
int adapt_format_search(const float* const* tensors, const int64_t* lens, int n_layers,
                        const adapt_format* formats, int n_formats, int n_bins,
                        double* kld_out, int64_t* zeros_out, int32_t* b_out,
                        int32_t* best_out, const adapt_search_opts* opts);

/* Quantize(L, format): maps x[0..n) to the representable values of one format.
 *   x           DEVICE float[n]
 *   kind, a, b  the format; for ADAPT_FMT_BFP b is the scale s (as b_out / best_out
 *               of adapt_format_search report it), -100 <= s <= 100
 *   layer       hash layer id for stochastic rounding
 *   values_out  DEVICE float[n]: the values (code * 2^-b, or the <E,M> value)
 *   stream      cudaStream_t or NULL */
int adapt_format_quantize(const float* x, int64_t n, int kind, int a, int b, int round_mode,
                          uint64_t seed, int layer, float* values_out, void* stream);

/* The bounds-checking build of the library (libadapt_b200_check.so, made by
 * `python -m paper_2107_13490_b200.build --check`; the stand-in for a memory checker
 * where none can be run).  In it every table index that the kernels form from
 * the data - cell positions taken from float bit patterns, bins, sub-cells, queue
 * slots - is tested against its table's size; an index outside is skipped (never
 * dereferenced, nothing traps) and the first such event is kept in a device word.
 *   out  HOST uint32[4] or NULL: {events since the library was loaded or the word
 *        was last cleared, site number of the first event, its index, its limit}
 *   clear non-zero resets the word after reading
 * Returns 1 in the bounds-checking build, 0 in the normal build (out is then all
 * zero), a negative adapt_status on a CUDA error.  Synchronises the device. */
int adapt_bounds_check_status(uint32_t* out, int clear);

/* Frees every library-owned device and pinned buffer of the current device's
 * caches.  Safe to call at any time no library work is in flight. */
int adapt_release(void);

#ifdef __cplusplus
}
#endif
#endif /* ADAPT_B200_H_ */
