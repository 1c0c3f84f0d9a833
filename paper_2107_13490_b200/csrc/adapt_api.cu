// C-ABI entry points of libadapt_b200.so: argument checks, workspace layout,
// kernel launches.  Declarations and argument contracts live in adapt.h.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <numeric>
#include <vector>

#include "../../include/adapt.h"
#include "common.cuh"
#include "k_diversity.cuh"
#include "k_expand.cuh"
#include "k_formats.cuh"
#include "k_kld_select.cuh"
#include "k_plan.cuh"
#include "k_quantize.cuh"
#include "k_range.cuh"
#include "k_search_direct.cuh"
#include "k_search_keyed.cuh"
#include "k_search_sr.cuh"

namespace {

using namespace adapt;

std::mutex g_mutex;                     // serialises calls that touch library-owned state
std::atomic<uint64_t> g_launches{0};
thread_local char g_last_error[512] = "";   // per calling thread

// Optional per-kernel device timing: events around each launch, on its stream.
struct TimedLaunch { int kind; cudaEvent_t start, stop; };
std::atomic<bool> g_timing{false};
std::mutex g_timing_mutex;
std::vector<TimedLaunch> g_pending;
std::vector<cudaEvent_t> g_event_pool;
double g_kind_ms[ADAPT_KERNEL_KINDS] = {0};
uint64_t g_kind_launches[ADAPT_KERNEL_KINDS] = {0};

cudaEvent_t pooled_event() {
  if (!g_event_pool.empty()) { cudaEvent_t e = g_event_pool.back(); g_event_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

// Brackets one kernel launch; counts it, and times it when timing is on.
struct LaunchScope {
  int kind; cudaStream_t stream; cudaEvent_t start = nullptr;
  LaunchScope(int k, cudaStream_t s) : kind(k), stream(s) {
    if (g_timing.load()) {
      std::lock_guard<std::mutex> l(g_timing_mutex);
      start = pooled_event();
      if (start) cudaEventRecord(start, stream);
    }
  }
  ~LaunchScope() {
    ++g_launches;
    if (start) {
      std::lock_guard<std::mutex> l(g_timing_mutex);
      cudaEvent_t stop = pooled_event();
      if (stop) { cudaEventRecord(stop, stream); g_pending.push_back({kind, start, stop}); }
    }
  }
};

int cuda_fail(cudaError_t e, const char* what) {
  std::snprintf(g_last_error, sizeof(g_last_error), "%s: %s", what, cudaGetErrorString(e));
  return ADAPT_ERR_CUDA;
}
#define ADAPT_CUDA(call)                                     \
  do {                                                       \
    cudaError_t e_ = (call);                                 \
    if (e_ != cudaSuccess) return cuda_fail(e_, #call);      \
  } while (0)

// after a kernel launch: report which launch was refused
#define ADAPT_LAUNCH_OK(what)                                \
  do {                                                       \
    cudaError_t e_ = cudaGetLastError();                     \
    if (e_ != cudaSuccess) return cuda_fail(e_, what);       \
  } while (0)

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---- per-device caches --------------------------------------------------------

constexpr int kMaxDevices = 64;
constexpr int kRingSlots = 4;

struct PinnedSlot {
  void* host = nullptr;
  size_t bytes = 0;
  cudaEvent_t done = nullptr;
};

struct DeviceCache {
  bool props_ready = false;
  int sm_count = 0;
  int max_smem_optin = 0;
  void* workspace = nullptr;   size_t workspace_bytes = 0;
  void* stage_in = nullptr;    size_t stage_in_bytes = 0;    // host-form calls: inputs
  void* stage_out = nullptr;   size_t stage_out_bytes = 0;   // host-form calls: outputs
  void* batch_tab = nullptr;   size_t batch_tab_bytes = 0;   // batched quantize: layer table
  std::vector<unsigned char> batch_tab_image;   // host copy of what batch_tab holds (empty: unknown)
  cudaStream_t batch_tab_stream = nullptr;      // the stream that uploaded it
  void* stage_codes = nullptr; size_t stage_codes_bytes = 0; // host-form calls: codes
  void* div_buf = nullptr;     size_t div_buf_bytes = 0;     // gradient diversity: tables + sums
  PinnedSlot ring[kRingSlots];
  int ring_next = 0;
  cudaStream_t copy_stream = nullptr;   // host-form calls: downloads that overlap the kernels
  cudaEvent_t slice_done[2] = {nullptr, nullptr};
  cudaEvent_t copies_done = nullptr;
  cudaStream_t side_stream = nullptr;   // search: the direct kernel runs beside the keyed kernels
  cudaEvent_t side_fork = nullptr, side_join = nullptr;
};

DeviceCache g_cache[kMaxDevices];

int current_cache(DeviceCache** out) {
  int dev = 0;
  ADAPT_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) {
    std::snprintf(g_last_error, sizeof(g_last_error), "device index %d not supported", dev);
    return ADAPT_ERR_CUDA;
  }
  DeviceCache& c = g_cache[dev];
  if (!c.props_ready) {
    ADAPT_CUDA(cudaDeviceGetAttribute(&c.sm_count, cudaDevAttrMultiProcessorCount, dev));
    ADAPT_CUDA(cudaDeviceGetAttribute(&c.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    c.props_ready = true;
  }
  *out = &c;
  return ADAPT_OK;
}

int grow_device(void** ptr, size_t* have, size_t need) {
  if (*have >= need) return ADAPT_OK;
  if (*ptr) { ADAPT_CUDA(cudaFree(*ptr)); *ptr = nullptr; *have = 0; }
  ADAPT_CUDA(cudaMalloc(ptr, need));
  *have = need;
  return ADAPT_OK;
}

// A pinned host slot whose previous upload has finished.
int acquire_slot(DeviceCache& c, size_t bytes, PinnedSlot** out) {
  PinnedSlot& s = c.ring[c.ring_next];
  c.ring_next = (c.ring_next + 1) % kRingSlots;
  if (!s.done) ADAPT_CUDA(cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming));
  ADAPT_CUDA(cudaEventSynchronize(s.done));
  if (s.bytes < bytes) {
    if (s.host) { ADAPT_CUDA(cudaFreeHost(s.host)); s.host = nullptr; s.bytes = 0; }
    size_t want = align_up(std::max<size_t>(bytes, 16384), 4096);
    ADAPT_CUDA(cudaMallocHost(&s.host, want));
    s.bytes = want;
  }
  *out = &s;
  return ADAPT_OK;
}

// ---- search plan ----------------------------------------------------------------

constexpr int kMaxBins = 16384;
#ifndef ADAPT_D_LEVELS_MAX
#define ADAPT_D_LEVELS_MAX 0   // fine levels of the main segment whose corrections stay in shared memory
                               // (none: the table is worth more as cells; the corrections are few)
#endif
constexpr long long kKeyedMinElements = 32768;  // smaller layers take the direct kernel
#ifndef ADAPT_EXPAND_FILL
#define ADAPT_EXPAND_FILL 3    // CTAs of the expand kernel per SM, over all layers, slices and roles
#endif
constexpr int kMaxKeyedGrid = 1023;             // CTAs of the keyed kernel (one per SM) whose tile ranges fit the descriptor block
// What it costs a CTA of the keyed kernel to take up one more layer (context, table set-up, flush),
// in tiles' worth of counting: the tile ranges of the CTAs are balanced with it.
#ifndef ADAPT_LAYER_COST_TILES
#define ADAPT_LAYER_COST_TILES 6.0
#endif
constexpr double kLayerCostTiles = ADAPT_LAYER_COST_TILES;
// Stochastic rounding: the keyed route saves about 10 us per 2^20 elements over the direct kernel and
// costs three more launches, so it takes layers of 2^20 elements up, and only 2^22 of them together.
constexpr long long kSrKeyedMinElements = 1ll << 20;
constexpr long long kSrKeyedMinTotal = 1ll << 22;
constexpr int kKeyedMaxBins = 8192;
constexpr size_t kKeyedSmemBudget = 224 * 1024; // one CTA per SM owns its shared memory

struct Plan {
  int n_layers = 0, n_cand = 0, n_levels = 0, n_bins = 0;
  std::vector<int> slot, order, by_fl, fl_begin;
  // keyed-kernel shared-memory shape
  int cell_cap = 0, value_cap = 0, d_levels = 0;
  size_t keyed_smem = 0;
  // stochastic-rounding kernel's shared-memory shape
  int sr_cap = 0, sr_d_levels = 0;
  size_t sr_smem = 0;
  // byte offsets inside the workspace -- descriptor block (uploaded)
  size_t off_layers = 0, off_keyed = 0, off_direct = 0, off_wl = 0, off_fl = 0, off_slot = 0,
         off_order = 0, off_by_fl = 0, off_fl_begin = 0, off_start = 0, off_cta = 0, off_state = 0, blob_bytes = 0;
  // written by kernels, not cleared
  size_t off_plan = 0, off_edges = 0;
  // accumulators (cleared every call)
  size_t off_coarse = 0, off_sub = 0, off_zeros = 0, off_q = 0, off_u = 0, off_cells = 0, off_qe = 0,
         off_zclass = 0, off_nzero = 0, accum_begin = 0, accum_bytes = 0;
  size_t total = 0;
};

static_assert(ADAPT_ERR_NONFINITE == 2 && ADAPT_ERR_RANGE == 3, "the kernels write these codes into status_out");

bool valid_format(int wl, int fl) { return wl >= 2 && wl <= 32 && fl >= 0 && fl < wl; }

// Validates sizes and fills the layout.  Returns false on invalid arguments.
bool make_plan(const int64_t* lens, int n_layers, const adapt_grid* grid, int n_bins, Plan* p) {
  if (!lens || !grid || !grid->wl || !grid->fl) return false;
  if (n_layers < 1 || n_layers > 65535) return false;
  if (grid->n_cand < 1 || grid->n_cand > 65535) return false;
  if (n_bins < 1 || n_bins > kMaxBins) return false;
  int fmax = 0;
  for (int c = 0; c < grid->n_cand; ++c) {
    if (!valid_format(grid->wl[c], grid->fl[c])) return false;
    fmax = std::max(fmax, grid->fl[c]);
  }
  for (int l = 0; l < n_layers; ++l)
    if (lens[l] < 0 || lens[l] >= (1ll << 32)) return false;
  p->n_layers = n_layers; p->n_cand = grid->n_cand; p->n_bins = n_bins;
  p->n_levels = fmax + 1;   // fraction lengths 0..fmax get a histogram each

  p->slot.assign(grid->fl, grid->fl + grid->n_cand);
  p->order.resize(grid->n_cand);
  std::iota(p->order.begin(), p->order.end(), 0);
  std::stable_sort(p->order.begin(), p->order.end(), [&](int a, int b) {
    if (grid->wl[a] != grid->wl[b]) return grid->wl[a] < grid->wl[b];
    return grid->fl[a] < grid->fl[b];
  });

  p->by_fl.resize(grid->n_cand);
  std::iota(p->by_fl.begin(), p->by_fl.end(), 0);
  std::stable_sort(p->by_fl.begin(), p->by_fl.end(),
                   [&](int a, int b) { return grid->fl[a] < grid->fl[b]; });
  p->fl_begin.assign(p->n_levels + 1, 0);
  for (int c = 0; c < grid->n_cand; ++c) p->fl_begin[grid->fl[c] + 1] += 1;
  for (int f = 0; f < p->n_levels; ++f) p->fl_begin[f + 1] += p->fl_begin[f];

  // shared-memory shape of the keyed kernel: queue + bin edges + Qe + a few correction levels + cells
  const size_t hist = sizeof(unsigned) * n_bins;
  const size_t queue = keyed_smem_bytes(0, 0, 0);
  p->d_levels = static_cast<int>(std::min<size_t>(ADAPT_D_LEVELS_MAX, (32 * 1024) / hist));
  p->d_levels = std::min(p->d_levels, p->n_levels);
  if (n_bins <= kKeyedMaxBins) {
    p->cell_cap = static_cast<int>((kKeyedSmemBudget - queue - hist * (2 + p->d_levels)) / 4) - 64;
    p->cell_cap = std::min(p->cell_cap, 1 << 16) & ~3;   // rows of the cell arrays stay 16-byte aligned
  } else {
    p->cell_cap = 0;
  }
  p->keyed_smem = keyed_smem_bytes(p->cell_cap, n_bins, p->d_levels);
  p->value_cap = p->cell_cap ? keyed_value_cap(p->cell_cap, n_bins, p->d_levels) : 0;
  if (n_bins <= kKeyedMaxBins) {
    p->sr_d_levels = std::min(static_cast<int>(std::min<size_t>(4, (16 * 1024) / hist)), p->n_levels);
    const size_t fixed = sr_smem_bytes(0, n_bins, p->sr_d_levels);
    // (the kernel's static tables - lane-private counters of the central values - take 13 KB more)
    p->sr_cap = static_cast<int>((kKeyedSmemBudget - 14 * 1024 - fixed) / 8) & ~3;
    p->sr_cap = std::min(p->sr_cap, p->value_cap);      // rows of the global tables are value_cap long
    p->sr_smem = sr_smem_bytes(p->sr_cap, n_bins, p->sr_d_levels);
  }

  // K: row length of the global cell arrays (the largest table a layer may use)
  const size_t C = grid->n_cand, L = n_layers, B = n_bins, F = p->n_levels, K = p->value_cap;
  size_t o = 0;
  p->off_layers = o;  o = align_up(o + sizeof(LayerDesc) * (L + 1), 16);
  p->off_keyed = o;   o = align_up(o + sizeof(LayerDesc) * (L + 1), 16);
  p->off_direct = o;  o = align_up(o + sizeof(LayerDesc) * (L + 1), 16);
  p->off_wl = o;      o = align_up(o + sizeof(int) * C, 16);
  p->off_fl = o;      o = align_up(o + sizeof(int) * C, 16);
  p->off_slot = o;    o = align_up(o + sizeof(int) * C, 16);
  p->off_order = o;   o = align_up(o + sizeof(int) * C, 16);
  p->off_by_fl = o;   o = align_up(o + sizeof(int) * C, 16);
  p->off_fl_begin = o; o = align_up(o + sizeof(int) * (F + 1), 16);
  p->off_start = o;   o = align_up(o + sizeof(int) * 2 * L, 16);
  p->off_cta = o;     o = align_up(o + sizeof(long long) * (kMaxKeyedGrid + 1), 16);
  p->off_state = o;   o = align_up(o + sizeof(LayerState) * L, 256);
  p->blob_bytes = o;
  p->off_plan = o;      o = align_up(o + sizeof(LayerPlan) * L, 256);
  p->off_edges = o;     o = align_up(o + sizeof(float) * L * (B + 1), 256);
  p->accum_begin = o;
  p->off_zeros = o;   o = align_up(o + sizeof(unsigned long long) * L * F, 256);
  p->off_zclass = o;  o = align_up(o + sizeof(unsigned long long) * L * kZeroClasses, 256);
  p->off_nzero = o;   o = align_up(o + sizeof(unsigned long long) * L, 256);
  p->off_q = o;       o = align_up(o + sizeof(unsigned) * L * B, 256);
  p->off_qe = o;      o = align_up(o + sizeof(unsigned) * L * B * 2, 256);
  p->off_cells = o;   o = align_up(o + sizeof(unsigned) * L * K, 256);
  p->off_coarse = o;  o = align_up(o + sizeof(unsigned) * L * K, 256);
  p->off_sub = o;     o = align_up(o + sizeof(unsigned) * (K ? L * 2 * B * kSubCells : 0), 256);
  p->off_u = o;       o = align_up(o + sizeof(unsigned) * L * F * B, 256);
  p->accum_bytes = o - p->accum_begin;
  p->total = o;
  return true;
}

}  // namespace

// Launch of a kernel that follows another kernel of this library in the stream and begins with
// grid_dependency_wait(): with programmatic stream serialization its CTAs may be scheduled while
// the earlier kernel's last CTAs are still running, which hides the launch latency between the
// dependent kernels of a search.  (Not while per-kernel events are recorded between them.)
template <typename... Params, typename... Args>
cudaError_t launch_dependent(void (*kern)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                             Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = g_timing.load() ? 0 : 1;
  return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// ---- search driver ----------------------------------------------------------------

namespace {

// Grid of the range scan, and for every layer of its list the number of CTAs that hold tiles of
// the layer (each CTA walks a contiguous slice of `per` tiles; the last CTA of a layer to finish
// settles it).  list: n_layers descriptors + sentinel, tile_begin filled in.
int plan_range_grid(LayerDesc* list, int n_layers, long long tiles, int sm_count) {
  const int grid = static_cast<int>(std::max<long long>(1, std::min<long long>(tiles, 16ll * sm_count)));
  const long long per = (tiles + grid - 1) / grid;
  for (int k = 0; k < n_layers; ++k) {
    const long long b = list[k].tile_begin, e = list[k + 1].tile_begin;
    list[k].range_ctas = (e > b && per > 0) ? static_cast<int>((e - 1) / per - b / per + 1) : 0;
  }
  return grid;
}

struct SearchArgs {
  const float* const* tensors;  // host array of device pointers
  const int64_t* lens;
  int n_layers;
  const adapt_grid* grid;
  int n_bins;
  double* kld_out;
  int64_t* zeros_out;
  int32_t* best_out;
  adapt_search_opts opts;
};

adapt_search_opts default_opts() {
  adapt_search_opts o;
  std::memset(&o, 0, sizeof(o));
  return o;
}

// Fills a layer list (descriptors + sentinel) from the chosen layers; returns its tile count.
long long fill_list(LayerDesc* out, const std::vector<int>& pick, const SearchArgs& a,
                    int tile) {
  long long tiles = 0;
  size_t k = 0;
  for (int l : pick) {
    const int mis = static_cast<int>((reinterpret_cast<uintptr_t>(a.tensors[l]) >> 2) & 3u);
    LayerDesc& d = out[k++];
    d.ptr = a.tensors[l];
    d.n = a.lens[l];
    d.tile_begin = tiles;
    d.mis = a.lens[l] > 0 ? mis : 0;
    d.layer_id = a.opts.layer_base + l;
    d.index = l;
    d.n_bins = a.opts.n_bins_per_layer ? a.opts.n_bins_per_layer[l] : a.n_bins;
    d.range_ctas = 0; d.via_plan = 0; d.pad_ = 0;
    if (a.lens[l] > 0) tiles += (a.lens[l] + mis + tile - 1) / tile;
  }
  LayerDesc& s = out[k];
  s.ptr = nullptr; s.n = 0; s.tile_begin = tiles; s.mis = 0; s.layer_id = 0; s.index = 0; s.n_bins = 1;
  s.range_ctas = 0; s.via_plan = 0; s.pad_ = 0;
  return tiles;
}

// Contiguous tile ranges for the CTAs of the keyed kernel, balanced by cost: a tile costs 1, and
// every layer a CTA touches costs kLayerCostTiles more (so CTAs in a stretch of small layers get
// fewer tiles).  list: the keyed layer list with its sentinel; out: grid + 1 first tiles.  The
// smallest per-CTA budget under which a greedy walk places all tiles is found by bisection.
void balance_keyed_ctas(const LayerDesc* list, int n_layers, long long tiles, int grid, long long* out) {
  auto walk = [&](double budget, long long* begin) {
    int k = 0;
    long long t = 0;
    for (int cta = 0; cta < grid; ++cta) {
      if (begin) begin[cta] = t;
      double load = 0.0;
      while (t < tiles) {
        while (k < n_layers && list[k + 1].tile_begin <= t) ++k;
        if (load > 0.0 && load + kLayerCostTiles + 1.0 > budget) break;
        load += kLayerCostTiles;
        const long long left = list[k + 1].tile_begin - t;
        const long long take = std::max<long long>(1, std::min<long long>(left, static_cast<long long>(budget - load)));
        t += take;
        load += static_cast<double>(take);
        if (take < left) break;
      }
    }
    if (begin) begin[grid] = tiles;
    return t >= tiles;
  };
  double lo = static_cast<double>(tiles) / grid, hi = static_cast<double>(tiles) + kLayerCostTiles * (n_layers + 1) + 1.0;
  for (int it = 0; it < 40 && hi - lo > 0.25; ++it) {
    const double mid = 0.5 * (lo + hi);
    if (walk(mid, nullptr)) hi = mid; else lo = mid;
  }
  walk(hi, out);
}

// Enqueues the whole search on opts.stream.  Caller holds g_mutex.
int run_search(DeviceCache& dc, const SearchArgs& a) {
  const adapt_search_opts& o = a.opts;
  if (!a.tensors || !a.kld_out || !a.zeros_out || !a.best_out) return ADAPT_ERR_INVALID_ARG;
  if (o.round_mode != ADAPT_ROUND_RNE && o.round_mode != ADAPT_ROUND_STOCHASTIC)
    return ADAPT_ERR_INVALID_ARG;
  if (!(o.eps >= 0.0) || !(o.pseudo_count >= 0.0)) return ADAPT_ERR_INVALID_ARG;
  const double base = (o.log_base == 0.0) ? 2.0 : o.log_base;
  if (!(base > 0.0) || base == 1.0 || !std::isfinite(base)) return ADAPT_ERR_INVALID_ARG;

  // per-layer resolutions: the arrays are laid out with the largest one as their stride
  int bins_stride = a.n_bins;
  if (o.n_bins_per_layer) {
    if (a.n_layers < 1) return ADAPT_ERR_INVALID_ARG;
    bins_stride = 0;
    for (int l = 0; l < a.n_layers; ++l) {
      if (o.n_bins_per_layer[l] < 1 || o.n_bins_per_layer[l] > kMaxBins) return ADAPT_ERR_INVALID_ARG;
      bins_stride = std::max(bins_stride, o.n_bins_per_layer[l]);
    }
  }
  Plan plan;
  if (!make_plan(a.lens, a.n_layers, a.grid, bins_stride, &plan)) return ADAPT_ERR_INVALID_ARG;
  for (int l = 0; l < a.n_layers; ++l) {
    if (a.lens[l] > 0 && !a.tensors[l]) return ADAPT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(a.tensors[l]) & 3u) return ADAPT_ERR_INVALID_ARG;
  }

  char* ws = nullptr;
  if (o.workspace) {
    if (reinterpret_cast<uintptr_t>(o.workspace) & 255u) return ADAPT_ERR_INVALID_ARG;
    if (o.workspace_bytes < plan.total) return ADAPT_ERR_WORKSPACE;
    ws = static_cast<char*>(o.workspace);
  } else {
    int rc = grow_device(&dc.workspace, &dc.workspace_bytes, plan.total);
    if (rc != ADAPT_OK) return rc;
    ws = static_cast<char*>(dc.workspace);
  }
  cudaStream_t stream = static_cast<cudaStream_t>(o.stream);

  // which kernel serves which layer
  if (o.algorithm != ADAPT_ALGO_AUTO && o.algorithm != ADAPT_ALGO_KEYED &&
      o.algorithm != ADAPT_ALGO_DIRECT) return ADAPT_ERR_INVALID_ARG;
  const bool stochastic = o.round_mode == ADAPT_ROUND_STOCHASTIC;
  const bool keyed_possible =
      (o.algorithm == ADAPT_ALGO_AUTO || o.algorithm == ADAPT_ALGO_KEYED) &&
      (stochastic ? (plan.sr_cap >= 2048 && plan.sr_smem + 15 * 1024 <= static_cast<size_t>(dc.max_smem_optin))
                  : (plan.cell_cap >= 1024 && plan.keyed_smem + 2048 <= static_cast<size_t>(dc.max_smem_optin)));
  const long long keyed_min = (o.algorithm == ADAPT_ALGO_KEYED) ? 1
                              : stochastic ? kSrKeyedMinElements : kKeyedMinElements;
  std::vector<int> all(a.n_layers), keyed, direct;
  std::iota(all.begin(), all.end(), 0);
  bool keyed_pays = keyed_possible;
  if (stochastic && o.algorithm == ADAPT_ALGO_AUTO) {
    long long total = 0;
    for (int l = 0; l < a.n_layers; ++l) total += a.lens[l] >= keyed_min ? a.lens[l] : 0;
    keyed_pays = keyed_pays && total >= kSrKeyedMinTotal;
  }
  for (int l = 0; l < a.n_layers; ++l) {
    const bool k = keyed_pays && a.lens[l] >= keyed_min;
    if (k) keyed.push_back(l);
    // Stochastic rounding: whether the keyed kernel can serve a layer is only known on the
    // device (its cell indices must be exact in a float), so its layers also stand in the
    // direct kernel's list, which skips those whose plan says "keyed"
    if (!k || stochastic) direct.push_back(l);
  }

  // host image of the descriptor block
  PinnedSlot* slot = nullptr;
  int rc = acquire_slot(dc, plan.blob_bytes, &slot);
  if (rc != ADAPT_OK) return rc;
  char* h = static_cast<char*>(slot->host);
  std::memset(h, 0, plan.blob_bytes);
  const long long tiles = fill_list(reinterpret_cast<LayerDesc*>(h + plan.off_layers), all, a, kTile);
  const int range_grid = plan_range_grid(reinterpret_cast<LayerDesc*>(h + plan.off_layers), a.n_layers, tiles, dc.sm_count);
  const long long keyed_tiles = fill_list(reinterpret_cast<LayerDesc*>(h + plan.off_keyed), keyed, a,
                                          stochastic ? kSrTile : kKeyedTile);
  const long long direct_tiles = fill_list(reinterpret_cast<LayerDesc*>(h + plan.off_direct), direct, a, kTile);
  if (stochastic && !keyed.empty()) {
    LayerDesc* dl = reinterpret_cast<LayerDesc*>(h + plan.off_direct);
    size_t k = 0;
    for (size_t i = 0; i < direct.size(); ++i) {
      while (k < keyed.size() && keyed[k] < direct[i]) ++k;
      if (k < keyed.size() && keyed[k] == direct[i]) dl[i].via_plan = 1;
    }
  }
  const int keyed_grid = static_cast<int>(std::max<long long>(
      1, std::min<long long>(keyed_tiles, std::min(dc.sm_count, kMaxKeyedGrid))));
  if (!stochastic && keyed_tiles > 0)
    balance_keyed_ctas(reinterpret_cast<const LayerDesc*>(h + plan.off_keyed), static_cast<int>(keyed.size()),
                       keyed_tiles, keyed_grid, reinterpret_cast<long long*>(h + plan.off_cta));
  std::memcpy(h + plan.off_wl, a.grid->wl, sizeof(int) * plan.n_cand);
  std::memcpy(h + plan.off_fl, a.grid->fl, sizeof(int) * plan.n_cand);
  std::memcpy(h + plan.off_slot, plan.slot.data(), sizeof(int) * plan.n_cand);
  std::memcpy(h + plan.off_order, plan.order.data(), sizeof(int) * plan.n_cand);
  std::memcpy(h + plan.off_by_fl, plan.by_fl.data(), sizeof(int) * plan.n_cand);
  std::memcpy(h + plan.off_fl_begin, plan.fl_begin.data(), sizeof(int) * (plan.n_levels + 1));
  if (o.start_wl_fl) std::memcpy(h + plan.off_start, o.start_wl_fl, sizeof(int) * 2 * a.n_layers);
  LayerState* hs = reinterpret_cast<LayerState*>(h + plan.off_state);
  for (int l = 0; l < a.n_layers; ++l) { hs[l].min_key = 0xFFFFFFFFu; hs[l].max_key = 0u; }

  ADAPT_CUDA(cudaMemcpyAsync(ws, h, plan.blob_bytes, cudaMemcpyHostToDevice, stream));
  ADAPT_CUDA(cudaEventRecord(slot->done, stream));

  const LayerDesc* d_layers = reinterpret_cast<const LayerDesc*>(ws + plan.off_layers);
  const LayerDesc* d_keyed = reinterpret_cast<const LayerDesc*>(ws + plan.off_keyed);
  const LayerDesc* d_direct = reinterpret_cast<const LayerDesc*>(ws + plan.off_direct);
  LayerState* d_state = reinterpret_cast<LayerState*>(ws + plan.off_state);
  LayerPlan* d_plan = reinterpret_cast<LayerPlan*>(ws + plan.off_plan);
  float* d_edges = reinterpret_cast<float*>(ws + plan.off_edges);
  unsigned long long* d_zeros = reinterpret_cast<unsigned long long*>(ws + plan.off_zeros);
  unsigned long long* d_zclass = reinterpret_cast<unsigned long long*>(ws + plan.off_zclass);
  unsigned* d_q = reinterpret_cast<unsigned*>(ws + plan.off_q);
  unsigned* d_qe = reinterpret_cast<unsigned*>(ws + plan.off_qe);
  unsigned* d_cells = reinterpret_cast<unsigned*>(ws + plan.off_cells);
  unsigned* d_sub = reinterpret_cast<unsigned*>(ws + plan.off_sub);
  unsigned* d_u = reinterpret_cast<unsigned*>(ws + plan.off_u);

  ADAPT_CUDA(cudaMemsetAsync(ws + plan.accum_begin, 0, plan.accum_bytes, stream));

  // K1: range scan over every layer; its last CTA per layer derives the bin origin and scale
  {
    RangeParams rp;
    rp.layers = d_layers; rp.n_layers = a.n_layers; rp.n_tiles = tiles; rp.state = d_state;
    rp.range_out = o.range_out;
    LaunchScope ls(ADAPT_KERNEL_RANGE, stream);
    range_scan_kernel<<<range_grid, kRangeThreads, 0, stream>>>(rp);
    ADAPT_CUDA(cudaGetLastError());
  }

  // Layers of both forms in one call (round-to-nearest-even): the direct kernel needs only the
  // ranges, so it runs on a stream of the library's own beside plan -> counting -> expansion and
  // joins before the divergences.  (Under stochastic rounding it reads the plans: no overlap.)
  const bool beside = !stochastic && !keyed.empty() && keyed_tiles > 0 && !direct.empty() && direct_tiles > 0;
  cudaStream_t direct_stream = stream;

  // K2, keyed form: plan -> cell counting -> expansion
  const long long elems_per_cta = (keyed_tiles + keyed_grid - 1) / keyed_grid * kKeyedTile;
  if (!keyed.empty() && keyed_tiles > 0) {
    const int nk = static_cast<int>(keyed.size());
    {
      PlanParams pp;
      pp.layers = d_keyed; pp.state = d_state; pp.plan = d_plan; pp.edges = d_edges;
      pp.n_bins = bins_stride; pp.value_cap = plan.value_cap;
      // stochastic rounding: cells and coarse tables share the limit; a little room for the
      // three spare entries of every coarse level
      pp.stochastic = stochastic ? 1 : 0;
      pp.cell_cap = stochastic ? plan.sr_cap - 128 : plan.cell_cap;
      pp.fine_ratio = ADAPT_FINE_RATIO;
      pp.elems_per_cta = elems_per_cta;
      LaunchScope ls(ADAPT_KERNEL_PLAN, stream);
      const int plan_slices = std::max(1, std::min(8, (bins_stride + kPlanThreads - 1) / kPlanThreads));
      ADAPT_CUDA(launch_dependent(plan_kernel, dim3(nk, plan_slices), dim3(kPlanThreads), 0, stream, pp));
    }
    // (the branch comes after the plan kernel so that nothing stands between the range scan and it)
    if (beside) {
      if (!dc.side_stream) {
        ADAPT_CUDA(cudaStreamCreateWithFlags(&dc.side_stream, cudaStreamNonBlocking));
        ADAPT_CUDA(cudaEventCreateWithFlags(&dc.side_fork, cudaEventDisableTiming));
        ADAPT_CUDA(cudaEventCreateWithFlags(&dc.side_join, cudaEventDisableTiming));
      }
      ADAPT_CUDA(cudaEventRecord(dc.side_fork, stream));
      ADAPT_CUDA(cudaStreamWaitEvent(dc.side_stream, dc.side_fork, 0));
      direct_stream = dc.side_stream;
    }
    if (stochastic) {
      SrParams sp;
      sp.layers = d_keyed; sp.n_layers = nk; sp.n_tiles = keyed_tiles; sp.state = d_state;
      sp.plan = d_plan; sp.edges = d_edges; sp.cell_count = d_cells;
      sp.coarse_count = reinterpret_cast<unsigned*>(ws + plan.off_coarse);
      sp.qe_hist = d_qe; sp.u_hist = d_u; sp.zeros = d_zeros;
      sp.cell_total = reinterpret_cast<unsigned long long*>(ws + plan.off_nzero);
      sp.seed = o.seed; sp.n_bins = bins_stride; sp.n_levels = plan.n_levels;
      sp.table_cap = plan.sr_cap; sp.cell_stride = plan.value_cap; sp.d_levels = plan.sr_d_levels;
      ADAPT_CUDA(cudaFuncSetAttribute(search_sr_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      static_cast<int>(plan.sr_smem)));
      {
        LaunchScope ls(ADAPT_KERNEL_SEARCH, stream);
        ADAPT_CUDA(launch_dependent(search_sr_kernel, dim3(keyed_grid), dim3(kSrThreads), plan.sr_smem, stream, sp));
      }
      SrExpandParams ep;
      ep.layers = d_keyed; ep.state = d_state; ep.plan = d_plan; ep.cell_count = d_cells;
      ep.coarse_count = sp.coarse_count; ep.qe_hist = d_qe; ep.cell_total = sp.cell_total;
      ep.q_hist = d_q; ep.u_hist = d_u; ep.zeros = d_zeros;
      ep.n_bins = bins_stride; ep.n_levels = plan.n_levels; ep.cell_stride = plan.value_cap;
      {
        LaunchScope ls(ADAPT_KERNEL_EXPAND, stream);
        ADAPT_CUDA(launch_dependent(expand_sr_kernel, dim3(plan.n_levels + 1, nk), dim3(kSrExpandThreads),
                                    sizeof(unsigned) * bins_stride, stream, ep));
      }
    } else {
    KeyedParams kp;
    kp.layers = d_keyed; kp.n_layers = nk; kp.n_tiles = keyed_tiles; kp.state = d_state;
    kp.plan = d_plan; kp.edges = d_edges; kp.cell_count = d_cells;
    kp.qe_hist = d_qe; kp.u_hist = d_u; kp.q_hist = d_q; kp.zeros = d_zeros; kp.zero_class = d_zclass;
    kp.sub_count = d_sub;
    kp.cell_total = reinterpret_cast<unsigned long long*>(ws + plan.off_nzero);
    kp.n_bins = bins_stride; kp.n_levels = plan.n_levels;
    kp.cell_cap = plan.cell_cap; kp.cell_stride = plan.value_cap; kp.d_levels = plan.d_levels;
    kp.cta_begin = reinterpret_cast<const long long*>(ws + plan.off_cta);
    ADAPT_CUDA(cudaFuncSetAttribute(search_keyed_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(plan.keyed_smem)));
    {
      const int grid = keyed_grid;
      LaunchScope ls(ADAPT_KERNEL_SEARCH, stream);
      ADAPT_CUDA(launch_dependent(search_keyed_kernel, dim3(grid), dim3(kKeyedThreads), plan.keyed_smem, stream, kp));
    }
    ExpandParams ep;
    ep.layers = d_keyed; ep.n_layers = nk; ep.state = d_state; ep.plan = d_plan;
    ep.cell_count = d_cells; ep.qe_hist = d_qe;
    ep.sub_count = d_sub; ep.edges = d_edges;
    ep.q_hist = d_q; ep.u_hist = d_u; ep.zeros = d_zeros; ep.zero_class = d_zclass;
    ep.cell_total = reinterpret_cast<const unsigned long long*>(ws + plan.off_nzero);
    ep.n_bins = bins_stride; ep.n_levels = plan.n_levels; ep.cell_stride = plan.value_cap;
    {
      // pyramid form: enough slices (times six roles) per layer to fill the GPU, and at least as many as keep
      // a slice's cells (1.5 words each) and the fine histogram inside one CTA's shared memory
      const size_t room = static_cast<size_t>(dc.max_smem_optin) - 2048 - sizeof(unsigned) * bins_stride;
      const int cap_max = static_cast<int>(std::min<size_t>(room / 6, 1u << 20)) & ~3;
      int slices = std::max(1, std::min(32, (ADAPT_EXPAND_FILL * dc.sm_count + nk * kExpandRoles - 1) / (nk * kExpandRoles)));
      slices = std::max(slices, (plan.cell_cap + cap_max - 1) / std::max(cap_max, 4));
      ep.slices = slices;
      // the largest table a layer of the pyramid form can have: the cap its plan works with
      // (make_layer_plan: cells ~ sqrt(balance * bins * elements one CTA sees), at most cell_cap)
      long long cells_bound = 2048;
      for (int l : keyed) {
        const int bins_l = o.n_bins_per_layer ? o.n_bins_per_layer[l] : a.n_bins;
        const double seen = static_cast<double>(std::min<long long>(a.lens[l], elems_per_cta));
        const long long want = static_cast<long long>(std::sqrt(ADAPT_CELL_BALANCE * static_cast<double>(bins_l) * seen)) + 16;
        cells_bound = std::max(cells_bound, std::min<long long>(plan.cell_cap, std::max<long long>(2048, want)));
      }
      ep.slice_cap = (static_cast<int>((cells_bound + slices - 1) / slices) + 3) & ~3;
      const size_t smem = sizeof(unsigned) * (static_cast<size_t>(bins_stride) + ep.slice_cap + ep.slice_cap / 2 + 2);
      if (smem + 1024 > static_cast<size_t>(dc.max_smem_optin)) return ADAPT_ERR_INVALID_ARG;
      ADAPT_CUDA(cudaFuncSetAttribute(expand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      static_cast<int>(smem)));
      LaunchScope ls(ADAPT_KERNEL_EXPAND, stream);
      ADAPT_CUDA(launch_dependent(expand_kernel, dim3(slices * kExpandRoles, nk), dim3(kExpandThreads), smem, stream, ep));
    }
    }
  }

  // K2, direct form: stochastic rounding, small layers, very large bin counts
  if (!direct.empty() && direct_tiles > 0) {
    SearchParams sp;
    sp.layers = d_direct; sp.state = d_state;
    sp.n_layers = static_cast<int>(direct.size()); sp.n_fl = plan.n_levels; sp.n_bins = bins_stride;
    sp.n_tiles = direct_tiles;
    sp.q_hist = d_q; sp.u_hist = d_u; sp.zeros = d_zeros; sp.seed = o.seed; sp.plan = d_plan;
    const size_t per_hist = sizeof(unsigned) * bins_stride;
    // When the histograms of all fraction lengths overflow half an SM's shared memory and there
    // is work for every SM, one CTA of 1024 threads takes the whole of it: fewer FL groups (each
    // group re-reads the tensors) and twice the resident warps of two 256-thread CTAs.
    const bool wide = per_hist * (plan.n_levels + 1) > 100 * 1024 && direct_tiles >= 2ll * dc.sm_count &&
                      dc.max_smem_optin >= 200 * 1024 + 1024;
    const int threads = wide ? kSearchThreadsWide : kSearchThreads;
    const size_t budget = (wide ? 200 : 100) * 1024;
    int fg = static_cast<int>(budget / per_hist) - 1;
    fg = std::max(1, std::min(fg, plan.n_levels));
    // few tiles: spread the fraction lengths over more CTAs instead of looping over them in one
    const long long want_groups = std::min<long long>(
        plan.n_levels, std::max<long long>(1, (2ll * dc.sm_count + direct_tiles - 1) / direct_tiles));
    fg = std::min<int>(fg, static_cast<int>((plan.n_levels + want_groups - 1) / want_groups));
    sp.fl_per_group = fg;
    const int groups = (plan.n_levels + fg - 1) / fg;
    const size_t smem = per_hist * (fg + 1);
    if (smem + 1024 > static_cast<size_t>(dc.max_smem_optin)) return ADAPT_ERR_INVALID_ARG;
    auto kern = (o.round_mode == ADAPT_ROUND_STOCHASTIC) ? search_direct_kernel<true>
                                                         : search_direct_kernel<false>;
    ADAPT_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(smem)));
    const int ctas_per_sm = wide ? 1 : std::max<int>(1, std::min<size_t>(8, (200 * 1024) / (smem + 1024)));
    dim3 grid(static_cast<unsigned>(std::min<long long>(direct_tiles, 1ll * ctas_per_sm * dc.sm_count)),
              groups);
    {
      LaunchScope ls(ADAPT_KERNEL_SEARCH_DIRECT, direct_stream);
      ADAPT_CUDA(launch_dependent(kern, grid, dim3(threads), smem, direct_stream, sp));
    }
    if (beside) {
      ADAPT_CUDA(cudaEventRecord(dc.side_join, dc.side_stream));
      ADAPT_CUDA(cudaStreamWaitEvent(stream, dc.side_join, 0));
    }
  }

  // K3: divergence per (layer, candidate); the last CTA of a layer selects its format
  KldParams kp;
  kp.layers = d_layers; kp.state = d_state;
  kp.cand_wl = reinterpret_cast<const int*>(ws + plan.off_wl);
  kp.cand_fl = reinterpret_cast<const int*>(ws + plan.off_fl);
  kp.cand_slot = reinterpret_cast<const int*>(ws + plan.off_slot);
  kp.cand_order = reinterpret_cast<const int*>(ws + plan.off_order);
  kp.cand_by_fl = reinterpret_cast<const int*>(ws + plan.off_by_fl);
  kp.fl_begin = reinterpret_cast<const int*>(ws + plan.off_fl_begin);
  kp.n_layers = a.n_layers; kp.n_cand = plan.n_cand; kp.n_fl = plan.n_levels; kp.n_bins = bins_stride;
  kp.q_hist = d_q; kp.u_hist = d_u; kp.zeros = d_zeros;
  kp.alpha = o.pseudo_count; kp.inv_ln_base = 1.0 / std::log(base); kp.eps = o.eps;
  kp.kld_out = a.kld_out; kp.zeros_out = reinterpret_cast<long long*>(a.zeros_out);
  kp.best_out = a.best_out; kp.hist_out = o.hist_out;
  kp.start = o.start_wl_fl ? reinterpret_cast<const int*>(ws + plan.off_start) : nullptr;
  kp.status_out = o.status_out;
  {
    LaunchScope ls(ADAPT_KERNEL_KLD, stream);
    // enough CTAs to fill the GPU when there are few (FL, layer) pairs
    const int slices = std::max(1, std::min(16, (4 * dc.sm_count) / std::max(1, plan.n_levels * a.n_layers)));
    ADAPT_CUDA(launch_dependent(kld_kernel, dim3(plan.n_levels, a.n_layers, slices), dim3(kKldThreads), 0, stream, kp));
  }
  return ADAPT_OK;
}

template <typename T>
int launch_quantize_t(const QuantParams& qp, bool stochastic, bool vec, int grid, cudaStream_t s) {
  LaunchScope ls(ADAPT_KERNEL_QUANTIZE, s);
  if (stochastic) {
    if (vec) quantize_kernel<T, true, true><<<grid, kQuantThreads, 0, s>>>(qp);
    else quantize_kernel<T, true, false><<<grid, kQuantThreads, 0, s>>>(qp);
  } else {
    if (vec) quantize_kernel<T, false, true><<<grid, kQuantThreads, 0, s>>>(qp);
    else quantize_kernel<T, false, false><<<grid, kQuantThreads, 0, s>>>(qp);
  }
  ADAPT_CUDA(cudaGetLastError());
  return ADAPT_OK;
}

int run_quantize(const float* x, int64_t n, int wl, int fl, const int32_t* selected,
                 int round_mode, uint64_t seed, int32_t layer, int code_bits, void* codes_out,
                 void* stream) {
  if (n < 0) return ADAPT_ERR_INVALID_ARG;
  if (round_mode != ADAPT_ROUND_RNE && round_mode != ADAPT_ROUND_STOCHASTIC)
    return ADAPT_ERR_INVALID_ARG;
  if (code_bits != 8 && code_bits != 16 && code_bits != 32) return ADAPT_ERR_INVALID_ARG;
  if (!selected && (!valid_format(wl, fl) || wl > code_bits)) return ADAPT_ERR_INVALID_ARG;
  if (n == 0) return ADAPT_OK;
  if (!x || !codes_out) return ADAPT_ERR_INVALID_ARG;
  const int ob = code_bits / 8;
  if ((reinterpret_cast<uintptr_t>(x) & 3u) || (reinterpret_cast<uintptr_t>(codes_out) & (ob - 1)))
    return ADAPT_ERR_INVALID_ARG;
  DeviceCache* dc = nullptr;
  int rc = current_cache(&dc);
  if (rc != ADAPT_OK) return rc;

  QuantParams qp;
  qp.x = x; qp.out = codes_out; qp.n = n; qp.wl = wl; qp.fl = fl; qp.selected = selected;
  qp.seed = seed; qp.layer_id = layer;
  const bool vec = !(reinterpret_cast<uintptr_t>(x) & 15u) &&
                   !(reinterpret_cast<uintptr_t>(codes_out) & (4 * ob - 1));
  const long long work = vec ? std::max<long long>(1, n / 4) : n;
  const long long want = (work + kQuantThreads - 1) / kQuantThreads;
  const int grid = static_cast<int>(std::min<long long>(want, 16ll * dc->sm_count));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool st = round_mode == ADAPT_ROUND_STOCHASTIC;
  if (code_bits == 8) return launch_quantize_t<int8_t>(qp, st, vec, grid, s);
  if (code_bits == 16) return launch_quantize_t<int16_t>(qp, st, vec, grid, s);
  return launch_quantize_t<int32_t>(qp, st, vec, grid, s);
}

}  // namespace

// ---- exported entry points ---------------------------------------------------------

extern "C" {

const char* adapt_version(void) { return "adapt-b200 0.9"; }

const char* adapt_status_string(int status) {
  switch (status) {
    case ADAPT_OK: return "ok";
    case ADAPT_ERR_INVALID_ARG: return "invalid argument";
    case ADAPT_ERR_NONFINITE: return "input holds NaN or Inf";
    case ADAPT_ERR_RANGE: return "input holds |x| >= 2^64";
    case ADAPT_ERR_CUDA: return "CUDA runtime error";
    case ADAPT_ERR_WORKSPACE: return "workspace too small";
    default: return "unknown status";
  }
}

const char* adapt_last_error(void) { return g_last_error; }

uint64_t adapt_kernel_launch_count(void) { return g_launches.load(); }

int adapt_kernel_timing(int enable) {
  g_timing.store(enable != 0);
  return ADAPT_OK;
}

int adapt_kernel_times(double* ms_out, uint64_t* launches_out, int reset) {
  std::lock_guard<std::mutex> l(g_timing_mutex);
  for (const TimedLaunch& t : g_pending) {
    ADAPT_CUDA(cudaEventSynchronize(t.stop));
    float ms = 0.0f;
    ADAPT_CUDA(cudaEventElapsedTime(&ms, t.start, t.stop));
    g_kind_ms[t.kind] += ms;
    g_kind_launches[t.kind] += 1;
    g_event_pool.push_back(t.start);
    g_event_pool.push_back(t.stop);
  }
  g_pending.clear();
  for (int k = 0; k < ADAPT_KERNEL_KINDS; ++k) {
    if (ms_out) ms_out[k] = g_kind_ms[k];
    if (launches_out) launches_out[k] = g_kind_launches[k];
    if (reset) { g_kind_ms[k] = 0.0; g_kind_launches[k] = 0; }
  }
  return ADAPT_OK;
}

int adapt_quantize(const float* x, int64_t n, int wl, int fl, int round_mode, uint64_t seed,
                   int32_t* codes_out) {
  return run_quantize(x, n, wl, fl, nullptr, round_mode, seed, 0, 32, codes_out, nullptr);
}

int adapt_quantize_ex(const float* x, int64_t n, int wl, int fl, int round_mode, uint64_t seed,
                      int32_t layer, int code_bits, void* codes_out, void* stream) {
  return run_quantize(x, n, wl, fl, nullptr, round_mode, seed, layer, code_bits, codes_out, stream);
}

int adapt_quantize_selected(const float* x, int64_t n, const int32_t* selected, int round_mode,
                            uint64_t seed, int32_t layer, int32_t* codes_out, void* stream) {
  if (!selected) return ADAPT_ERR_INVALID_ARG;
  return run_quantize(x, n, 0, 0, selected, round_mode, seed, layer, 32, codes_out, stream);
}

}  // extern "C"

namespace {
// Body of adapt_quantize_selected_batch.  Caller holds g_mutex.
// out_bits: 8, 16 or 32 for integer codes of that width, 0 for dequantized fp32 values.
int run_quantize_batch(const float* const* tensors, const int64_t* lens, int n_layers,
                       const int32_t* best, int round_mode, uint64_t seed, int32_t layer_base,
                       void* const* codes_out, int out_bits, int32_t* unfit, void* stream_handle) {
  if (!tensors || !lens || !best || !codes_out) return ADAPT_ERR_INVALID_ARG;
  if (n_layers < 1 || n_layers > 65535) return ADAPT_ERR_INVALID_ARG;
  if (round_mode != ADAPT_ROUND_RNE && round_mode != ADAPT_ROUND_STOCHASTIC)
    return ADAPT_ERR_INVALID_ARG;
  if (out_bits != 0 && out_bits != 8 && out_bits != 16 && out_bits != 32) return ADAPT_ERR_INVALID_ARG;
  const uintptr_t elem = out_bits == 0 ? 4u : static_cast<uintptr_t>(out_bits / 8);
  for (int l = 0; l < n_layers; ++l) {
    if (lens[l] < 0) return ADAPT_ERR_INVALID_ARG;
    if (lens[l] > 0 && (!tensors[l] || !codes_out[l])) return ADAPT_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(tensors[l]) & 3u) ||
        (reinterpret_cast<uintptr_t>(codes_out[l]) & (elem - 1u)))
      return ADAPT_ERR_INVALID_ARG;
  }
  DeviceCache* dc = nullptr;
  int rc = current_cache(&dc);
  if (rc != ADAPT_OK) return rc;
  const size_t bytes = sizeof(QuantLayer) * static_cast<size_t>(n_layers);
  void* const tab_before = dc->batch_tab;
  rc = grow_device(&dc->batch_tab, &dc->batch_tab_bytes, align_up(bytes, 4096));
  if (rc != ADAPT_OK) return rc;
  if (dc->batch_tab != tab_before) dc->batch_tab_image.clear();
  std::vector<unsigned char> image(bytes);
  QuantLayer* h = reinterpret_cast<QuantLayer*>(image.data());
  long long tiles = 0;
  for (int l = 0; l < n_layers; ++l) {
    h[l].x = tensors[l]; h[l].out = codes_out[l]; h[l].n = lens[l]; h[l].tile_begin = tiles;
    h[l].layer_id = layer_base + l; h[l].select = l; h[l].pad_ = 0; h[l].index_base = 0;
    h[l].vec = !(reinterpret_cast<uintptr_t>(tensors[l]) & 15u) &&
               !(reinterpret_cast<uintptr_t>(codes_out[l]) & (4u * elem - 1u));
    tiles += (lens[l] + kQuantTile - 1) / kQuantTile;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_handle);
  if (unfit) ADAPT_CUDA(cudaMemsetAsync(unfit, 0, sizeof(int32_t) * static_cast<size_t>(n_layers), stream));
  if (tiles == 0) return ADAPT_OK;
  // The same layer list as in the call before, on the same stream (a training loop's case): the
  // table on the device is still the right one, and with no copy in between the kernel can follow
  // the search's last kernel as a dependent launch.
  const bool same = dc->batch_tab_stream == stream && dc->batch_tab_image.size() == bytes &&
                    std::memcmp(dc->batch_tab_image.data(), image.data(), bytes) == 0;
  if (!same) {
    PinnedSlot* slot = nullptr;
    rc = acquire_slot(*dc, bytes, &slot);
    if (rc != ADAPT_OK) return rc;
    std::memcpy(slot->host, image.data(), bytes);
    dc->batch_tab_image.clear();
    ADAPT_CUDA(cudaMemcpyAsync(dc->batch_tab, slot->host, bytes, cudaMemcpyHostToDevice, stream));
    ADAPT_CUDA(cudaEventRecord(slot->done, stream));
    dc->batch_tab_image.swap(image);
    dc->batch_tab_stream = stream;
  }
  const int grid = static_cast<int>(std::min<long long>(tiles, 32ll * dc->sm_count));
  const QuantLayer* d = static_cast<const QuantLayer*>(dc->batch_tab);
  LaunchScope ls(ADAPT_KERNEL_QUANTIZE, stream);
  const bool sr = round_mode == ADAPT_ROUND_STOCHASTIC;
  void (*kern)(const QuantLayer*, int, long long, const int*, unsigned long long, int*) = nullptr;
  switch (out_bits) {
    case 0:  kern = sr ? quantize_batch_kernel<true, float>   : quantize_batch_kernel<false, float>;   break;
    case 8:  kern = sr ? quantize_batch_kernel<true, int8_t>  : quantize_batch_kernel<false, int8_t>;  break;
    case 16: kern = sr ? quantize_batch_kernel<true, int16_t> : quantize_batch_kernel<false, int16_t>; break;
    default: kern = sr ? quantize_batch_kernel<true, int32_t> : quantize_batch_kernel<false, int32_t>; break;
  }
  ADAPT_CUDA(launch_dependent(kern, dim3(grid), dim3(kQuantThreads), 0, stream, d, n_layers, tiles, best,
                              static_cast<unsigned long long>(seed), unfit));
  return ADAPT_OK;
}
}  // namespace

extern "C" {

int adapt_quantize_selected_batch(const float* const* tensors, const int64_t* lens, int n_layers,
                                  const int32_t* best, int round_mode, uint64_t seed,
                                  int32_t layer_base, int32_t* const* codes_out, void* stream_handle) {
  std::lock_guard<std::mutex> lock(g_mutex);
  return run_quantize_batch(tensors, lens, n_layers, best, round_mode, seed, layer_base,
                            reinterpret_cast<void* const*>(codes_out), 32, nullptr, stream_handle);
}

int adapt_quantize_selected_batch_packed(const float* const* tensors, const int64_t* lens,
                                         int n_layers, const int32_t* best, int round_mode,
                                         uint64_t seed, int32_t layer_base, int code_bits,
                                         void* const* codes_out, int32_t* unfit_out,
                                         void* stream_handle) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (code_bits != 8 && code_bits != 16 && code_bits != 32) return ADAPT_ERR_INVALID_ARG;
  return run_quantize_batch(tensors, lens, n_layers, best, round_mode, seed, layer_base, codes_out,
                            code_bits, unfit_out, stream_handle);
}

int adapt_requantize_selected_batch(const float* const* tensors, const int64_t* lens, int n_layers,
                                    const int32_t* best, int round_mode, uint64_t seed,
                                    int32_t layer_base, float* const* values_out, void* stream_handle) {
  std::lock_guard<std::mutex> lock(g_mutex);
  return run_quantize_batch(tensors, lens, n_layers, best, round_mode, seed, layer_base,
                            reinterpret_cast<void* const*>(values_out), 0, nullptr, stream_handle);
}

int adapt_gradient_diversity(const float* const* grads, const int64_t* lens, int n_layers,
                             int n_grads, double* out, void* stream_handle) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!grads || !lens || !out) return ADAPT_ERR_INVALID_ARG;
  if (n_layers < 1 || n_layers > 65535 || n_grads < 1 || n_grads > kDivMaxGrads)
    return ADAPT_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) {
    if (lens[l] < 0) return ADAPT_ERR_INVALID_ARG;
    for (int k = 0; k < n_grads; ++k) {
      const float* g = grads[static_cast<size_t>(l) * n_grads + k];
      if ((lens[l] > 0 && !g) || (reinterpret_cast<uintptr_t>(g) & 3u)) return ADAPT_ERR_INVALID_ARG;
    }
  }
  DeviceCache* dc = nullptr;
  int rc = current_cache(&dc);
  if (rc != ADAPT_OK) return rc;
  const size_t L = n_layers, K = n_grads;
  const size_t off_ptrs = align_up(sizeof(DivLayer) * (L + 1), 256);
  const size_t blob = align_up(off_ptrs + sizeof(float*) * L * K, 256);
  const size_t sums = sizeof(double) * L * (K + 1);
  rc = grow_device(&dc->div_buf, &dc->div_buf_bytes, align_up(blob + sums, 4096));
  if (rc != ADAPT_OK) return rc;
  PinnedSlot* slot = nullptr;
  rc = acquire_slot(*dc, blob, &slot);
  if (rc != ADAPT_OK) return rc;
  char* h = static_cast<char*>(slot->host);
  DivLayer* hl = reinterpret_cast<DivLayer*>(h);
  long long tiles = 0;
  for (int l = 0; l < n_layers; ++l) {
    hl[l].n = lens[l]; hl[l].tile_begin = tiles; hl[l].vec = 1; hl[l].pad_ = 0;
    for (int k = 0; k < n_grads; ++k)
      if (reinterpret_cast<uintptr_t>(grads[static_cast<size_t>(l) * n_grads + k]) & 15u) hl[l].vec = 0;
    tiles += (lens[l] + kDivTile - 1) / kDivTile;
  }
  hl[n_layers].n = 0; hl[n_layers].tile_begin = tiles; hl[n_layers].vec = 0; hl[n_layers].pad_ = 0;
  std::memcpy(h + off_ptrs, grads, sizeof(float*) * L * K);
  cudaStream_t stream = static_cast<cudaStream_t>(stream_handle);
  char* d = static_cast<char*>(dc->div_buf);
  ADAPT_CUDA(cudaMemcpyAsync(d, h, blob, cudaMemcpyHostToDevice, stream));
  ADAPT_CUDA(cudaEventRecord(slot->done, stream));
  ADAPT_CUDA(cudaMemsetAsync(d + blob, 0, sums, stream));
  DivParams dp;
  dp.layers = reinterpret_cast<const DivLayer*>(d);
  dp.grads = reinterpret_cast<const float* const*>(d + off_ptrs);
  dp.sumsq = reinterpret_cast<double*>(d + blob);
  dp.n_layers = n_layers; dp.n_grads = n_grads; dp.n_tiles = tiles;
  if (tiles > 0) {
    const int grid = static_cast<int>(std::min<long long>(tiles, 16ll * dc->sm_count));
    LaunchScope ls(ADAPT_KERNEL_DIVERSITY, stream);
    diversity_kernel<<<grid, kDivThreads, 0, stream>>>(dp);
    ADAPT_CUDA(cudaGetLastError());
  }
  {
    LaunchScope ls(ADAPT_KERNEL_DIVERSITY, stream);
    diversity_finalize_kernel<<<(n_layers + 127) / 128, 128, 0, stream>>>(dp.sumsq, n_layers, n_grads, out);
    ADAPT_CUDA(cudaGetLastError());
  }
  return ADAPT_OK;
}

int adapt_pushup(const double* diversity, const int32_t* best, int n_layers, int strategy,
                 int buff, int32_t* wl_fl_out, int32_t* suggestion_out) {
  if (!diversity || !best || !wl_fl_out || n_layers < 1) return ADAPT_ERR_INVALID_ARG;
  if (strategy != ADAPT_STRATEGY_MIN && strategy != ADAPT_STRATEGY_MEAN &&
      strategy != ADAPT_STRATEGY_MAX) return ADAPT_ERR_INVALID_ARG;
  if (buff < 0 || buff > 31) return ADAPT_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (!valid_format(best[4 * l], best[4 * l + 1])) return ADAPT_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) {
    const double d = diversity[4 * l + 3];
    const int wl_min = best[4 * l], fl_min = best[4 * l + 1];
    int first = 0, second = 0, step = 1;
    if (d > 0.0) {
      // first suggestion: the reciprocal of d - 1, rounded up, between 1 and 32
      const double recip = 1.0 / (d - 1.0);
      first = 32;
      if (recip < 32.0) first = recip > 1.0 ? static_cast<int>(std::ceil(recip)) : 1;
      // second suggestion: 32 d^2 - 1 (at most 32), rounded up, less the present fraction length
      double target = 32.0 * (d * d) - 1.0;
      if (target > 32.0) target = 32.0;
      second = static_cast<int>(std::ceil(target)) - fl_min;
      second = std::max(1, std::min(second, 32));
      if (strategy == ADAPT_STRATEGY_MIN) step = std::min(first, second);
      else if (strategy == ADAPT_STRATEGY_MAX) step = std::max(first, second);
      else step = (first + second) / 2 + ((first + second) & 1);
    }
    int fl = std::min(fl_min + step, 32);
    int wl = std::min(std::max(wl_min, fl) + 1, 32);
    if (fl > 32 - buff) fl = 32 - buff;                 // room for the buffer bits
    wl = std::max(wl, std::min(fl + buff, 32));
    if (fl > wl - 1) fl = wl - 1;                       // the sign bit stays
    wl_fl_out[2 * l] = wl;
    wl_fl_out[2 * l + 1] = fl;
    if (suggestion_out) {
      suggestion_out[3 * l] = first; suggestion_out[3 * l + 1] = second; suggestion_out[3 * l + 2] = step;
    }
  }
  return ADAPT_OK;
}

int adapt_normalize_gradients(const float* const* grads, const int64_t* lens, int n_layers,
                              float* const* out, double* norms_out, void* stream_handle) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!grads || !lens || !out) return ADAPT_ERR_INVALID_ARG;
  if (n_layers < 1 || n_layers > 65535) return ADAPT_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) {
    if (lens[l] < 0) return ADAPT_ERR_INVALID_ARG;
    if (lens[l] > 0 && (!grads[l] || !out[l])) return ADAPT_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(grads[l]) & 3u) || (reinterpret_cast<uintptr_t>(out[l]) & 3u))
      return ADAPT_ERR_INVALID_ARG;
  }
  DeviceCache* dc = nullptr;
  int rc = current_cache(&dc);
  if (rc != ADAPT_OK) return rc;
  // layer table, the two pointer lists, then the sums of squares (two doubles per layer)
  const size_t L = n_layers;
  const size_t off_g = align_up(sizeof(DivLayer) * (L + 1), 256);
  const size_t off_o = align_up(off_g + sizeof(float*) * L, 256);
  const size_t blob = align_up(off_o + sizeof(float*) * L, 256);
  const size_t sums = sizeof(double) * L * 2;
  rc = grow_device(&dc->div_buf, &dc->div_buf_bytes, align_up(blob + sums, 4096));
  if (rc != ADAPT_OK) return rc;
  PinnedSlot* slot = nullptr;
  rc = acquire_slot(*dc, blob, &slot);
  if (rc != ADAPT_OK) return rc;
  char* h = static_cast<char*>(slot->host);
  DivLayer* hl = reinterpret_cast<DivLayer*>(h);
  long long tiles = 0;
  for (int l = 0; l < n_layers; ++l) {
    hl[l].n = lens[l]; hl[l].tile_begin = tiles; hl[l].pad_ = 0;
    hl[l].vec = !(reinterpret_cast<uintptr_t>(grads[l]) & 15u) && !(reinterpret_cast<uintptr_t>(out[l]) & 15u);
    tiles += (lens[l] + kDivTile - 1) / kDivTile;
  }
  hl[n_layers].n = 0; hl[n_layers].tile_begin = tiles; hl[n_layers].vec = 0; hl[n_layers].pad_ = 0;
  std::memcpy(h + off_g, grads, sizeof(float*) * L);
  std::memcpy(h + off_o, out, sizeof(float*) * L);
  cudaStream_t stream = static_cast<cudaStream_t>(stream_handle);
  char* d = static_cast<char*>(dc->div_buf);
  ADAPT_CUDA(cudaMemcpyAsync(d, h, blob, cudaMemcpyHostToDevice, stream));
  ADAPT_CUDA(cudaEventRecord(slot->done, stream));
  ADAPT_CUDA(cudaMemsetAsync(d + blob, 0, sums, stream));
  DivParams dp;
  dp.layers = reinterpret_cast<const DivLayer*>(d);
  dp.grads = reinterpret_cast<const float* const*>(d + off_g);
  dp.sumsq = reinterpret_cast<double*>(d + blob);
  dp.n_layers = n_layers; dp.n_grads = 1; dp.n_tiles = tiles;
  if (tiles > 0) {
    const int grid = static_cast<int>(std::min<long long>(tiles, 16ll * dc->sm_count));
    {
      LaunchScope ls(ADAPT_KERNEL_DIVERSITY, stream);
      diversity_kernel<<<grid, kDivThreads, 0, stream>>>(dp);
      ADAPT_CUDA(cudaGetLastError());
    }
    LaunchScope ls(ADAPT_KERNEL_DIVERSITY, stream);
    normalize_kernel<<<grid, kDivThreads, 0, stream>>>(dp.layers, dp.grads,
                                                       reinterpret_cast<float* const*>(d + off_o),
                                                       dp.sumsq, n_layers, tiles);
    ADAPT_CUDA(cudaGetLastError());
  }
  if (norms_out)   // the sums of squares sit two doubles apart: strided copy of the first of each
    ADAPT_CUDA(cudaMemcpy2DAsync(norms_out, sizeof(double), dp.sumsq, 2 * sizeof(double),
                                 sizeof(double), L, cudaMemcpyDeviceToDevice, stream));
  return ADAPT_OK;
}

size_t adapt_search_workspace_bytes(const int64_t* lens, int n_layers, const adapt_grid* grid,
                                    int n_bins) {
  Plan plan;
  if (!make_plan(lens, n_layers, grid, n_bins, &plan)) return 0;
  return plan.total;
}

int adapt_precision_search_ex(const float* const* tensors, const int64_t* lens, int n_layers,
                              const adapt_grid* grid, int n_bins, double* kld_out,
                              int64_t* zeros_out, int32_t* best_out,
                              const adapt_search_opts* opts) {
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceCache* dc = nullptr;
  int rc = current_cache(&dc);
  if (rc != ADAPT_OK) return rc;
  SearchArgs a{tensors, lens, n_layers, grid, n_bins, kld_out, zeros_out, best_out,
               opts ? *opts : default_opts()};
  return run_search(*dc, a);
}

int adapt_precision_search(const float* const* tensors, const int64_t* lens, int n_layers,
                           const adapt_grid* grid, int n_bins, double* kld_out,
                           int64_t* zeros_out, int32_t* best_out) {
  return adapt_precision_search_ex(tensors, lens, n_layers, grid, n_bins, kld_out, zeros_out,
                                   best_out, nullptr);
}

}  // extern "C"

namespace {

// Launches the batched quantize kernel over table entries [first, first + count) of a device
// table whose tile numbering restarts at `first`.  Caller holds g_mutex.
int launch_quantize_entries(const QuantLayer* d_table, int count, long long tiles, const int32_t* best,
                            int round_mode, uint64_t seed, int out_bits, int32_t* unfit, int sm_count,
                            cudaStream_t stream) {
  if (tiles == 0) return ADAPT_OK;
  const int grid = static_cast<int>(std::min<long long>(tiles, 32ll * sm_count));
  LaunchScope ls(ADAPT_KERNEL_QUANTIZE, stream);
  const bool sr = round_mode == ADAPT_ROUND_STOCHASTIC;
  void (*kern)(const QuantLayer*, int, long long, const int*, unsigned long long, int*) = nullptr;
  switch (out_bits) {
    case 8:  kern = sr ? quantize_batch_kernel<true, int8_t>  : quantize_batch_kernel<false, int8_t>;  break;
    case 16: kern = sr ? quantize_batch_kernel<true, int16_t> : quantize_batch_kernel<false, int16_t>; break;
    default: kern = sr ? quantize_batch_kernel<true, int32_t> : quantize_batch_kernel<false, int32_t>; break;
  }
  kern<<<grid, kQuantThreads, 0, stream>>>(d_table, count, tiles, best, seed, unfit);
  ADAPT_CUDA(cudaGetLastError());
  return ADAPT_OK;
}

// Host-buffer search, optionally followed by the quantization of every layer at its selected
// format from the same device copy (codes_out: HOST array of HOST buffers of code_bits-wide codes,
// or null).  The codes are produced slice by slice (a slice is a run of whole small layers or a
// piece of a large one, about 64 MB of input) and each slice's download runs on a second stream
// while the next slice is quantized.
int run_search_host(const float* const* tensors, const int64_t* lens, int n_layers,
                    const adapt_grid* grid, int n_bins, double* kld_out, int64_t* zeros_out,
                    int32_t* best_out, void* const* codes_out, int code_bits, int32_t* unfit_out,
                    const adapt_search_opts* opts) {
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceCache* dc = nullptr;
  int rc = current_cache(&dc);
  if (rc != ADAPT_OK) return rc;
  adapt_search_opts o = opts ? *opts : default_opts();
  if (o.workspace || o.workspace_bytes || o.hist_out || o.range_out || o.status_out) return ADAPT_ERR_INVALID_ARG;
  if (!tensors || !kld_out || !zeros_out || !best_out) return ADAPT_ERR_INVALID_ARG;
  if (codes_out && code_bits != 8 && code_bits != 16 && code_bits != 32) return ADAPT_ERR_INVALID_ARG;
  Plan plan;
  if (!make_plan(lens, n_layers, grid, n_bins, &plan)) return ADAPT_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l) {
    if (lens[l] > 0 && !tensors[l]) return ADAPT_ERR_INVALID_ARG;
    if (codes_out && lens[l] > 0 && !codes_out[l]) return ADAPT_ERR_INVALID_ARG;
  }

  // device copies of the layers, 256-byte aligned each
  std::vector<size_t> off(n_layers);
  size_t in_bytes = 0;
  for (int l = 0; l < n_layers; ++l) {
    off[l] = in_bytes;
    in_bytes = align_up(in_bytes + sizeof(float) * static_cast<size_t>(lens[l]), 256);
  }
  const size_t C = plan.n_cand, L = n_layers;
  const size_t kld_bytes = align_up(sizeof(double) * L * C, 256);
  const size_t zeros_bytes = align_up(sizeof(int64_t) * L * C, 256);
  const size_t best_bytes = align_up(sizeof(int32_t) * 4 * L, 256);
  const size_t unfit_bytes = align_up(sizeof(int32_t) * L, 256);
  rc = grow_device(&dc->stage_in, &dc->stage_in_bytes, std::max<size_t>(in_bytes, 256));
  if (rc != ADAPT_OK) return rc;
  rc = grow_device(&dc->stage_out, &dc->stage_out_bytes, kld_bytes + zeros_bytes + best_bytes + unfit_bytes);
  if (rc != ADAPT_OK) return rc;

  cudaStream_t stream = static_cast<cudaStream_t>(o.stream);
  std::vector<const float*> dptr(n_layers);
  for (int l = 0; l < n_layers; ++l) {
    dptr[l] = reinterpret_cast<const float*>(static_cast<char*>(dc->stage_in) + off[l]);
    if (lens[l] > 0)
      ADAPT_CUDA(cudaMemcpyAsync(const_cast<float*>(dptr[l]), tensors[l],
                                 sizeof(float) * static_cast<size_t>(lens[l]),
                                 cudaMemcpyHostToDevice, stream));
  }
  char* so = static_cast<char*>(dc->stage_out);
  SearchArgs a{dptr.data(), lens, n_layers, grid, n_bins, reinterpret_cast<double*>(so),
               reinterpret_cast<int64_t*>(so + kld_bytes),
               reinterpret_cast<int32_t*>(so + kld_bytes + zeros_bytes), o};
  rc = run_search(*dc, a);
  if (rc != ADAPT_OK) return rc;
  std::vector<int32_t> fits(n_layers, 0);       // 1: the layer's codes are produced and downloaded
  if (codes_out) {
    const size_t cb = static_cast<size_t>(code_bits / 8);
    // the selected word lengths decide which layers get codes: fetch them (16 bytes per layer)
    ADAPT_CUDA(cudaMemcpyAsync(best_out, a.best_out, sizeof(int32_t) * 4 * L, cudaMemcpyDeviceToHost, stream));
    ADAPT_CUDA(cudaStreamSynchronize(stream));
    for (int l = 0; l < n_layers; ++l) {
      const int wl_sel = best_out[4 * l], fl_sel = best_out[4 * l + 1];
      const bool valid_sel = valid_format(wl_sel, fl_sel) &&
                             !(best_out[4 * l + 3] & (ADAPT_FLAG_NONFINITE | ADAPT_FLAG_RANGE));
      fits[l] = (valid_sel && wl_sel <= code_bits) ? 1 : 0;
      if (unfit_out) unfit_out[l] = (valid_sel && wl_sel > code_bits) ? wl_sel : 0;
    }
    // codes of all layers in one more library-owned buffer: layer l at off[l] / 4 * cb
    rc = grow_device(&dc->stage_codes, &dc->stage_codes_bytes, std::max<size_t>(in_bytes / 4 * cb, 256));
    if (rc != ADAPT_OK) return rc;
    if (!dc->copy_stream) {
      ADAPT_CUDA(cudaStreamCreateWithFlags(&dc->copy_stream, cudaStreamNonBlocking));
      for (cudaEvent_t& e : dc->slice_done) ADAPT_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
      ADAPT_CUDA(cudaEventCreateWithFlags(&dc->copies_done, cudaEventDisableTiming));
    }
    // table entries: pieces of at most kSliceElems elements, in layer order
    constexpr long long kSliceElems = 16ll << 20;
    std::vector<QuantLayer> table;
    std::vector<int> group_first;           // first entry of every launch group
    std::vector<long long> group_tiles;
    long long in_group = 0, tiles = 0;
    for (int l = 0; l < n_layers; ++l) {
      if (!fits[l]) continue;
      for (long long at = 0; at < lens[l]; at += kSliceElems) {
        const long long n = std::min<long long>(kSliceElems, lens[l] - at);
        if (group_first.empty() || in_group + n > kSliceElems) {
          if (!group_first.empty()) group_tiles.push_back(tiles);
          group_first.push_back(static_cast<int>(table.size()));
          in_group = 0; tiles = 0;
        }
        QuantLayer q;
        q.x = dptr[l] + at;
        q.out = static_cast<char*>(dc->stage_codes) + off[l] / 4 * cb + static_cast<size_t>(at) * cb;
        q.n = n; q.tile_begin = tiles; q.layer_id = o.layer_base + l; q.vec = 1;   // 256-byte aligned pieces
        q.select = l; q.pad_ = 0; q.index_base = at;
        table.push_back(q);
        tiles += (n + kQuantTile - 1) / kQuantTile;
        in_group += n;
      }
    }
    if (!group_first.empty()) group_tiles.push_back(tiles);
    if (!table.empty()) {
      const size_t bytes = sizeof(QuantLayer) * table.size();
      rc = grow_device(&dc->batch_tab, &dc->batch_tab_bytes, align_up(bytes, 4096));
      if (rc != ADAPT_OK) return rc;
      PinnedSlot* slot = nullptr;
      rc = acquire_slot(*dc, bytes, &slot);
      if (rc != ADAPT_OK) return rc;
      std::memcpy(slot->host, table.data(), bytes);
      dc->batch_tab_image.clear();
      ADAPT_CUDA(cudaMemcpyAsync(dc->batch_tab, slot->host, bytes, cudaMemcpyHostToDevice, stream));
      ADAPT_CUDA(cudaEventRecord(slot->done, stream));
      const QuantLayer* d_table = static_cast<const QuantLayer*>(dc->batch_tab);
      for (size_t g = 0; g < group_first.size(); ++g) {
        const int first = group_first[g];
        const int count = (g + 1 < group_first.size() ? group_first[g + 1] : static_cast<int>(table.size())) - first;
        rc = launch_quantize_entries(d_table + first, count, group_tiles[g], a.best_out, o.round_mode, o.seed,
                                     code_bits, nullptr, dc->sm_count, stream);
        if (rc != ADAPT_OK) return rc;
        // the group's download starts when its kernel is done and overlaps the next group's kernel
        cudaEvent_t ev = dc->slice_done[g & 1];
        ADAPT_CUDA(cudaEventRecord(ev, stream));
        ADAPT_CUDA(cudaStreamWaitEvent(dc->copy_stream, ev, 0));
        for (int e = first; e < first + count; ++e) {
          const QuantLayer& q = table[e];
          char* host_at = static_cast<char*>(codes_out[q.select]) + static_cast<size_t>(q.index_base) * cb;
          ADAPT_CUDA(cudaMemcpyAsync(host_at, q.out, static_cast<size_t>(q.n) * cb, cudaMemcpyDeviceToHost,
                                     dc->copy_stream));
        }
      }
      ADAPT_CUDA(cudaEventRecord(dc->copies_done, dc->copy_stream));
      ADAPT_CUDA(cudaStreamWaitEvent(stream, dc->copies_done, 0));
    }
  }
  ADAPT_CUDA(cudaMemcpyAsync(kld_out, a.kld_out, sizeof(double) * L * C, cudaMemcpyDeviceToHost, stream));
  ADAPT_CUDA(cudaMemcpyAsync(zeros_out, a.zeros_out, sizeof(int64_t) * L * C, cudaMemcpyDeviceToHost, stream));
  ADAPT_CUDA(cudaMemcpyAsync(best_out, a.best_out, sizeof(int32_t) * 4 * L, cudaMemcpyDeviceToHost, stream));
  ADAPT_CUDA(cudaStreamSynchronize(stream));
  int status = ADAPT_OK;
  for (int l = 0; l < n_layers; ++l) {
    if (best_out[4 * l + 3] & ADAPT_FLAG_NONFINITE) return ADAPT_ERR_NONFINITE;
    if (best_out[4 * l + 3] & ADAPT_FLAG_RANGE) status = ADAPT_ERR_RANGE;
  }
  return status;
}
}  // namespace

extern "C" {

int adapt_precision_search_host(const float* const* tensors, const int64_t* lens, int n_layers,
                                const adapt_grid* grid, int n_bins, double* kld_out,
                                int64_t* zeros_out, int32_t* best_out,
                                const adapt_search_opts* opts) {
  return run_search_host(tensors, lens, n_layers, grid, n_bins, kld_out, zeros_out, best_out,
                         nullptr, 32, nullptr, opts);
}

int adapt_precision_switch_host(const float* const* tensors, const int64_t* lens, int n_layers,
                                const adapt_grid* grid, int n_bins, double* kld_out,
                                int64_t* zeros_out, int32_t* best_out, int32_t* const* codes_out,
                                const adapt_search_opts* opts) {
  if (!codes_out) return ADAPT_ERR_INVALID_ARG;
  return run_search_host(tensors, lens, n_layers, grid, n_bins, kld_out, zeros_out, best_out,
                         reinterpret_cast<void* const*>(codes_out), 32, nullptr, opts);
}

int adapt_precision_switch_host_packed(const float* const* tensors, const int64_t* lens, int n_layers,
                                       const adapt_grid* grid, int n_bins, double* kld_out,
                                       int64_t* zeros_out, int32_t* best_out, int code_bits,
                                       void* const* codes_out, int32_t* unfit_out,
                                       const adapt_search_opts* opts) {
  if (!codes_out) return ADAPT_ERR_INVALID_ARG;
  return run_search_host(tensors, lens, n_layers, grid, n_bins, kld_out, zeros_out, best_out,
                         codes_out, code_bits, unfit_out, opts);
}

int adapt_quantize_host(const float* x, int64_t n, int wl, int fl, int round_mode, uint64_t seed,
                        int32_t layer, int code_bits, void* codes_out) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (n < 0 || (code_bits != 8 && code_bits != 16 && code_bits != 32)) return ADAPT_ERR_INVALID_ARG;
  if (!valid_format(wl, fl) || wl > code_bits) return ADAPT_ERR_INVALID_ARG;
  if (n == 0) return ADAPT_OK;
  if (!x || !codes_out) return ADAPT_ERR_INVALID_ARG;
  DeviceCache* dc = nullptr;
  int rc = current_cache(&dc);
  if (rc != ADAPT_OK) return rc;
  const size_t in_bytes = sizeof(float) * static_cast<size_t>(n);
  const size_t out_bytes = static_cast<size_t>(code_bits / 8) * static_cast<size_t>(n);
  rc = grow_device(&dc->stage_in, &dc->stage_in_bytes, in_bytes);
  if (rc != ADAPT_OK) return rc;
  rc = grow_device(&dc->stage_out, &dc->stage_out_bytes, out_bytes);
  if (rc != ADAPT_OK) return rc;
  ADAPT_CUDA(cudaMemcpyAsync(dc->stage_in, x, in_bytes, cudaMemcpyHostToDevice, nullptr));
  rc = run_quantize(static_cast<const float*>(dc->stage_in), n, wl, fl, nullptr, round_mode, seed,
                    layer, code_bits, dc->stage_out, nullptr);
  if (rc != ADAPT_OK) return rc;
  ADAPT_CUDA(cudaMemcpyAsync(codes_out, dc->stage_out, out_bytes, cudaMemcpyDeviceToHost, nullptr));
  ADAPT_CUDA(cudaStreamSynchronize(nullptr));
  return ADAPT_OK;
}

}  // extern "C"

// ---- other number formats -----------------------------------------------------------------

namespace {

struct FormatPlan {
  int n_layers = 0, n_cand = 0, n_rules = 0, n_bins = 0;
  std::vector<FormatCand> cands;
  std::vector<FormatRule> rules;
  size_t off_layers = 0, off_cands = 0, off_rules = 0, off_state = 0, blob_bytes = 0;
  size_t off_level = 0, off_clamp = 0, off_b = 0;
  size_t accum_begin = 0, off_zeros = 0, off_hist = 0, accum_bytes = 0, total = 0;
};

bool valid_any_format(const adapt_format& f) {
  if (f.kind == ADAPT_FMT_FIXED) return valid_format(f.a, f.b);
  if (f.kind == ADAPT_FMT_BFP) return f.a >= 2 && f.a <= 32;
  if (f.kind == ADAPT_FMT_FLOAT) return f.a >= 2 && f.a <= 8 && f.b >= 1 && f.b <= 23;
  return false;
}

// Validates the sizes, finds the distinct rounding rules and lays out the workspace.
bool make_format_plan(const int64_t* lens, int n_layers, const adapt_format* formats,
                      int n_formats, int n_bins, FormatPlan* p) {
  if (!lens || !formats) return false;
  if (n_layers < 1 || n_layers > 65535) return false;
  if (n_formats < 1 || n_formats > ADAPT_MAX_FORMATS) return false;
  if (n_bins < 1 || n_bins > kMaxBins) return false;
  for (int l = 0; l < n_layers; ++l)
    if (lens[l] < 0 || lens[l] >= (1ll << 32)) return false;
  p->n_layers = n_layers; p->n_cand = n_formats; p->n_bins = n_bins;
  p->rules.clear();
  p->rules.push_back(FormatRule{kRuleIdentity, 0, 0, 0});
  p->cands.resize(n_formats);
  for (int c = 0; c < n_formats; ++c) {
    const adapt_format& f = formats[c];
    if (!valid_any_format(f)) return false;
    // fixed: one rule per FL; block floating point: per WL; floating point: per (E, M)
    FormatRule want{f.kind, f.kind == ADAPT_FMT_FIXED ? f.b : f.a,
                    f.kind == ADAPT_FMT_FLOAT ? f.b : 0, 0};
    int r = -1;
    for (size_t i = 1; i < p->rules.size(); ++i)
      if (p->rules[i].kind == want.kind && p->rules[i].p0 == want.p0 && p->rules[i].p1 == want.p1) {
        r = static_cast<int>(i);
        break;
      }
    if (r < 0) { r = static_cast<int>(p->rules.size()); p->rules.push_back(want); }
    p->cands[c] = FormatCand{f.kind, f.a, f.b, r};
  }
  p->n_rules = static_cast<int>(p->rules.size());
  const size_t C = n_formats, L = n_layers, B = n_bins, R = p->n_rules;
  size_t o = 0;
  p->off_layers = o;  o = align_up(o + sizeof(LayerDesc) * (L + 1), 16);
  p->off_cands = o;   o = align_up(o + sizeof(FormatCand) * C, 16);
  p->off_rules = o;   o = align_up(o + sizeof(FormatRule) * R, 16);
  p->off_state = o;   o = align_up(o + sizeof(LayerState) * L, 256);
  p->blob_bytes = o;
  p->off_level = o;   o = align_up(o + sizeof(int) * L * R, 256);
  p->off_clamp = o;   o = align_up(o + sizeof(float2) * L * C, 256);
  p->off_b = o;       o = align_up(o + sizeof(int) * L * C, 256);
  p->accum_begin = o;
  p->off_zeros = o;   o = align_up(o + sizeof(unsigned long long) * L * R, 256);
  p->off_hist = o;    o = align_up(o + sizeof(unsigned) * L * R * B, 256);
  p->accum_bytes = o - p->accum_begin;
  p->total = o;
  return true;
}

struct FormatArgs {
  const float* const* tensors;
  const int64_t* lens;
  int n_layers;
  const adapt_format* formats;
  int n_formats, n_bins;
  double* kld_out;
  int64_t* zeros_out;
  int32_t* b_out;
  int32_t* best_out;
  adapt_search_opts opts;
};

// Enqueues the whole format search on opts.stream.  Caller holds g_mutex.
int run_format_search(DeviceCache& dc, const FormatArgs& a) {
  const adapt_search_opts& o = a.opts;
  if (!a.tensors || !a.kld_out || !a.zeros_out || !a.best_out) return ADAPT_ERR_INVALID_ARG;
  if (o.round_mode != ADAPT_ROUND_RNE && o.round_mode != ADAPT_ROUND_STOCHASTIC)
    return ADAPT_ERR_INVALID_ARG;
  if (!(o.eps >= 0.0) || !(o.pseudo_count >= 0.0)) return ADAPT_ERR_INVALID_ARG;
  if (o.n_bins_per_layer || o.start_wl_fl || o.algorithm != 0) return ADAPT_ERR_INVALID_ARG;
  const double base = (o.log_base == 0.0) ? 2.0 : o.log_base;
  if (!(base > 0.0) || base == 1.0 || !std::isfinite(base)) return ADAPT_ERR_INVALID_ARG;
  FormatPlan plan;
  if (!make_format_plan(a.lens, a.n_layers, a.formats, a.n_formats, a.n_bins, &plan))
    return ADAPT_ERR_INVALID_ARG;
  for (int l = 0; l < a.n_layers; ++l) {
    if (a.lens[l] > 0 && !a.tensors[l]) return ADAPT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(a.tensors[l]) & 3u) return ADAPT_ERR_INVALID_ARG;
  }
  // shared-memory shape: as many rule histograms per group as fit, at most kMaxRulesPerGroup
  const size_t per_hist = sizeof(unsigned) * plan.n_bins;
  const size_t budget = std::min<size_t>(200 * 1024, static_cast<size_t>(dc.max_smem_optin) - 4096);
  if (per_hist > budget) return ADAPT_ERR_INVALID_ARG;

  char* ws = nullptr;
  if (o.workspace) {
    if (reinterpret_cast<uintptr_t>(o.workspace) & 255u) return ADAPT_ERR_INVALID_ARG;
    if (o.workspace_bytes < plan.total) return ADAPT_ERR_WORKSPACE;
    ws = static_cast<char*>(o.workspace);
  } else {
    int rc = grow_device(&dc.workspace, &dc.workspace_bytes, plan.total);
    if (rc != ADAPT_OK) return rc;
    ws = static_cast<char*>(dc.workspace);
  }
  cudaStream_t stream = static_cast<cudaStream_t>(o.stream);

  PinnedSlot* slot = nullptr;
  int rc = acquire_slot(dc, plan.blob_bytes, &slot);
  if (rc != ADAPT_OK) return rc;
  char* h = static_cast<char*>(slot->host);
  std::memset(h, 0, plan.blob_bytes);
  std::vector<int> all(a.n_layers);
  std::iota(all.begin(), all.end(), 0);
  SearchArgs la{a.tensors, a.lens, a.n_layers, nullptr, a.n_bins, nullptr, nullptr, nullptr, o};
  const long long tiles = fill_list(reinterpret_cast<LayerDesc*>(h + plan.off_layers), all, la, kTile);
  const int range_grid = plan_range_grid(reinterpret_cast<LayerDesc*>(h + plan.off_layers), a.n_layers, tiles, dc.sm_count);
  std::memcpy(h + plan.off_cands, plan.cands.data(), sizeof(FormatCand) * plan.n_cand);
  std::memcpy(h + plan.off_rules, plan.rules.data(), sizeof(FormatRule) * plan.n_rules);
  LayerState* hs = reinterpret_cast<LayerState*>(h + plan.off_state);
  for (int l = 0; l < a.n_layers; ++l) { hs[l].min_key = 0xFFFFFFFFu; hs[l].max_key = 0u; }
  ADAPT_CUDA(cudaMemcpyAsync(ws, h, plan.blob_bytes, cudaMemcpyHostToDevice, stream));
  ADAPT_CUDA(cudaEventRecord(slot->done, stream));
  ADAPT_CUDA(cudaMemsetAsync(ws + plan.accum_begin, 0, plan.accum_bytes, stream));

  FormatParams fp;
  fp.layers = reinterpret_cast<const LayerDesc*>(ws + plan.off_layers);
  LayerState* d_state = reinterpret_cast<LayerState*>(ws + plan.off_state);
  fp.state = d_state;
  fp.cands = reinterpret_cast<const FormatCand*>(ws + plan.off_cands);
  fp.rules = reinterpret_cast<const FormatRule*>(ws + plan.off_rules);
  fp.n_layers = a.n_layers; fp.n_cand = plan.n_cand; fp.n_rules = plan.n_rules; fp.n_bins = plan.n_bins;
  fp.n_tiles = tiles;
  fp.level = reinterpret_cast<int*>(ws + plan.off_level);
  fp.clamp = reinterpret_cast<float2*>(ws + plan.off_clamp);
  fp.b_used = reinterpret_cast<int*>(ws + plan.off_b);
  fp.hist = reinterpret_cast<unsigned*>(ws + plan.off_hist);
  fp.zeros = reinterpret_cast<unsigned long long*>(ws + plan.off_zeros);
  fp.seed = o.seed;
  fp.alpha = o.pseudo_count; fp.inv_ln_base = 1.0 / std::log(base); fp.eps = o.eps;
  fp.kld_out = a.kld_out; fp.zeros_out = reinterpret_cast<long long*>(a.zeros_out);
  fp.b_out = a.b_out; fp.best_out = a.best_out; fp.hist_out = o.hist_out; fp.status_out = o.status_out;

  // rule groups: few tiles spread the rules over more CTAs, many tiles fill shared memory
  int rpg = static_cast<int>(std::min<size_t>(kMaxRulesPerGroup, budget / per_hist));
  rpg = std::max(1, std::min(rpg, plan.n_rules));
  const long long want_groups = std::min<long long>(
      plan.n_rules, std::max<long long>(1, (2ll * dc.sm_count + std::max(1ll, tiles) - 1) / std::max(1ll, tiles)));
  rpg = std::min<int>(rpg, static_cast<int>((plan.n_rules + want_groups - 1) / want_groups));
  fp.rules_per_group = rpg;
  const int groups = (plan.n_rules + rpg - 1) / rpg;
  const size_t smem = per_hist * rpg;

  {
    RangeParams rp;
    rp.layers = fp.layers; rp.n_layers = a.n_layers; rp.n_tiles = tiles; rp.state = d_state;
    rp.range_out = o.range_out;
    LaunchScope ls(ADAPT_KERNEL_RANGE, stream);
    range_scan_kernel<<<range_grid, kRangeThreads, 0, stream>>>(rp);
    ADAPT_CUDA(cudaGetLastError());
  }
  {
    LaunchScope ls(ADAPT_KERNEL_FORMAT_RESOLVE, stream);
    ADAPT_CUDA(launch_dependent(format_resolve_kernel, dim3(a.n_layers), dim3(128), 0, stream, fp));
  }
  if (tiles > 0) {
    auto kern = (o.round_mode == ADAPT_ROUND_STOCHASTIC) ? format_search_kernel<true>
                                                         : format_search_kernel<false>;
    ADAPT_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(smem)));
    const int ctas_per_sm = std::max<int>(1, std::min<size_t>(2, (200 * 1024) / (smem + 2048)));
    dim3 grid(static_cast<unsigned>(std::min<long long>(tiles, 1ll * ctas_per_sm * dc.sm_count)), groups);
    LaunchScope ls(ADAPT_KERNEL_FORMAT_SEARCH, stream);
    ADAPT_CUDA(launch_dependent(kern, grid, dim3(kFormatThreads), smem, stream, fp));
  }
  {
    LaunchScope ls(ADAPT_KERNEL_FORMAT_KLD, stream);
    ADAPT_CUDA(launch_dependent(format_kld_kernel, dim3(plan.n_cand, a.n_layers), dim3(kKldThreads), 0, stream, fp));
  }
  {
    LaunchScope ls(ADAPT_KERNEL_SELECT, stream);
    ADAPT_CUDA(launch_dependent(format_select_kernel, dim3(a.n_layers), dim3(32), 0, stream, fp));
  }
  return ADAPT_OK;
}

}  // namespace

extern "C" {

size_t adapt_format_search_workspace_bytes(const int64_t* lens, int n_layers,
                                           const adapt_format* formats, int n_formats,
                                           int n_bins) {
  FormatPlan plan;
  if (!make_format_plan(lens, n_layers, formats, n_formats, n_bins, &plan)) return 0;
  return plan.total;
}

int adapt_format_search(const float* const* tensors, const int64_t* lens, int n_layers,
                        const adapt_format* formats, int n_formats, int n_bins,
                        double* kld_out, int64_t* zeros_out, int32_t* b_out,
                        int32_t* best_out, const adapt_search_opts* opts) {
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceCache* dc = nullptr;
  int rc = current_cache(&dc);
  if (rc != ADAPT_OK) return rc;
  FormatArgs a{tensors, lens, n_layers, formats, n_formats, n_bins, kld_out, zeros_out, b_out,
               best_out, opts ? *opts : default_opts()};
  return run_format_search(*dc, a);
}

int adapt_format_quantize(const float* x, int64_t n, int kind, int a, int b, int round_mode,
                          uint64_t seed, int layer, float* values_out, void* stream) {
  if (n < 0 || (n > 0 && (!x || !values_out))) return ADAPT_ERR_INVALID_ARG;
  if (round_mode != ADAPT_ROUND_RNE && round_mode != ADAPT_ROUND_STOCHASTIC)
    return ADAPT_ERR_INVALID_ARG;
  adapt_format f{kind, a, b};
  if (kind == ADAPT_FMT_BFP) {
    if (a < 2 || a > 32 || b < -kBfpScaleLimit || b > kBfpScaleLimit) return ADAPT_ERR_INVALID_ARG;
  } else if (!valid_any_format(f)) {
    return ADAPT_ERR_INVALID_ARG;
  }
  if (n == 0) return ADAPT_OK;
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceCache* dc = nullptr;
  int rc = current_cache(&dc);
  if (rc != ADAPT_OK) return rc;
  FormatQuantParams qp{x, values_out, n, kind, a, b, layer, seed};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int grid = static_cast<int>(std::min<long long>((n + 255) / 256, 16ll * dc->sm_count));
  LaunchScope ls(ADAPT_KERNEL_FORMAT_QUANTIZE, s);
  if (round_mode == ADAPT_ROUND_STOCHASTIC) format_quantize_kernel<true><<<grid, 256, 0, s>>>(qp);
  else format_quantize_kernel<false><<<grid, 256, 0, s>>>(qp);
  ADAPT_CUDA(cudaGetLastError());
  return ADAPT_OK;
}

}  // extern "C"

// ---- search without any allocation ------------------------------------------------
//
// Scratch of adapt_precision_search_static: one fixed device array, part of the library
// image, so every GPU that loads the library holds it until the process exits.

namespace {

constexpr int kStaticMaxLayers = ADAPT_STATIC_MAX_LAYERS;
constexpr int kStaticMaxBins = ADAPT_STATIC_MAX_BINS;
constexpr int kStaticMaxCand = ADAPT_STATIC_MAX_CAND;

// layout (bytes): descriptor block, then the accumulators that every call clears
constexpr size_t kStLayers = 0;                                                   // LayerDesc[L + 1]
constexpr size_t kStWl = kStLayers + 64 * (kStaticMaxLayers + 1);
constexpr size_t kStFl = kStWl + 4 * kStaticMaxCand;
constexpr size_t kStSlot = kStFl + 4 * kStaticMaxCand;
constexpr size_t kStOrder = kStSlot + 4 * kStaticMaxCand;
constexpr size_t kStByFl = kStOrder + 4 * kStaticMaxCand;
constexpr size_t kStFlBegin = kStByFl + 4 * kStaticMaxCand;                       // int[33]
constexpr size_t kStState = kStFlBegin + 4 * 64;                                  // LayerState[L]
constexpr size_t kStBlobEnd = kStState + 64 * kStaticMaxLayers;
constexpr size_t kStZeros = (kStBlobEnd + 255) / 256 * 256;                       // u64[L][32]
constexpr size_t kStQ = kStZeros + 8 * kStaticMaxLayers * kMaxFl;                 // u32[L][B]
constexpr size_t kStU = kStQ + 4 * static_cast<size_t>(kStaticMaxLayers) * kStaticMaxBins;
constexpr size_t kStEnd = kStU + 4 * static_cast<size_t>(kStaticMaxLayers) * kMaxFl * kStaticMaxBins;
static_assert((kStEnd - kStZeros) % 16 == 0, "the accumulators are cleared in 16-byte units");
static_assert(sizeof(LayerDesc) <= 64 && sizeof(LayerState) <= 64, "descriptor slots too small");

static __device__ __align__(256) unsigned char g_static_scratch[kStEnd];

// The array's name is only a host-side handle; kernels need its device address, looked up
// once per device (with that device current) and kept here.
unsigned char* g_static_ptr[kMaxDevices] = {nullptr};
unsigned char g_static_blob[kStBlobEnd];   // host image of the descriptor block (under g_mutex)

int static_scratch_address(unsigned char** out) {
  int dev = 0;
  ADAPT_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) {
    std::snprintf(g_last_error, sizeof(g_last_error), "device index %d not supported", dev);
    return ADAPT_ERR_CUDA;
  }
  if (!g_static_ptr[dev]) {
    void* ptr = nullptr;
    ADAPT_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
    g_static_ptr[dev] = static_cast<unsigned char*>(ptr);
  }
  *out = g_static_ptr[dev];
  return ADAPT_OK;
}

}  // namespace

extern "C" {

int adapt_precision_search_static(const float* const* tensors, const int64_t* lens, int n_layers,
                                  const adapt_grid* grid, int n_bins, double* kld_out,
                                  int64_t* zeros_out, int32_t* best_out, void* stream_handle) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!tensors || !lens || !grid || !grid->wl || !grid->fl || !kld_out || !zeros_out || !best_out)
    return ADAPT_ERR_INVALID_ARG;
  if (n_layers < 1 || n_layers > kStaticMaxLayers || grid->n_cand < 1 ||
      grid->n_cand > kStaticMaxCand || n_bins < 1 || n_bins > kStaticMaxBins) {
    std::snprintf(g_last_error, sizeof(g_last_error),
                  "adapt_precision_search_static: sizes beyond the fixed scratch (at most %d layers, "
                  "%d candidates, %d bins; got %d, %d, %d)", kStaticMaxLayers, kStaticMaxCand,
                  kStaticMaxBins, n_layers, grid->n_cand, n_bins);
    return ADAPT_ERR_WORKSPACE;
  }
  int fmax = 0;
  for (int c = 0; c < grid->n_cand; ++c) {
    if (!valid_format(grid->wl[c], grid->fl[c])) return ADAPT_ERR_INVALID_ARG;
    fmax = std::max(fmax, grid->fl[c]);
  }
  for (int l = 0; l < n_layers; ++l) {
    if (lens[l] < 0 || lens[l] >= (1ll << 32)) return ADAPT_ERR_INVALID_ARG;
    if (lens[l] > 0 && !tensors[l]) return ADAPT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(tensors[l]) & 3u) return ADAPT_ERR_INVALID_ARG;
  }
  const int n_levels = fmax + 1, C = grid->n_cand;
  DeviceCache* dc = nullptr;
  int rc = current_cache(&dc);
  if (rc != ADAPT_OK) return rc;
  unsigned char* ws = nullptr;
  rc = static_scratch_address(&ws);
  if (rc != ADAPT_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_handle);
  // the descriptor block below is re-read from a host array that the next call overwrites:
  // a captured copy of it would replay stale or foreign contents
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  ADAPT_CUDA(cudaStreamIsCapturing(stream, &capturing));
  if (capturing != cudaStreamCaptureStatusNone) {
    std::snprintf(g_last_error, sizeof(g_last_error),
                  "adapt_precision_search_static: the stream is being captured");
    return ADAPT_ERR_INVALID_ARG;
  }

  // descriptor block: layer list, candidates (slot = FL, order by (WL, FL, index)), fresh state
  unsigned char* h = g_static_blob;
  std::memset(h, 0, kStBlobEnd);
  LayerDesc* hl = reinterpret_cast<LayerDesc*>(h + kStLayers);
  long long tiles = 0;
  for (int l = 0; l < n_layers; ++l) {
    const int mis = static_cast<int>((reinterpret_cast<uintptr_t>(tensors[l]) >> 2) & 3u);
    hl[l].ptr = tensors[l]; hl[l].n = lens[l]; hl[l].tile_begin = tiles;
    hl[l].mis = lens[l] > 0 ? mis : 0; hl[l].layer_id = l; hl[l].index = l; hl[l].n_bins = n_bins;
    hl[l].via_plan = 0; hl[l].pad_ = 0;
    if (lens[l] > 0) tiles += (lens[l] + mis + kTile - 1) / kTile;
  }
  hl[n_layers].tile_begin = tiles;
  const int range_grid = plan_range_grid(hl, n_layers, tiles, dc->sm_count);
  int* h_wl = reinterpret_cast<int*>(h + kStWl);
  int* h_fl = reinterpret_cast<int*>(h + kStFl);
  int* h_slot = reinterpret_cast<int*>(h + kStSlot);
  int* h_order = reinterpret_cast<int*>(h + kStOrder);
  for (int c = 0; c < C; ++c) { h_wl[c] = grid->wl[c]; h_fl[c] = grid->fl[c]; h_slot[c] = grid->fl[c]; h_order[c] = c; }
  std::stable_sort(h_order, h_order + C, [&](int a, int b) {
    if (grid->wl[a] != grid->wl[b]) return grid->wl[a] < grid->wl[b];
    return grid->fl[a] < grid->fl[b];
  });
  int* h_by_fl = reinterpret_cast<int*>(h + kStByFl);
  int* h_fl_begin = reinterpret_cast<int*>(h + kStFlBegin);
  for (int c = 0; c < C; ++c) h_by_fl[c] = c;
  std::stable_sort(h_by_fl, h_by_fl + C, [&](int a, int b) { return grid->fl[a] < grid->fl[b]; });
  for (int c = 0; c < C; ++c) h_fl_begin[grid->fl[c] + 1] += 1;
  for (int f = 0; f < n_levels; ++f) h_fl_begin[f + 1] += h_fl_begin[f];
  LayerState* hs = reinterpret_cast<LayerState*>(h + kStState);
  for (int l = 0; l < n_layers; ++l) { hs[l].min_key = 0xFFFFFFFFu; hs[l].max_key = 0u; }

  // the block is ordinary host memory: the copy is staged before the call returns
  ADAPT_CUDA(cudaMemcpyAsync(ws, h, kStBlobEnd, cudaMemcpyHostToDevice, stream));
  // the scratch keeps the previous call's counts: clear every accumulator
  ADAPT_CUDA(cudaMemsetAsync(ws + kStZeros, 0, kStEnd - kStZeros, stream));
  const LayerDesc* d_layers = reinterpret_cast<const LayerDesc*>(ws + kStLayers);
  LayerState* d_state = reinterpret_cast<LayerState*>(ws + kStState);
  unsigned long long* d_zeros = reinterpret_cast<unsigned long long*>(ws + kStZeros);
  unsigned* d_q = reinterpret_cast<unsigned*>(ws + kStQ);
  unsigned* d_u = reinterpret_cast<unsigned*>(ws + kStU);

  {
    RangeParams rp;
    rp.layers = d_layers; rp.n_layers = n_layers; rp.n_tiles = tiles; rp.state = d_state;
    rp.range_out = nullptr;
    range_scan_kernel<<<range_grid, kRangeThreads, 0, stream>>>(rp);
    ADAPT_LAUNCH_OK("range scan launch");
    ++g_launches;
  }
  if (tiles > 0) {
    SearchParams sp;
    sp.layers = d_layers; sp.state = d_state; sp.n_layers = n_layers; sp.n_fl = n_levels;
    sp.n_bins = n_bins; sp.n_tiles = tiles; sp.q_hist = d_q; sp.u_hist = d_u; sp.zeros = d_zeros;
    sp.seed = 0; sp.plan = nullptr;
    const size_t per_hist = sizeof(unsigned) * n_bins;
    int fg = static_cast<int>((40 * 1024) / per_hist) - 1;   // stays under the 48 KB default limit
    fg = std::max(1, std::min(fg, n_levels));
    sp.fl_per_group = fg;
    const int groups = (n_levels + fg - 1) / fg;
    const size_t smem = per_hist * (fg + 1);
    dim3 g(static_cast<unsigned>(std::min<long long>(tiles, 4ll * dc->sm_count)), groups);
    // the other search calls leave their own dynamic shared-memory limit on this kernel
    // (possibly a smaller one): state the one this launch needs (not an allocation)
    ADAPT_CUDA(cudaFuncSetAttribute(search_direct_kernel<false>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    static_cast<int>(smem)));
    search_direct_kernel<false><<<g, kSearchThreads, smem, stream>>>(sp);
    ADAPT_LAUNCH_OK("direct search launch");
    ++g_launches;
  }
  KldParams kp;
  kp.layers = d_layers; kp.state = d_state;
  kp.cand_wl = reinterpret_cast<const int*>(ws + kStWl);
  kp.cand_fl = reinterpret_cast<const int*>(ws + kStFl);
  kp.cand_slot = reinterpret_cast<const int*>(ws + kStSlot);
  kp.cand_order = reinterpret_cast<const int*>(ws + kStOrder);
  kp.cand_by_fl = reinterpret_cast<const int*>(ws + kStByFl);
  kp.fl_begin = reinterpret_cast<const int*>(ws + kStFlBegin);
  kp.n_layers = n_layers; kp.n_cand = C; kp.n_fl = n_levels; kp.n_bins = n_bins;
  kp.q_hist = d_q; kp.u_hist = d_u; kp.zeros = d_zeros;
  kp.alpha = 0.0; kp.inv_ln_base = 1.0 / std::log(2.0); kp.eps = 0.0;
  kp.kld_out = kld_out; kp.zeros_out = reinterpret_cast<long long*>(zeros_out);
  kp.best_out = best_out; kp.hist_out = nullptr; kp.start = nullptr; kp.status_out = nullptr;
  kld_kernel<<<dim3(n_levels, n_layers), kKldThreads, 0, stream>>>(kp);
  ADAPT_LAUNCH_OK("kld launch");
  ++g_launches;
  return ADAPT_OK;
}

int adapt_bounds_check_status(uint32_t* out, int clear) {
  if (out) out[0] = out[1] = out[2] = out[3] = 0;
#ifdef ADAPT_CHECK_BOUNDS
  unsigned word[4] = {0, 0, 0, 0};
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpyFromSymbol(word, adapt::g_bounds_error, sizeof(word)) != cudaSuccess)
    return -ADAPT_ERR_CUDA;
  if (out) for (int i = 0; i < 4; ++i) out[i] = word[i];
  if (clear) {
    const unsigned zero[4] = {0, 0, 0, 0};
    if (cudaMemcpyToSymbol(adapt::g_bounds_error, zero, sizeof(zero)) != cudaSuccess) return -ADAPT_ERR_CUDA;
  }
  return 1;
#else
  (void)clear;
  return 0;
#endif
}

int adapt_release(void) {
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceCache* dc = nullptr;
  int rc = current_cache(&dc);
  if (rc != ADAPT_OK) return rc;
  ADAPT_CUDA(cudaDeviceSynchronize());
  if (dc->workspace) { ADAPT_CUDA(cudaFree(dc->workspace)); dc->workspace = nullptr; dc->workspace_bytes = 0; }
  if (dc->stage_in) { ADAPT_CUDA(cudaFree(dc->stage_in)); dc->stage_in = nullptr; dc->stage_in_bytes = 0; }
  if (dc->stage_out) { ADAPT_CUDA(cudaFree(dc->stage_out)); dc->stage_out = nullptr; dc->stage_out_bytes = 0; }
  if (dc->batch_tab) { ADAPT_CUDA(cudaFree(dc->batch_tab)); dc->batch_tab = nullptr; dc->batch_tab_bytes = 0; }
  dc->batch_tab_image.clear();
  if (dc->div_buf) { ADAPT_CUDA(cudaFree(dc->div_buf)); dc->div_buf = nullptr; dc->div_buf_bytes = 0; }
  if (dc->stage_codes) { ADAPT_CUDA(cudaFree(dc->stage_codes)); dc->stage_codes = nullptr; dc->stage_codes_bytes = 0; }
  if (dc->side_stream) {
    ADAPT_CUDA(cudaStreamDestroy(dc->side_stream)); dc->side_stream = nullptr;
    ADAPT_CUDA(cudaEventDestroy(dc->side_fork)); dc->side_fork = nullptr;
    ADAPT_CUDA(cudaEventDestroy(dc->side_join)); dc->side_join = nullptr;
  }
  if (dc->copy_stream) {
    ADAPT_CUDA(cudaStreamDestroy(dc->copy_stream)); dc->copy_stream = nullptr;
    for (cudaEvent_t& e : dc->slice_done) { ADAPT_CUDA(cudaEventDestroy(e)); e = nullptr; }
    ADAPT_CUDA(cudaEventDestroy(dc->copies_done)); dc->copies_done = nullptr;
  }
  for (PinnedSlot& s : dc->ring) {
    if (s.host) { ADAPT_CUDA(cudaFreeHost(s.host)); s.host = nullptr; s.bytes = 0; }
    if (s.done) { ADAPT_CUDA(cudaEventDestroy(s.done)); s.done = nullptr; }
  }
  return ADAPT_OK;
}

}  // extern "C"
