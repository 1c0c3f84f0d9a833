// Shared device helpers of the precision-switch search kernels (sm_100a).
//
// Every floating-point step that decides an integer (a code, a bin) is a
// single IEEE fp32 round-to-nearest operation written with an explicit
// intrinsic, so the compiler can neither contract it into an FMA nor
// reassociate it.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace adapt {

constexpr int kMaxFl = 32;  // FL in 0..31
constexpr int kTile = 4096; // elements per tile of the range scan and the direct kernels (in aligned indexing)

// LayerState::flags (the same bits as ADAPT_FLAG_* of the C interface)
constexpr unsigned kFlagDegenerate = 2u;
constexpr unsigned kFlagNonfinite = 4u;
constexpr unsigned kFlagRange = 8u;

// Per-layer descriptor, written by the host into the workspace.
struct LayerDesc {
  const float* ptr;      // first element (4-byte aligned)
  long long n;           // elements
  long long tile_begin;  // index of the layer's first tile in the global tile list
  int mis;               // elements between the 16-byte boundary below ptr and ptr (0..3)
  int layer_id;          // hash layer id
  int index;             // position in the caller's tensor list (addresses state and outputs)
  int n_bins;            // bins of this layer's histograms (<= the stride the arrays use)
  int range_ctas;        // CTAs of the range scan that hold tiles of this layer (set by the host for
                         // the list that kernel walks; the last of them to finish settles the layer)
  int via_plan;          // direct kernel's list: 1 = the layer also stands in the stochastic-rounding
                         // kernel's list and is served here only if its plan says "not keyed"
  int pad_;
};

// Per-layer state produced on the device by the range scan.
struct LayerState {
  unsigned min_key;  // order-preserving image of the minimum
  unsigned max_key;  // ... of the maximum
  unsigned flags;    // ADAPT_FLAG_NONFINITE / ADAPT_FLAG_RANGE / ADAPT_FLAG_DEGENERATE
  float lo, hi, scale, bmax;
  unsigned pad_;
  unsigned zero_count;  // estimate of the exact zeros (the range scan samples one element in
                        // eight; steers the choice of loop form only, never results)
  unsigned ticket;      // range scan: CTAs that have added their part of this layer (the last one
                        // turns the extremes into the bin origin and scale)
  unsigned kld_ticket;  // divergence kernel: CTAs that have written their candidates of this layer
                        // (the last one selects the layer's format)
};

// Index checks of the bounds-checking build (-DADAPT_CHECK_BOUNDS; the stand-in for a memory
// checker): every table index that is formed from the data - a cell position from a float's
// bit pattern, a bin, a sub-cell, a queue slot - goes through ADAPT_IN_BOUNDS, which in that
// build skips an access outside [0, limit) and records the first such event in a device word
// that adapt_bounds_check_status returns; nothing traps.  In the normal build the macro is
// `true` and the checks cost nothing.
#ifdef ADAPT_CHECK_BOUNDS
__device__ unsigned g_bounds_error[4];   // {events, site of the first, its index, its limit}
__device__ __forceinline__ bool index_in_bounds(long long idx, long long limit, int site) {
  if (idx >= 0 && idx < limit) return true;
  if (atomicAdd(&g_bounds_error[0], 1u) == 0u) {
    g_bounds_error[1] = static_cast<unsigned>(site);
    g_bounds_error[2] = static_cast<unsigned>(idx);
    g_bounds_error[3] = static_cast<unsigned>(limit);
  }
  return false;
}
#define ADAPT_IN_BOUNDS(idx, limit, site) \
  ::adapt::index_in_bounds(static_cast<long long>(idx), static_cast<long long>(limit), (site))
#else
#define ADAPT_IN_BOUNDS(idx, limit, site) true
#endif

// Shared-memory atomics by 32-bit shared address.  A table pointer that a kernel keeps in a
// context structure is a generic pointer to the compiler, and atomics through generic pointers
// are far slower than the shared-memory forms; kernels therefore keep shared addresses
// (smem_addr of the table's first word) and add byte offsets.
__device__ __forceinline__ unsigned smem_addr(const void* p) {
  return static_cast<unsigned>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned smem_atom_add(unsigned addr, unsigned v) {
  unsigned o;
  asm volatile("atom.shared.add.u32 %0, [%1], %2;" : "=r"(o) : "r"(addr), "r"(v) : "memory");
  return o;
}
__device__ __forceinline__ void smem_red_add(unsigned addr, unsigned v) {
  asm volatile("red.shared.add.u32 [%0], %1;" :: "r"(addr), "r"(v) : "memory");
}

// A kernel that may be launched with programmatic stream serialization (its CTAs may become
// resident while the kernel before it in the stream is still draining) calls this before it
// touches anything that kernel wrote: it returns once the earlier grid has completed and its
// writes are visible.  Without the launch attribute it returns at once.
__device__ __forceinline__ void grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Adds the u32 words of a shared-memory array to a global array through the bulk-copy engine
// (cp.reduce.async.bulk: the addition happens at the L2, no thread touches the words).  Both
// addresses are 16-byte aligned and n_bytes is a multiple of 16.  Called by one thread, after a
// barrier behind the last ordinary write to the array; the caller commits the group and waits for
// it (bulk_reduce_wait_read) before the array is written again.
__device__ __forceinline__ void bulk_reduce_add_u32(unsigned* dst, unsigned smem_src, unsigned n_bytes) {
  const unsigned long long gdst = static_cast<unsigned long long>(__cvta_generic_to_global(dst));
  constexpr unsigned kPiece = 32768u;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  for (unsigned at = 0; at < n_bytes; at += kPiece) {
    const unsigned len = min(kPiece, n_bytes - at);
    asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.u32 [%0], [%1], %2;"
                 :: "l"(gdst + at), "r"(smem_src + at), "r"(len) : "memory");
  }
}
__device__ __forceinline__ void bulk_reduce_commit() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// The engine has read the shared-memory sources of every committed group (they may be reused).
__device__ __forceinline__ void bulk_reduce_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
// Every committed group is complete.
__device__ __forceinline__ void bulk_reduce_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// Monotone map float -> uint32 (a < b  <=>  key(a) < key(b) for non-NaN a, b).
__device__ __forceinline__ unsigned float_key(float v) {
  unsigned b = __float_as_uint(v);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_float(unsigned k) {
  unsigned b = (k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k;
  return __uint_as_float(b);
}

// Index of the bin of value v among the shared equal-width bins (Sec. 3.3):
// floor((v - lo) * scale) clamped to [0, n_bins-1], scale = n_bins / (hi - lo).
// fmaxf returns its non-NaN operand, so 0 * inf lands in bin 0.
__device__ __forceinline__ int bin_of(float v, float lo, float scale, float bmax) {
  float t = __fsub_rn(v, lo);
  float u = __fmul_rn(t, scale);
  float bf = floorf(u);
  bf = fmaxf(bf, 0.0f);
  bf = fminf(bf, bmax);
  return __float2int_rz(bf);
}

// 2^e for -126 <= e <= 127 by exponent-field construction.
__device__ __forceinline__ float pow2f(int e) {
  return __uint_as_float(static_cast<unsigned>(e + 127) << 23);
}

// Counter hash (seed, layer, element index) -> 24 uniform bits; P = k * 2^-24.
__device__ __forceinline__ unsigned hash24(unsigned long long seed, unsigned long long layer,
                                           unsigned long long index) {
  const unsigned long long c1 = 0x9E3779B97F4A7C15ull;
  const unsigned long long c2 = 0x6A09E667F3BCC909ull;
  const unsigned long long c3 = 0xBB67AE8584CAA73Bull;
  unsigned long long z = seed ^ ((layer + 1ull) * c1);
  z += index * c2;
  z ^= z >> 32;
  z *= c1;
  z ^= z >> 29;
  z *= c3;
  z ^= z >> 32;
  return static_cast<unsigned>(z >> 40);
}

// Unsaturated rounded value of x * 2^FL (an integer held in a float).
// RNE: ties to even.  Stochastic (Sec. 3.2, SR(x)): floor + (P < y - floor(y)).
template <bool kStochastic>
__device__ __forceinline__ float round_scaled(float x, float two_fl, float p) {
  float y = __fmul_rn(x, two_fl);
  if (!kStochastic) return rintf(y);
  float f = floorf(y);
  float frac = __fsub_rn(y, f);
  return (p < frac) ? __fadd_rn(f, 1.0f) : f;
}

// Two's-complement saturation of an integral float r to WL bits.
__device__ __forceinline__ int saturate_code(float r, int wl) {
  float top = pow2f(wl - 1);
  int hi_code = static_cast<int>((1ll << (wl - 1)) - 1);
  int lo_code = static_cast<int>(-(1ll << (wl - 1)));
  if (r >= top) return hi_code;
  if (r <= -top) return lo_code;
  return __float2int_rz(r);
}

__device__ __forceinline__ float dequantize(int code, int fl) {
  return __fmul_rn(__int2float_rn(code), pow2f(-fl));
}

// Loads the four elements j0..j0+3 of a layer in "aligned" indexing: j counts
// from the 16-byte boundary at or below the layer's first element, the layer
// owns j in [jbeg, jend).  Interior quads use one 128-bit load; quads that
// straddle an end fall back to guarded scalar loads.  Returns the mask of
// valid elements (bit k = element j0+k); invalid slots hold 0.
__device__ __forceinline__ unsigned load_quad(const float* aligned_base, long long j0,
                                              long long jbeg, long long jend, float (&v)[4]) {
  if (j0 >= jbeg && j0 + 4 <= jend) {
    float4 q = __ldg(reinterpret_cast<const float4*>(aligned_base + j0));
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
    return 0xFu;
  }
  unsigned m = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    long long j = j0 + k;
    bool ok = (j >= jbeg) && (j < jend);
    v[k] = ok ? __ldg(aligned_base + j) : 0.0f;
    m |= ok ? (1u << k) : 0u;
  }
  return m;
}

// Finds the layer that owns global tile t (tile_begin is ascending; the entry
// after the last layer holds the total tile count).
__device__ __forceinline__ int layer_of_tile(const LayerDesc* layers, int n_layers, long long t) {
  int lo = 0, hi = n_layers - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (layers[mid].tile_begin <= t) lo = mid; else hi = mid - 1;
  }
  return lo;
}

}  // namespace adapt
