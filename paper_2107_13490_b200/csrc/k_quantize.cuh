// K4: stand-alone Quantize(L, <WL,FL>) writing int8 / int16 / int32 codes
// (Algorithm 1, the re-quantisation of each layer; Sec. 2.1 / 3.2).
// Streaming: 4 bytes read and 1/2/4 bytes written per element.
#pragma once

#include "common.cuh"

namespace adapt {

constexpr int kQuantThreads = 256;

template <typename T> struct Pack4;
template <> struct Pack4<int8_t>  { using type = char4;  };
template <> struct Pack4<int16_t> { using type = short4; };
template <> struct Pack4<int32_t> { using type = int4;   };

struct QuantParams {
  const float* x;
  void* out;
  long long n;
  int wl, fl;
  const int* selected;  // optional device {wl, fl, ...}: overrides wl/fl
  unsigned long long seed;
  int layer_id;
};

template <bool kStochastic>
__device__ __forceinline__ int quantize_one(float x, float two_fl, int wl, unsigned long long seed,
                                            int layer_id, long long i) {
  float pr = 0.0f;
  if (kStochastic) {
    unsigned h = hash24(seed, static_cast<unsigned long long>(layer_id),
                        static_cast<unsigned long long>(i));
    pr = __fmul_rn(__uint2float_rn(h), 5.9604644775390625e-8f);
  }
  return saturate_code(round_scaled<kStochastic>(x, two_fl, pr), wl);
}

// kVec: x is 16-byte aligned and out is aligned for a 4-element store; each
// thread then handles whole quads, the last (n % 4) elements go through the
// scalar tail.  Otherwise every element takes the scalar path.
template <typename T, bool kStochastic, bool kVec>
__global__ void __launch_bounds__(kQuantThreads) quantize_kernel(const QuantParams p) {
  int wl = p.wl, fl = p.fl;
  if (p.selected) { wl = p.selected[0]; fl = p.selected[1]; }
  if (wl < 2 || wl > 32 || fl < 0 || fl >= wl) return;  // never true for validated input
  const float two_fl = pow2f(fl);
  T* out = static_cast<T*>(p.out);
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (kVec) {
    using P4 = typename Pack4<T>::type;
    const long long nq = p.n >> 2;
    const float4* x4 = reinterpret_cast<const float4*>(p.x);
    P4* o4 = reinterpret_cast<P4*>(out);
    for (long long q = tid; q < nq; q += stride) {
      const float4 v = __ldcs(x4 + q);
      P4 c;
      c.x = static_cast<T>(quantize_one<kStochastic>(v.x, two_fl, wl, p.seed, p.layer_id, 4 * q + 0));
      c.y = static_cast<T>(quantize_one<kStochastic>(v.y, two_fl, wl, p.seed, p.layer_id, 4 * q + 1));
      c.z = static_cast<T>(quantize_one<kStochastic>(v.z, two_fl, wl, p.seed, p.layer_id, 4 * q + 2));
      c.w = static_cast<T>(quantize_one<kStochastic>(v.w, two_fl, wl, p.seed, p.layer_id, 4 * q + 3));
      __stcs(o4 + q, c);
    }
    for (long long i = (nq << 2) + tid; i < p.n; i += stride)
      out[i] = static_cast<T>(quantize_one<kStochastic>(p.x[i], two_fl, wl, p.seed, p.layer_id, i));
  } else {
    for (long long i = tid; i < p.n; i += stride)
      out[i] = static_cast<T>(quantize_one<kStochastic>(__ldcs(p.x + i), two_fl, wl, p.seed,
                                                        p.layer_id, i));
  }
}

// Batched form: every layer of a list is quantized at the <WL,FL> a search left on the
// device for it, in one launch (Algorithm 1: for l in L: L^[l] = Quantize(L[l], Q[l].quant)).
struct QuantLayer {
  const float* x;
  void* out;              // int8 / int16 / int32 codes, or fp32 dequantized values
  long long n;
  long long tile_begin;   // first tile of the layer in the launch's tile list (4096 elements each)
  int layer_id;           // hash layer id
  int vec;                // x is 16-byte aligned and out aligned for a 4-element store
  int select;             // row of `best` (and of `unfit`) that holds this entry's <WL,FL>
  int pad_;
  long long index_base;   // element index of x[0] inside its layer (an entry may be a slice of one)
};

constexpr int kQuantTile = 4096;

// Output of the batched kernel: int32 / int16 / int8 codes, or (float) the dequantized values
// code * 2^-FL as fp32 - the tensor a float32 simulation of fixed-point training goes on with
// (Sec. 4.1); the float output may be x itself (every element is read and written by the same
// thread).  A layer whose selected word length does not fit the code type is left untouched
// and, if `unfit` is given, reported there (unfit[layer] = its word length).
template <typename T> struct Pack4;
template <> struct Pack4<float> { using type = float4; };

template <typename T>
__device__ __forceinline__ T quant_out(int code, int fl) { return static_cast<T>(code); }
template <>
__device__ __forceinline__ float quant_out<float>(int code, int fl) { return dequantize(code, fl); }

template <bool kStochastic, typename T>
__global__ void __launch_bounds__(kQuantThreads)
quantize_batch_kernel(const QuantLayer* __restrict__ layers, int n_layers, long long n_tiles,
                      const int* __restrict__ best, unsigned long long seed, int* __restrict__ unfit) {
  grid_dependency_wait();
  constexpr int kBits = sizeof(T) == 1 ? 8 : (sizeof(T) == 2 ? 16 : 32);   // float carries any code
  for (long long t = blockIdx.x; t < n_tiles; t += gridDim.x) {
    int lo = 0, hi = n_layers - 1;                 // layer that owns tile t
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (layers[mid].tile_begin <= t) lo = mid; else hi = mid - 1;
    }
    const QuantLayer L = layers[lo];
    const int wl = best[4 * L.select], fl = best[4 * L.select + 1];
    if (wl < 2 || wl > 32 || fl < 0 || fl >= wl) continue;   // layer without a valid selection
    if (wl > kBits) {
      if (unfit && t == L.tile_begin && threadIdx.x == 0) unfit[L.select] = wl;
      continue;
    }
    const float two_fl = pow2f(fl);
    const long long i0 = (t - L.tile_begin) * kQuantTile;
    const long long i1 = min(L.n, i0 + kQuantTile);
    T* out = static_cast<T*>(L.out);
    if (L.vec && i1 - i0 == kQuantTile) {
      using P4 = typename Pack4<T>::type;
      const float4* x4 = reinterpret_cast<const float4*>(L.x + i0);
      P4* o4 = reinterpret_cast<P4*>(out + i0);
      for (int q = threadIdx.x; q < kQuantTile / 4; q += kQuantThreads) {
        const float4 v = __ldcs(x4 + q);
        const long long i = L.index_base + i0 + 4ll * q;
        P4 c;
        c.x = quant_out<T>(quantize_one<kStochastic>(v.x, two_fl, wl, seed, L.layer_id, i + 0), fl);
        c.y = quant_out<T>(quantize_one<kStochastic>(v.y, two_fl, wl, seed, L.layer_id, i + 1), fl);
        c.z = quant_out<T>(quantize_one<kStochastic>(v.z, two_fl, wl, seed, L.layer_id, i + 2), fl);
        c.w = quant_out<T>(quantize_one<kStochastic>(v.w, two_fl, wl, seed, L.layer_id, i + 3), fl);
        __stcs(o4 + q, c);
      }
    } else {
      for (long long i = i0 + threadIdx.x; i < i1; i += kQuantThreads)
        out[i] = quant_out<T>(quantize_one<kStochastic>(__ldcs(L.x + i), two_fl, wl, seed, L.layer_id,
                                                        L.index_base + i), fl);
    }
  }
}

}  // namespace adapt
