// Shared device helpers for the TensorGRaD step kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace tg {

typedef float2 cf;   // complex fp32: x = re, y = im

__device__ __forceinline__ cf cmul(cf a, cf b) { return make_float2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x); }
// acc += a * b
__device__ __forceinline__ void cfma(cf& acc, cf a, cf b) {
  acc.x = fmaf(a.x, b.x, acc.x); acc.x = fmaf(-a.y, b.y, acc.x);
  acc.y = fmaf(a.x, b.y, acc.y); acc.y = fmaf(a.y, b.x, acc.y);
}
// acc += a * conj(b)
__device__ __forceinline__ void cfma_conj(cf& acc, cf a, cf b) {
  acc.x = fmaf(a.x, b.x, acc.x); acc.x = fmaf(a.y, b.y, acc.x);
  acc.y = fmaf(a.y, b.x, acc.y); acc.y = fmaf(-a.x, b.y, acc.y);
}

// Storage adaptors for W and G: interleaved 2 x fp32, 2 x fp16 or 2 x bfloat16.  widen() is exact; narrow() rounds
// to nearest even (the identity for fp32).
struct StoreC64 {
  typedef float2 elem;
  static constexpr int kBytes = 8;
  static constexpr bool kBf16 = false;
  __device__ static __forceinline__ cf widen(const elem& e) { return e; }
  __device__ static __forceinline__ cf narrow(cf v) { return v; }
  __device__ static __forceinline__ cf load(const void* p, size_t i) { return reinterpret_cast<const float2*>(p)[i]; }
  __device__ static __forceinline__ void store(void* p, size_t i, cf v) { reinterpret_cast<float2*>(p)[i] = v; }
};
struct StoreC32H {
  typedef __half2 elem;
  static constexpr int kBytes = 4;
  static constexpr bool kBf16 = false;
  __device__ static __forceinline__ cf widen(const elem& e) { return __half22float2(e); }
  __device__ static __forceinline__ cf narrow(cf v) { return __half22float2(__floats2half2_rn(v.x, v.y)); }
  __device__ static __forceinline__ cf load(const void* p, size_t i) {
    return __half22float2(reinterpret_cast<const __half2*>(p)[i]);
  }
  __device__ static __forceinline__ void store(void* p, size_t i, cf v) {
    reinterpret_cast<__half2*>(p)[i] = __floats2half2_rn(v.x, v.y);
  }
};

struct StoreC32B {
  typedef __nv_bfloat162 elem;
  static constexpr int kBytes = 4;
  static constexpr bool kBf16 = true;
  __device__ static __forceinline__ cf widen(const elem& e) { return __bfloat1622float2(e); }
  __device__ static __forceinline__ cf narrow(cf v) { return __bfloat1622float2(__floats2bfloat162_rn(v.x, v.y)); }
  __device__ static __forceinline__ cf load(const void* p, size_t i) {
    return __bfloat1622float2(reinterpret_cast<const __nv_bfloat162*>(p)[i]);
  }
  __device__ static __forceinline__ void store(void* p, size_t i, cf v) {
    reinterpret_cast<__nv_bfloat162*>(p)[i] = __floats2bfloat162_rn(v.x, v.y);
  }
};

// Magnitude key of the top-k selection: fl(fl(re*re) + fl(im*im)) in fp32 with
// no fused multiply-add; for non-negative floats the bit pattern orders like
// the value.
__device__ __forceinline__ uint32_t mag_key(cf v) {
  return __float_as_uint(__fadd_rn(__fmul_rn(v.x, v.x), __fmul_rn(v.y, v.y)));
}

__device__ __forceinline__ int lower_bound_u32(const uint32_t* __restrict__ a, int n, uint32_t key) {
  int lo = 0, hi = n;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (a[mid] < key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

}  // namespace tg
