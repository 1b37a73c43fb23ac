// Shared device helpers for the sparse FFN decode kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace ls {

constexpr int WD_BF16 = 0;
constexpr int WD_FP16 = 1;

// Device-side status codes recorded by kernels (mirrors the LS_ERR_* values of the public header).
constexpr int ST_OK = 0;
constexpr int ST_BAD_INDEX = -1;
constexpr int ST_CAPACITY = -5;
constexpr int ST_TIMEOUT = -6;
constexpr int ST_INTERNAL = -7;

__device__ __forceinline__ void set_status(int* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

// Eight consecutive 16-bit weights (one 128-bit load) widened exactly to fp32.
template <int WD>
__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (WD == WD_BF16) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    } else {
      const __half2 h = *reinterpret_cast<const __half2*>(&w[i]);
      const float2 t = __half22float2(h);
      f[2 * i] = t.x;
      f[2 * i + 1] = t.y;
    }
  }
}

__device__ __forceinline__ uint4 ldg128(const void* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }

// Streaming 128-bit load: weight rows are read once per token, keep them out of L1.
__device__ __forceinline__ uint4 ld_stream128(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Score canonicalisation for ranking: NaN ranks last (as -inf), -0.0 and +0.0 are one value.
__device__ __forceinline__ double canonical_score(double s) {
  if (s != s) return __longlong_as_double((long long)0xfff0000000000000ULL);  // -inf
  return s + 0.0;
}
// Order-preserving map of a canonical fp64 score to an unsigned 64-bit key (larger score -> larger key).
__device__ __forceinline__ unsigned long long ordered_key(double s) {
  const unsigned long long b = (unsigned long long)__double_as_longlong(s);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ULL);
}

// Rank range of stage c of K over `count` ranked entries: m = ceil(count/K) entries per stage.
__device__ __forceinline__ void stage_bounds(int count, int K, int c, int& lo, int& hi) {
  const int m = count > 0 ? (count + K - 1) / K : 0;
  lo = min(count, c * m);
  hi = min(count, (c + 1) * m);
}

}  // namespace ls
