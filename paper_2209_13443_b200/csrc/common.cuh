// Shared device/host helpers of the early-exit CNN library (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ee.h"

namespace ee {

typedef __nv_bfloat16 bf16;

template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kVec = 4;  // elements per 16-byte access
  __device__ __forceinline__ static float ld(const float* p) { return *p; }
  __device__ __forceinline__ static void st(float* p, float v) { *p = v; }
};
template <> struct Elem<bf16> {
  static constexpr int kVec = 8;
  __device__ __forceinline__ static float ld(const bf16* p) { return __bfloat162float(*p); }
  __device__ __forceinline__ static void st(bf16* p, float v) { *p = __float2bfloat16_rn(v); }
};

// 16 bytes of T as floats.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  float v[4];
  __device__ __forceinline__ void load(const float* p) {
    float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
  __device__ __forceinline__ void store(float* p) const { *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]); }
};
template <> struct Vec16<bf16> {
  float v[8];
  __device__ __forceinline__ void load(const bf16* p) {
    uint4 t = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {  // bf16 -> f32 is a 16-bit shift
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ __forceinline__ void store(bf16* p) const {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

// Accumulator type of the CUDA-core kernels: the fp32 model sums in fp64 (products of two floats are exact in a double,
// so a sum is rounded once, to fp32, at the store: the 1e-5 parity bar then holds for every element, however small
// against its tensor); bf16 models sum in fp32 (their bar is the bf16 rounding of the result).
template <typename T> struct Accum { typedef float type; };
template <> struct Accum<float> { typedef double type; };
__device__ __forceinline__ float acc_fma(float a, float b, float c) { return fmaf(a, b, c); }
__device__ __forceinline__ double acc_fma(float a, float b, double c) { return fma((double)a, (double)b, c); }
__device__ __forceinline__ double apply_act(double v, int act) {
  if (act == EE_ACT_RELU) return fmax(v, 0.0);
  if (act == EE_ACT_RELU6) return fmin(fmax(v, 0.0), 6.0);
  return v;
}

__device__ __forceinline__ float apply_act(float v, int act) {
  if (act == EE_ACT_RELU) return fmaxf(v, 0.f);
  if (act == EE_ACT_RELU6) return fminf(fmaxf(v, 0.f), 6.f);
  return v;
}

static inline int cdiv(long a, long b) { return (int)((a + b - 1) / b); }
static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace ee
