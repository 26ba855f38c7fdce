// CUDA-core convolution kernels: fp32 implicit GEMM (the fp32 model path, and layers whose
// channel counts no tensor-core tile covers, e.g. a 3-channel stem), depthwise 3x3 and max-pool.
//
// The convolution is the product of the implicit Toeplitz matrix A [M = B*Ho*Wo][K = kh*kw*Cin]
// with the weight matrix W [N = Cout][K] (paper Section II-C); A is never materialised.
// Every output sums its K terms in ascending k with fp32 FMAs, independent of the batch size,
// so a sample's result does not depend on which batch it rides in.
#pragma once
#include "common.cuh"

namespace ee {

struct ConvGeom {
  int B, H, W, Cin, Ho, Wo, Cout, kh, kw, stride, pad, act;
};

constexpr int kSimtBM = 64, kSimtBN = 64, kSimtBK = 16, kSimtThreads = 256, kSimtPad = 4;

template <typename T>
__global__ void __launch_bounds__(kSimtThreads)
conv_igemm_simt_kernel(const T* __restrict__ x, const T* __restrict__ w, const float* __restrict__ scale,
                       const float* __restrict__ bias, const T* __restrict__ residual, T* __restrict__ y, ConvGeom g) {
  __shared__ __align__(16) float As[kSimtBK][kSimtBM + kSimtPad];
  __shared__ __align__(16) float Bs[kSimtBK][kSimtBN + kSimtPad];
  const int t = threadIdx.x;
  const long M = (long)g.B * g.Ho * g.Wo;
  const int N = g.Cout, K = g.kh * g.kw * g.Cin;
  const long m0 = (long)blockIdx.x * kSimtBM;
  const int n0 = blockIdx.y * kSimtBN;

  // this thread's four A rows (fixed for the whole K loop)
  const int kk = t & 15, rb = t >> 4;
  long a_base[4];
  int a_hi0[4], a_wi0[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long m = m0 + rb + 16 * i;
    if (m < M) {
      const int wo = (int)(m % g.Wo);
      const long q = m / g.Wo;
      const int ho = (int)(q % g.Ho);
      const long b = q / g.Ho;
      a_base[i] = b * g.H * g.W;
      a_hi0[i] = ho * g.stride - g.pad;
      a_wi0[i] = wo * g.stride - g.pad;
    } else {
      a_base[i] = -1;
      a_hi0[i] = a_wi0[i] = 0;
    }
  }

  const int tx = t & 15, ty = t >> 4;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += kSimtBK) {
    const int k = k0 + kk;
    int r = 0, s = 0, ci = 0;
    const bool kin = k < K;
    if (kin) {
      const int tap = k / g.Cin;
      ci = k - tap * g.Cin;
      r = tap / g.kw;
      s = tap - r * g.kw;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float v = 0.f;
      if (kin && a_base[i] >= 0) {
        const int hi = a_hi0[i] + r, wi = a_wi0[i] + s;
        if (hi >= 0 && hi < g.H && wi >= 0 && wi < g.W) v = Elem<T>::ld(x + ((a_base[i] + (long)hi * g.W + wi) * g.Cin + ci));
      }
      As[kk][rb + 16 * i] = v;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int n = n0 + rb + 16 * i;
      Bs[kk][rb + 16 * i] = (kin && n < N) ? Elem<T>::ld(w + (long)n * K + k) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < kSimtBK; ++q) {
      const float4 a = *reinterpret_cast<const float4*>(&As[q][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Bs[q][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= N) continue;
      float v = fmaf(scale ? scale[n] : 1.f, acc[i][j], bias ? bias[n] : 0.f);
      if (residual) v += Elem<T>::ld(residual + m * N + n);
      Elem<T>::st(y + m * N + n, apply_act(v, g.act));
    }
  }
}

// Depthwise k x k convolution, NHWC, one thread per (output pixel, 16-byte channel vector).
// Weights [C][kh][kw]; taps summed in ascending (r, s) with fp32 FMAs.
template <typename T, int VEC>
__global__ void __launch_bounds__(256)
dwconv_kernel(const T* __restrict__ x, const T* __restrict__ w, const float* __restrict__ scale,
              const float* __restrict__ bias, T* __restrict__ y, ConvGeom g) {
  const int cv = g.Cin / VEC;
  const long total = (long)g.B * g.Ho * g.Wo * cv;
  for (long idx = (long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % cv) * VEC;
    long p = idx / cv;
    const int wo = (int)(p % g.Wo);
    p /= g.Wo;
    const int ho = (int)(p % g.Ho);
    const long b = p / g.Ho;
    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
    for (int r = 0; r < g.kh; ++r) {
      const int hi = ho * g.stride - g.pad + r;
      if (hi < 0 || hi >= g.H) continue;
      for (int s = 0; s < g.kw; ++s) {
        const int wi = wo * g.stride - g.pad + s;
        if (wi < 0 || wi >= g.W) continue;
        const T* xp = x + ((b * g.H + hi) * g.W + wi) * g.Cin + c;
        if constexpr (VEC > 1) {
          Vec16<T> xv;
          xv.load(xp);
#pragma unroll
          for (int e = 0; e < VEC; ++e) acc[e] = fmaf(xv.v[e], Elem<T>::ld(w + ((long)(c + e) * g.kh + r) * g.kw + s), acc[e]);
        } else {
          acc[0] = fmaf(Elem<T>::ld(xp), Elem<T>::ld(w + ((long)c * g.kh + r) * g.kw + s), acc[0]);
        }
      }
    }
    T* yp = y + ((b * g.Ho + ho) * g.Wo + wo) * g.Cout + c;
    if constexpr (VEC > 1) {
      Vec16<T> o;
#pragma unroll
      for (int e = 0; e < VEC; ++e) o.v[e] = apply_act(fmaf(scale ? scale[c + e] : 1.f, acc[e], bias ? bias[c + e] : 0.f), g.act);
      o.store(yp);
    } else {
      Elem<T>::st(yp, apply_act(fmaf(scale ? scale[c] : 1.f, acc[0], bias ? bias[c] : 0.f), g.act));
    }
  }
}

// Window maximum over in-range taps, NHWC, one thread per (output pixel, channel vector).
template <typename T, int VEC>
__global__ void __launch_bounds__(256)
maxpool_kernel(const T* __restrict__ x, T* __restrict__ y, ConvGeom g) {
  const int cv = g.Cin / VEC;
  const long total = (long)g.B * g.Ho * g.Wo * cv;
  for (long idx = (long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % cv) * VEC;
    long p = idx / cv;
    const int wo = (int)(p % g.Wo);
    p /= g.Wo;
    const int ho = (int)(p % g.Ho);
    const long b = p / g.Ho;
    float m[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) m[e] = -INFINITY;
    for (int r = 0; r < g.kh; ++r) {
      const int hi = ho * g.stride - g.pad + r;
      if (hi < 0 || hi >= g.H) continue;
      for (int s = 0; s < g.kw; ++s) {
        const int wi = wo * g.stride - g.pad + s;
        if (wi < 0 || wi >= g.W) continue;
        const T* xp = x + ((b * g.H + hi) * g.W + wi) * g.Cin + c;
        if constexpr (VEC > 1) {
          Vec16<T> xv;
          xv.load(xp);
#pragma unroll
          for (int e = 0; e < VEC; ++e) m[e] = fmaxf(m[e], xv.v[e]);
        } else {
          m[0] = fmaxf(m[0], Elem<T>::ld(xp));
        }
      }
    }
    T* yp = y + ((b * g.Ho + ho) * g.Wo + wo) * g.Cin + c;
    if constexpr (VEC > 1) {
      Vec16<T> o;
#pragma unroll
      for (int e = 0; e < VEC; ++e) o.v[e] = m[e];
      o.store(yp);
    } else {
      Elem<T>::st(yp, m[0]);
    }
  }
}

}  // namespace ee
