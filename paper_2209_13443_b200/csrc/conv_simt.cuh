// CUDA-core convolution kernels: fp32 implicit GEMM (the fp32 model path, and layers whose
// channel counts no tensor-core tile covers, e.g. a 3-channel stem), depthwise 3x3 and max-pool.
//
// The convolution is the product of the implicit Toeplitz matrix A [M = B*Ho*Wo][K = kh*kw*Cin]
// with the weight matrix W [N = Cout][K] (paper Section II-C); A is never materialised.
// Every output sums its K terms in ascending k (fp32 FMAs for bf16 models, fp64 for the fp32 model: see Accum),
// independent of the batch size, so a sample's result does not depend on which batch it rides in.
#pragma once
#include "common.cuh"

namespace ee {

struct ConvGeom {
  int B, H, W, Cin, Ho, Wo, Cout, kh, kw, stride, pad, pad_w, act;   // pad: rows, pad_w: columns (equal except for dense convolutions)
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
      a_wi0[i] = wo * g.stride - g.pad_w;
    } else {
      a_base[i] = -1;
      a_hi0[i] = a_wi0[i] = 0;
    }
  }

  const int tx = t & 15, ty = t >> 4;
  typedef typename Accum<T>::type A;
  A acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = (A)0;

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
        for (int j = 0; j < 4; ++j) acc[i][j] = acc_fma(av[i], bv[j], acc[i][j]);
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
      A v = (A)(scale ? scale[n] : 1.f) * acc[i][j] + (A)(bias ? bias[n] : 0.f);   // float: one FMA; double: exact product, one add
      if (residual) v += (A)Elem<T>::ld(residual + m * N + n);
      Elem<T>::st(y + m * N + n, (float)apply_act(v, g.act));
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
    typedef typename Accum<T>::type A;
    A acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = (A)0;
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
          for (int e = 0; e < VEC; ++e) acc[e] = acc_fma(xv.v[e], Elem<T>::ld(w + ((long)(c + e) * g.kh + r) * g.kw + s), acc[e]);
        } else {
          acc[0] = acc_fma(Elem<T>::ld(xp), Elem<T>::ld(w + ((long)c * g.kh + r) * g.kw + s), acc[0]);
        }
      }
    }
    T* yp = y + ((b * g.Ho + ho) * g.Wo + wo) * g.Cout + c;
    if constexpr (VEC > 1) {
      Vec16<T> o;
#pragma unroll
      for (int e = 0; e < VEC; ++e)
        o.v[e] = (float)apply_act((A)(scale ? scale[c + e] : 1.f) * acc[e] + (A)(bias ? bias[c + e] : 0.f), g.act);
      o.store(yp);
    } else {
      Elem<T>::st(yp, (float)apply_act((A)(scale ? scale[c] : 1.f) * acc[0] + (A)(bias ? bias[c] : 0.f), g.act));
    }
  }
}

// Depthwise 3x3 pad-1 convolution on bf16, stride 1 or 2: the layers of the inverted-residual blocks.  The kernel
// above issues one 2-byte load per (tap, channel) for the weights and one 16-byte load per tap for the input: 81
// loads for 72 FMAs, which makes the load/store units, not memory, the bound.  Here a thread owns one vector of
// eight channels for its whole life: it reads that vector's 72 weights once (144 contiguous bytes of the
// [C][3][3] array) and keeps them in registers as stored, then walks items of kDwStrip consecutive output pixels of one
// output row.  Per item it requests all 3 x ((kDwStrip - 1) * STRIDE + 3) input vectors up front (enough bytes in
// flight per SM to cover the memory latency) and uses each for every output it overlaps.  Every output still sums its nine taps in ascending (r, s) with fp32 FMAs.
// Block (x, y): x runs over channel vectors (adjacent threads read adjacent 16-byte vectors), y over items.
constexpr int kDwStrip = 4;

template <int STRIDE>
__global__ void __launch_bounds__(256)
dwconv3x3_bf16_kernel(const bf16* __restrict__ x, const bf16* __restrict__ w, const float* __restrict__ scale,
                      const float* __restrict__ bias, bf16* __restrict__ y, ConvGeom g, int strips) {
  constexpr int P = kDwStrip, COLS = (P - 1) * STRIDE + 3;
  const int cv = g.Cin / 8;
  const int c8 = blockIdx.y * blockDim.x + threadIdx.x;
  if (c8 >= cv) return;
  const int c = c8 * 8;
  uint32_t raw[36];   // the vector's 72 weights as stored: element e = channel e / 9, tap e % 9
  {
    const uint4* wp = reinterpret_cast<const uint4*>(w + (size_t)c * 9);   // 9 x 16 bytes, 16-byte aligned
#pragma unroll
    for (int i = 0; i < 9; ++i) {
      const uint4 v = __ldg(wp + i);
      raw[4 * i] = v.x, raw[4 * i + 1] = v.y, raw[4 * i + 2] = v.z, raw[4 * i + 3] = v.w;
    }
  }
  auto weight = [&](int tap, int ch) {   // indices are compile-time constants after unrolling
    const int e = ch * 9 + tap;
    return (e & 1) ? __uint_as_float(raw[e >> 1] & 0xffff0000u) : __uint_as_float(raw[e >> 1] << 16);
  };
  float sc[8], bi[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    sc[e] = scale ? scale[c + e] : 1.f;
    bi[e] = bias ? bias[c + e] : 0.f;
  }
  const long items = (long)g.B * g.Ho * strips;
  for (long item = (long)blockIdx.x * blockDim.y + threadIdx.y; item < items; item += (long)gridDim.x * blockDim.y) {
    const int st = (int)(item % strips);
    const long t = item / strips;
    const int ho = (int)(t % g.Ho);
    const long b = t / g.Ho;
    const int wo0 = st * P;
    const int hi0 = ho * STRIDE - 1, wi0 = wo0 * STRIDE - 1;
    float acc[P][8];
#pragma unroll
    for (int pp = 0; pp < P; ++pp)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[pp][e] = 0.f;
    uint4 v[3][COLS];   // every input vector of the item is requested before the first FMA
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      const int hi = hi0 + r;
      const bool row_in = hi >= 0 && hi < g.H;
      const bf16* row = x + ((b * g.H + (row_in ? hi : 0)) * g.W) * (long)g.Cin + c;
#pragma unroll
      for (int j = 0; j < COLS; ++j) {
        const int wi = wi0 + j;
        v[r][j] = (row_in && wi >= 0 && wi < g.W) ? __ldg(reinterpret_cast<const uint4*>(row + (long)wi * g.Cin)) : make_uint4(0u, 0u, 0u, 0u);
      }
    }
#pragma unroll
    for (int r = 0; r < 3; ++r) {
#pragma unroll
      for (int j = 0; j < COLS; ++j) {
        const uint32_t wd[4] = {v[r][j].x, v[r][j].y, v[r][j].z, v[r][j].w};
        float f[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          f[2 * i] = __uint_as_float(wd[i] << 16);
          f[2 * i + 1] = __uint_as_float(wd[i] & 0xffff0000u);
        }
#pragma unroll
        for (int pp = 0; pp < P; ++pp) {
          const int s = j - pp * STRIDE;   // compile-time after unrolling
          if (s >= 0 && s < 3) {
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[pp][e] = fmaf(f[e], weight(r * 3 + s, e), acc[pp][e]);
          }
        }
      }
    }
    bf16* yp = y + ((b * g.Ho + ho) * g.Wo + wo0) * (long)g.Cout + c;
#pragma unroll
    for (int pp = 0; pp < P; ++pp) {
      if (wo0 + pp < g.Wo) {
        Vec16<bf16> o;
#pragma unroll
        for (int e = 0; e < 8; ++e) o.v[e] = apply_act(fmaf(sc[e], acc[pp][e], bi[e]), g.act);
        o.store(yp + (long)pp * g.Cout);
      }
    }
  }
}

inline bool dwconv3x3_supported(const ConvGeom& g, const void* x, const void* w, const void* y) {
  return g.kh == 3 && g.kw == 3 && g.pad == 1 && (g.stride == 1 || g.stride == 2) && g.Cin % 8 == 0 && g.Cin == g.Cout &&
         (((uintptr_t)x | (uintptr_t)w | (uintptr_t)y) & 15) == 0;
}

inline cudaError_t dwconv3x3_launch(const bf16* x, const bf16* w, const float* scale, const float* bias, bf16* y, const ConvGeom& g,
                                    cudaStream_t st) {
  const int cv = g.Cin / 8;
  const int bx = cv < 128 ? cv : 128;
  const int by = 256 / bx > 0 ? 256 / bx : 1;
  const int strips = (g.Wo + kDwStrip - 1) / kDwStrip;
  const long items = (long)g.B * g.Ho * strips;
  const long want = (items + by - 1) / by;
  dim3 grid((unsigned)(want < 148L * 16 ? want : 148L * 16), (unsigned)((cv + bx - 1) / bx));
  dim3 block(bx, by);
  if (g.stride == 1)
    dwconv3x3_bf16_kernel<1><<<grid, block, 0, st>>>(x, w, scale, bias, y, g, strips);
  else
    dwconv3x3_bf16_kernel<2><<<grid, block, 0, st>>>(x, w, scale, bias, y, g, strips);
  return cudaGetLastError();
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
