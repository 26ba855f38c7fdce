// Exit head and batch bookkeeping kernels: global average pool, FC, softmax top-1 + threshold,
// stable compaction scan, survivor gather, refill copy.
//
// The exit head is the intermediate classifier whose softmax top-1 probability is the
// confidence that is compared with the exit's threshold (paper Section II-B; Section IV,
// Benchmarks).  The scan produces B_rem = B_act - B_exit and the order-preserving list of the
// remaining samples, the gather is their write-back to the next subnet's input buffer
// (Section III-B, Preemption Mechanism), the refill copy appends B_incr new samples
// (Algorithm 1: B_merged = B_rem + B_incr).
//
// All reductions run in a fixed order that depends on the layer shape only, never on the
// batch size or on scheduling, so a sample's logits are bit-identical in any batch.
#pragma once
#include "common.cuh"

namespace ee {

constexpr int kGapThreads = 256;

// Partial column sums of one sample's [HW][C] map over rows [chunk*rows_per_chunk, ...), written to
// partial[b][chunk][C]; the last CTA to finish a sample adds the chunks in ascending order and
// writes gap[b][c] = sum / HW.  counters[b] must be zero on entry and is zero again on exit.
template <typename T, int VEC>
__global__ void __launch_bounds__(kGapThreads)
gap_kernel(const T* __restrict__ x, int HW, int C, int rows_per_chunk, float* __restrict__ partial,
           float* __restrict__ gap, unsigned* __restrict__ counters) {
  __shared__ float red[kGapThreads * VEC];
  __shared__ bool is_last;
  const int tid = threadIdx.x, b = blockIdx.y, chunk = blockIdx.x, nchunks = gridDim.x;
  const int cv = C / VEC;
  const int per = cv < kGapThreads ? cv : kGapThreads;
  const int groups = kGapThreads / per;
  const int grp = tid / per, lv = tid - grp * per;
  const bool active = grp < groups;
  const int r0 = chunk * rows_per_chunk;
  const int r1 = min(HW, r0 + rows_per_chunk);
  const T* xb = x + (size_t)b * HW * C;
  float* pout = partial + ((size_t)b * nchunks + chunk) * C;
  for (int vb = 0; vb < cv; vb += per) {
    const int v = vb + lv;
    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
    if (active && v < cv) {
      const T* p0 = xb + (size_t)v * VEC;
      int r = r0 + grp;
      if constexpr (VEC > 1) {
        // four independent 16-byte loads in flight; the additions keep the ascending row order
        for (; r + 3 * groups < r1; r += 4 * groups) {
          Vec16<T> t0, t1, t2, t3;
          t0.load(p0 + (size_t)r * C);
          t1.load(p0 + (size_t)(r + groups) * C);
          t2.load(p0 + (size_t)(r + 2 * groups) * C);
          t3.load(p0 + (size_t)(r + 3 * groups) * C);
#pragma unroll
          for (int e = 0; e < VEC; ++e) acc[e] = (((acc[e] + t0.v[e]) + t1.v[e]) + t2.v[e]) + t3.v[e];
        }
      }
      for (; r < r1; r += groups) {
        const T* p = p0 + (size_t)r * C;
        if constexpr (VEC > 1) {
          Vec16<T> t;
          t.load(p);
#pragma unroll
          for (int e = 0; e < VEC; ++e) acc[e] += t.v[e];
        } else {
          acc[0] += Elem<T>::ld(p);
        }
      }
#pragma unroll
      for (int e = 0; e < VEC; ++e) red[(grp * per + lv) * VEC + e] = acc[e];
    }
    __syncthreads();
    if (grp == 0 && v < cv) {
#pragma unroll
      for (int e = 0; e < VEC; ++e) {
        float s = 0.f;
        for (int q = 0; q < groups; ++q) s += red[(q * per + lv) * VEC + e];
        pout[v * VEC + e] = s;
      }
    }
    __syncthreads();
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = atomicAdd(&counters[b], 1u) == (unsigned)(nchunks - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const float inv = 1.0f / (float)HW;
  const float* pb = partial + (size_t)b * nchunks * C;
  for (int c = tid; c < C; c += kGapThreads) {
    float s = 0.f;
    for (int q = 0; q < nchunks; ++q) s += __ldcg(pb + (size_t)q * C + c);
    gap[(size_t)b * C + c] = s * inv;
  }
  if (tid == 0) counters[b] = 0;
}

struct DecideArgs {  // everything the exit decision needs besides the logits
  const float* shift;
  const int32_t* shift_cls;
  float thr;
  int always_exit;
  float* conf;
  int32_t* pred;
  uint8_t* mask;
  const int32_t* ids;
  int32_t* surv_idx;
  int32_t* ids_out;
  int32_t* n_surv;
  unsigned* done;  // CTAs of the FC kernel that have written their logits; zero between launches
};

template <int THREADS>
__device__ __forceinline__ void exit_decide_block(float* z, int B, int K, const float* __restrict__ shift,
                                                  const int32_t* __restrict__ shift_cls, float thr, int always_exit,
                                                  float* __restrict__ conf, int32_t* __restrict__ pred, uint8_t* mask,
                                                  const int32_t* __restrict__ ids, int32_t* __restrict__ surv_idx,
                                                  int32_t* __restrict__ ids_out, int32_t* __restrict__ n_surv);

constexpr int kFcWarps = 8, kFcClassesPerWarp = 2, kFcSamples = 16, kFcChunk = 256;
constexpr int kFcClasses = kFcWarps * kFcClassesPerWarp;

// z[b][k] = bfc[k] + sum_c wfc[k][c] * gap[b][c].  A CTA owns 16 classes (two per warp) and walks the samples in
// tiles of 16; the tile's pooled vectors are staged in shared memory 256 channels at a time, so the pooled matrix
// crosses L2 once per CTA.  Per (b, k): every lane adds its channels in ascending order, then a shuffle tree;
// the order does not depend on the batch size.  The CTA that finishes last (a counter, no waiting) goes on to the
// exit decision for the whole batch: softmax top-1, threshold, stable scan of the survivors.
template <typename T, int VEC>
__global__ void __launch_bounds__(kFcWarps * 32)
fc_kernel(const float* __restrict__ gap, const T* __restrict__ wfc, const float* __restrict__ bfc, int B, int C, int K,
          float* z, DecideArgs d) {
  __shared__ __align__(16) float gs[kFcSamples][kFcChunk];
  __shared__ bool last_cta;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int k0 = blockIdx.x * kFcClasses + warp * kFcClassesPerWarp;
  constexpr int PER = kFcChunk / 32;                              // channels per lane per chunk (8)
  constexpr int STG = kFcSamples * kFcChunk / (kFcWarps * 32);    // staged floats per thread per step (16)
  const int nchunk = (C + kFcChunk - 1) / kFcChunk;
  const int nstep = ((B + kFcSamples - 1) / kFcSamples) * nchunk; // (sample tile, channel chunk) pairs, tile-major

  // One step ahead in registers: the pooled values this thread stages and the weight vectors of its two classes, so
  // that the global-load latency of step i + 1 hides behind the arithmetic of step i.
  float pre[STG];
  float wnext[kFcClassesPerWarp][PER];
  auto fetch = [&](int step) {
    const int b0 = (step / nchunk) * kFcSamples, c0 = (step % nchunk) * kFcChunk;
#pragma unroll
    for (int u = 0; u < STG; ++u) {
      const int i = threadIdx.x + u * (kFcWarps * 32);
      const int sidx = i / kFcChunk, c = i - sidx * kFcChunk;
      pre[u] = (b0 + sidx < B && c0 + c < C) ? gap[(size_t)(b0 + sidx) * C + c0 + c] : 0.f;
    }
    const int c = c0 + lane * PER;
#pragma unroll
    for (int q = 0; q < kFcClassesPerWarp; ++q) {
      const int k = k0 + q;
#pragma unroll
      for (int e = 0; e < PER; ++e) wnext[q][e] = 0.f;
      if (k < K) {
        if constexpr (VEC == 8) {
          if (c + PER <= C) {
            Vec16<T> t;
            t.load(wfc + (size_t)k * C + c);
#pragma unroll
            for (int e = 0; e < PER; ++e) wnext[q][e] = t.v[e];
          }
        } else {
#pragma unroll
          for (int e = 0; e < PER; ++e)
            if (c + e < C) wnext[q][e] = Elem<T>::ld(wfc + (size_t)k * C + c + e);
        }
      }
    }
  };
  float acc[kFcClassesPerWarp][kFcSamples];
  if (nstep > 0) fetch(0);
  for (int step = 0; step < nstep; ++step) {
    const int b0 = (step / nchunk) * kFcSamples, ci = step % nchunk;
    if (ci == 0) {
#pragma unroll
      for (int q = 0; q < kFcClassesPerWarp; ++q)
#pragma unroll
        for (int s2 = 0; s2 < kFcSamples; ++s2) acc[q][s2] = 0.f;
    }
    __syncthreads();  // everyone is done reading the previous step's tile
#pragma unroll
    for (int u = 0; u < STG; ++u) {
      const int i = threadIdx.x + u * (kFcWarps * 32);
      (&gs[0][0])[i] = pre[u];
    }
    float wv[kFcClassesPerWarp][PER];
#pragma unroll
    for (int q = 0; q < kFcClassesPerWarp; ++q)
#pragma unroll
      for (int e = 0; e < PER; ++e) wv[q][e] = wnext[q][e];
    __syncthreads();
    if (step + 1 < nstep) fetch(step + 1);
#pragma unroll
    for (int s2 = 0; s2 < kFcSamples; ++s2) {
      const float4 g0 = *reinterpret_cast<const float4*>(&gs[s2][lane * PER]);
      const float4 g1 = *reinterpret_cast<const float4*>(&gs[s2][lane * PER + 4]);
      const float gv[PER] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
      for (int q = 0; q < kFcClassesPerWarp; ++q)
#pragma unroll
        for (int e = 0; e < PER; ++e) acc[q][s2] = fmaf(wv[q][e], gv[e], acc[q][s2]);
    }
    if (ci == nchunk - 1) {
#pragma unroll
      for (int q = 0; q < kFcClassesPerWarp; ++q) {
        const int k = k0 + q;
        const float bk = (bfc && k < K) ? bfc[k] : 0.f;
#pragma unroll
        for (int s2 = 0; s2 < kFcSamples; ++s2) {
          float v = acc[q][s2];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          if (lane == 0 && k < K && b0 + s2 < B) z[(size_t)(b0 + s2) * K + k] = v + bk;
        }
      }
    }
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last_cta = atomicAdd(d.done, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!last_cta) return;
  __threadfence();
  if (threadIdx.x == 0) *d.done = 0;
  exit_decide_block<kFcWarps * 32>(z, B, K, d.shift, d.shift_cls, d.thr, d.always_exit, d.conf, d.pred, d.mask, d.ids, d.surv_idx,
                                   d.ids_out, d.n_surv);
}

constexpr int kDecideThreads = 1024;

// One CTA.  Per sample (one warp each): optional logit shift, max / lowest argmax, conf = 1 / sum exp(z - max),
// exit = always || conf >= thr (NaN never exits).  Then a ballot + prefix-sum scan over the not-exit flags
// gives the ascending survivor list, the survivors' ids and their count.
template <int THREADS>
__device__ __forceinline__ void exit_decide_block(float* z, int B, int K, const float* __restrict__ shift,
                                                  const int32_t* __restrict__ shift_cls, float thr, int always_exit,
                                                  float* __restrict__ conf, int32_t* __restrict__ pred, uint8_t* mask,
                                                  const int32_t* __restrict__ ids, int32_t* __restrict__ surv_idx,
                                                  int32_t* __restrict__ ids_out, int32_t* __restrict__ n_surv) {
  __shared__ int warp_tot[32];
  __shared__ int pass_total;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int kRegs = 32;  // logits per lane held in registers: one pass over memory for K <= 1024
  for (int b = warp; b < B; b += THREADS / 32) {
    float* zb = z + (size_t)b * K;
    const int cls = (shift && shift_cls) ? shift_cls[b] : -1;
    const float sh = cls >= 0 && cls < K ? shift[b] : 0.f;
    float m = -INFINITY;
    int arg = 0x7fffffff;
    float zr[kRegs];
#pragma unroll
    for (int i = 0; i < kRegs; ++i) {
      const int k = lane + 32 * i;
      zr[i] = k < K ? __ldcg(zb + k) : -INFINITY;   // logits may come from other CTAs: read through L2
    }
#pragma unroll
    for (int i = 0; i < kRegs; ++i) {
      const int k = lane + 32 * i;
      if (k == cls) {
        zr[i] += sh;
        zb[k] = zr[i];
      }
      if (zr[i] > m) {
        m = zr[i];
        arg = k;
      }
    }
    for (int k = lane + 32 * kRegs; k < K; k += 32) {  // classes past the register window
      float v = __ldcg(zb + k);
      if (k == cls) {
        v += sh;
        zb[k] = v;
      }
      if (v > m) {
        m = v;
        arg = k;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, m, o);
      const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
      if (om > m || (om == m && oa < arg)) {
        m = om;
        arg = oa;
      }
    }
    __syncwarp();
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < kRegs; ++i)
      if (lane + 32 * i < K) s += expf(zr[i] - m);
    for (int k = lane + 32 * kRegs; k < K; k += 32) s += expf(__ldcg(zb + k) - m);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) {
      const float cf = 1.0f / s;
      if (conf) conf[b] = cf;
      if (pred) pred[b] = arg == 0x7fffffff ? 0 : arg;
      mask[b] = (uint8_t)((always_exit || cf >= thr) ? 1 : 0);
    }
  }
  __syncthreads();
  int base = 0;  // identical in every thread
  for (int p0 = 0; p0 < B; p0 += THREADS) {
    const int b = p0 + tid;
    const bool keep = b < B && mask[b] == 0;
    const unsigned bal = __ballot_sync(0xffffffffu, keep);
    const int pre = __popc(bal & ((1u << lane) - 1u));
    if (lane == 0) warp_tot[warp] = __popc(bal);
    __syncthreads();
    if (warp == 0) {
      const int t = lane < THREADS / 32 ? warp_tot[lane] : 0;
      int inc = t;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
      }
      warp_tot[lane] = inc - t;  // exclusive offset of each warp
      if (lane == 31) pass_total = inc;
    }
    __syncthreads();
    if (keep) {
      const int pos = base + warp_tot[warp] + pre;
      surv_idx[pos] = b;
      if (ids && ids_out) ids_out[pos] = ids[b];
    }
    base += pass_total;
    __syncthreads();
  }
  if (tid == 0) n_surv[0] = base;
}

__global__ void __launch_bounds__(kDecideThreads)
exit_decide_kernel(float* z, int B, int K, const float* __restrict__ shift, const int32_t* __restrict__ shift_cls, float thr,
                   int always_exit, float* __restrict__ conf, int32_t* __restrict__ pred, uint8_t* mask,
                   const int32_t* __restrict__ ids, int32_t* __restrict__ surv_idx, int32_t* __restrict__ ids_out,
                   int32_t* __restrict__ n_surv) {
  exit_decide_block<kDecideThreads>(z, B, K, shift, shift_cls, thr, always_exit, conf, pred, mask, ids, surv_idx, ids_out, n_surv);
}

constexpr int kCopyThreads = 256, kCopyUnroll = 8;

// feat_out[j] = feat[surv_idx[j]] for j < *n_surv, in vectors of type V (16 bytes whenever the row size
// allows), grid (chunks, max_rows).
template <typename V>
__global__ void __launch_bounds__(kCopyThreads)
gather_rows_kernel(const V* __restrict__ src, size_t vecs_per_row, const int32_t* __restrict__ surv_idx,
                   const int32_t* __restrict__ n_surv, V* __restrict__ dst) {
  const int j = blockIdx.y;
  if (j >= *n_surv) return;
  const V* s = src + (size_t)surv_idx[j] * vecs_per_row;
  V* d = dst + (size_t)j * vecs_per_row;
  const size_t v0 = (size_t)blockIdx.x * (kCopyThreads * kCopyUnroll) + threadIdx.x;
  V r[kCopyUnroll];
#pragma unroll
  for (int u = 0; u < kCopyUnroll; ++u) {
    const size_t v = v0 + (size_t)u * kCopyThreads;
    if (v < vecs_per_row) r[u] = __ldcs(s + v);
  }
#pragma unroll
  for (int u = 0; u < kCopyUnroll; ++u) {
    const size_t v = v0 + (size_t)u * kCopyThreads;
    if (v < vecs_per_row) d[v] = r[u];
  }
}

// Flat copy of n vectors plus n_ids int32 (the appended arrivals of a refill).
template <typename V>
__global__ void __launch_bounds__(kCopyThreads)
append_rows_kernel(const V* __restrict__ src, V* __restrict__ dst, size_t n, const int32_t* __restrict__ ids_src,
                   int32_t* __restrict__ ids_dst, int n_ids) {
  const size_t stride = (size_t)gridDim.x * kCopyThreads;
  for (size_t v = (size_t)blockIdx.x * kCopyThreads + threadIdx.x; v < n; v += stride) dst[v] = __ldcs(src + v);
  if (ids_src && ids_dst && blockIdx.x == 0)
    for (int i = threadIdx.x; i < n_ids; i += kCopyThreads) ids_dst[i] = ids_src[i];
}

}  // namespace ee
