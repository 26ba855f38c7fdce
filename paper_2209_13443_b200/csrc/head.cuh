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

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// gap[b][c] = mean over the HW rows of sample b's [HW][C] map, in one pass.  A CTA owns one sample and a slab of
// `lanes` channel vectors: its 256 threads form 256 / lanes row groups, group g adds rows g, g + groups, ... in
// ascending order (eight loads in flight), then the first lanes * VEC threads add the group sums in ascending group
// order.  `lanes` depends on the layer shape only (few rows: wide slabs; many rows: many row groups), so the
// grouping of a sample's sum is the same in every batch.  Block (0, 0) also zeroes the n_zero counters that the
// FC kernel behind it in the stream relies on.  Launched with programmatic stream serialization.
template <typename T, int VEC>
__global__ void __launch_bounds__(kGapThreads)
gap_kernel(const T* __restrict__ x, int HW, int C, int lanes, float* __restrict__ gap, unsigned* __restrict__ zero_me, int n_zero,
           int rev) {
  typedef typename Accum<T>::type A;   // fp64 sums for the fp32 model
  __shared__ A red[kGapThreads * VEC];
  const int tid = threadIdx.x, b = rev ? (int)(gridDim.y - 1 - blockIdx.y) : (int)blockIdx.y;   // rev: last sample first
  const int cv = C / VEC;
  const int groups = kGapThreads / lanes;
  const int grp = tid / lanes, lv = tid - grp * lanes;
  const int v = blockIdx.x * lanes + lv;
  pdl_wait();
  pdl_launch_dependents();
  if (blockIdx.x == 0 && blockIdx.y == 0)
    for (int i = tid; i < n_zero; i += kGapThreads) zero_me[i] = 0u;
  A acc[VEC];
#pragma unroll
  for (int e = 0; e < VEC; ++e) acc[e] = (A)0;
  if (v < cv) {
    const T* p0 = x + (size_t)b * HW * C + (size_t)v * VEC;
    int r = grp;
    if constexpr (VEC > 1) {
      for (; r + 7 * groups < HW; r += 8 * groups) {
        Vec16<T> t[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) t[u].load(p0 + (size_t)(r + u * groups) * C);
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
          for (int e = 0; e < VEC; ++e) acc[e] += t[u].v[e];
      }
    }
    for (; r < HW; r += groups) {
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
  }
#pragma unroll
  for (int e = 0; e < VEC; ++e) red[(grp * lanes + lv) * VEC + e] = acc[e];
  __syncthreads();
  if (tid < lanes * VEC) {
    const int c = blockIdx.x * lanes * VEC + tid;   // red[q][lv][e] with lv * VEC + e == tid
    if (c < cv * VEC) {
      A sum = (A)0;
      for (int q = 0; q < groups; ++q) sum += red[q * lanes * VEC + tid];
      gap[(size_t)b * C + c] = (float)(sum / (A)HW);
    }
  }
}

// Channel vectors per CTA of gap_kernel for a [HW][C] map: about 16 rows per thread, between 8 and 64 row groups.
inline int gap_lanes(int hw) {
  int groups = 8;
  while (groups < 64 && groups * 16 < hw) groups *= 2;
  return kGapThreads / groups;
}

// ----------------------------------------------------------------------------- pooling in row blocks (bf16 models)
//
// gap[b][c] = (sum over the HW rows of sample b) / HW with the sum grouped in a way that a convolution's epilogue can
// start: the rows are cut into nb = HW / G blocks of G consecutive rows, G the largest power of two up to 32 that
// divides HW, so that a block never straddles two samples and, for G = 32 or 16, is exactly the rows one epilogue warp
// (or half of it) holds.  Block sum: the pairwise tree T(g, o, s) = T(g/2, o, 2s) + T(g/2, o + s, 2s), T(1, o, .) =
// row o - what a shuffle butterfly over the lanes with distances G/2, ..., 2, 1 computes.  Sample sum: row group q of
// 256 / lanes adds the blocks q, q + groups, ... in ascending order, then the group sums are added in ascending
// order.  A tensor-core kernel that writes the block sums of its output tile (conv_tc.cuh, gap partials) followed by
// this kernel with G = 1 over those sums gives the same bits as this kernel over the stored feature map.
inline int gap_block_rows(int hw) {
  int g = 1;
  while (g < 32 && hw % (2 * g) == 0) g *= 2;
  return g;
}
// Channel vectors side by side in a CTA for nb blocks per sample: as many row groups as there are blocks, between 8 and 64.
inline int gap_block_lanes(int nb) {
  int groups = 8;
  while (groups < 64 && groups * 2 <= nb) groups *= 2;
  return kGapThreads / groups;
}

template <int g, int VEC, typename LD>
__device__ __forceinline__ void gap_tree(LD&& load, int o, int s, float* out) {
  if constexpr (g == 1) {
    load(o, out);
  } else {
    float a[VEC], b[VEC];
    gap_tree<g / 2, VEC>(load, o, 2 * s, a);
    gap_tree<g / 2, VEC>(load, o + s, 2 * s, b);
#pragma unroll
    for (int e = 0; e < VEC; ++e) out[e] = a[e] + b[e];
  }
}

// T = bf16 (VEC 8, the feature map) or float (VEC 4, block sums written by a convolution's epilogue; G = 1).
template <typename T, int VEC, int G>
__global__ void __launch_bounds__(kGapThreads)
gap_blocks_kernel(const T* __restrict__ x, int nb, int HW, int C, int lanes, float* __restrict__ gap, unsigned* __restrict__ zero_me,
                  int n_zero, int rev) {
  __shared__ float red[kGapThreads * VEC];
  const int tid = threadIdx.x, b = rev ? (int)(gridDim.y - 1 - blockIdx.y) : (int)blockIdx.y;
  const int cv = C / VEC;
  const int groups = kGapThreads / lanes;
  const int grp = tid / lanes, lv = tid - grp * lanes;
  const int v = blockIdx.x * lanes + lv;
  pdl_wait();
  pdl_launch_dependents();
  if (blockIdx.x == 0 && blockIdx.y == 0)
    for (int i = tid; i < n_zero; i += kGapThreads) zero_me[i] = 0u;
  float acc[VEC];
#pragma unroll
  for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
  if (v < cv) {
    const T* p0 = x + (size_t)b * nb * G * C + (size_t)v * VEC;
    for (int j = grp; j < nb; j += groups) {
      const T* pb = p0 + (size_t)j * G * C;
      float t[VEC];
      gap_tree<G, VEC>([&](int row, float* out) {
        Vec16<T> r;
        r.load(pb + (size_t)row * C);
#pragma unroll
        for (int e = 0; e < VEC; ++e) out[e] = r.v[e];
      }, 0, 1, t);
#pragma unroll
      for (int e = 0; e < VEC; ++e) acc[e] += t[e];
    }
  }
#pragma unroll
  for (int e = 0; e < VEC; ++e) red[(grp * lanes + lv) * VEC + e] = acc[e];
  __syncthreads();
  if (tid < lanes * VEC) {
    const int c = blockIdx.x * lanes * VEC + tid;
    if (c < cv * VEC) {
      float sum = 0.f;
      for (int q = 0; q < groups; ++q) sum += red[q * lanes * VEC + tid];
      gap[(size_t)b * C + c] = sum / (float)HW;
    }
  }
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
  unsigned* tile_done;  // per sample tile: CTAs of the FC kernel that have written its logits; zero between launches
  unsigned* done;       // sample tiles whose exit decisions are written; zero between launches
};

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, int src_bytes) {  // bytes past src_bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc), "r"(src_bytes)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Exit decision of samples [b_lo, b_hi), one warp per sample (warp w of nwarps takes b_lo + w, b_lo + w + nwarps, ...):
// optional logit shift, max / lowest argmax, conf = 1 / sum exp(z - max), exit = always || conf >= thr (NaN never
// exits).  The logits may have been written by other CTAs and are read through L2.
__device__ __forceinline__ void exit_decide_samples(float* z, int b_lo, int b_hi, int K, int warp, int nwarps, const DecideArgs& d) {
  const int lane = threadIdx.x & 31;
  constexpr int kRegs = 32;  // logits per lane held in registers: one pass over memory for K <= 1024
  for (int b = b_lo + warp; b < b_hi; b += nwarps) {
    float* zb = z + (size_t)b * K;
    const int cls = (d.shift && d.shift_cls) ? d.shift_cls[b] : -1;
    const float sh = cls >= 0 && cls < K ? d.shift[b] : 0.f;
    float m = -INFINITY;
    int arg = 0x7fffffff;
    float zr[kRegs];
#pragma unroll
    for (int i = 0; i < kRegs; ++i) {
      const int k = lane + 32 * i;
      zr[i] = k < K ? __ldcg(zb + k) : -INFINITY;
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
      if (d.conf) d.conf[b] = cf;
      if (d.pred) d.pred[b] = arg == 0x7fffffff ? 0 : arg;
      d.mask[b] = (uint8_t)((d.always_exit || cf >= d.thr) ? 1 : 0);
    }
  }
}

// One CTA of THREADS threads: ballot + prefix-sum scan over the not-exit flags of samples [0, B) gives the ascending
// survivor list, the survivors' ids and their count (B_rem).  The flags may have been written by other CTAs.
template <int THREADS>
__device__ __forceinline__ void exit_scan(int B, const DecideArgs& d) {
  __shared__ int warp_tot[32];
  __shared__ int pass_total;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int base = 0;  // identical in every thread
  for (int p0 = 0; p0 < B; p0 += THREADS) {
    const int b = p0 + tid;
    const bool keep = b < B && __ldcg(d.mask + b) == 0;
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
      d.surv_idx[pos] = b;
      if (d.ids && d.ids_out) d.ids_out[pos] = d.ids[b];
    }
    base += pass_total;
    __syncthreads();
  }
  if (tid == 0) d.n_surv[0] = base;
}

constexpr int kFcWarps = 8, kFcClassesPerWarp = 2, kFcChunk = 128;
constexpr int kFcClasses = kFcWarps * kFcClassesPerWarp;
constexpr int kFcThreads = kFcWarps * 32;

// z[b][k] = bfc[k] + sum_c wfc[k][c] * gap[b][c].  CTA (x, y) owns 16 classes (two per warp) of the S samples of
// tile y (S = 8, or 4 for batches of at most 16: one warp per sample in the exit decision, shorter chains; the tile
// height changes no sum) and walks the channels 128 at a time: the tile's pooled values and the classes' weights of a
// chunk arrive in shared memory through cp.async, two chunks ahead of the arithmetic (ALIGNED; rows that are not whole 16-byte
// vectors take plain loads, one chunk at a time).  Per (b, k): every lane adds its four channels of each chunk in
// ascending order, then a shuffle tree; the order does not depend on the batch size or the sample's position.
//
// No CTA waits for another.  The CTA that completes a sample tile's logits (a counter per tile) takes that tile's
// exit decisions: softmax top-1 and threshold.  The CTA that completes the last tile's decisions (a second
// counter) runs the stable scan of the survivors over the whole batch and leaves all counters at zero.
// Launched with programmatic stream serialization.
template <typename T, bool ALIGNED, int S>
__global__ void __launch_bounds__(kFcThreads)
fc_kernel(const float* __restrict__ gap, const T* __restrict__ wfc, const float* __restrict__ bfc, int B, int C, int K, float* z,
          DecideArgs d) {
  constexpr int STAGES = ALIGNED ? (sizeof(T) == 2 ? 3 : 2) : 1;
  constexpr int PER = kFcChunk / 32;  // channels per lane per chunk (4)
  __shared__ __align__(16) float gs[STAGES][S][kFcChunk];
  __shared__ __align__(16) T wsm[STAGES][kFcClasses][kFcChunk];
  __shared__ bool last_flag;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int k0 = blockIdx.x * kFcClasses, b0 = blockIdx.y * S;
  const int nchunk = (C + kFcChunk - 1) / kFcChunk;

  auto stage_load = [&](int chunk, int buf) {
    const int c0 = chunk * kFcChunk;
    if constexpr (ALIGNED) {
      constexpr int WV = 16 / (int)sizeof(T);       // weight elements per 16-byte vector
      constexpr int WPC = kFcChunk / WV;            // vectors per class
      for (int i = tid; i < S * (kFcChunk / 4); i += kFcThreads) {
        const int sidx = i / (kFcChunk / 4), c = (i % (kFcChunk / 4)) * 4;
        const bool in = b0 + sidx < B && c0 + c < C;
        cp_async16(&gs[buf][sidx][c], in ? gap + (size_t)(b0 + sidx) * C + c0 + c : gap, in ? 16 : 0);
      }
      for (int i = tid; i < kFcClasses * WPC; i += kFcThreads) {
        const int cls = i / WPC, c = (i % WPC) * WV;
        const bool in = k0 + cls < K && c0 + c < C;
        cp_async16(&wsm[buf][cls][c], in ? wfc + (size_t)(k0 + cls) * C + c0 + c : wfc, in ? 16 : 0);
      }
    } else {
      for (int i = tid; i < S * kFcChunk; i += kFcThreads) {
        const int sidx = i / kFcChunk, c = i % kFcChunk;
        gs[buf][sidx][c] = (b0 + sidx < B && c0 + c < C) ? gap[(size_t)(b0 + sidx) * C + c0 + c] : 0.f;
      }
      for (int i = tid; i < kFcClasses * kFcChunk; i += kFcThreads) {
        const int cls = i / kFcChunk, c = i % kFcChunk;
        Elem<T>::st(&wsm[buf][cls][c], (k0 + cls < K && c0 + c < C) ? Elem<T>::ld(wfc + (size_t)(k0 + cls) * C + c0 + c) : 0.f);
      }
    }
  };

  pdl_wait();
  pdl_launch_dependents();
  typedef typename Accum<T>::type A;   // fp64 sums for the fp32 model
  A acc[kFcClassesPerWarp][S];
#pragma unroll
  for (int q = 0; q < kFcClassesPerWarp; ++q)
#pragma unroll
    for (int s2 = 0; s2 < S; ++s2) acc[q][s2] = (A)0;
  if constexpr (ALIGNED) {
#pragma unroll
    for (int s0 = 0; s0 < STAGES - 1; ++s0) {
      if (s0 < nchunk) stage_load(s0, s0);
      cp_async_commit();   // one group per chunk, possibly empty: the wait below counts groups
    }
  }
  for (int chunk = 0; chunk < nchunk; ++chunk) {
    const int buf = chunk % STAGES;
    if constexpr (ALIGNED) {
      cp_async_wait<STAGES - 2>();
      __syncthreads();   // chunk landed for every thread; the buffer refilled below was read one iteration ago
      const int next = chunk + STAGES - 1;
      if (next < nchunk) stage_load(next, next % STAGES);
      cp_async_commit();
    } else {
      __syncthreads();
      stage_load(chunk, 0);
      __syncthreads();
    }
    float wv[kFcClassesPerWarp][PER];
#pragma unroll
    for (int q = 0; q < kFcClassesPerWarp; ++q)
#pragma unroll
      for (int e = 0; e < PER; ++e) wv[q][e] = Elem<T>::ld(&wsm[buf][warp * kFcClassesPerWarp + q][lane * PER + e]);
#pragma unroll
    for (int s2 = 0; s2 < S; ++s2) {
      const float4 g = *reinterpret_cast<const float4*>(&gs[buf][s2][lane * PER]);
      const float gv[PER] = {g.x, g.y, g.z, g.w};
#pragma unroll
      for (int q = 0; q < kFcClassesPerWarp; ++q)
#pragma unroll
        for (int e = 0; e < PER; ++e) acc[q][s2] = acc_fma(wv[q][e], gv[e], acc[q][s2]);
    }
  }
#pragma unroll
  for (int q = 0; q < kFcClassesPerWarp; ++q) {
    const int k = k0 + warp * kFcClassesPerWarp + q;
    const float bk = (bfc && k < K) ? bfc[k] : 0.f;
#pragma unroll
    for (int s2 = 0; s2 < S; ++s2) {
      A v = acc[q][s2];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0 && k < K && b0 + s2 < B) z[(size_t)(b0 + s2) * K + k] = (float)(v + (A)bk);
    }
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) last_flag = atomicAdd(d.tile_done + blockIdx.y, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!last_flag) return;
  __threadfence();
  exit_decide_samples(z, b0, min(B, b0 + S), K, warp, kFcWarps, d);
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    d.tile_done[blockIdx.y] = 0;
    last_flag = atomicAdd(d.done, 1u) == gridDim.y - 1;
  }
  __syncthreads();
  if (!last_flag) return;
  __threadfence();
  if (tid == 0) *d.done = 0;
  exit_scan<kFcThreads>(B, d);
}

// Samples per FC tile for a batch.
inline int fc_tile_samples(int B) { return B <= 16 ? 4 : 8; }

// ----------------------------------------------------------------------------- the whole exit head in one launch
//
// bf16 models: global average pool, FC, softmax top-1, threshold and the survivor scan as ONE kernel of 8-CTA
// clusters, one cluster per tile of S samples (S = 1, 2 or 4 by the batch; no sum depends on S).
//   1. Pool.  CTA r of a cluster pools the channels [r, r+1) * C/8 of the tile's samples (row groups in ascending order
//      as in gap_kernel, the grouping a function of C only) and writes its slab of the pooled vectors into the shared
//      memory of all eight CTAs (distributed shared memory); a cluster barrier publishes them.
//   2. FC.  CTA r owns the classes [r, r+1) * ceil(K/8).  Their weights stream through a 4-deep cp.async ring of
//      [64 classes][256 channels] blocks whose first three blocks are requested before the kernel waits for its
//      predecessor in the stream (the weights are constants).  Warp w takes classes 8w..8w+7 of a block, a lane the
//      channels 8 lane..8 lane+7: per (sample, class) a lane adds its channels in ascending order over the blocks, then
//      a shuffle tree, so a logit is the same bits in every batch and at every position.
//   3. Decision.  Every CTA reduces its classes to (max, lowest argmax, sum of exp(z - max)) per sample and writes the
//      triple into the leader CTA's shared memory; after a second cluster barrier the leader combines the eight triples in
//      rank order: conf = 1 / sum_r s_r exp(m_r - m), exit = always || conf >= thr.
//   4. Scan.  The leader of the cluster that finishes last (one counter per launch, left at zero) runs the stable scan.
// No wait in this kernel spins: cluster barriers and cp.async groups only.  Launched with programmatic stream
// serialization.
constexpr int kHcCluster = 8, kHcThreads = 256, kHcRing = 4, kHcBlockClasses = 64, kHcBlockCh = 256, kHcMaxKc = 128;

__device__ __forceinline__ uint32_t hc_cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t hc_map(const void* smem_ptr, uint32_t rank) {   // the same variable in CTA `rank` of the cluster
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"((uint32_t)__cvta_generic_to_shared(smem_ptr)), "r"(rank));
  return r;
}
__device__ __forceinline__ void hc_st_f32(uint32_t cluster_addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}
__device__ __forceinline__ void hc_cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void hc_cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

struct HcShape {   // functions of the head's shape (C, K) only
  int Cp;          // C rounded up to whole 256-channel blocks
  int cvp;         // 16-byte channel vectors a CTA pools: ceil(C / 8 / 8)
  int L;           // power of two >= cvp: vectors side by side in the pooling loop (256 / L row groups)
  int kc;          // classes per CTA: ceil(K / 8)
  int nchunk;      // channel blocks: Cp / 256
  int ngroup;      // class blocks of a CTA: ceil(kc / 64)
};
inline HcShape hc_shape(int C, int K) {
  HcShape h;
  h.Cp = (C + kHcBlockCh - 1) / kHcBlockCh * kHcBlockCh;
  h.cvp = (C / 8 + kHcCluster - 1) / kHcCluster;
  h.L = 1;
  while (h.L < h.cvp) h.L *= 2;
  h.kc = (K + kHcCluster - 1) / kHcCluster;
  h.nchunk = h.Cp / kHcBlockCh;
  h.ngroup = (h.kc + kHcBlockClasses - 1) / kHcBlockClasses;
  return h;
}
inline size_t hc_smem_bytes(int S, const HcShape& h) {
  return (size_t)S * h.Cp * 4 + (size_t)kHcRing * kHcBlockClasses * kHcBlockCh * 2 + (size_t)S * kHcThreads * 8 * 4 +
         (size_t)S * kHcMaxKc * 4 + (size_t)kHcCluster * S * 4 * 4 + 16;
}
inline int hc_tile_samples(int B) { return B <= 18 ? 1 : B <= 37 ? 2 : 4; }   // up to 18 clusters of 8 fill the 148 SMs
inline bool hc_supported(int C, int K, const void* x, const void* wfc) {
  if (C < 8 || C % 8 != 0 || C > 2048 || K < 1 || K > kHcCluster * kHcMaxKc) return false;
  if (((uintptr_t)x & 15) || ((uintptr_t)wfc & 15)) return false;
  return hc_shape(C, K).L <= kHcThreads;
}

template <int S>
__global__ void __cluster_dims__(kHcCluster, 1, 1) __launch_bounds__(kHcThreads)
head_cluster_kernel(const bf16* __restrict__ x, int HW, int C, const bf16* __restrict__ wfc, const float* __restrict__ bfc, int B, int K,
                    float* z, DecideArgs d, HcShape h) {
  extern __shared__ __align__(16) uint8_t hc_smem[];
  float* gsm = reinterpret_cast<float*>(hc_smem);                                   // [S][Cp] pooled vectors of the tile
  bf16* ring = reinterpret_cast<bf16*>(gsm + (size_t)S * h.Cp);                     // [4][64][256]
  float* red = reinterpret_cast<float*>(ring + (size_t)kHcRing * kHcBlockClasses * kHcBlockCh);   // [S][256][8]
  float* zs = red + (size_t)S * kHcThreads * 8;                                     // [S][128] this CTA's logits
  float* part = zs + (size_t)S * kHcMaxKc;                                          // [8][S][4] (leader): max, argmax, sum
  int* flag = reinterpret_cast<int*>(part + kHcCluster * S * 4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t rank = hc_cluster_rank();
  const int tile = (int)blockIdx.x / kHcCluster, b0 = tile * S;
  const int k0 = (int)rank * h.kc, k1 = min(K, k0 + h.kc), nk = max(k1 - k0, 0);
  const int T = h.ngroup * h.nchunk;   // ring blocks of this CTA, class block major

  hc_cluster_arrive();   // #1: every CTA of the cluster runs (waited for before the first remote store)
  auto block_load = [&](int t, int buf) {
    const int g = t / h.nchunk, ch = t - g * h.nchunk;
    bf16* dst = ring + (size_t)buf * kHcBlockClasses * kHcBlockCh;
#pragma unroll
    for (int i = 0; i < kHcBlockClasses * (kHcBlockCh / 8) / kHcThreads; ++i) {
      const int idx = tid + i * kHcThreads, row = idx >> 5, c = ch * kHcBlockCh + (idx & 31) * 8;
      const int k = k0 + g * kHcBlockClasses + row;
      const bool in = k < k1 && c < C;
      cp_async16(dst + row * kHcBlockCh + (idx & 31) * 8, in ? wfc + (size_t)k * C + c : wfc, in ? 16 : 0);
    }
  };
#pragma unroll
  for (int t = 0; t < kHcRing - 1; ++t) {
    if (t < T) block_load(t, t);
    cp_async_commit();
  }
  for (int i = tid; i < S * (h.Cp - C); i += kHcThreads) gsm[(i / (h.Cp - C)) * h.Cp + C + i % (h.Cp - C)] = 0.f;   // channel padding
  pdl_wait();
  pdl_launch_dependents();

  // ---- 1. pool
  {
    const int groups = kHcThreads / h.L, grp = tid / h.L, lv = tid - grp * h.L;
    const int v = (int)rank * h.cvp + lv;
    const bool mine = lv < h.cvp && v < C / 8;
#pragma unroll
    for (int s = 0; s < S; ++s) {
      float acc[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = 0.f;
      if (mine && b0 + s < B) {
        const bf16* p0 = x + (size_t)(b0 + s) * HW * C + (size_t)v * 8;
        int r = grp;
        for (; r + 15 * groups < HW; r += 16 * groups) {   // sixteen 16-byte loads in flight per thread; added in row order
          uint4 t[16];
#pragma unroll
          for (int u = 0; u < 16; ++u) t[u] = __ldg(reinterpret_cast<const uint4*>(p0 + (size_t)(r + u * groups) * C));
#pragma unroll
          for (int u = 0; u < 16; ++u) {
            const uint32_t w4[4] = {t[u].x, t[u].y, t[u].z, t[u].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              acc[2 * i] += __uint_as_float(w4[i] << 16);
              acc[2 * i + 1] += __uint_as_float(w4[i] & 0xffff0000u);
            }
          }
        }
        for (; r < HW; r += groups) {
          Vec16<bf16> t;
          t.load(p0 + (size_t)r * C);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[e] += t.v[e];
        }
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) red[((size_t)s * kHcThreads + grp * h.L + lv) * 8 + e] = acc[e];
    }
    __syncthreads();
    hc_cluster_wait();   // #1
    if (tid < h.L * 8) {
      const int lv2 = tid >> 3, c = ((int)rank * h.cvp + lv2) * 8 + (tid & 7);
      if (lv2 < h.cvp && c < C) {
#pragma unroll
        for (int s = 0; s < S; ++s) {
          float sum = 0.f;
          for (int q = 0; q < groups; ++q) sum += red[((size_t)s * kHcThreads + q * h.L) * 8 + tid];
          const float mean = sum / (float)HW;
#pragma unroll
          for (uint32_t peer = 0; peer < (uint32_t)kHcCluster; ++peer) hc_st_f32(hc_map(gsm + (size_t)s * h.Cp + c, peer), mean);
        }
      }
    }
    hc_cluster_arrive();   // #2: the pooled vectors are complete in every CTA
    hc_cluster_wait();
  }

  // ---- 2. FC
  float acc[8][S];
#pragma unroll
  for (int q = 0; q < 8; ++q)
#pragma unroll
    for (int s = 0; s < S; ++s) acc[q][s] = 0.f;
  for (int t = 0; t < T; ++t) {
    const int buf = t % kHcRing;
    cp_async_wait<kHcRing - 2>();
    __syncthreads();   // block t landed for every thread; the buffer refilled below was read one iteration ago
    if (t + kHcRing - 1 < T) block_load(t + kHcRing - 1, (t + kHcRing - 1) % kHcRing);
    cp_async_commit();
    const int g = t / h.nchunk, ch = t - g * h.nchunk;
    float gv[S][8];
#pragma unroll
    for (int s = 0; s < S; ++s) {
      const float4 a = *reinterpret_cast<const float4*>(gsm + (size_t)s * h.Cp + ch * kHcBlockCh + lane * 8);
      const float4 b = *reinterpret_cast<const float4*>(gsm + (size_t)s * h.Cp + ch * kHcBlockCh + lane * 8 + 4);
      gv[s][0] = a.x, gv[s][1] = a.y, gv[s][2] = a.z, gv[s][3] = a.w, gv[s][4] = b.x, gv[s][5] = b.y, gv[s][6] = b.z, gv[s][7] = b.w;
    }
    const bf16* wb = ring + (size_t)buf * kHcBlockClasses * kHcBlockCh + (warp * 8) * kHcBlockCh + lane * 8;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      Vec16<bf16> w;
      w.load(wb + q * kHcBlockCh);
#pragma unroll
      for (int s = 0; s < S; ++s)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[q][s] = fmaf(w.v[e], gv[s][e], acc[q][s]);
    }
    if (ch == h.nchunk - 1) {   // the classes of this block are complete
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int kl = g * kHcBlockClasses + warp * 8 + q;
        const float bk = (bfc && kl < nk) ? bfc[k0 + kl] : 0.f;
#pragma unroll
        for (int s = 0; s < S; ++s) {
          float v = acc[q][s];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          if (lane == 0 && kl < nk) zs[s * kHcMaxKc + kl] = v + bk;
          acc[q][s] = 0.f;
        }
      }
    }
  }
  cp_async_wait<0>();
  __syncthreads();

  // ---- 3. decision
  if (warp < S && b0 + warp < B) {
    const int s = warp, b = b0 + s;
    const int cls = (d.shift && d.shift_cls) ? d.shift_cls[b] : -1;
    const float sh = cls >= 0 && cls < K ? d.shift[b] : 0.f;
    float zr[kHcMaxKc / 32];
    float m = -INFINITY;
    int arg = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < kHcMaxKc / 32; ++i) {
      const int j = lane + 32 * i;
      zr[i] = j < nk ? zs[s * kHcMaxKc + j] : -INFINITY;
      if (j < nk) {
        if (k0 + j == cls) zr[i] += sh;
        if (z) z[(size_t)b * K + k0 + j] = zr[i];
        if (zr[i] > m) m = zr[i], arg = k0 + j;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, m, o);
      const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
      if (om > m || (om == m && oa < arg)) m = om, arg = oa;
    }
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < kHcMaxKc / 32; ++i)
      if (lane + 32 * i < nk) sum += expf(zr[i] - m);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) {
      float* mine = part + ((size_t)rank * S + s) * 4;
      hc_st_f32(hc_map(mine, 0), m);
      hc_st_f32(hc_map(mine + 1, 0), __int_as_float(arg));
      hc_st_f32(hc_map(mine + 2, 0), sum);
    }
  }
  hc_cluster_arrive();   // #3: the leader holds every CTA's triple
  hc_cluster_wait();
  if (rank != 0) return;
  if (tid < S && b0 + tid < B) {
    const int s = tid, b = b0 + s;
    float m = -INFINITY;
    int arg = 0x7fffffff;
    for (int r = 0; r < kHcCluster; ++r) {   // ranks hold ascending classes: strict > keeps the lowest argmax
      const float mr = part[(r * S + s) * 4];
      if (mr > m) m = mr, arg = __float_as_int(part[(r * S + s) * 4 + 1]);
    }
    float tot = 0.f;
    for (int r = 0; r < kHcCluster; ++r) {
      const float mr = part[(r * S + s) * 4];
      if (mr != -INFINITY) tot += part[(r * S + s) * 4 + 2] * expf(mr - m);   // a rank without classes holds -inf
    }
    const float cf = 1.0f / tot;
    if (d.conf) d.conf[b] = cf;
    if (d.pred) d.pred[b] = arg == 0x7fffffff ? 0 : arg;
    d.mask[b] = (uint8_t)((d.always_exit || cf >= d.thr) ? 1 : 0);
  }
  // ---- 4. scan, by the last tile
  __threadfence();
  __syncthreads();
  if (tid == 0) *flag = atomicAdd(d.done, 1u) == gridDim.x / kHcCluster - 1 ? 1 : 0;
  __syncthreads();
  if (!*flag) return;
  __threadfence();
  if (tid == 0) *d.done = 0;
  exit_scan<kHcThreads>(B, d);
}

template <int S>
inline cudaError_t hc_launch_t(const bf16* x, int HW, int C, const bf16* wfc, const float* bfc, int B, int K, float* z, const DecideArgs& d,
                               cudaStream_t st) {
  const HcShape h = hc_shape(C, K);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((B + S - 1) / S * kHcCluster));
  cfg.blockDim = dim3(kHcThreads);
  cfg.dynamicSmemBytes = hc_smem_bytes(S, h);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, head_cluster_kernel<S>, x, HW, C, wfc, bfc, B, K, z, d, h);
}
// d.done must be zero when the kernel starts and is zero again when it ends; d.tile_done is not used.
inline cudaError_t hc_launch(const bf16* x, int HW, int C, const bf16* wfc, const float* bfc, int B, int K, float* z, const DecideArgs& d,
                             cudaStream_t st) {
  switch (hc_tile_samples(B)) {
    case 1: return hc_launch_t<1>(x, HW, C, wfc, bfc, B, K, z, d, st);
    case 2: return hc_launch_t<2>(x, HW, C, wfc, bfc, B, K, z, d, st);
    default: return hc_launch_t<4>(x, HW, C, wfc, bfc, B, K, z, d, st);
  }
}
inline cudaError_t hc_context_init() {
  const size_t most = hc_smem_bytes(4, hc_shape(2048, kHcCluster * kHcMaxKc));
  cudaError_t e = cudaFuncSetAttribute(head_cluster_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(head_cluster_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(head_cluster_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most);
  return e;
}

constexpr int kCopyThreads = 256, kCopyUnroll = 8;

// feat_out[j] = feat[surv_idx[j]] for j < *n_surv, in vectors of type V (16 bytes whenever the row size
// allows), grid (chunks, max_rows).
template <typename V>
__global__ void __launch_bounds__(kCopyThreads)
gather_rows_kernel(const V* __restrict__ src, size_t vecs_per_row, const int32_t* __restrict__ surv_idx,
                   const int32_t* __restrict__ n_surv, V* __restrict__ dst, int rev) {
  const int j = rev ? (int)(gridDim.y - 1 - blockIdx.y) : (int)blockIdx.y;   // rev: last row first, each row from its end
  const unsigned bx = rev ? gridDim.x - 1 - blockIdx.x : blockIdx.x;
  if (j >= *n_surv) return;
  const V* s = src + (size_t)surv_idx[j] * vecs_per_row;
  V* d = dst + (size_t)j * vecs_per_row;
  const size_t v0 = (size_t)bx * (kCopyThreads * kCopyUnroll) + threadIdx.x;
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
