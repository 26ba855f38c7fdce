// Tensor-core convolution on CTA pairs: tcgen05.mma cta_group::2 over 256 x BN output tiles, persistent, with
// (tile, K-range) work units and a fixed-order split-K reduction through global memory.
//
// Why pairs.  In the one-CTA kernels of conv_tc.cuh a 128 x 128 x 64 K block moves 64 KB through the SM's shared
// memory (32 KB written by TMA, 32 KB read by the MMAs) for 256 clocks of MMA time, so the tile is bound by the 128 B/clk
// of shared memory at half the tensor rate.  Two CTAs of a cluster that issue one MMA of M = 256 hold half of the
// weight tile each: per CTA and K block 16 KB of activations and BN/2 rows of weights are staged and read while the
// tensor core does a 128 x BN x 64 product, twice the MMA time per staged byte at BN = 256.
//
// Why units.  The layers of the deep stages have few output tiles (23 to 368 pair tiles at the benchmark's batch
// sizes) and long K loops.  The K loop of every tile is cut into `splits` fixed ranges of kb_per K blocks (a property
// of the layer, never of the batch, so the grouping of every sum is the same in any batch), and the (tile, range)
// units are dealt round-robin to one persistent CTA pair per SM pair.  A unit whose tile has several ranges leaves
// its fp32 partial tile in global memory (each epilogue warp its own 32-row x BN/2-column region, stored so that a
// warp's accesses are contiguous) and bumps that region's counter; the warp that finds the counter complete adds the
// partials in ascending range order, applies the epilogue and stores.  Nobody waits for anybody: the last arriver
// does the work.  The counters return to zero for the next launch.
//
// Warp roles per CTA (320 threads): warp 0 issues the TMA loads of its own half of the operands (signalling the
// leader CTA's barrier), warp 1 owns the TMEM allocation and, in the leader CTA, issues the MMAs for both CTAs,
// warps 2-9 run the epilogue: two warps per TMEM lane quarter, one per half of the columns.  The accumulator is
// double-buffered in TMEM (2 x BN columns), so the epilogue of unit i overlaps the MMAs of unit i + 1.  Residual tiles
// are fetched by the epilogue warps themselves (TMA into their staging chunks) while the MMAs of the unit still run.
// No TMA load uses cluster multicast: every CTA fetches its own tiles.  Every wait on an mbarrier is bounded.
#pragma once
#include "conv_tc.cuh"

namespace ee {

constexpr int kPairThreads = 320;   // producer warp, MMA warp, eight epilogue warps
constexpr int kPairEpiWarps = 8;

struct PairParams {
  int M, N;             // valid rows (B*Ho*Wo) and Cout
  int taps, kw;         // kh*kw and kw
  int cblocks;          // ceil(Cin / 64)
  int Ho, Wo, stride, pad, pad_w;
  int im2col;           // 0: A is a plain [rows][Cin] matrix, 1: im2col tensor map
  int act;
  int has_res;
  const float* scale;
  const float* bias;
  int* err_flag;
  int splits, kb_per;   // K ranges per tile and K blocks per range (fixed per layer)
  int m_tiles, n_tiles; // pair tiles: ceil(M / 256) x ceil(N / BN)
  int rev;              // 1: walk the units from the last one down
  float* partial;       // split-K partial tiles (splits > 1)
  unsigned* counters;   // per (tile, CTA of the pair, epilogue warp); zero between launches
  int res_late;         // the residual operand is written by the layer just before this one in the same launch
};

template <int BN>
struct PairSmem {
  static constexpr int kStages = BN == 256 ? 4 : 6;
  static constexpr int kABytes = kTcBM * kTcBK * 2;         // this CTA's 128 rows of the A tile
  static constexpr int kBBytes = (BN / 2) * kTcBK * 2;      // this CTA's half of the weight tile
  static constexpr int kStage = kABytes + kBBytes;
  static constexpr int kTiles = kStages * kStage;
  static constexpr int kChunks = BN / 128;                  // 64-column chunks per epilogue warp
  static constexpr int kWarpIo = kChunks * 4096;            // staging of one warp: chunks of 32 rows x 128 bytes
  static constexpr int kIoOff = kTiles;
  static constexpr int kSbOff = kIoOff + kPairEpiWarps * kWarpIo;
  static constexpr int kBarOff = kSbOff + kPairEpiWarps * 2 * (BN / 2) * 4;   // scale | bias of each warp's columns
  static constexpr int kNumBars = 2 * kStages + 4 + kPairEpiWarps;
  static constexpr int kBytes = kBarOff + kNumBars * 8 + 16 + 1024;
  static_assert(kBytes <= 227 * 1024, "exceeds the shared memory of an SM");
};

// ----------------------------------------------------------------------------- PTX wrappers (pair forms)

__device__ __forceinline__ bool mbar_wait_for(uint32_t bar, uint32_t parity, int* err_flag, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > limit) {
      atomicExch(err_flag, (int)EE_ERR_TIMEOUT);
      return false;
    }
  }
  return true;
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in the CTA of rank `rank`
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
  uint32_t d;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(d) : "r"(addr), "r"(rank));
  return d;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;\n barrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Loads of a CTA pair: the destination is this CTA's shared memory, the barrier may live in either CTA of the pair.
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void tma2_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
               ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
__device__ __forceinline__ void tma2_load_im2col_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c, int w, int h, int n,
                                                    uint16_t woff, uint16_t hoff) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(woff), "h"(hoff)
      : "memory");
}
// One MMA over both CTAs of the pair: D (256 x N, rows 0-127 in the leader's TMEM, 128-255 in the peer's) (+)= A * B^T with
// each CTA's A rows and its half of B read from that CTA's shared memory at the descriptors' addresses.
__device__ __forceinline__ void umma2_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the barrier at this shared-memory offset in both CTAs once all MMAs issued so far have completed.
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"((uint16_t)3)
               : "memory");
}
__host__ __device__ constexpr uint32_t umma2_idesc(int n) {   // bf16 x bf16 -> fp32, K-major operands, M = 256 over the pair, N = n
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

// ----------------------------------------------------------------------------- kernel

constexpr int kPairMaxLayers = 20;

// Everything the kernel needs for a run of consecutive layers (one layer in the plain case).  Passed as one
// __grid_constant__ argument: the tensor maps are used in place from the parameter space.
struct PairStageArgs {
  int n_layers;
  unsigned* grid_bar;       // [kPairMaxLayers + 1] arrival counters of the barriers between layers; zero between launches
  int* err_flag;
  long long wait_cycles;
  PairParams layer[kPairMaxLayers];
  CUtensorMap tmA[kPairMaxLayers], tmW[kPairMaxLayers], tmR[kPairMaxLayers], tmO[kPairMaxLayers];
};

// Bounded spin on a global arrival counter (acquire at GPU scope).
__device__ __forceinline__ bool grid_bar_wait(const unsigned* ctr, unsigned target, int* err_flag, long long limit) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
  if (v >= target) return true;
  const long long t0 = clock64();
  for (;;) {
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
    if (v >= target) return true;
    if (clock64() - t0 > limit) {
      atomicExch(err_flag, (int)EE_ERR_TIMEOUT);
      return false;
    }
  }
}

// A run of layers in one launch.  Layer l + 1 reads what layer l wrote, so between two layers every CTA's epilogue
// warps wait for their own output stores to complete and the CTA arrives on a global counter; a CTA's producer
// requests the first weight tiles of the next layer at once (nobody writes weights) and spins on the counter only
// before its first activation tile.  The ring, the accumulator parity and the staging chunks carry on across layers.
// All CTAs of the grid must be resident together (the grid is never larger than one CTA per SM); the spin is bounded
// like every other wait.  With n_layers = 1 there is no barrier at all.
template <int BN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
conv_igemm_tcgen05_pair_kernel(const __grid_constant__ PairStageArgs A) {
  extern __shared__ uint8_t smem_raw[];
  using S = PairSmem<BN>;
  constexpr int kStages = S::kStages;
  constexpr int HALF = BN / 2;   // columns per epilogue warp = weight rows per CTA
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t bar0 = base + S::kBarOff;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * kStages + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * kStages + 2 + b); };
  auto res_bar = [&](int w) { return bar0 + 8u * (2 * kStages + 4 + w); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + S::kBarOff + S::kNumBars * 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();        // 0: leader (issues the MMAs), 1: peer
  const int pair = (int)(blockIdx.x >> 1), n_pairs = (int)(gridDim.x >> 1);
  const long long limit = A.wait_cycles;
  const int L = A.n_layers;
  int* const err_flag = A.err_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);    // the leader's expect_tx arrive; both CTAs' loads complete_tx on the leader's barrier
      mbar_init(empty_bar(s), 1);   // the MMA commit, delivered to both CTAs
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full(b), 1);
      mbar_init(acc_empty(b), 2 * kPairEpiWarps);   // every epilogue warp of both CTAs (used in the leader only)
    }
    for (int w = 0; w < kPairEpiWarps; ++w) mbar_init(res_bar(w), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&A.tmA[0]) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&A.tmW[0]) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&A.tmO[0]) : "memory");
  }
  if (warp == 1) {  // two accumulators of BN fp32 columns, allocated in both CTAs of the pair
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(2 * BN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  cluster_sync_all();   // barriers of both CTAs initialised, both TMEM allocations done
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // units of this pair in layer `l`: unit i -> (tile, K range)
  auto units_of = [&](const PairParams& p) {
    const int total = p.m_tiles * p.n_tiles * p.splits;
    return pair < total ? (total - 1 - pair) / n_pairs + 1 : 0;
  };
  auto unit_of = [&](const PairParams& p, int i, int& mt, int& nt, int& z) {
    const int total = p.m_tiles * p.n_tiles * p.splits;
    const int uf = pair + i * n_pairs, u = p.rev ? total - 1 - uf : uf;
    const int t = u / p.splits;
    z = u - t * p.splits;
    mt = t / p.n_tiles;
    nt = t - mt * p.n_tiles;
  };

  if (warp == 0) {
    if (lane == 0) {
      int g = 0;   // K blocks issued so far, across units and layers: the ring never drains at a boundary
      bool ok = true;
      for (int l = 0; l < L && ok; ++l) {
        const PairParams& p = A.layer[l];
        const CUtensorMap* tmA = &A.tmA[l];
        const CUtensorMap* tmW = &A.tmW[l];
        const int num_kb_all = p.taps * p.cblocks;
        const int my_units = units_of(p);
        bool inputs_ready = l == 0;   // layer 0: the dependency wait above
        for (int i = 0; i < my_units && ok; ++i) {
          int mt, nt, z;
          unit_of(p, i, mt, nt, z);
          const int m0 = mt * 256 + (int)rank * kTcBM;       // this CTA's rows
          const int nb0 = nt * BN + (int)rank * HALF;        // this CTA's weight rows
          const bool rows = m0 < p.M;                        // a peer whose rows all lie past M loads no A tile
          const bool peer_rows = mt * 256 + kTcBM < p.M;
          const int kb_begin = z * p.kb_per, kb_end = min(num_kb_all, kb_begin + p.kb_per);
          int cw = 0, ch = 0, cn = 0;
          if (p.im2col && rows) {
            const int hw = p.Ho * p.Wo;
            cn = m0 / hw;
            const int rem = m0 - cn * hw;
            const int ho = rem / p.Wo;
            cw = (rem - ho * p.Wo) * p.stride - p.pad_w;
            ch = ho * p.stride - p.pad;
          }
          auto arm_and_load_w = [&](int kb, int gg) -> bool {
            const int s = gg % kStages;
            const uint32_t ph = (uint32_t)(gg / kStages) & 1u;
            const int tap = kb / p.cblocks, cb = kb - tap * p.cblocks;
            if (!mbar_wait_for(empty_bar(s), ph ^ 1u, err_flag, limit)) return false;
            if (rank == 0) mbar_expect_tx(full_bar(s), (uint32_t)(2 * S::kBBytes + S::kABytes + (peer_rows ? S::kABytes : 0)));
            tma2_load_3d(base + (uint32_t)s * S::kStage + S::kABytes, tmW, map_to_rank(full_bar(s), 0), cb * kTcBK, tap, nb0);
            return true;
          };
          auto load_a = [&](int kb, int gg) {
            if (!rows) return;
            const int s = gg % kStages;
            const int tap = kb / p.cblocks, cb = kb - tap * p.cblocks;
            const uint32_t sa = base + (uint32_t)s * S::kStage, fb = map_to_rank(full_bar(s), 0);
            if (p.im2col) {
              const int r = tap / p.kw;
              tma2_load_im2col_4d(sa, tmA, fb, cb * kTcBK, cw, ch, cn, (uint16_t)(tap - r * p.kw), (uint16_t)r);
            } else {
              tma2_load_2d(sa, tmA, fb, cb * kTcBK, m0);
            }
          };
          int kb = kb_begin;
          if (!inputs_ready) {
            // first unit of a later layer: weight tiles of the first ring slots now, activation tiles once every CTA
            // of the grid has finished the layer before
            const int ahead = min(kStages, kb_end - kb_begin);
            for (int j = 0; j < ahead && ok; ++j) ok = arm_and_load_w(kb_begin + j, g + j);
            if (ok) ok = grid_bar_wait(A.grid_bar + (l - 1), gridDim.x, err_flag, limit);
            if (!ok) break;
            asm volatile("fence.proxy.async.global;" ::: "memory");   // the acquire above orders the TMA reads below
            for (int j = 0; j < ahead; ++j) load_a(kb_begin + j, g + j);
            kb += ahead;
            g += ahead;
            inputs_ready = true;
          }
          for (; kb < kb_end; ++kb, ++g) {
            ok = arm_and_load_w(kb, g);
            if (!ok) break;
            load_a(kb, g);
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = umma2_idesc(BN);
      int g = 0, ui = 0;   // K blocks and units so far, across layers
      bool ok = true;
      for (int l = 0; l < L && ok; ++l) {
        const PairParams& p = A.layer[l];
        const int num_kb_all = p.taps * p.cblocks;
        const int my_units = units_of(p);
        for (int i = 0; i < my_units && ok; ++i, ++ui) {
          int mt, nt, z;
          unit_of(p, i, mt, nt, z);
          const int kb_begin = z * p.kb_per, kb_end = min(num_kb_all, kb_begin + p.kb_per);
          const int b = ui & 1;
          if (ui >= 2) {  // the epilogue warps of both CTAs must have drained this accumulator (unit ui - 2)
            ok = mbar_wait_for(acc_empty(b), (uint32_t)((ui >> 1) - 1) & 1u, err_flag, limit);
            if (!ok) break;
            tc_fence_after();
          }
          const uint32_t acc = tmem_base + (uint32_t)(b * BN);
          for (int kb = kb_begin; kb < kb_end; ++kb, ++g) {
            const int s = g % kStages;
            const uint32_t ph = (uint32_t)(g / kStages) & 1u;
            ok = mbar_wait_for(full_bar(s), ph, err_flag, limit);
            if (!ok) break;
            tc_fence_after();
            const uint32_t sa = base + (uint32_t)s * S::kStage, sb = sa + S::kABytes;
#pragma unroll
            for (int k = 0; k < kTcBK / 16; ++k)
              umma2_bf16(acc, umma_desc(sa + k * 32), umma_desc(sb + k * 32), idesc, (uint32_t)((kb > kb_begin) | (k != 0)));
            umma2_commit_both(empty_bar(s));   // frees the slot in both CTAs once these MMAs have read it
          }
          if (ok) umma2_commit_both(acc_full(b));
        }
      }
    }
  } else {
    const int ew = warp - 2;                 // 0..7
    const int q = warp & 3;                  // TMEM lane quarter this warp may read
    const int h = ew >> 2;                   // which half of the tile's columns
    float* sc = reinterpret_cast<float*>(gen + S::kSbOff) + ew * 2 * HALF;   // this warp's scale | bias
    uint8_t* io = gen + S::kIoOff + ew * S::kWarpIo;
    const uint32_t io_s = base + S::kIoOff + ew * S::kWarpIo;
    const uint32_t acc_empty_leader0 = map_to_rank(acc_empty(0), 0), acc_empty_leader1 = map_to_rank(acc_empty(1), 0);
    bool ok = true;
    bool pending = false;      // lane 0: a bulk store group of this warp may still be in flight
    uint32_t res_phase = 0;
    int ui = 0;
    int prev_units = 0;
    for (int l = 0; l < L; ++l) {   // a warp whose wait ran out skips the work but still meets the others at the layer's end
      const PairParams& p = A.layer[l];
      const CUtensorMap* tmR = &A.tmR[l];
      const CUtensorMap* tmO = &A.tmO[l];
      const int my_units = units_of(p);
      int sc_n0 = -1;
      for (int i = 0; i < my_units && ok; ++i, ++ui) {
        int mt, nt, z;
        unit_of(p, i, mt, nt, z);
        const int m0 = mt * 256 + (int)rank * kTcBM, n0 = nt * BN, c_base = n0 + h * HALF;   // this warp's first column
        const int b = ui & 1;
        const bool live = m0 + q * 32 < p.M && c_base < p.N;    // this warp has something to store
        const bool split = p.splits > 1;
        if (c_base != sc_n0) {
          __syncwarp();
          for (int j = lane; j < HALF; j += 32) {
            const bool in = c_base + j < p.N;
            sc[j] = (p.scale && in) ? p.scale[c_base + j] : 1.f;
            sc[HALF + j] = (p.bias && in) ? p.bias[c_base + j] : 0.f;
          }
          sc_n0 = c_base;
        }
        __syncwarp();
        // the staging chunks are about to be rewritten (residual load or output): the previous store must have read them
        if (lane == 0 && pending) {
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          pending = false;
        }
        __syncwarp();
        auto fetch_residual = [&]() {   // this warp's 32 rows x HALF columns of the residual operand, into the staging chunks
          if (lane == 0) {
            int chunks = 0;
            for (int c = 0; c < S::kChunks; ++c)
              if (c_base + c * 64 < p.N) ++chunks;
            mbar_expect_tx(res_bar(ew), (uint32_t)(chunks * 4096));
            for (int c = 0; c < S::kChunks; ++c)
              if (c_base + c * 64 < p.N) tma_load_2d(io_s + c * 4096, tmR, res_bar(ew), c_base + c * 64, m0 + q * 32);
          }
        };
        // res_late: the residual operand was written by the layer just before this one in the same launch, so it may
        // only be requested once this unit's accumulator is complete (its activation tiles came after the grid barrier)
        // Early request only when the layer that wrote the residual operand is known to be complete on the whole grid:
        // in layer 0, behind this layer's first unit (its accumulator implies the barrier before this layer), or
        // when this CTA worked in the layer before and the operand is older than that layer.
        const bool res_early = l == 0 || i > 0 || (prev_units > 0 && !p.res_late);
        const bool res_now = p.has_res && live && !split && res_early;
        if (res_now) fetch_residual();
        ok = __all_sync(0xffffffffu, mbar_wait_for(acc_full(b), (uint32_t)(ui >> 1) & 1u, err_flag, limit));
        if (!ok) break;
        tc_fence_after();
        if (p.has_res && live && !split && !res_early) {
          asm volatile("fence.proxy.async.global;" ::: "memory");
          fetch_residual();
        }
        const uint32_t acc = tmem_base + (uint32_t)(b * BN + h * HALF) + ((uint32_t)(q * 32) << 16);
        bool reduce = !split;
        float* part = nullptr;
        if (split) {
          // region of this warp in the partial tile of (tile, range z, CTA rank): [HALF / 4 column groups][32 lanes][4] fp32
          const size_t region = (size_t)32 * HALF;
          const size_t tile = (size_t)mt * p.n_tiles + nt;
          part = p.partial + (((tile * p.splits) * 2 + rank) * kPairEpiWarps + ew) * region;   // range 0; range z at + z * 2 * 8 * region
          float* mine = part + (size_t)z * 2 * kPairEpiWarps * region;
#pragma unroll 1
          for (int c = 0; c < S::kChunks; ++c) {
            float va[32], vb[32];
            tmem_ld32_issue(acc + (uint32_t)(c * 64), va);
            tmem_ld32_issue(acc + (uint32_t)(c * 64 + 32), vb);
            tmem_ld_wait(va, vb);
            if (live) {
#pragma unroll
              for (int g4 = 0; g4 < 8; ++g4) {
                __stcg(reinterpret_cast<float4*>(mine) + (size_t)(c * 16 + g4) * 32 + lane, make_float4(va[4 * g4], va[4 * g4 + 1], va[4 * g4 + 2], va[4 * g4 + 3]));
                __stcg(reinterpret_cast<float4*>(mine) + (size_t)(c * 16 + 8 + g4) * 32 + lane, make_float4(vb[4 * g4], vb[4 * g4 + 1], vb[4 * g4 + 2], vb[4 * g4 + 3]));
              }
            }
          }
          tc_fence_before();
          __threadfence();
          __syncwarp();
          unsigned old = 0;
          if (lane == 0) {
            mbar_arrive_cluster(b ? acc_empty_leader1 : acc_empty_leader0);   // accumulator drained
            if (live) old = atomicAdd(p.counters + (tile * 2 + rank) * kPairEpiWarps + ew, 1u);
          }
          old = __shfl_sync(0xffffffffu, old, 0);
          reduce = live && old == (unsigned)(p.splits - 1);
          if (reduce) {
            __threadfence();
            if (lane == 0) p.counters[(tile * 2 + rank) * kPairEpiWarps + ew] = 0u;   // ready for the next launch
            if (p.has_res) {
              asm volatile("fence.proxy.async.global;" ::: "memory");
              fetch_residual();
            }
          }
        }
        if (reduce && (p.has_res && live)) {
          ok = __all_sync(0xffffffffu, mbar_wait_for(res_bar(ew), res_phase, err_flag, limit));
          res_phase ^= 1u;
          if (!ok) break;
        }
#pragma unroll 1
        for (int c = 0; c < S::kChunks; ++c) {
          float va[32], vb[32];
          if (!split) {
            tmem_ld32_issue(acc + (uint32_t)(c * 64), va);
            tmem_ld32_issue(acc + (uint32_t)(c * 64 + 32), vb);
            tmem_ld_wait(va, vb);
            if (c == S::kChunks - 1) {  // this warp's share of the accumulator is in registers: the MMA warp may refill it
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive_cluster(b ? acc_empty_leader1 : acc_empty_leader0);
            }
          } else if (reduce) {
            // partials of ranges 0, 1, ... in ascending order (range 0 first, so the sum starts from it)
            const size_t zs = (size_t)2 * kPairEpiWarps * 32 * HALF / 4;   // float4 stride between ranges
            const float4* p4 = reinterpret_cast<const float4*>(part) + (size_t)(c * 16) * 32 + lane;
#pragma unroll
            for (int g4 = 0; g4 < 8; ++g4) {
              const float4 x = __ldcg(p4 + (size_t)g4 * 32), y = __ldcg(p4 + (size_t)(8 + g4) * 32);
              va[4 * g4] = x.x, va[4 * g4 + 1] = x.y, va[4 * g4 + 2] = x.z, va[4 * g4 + 3] = x.w;
              vb[4 * g4] = y.x, vb[4 * g4 + 1] = y.y, vb[4 * g4 + 2] = y.z, vb[4 * g4 + 3] = y.w;
            }
            for (int zz = 1; zz < p.splits; ++zz) {
#pragma unroll
              for (int g4 = 0; g4 < 8; ++g4) {
                const float4 x = __ldcg(p4 + zz * zs + (size_t)g4 * 32), y = __ldcg(p4 + zz * zs + (size_t)(8 + g4) * 32);
                va[4 * g4] += x.x, va[4 * g4 + 1] += x.y, va[4 * g4 + 2] += x.z, va[4 * g4 + 3] += x.w;
                vb[4 * g4] += y.x, vb[4 * g4 + 1] += y.y, vb[4 * g4 + 2] += y.z, vb[4 * g4 + 3] += y.w;
              }
            }
          }
          if (!reduce || !live || c_base + c * 64 >= p.N) continue;
          uint8_t* line = io + c * 4096 + lane * 128;   // this thread's 128-byte row of the chunk, 16-byte groups XOR-swizzled with the row
#pragma unroll
          for (int sub = 0; sub < 2; ++sub) {
            const float* v = sub ? vb : va;
#pragma unroll
            for (int gq = 0; gq < 4; ++gq) {
              const int col = c * 64 + sub * 32 + gq * 8;    // within this warp's HALF columns
              if (c_base + col >= p.N) break;
              uint4* chunk = reinterpret_cast<uint4*>(line + (((sub * 4 + gq) ^ (lane & 7)) << 4));
              if (p.has_res)
                *chunk = epilogue8_act<true>(p.act, v + gq * 8, sc + col, sc + HALF + col, *chunk);
              else
                *chunk = epilogue8_act<false>(p.act, v + gq * 8, sc + col, sc + HALF + col, make_uint4(0u, 0u, 0u, 0u));
            }
          }
        }
        if (reduce && live) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the TMA unit
          __syncwarp();
          if (lane == 0) {
            for (int c = 0; c < S::kChunks; ++c)
              if (c_base + c * 64 < p.N) tma_store_2d(tmO, io_s + c * 4096, c_base + c * 64, m0 + q * 32);   // rows past M, columns past N: clipped
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            pending = true;
          }
        }
      }
      prev_units = my_units;
      if (l + 1 < L) {
        // end of a layer: this warp's stores must be complete (not merely read from shared memory) before the CTA tells
        // the grid that its part of the layer's output is in place
        if (lane == 0) {
          asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
          pending = false;
        }
        __threadfence();
        asm volatile("bar.sync 2, 256;" ::: "memory");   // the eight epilogue warps of this CTA
        if (ew == 0 && lane == 0) {
          asm volatile("fence.proxy.async.global;" ::: "memory");
          asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(A.grid_bar + l) : "memory");
        }
      }
    }
    if (lane == 0 && pending) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  }
  // Both CTAs stay until the other is done with their barriers and tensor memory.
  tc_fence_before();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * BN) : "memory");
  }
  // the last CTA to leave puts the barrier counters back to zero for the next launch
  if (L > 1 && threadIdx.x == 0) {
    __threadfence();
    const unsigned done = atomicAdd(A.grid_bar + kPairMaxLayers, 1u);
    if (done == gridDim.x - 1) {
      for (int l = 0; l <= kPairMaxLayers; ++l) A.grid_bar[l] = 0u;
      __threadfence();
    }
  }
}

// Self-test of the bounded wait: one thread waits on a barrier nobody will ever signal.  The wait must run out after
// `limit` cycles, record EE_ERR_TIMEOUT in the error word and let the kernel return normally.
__global__ void wait_selftest_kernel(int* err_flag, long long limit, int* reached_end) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait_for(smem_u32(&bar), 0, err_flag, limit);
    *reached_end = ok ? 2 : 1;   // 1: the wait gave up and the thread went on
  }
}

// ----------------------------------------------------------------------------- host side

// Kernel variants a tensor-core layer can run as (the per-(layer, batch) table of LayerPlan holds one of these).
enum TcVariant { TCV_AUTO = 0, TCV_PAIR256 = 1, TCV_PAIR128 = 2, TCV_RANGES_CLUSTER = 3, TCV_RANGES_LOCAL = 4, TCV_COUNT = 5 };

inline ee_status_t pair_context_init() {
  if (cudaFuncSetAttribute(conv_igemm_tcgen05_pair_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairSmem<256>::kBytes) != cudaSuccess ||
      cudaFuncSetAttribute(conv_igemm_tcgen05_pair_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairSmem<128>::kBytes) != cudaSuccess)
    return EE_ERR_CUDA;
  return EE_OK;
}

// Layers the pair kernel covers: what the one-CTA tensor-core kernel covers, without the gather mode.
inline bool pair_supported(const TcLayer& L, int variant) {
  if (L.gather || L.halo || L.stem7) return false;
  return variant == TCV_PAIR256 ? L.cout > 128 : L.cout > 64;
}

// Bytes of split-K partial tiles the pair kernel needs for this layer at batch B (0 when the layer is not split).
inline size_t pair_partial_bytes(const TcLayer& L, int B, int bn) {
  if (L.splits <= 1) return 0;
  const long tiles = (long)cdiv((long)B * L.out_h * L.out_w, 256) * cdiv(L.cout, bn);
  return (size_t)tiles * L.splits * 256 * bn * sizeof(float);
}
inline size_t pair_counter_words(const TcLayer& L, int B) {   // BN = 128 has the most tiles
  return (size_t)cdiv((long)B * L.out_h * L.out_w, 256) * cdiv(L.cout, 128) * 2 * kPairEpiWarps;
}

// Fills layer slot `slot` of `args` for one layer at batch B.
inline ee_status_t pair_fill_layer(TcContext& c, const TcLayer& L, int bn, const void* src, const void* res, void* dst, int B,
                                   const float* scale, const float* bias, float* partial, size_t partial_bytes, unsigned* counters,
                                   bool res_late, PairStageArgs* args, int slot) {
  if (((uintptr_t)src & 15) || ((uintptr_t)dst & 15) || ((uintptr_t)res & 15)) return EE_ERR_INVALID_ARG;
  const CUtensorMap* t = nullptr;
  ee_status_t s = tc_buffer_map(c, L, dst, B, 1, &t);
  if (s != EE_OK) return s;
  args->tmO[slot] = *t;
  if ((s = tc_buffer_map(c, L, src, B, 0, &t)) != EE_OK) return s;
  args->tmA[slot] = *t;
  args->tmR[slot] = args->tmO[slot];
  if (res) {
    if ((s = tc_buffer_map(c, L, res, B, 1, &t)) != EE_OK) return s;
    args->tmR[slot] = *t;
  }
  args->tmW[slot] = bn == 256 ? L.tm_w_half[0] : L.tm_w_half[1];
  PairParams& p = args->layer[slot];
  p.M = B * L.out_h * L.out_w;
  p.N = L.cout;
  p.taps = L.kh * L.kw;
  p.kw = L.kw;
  p.cblocks = cdiv(L.cin, kTcBK);
  p.Ho = L.out_h, p.Wo = L.out_w, p.stride = L.stride, p.pad = L.pad, p.pad_w = L.pad_w;
  p.im2col = L.im2col ? 1 : 0;
  p.act = L.act;
  p.has_res = res ? 1 : 0;
  p.scale = scale, p.bias = bias;
  p.err_flag = nullptr;
  p.splits = L.splits, p.kb_per = L.kb_per;
  p.m_tiles = cdiv(p.M, 256), p.n_tiles = cdiv(p.N, bn);
  p.rev = L.rev ? 1 : 0;
  p.partial = partial;
  p.counters = counters;
  p.res_late = res_late ? 1 : 0;
  if (p.splits > 1 && (!partial || !counters || partial_bytes < pair_partial_bytes(L, B, bn))) return EE_ERR_CAPACITY;
  return EE_OK;
}

// Launches the layers filled into `args` (n_layers of them) as one kernel.
inline ee_status_t pair_launch_args(TcContext& c, PairStageArgs& args, int bn, int* err_flag, unsigned* grid_bar, long long wait_cycles,
                                    cudaStream_t st) {
  if (args.n_layers < 1 || args.n_layers > kPairMaxLayers || (args.n_layers > 1 && !grid_bar)) return EE_ERR_INTERNAL;
  args.err_flag = err_flag;
  args.grid_bar = grid_bar;
  args.wait_cycles = wait_cycles;
  long units = 0;
  for (int l = 0; l < args.n_layers; ++l) units = std::max(units, (long)args.layer[l].m_tiles * args.layer[l].n_tiles * args.layer[l].splits);
  const int pairs = (int)std::min<long>(units, c.sm_count / 2);   // never more than one CTA per SM: the grid is co-resident
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = bn == 256 ? PairSmem<256>::kBytes : PairSmem<128>::kBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = bn == 256 ? cudaLaunchKernelEx(&cfg, conv_igemm_tcgen05_pair_kernel<256>, args)
                            : cudaLaunchKernelEx(&cfg, conv_igemm_tcgen05_pair_kernel<128>, args);
  return e == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

inline ee_status_t pair_launch(TcContext& c, const TcLayer& L, int variant, const void* src, const void* res, void* dst, int B,
                               const float* scale, const float* bias, int* err_flag, float* partial, size_t partial_bytes,
                               unsigned* counters, long long wait_cycles, cudaStream_t st) {
  const int bn = variant == TCV_PAIR256 ? 256 : 128;
  static thread_local PairStageArgs args;   // 13 KB: kept off the stack
  args.n_layers = 1;
  ee_status_t s = pair_fill_layer(c, L, bn, src, res, dst, B, scale, bias, partial, partial_bytes, counters, false, &args, 0);
  if (s != EE_OK) return s;
  return pair_launch_args(c, args, bn, err_flag, nullptr, wait_cycles, st);
}

}  // namespace ee
