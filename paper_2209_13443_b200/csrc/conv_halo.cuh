// 3x3 stride-1 pad-1 convolution over 64 input channels (bf16) as an implicit GEMM on tcgen05.mma whose A operand is
// read from shared memory nine times but fetched from L2 once.
//
// The generic kernel of conv_tc.cuh gathers one 128-pixel x 64-channel A tile per filter tap (im2col tensor map):
// nine loads of 16 KB per output tile, which makes a 64-channel 3x3 layer wait on its SM's L2 port, not on the
// tensor pipe.  Here one persistent CTA per SM keeps the layer's nine 64 x 64 weight tiles resident in shared memory
// and walks output tiles of R whole image rows.  Per tile the TMA unit brings the R + 2 input rows the tile touches,
// each with one zero pixel left and right (coordinates start at -1; the unit zero-fills outside the image), as one
// dense [R + 2][Wp = W + 2][64] block.  With 64 channels a pixel is exactly one 128-byte row of the K-major,
// 128-byte-swizzled operand layout, so the A operand of filter tap (r, s) is the same block viewed from pixel
// r * Wp + s on: output position m = y * Wp + x of the tile reads block row m + r * Wp + s.  The nine taps are nine
// descriptor offsets, not nine loads (paper Section II-C maps a convolution to a GEMM over a Toeplitz matrix; the
// overlapping rows of that matrix are never materialised, not even in shared memory).  Positions with x >= W are the
// padding columns of the flattened rows: they are computed and dropped (2 of every Wp rows).
//
// Warp roles as in conv_tc.cuh: warp 0 issues TMA loads into a ring of blocks, warp 1 owns TMEM and issues the MMAs
// into a double-buffered accumulator (2 x 64 columns), warps 2-5 run the epilogue (tcgen05.ld, folded-BN scale/bias,
// activation, one rounding to bf16) and store each pixel's 128 bytes straight to global memory.  Every wait on an
// mbarrier is bounded; on expiry the thread records EE_ERR_TIMEOUT and falls through to the common exit.
#pragma once
#include "conv_tc.cuh"

namespace ee {

struct HaloParams {
  int tiles;          // B * tiles_per_img
  int tiles_per_img;  // ceil(H / R)
  int H, W, Wp, R;    // image size, padded row length W + 2, output rows per tile
  int N;              // Cout (<= 64, a multiple of 8)
  int act;
  int rev;            // 1: walk the tiles from the last one down
  const float* scale;
  const float* bias;
  bf16* out;          // [B][H][W][N]
  int* err_flag;
};

constexpr int kHaloThreads = 192;                    // producer warp, MMA warp, four epilogue warps
constexpr int kHaloStages = 4;
constexpr int kHaloBlockRows = 256;                  // pixel rows of one ring slot: 128 + 2 * Wp + 2 <= 256
constexpr int kHaloBlockBytes = kHaloBlockRows * 128;
constexpr int kHaloTaps = 9;
constexpr int kHaloWTapBytes = 64 * kTcBK * 2;       // one tap: 64 filters x 64 channels

struct HaloSmem {
  static constexpr int kWOff = 0;
  static constexpr int kAOff = kWOff + kHaloTaps * kHaloWTapBytes;
  static constexpr int kScaleOff = kAOff + kHaloStages * kHaloBlockBytes;
  static constexpr int kBarOff = kScaleOff + 2 * 64 * 4;
  static constexpr int kBytes = kBarOff + 256 + 1024;
  static_assert(kAOff % 1024 == 0 && kBarOff % 8 == 0, "alignment");
  static_assert(kBytes <= 227 * 1024, "exceeds the shared memory of an SM");
};

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

// A descriptor may start at any 128-byte row of a swizzled block, not only at a multiple of 1024 bytes: the TMA unit
// and the tensor core both derive the 16-byte chunk permutation from the shared-memory address itself (address
// bits 7-9 select the permutation of bits 4-6), so a view shifted by whole rows finds every chunk where the load put
// it.  The descriptor's base-offset field stays zero (checked on the device: bit-exact against the oracle).

__global__ void __launch_bounds__(kHaloThreads, 1)
conv3x3_halo_tcgen05_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, HaloParams p) {
  extern __shared__ uint8_t smem_raw[];
  using S = HaloSmem;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  float* s_scale = reinterpret_cast<float*>(gen + S::kScaleOff);
  float* s_bias = s_scale + 64;
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen + S::kBarOff);
  const uint32_t bar0 = base + S::kBarOff;
  auto a_full = [&](int s) { return bar0 + 8u * s; };
  auto a_empty = [&](int s) { return bar0 + 8u * (kHaloStages + s); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * kHaloStages + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * kHaloStages + 2 + b); };
  const uint32_t w_bar = bar0 + 8u * (2 * kHaloStages + 4);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kHaloStages + 5);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int my_tiles = (int)blockIdx.x < p.tiles ? (p.tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kHaloStages; ++s) {
      mbar_init(a_full(s), 1);
      mbar_init(a_empty(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full(b), 1);
      mbar_init(acc_empty(b), 4);   // lane 0 of each epilogue warp
    }
    mbar_init(w_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
  }
  if (warp == 1) {  // two accumulators of 64 fp32 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(128) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // the weights are written by no kernel: request all nine taps before the dependency wait
  if (warp == 0 && lane == 0 && my_tiles > 0) {
    mbar_expect_tx(w_bar, kHaloTaps * kHaloWTapBytes);
    for (int tap = 0; tap < kHaloTaps; ++tap) tma_load_3d(base + S::kWOff + tap * kHaloWTapBytes, &tmW, w_bar, 0, tap, 0);
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    if (lane == 0) {
      const uint32_t block_bytes = (uint32_t)(p.Wp * (p.R + 2) * 128);
      for (int j = 0; j < my_tiles; ++j) {
        const int tf = (int)blockIdx.x + j * (int)gridDim.x, t = p.rev ? p.tiles - 1 - tf : tf;
        const int n = t / p.tiles_per_img, h0 = (t - n * p.tiles_per_img) * p.R;
        const int s = j % kHaloStages;
        const uint32_t ph = (uint32_t)(j / kHaloStages) & 1u;
        if (!mbar_wait(a_empty(s), ph ^ 1u, p.err_flag)) break;
        mbar_expect_tx(a_full(s), block_bytes);
        tma_load_4d(base + S::kAOff + (uint32_t)s * kHaloBlockBytes, &tmX, a_full(s), 0, -1, h0 - 1, n);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc(64);
      bool ok = my_tiles > 0 ? mbar_wait(w_bar, 0, p.err_flag) : true;
      for (int j = 0; j < my_tiles && ok; ++j) {
        const int b = j & 1;
        const int s = j % kHaloStages;
        const uint32_t ph = (uint32_t)(j / kHaloStages) & 1u;
        if (j >= 2) {  // the epilogue must have drained this accumulator (tile j - 2)
          ok = mbar_wait(acc_empty(b), (uint32_t)((j >> 1) - 1) & 1u, p.err_flag);
          if (!ok) break;
        }
        ok = mbar_wait(a_full(s), ph, p.err_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t acc = tmem_base + (uint32_t)(b * 64);
        const uint32_t sa = base + S::kAOff + (uint32_t)s * kHaloBlockBytes;
#pragma unroll
        for (int tap = 0; tap < kHaloTaps; ++tap) {
          const uint32_t a_tap = sa + (uint32_t)(((tap / 3) * p.Wp + (tap % 3)) * 128);
          const uint32_t w_tap = base + S::kWOff + tap * kHaloWTapBytes;
#pragma unroll
          for (int k = 0; k < kTcBK / 16; ++k)
            umma_bf16(acc, umma_desc(a_tap + k * 32), umma_desc(w_tap + k * 32), idesc, (uint32_t)((tap | k) != 0));
        }
        umma_commit(a_empty(s));    // frees the block once these MMAs have read it
        umma_commit(acc_full(b));
      }
    }
  } else {
    const int et = threadIdx.x - 64;  // 0..127
    if (et < 64) {
      const bool in = et < p.N;
      s_scale[et] = (p.scale && in) ? p.scale[et] : 1.f;
      s_bias[et] = (p.bias && in) ? p.bias[et] : 0.f;
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    const int q = warp & 3;           // TMEM lane quarter of this warp
    const int row = q * 32 + lane;    // position y * Wp + x of the tile
    const int y = row / p.Wp, x = row - y * p.Wp;
    const bool inside = y < p.R && x < p.W;
    for (int j = 0; j < my_tiles; ++j) {
      const int tf = (int)blockIdx.x + j * (int)gridDim.x, t = p.rev ? p.tiles - 1 - tf : tf;
      const int n = t / p.tiles_per_img, h0 = (t - n * p.tiles_per_img) * p.R;
      const int b = j & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(acc_full(b), (uint32_t)(j >> 1) & 1u, p.err_flag))) break;
      tc_fence_after();
      const uint32_t acc = tmem_base + (uint32_t)(b * 64) + ((uint32_t)(q * 32) << 16);
      float va[32], vb[32];
      tmem_ld32_issue(acc, va);
      tmem_ld32_issue(acc + 32u, vb);
      tmem_ld_wait(va, vb);
      tc_fence_before();   // the accumulator is in registers: the MMA warp may refill it
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acc_empty(b)) : "memory");
      if (inside && h0 + y < p.H) {
        bf16* dst = p.out + ((size_t)((size_t)n * p.H + h0 + y) * p.W + x) * p.N;
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          if (g * 8 < p.N) {
            const float* v = g < 4 ? va + g * 8 : vb + (g - 4) * 8;
            *reinterpret_cast<uint4*>(dst + g * 8) = epilogue8_act<false>(p.act, v, s_scale + g * 8, s_bias + g * 8, make_uint4(0u, 0u, 0u, 0u));
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(128) : "memory");
  }
}

// Layers this kernel takes: 3x3, stride 1, pad 1, exactly 64 input channels (one 128-byte row per pixel), at most 64
// output channels, no residual operand, and an image row short enough that a ring slot holds 128 positions plus the
// two rows and two pixels the last tap reaches past them.
inline bool halo_supported(const ee_layer_desc_t& d, int in_w) {
  return d.op == EE_OP_CONV && d.kh == 3 && d.kw == 3 && d.stride == 1 && d.pad == 1 && d.pad_w == 1 && d.cin == 64 && d.cout <= 64 && d.cout % 8 == 0 &&
         d.residual_from == EE_NO_RESIDUAL && kTcBM + 2 * (in_w + 2) + 2 <= kHaloBlockRows;
}

inline ee_status_t halo_context_init() {
  return cudaFuncSetAttribute(conv3x3_halo_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, HaloSmem::kBytes) == cudaSuccess
             ? EE_OK
             : EE_ERR_CUDA;
}

inline ee_status_t halo_launch(TcContext& c, const TcLayer& L, const void* src, void* dst, int B, const float* scale, const float* bias,
                               int* err_flag, cudaStream_t st) {
  if (((uintptr_t)src & 15) || ((uintptr_t)dst & 15)) return EE_ERR_INVALID_ARG;
  const CUtensorMap* t = nullptr;
  ee_status_t s = tc_buffer_map(c, L, src, B, 4, &t);
  if (s != EE_OK) return s;
  const CUtensorMap tmX = *t;
  HaloParams p;
  p.H = L.in_h, p.W = L.in_w, p.Wp = L.in_w + 2;
  p.R = kTcBM / p.Wp;
  p.tiles_per_img = cdiv(p.H, p.R);
  p.tiles = B * p.tiles_per_img;
  p.N = L.cout;
  p.act = L.act;
  p.rev = L.rev ? 1 : 0;
  p.scale = scale, p.bias = bias;
  p.out = (bf16*)dst;
  p.err_flag = err_flag;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(std::min(p.tiles, c.sm_count));
  cfg.blockDim = dim3(kHaloThreads);
  cfg.dynamicSmemBytes = HaloSmem::kBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, conv3x3_halo_tcgen05_kernel, tmX, L.tm_w, p) == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace ee
