// Depthwise 3x3 pad-1 convolution on bf16 (stride 1 or 2) with the input staged in shared memory by TMA: the
// bandwidth-bound layers of the inverted-residual blocks.
//
// A depthwise layer does 9 MACs per element, so its only bound is HBM: what matters is how many bytes an SM keeps in
// flight.  A kernel that loads through registers holds one item's inputs per thread and stalls on every item.  Here
// one producer warp per persistent CTA asks the TMA unit for whole input tiles, a band of output rows x all columns x
// one block of up to 64 channels, including the one-pixel frame of the padding (coordinates start at -1; the unit
// zero-fills outside the image), into a ring of three slots: two or three tiles (up to 72 KB each) are in flight per
// SM whatever the consumers do.  Eight consumer warps compute from shared memory: a thread owns one vector of eight
// channels (its 72 weights stay in registers as stored) and walks strips of four consecutive output pixels of the
// tile, reading each of the 3 x 6 (stride 2: 3 x 9) input vectors of a strip once.  A quarter warp reads the eight
// channel vectors of one pixel, 128 contiguous bytes, so the reads are conflict-free without swizzling.  Every output
// sums its nine taps in ascending (r, s) with fp32 FMAs, scale / bias / activation in fp32, one rounding to bf16.
#pragma once
#include "conv_tc.cuh"

namespace ee {

struct DwParams {
  int H, W, C, Ho, Wo;
  int RB;          // output rows per tile
  int bands;       // ceil(Ho / RB)
  int tiles;       // B * bands, per channel block
  int cb;          // channels per block (dw_block_channels)
  int tile_bytes;  // ((RB - 1) * stride + 3) * (W + 2) * cb * 2
  int slot_bytes;  // tile_bytes rounded up to 128
  int act;
  int rev;         // 1: walk the tiles from the last one down
  const bf16* w;   // [C][3][3]
  const float* scale;
  const float* bias;
  bf16* y;         // [B][Ho][Wo][C]
  int* err_flag;
};

constexpr int kDwStages = 3;
constexpr int kDwConsumers = 256;
constexpr int kDwThreads = 32 + kDwConsumers;
constexpr int kDwMaxTileBytes = 72 * 1024;

__device__ __forceinline__ void tma_load_4d_tile(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

// POOL: the same staging for a 3x3 pad-1 window maximum (the max-pool behind a ResNet-style stem): taps outside the
// image are skipped (the frame's zeros must not win against negative inputs), no weights, no epilogue arithmetic.
template <int STRIDE, bool POOL>
__global__ void __launch_bounds__(kDwThreads, 1)
dwconv3x3_tma_kernel(const __grid_constant__ CUtensorMap tmX, DwParams p) {
  constexpr int P = kDwStrip, COLS = (P - 1) * STRIDE + 3;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_s = smem_u32(smem_raw);
  const uint32_t base = (raw_s + 127u) & ~127u;
  uint8_t* gen = smem_raw + (base - raw_s);
  const int bar_off = kDwStages * p.slot_bytes;
  const uint32_t bar0 = base + bar_off;
  auto full = [&](int s) { return bar0 + 8u * s; };
  auto empty = [&](int s) { return bar0 + 8u * (kDwStages + s); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int my_tiles = (int)blockIdx.x < p.tiles ? (p.tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  const int c0 = (int)blockIdx.y * p.cb;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kDwStages; ++s) {
      mbar_init(full(s), 1);
      mbar_init(empty(s), kDwConsumers / 32);   // lane 0 of each consumer warp
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX) : "memory");
  }
  __syncthreads();
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    if (lane == 0) {
      for (int j = 0; j < my_tiles; ++j) {
        const int tf = (int)blockIdx.x + j * (int)gridDim.x, t = p.rev ? p.tiles - 1 - tf : tf;
        const int b = t / p.bands, band = t - b * p.bands;
        const int s = j % kDwStages;
        if (!mbar_wait(empty(s), ((uint32_t)(j / kDwStages) & 1u) ^ 1u, p.err_flag)) break;
        mbar_expect_tx(full(s), (uint32_t)p.tile_bytes);
        tma_load_4d_tile(base + (uint32_t)(s * p.slot_bytes), &tmX, full(s), c0, -1, band * p.RB * STRIDE - 1, b);
      }
    }
    return;
  }

  const int tid = (int)threadIdx.x - 32;
  const int nv = p.cb >> 3;                 // channel vectors per block
  const int cvec = tid % nv, item0 = tid / nv, item_step = kDwConsumers / nv;
  const bool live = item0 < item_step;      // nv need not divide 256: the threads of the ragged tail idle
  const int c = c0 + cvec * 8;
  const bool c_in = c < p.C;
  uint32_t wr[36];   // the vector's 72 weights as stored: element e = channel e / 9, tap e % 9
#pragma unroll
  for (int i = 0; i < 9; ++i) {
    const uint4 v = (!POOL && c_in) ? __ldg(reinterpret_cast<const uint4*>(p.w + (size_t)c * 9) + i) : make_uint4(0u, 0u, 0u, 0u);
    wr[4 * i] = v.x, wr[4 * i + 1] = v.y, wr[4 * i + 2] = v.z, wr[4 * i + 3] = v.w;
  }
  auto weight = [&](int tap, int ch) {   // indices are compile-time constants after unrolling
    const int e = ch * 9 + tap;
    return (e & 1) ? __uint_as_float(wr[e >> 1] & 0xffff0000u) : __uint_as_float(wr[e >> 1] << 16);
  };
  float sc[8], bi[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    sc[e] = (p.scale && c_in) ? p.scale[c + e] : 1.f;
    bi[e] = (p.bias && c_in) ? p.bias[c + e] : 0.f;
  }
  const int strips = (p.Wo + P - 1) / P;
  const int Wc = p.W + 2;
  const int items = p.RB * strips;
  for (int j = 0; j < my_tiles; ++j) {
    const int tf = (int)blockIdx.x + j * (int)gridDim.x, t = p.rev ? p.tiles - 1 - tf : tf;
    const int b = t / p.bands, band = t - b * p.bands;
    const int s = j % kDwStages;
    if (!__all_sync(0xffffffffu, mbar_wait(full(s), (uint32_t)(j / kDwStages) & 1u, p.err_flag))) break;
    const uint8_t* tile = gen + (size_t)s * p.slot_bytes;
    if (live) {
      for (int it = item0; it < items; it += item_step) {
        const int ro = it / strips, st = it - ro * strips;
        const int wo0 = st * P;
        const int ho = band * p.RB + ro;
        uint4 v[3][COLS];
#pragma unroll
        for (int r = 0; r < 3; ++r) {
          const uint8_t* row = tile + (size_t)((ro * STRIDE + r) * Wc) * p.cb * 2 + cvec * 16;
#pragma unroll
          for (int q = 0; q < COLS; ++q) {
            const int col = min(wo0 * STRIDE + q, Wc - 1);   // columns past the frame only feed outputs that are not stored
            v[r][q] = *reinterpret_cast<const uint4*>(row + (size_t)col * p.cb * 2);
          }
        }
        float acc[P][8];
#pragma unroll
        for (int pp = 0; pp < P; ++pp)
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[pp][e] = POOL ? -INFINITY : 0.f;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
          const int hi = ho * STRIDE - 1 + r;
          const bool row_in = hi >= 0 && hi < p.H;
#pragma unroll
          for (int q = 0; q < COLS; ++q) {
            const uint32_t wd[4] = {v[r][q].x, v[r][q].y, v[r][q].z, v[r][q].w};
            float f[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              f[2 * i] = __uint_as_float(wd[i] << 16);
              f[2 * i + 1] = __uint_as_float(wd[i] & 0xffff0000u);
            }
#pragma unroll
            for (int pp = 0; pp < P; ++pp) {
              const int sx = q - pp * STRIDE;   // compile-time after unrolling
              if (sx >= 0 && sx < 3) {
                if constexpr (POOL) {
                  const int wi = wo0 * STRIDE - 1 + q;
                  if (row_in && wi >= 0 && wi < p.W) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[pp][e] = fmaxf(acc[pp][e], f[e]);
                  }
                } else {
#pragma unroll
                  for (int e = 0; e < 8; e += 2) {   // two independent round-to-nearest FMAs per instruction
                    float a0 = f[e], a1 = f[e + 1];
                    ffma2(a0, a1, weight(r * 3 + sx, e), weight(r * 3 + sx, e + 1), acc[pp][e], acc[pp][e + 1]);
                    acc[pp][e] = a0, acc[pp][e + 1] = a1;
                  }
                }
              }
            }
          }
        }
        if (c_in && ho < p.Ho) {
          bf16* yp = p.y + (((size_t)b * p.Ho + ho) * p.Wo + wo0) * p.C + c;
#pragma unroll
          for (int pp = 0; pp < P; ++pp) {
            if (wo0 + pp < p.Wo) {
              Vec16<bf16> o;
#pragma unroll
              for (int e = 0; e < 8; ++e) o.v[e] = POOL ? acc[pp][e] : apply_act(fmaf(sc[e], acc[pp][e], bi[e]), p.act);
              o.store(yp + (size_t)pp * p.C);
            }
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty(s)) : "memory");
  }
}

// Layers this kernel takes: depthwise 3x3 (or a 3x3 max-pool, w == nullptr), pad 1, stride 1 or 2, channels a multiple
// of 8, at most 254 columns, and a tile of one output row that fits a ring slot.
// Channels per block: the channels are cut into ceil(C / 64) blocks of equal size (a multiple of 8), so that no block
// is mostly empty (144 channels: 3 x 48, not 64 + 64 + 16).
inline int dw_block_channels(int C) {
  const int blocks = (C + 63) / 64;
  return ((C + blocks - 1) / blocks + 7) / 8 * 8;
}

inline bool dw_tma_supported(const ConvGeom& g, const void* x, const void* w, const void* y) {
  if (!(g.kh == 3 && g.kw == 3 && g.pad == 1 && (g.stride == 1 || g.stride == 2) && g.Cin % 8 == 0 && g.Cin == g.Cout)) return false;
  if ((((uintptr_t)x | (uintptr_t)w | (uintptr_t)y) & 15) != 0 || g.W + 2 > 256) return false;
  const int cb = dw_block_channels(g.Cin);
  return 3 * (g.W + 2) * cb * 2 <= kDwMaxTileBytes;
}

inline ee_status_t dw_context_init() {
  const int bytes = kDwStages * kDwMaxTileBytes + 256 + 128;
  cudaError_t e = cudaFuncSetAttribute(dwconv3x3_tma_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(dwconv3x3_tma_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(dwconv3x3_tma_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(dwconv3x3_tma_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  return e == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

// Tensor map of a depthwise layer's input, NHWC as (C, W, H, B), box = (cb, W + 2, rows, 1), no swizzle; cached in the
// layer like the other maps of caller buffers.
inline ee_status_t dw_input_map(const TcContext& c, const TcLayer& L, const void* ptr, int batch, int C, int H, int W, int cb, int rows,
                                const CUtensorMap** out) {
  for (auto& e : L.a_maps)
    if (e.ptr == ptr && e.batch == batch && e.kind == 5) {
      *out = &e.tm;
      return EE_OK;
    }
  TcLayer::Cached e;
  e.ptr = ptr, e.batch = batch, e.kind = 5;
  const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)batch};
  const cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)C * 2 * W, (cuuint64_t)C * 2 * W * H};
  const cuuint32_t box[4] = {(cuuint32_t)cb, (cuuint32_t)(W + 2), (cuuint32_t)rows, 1};
  const cuuint32_t es[4] = {1, 1, 1, 1};
  if (c.encode_tiled(&e.tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return EE_ERR_CUDA;
  if (L.a_maps.size() < 48) {
    L.a_maps.push_back(e);
    *out = &L.a_maps.back().tm;
  } else {
    L.a_maps[L.next_evict] = e;
    *out = &L.a_maps[L.next_evict].tm;
    L.next_evict = (L.next_evict + 1) % L.a_maps.size();
  }
  return EE_OK;
}

// L: only its map cache is used (a depthwise layer has no tensor-core plan).
inline ee_status_t dw_tma_launch(TcContext& c, const TcLayer& L, const ConvGeom& g, const void* x, const void* w, const float* scale,
                                 const float* bias, void* y, int* err_flag, cudaStream_t st) {
  DwParams p;
  p.H = g.H, p.W = g.W, p.C = g.Cin, p.Ho = g.Ho, p.Wo = g.Wo;
  p.cb = dw_block_channels(g.Cin);
  const int row_bytes = (g.W + 2) * p.cb * 2;
  int in_rows = kDwMaxTileBytes / row_bytes;                      // input rows a slot holds
  if (in_rows > 256) in_rows = 256;
  int rb_max = (in_rows - 3) / g.stride + 1;
  if (rb_max > g.Ho) rb_max = g.Ho;
  // Band height: a CTA's eight consumer warps take 256 / (cb / 8) strips per pass over a tile, a tile costs about one
  // more pass (waiting for the slot, hand-over), and the busiest CTA walks ceil(tiles / CTAs) tiles.  Take the height
  // that minimises that CTA's passes (bytes moved rise with shorter bands: each band re-reads two frame rows).
  const int chunks = cdiv(g.Cin, p.cb);
  const int ctas_x = std::max(1, c.sm_count / chunks);
  const int strips = (g.Wo + kDwStrip - 1) / kDwStrip;
  const int per_pass = kDwConsumers / std::max(1, p.cb / 8);
  long best = -1;
  p.RB = 1;
  for (int rb = 1; rb <= rb_max; ++rb) {
    const long tiles = (long)g.B * cdiv(g.Ho, rb);
    const long cost = cdiv(tiles, std::min<long>(tiles, ctas_x)) * (cdiv((long)rb * strips, per_pass) + 1);
    if (best < 0 || cost <= best) best = cost, p.RB = rb;   // ties: the taller band (fewer frame rows re-read)
  }
  const int rows = (p.RB - 1) * g.stride + 3;
  p.bands = cdiv(g.Ho, p.RB);
  p.tiles = g.B * p.bands;
  p.tile_bytes = rows * row_bytes;
  p.slot_bytes = (int)align_up((size_t)p.tile_bytes, 128);
  p.act = g.act;
  p.rev = L.rev ? 1 : 0;
  p.w = (const bf16*)w, p.scale = scale, p.bias = bias, p.y = (bf16*)y;
  p.err_flag = err_flag;
  const CUtensorMap* t = nullptr;
  ee_status_t s = dw_input_map(c, L, x, g.B, g.Cin, g.H, g.W, p.cb, rows, &t);
  if (s != EE_OK) return s;
  const CUtensorMap tmX = *t;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(std::min(p.tiles, std::max(1, c.sm_count / chunks)), chunks);
  cfg.blockDim = dim3(kDwThreads);
  cfg.dynamicSmemBytes = kDwStages * p.slot_bytes + 256 + 128;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e;
  if (w)
    e = g.stride == 1 ? cudaLaunchKernelEx(&cfg, dwconv3x3_tma_kernel<1, false>, tmX, p) : cudaLaunchKernelEx(&cfg, dwconv3x3_tma_kernel<2, false>, tmX, p);
  else
    e = g.stride == 1 ? cudaLaunchKernelEx(&cfg, dwconv3x3_tma_kernel<1, true>, tmX, p) : cudaLaunchKernelEx(&cfg, dwconv3x3_tma_kernel<2, true>, tmX, p);
  return e == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace ee
