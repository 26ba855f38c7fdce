// Tensor-core convolution for bf16 models on sm_100a: implicit GEMM on tcgen05.mma with the
// accumulator in TMEM, both operands staged in shared memory by TMA.
//
// GEMM view (paper Section II-C): D[M = B*Ho*Wo][N = Cout] = A[M][K] * W[N][K]^T with
// K = kh*kw*Cin.  The Toeplitz matrix A is never built: the TMA unit gathers each 128-pixel x
// 64-channel tile of it straight from the NHWC feature map (im2col tensor map: one filter tap per
// K block, zero fill for the padding halo), or reads it as a plain 2-D tile for 1x1 stride-1
// layers.  Batching appends samples along M, so one weight tile serves every sample of the batch.
//
// One CTA computes one 128 x BN output tile (or, in the persistent variant, walks many).  Warp roles: warp 0 issues
// TMA loads into a ring of shared-memory slots, warp 1 owns the TMEM allocation and issues the MMAs (one thread),
// the remaining warps run the epilogue: tcgen05.ld of the fp32 accumulator, folded-BN scale/bias, residual add (the
// residual tile was brought into shared memory by TMA while the main loop ran), activation, one rounding to bf16,
// then a TMA store of the tile from shared memory.  The K loop visits (tap, channel block) in a fixed order that
// does not depend on the batch size.  Variants (chosen per launch from the grid size, see tc_launch): shallow or
// deep ring, cluster split-K with a reduce-scatter through distributed shared memory, gather-mode A operand for
// 3-channel stems, and a persistent kernel with double-buffered TMEM accumulators for multi-wave 1x1 layers.
//
// Every wait on an mbarrier is bounded by a clock: on expiry the thread records EE_ERR_TIMEOUT in
// the model's error word and falls through to the common exit, which frees the TMEM columns.
#pragma once
#include <cuda.h>

#include <algorithm>
#include <vector>

#include "common.cuh"

namespace ee {

constexpr int kTcBM = 128;       // output pixels per CTA (= TMEM lanes)
constexpr int kTcBK = 64;        // bf16 elements per K block: 128 bytes = one swizzle span
constexpr int kTcThreads = 192;  // producer warp, MMA warp, four epilogue warps
constexpr long long kTcWaitCycles = 4000000000LL;  // ~2 s at boost clock; far beyond any healthy wait

struct TcParams {
  int M, N;             // valid rows (B*Ho*Wo) and Cout
  int taps, kw;         // kh*kw and kw
  int cblocks;          // ceil(Cin / 64); the TMA unit zero-fills channels past Cin in both operands
  int Ho, Wo, stride, pad, pad_w;   // pad: rows, pad_w: columns
  int im2col;           // 0: A is a plain [rows][Cin] matrix, 1: im2col tensor map
  int act;
  const float* scale;
  const float* bias;
  const bf16* residual;
  bf16* out;
  int* err_flag;
  int kb_per;           // split-K: K blocks per range (a property of the layer)
  int ranges;           // > 1 (one-CTA kernel without SPLIT): this CTA runs all `ranges` K ranges of its tile itself, each
                        // into an accumulator of its own, and adds them in ascending order in the epilogue - the same
                        // bits as `ranges` CTAs of a cluster reducing their partial tiles
  int rev;              // 1: walk the M tiles from the last one down (start where the producer of the input finished: its
                        // newest rows are the ones still in L2)
  // gather mode (layers whose pixel rows are not 16-byte units, e.g. a 3-channel stem): the epilogue warps build the A tile
  const bf16* gx;       // input feature map [B][gH][gW][gCin]
  int gH, gW, gCin, gkh, grun, grunp;  // run = kw*Cin contiguous taps of one filter row, zero-padded to runp columns
  // projection mode of the persistent kernel: the residual operand is itself a 1x1 convolution (stride stride2, no
  // padding, scale2 / bias2 / act2) of a second input with the same output geometry, computed into a second accumulator
  int cblocks2, im2col2, stride2, act2;
  const float* scale2;
  const float* bias2;
  // pooling partials of the persistent kernel: gap_g = 32 or 16 (0 = off): the epilogue also writes, for every block of
  // gap_g consecutive output rows, the column sums of the bf16-rounded outputs to gap_part[row / gap_g][N] (fp32), summed
  // pairwise over the rows with distances gap_g/2, ..., 2, 1 - the block sums of gap_blocks_kernel (head.cuh)
  int gap_g;
  float* gap_part;
};

// ----------------------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and records the fault) if the phase did not complete in time.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* err_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kTcWaitCycles) {
      atomicExch(err_flag, (int)EE_ERR_TIMEOUT);
      return false;
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
               ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
// im2col gather: 128 consecutive output pixels starting at base pixel (w, h, n), channels [c, c+64), filter tap (woff, hoff).
__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c, int w, int h, int n,
                                                   uint16_t woff, uint16_t hoff) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(woff), "h"(hoff)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile, rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);   // start address
  d |= (uint64_t)(1024 >> 4) << 32;              // stride between 8-row groups
  d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                        // 128-byte swizzle
  return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t umma_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTcBM >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.  Load and wait sit in one statement so that no
// use of the registers can be scheduled before the wait.
// Issue only; pair with tmem_ld_wait() before the registers are read.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// The "+r" ties make every later use of the 64 registers depend on the wait.
__device__ __forceinline__ void tmem_ld_wait(float* a, float* b) {
  uint32_t* x = reinterpret_cast<uint32_t*>(a);
  uint32_t* y = reinterpret_cast<uint32_t*>(b);
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) asm volatile("" : "+r"(x[i]), "+r"(y[i]));
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}

// v[i] = scale[i] * v[i] + bias[i] over N columns (a multiple of 4).  scale and bias are 16-byte aligned rows in shared
// memory that every lane reads at the same address: as float4 a load is one broadcast wavefront for four columns.
template <int N>
__device__ __forceinline__ void scale_bias(float* v, const float* scale, const float* bias) {
  const float4* s4 = reinterpret_cast<const float4*>(scale);
  const float4* b4 = reinterpret_cast<const float4*>(bias);
#pragma unroll
  for (int i = 0; i < N / 4; ++i) {
    const float4 s = s4[i], b = b4[i];
    v[4 * i] = fmaf(s.x, v[4 * i], b.x);
    v[4 * i + 1] = fmaf(s.y, v[4 * i + 1], b.y);
    v[4 * i + 2] = fmaf(s.z, v[4 * i + 2], b.z);
    v[4 * i + 3] = fmaf(s.w, v[4 * i + 3], b.w);
  }
}

// Epilogue arithmetic of eight output channels of one pixel: y = act(scale * acc + bias (+ residual)), one rounding to
// bf16, packed into 16 bytes.  Two fp32 FMAs per instruction (fma.rn.f32x2: two independent round-to-nearest FMAs, bit
// for bit the scalar result), and for ReLU the clamp rides on the conversion (cvt.rn.relu.bf16x2.f32: negative -> 0,
// then round; rounding is monotone and keeps 0, so this equals round(max(y, 0))).  scale / bias: 32-byte aligned
// shared-memory rows every lane reads at the same address (broadcast).  res: eight bf16 of the residual operand.
__device__ __forceinline__ void ffma2(float& x0, float& x1, float s0, float s1, float b0, float b1) {
  asm("{\n .reg .b64 a, s, b, d;\n mov.b64 a, {%0, %1};\n mov.b64 s, {%2, %3};\n mov.b64 b, {%4, %5};\n fma.rn.f32x2 d, a, s, b;\n"
      " mov.b64 {%0, %1}, d;\n}"
      : "+f"(x0), "+f"(x1)
      : "f"(s0), "f"(s1), "f"(b0), "f"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ uint32_t pack_bf16x2_relu(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
template <int ACT, bool RES>
__device__ __forceinline__ uint4 epilogue8(const float* acc, const float* scale, const float* bias, uint4 res) {
  const float4 s0 = *reinterpret_cast<const float4*>(scale), s1 = *reinterpret_cast<const float4*>(scale + 4);
  const float4 b0 = *reinterpret_cast<const float4*>(bias), b1 = *reinterpret_cast<const float4*>(bias + 4);
  float v[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) v[e] = acc[e];
  ffma2(v[0], v[1], s0.x, s0.y, b0.x, b0.y);
  ffma2(v[2], v[3], s0.z, s0.w, b0.z, b0.w);
  ffma2(v[4], v[5], s1.x, s1.y, b1.x, b1.y);
  ffma2(v[6], v[7], s1.z, s1.w, b1.z, b1.w);
  if (RES) {
    const uint32_t w[4] = {res.x, res.y, res.z, res.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {  // bf16 -> f32 is a 16-bit shift
      v[2 * i] += __uint_as_float(w[i] << 16);
      v[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (ACT == EE_ACT_RELU) {
      o[i] = pack_bf16x2_relu(v[2 * i], v[2 * i + 1]);
    } else if (ACT == EE_ACT_RELU6) {
      o[i] = pack_bf16x2(fminf(fmaxf(v[2 * i], 0.f), 6.f), fminf(fmaxf(v[2 * i + 1], 0.f), 6.f));
    } else {
      o[i] = pack_bf16x2(v[2 * i], v[2 * i + 1]);
    }
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}
// The same with the activation chosen at run time (one uniform branch per call site, not per element).
template <bool RES>
__device__ __forceinline__ uint4 epilogue8_act(int act, const float* acc, const float* scale, const float* bias, uint4 res) {
  if (act == EE_ACT_RELU) return epilogue8<EE_ACT_RELU, RES>(acc, scale, bias, res);
  if (act == EE_ACT_RELU6) return epilogue8<EE_ACT_RELU6, RES>(acc, scale, bias, res);
  return epilogue8<EE_ACT_NONE, RES>(acc, scale, bias, res);
}

// Column sums over the 32 rows a warp holds (ov: this lane's row, 64 bf16 columns as eight 16-byte groups), written as
// block sums of G rows (see TcParams::gap_g).  Halving butterfly: in the step of distance d a lane keeps half of its
// columns and receives its partner's values for them, so that every (block, column) sum is formed once, by the tree
// ((r, r + G/2), then distance G/4, ...).  Afterwards lane l holds columns [2l, 2l + 2) of the block (G = 32) or
// columns [4 (l % 16), + 4) of block l / 16 (G = 16).
template <int G>
__device__ __forceinline__ void gap_partial_store(const uint4* ov, int lane, float* dst, int cols_left, size_t block_stride, bool rows_ok) {
  float f[64];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t w[4] = {ov[i].x, ov[i].y, ov[i].z, ov[i].w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      f[8 * i + 2 * k] = __uint_as_float(w[k] << 16);
      f[8 * i + 2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
  }
#pragma unroll
  for (int d = G / 2, n = 32; d >= 1; d >>= 1, n >>= 1) {
    const bool up = (lane & d) != 0;
#pragma unroll
    for (int i = 0; i < n; ++i) {
      const float send = up ? f[i] : f[i + n], keep = up ? f[i + n] : f[i];
      f[i] = keep + __shfl_xor_sync(0xffffffffu, send, d);
    }
  }
  if (!rows_ok) return;
  if (G == 32) {
    if (2 * lane < cols_left) *reinterpret_cast<float2*>(dst + 2 * lane) = make_float2(f[0], f[1]);
  } else {
    const int c = 4 * (lane & 15);
    if (c < cols_left) *reinterpret_cast<float4*>(dst + (size_t)(lane >> 4) * block_stride + c) = make_float4(f[0], f[1], f[2], f[3]);
  }
}

// ----------------------------------------------------------------------------- kernel

// Gather-mode row builders (see the GATHER note on the kernel).  Thread `grow` writes row `grow` of the A tile of
// every K block: 64 bf16 = eight 16-byte chunks, chunk c stored at position c ^ (row & 7) of the 128-byte line, which
// is where the 128-byte swizzle of the MMA descriptor looks for it.  full barrier of slot s sits at bar0 + 8 s, the
// empty barrier at bar0 + 8 (STAGES + s).
template <int STAGES>
__device__ __forceinline__ void gather_rows_generic(const TcParams& p, const bf16* xb, bool row_in, int hi0, int off0, int row_elems,
                                                    uint8_t* gen, int stage_bytes, int grow, uint32_t bar0, int num_kb) {
  const __nv_bfloat16 zero = __float2bfloat16_rn(0.f);
  for (int i = 0; i < num_kb; ++i) {
    const int s = i % STAGES;
    const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
    if (!mbar_wait(bar0 + 8u * (STAGES + s), ph ^ 1u, p.err_flag)) break;
    uint8_t* line = gen + (size_t)s * stage_bytes + grow * 128;
    int rf = (i * kTcBK) / p.grunp, j = i * kTcBK - rf * p.grunp;   // filter row and column within its run
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
      __align__(16) bf16 v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int hi = hi0 + rf, off = off0 + j;
        const bool in = row_in && rf < p.gkh && j < p.grun && hi >= 0 && hi < p.gH && off >= 0 && off < row_elems;
        v[e] = in ? xb[(size_t)hi * row_elems + off] : zero;
        if (++j == p.grunp) {
          j = 0;
          ++rf;
        }
      }
      *reinterpret_cast<uint4*>(line + ((c ^ (grow & 7)) << 4)) = *reinterpret_cast<const uint4*>(v);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar0 + 8u * s) : "memory");
  }
}

// Same with the run geometry known at compile time: every (filter row, column) of every chunk is a constant, a pixel
// whose taps all lie inside the image row takes the check-free path, and loads carry immediate offsets.
template <int RUN, int RUNP, int KH, int NUMKB, int STAGES>
__device__ __forceinline__ void gather_rows_static(const TcParams& p, const bf16* xb, bool row_in, int hi0, int off0, int row_elems,
                                                   uint8_t* gen, int stage_bytes, int grow, uint32_t bar0) {
  const __nv_bfloat16 zero = __float2bfloat16_rn(0.f);
  const bool interior = off0 >= 0 && off0 + RUN <= row_elems;
  unsigned rows_ok = 0;  // bit r: filter row r lies inside the image
#pragma unroll
  for (int r = 0; r < KH; ++r)
    if (row_in && hi0 + r >= 0 && hi0 + r < p.gH) rows_ok |= 1u << r;
  const bf16* x0 = xb + (long)hi0 * row_elems + off0;  // tap (0, 0); only dereferenced where in range
#pragma unroll
  for (int i = 0; i < NUMKB; ++i) {
    const int s = i % STAGES;
    const uint32_t ph = (uint32_t)(i / STAGES) & 1u;
    if (!mbar_wait(bar0 + 8u * (STAGES + s), ph ^ 1u, p.err_flag)) break;
    uint8_t* line = gen + (size_t)s * stage_bytes + grow * 128;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      __align__(16) bf16 v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int k = i * kTcBK + c * 8 + e;
        const int rf = k / RUNP, j = k % RUNP;     // compile-time after unrolling
        if (rf < KH && j < RUN) {
          const bool in = ((rows_ok >> rf) & 1u) && (interior || (off0 + j >= 0 && off0 + j < row_elems));
          v[e] = in ? x0[(long)rf * row_elems + j] : zero;
        } else {
          v[e] = zero;
        }
      }
      *reinterpret_cast<uint4*>(line + ((c ^ (grow & 7)) << 4)) = *reinterpret_cast<const uint4*>(v);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar0 + 8u * s) : "memory");
  }
}

// Shared-memory plan of one CTA: a ring of STAGES operand slots (A 16 KB + W BN*128 B each), then, for layers whose
// residual operand is prefetched (RES), a dedicated 128 x BN bf16 tile that the producer fills with the residual at
// kernel start and the epilogue overwrites in place with the output.  Without it the output is staged in ring slot
// 0 once the main loop has drained it.  The shallow variants (3 slots, or 2 + residual tile: 96 KB at BN = 128) let
// two CTAs share an SM so one's epilogue overlaps the other's main loop; the deep variants (6, or 5 + tile) are
// used when the grid has at most one CTA per SM anyway and a longer ring hides more TMA latency.
template <int BN, int STAGES, bool RES>
struct TcSmem {
  static constexpr int kStages = STAGES;
  static constexpr int kABytes = kTcBM * kTcBK * 2;
  static constexpr int kBBytes = BN * kTcBK * 2;
  static constexpr int kStage = kABytes + kBBytes;
  static constexpr int kTiles = kStages * kStage;
  static constexpr int kIoBytes = kTcBM * BN * 2;
  static constexpr int kIoOff = RES ? kTiles : 0;
  static constexpr int kAfter = kTiles + (RES ? kIoBytes : 0);
  static constexpr int kBytes = kAfter + 2 * BN * 4 + 256 + 1024;  // + scale/bias, barriers, alignment slack
  static_assert(RES || kIoBytes <= kStage, "output staging must fit in ring slot 0");
  static_assert(kBytes <= 227 * 1024, "exceeds the shared memory of an SM");
};

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(tm), "r"(src), "r"(c0), "r"(c1)
               : "memory");
}

// tmA: activations (2-D tile map or im2col map), tmW: weights [Cin][taps][Cout], tmR / tmO: residual and output as
// [rows][Cout] matrices with a 64-column x 32-row box (128-byte swizzle).
//
// SPLIT: the K loop of one output tile is cut into gridDim.z (2 to 8) fixed ranges of p.kb_per K blocks, a
// property of the layer and never of the batch.  The CTAs of a tile form a thread-block cluster along z.  CTA z owns
// a slice of the tile's rows: once every CTA has drained its ring (first cluster barrier), each thread sends its row
// of the fp32 partial tile to the owner's shared memory through distributed shared memory; after the second
// barrier every CTA adds the partials of its rows in ascending range order, all from its own shared memory (a
// reduce-scatter), applies the epilogue to that slice and stores it.
//
// GATHER: operand A comes from CUDA cores instead of TMA, for layers whose pixel rows are not whole 16-byte units
// (a 3-channel stem).  K is laid out as kh runs of runp columns: run r holds the kw*Cin taps of filter row r, which
// are contiguous in the NHWC input, then zeros; the weights are packed the same way.  While the main loop runs, the
// four epilogue warps (one thread per tile row) read their pixel's taps and write them into the ring slot at the
// position the 128-byte swizzle expects; the Toeplitz matrix still never touches global memory.
template <int BN, int STAGES, bool RES, bool SPLIT, bool GATHER, bool LOCAL = false>   // LOCAL: TcParams::ranges accumulators in this CTA
__global__ void __launch_bounds__(kTcThreads, 2)
conv_igemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                          const __grid_constant__ CUtensorMap tmR, const __grid_constant__ CUtensorMap tmO, TcParams p) {
  static_assert(!(RES && SPLIT), "split-K tiles read their residual with plain loads");
  static_assert(!GATHER || (!RES && !SPLIT), "gather mode is for plain stem layers");
  extern __shared__ uint8_t smem_raw[];
  using S = TcSmem<BN, STAGES, RES>;
  constexpr int kStages = S::kStages;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
  uint8_t* gen = smem_raw + (base - raw);
  float* s_scale = reinterpret_cast<float*>(gen + S::kAfter);
  float* s_bias = s_scale + BN;
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen + S::kAfter + 2 * BN * 4);
  const uint32_t bar0 = base + S::kAfter + 2 * BN * 4;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  const uint32_t accum_bar = bar0 + 8u * (2 * kStages);
  const uint32_t res_bar = bar0 + 8u * (2 * kStages + 1);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = (p.rev ? (int)(gridDim.x - 1 - blockIdx.x) : (int)blockIdx.x) * kTcBM, n0 = blockIdx.y * BN;
  const int num_kb_all = p.taps * p.cblocks;
  const int kb_begin = SPLIT ? (int)blockIdx.z * p.kb_per : 0;
  const int kb_end = SPLIT ? min(num_kb_all, kb_begin + p.kb_per) : num_kb_all;
  const int num_kb = kb_end - kb_begin;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), GATHER ? 129 : 1);  // gather: 128 row writers + the weight tile's expect_tx
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(accum_bar, 1);
    mbar_init(res_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0 && lane == 0) {  // descriptor fetches overlap the rest of the prologue
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmO) : "memory");
    if (RES) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmR) : "memory");
  }
  static_assert(!LOCAL || (!SPLIT && !GATHER), "local K ranges are a mode of the plain one-CTA kernel");
  const int n_acc = LOCAL ? max(p.ranges, 1) : 1;   // accumulators of BN fp32 columns
  uint32_t acc_cols = BN;                           // TMEM allocations are powers of two
  if (LOCAL)
    while ((int)acc_cols < n_acc * BN) acc_cols *= 2;
  if (warp == 1) {  // TMEM: acc_cols fp32 columns x 128 lanes
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(acc_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Programmatic dependent launch: everything above overlapped the tail of the previous kernel in the stream, and
  // so do the weight tiles of the first ring slots, which no kernel writes.  From the wait on this kernel touches
  // activations, so it needs that kernel's memory; the next kernel in the stream may begin its own prologue now.
  const int w_ahead = min(num_kb, kStages);
  if (warp == 0 && lane == 0) {
    for (int i = 0; i < w_ahead; ++i) {   // the slots start out empty
      const int kb = kb_begin + i;
      const int tap = kb / p.cblocks, cb = kb - tap * p.cblocks;
      mbar_expect_tx(full_bar(i), GATHER ? S::kBBytes : S::kStage);
      tma_load_3d(base + (uint32_t)i * S::kStage + S::kABytes, &tmW, full_bar(i), cb * kTcBK, tap, n0);
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    if (lane == 0) {
      if (RES) {
        mbar_expect_tx(res_bar, S::kIoBytes);
#pragma unroll
        for (int h = 0; h < BN / 64; ++h)
#pragma unroll
          for (int q = 0; q < 4; ++q)
            tma_load_2d(base + S::kIoOff + h * 16384 + q * 4096, &tmR, res_bar, n0 + h * 64, m0 + q * 32);
      }
      int cw = 0, ch = 0, cn = 0;
      if (p.im2col) {
        const int hw = p.Ho * p.Wo;
        cn = m0 / hw;
        const int rem = m0 - cn * hw;
        const int ho = rem / p.Wo;
        cw = (rem - ho * p.Wo) * p.stride - p.pad_w;
        ch = ho * p.stride - p.pad;
      }
      for (int i = 0; i < num_kb; ++i) {
        const int kb = kb_begin + i;
        const int s = i % kStages;
        const uint32_t ph = (uint32_t)(i / kStages) & 1u;
        const int tap = kb / p.cblocks, cb = kb - tap * p.cblocks;
        const uint32_t sa = base + (uint32_t)s * S::kStage, sb = sa + S::kABytes;
        if (i >= w_ahead) {   // earlier slots: armed and their weight tile requested before the dependency wait
          if (!mbar_wait(empty_bar(s), ph ^ 1u, p.err_flag)) break;
          mbar_expect_tx(full_bar(s), GATHER ? S::kBBytes : S::kStage);
          tma_load_3d(sb, &tmW, full_bar(s), cb * kTcBK, tap, n0);
        }
        if (GATHER) {
        } else if (p.im2col) {
          const int r = tap / p.kw;
          tma_load_im2col_4d(sa, &tmA, full_bar(s), cb * kTcBK, cw, ch, cn, (uint16_t)(tap - r * p.kw), (uint16_t)r);
        } else {
          tma_load_2d(sa, &tmA, full_bar(s), cb * kTcBK, m0);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc(BN);
      bool ok = true;
      for (int i = 0; i < num_kb; ++i) {
        const int s = i % kStages;
        const uint32_t ph = (uint32_t)(i / kStages) & 1u;
        ok = mbar_wait(full_bar(s), ph, p.err_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = base + (uint32_t)s * S::kStage, sb = sa + S::kABytes;
        const int r = LOCAL ? i / p.kb_per : 0, ir = i - r * p.kb_per;   // local K range and position inside it
#pragma unroll
        for (int k = 0; k < kTcBK / 16; ++k)
          umma_bf16(tmem_base + (uint32_t)(r * BN), umma_desc(sa + k * 32), umma_desc(sb + k * 32), idesc, (uint32_t)((ir | k) != 0));
        umma_commit(empty_bar(s));  // frees the stage once these MMAs have read it
      }
      if (ok && num_kb > 0) umma_commit(accum_bar);  // accumulator complete: every MMA has also finished reading the ring
    }
  } else {
    const int et = threadIdx.x - 64;  // 0..127
    for (int i = et; i < BN; i += 128) {
      const bool in = n0 + i < p.N;
      s_scale[i] = (p.scale && in) ? p.scale[n0 + i] : 1.f;
      s_bias[i] = (p.bias && in) ? p.bias[n0 + i] : 0.f;
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (GATHER) {
      const int grow = (warp & 3) * 32 + lane;  // tile row = output pixel built by this thread
      const int m = m0 + grow;
      const bool row_in = m < p.M;
      const int hw = p.Ho * p.Wo;
      const int b = m / hw, rem = m - b * hw, ho = rem / p.Wo, wo = rem - ho * p.Wo;
      const int hi0 = ho * p.stride - p.pad;
      const int off0 = (wo * p.stride - p.pad) * p.gCin;  // flat element offset of tap 0 within an input row (may be negative)
      const int row_elems = p.gW * p.gCin;
      const bf16* xb = p.gx + (size_t)(row_in ? b : 0) * p.gH * row_elems;
      if (p.grun == 21 && p.grunp == 24 && p.gkh == 7 && num_kb == 3)        // 7x7 stem on 3 channels
        gather_rows_static<21, 24, 7, 3, STAGES>(p, xb, row_in, hi0, off0, row_elems, gen, S::kStage, grow, bar0);
      else if (p.grun == 9 && p.grunp == 16 && p.gkh == 3 && num_kb == 1)    // 3x3 stem on 3 channels
        gather_rows_static<9, 16, 3, 1, STAGES>(p, xb, row_in, hi0, off0, row_elems, gen, S::kStage, grow, bar0);
      else
        gather_rows_generic<STAGES>(p, xb, row_in, hi0, off0, row_elems, gen, S::kStage, grow, bar0, num_kb);
    }
    // warp-uniform outcomes: tcgen05.ld is a warp-wide instruction
    bool ok = num_kb > 0 ? __all_sync(0xffffffffu, mbar_wait(accum_bar, 0, p.err_flag)) : true;
    if (RES) ok = __all_sync(0xffffffffu, mbar_wait(res_bar, 0, p.err_flag)) && ok;
    tc_fence_after();
    const int q = warp & 3;  // TMEM lane quarter this warp may read = rows [32q, 32q + 32) of the tile
    const int row = q * 32 + lane;
    if (SPLIT) {
      // Reduce-scatter, push side.  CTA z of the cluster owns tile rows [z * rows_per, (z + 1) * rows_per); this thread
      // sends its row of the fp32 partial tile to the owner's shared memory (slot `rank` of the owner's receive
      // buffer, which overlays the drained ring), 16-byte chunks XOR-swizzled with the row so that neither these
      // row-wise stores nor the owner's reads pile onto one bank.  The first cluster barrier guarantees that every
      // peer has finished with its ring before anybody writes into it.
      constexpr int CH = BN / 4;
      const int nsplit = (int)gridDim.z;
      const int rows_per = (kTcBM + nsplit - 1) / nsplit;
      uint32_t rank;
      asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
      const int owner = row / rows_per, rloc = row - owner * rows_per;
      uint32_t dst;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(base + (uint32_t)(((int)rank * rows_per + rloc) * (BN * 4))), "r"(owner));
      asm volatile("barrier.cluster.arrive.release;" ::: "memory");
      bool waited = false;
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        float v[32];
        if (ok && num_kb > 0) {
          tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0.f;
        }
        if (!waited) {
          asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
          waited = true;
        }
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const int c = (c0 >> 2) + g;
          asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (uint32_t)((c ^ (rloc & (CH - 1))) << 4)), "f"(v[4 * g]),
                       "f"(v[4 * g + 1]), "f"(v[4 * g + 2]), "f"(v[4 * g + 3])
                       : "memory");
        }
      }
    } else if (ok) {
      uint8_t* io = gen + S::kIoOff;
      const uint32_t io_s = base + S::kIoOff;
      bool stored = false;
#pragma unroll 1
      for (int h = 0; h < BN / 64; ++h) {
        if (n0 + h * 64 >= p.N) break;
        // this thread's 128-byte line of the 64-column half; its eight 16-byte chunks are XOR-swizzled with the
        // row index so that the TMA unit (128-byte swizzle) finds row-major data
        uint8_t* line = io + h * 16384 + row * 128;
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          const int c0 = h * 64 + sub * 32;
          float v[32];
          tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
          if constexpr (LOCAL) {   // local K ranges: 0 + range 0 + range 1 + ... as the cluster reduction adds them
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = 0.f + v[e];
            for (int r = 1; r < n_acc; ++r) {
              float t[32];
              tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(r * BN + c0), t);
#pragma unroll
              for (int e = 0; e < 32; ++e) v[e] += t[e];
            }
          }
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            if (n0 + c0 + g * 8 >= p.N) break;   // columns past Cout: nothing to compute, the store clips them
            uint4* chunk = reinterpret_cast<uint4*>(line + (((sub * 4 + g) ^ (lane & 7)) << 4));
            *chunk = epilogue8_act<RES>(p.act, v + g * 8, s_scale + c0 + g * 8, s_bias + c0 + g * 8, RES ? *chunk : make_uint4(0u, 0u, 0u, 0u));
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the TMA unit
        __syncwarp();
        if (lane == 0 && m0 + q * 32 < p.M) {  // rows past M and columns past N are clipped by the TMA unit
          tma_store_2d(&tmO, io_s + h * 16384 + q * 4096, n0 + h * 64, m0 + q * 32);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          stored = true;
        }
      }
      if (stored) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // shared memory is read before the CTA retires
    }
  }
  if (SPLIT) {
    // Every thread of every CTA of the cluster passes both barriers, whatever happened above: the first one before
    // any remote store (epilogue threads took it inside their push loop), the second once all partials have landed.
    if (warp < 2) asm volatile("barrier.cluster.arrive.release;\n barrier.cluster.wait.acquire;" ::: "memory");
    asm volatile("barrier.cluster.arrive.release;\n barrier.cluster.wait.acquire;" ::: "memory");
    if (warp >= 2) {
      // Pull side, all local: this CTA adds the nsplit partials of its rows in ascending range order (the grouping
      // of the sum is fixed by the layer), applies the epilogue and stores.
      constexpr int CH = BN / 4, G = BN / 8;     // 16-byte fp32 chunks and 8-column groups per row
      const int et = threadIdx.x - 64;
      const int nsplit = (int)gridDim.z;
      const int rows_per = (kTcBM + nsplit - 1) / nsplit;
      uint32_t rank;
      asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
      const float* part = reinterpret_cast<const float*>(gen);
      for (int item = et; item < rows_per * G; item += 128) {
        const int r = item / G, g = item - r * G;
        const int trow = (int)rank * rows_per + r;
        if (trow >= kTcBM) break;
        const int m = m0 + trow, n = n0 + g * 8;
        const int o0 = ((2 * g) ^ (r & (CH - 1))) << 2, o1 = ((2 * g + 1) ^ (r & (CH - 1))) << 2;
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = 0.f;
#pragma unroll 4
        for (int z = 0; z < nsplit; ++z) {
          const float* pr = part + (size_t)(z * rows_per + r) * BN;
          const float4 x0 = *reinterpret_cast<const float4*>(pr + o0);
          const float4 x1 = *reinterpret_cast<const float4*>(pr + o1);
          v[0] += x0.x; v[1] += x0.y; v[2] += x0.z; v[3] += x0.w;
          v[4] += x1.x; v[5] += x1.y; v[6] += x1.z; v[7] += x1.w;
        }
        if (m < p.M && n < p.N) {
          scale_bias<8>(v, s_scale + g * 8, s_bias + g * 8);
          if (p.residual) {
            Vec16<bf16> rr;
            rr.load(p.residual + (size_t)m * p.N + n);
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] += rr.v[e];
          }
          Vec16<bf16> o;
#pragma unroll
          for (int e = 0; e < 8; ++e) o.v[e] = apply_act(v[e], p.act);
          o.store(p.out + (size_t)m * p.N + n);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(acc_cols) : "memory");
  }
}

// ----------------------------------------------------------------------------- persistent variant
//
// For grids of several waves (large B*Ho*Wo): one CTA per SM walks output tiles t = blockIdx.x, + gridDim.x, ...
// (tile t -> M tile t / n_tiles, N tile t % n_tiles, so CTAs running side by side share A rows in L2).  The operand
// ring keeps streaming across tile boundaries and the accumulator is double-buffered in TMEM: while the epilogue warps
// drain accumulator j & 1 of tile j, the MMA warp already fills the other one with tile j + 1, and the producer is
// further ahead still.  A tile then costs max(load, MMA, epilogue) instead of their sum, and the per-CTA prologue
// (barriers, TMEM allocation, descriptor fetch) is paid once per SM instead of once per tile.
// Staged outputs leave through TMA stores; a staging tile is rewritten only after the warp has seen its previous store
// finish reading it.  Residual tiles are prefetched by the producer into two buffers of their own, which return to it
// (res_free) as soon as all four epilogue warps have read them.
template <int BN, bool RES, bool PROJ = false>
struct TcPersistSmem {
  // without a residual: a longer ring and two output staging tiles; with one: two residual tiles the producer
  // prefetches (free again as soon as the epilogue has read them) and a single staging tile
  static constexpr int kEpiWarps = BN == 128 ? 8 : 4;   // at BN = 128 two warps share a TMEM lane quarter, one per 64-column half
  static constexpr int kThreads = 64 + 32 * kEpiWarps;
  static constexpr int kStages = RES ? (BN == 128 ? 3 : 5) : (BN == 128 ? 4 : 7);
  static constexpr int kABytes = kTcBM * kTcBK * 2;
  static constexpr int kBBytes = BN * kTcBK * 2;
  static constexpr int kStage = kABytes + kBBytes;
  static constexpr int kTiles = kStages * kStage;
  static constexpr int kIoBytes = kTcBM * BN * 2;
  static constexpr int kROff = kTiles;
  static constexpr int kOOff = kTiles + (RES ? 2 * kIoBytes : 0);
  static constexpr int kAfter = kOOff + (RES ? 1 : 2) * kIoBytes;
  static constexpr int kSb = (PROJ ? 4 : 2) * BN;   // floats per epilogue warp: scale | bias (| scale2 | bias2)
  static constexpr int kBytes = kAfter + kEpiWarps * kSb * 4 + 256 + 1024;  // + one scale/bias copy per epilogue warp, barriers, slack
  static_assert(!(RES && PROJ), "the projection replaces the residual tile");
  static_assert(kBytes <= 227 * 1024, "exceeds the shared memory of an SM");
};

// PROJ: the residual operand is computed here instead of read: after the K blocks of the layer the ring carries the K
// blocks of a 1x1 projection (tmA2: its input, tile or im2col map; tmW2: its weights) into a second accumulator, and
// the epilogue rounds scale2 * acc2 + bias2 (act2) to bf16 - the value the projection layer would have stored - before
// it adds it: the same bits as the two layers run apart, without the projection's output ever reaching global memory.
template <int BN, bool RES, bool PROJ = false>
__global__ void __launch_bounds__(TcPersistSmem<BN, RES, PROJ>::kThreads, 1)
conv_igemm_tcgen05_persistent_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                                     const __grid_constant__ CUtensorMap tmR, const __grid_constant__ CUtensorMap tmO,
                                     const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmW2, TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  using S = TcPersistSmem<BN, RES, PROJ>;
  constexpr int kAccs = PROJ ? 2 : 1;   // accumulators per tile
  constexpr int kStages = S::kStages;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  float* s_sb = reinterpret_cast<float*>(gen + S::kAfter);  // [epilogue warps][scale BN | bias BN]
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen + S::kAfter + S::kEpiWarps * S::kSb * 4);
  const uint32_t bar0 = base + S::kAfter + S::kEpiWarps * S::kSb * 4;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * kStages + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * kStages + 2 + b); };
  auto res_full = [&](int b) { return bar0 + 8u * (2 * kStages + 4 + b); };
  auto res_free = [&](int b) { return bar0 + 8u * (2 * kStages + 6 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = p.taps * p.cblocks;
  const int num_kb2 = PROJ ? p.cblocks2 : 0;   // K blocks of the projection (one tap)
  const int n_tiles = (p.N + BN - 1) / BN;
  const int m_tiles = (p.M + kTcBM - 1) / kTcBM;
  const int total = n_tiles * m_tiles;
  const int my_tiles = (int)blockIdx.x < total ? (total - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full(b), 1);
      mbar_init(acc_empty(b), S::kEpiWarps);   // lane 0 of each epilogue warp
      mbar_init(res_full(b), 1);
      mbar_init(res_free(b), S::kEpiWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmO) : "memory");
    if (RES) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmR) : "memory");
    if (PROJ) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA2) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW2) : "memory");
    }
  }
  if (warp == 1) {  // two tiles in flight, each with kAccs accumulators of BN fp32 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(2 * kAccs * BN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // weight tiles of the first ring slots (first tile of this CTA) are requested before the dependency wait: no
  // kernel writes them
  const int w_ahead = my_tiles > 0 ? min(num_kb, kStages) : 0;
  if (warp == 0 && lane == 0) {
    const int n0 = ((p.rev ? total - 1 - (int)blockIdx.x : (int)blockIdx.x) % n_tiles) * BN;
    for (int i = 0; i < w_ahead; ++i) {
      const int tap = i / p.cblocks, cb = i - tap * p.cblocks;
      mbar_expect_tx(full_bar(i), S::kStage);
      tma_load_3d(base + (uint32_t)i * S::kStage + S::kABytes, &tmW, full_bar(i), cb * kTcBK, tap, n0);
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    if (lane == 0) {
      int g = 0;  // K blocks issued so far, across tiles: the ring never drains at a tile boundary
      bool ok = true;
      for (int j = 0; j < my_tiles && ok; ++j) {
        const int tf = (int)blockIdx.x + j * (int)gridDim.x, t = p.rev ? total - 1 - tf : tf;
        const int m0 = (t / n_tiles) * kTcBM, n0 = (t % n_tiles) * BN;
        const int b = j & 1;
        if (RES) {
          if (j >= 2) ok = mbar_wait(res_free(b), (uint32_t)((j >> 1) - 1) & 1u, p.err_flag);
          if (!ok) break;
          mbar_expect_tx(res_full(b), S::kIoBytes);
#pragma unroll
          for (int h = 0; h < BN / 64; ++h)
#pragma unroll
            for (int q = 0; q < 4; ++q)
              tma_load_2d(base + S::kROff + b * S::kIoBytes + h * 16384 + q * 4096, &tmR, res_full(b), n0 + h * 64, m0 + q * 32);
        }
        int cw = 0, ch = 0, cn = 0;
        if (p.im2col) {
          const int hw = p.Ho * p.Wo;
          cn = m0 / hw;
          const int rem = m0 - cn * hw;
          const int ho = rem / p.Wo;
          cw = (rem - ho * p.Wo) * p.stride - p.pad_w;
          ch = ho * p.stride - p.pad;
        }
        for (int kb = 0; kb < num_kb; ++kb, ++g) {
          const int s = g % kStages;
          const uint32_t ph = (uint32_t)(g / kStages) & 1u;
          const int tap = kb / p.cblocks, cb = kb - tap * p.cblocks;
          const uint32_t sa = base + (uint32_t)s * S::kStage, sb = sa + S::kABytes;
          if (g >= w_ahead) {   // earlier slots were armed before the dependency wait
            ok = mbar_wait(empty_bar(s), ph ^ 1u, p.err_flag);
            if (!ok) break;
            mbar_expect_tx(full_bar(s), S::kStage);
            tma_load_3d(sb, &tmW, full_bar(s), cb * kTcBK, tap, n0);
          }
          if (p.im2col) {
            const int r = tap / p.kw;
            tma_load_im2col_4d(sa, &tmA, full_bar(s), cb * kTcBK, cw, ch, cn, (uint16_t)(tap - r * p.kw), (uint16_t)r);
          } else {
            tma_load_2d(sa, &tmA, full_bar(s), cb * kTcBK, m0);
          }
        }
        if (PROJ && ok) {   // the projection's K blocks follow in the same ring
          int cw2 = 0, ch2 = 0, cn2 = 0;
          if (p.im2col2) {
            const int hw = p.Ho * p.Wo;
            cn2 = m0 / hw;
            const int rem = m0 - cn2 * hw;
            const int ho = rem / p.Wo;
            cw2 = (rem - ho * p.Wo) * p.stride2;
            ch2 = ho * p.stride2;
          }
          for (int kb = 0; kb < num_kb2; ++kb, ++g) {
            const int s = g % kStages;
            const uint32_t ph = (uint32_t)(g / kStages) & 1u;
            const uint32_t sa = base + (uint32_t)s * S::kStage, sb = sa + S::kABytes;
            ok = mbar_wait(empty_bar(s), ph ^ 1u, p.err_flag);   // g >= num_kb >= w_ahead: never a pre-armed slot
            if (!ok) break;
            mbar_expect_tx(full_bar(s), S::kStage);
            tma_load_3d(sb, &tmW2, full_bar(s), kb * kTcBK, 0, n0);
            if (p.im2col2)
              tma_load_im2col_4d(sa, &tmA2, full_bar(s), kb * kTcBK, cw2, ch2, cn2, (uint16_t)0, (uint16_t)0);
            else
              tma_load_2d(sa, &tmA2, full_bar(s), kb * kTcBK, m0);
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc(BN);
      int g = 0;
      bool ok = true;
      for (int j = 0; j < my_tiles && ok; ++j) {
        const int b = j & 1;
        if (j >= 2) {  // the epilogue must have drained this accumulator (tile j - 2)
          ok = mbar_wait(acc_empty(b), (uint32_t)((j >> 1) - 1) & 1u, p.err_flag);
          if (!ok) break;
          tc_fence_after();
        }
        const uint32_t acc = tmem_base + (uint32_t)(b * kAccs * BN);
        for (int kb = 0; kb < num_kb; ++kb, ++g) {
          const int s = g % kStages;
          const uint32_t ph = (uint32_t)(g / kStages) & 1u;
          ok = mbar_wait(full_bar(s), ph, p.err_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = base + (uint32_t)s * S::kStage, sb = sa + S::kABytes;
#pragma unroll
          for (int k = 0; k < kTcBK / 16; ++k)
            umma_bf16(acc, umma_desc(sa + k * 32), umma_desc(sb + k * 32), idesc, (uint32_t)((kb | k) != 0));
          umma_commit(empty_bar(s));
        }
        if (PROJ) {
          for (int kb = 0; kb < num_kb2 && ok; ++kb, ++g) {
            const int s = g % kStages;
            const uint32_t ph = (uint32_t)(g / kStages) & 1u;
            ok = mbar_wait(full_bar(s), ph, p.err_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t sa = base + (uint32_t)s * S::kStage, sb = sa + S::kABytes;
#pragma unroll
            for (int k = 0; k < kTcBK / 16; ++k)
              umma_bf16(acc + (uint32_t)BN, umma_desc(sa + k * 32), umma_desc(sb + k * 32), idesc, (uint32_t)((kb | k) != 0));
            umma_commit(empty_bar(s));
          }
        }
        if (ok) umma_commit(acc_full(b));
      }
    }
  } else {
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const int ew = warp - 2;
    const int h0 = BN == 128 ? (ew >> 2) : 0, h1 = h0 + 1;  // the 64-column half (halves) this warp owns
    float* sc = s_sb + ew * S::kSb;  // this warp's own copy: no barrier across warps inside the tile loop
    bool ok = true;
    int sc_n0 = -1;
    bool pending = false;  // lane 0: a bulk store group of this warp may still be reading shared memory
    for (int j = 0; j < my_tiles; ++j) {
      const int tf = (int)blockIdx.x + j * (int)gridDim.x, t = p.rev ? total - 1 - tf : tf;
      const int m0 = (t / n_tiles) * kTcBM, n0 = (t % n_tiles) * BN;
      const int b = j & 1;
      if (n0 != sc_n0) {  // consecutive tiles of a CTA usually share the N tile: reload only on change
        __syncwarp();
        for (int i = lane; i < BN; i += 32) {
          const bool in = n0 + i < p.N;
          sc[i] = (p.scale && in) ? p.scale[n0 + i] : 1.f;
          sc[BN + i] = (p.bias && in) ? p.bias[n0 + i] : 0.f;
          if (PROJ) {
            sc[2 * BN + i] = (p.scale2 && in) ? p.scale2[n0 + i] : 1.f;
            sc[3 * BN + i] = (p.bias2 && in) ? p.bias2[n0 + i] : 0.f;
          }
        }
        sc_n0 = n0;
      }
      __syncwarp();  // scale/bias of this tile visible to the warp
      ok = __all_sync(0xffffffffu, mbar_wait(acc_full(b), (uint32_t)(j >> 1) & 1u, p.err_flag));
      if (RES && ok) ok = __all_sync(0xffffffffu, mbar_wait(res_full(b), (uint32_t)(j >> 1) & 1u, p.err_flag));
      if (!ok) break;
      tc_fence_after();
      if (!RES) {  // two staging tiles: all but this warp's latest store (tile j - 1, the other tile) must have been read
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        __syncwarp();
      }
      const int ob = RES ? 0 : b;  // output staging tile of this tile
      uint8_t* io = gen + S::kOOff + ob * S::kIoBytes;
      const uint32_t io_s = base + S::kOOff + ob * S::kIoBytes;
      const uint8_t* rin = gen + S::kROff + b * S::kIoBytes;
      const uint32_t acc = tmem_base + (uint32_t)(b * kAccs * BN) + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
      for (int h = h0; h < h1; ++h) {
        uint4 proj[8];   // PROJ: the projection's 64 values of this row, rounded to bf16 as the layer itself would store them
        if (PROJ) {
          float pa[32], pb[32];
          tmem_ld32_issue(acc + (uint32_t)(BN + h * 64), pa);
          tmem_ld32_issue(acc + (uint32_t)(BN + h * 64 + 32), pb);
          tmem_ld_wait(pa, pb);
#pragma unroll
          for (int sub = 0; sub < 2; ++sub) {
            const int c0 = h * 64 + sub * 32;
            const float* v = sub ? pb : pa;
#pragma unroll
            for (int gq = 0; gq < 4; ++gq)
              proj[sub * 4 + gq] = epilogue8_act<false>(p.act2, v + gq * 8, sc + 2 * BN + c0 + gq * 8, sc + 3 * BN + c0 + gq * 8, make_uint4(0u, 0u, 0u, 0u));
          }
        }
        uint4 ov[8];           // this row's 64 outputs of the half (kept for the pooling partials)
#pragma unroll
        for (int i = 0; i < 8; ++i) ov[i] = make_uint4(0u, 0u, 0u, 0u);
        float va[32], vb[32];  // both 32-column loads of the half in flight before one wait
        tmem_ld32_issue(acc + (uint32_t)(h * 64), va);
        tmem_ld32_issue(acc + (uint32_t)(h * 64 + 32), vb);
        tmem_ld_wait(va, vb);
        if (h == h1 - 1) {  // this warp's share of the accumulator is in registers: the MMA warp may refill it
          tc_fence_before();
          __syncwarp();
          if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acc_empty(b)) : "memory");
        }
        if (RES && h == h0) {  // single staging tile: this warp's previous store must have finished reading it
          if (lane == 0 && pending) {
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            pending = false;
          }
          __syncwarp();
        }
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          const int c0 = h * 64 + sub * 32;
          const float* v = sub ? vb : va;
#pragma unroll
          for (int gq = 0; gq < 4; ++gq) {
            if (n0 + c0 + gq * 8 >= p.N) break;   // columns past Cout: nothing to compute, the store clips them
            const int off = h * 16384 + row * 128 + (((sub * 4 + gq) ^ (lane & 7)) << 4);
            const uint4 r = RES ? *reinterpret_cast<const uint4*>(rin + off) : PROJ ? proj[sub * 4 + gq] : make_uint4(0u, 0u, 0u, 0u);
            ov[sub * 4 + gq] = epilogue8_act<RES || PROJ>(p.act, v + gq * 8, sc + c0 + gq * 8, sc + BN + c0 + gq * 8, r);
            *reinterpret_cast<uint4*>(io + off) = ov[sub * 4 + gq];
          }
        }
        if (p.gap_g) {   // rows past M hold zero-filled operands, but their bias and residual garbage must not be summed: whole blocks are skipped
          const int r0 = m0 + q * 32;
          if (p.gap_g == 32)
            gap_partial_store<32>(ov, lane, p.gap_part + (size_t)(r0 / 32) * p.N + n0 + h * 64, p.N - n0 - h * 64, 0, r0 < p.M);
          else
            gap_partial_store<16>(ov, lane, p.gap_part + (size_t)(r0 / 16) * p.N + n0 + h * 64, p.N - n0 - h * 64, (size_t)p.N,
                                  r0 + (lane >> 4) * 16 < p.M);
        }
      }
      if (RES) {  // the residual tile is consumed: the producer may prefetch the one of tile j + 2 into it
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(res_free(b)) : "memory");
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        if (m0 + q * 32 < p.M) {
          for (int h = h0; h < h1; ++h)
            if (n0 + h * 64 < p.N) tma_store_2d(&tmO, io_s + h * 16384 + q * 4096, n0 + h * 64, m0 + q * 32);
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");  // possibly empty: keeps the bookkeeping uniform
        pending = true;
      }
    }
    if (lane == 0 && pending) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * kAccs * BN) : "memory");
  }
}

// Pixel grouping for narrow 1x1 layers.  A pixel row of Cin <= 32 channels is 16-64 bytes, and a TMA box over such
// rows moves one short row per request (a 16-channel layer loads at a quarter of the rate of a 64-channel one).  g
// consecutive pixels are one contiguous row of g * Cin channels, so the layer is run as a 1x1 layer over M / g rows
// with Cin' = g * Cin and Cout' = g * Cout and the block-diagonal weight matrix below: row (j, n) holds w[n][:] in
// columns [j * Cin, (j + 1) * Cin) and zeros elsewhere.  Output row i, column j * Cout + n is channel n of pixel
// g * i + j, which is exactly where the dense [M][Cout] output keeps it.  The zero blocks add g - 1 idle MMA passes
// on layers that do not come near the tensor pipe's rate; each output is still the same sum of Cin products.
__global__ void pack_grouped_weights_kernel(const bf16* __restrict__ w, bf16* __restrict__ out, int cout, int cin, int g) {
  const long total = (long)g * cout * g * cin;
  for (long idx = (long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
    const int col = (int)(idx % ((long)g * cin));
    const int row = (int)(idx / ((long)g * cin));
    const int j = row / cout, n = row - j * cout, jc = col / cin, c = col - jc * cin;
    out[idx] = j == jc ? w[(long)n * cin + c] : __float2bfloat16_rn(0.f);
  }
}
__global__ void replicate_kernel(const float* __restrict__ src, float* __restrict__ dst, int n, int g) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n * g; i += gridDim.x * blockDim.x) dst[i] = src[i % n];
}
// Pixels per row for a 1x1 / stride 1 / pad 0 layer on hw pixels per sample: the largest g with g * Cin <= 64 that
// divides hw (so no row straddles two samples); 1 = leave the layer as it is.
inline int pixel_group(const ee_layer_desc_t& d, int hw) {
  if (!(d.kh == 1 && d.kw == 1 && d.stride == 1 && d.pad == 0 && d.pad_w == 0) || d.cin > 32) return 1;
  int g = kTcBK / d.cin;
  while (g > 1 && hw % g != 0) --g;
  return g;
}

// Gather mode: weight rows [Cout][kh][kw*Cin] copied into rows [Cout][kh][runp] padded to Kp columns, zeros elsewhere.
__global__ void pack_weights_kernel(const bf16* __restrict__ w, bf16* __restrict__ out, int rows, int kh, int run, int runp, int Kp) {
  const long total = (long)rows * Kp;
  for (long idx = (long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
    const int k = (int)(idx % Kp);
    const long co = idx / Kp;
    const int r = k / runp, j = k - r * runp;
    out[idx] = (r < kh && j < run) ? w[(co * kh + r) * run + j] : __float2bfloat16_rn(0.f);
  }
}

// ----------------------------------------------------------------------------- host side

typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*PFN_encodeIm2col)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                     const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*, CUtensorMapInterleave,
                                     CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcContext {
  PFN_encodeTiled encode_tiled = nullptr;
  PFN_encodeIm2col encode_im2col = nullptr;
  int sm_count = 148;
};

struct TcLayer {
  int cin = 0, cout = 0, kh = 1, kw = 1, stride = 1, pad = 0, pad_w = 0, act = 0;
  int in_h = 0, in_w = 0, out_h = 0, out_w = 0, max_batch = 0;
  int bn = 128;
  bool im2col = false;
  int splits = 1, kb_per = 0;    // split-K ranges of this layer (fixed per layer, independent of the batch)
  bool rev = false;              // walk the output tiles from the last one down (see TcParams::rev)
  // gather mode: geometry of the real convolution (cin/kh/... above then describe the packed 1x1 GEMM view)
  bool gather = false;
  bool stem7 = false;   // the 7x7/2 stem kernel of conv_stem.cuh takes this layer
  bool halo = false;    // the 3x3 halo-block kernel of conv_halo.cuh takes this layer
  int g_h = 0, g_w = 0, g_cin = 0, g_kh = 0, g_kw = 0, g_stride = 1, g_pad = 0, g_runp = 0;
  CUtensorMap tm_w;
  CUtensorMap tm_w_half[2];   // the same weights with boxes of 128 and 64 filters: one CTA's half of a 256- or 128-wide pair tile
  struct Cached {
    const void* ptr;
    int batch;
    int kind;  // 0: operand A, 1: residual / output matrix, 2: stem input rows, 3: stem output rows, 4: halo blocks
    CUtensorMap tm;
  };
  mutable std::vector<Cached> a_maps;  // tensor maps of caller buffers by (pointer, batch, kind)
  mutable size_t next_evict = 0;
};

inline ee_status_t tc_context_init(TcContext& c) {
  cudaDriverEntryPointQueryResult q;
  void* f = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess || !f) return EE_ERR_CUDA;
  c.encode_tiled = (PFN_encodeTiled)f;
  f = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f, cudaEnableDefault, &q) != cudaSuccess || !f) return EE_ERR_CUDA;
  c.encode_im2col = (PFN_encodeIm2col)f;
  {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
      c.sm_count = sms;
  }
  cudaError_t e = cudaSuccess;
  auto set = [&](auto kernel, int bytes) {
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  };
  set(conv_igemm_tcgen05_kernel<64, 3, false, false, true>, TcSmem<64, 3, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<128, 3, false, false, true>, TcSmem<128, 3, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<64, 3, false, false, false>, TcSmem<64, 3, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<64, 6, false, false, false>, TcSmem<64, 6, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<64, 2, true, false, false>, TcSmem<64, 2, true>::kBytes);
  set(conv_igemm_tcgen05_kernel<64, 5, true, false, false>, TcSmem<64, 5, true>::kBytes);
  set(conv_igemm_tcgen05_kernel<64, 6, false, true, false>, TcSmem<64, 6, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<64, 3, false, true, false>, TcSmem<64, 3, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<128, 3, false, false, false>, TcSmem<128, 3, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<128, 6, false, false, false>, TcSmem<128, 6, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<128, 2, true, false, false>, TcSmem<128, 2, true>::kBytes);
  set(conv_igemm_tcgen05_kernel<128, 5, true, false, false>, TcSmem<128, 5, true>::kBytes);
  set(conv_igemm_tcgen05_kernel<128, 6, false, true, false>, TcSmem<128, 6, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<128, 3, false, true, false>, TcSmem<128, 3, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<64, 3, false, false, false, true>, TcSmem<64, 3, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<64, 6, false, false, false, true>, TcSmem<64, 6, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<64, 2, true, false, false, true>, TcSmem<64, 2, true>::kBytes);
  set(conv_igemm_tcgen05_kernel<64, 5, true, false, false, true>, TcSmem<64, 5, true>::kBytes);
  set(conv_igemm_tcgen05_kernel<128, 3, false, false, false, true>, TcSmem<128, 3, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<128, 6, false, false, false, true>, TcSmem<128, 6, false>::kBytes);
  set(conv_igemm_tcgen05_kernel<128, 2, true, false, false, true>, TcSmem<128, 2, true>::kBytes);
  set(conv_igemm_tcgen05_kernel<128, 5, true, false, false, true>, TcSmem<128, 5, true>::kBytes);
  set(conv_igemm_tcgen05_persistent_kernel<64, false>, TcPersistSmem<64, false>::kBytes);
  set(conv_igemm_tcgen05_persistent_kernel<64, true>, TcPersistSmem<64, true>::kBytes);
  set(conv_igemm_tcgen05_persistent_kernel<128, false>, TcPersistSmem<128, false>::kBytes);
  set(conv_igemm_tcgen05_persistent_kernel<128, true>, TcPersistSmem<128, true>::kBytes);
  set(conv_igemm_tcgen05_persistent_kernel<64, false, true>, TcPersistSmem<64, false, true>::kBytes);
  set(conv_igemm_tcgen05_persistent_kernel<128, false, true>, TcPersistSmem<128, false, true>::kBytes);
  if (e != cudaSuccess) return EE_ERR_CUDA;
  return EE_OK;
}

// Layers this path covers: dense convolutions whose pixel rows are whole 16-byte units (Cin and Cout multiples
// of 8).  Channel counts need not fill the 64-wide K block or the N tile: the TMA unit zero-fills what lies past
// the tensor, and the epilogue masks columns past Cout.
inline bool tc_supported(const ee_layer_desc_t& d, int in_h, int in_w) {
  (void)in_h;
  (void)in_w;
  return d.op == EE_OP_CONV && d.cin % 8 == 0 && d.cout % 8 == 0 && d.kh <= 7 && d.kw <= 7 && d.stride <= 8 &&
         d.pad < d.kh && d.pad_w < d.kw;   // filters need not be square: the im2col map takes one corner pair per axis
}

inline ee_status_t tc_plan_layer(TcContext& c, const ee_layer_desc_t& d, int in_h, int in_w, int out_h, int out_w, int max_batch,
                                 const void* w_dev, TcLayer* L) {
  L->cin = d.cin, L->cout = d.cout, L->kh = d.kh, L->kw = d.kw, L->stride = d.stride, L->pad = d.pad, L->pad_w = d.pad_w, L->act = d.act;
  L->in_h = in_h, L->in_w = in_w, L->out_h = out_h, L->out_w = out_w, L->max_batch = max_batch;
  L->bn = d.cout > 64 ? 128 : 64;
  L->im2col = !(d.kh == 1 && d.kw == 1 && d.stride == 1 && d.pad == 0 && d.pad_w == 0);
  // Split-K: a lone CTA cannot pull operands faster than its SM's L2 port (about 126 GB/s: a 32 KB K block of a
  // 128x128 tile takes 0.26 us in tile mode and 0.36 us in im2col mode, against 0.13 us of MMA time), so a layer
  // whose grid leaves SMs idle spreads the K range of a tile over a cluster of 2..4 CTAs.  A split costs about
  // 4.5 us (cluster launch, two cluster barriers, the reduce-scatter), larger clusters gain nothing measurable, and
  // grids of more than two CTAs per SM lose to the unsplit kernel, hence the bounds.  The number of ranges is chosen
  // once per layer by this cost model summed over the batch sizes the model will see (max_batch, 3/4, 1/2 and 1/4
  // of it: the batch shrinks at every exit), the analogue of the per-layer objective sum_b w_b T(b) of the paper's
  // design-space exploration (Eq. 2).  It depends on the layer and on max_batch, never on the batch actually run,
  // so a sample's sums are grouped the same way in every call.
  {
    const int num_kb = d.kh * d.kw * cdiv(d.cin, kTcBK);
    const int n_tiles = cdiv(d.cout, L->bn);
    const double t_block = (L->im2col ? 0.36 : 0.26) * (16384.0 + L->bn * 128.0) / 32768.0;   // us per K block per SM
    const long tiles_max = (long)cdiv((long)max_batch * out_h * out_w, kTcBM) * n_tiles;
    double best = 0;
    L->splits = 1;
    L->kb_per = num_kb;
    for (int sp = 1; sp <= 4; ++sp) {
      const int per = cdiv(num_kb, sp);
      if (sp > 1 && (per < 4 || (sp - 1) * per >= num_kb || tiles_max * sp > 2 * c.sm_count + 4)) continue;
      double cost = 0;
      for (int f = 4; f >= 1; --f) {
        const int b = std::max(1, (max_batch * f + 3) / 4);
        const long tiles = (long)cdiv((long)b * out_h * out_w, kTcBM) * n_tiles;
        const long share = cdiv(tiles * sp, c.sm_count);   // CTAs that share the L2 port of the busiest SM
        cost += 2.4 + (sp > 1 ? 4.5 : 0.0) + (double)share * per * t_block + 0.8 * cdiv(tiles, c.sm_count);
      }
      if (sp == 1) {
        best = cost;
      } else if (cost < best) {
        best = cost;
        L->splits = sp;
        L->kb_per = per;
      }
    }
  }
  // weights [Cout][taps][Cin] as a 3-D tensor, box = 64 channels x 1 tap x BN filters
  const cuuint64_t dims[3] = {(cuuint64_t)d.cin, (cuuint64_t)(d.kh * d.kw), (cuuint64_t)d.cout};
  const cuuint64_t strides[2] = {(cuuint64_t)d.cin * 2, (cuuint64_t)d.cin * d.kh * d.kw * 2};
  const cuuint32_t box[3] = {kTcBK, 1, (cuuint32_t)L->bn};
  const cuuint32_t es[3] = {1, 1, 1};
  CUresult r = c.encode_tiled(&L->tm_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(w_dev), dims, strides, box, es,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  for (int i = 0; i < 2 && r == CUDA_SUCCESS; ++i) {
    const cuuint32_t hbox[3] = {kTcBK, 1, (cuuint32_t)(i == 0 ? 128 : 64)};
    r = c.encode_tiled(&L->tm_w_half[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(w_dev), dims, strides, hbox, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  return r == CUDA_SUCCESS ? EE_OK : EE_ERR_CUDA;
}

// Tensor map of a caller buffer, cached by (pointer, batch, kind).  kind 0: operand A of the layer; kind 1: a
// [batch*Ho*Wo][Cout] matrix (residual or output) with a 64 x 32 box.  A map covers exactly `batch` samples: rows
// past them are out of bounds for the TMA unit (reads give zero, writes are dropped), so no byte beyond the
// caller's [batch] samples is ever touched.
inline ee_status_t tc_buffer_map(const TcContext& c, const TcLayer& L, const void* ptr, int batch, int kind, const CUtensorMap** out) {
  for (auto& e : L.a_maps)
    if (e.ptr == ptr && e.batch == batch && e.kind == kind) {
      *out = &e.tm;
      return EE_OK;
    }
  TcLayer::Cached e;
  e.ptr = ptr;
  e.batch = batch;
  e.kind = kind;
  CUresult r;
  if (kind == 4) {
    // NHWC as (C, W, H, B); a box is the R + 2 rows of W + 2 pixels one output tile of R rows touches (zero fill outside)
    const int wp = L.in_w + 2, rows = kTcBM / wp + 2;
    const cuuint64_t dims[4] = {(cuuint64_t)L.cin, (cuuint64_t)L.in_w, (cuuint64_t)L.in_h, (cuuint64_t)batch};
    const cuuint64_t strides[3] = {(cuuint64_t)L.cin * 2, (cuuint64_t)L.cin * 2 * L.in_w, (cuuint64_t)L.cin * 2 * L.in_w * L.in_h};
    const cuuint32_t box[4] = {kTcBK, (cuuint32_t)wp, (cuuint32_t)rows, 1};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    r = c.encode_tiled(&e.tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else if (kind == 2) {
    // stem input as (W*Cin, H, B): 256 elements of 7 consecutive image rows per load, zero fill outside
    const cuuint64_t dims[3] = {(cuuint64_t)L.g_w * L.g_cin, (cuuint64_t)L.g_h, (cuuint64_t)batch};
    const cuuint64_t strides[2] = {(cuuint64_t)L.g_w * L.g_cin * 2, (cuuint64_t)L.g_w * L.g_cin * 2 * L.g_h};
    const cuuint32_t box[3] = {256, 7, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    r = c.encode_tiled(&e.tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else if (kind == 3) {
    // stem output as (Cout, Wo, B*Ho): a tile is one output row, pixels past Wo are clipped
    const cuuint64_t dims[3] = {(cuuint64_t)L.cout, (cuuint64_t)L.out_w, (cuuint64_t)batch * L.out_h};
    const cuuint64_t strides[2] = {(cuuint64_t)L.cout * 2, (cuuint64_t)L.cout * 2 * L.out_w};
    const cuuint32_t box[3] = {64, 32, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    r = c.encode_tiled(&e.tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else if (kind == 5) {
    // stem output behind its fused 3x3 stride-2 pad-1 max-pool, as (Cout, Wp, B*Hp): a store is up to 32 pixels of a pooled row
    const int hp = (L.out_h - 1) / 2 + 1, wp = (L.out_w - 1) / 2 + 1;
    const cuuint64_t dims[3] = {(cuuint64_t)L.cout, (cuuint64_t)wp, (cuuint64_t)batch * hp};
    const cuuint64_t strides[2] = {(cuuint64_t)L.cout * 2, (cuuint64_t)L.cout * 2 * wp};
    const cuuint32_t box[3] = {64, 32, 1};
    const cuuint32_t es[3] = {1, 1, 1};
    r = c.encode_tiled(&e.tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else if (kind == 1) {
    const cuuint64_t dims[2] = {(cuuint64_t)L.cout, (cuuint64_t)batch * L.out_h * L.out_w};
    const cuuint64_t strides[1] = {(cuuint64_t)L.cout * 2};
    const cuuint32_t box[2] = {64, 32};
    const cuuint32_t es[2] = {1, 1};
    r = c.encode_tiled(&e.tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else if (!L.im2col) {
    const cuuint64_t dims[2] = {(cuuint64_t)L.cin, (cuuint64_t)batch * L.in_h * L.in_w};
    const cuuint64_t strides[1] = {(cuuint64_t)L.cin * 2};
    const cuuint32_t box[2] = {kTcBK, kTcBM};
    const cuuint32_t es[2] = {1, 1};
    r = c.encode_tiled(&e.tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    // NHWC as (C, W, H, N).  Base pixels (filter tap 0,0) range over [-pad, dim - 1 + pad - (k - 1)] in steps of `stride`.
    const cuuint64_t dims[4] = {(cuuint64_t)L.cin, (cuuint64_t)L.in_w, (cuuint64_t)L.in_h, (cuuint64_t)batch};
    const cuuint64_t strides[3] = {(cuuint64_t)L.cin * 2, (cuuint64_t)L.cin * 2 * L.in_w, (cuuint64_t)L.cin * 2 * L.in_w * L.in_h};
    const int lower[2] = {-L.pad_w, -L.pad};                                 // (W, H) corners
    const int upper[2] = {L.pad_w - (L.kw - 1), L.pad - (L.kh - 1)};
    const cuuint32_t es[4] = {1, (cuuint32_t)L.stride, (cuuint32_t)L.stride, 1};
    r = c.encode_im2col(&e.tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, lower, upper, kTcBK,
                        kTcBM, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) return EE_ERR_CUDA;
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

template <int BN, int STAGES, bool RES, bool SPLIT, bool GATHER = false, bool LOCAL = false>
inline cudaError_t tc_launch_t(dim3 grid, cudaStream_t st, const CUtensorMap& a, const CUtensorMap& w, const CUtensorMap& r,
                               const CUtensorMap& o, const TcParams& p) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = TcSmem<BN, STAGES, RES>::kBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // prologue may overlap the previous kernel's tail
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (SPLIT) {  // the K ranges of one tile form a cluster along z
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = grid.z;
    cfg.numAttrs = 2;
  }
  return cudaLaunchKernelEx(&cfg, conv_igemm_tcgen05_kernel<BN, STAGES, RES, SPLIT, GATHER, LOCAL>, a, w, r, o, p);
}

template <int BN>
inline cudaError_t tc_launch_bn(bool deep, bool res, bool split, dim3 grid, cudaStream_t st, const CUtensorMap& a, const CUtensorMap& w,
                                const CUtensorMap& r, const CUtensorMap& o, const TcParams& p) {
  if (p.ranges > 1) {   // one CTA per tile with an accumulator per K range
    if (res) return deep ? tc_launch_t<BN, 5, true, false, false, true>(grid, st, a, w, r, o, p) : tc_launch_t<BN, 2, true, false, false, true>(grid, st, a, w, r, o, p);
    return deep ? tc_launch_t<BN, 6, false, false, false, true>(grid, st, a, w, r, o, p) : tc_launch_t<BN, 3, false, false, false, true>(grid, st, a, w, r, o, p);
  }
  if (split) return deep ? tc_launch_t<BN, 6, false, true>(grid, st, a, w, r, o, p) : tc_launch_t<BN, 3, false, true>(grid, st, a, w, r, o, p);
  if (res) return deep ? tc_launch_t<BN, 5, true, false>(grid, st, a, w, r, o, p) : tc_launch_t<BN, 2, true, false>(grid, st, a, w, r, o, p);
  return deep ? tc_launch_t<BN, 6, false, false>(grid, st, a, w, r, o, p) : tc_launch_t<BN, 3, false, false>(grid, st, a, w, r, o, p);
}

template <int BN, bool RES>
inline cudaError_t tc_launch_persistent(int ctas, cudaStream_t st, const CUtensorMap& a, const CUtensorMap& w, const CUtensorMap& r,
                                        const CUtensorMap& o, const TcParams& p) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctas);
  cfg.blockDim = dim3(TcPersistSmem<BN, RES>::kThreads);
  cfg.dynamicSmemBytes = TcPersistSmem<BN, RES>::kBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, conv_igemm_tcgen05_persistent_kernel<BN, RES, false>, a, w, r, o, a, w, p);
}

// The projection mode: a2 / w2 are the projection's input and weight maps.
template <int BN>
inline cudaError_t tc_launch_persistent_proj(int ctas, cudaStream_t st, const CUtensorMap& a, const CUtensorMap& w, const CUtensorMap& o,
                                             const CUtensorMap& a2, const CUtensorMap& w2, const TcParams& p) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctas);
  cfg.blockDim = dim3(TcPersistSmem<BN, false, true>::kThreads);
  cfg.dynamicSmemBytes = TcPersistSmem<BN, false, true>::kBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, conv_igemm_tcgen05_persistent_kernel<BN, false, true>, a, w, o, o, a2, w2, p);
}

// True when layer L at batch B has at least `waves` tiles per SM on the persistent kernel (1x1, one K range).  tc_launch
// itself takes that kernel from two waves on.
inline bool tc_runs_persistent(const TcContext& c, const TcLayer& L, int B, int waves = 2) {
  if (L.gather || L.halo || L.splits > 1 || L.kh * L.kw != 1) return false;
  const long tiles = (long)cdiv((long)B * L.out_h * L.out_w, kTcBM) * cdiv(L.cout, L.bn);
  return tiles >= (long)waves * c.sm_count;
}

// A layer L whose residual operand is the output of the 1x1 projection P (no padding, one K range, the same tile width
// and output geometry) can compute that operand itself on the persistent kernel (see its PROJ note).
inline bool tc_proj_supported(const TcLayer& L, const TcLayer& P) {
  return !P.gather && !P.halo && P.splits == 1 && P.kh == 1 && P.kw == 1 && P.pad == 0 && P.pad_w == 0 && P.bn == L.bn && P.cout == L.cout &&
         P.out_h == L.out_h && P.out_w == L.out_w && L.kh * L.kw == 1 && L.splits == 1 && !L.gather && !L.halo;
}

// L with the projection P in its launch: src -> L, src2 -> P; P's own output is never written.
inline ee_status_t tc_launch_proj(TcContext& c, const TcLayer& L, const TcLayer& P, const void* src, const void* src2, void* dst, int B,
                                  const float* scale, const float* bias, const float* scale2, const float* bias2, int* err_flag,
                                  cudaStream_t st, float* gap_part = nullptr, int gap_g = 0) {
  if (((uintptr_t)src & 15) || ((uintptr_t)src2 & 15) || ((uintptr_t)dst & 15)) return EE_ERR_INVALID_ARG;
  const CUtensorMap* t = nullptr;
  ee_status_t s = tc_buffer_map(c, L, dst, B, 1, &t);
  if (s != EE_OK) return s;
  const CUtensorMap tmO = *t;
  if ((s = tc_buffer_map(c, L, src, B, 0, &t)) != EE_OK) return s;
  const CUtensorMap tmA = *t;
  if ((s = tc_buffer_map(c, P, src2, B, 0, &t)) != EE_OK) return s;
  const CUtensorMap tmA2 = *t;
  TcParams p = {};
  p.M = B * L.out_h * L.out_w;
  p.N = L.cout;
  p.taps = 1, p.kw = 1;
  p.cblocks = cdiv(L.cin, kTcBK);
  p.Ho = L.out_h, p.Wo = L.out_w, p.stride = L.stride, p.pad = L.pad, p.pad_w = L.pad_w;
  p.im2col = L.im2col ? 1 : 0;
  p.act = L.act;
  p.scale = scale, p.bias = bias;
  p.residual = nullptr;
  p.out = (bf16*)dst;
  p.err_flag = err_flag;
  p.kb_per = L.kb_per;
  p.rev = L.rev ? 1 : 0;
  p.cblocks2 = cdiv(P.cin, kTcBK), p.im2col2 = P.im2col ? 1 : 0, p.stride2 = P.stride, p.act2 = P.act;
  p.scale2 = scale2, p.bias2 = bias2;
  p.gap_part = gap_part, p.gap_g = gap_part ? gap_g : 0;
  const cudaError_t e = L.bn == 128 ? tc_launch_persistent_proj<128>(c.sm_count, st, tmA, L.tm_w, tmO, tmA2, P.tm_w, p)
                                    : tc_launch_persistent_proj<64>(c.sm_count, st, tmA, L.tm_w, tmO, tmA2, P.tm_w, p);
  return e == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

// Sets the number of K ranges of a layer (1 = no split).  Ranges are equal runs of ceil(num_kb / splits) K blocks, the last
// one shorter; returns false when a range would be empty or shorter than two K blocks.
inline bool tc_set_splits(TcLayer& L, int splits) {
  const int num_kb = L.kh * L.kw * cdiv(L.cin, kTcBK);
  if (splits < 1 || splits > 8) return false;
  const int per = cdiv(num_kb, splits);
  if (splits > 1 && (per < 2 || (splits - 1) * per >= num_kb)) return false;
  L.splits = splits;
  L.kb_per = per;
  return true;
}

// gap_part / gap_g: pooling partials (TcParams::gap_g); only a launch on the persistent kernel (tc_runs_persistent) writes them.
inline ee_status_t tc_launch(TcContext& c, const TcLayer& L, const void* src, const void* res, void* dst, int B, const float* scale,
                             const float* bias, int* err_flag, cudaStream_t st, float* gap_part = nullptr, int gap_g = 0,
                             int range_mode = 0) {
  if (((uintptr_t)src & 15) || ((uintptr_t)dst & 15) || ((uintptr_t)res & 15)) return EE_ERR_INVALID_ARG;
  // copies: a later lookup may grow the cache and move its entries
  const CUtensorMap* t = nullptr;
  ee_status_t s = tc_buffer_map(c, L, dst, B, 1, &t);
  if (s != EE_OK) return s;
  const CUtensorMap tmO = *t;
  CUtensorMap tmA = tmO;  // unused in gather mode
  if (!L.gather) {
    if ((s = tc_buffer_map(c, L, src, B, 0, &t)) != EE_OK) return s;
    tmA = *t;
  }
  CUtensorMap tmR = tmO;
  if (res) {
    if ((s = tc_buffer_map(c, L, res, B, 1, &t)) != EE_OK) return s;
    tmR = *t;
  }
  TcParams p = {};
  p.gap_part = gap_part, p.gap_g = gap_part ? gap_g : 0;
  p.M = B * L.out_h * L.out_w;
  p.N = L.cout;
  p.taps = L.kh * L.kw;
  p.kw = L.kw;
  p.cblocks = cdiv(L.cin, kTcBK);
  p.Ho = L.out_h, p.Wo = L.out_w, p.stride = L.stride, p.pad = L.pad, p.pad_w = L.pad_w;
  p.im2col = L.im2col ? 1 : 0;
  p.act = L.act;
  p.scale = scale, p.bias = bias;
  p.residual = (const bf16*)res;
  p.out = (bf16*)dst;
  p.err_flag = err_flag;
  // A layer with several K ranges runs them as a cluster of CTAs per tile (more SMs pull operands: small grids) or, bit
  // for bit the same, in ONE CTA per tile with an accumulator per range (no cluster, no exchange: grids that fill the GPU
  // anyway).  range_mode: 0 = the cluster while the whole grid still fits one wave, 1 = cluster, 2 = one CTA.
  const long tiles_all = (long)cdiv(p.M, kTcBM) * cdiv(L.cout, L.bn);
  const bool can_local = L.splits > 1 && L.splits * L.bn <= 512 && !L.gather;
  // Measured (3x3 256->256 on 14x14, 2 and 4 ranges): the cluster wins while tiles x ranges stays within about 1.25 waves
  // and loses badly beyond; one CTA with 2 accumulators costs 1 us per layer over a single range, with 4 (all 512 TMEM
  // columns: no second CTA, no overlap with the neighbouring kernels' prologues) 17 us.
  const bool local = can_local && (range_mode == 2 || (range_mode == 0 && tiles_all * L.splits * 4 > 5L * c.sm_count));
  const bool split = L.splits > 1 && !local;
  p.ranges = local ? L.splits : 1;
  p.kb_per = L.kb_per;
  p.rev = L.rev ? 1 : 0;
  p.gx = (const bf16*)src;
  p.gH = L.g_h, p.gW = L.g_w, p.gCin = L.g_cin, p.gkh = L.g_kh, p.grun = L.g_kw * L.g_cin, p.grunp = L.g_runp;
  if (L.gather) p.stride = L.g_stride, p.pad = p.pad_w = L.g_pad;
  dim3 grid(cdiv(p.M, kTcBM), cdiv(L.cout, L.bn), split ? L.splits : 1);
  // At most one CTA per SM anyway: take the deep operand ring.  A cluster grid close to the SM count does not: its
  // clusters need all their CTAs inside one GPC, a 192 KB CTA owns its SM, and the last clusters then wait for a second
  // wave (measured: the split-3 3x3 layers of 132 CTAs lose 6 us each with the deep ring).
  const long n_ctas = (long)grid.x * grid.y * grid.z;
  const bool deep = split ? n_ctas * 4 <= 3L * c.sm_count : n_ctas <= c.sm_count;
  const bool tma_res = res && !split;
  if (L.gather) {
    if (res || split) return EE_ERR_INTERNAL;
    cudaError_t ge = L.bn == 128 ? tc_launch_t<128, 3, false, false, true>(grid, st, tmA, L.tm_w, tmR, tmO, p)
                                 : tc_launch_t<64, 3, false, false, true>(grid, st, tmA, L.tm_w, tmR, tmO, p);
    return ge == cudaSuccess ? EE_OK : EE_ERR_CUDA;
  }
  const long tiles = (long)grid.x * grid.y;
  if (!split && L.kh * L.kw == 1 && tiles >= 2 * c.sm_count) {  // several waves of short K loops: one persistent CTA per SM walks the tiles
    const int ctas = c.sm_count;
    cudaError_t pe;
    if (L.bn == 128)
      pe = res ? tc_launch_persistent<128, true>(ctas, st, tmA, L.tm_w, tmR, tmO, p) : tc_launch_persistent<128, false>(ctas, st, tmA, L.tm_w, tmR, tmO, p);
    else
      pe = res ? tc_launch_persistent<64, true>(ctas, st, tmA, L.tm_w, tmR, tmO, p) : tc_launch_persistent<64, false>(ctas, st, tmA, L.tm_w, tmR, tmO, p);
    return pe == cudaSuccess ? EE_OK : EE_ERR_CUDA;
  }
  cudaError_t e = L.bn == 128 ? tc_launch_bn<128>(deep, tma_res, split, grid, st, tmA, L.tm_w, tmR, tmO, p)
                              : tc_launch_bn<64>(deep, tma_res, split, grid, st, tmA, L.tm_w, tmR, tmO, p);
  return e == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace ee
