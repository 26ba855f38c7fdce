// 7x7 stride-2 pad-3 stem convolution on 3-channel bf16 images (the first layer of the ResNet-style backbones of
// paper Section V), as an implicit GEMM on tcgen05.mma.
//
// A 3-channel pixel is 6 bytes, so neither a tiled nor an im2col TMA load can fetch 16-byte pixel rows.  Instead
// one persistent CTA per half SM walks output rows: per output row (n, oy) the producer warp brings the 7 input
// rows it touches into shared memory by TMA (zero fill above, below, left and right of the image), four gather
// warps (one thread per output pixel) cut the Toeplitz rows out of that patch with aligned 32-bit shared-memory
// loads and write them where the 128-byte swizzle of the MMA descriptor expects them, one thread issues the MMAs
// into a double-buffered TMEM accumulator, and four epilogue warps apply scale/bias/activation and store the
// [Wo][Cout] row through a TMA store.  All four roles overlap across consecutive output rows.
//
// K layout: K = 7 runs (filter rows) of 24 columns: column 0 is a dummy, columns 1..21 are the kw*Cin = 21 taps of
// the filter row (contiguous in NHWC), columns 22..23 are padding; 168 columns padded to three K blocks of 64.  The
// dummy column makes every run start on a 4-byte boundary of the patch: the run of pixel ox begins at element
// 6 ox - 10 of the image row, and the patch boxes begin at multiples of 8 elements (16 before the row for the first).  Weights are packed the same way, with zeros in the dummy and
// padding columns; the gather warps zero those columns of A as well, so nothing but real taps enters a sum.
#pragma once
#include "conv_tc.cuh"

namespace ee {

struct StemParams {
  int tiles;            // B * Ho output rows
  int Ho, Wo, N;        // output height, width (<= kStemMaxWo) and Cout (<= 64)
  int act;
  int rev;              // 1: walk the output rows from the last one down
  int Hp, Wp, rows;     // fused pooling only: pooled height and width, rows = B * Hp pooled rows
  const float* scale;
  const float* bias;
  int* err_flag;
};

constexpr int kStemThreads = 320;      // producer, MMA, 4 gather warps, 4 epilogue warps
constexpr int kStemKh = 7, kStemKw = 7, kStemCin = 3, kStemStride = 2, kStemPad = 3;
constexpr int kStemRunWords = 12;      // 24 bf16 columns per filter row
constexpr int kStemLead = 16;          // zero elements in front of each patch row (a TMA load may start at x = -16)
// The patch is three TMA boxes of 7 rows x 256 elements whose first columns sit kStemBoxStep elements apart: they
// overlap by 32 elements, more than one pixel's 24-column run, so every pixel finds its whole run inside one box
// and addresses it with constant offsets.
constexpr int kStemBoxElems = 256, kStemBoxes = 3, kStemBoxStep = 224;
constexpr int kStemBoxRowBytes = kStemBoxElems * 2;
constexpr int kStemBoxBytes = kStemKh * kStemBoxRowBytes;
constexpr int kStemPatchBytes = kStemBoxes * kStemBoxBytes;
constexpr int kStemKBlocks = 3;
// image elements (before the lead-in shift) the boxes cover: [-kStemLead, kStemCover)
constexpr int kStemCover = (kStemBoxes - 1) * kStemBoxStep + kStemBoxElems - kStemLead;
// the run of pixel ox spans elements [6 ox - 10, 6 ox + 13] of the image row
constexpr int kStemMaxWo = (kStemCover - 14) / (kStemStride * kStemCin) + 1;

struct StemSmem {
  static constexpr int kABytes = kTcBM * kTcBK * 2;        // one K block of A
  static constexpr int kWBytes = 64 * kTcBK * 2;           // one K block of the weights
  static constexpr int kAOff = 0;
  static constexpr int kWOff = kAOff + kStemKBlocks * kABytes;
  static constexpr int kOOff = kWOff + kStemKBlocks * kWBytes;
  static constexpr int kPatchOff = kOOff + kTcBM * 64 * 2;
  static constexpr int kScaleOff = kPatchOff + 2 * kStemPatchBytes;
  static constexpr int kBarOff = kScaleOff + 2 * 64 * 4;
  static constexpr int kBytes = kBarOff + 256 + 1024;
  static_assert(kPatchOff % 128 == 0 && kBarOff % 8 == 0, "alignment");
  static_assert(2 * (kBytes + 1024) <= 228 * 1024, "two CTAs per SM");
};

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* tm, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(tm), "r"(src), "r"(c0), "r"(c1),
               "r"(c2)
               : "memory");
}

// The output rows a CTA computes, in order: body(j, n, oy, fresh, emit, t) for the CTA's j-th row, row oy of image n.
// Without pooling the rows of the batch are dealt round-robin (t = the row's index over the batch).  With the 3x3
// stride-2 pad-1 max-pool fused behind the convolution a CTA owns a contiguous range of POOLED rows (t = the pooled
// row's index over the batch) and walks the convolution rows they cover in ascending order: rows 2py-1 .. 2py+1 for
// the first pooled row of the range or of an image (`fresh` marks the row that starts a new running maximum), rows
// 2py and 2py+1 for the others (row 2py-1 was the row before); `emit` marks the last row of a pooled row.  body
// returns false to stop the walk.
template <bool POOL, typename F>
__device__ __forceinline__ void stem_walk(const StemParams& p, F&& body) {
  if constexpr (!POOL) {
    const int mine = (int)blockIdx.x < p.tiles ? (p.tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    for (int j = 0; j < mine; ++j) {
      const int tf = (int)blockIdx.x + j * (int)gridDim.x, t = p.rev ? p.tiles - 1 - tf : tf;
      const int n = t / p.Ho;
      if (!body(j, n, t - n * p.Ho, false, false, t)) return;
    }
  } else {
    const long g = p.rev ? (long)gridDim.x - 1 - blockIdx.x : (long)blockIdx.x;
    const int r0 = (int)(g * p.rows / gridDim.x), r1 = (int)((g + 1) * p.rows / gridDim.x);
    int j = 0;
    for (int r = r0; r < r1; ++r) {
      const int n = r / p.Hp, py = r - n * p.Hp;
      const bool first = r == r0 || py == 0;
      const int lo = first ? max(2 * py - 1, 0) : 2 * py, hi = min(2 * py + 1, p.Ho - 1);
      for (int c = lo; c <= hi; ++c, ++j)
        if (!body(j, n, c, first && c == lo, c == hi, r)) return;
    }
  }
}

__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
  const __nv_bfloat162 r = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
  return *reinterpret_cast<const uint32_t*>(&r);
}

// tmX: input as (W*3, H, B) with a 256 x 7 x 1 box, no swizzle; tmW: packed weights (192, 1, Cout) with a 64 x 1 x 64
// box, 128-byte swizzle; tmO: output as (Cout, Wo, B*Ho) with a 64 x 32 x 1 box, 128-byte swizzle, so that pixels past
// Wo are clipped by the TMA unit (POOL: the pooled tensor, (Cout, Wp, B*Hp), same box).
//
// POOL: the epilogue threads keep the running maximum over the convolution rows of a pooled row in registers (a
// thread owns one pixel column, all channels), and on the last of them put it in the staging tile, take the maximum
// over the three columns of every pooled pixel there and store the pooled row; the convolution's own output never
// reaches global memory.  max() of bf16 values is exact, so the result equals pooling the stored convolution output.
template <bool POOL>
__global__ void __launch_bounds__(kStemThreads, 2)
conv_stem7x7_tcgen05_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                            const __grid_constant__ CUtensorMap tmO, StemParams p) {
  extern __shared__ uint8_t smem_raw[];
  using S = StemSmem;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  float* s_scale = reinterpret_cast<float*>(gen + S::kScaleOff);
  float* s_bias = s_scale + 64;
  const uint32_t bar0 = base + S::kBarOff;
  const uint32_t w_bar = bar0;
  auto patch_full = [&](int b) { return bar0 + 8u * (1 + b); };
  auto patch_empty = [&](int b) { return bar0 + 8u * (3 + b); };
  auto a_full = [&](int i) { return bar0 + 8u * (5 + i); };
  auto a_empty = [&](int i) { return bar0 + 8u * (8 + i); };
  auto acc_full = [&](int b) { return bar0 + 8u * (11 + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (13 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + S::kBarOff + 8 * 15);
  volatile int* s_abort = reinterpret_cast<volatile int*>(gen + S::kBarOff + 8 * 16);   // POOL: an epilogue warp gave up

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    *s_abort = 0;
    mbar_init(w_bar, 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(patch_full(b), 1);
      mbar_init(patch_empty(b), 4);   // lane 0 of each gather warp
      mbar_init(acc_full(b), 1);
      mbar_init(acc_empty(b), 4);     // lane 0 of each epilogue warp
    }
    for (int i = 0; i < kStemKBlocks; ++i) {
      mbar_init(a_full(i), 128);      // every gather thread, after its own proxy fence
      mbar_init(a_empty(i), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmO) : "memory");
  }
  if (warp == 1) {  // two accumulators of 64 fp32 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(128) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (warp == 0 && lane == 0) {   // the whole weight matrix stays resident; no kernel writes it, so it need not wait
    mbar_expect_tx(w_bar, kStemKBlocks * S::kWBytes);
    for (int i = 0; i < kStemKBlocks; ++i) tma_load_3d(base + S::kWOff + i * S::kWBytes, &tmW, w_bar, i * kTcBK, 0, 0);
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    if (lane == 0) {
      stem_walk<POOL>(p, [&](int j, int n, int oy, bool, bool, int) {
        const int b = j & 1;
        if (j >= 2 && !mbar_wait(patch_empty(b), (uint32_t)((j >> 1) - 1) & 1u, p.err_flag)) return false;
        mbar_expect_tx(patch_full(b), kStemPatchBytes);
        const uint32_t dst = base + S::kPatchOff + b * kStemPatchBytes;
#pragma unroll
        for (int c = 0; c < kStemBoxes; ++c)   // rows outside the image and columns outside the row arrive as zeros
          tma_load_3d(dst + c * kStemBoxBytes, &tmX, patch_full(b), c * kStemBoxStep - kStemLead, oy * kStemStride - kStemPad, n);
        return true;
      });
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc(64);
      if (mbar_wait(w_bar, 0, p.err_flag))
        stem_walk<POOL>(p, [&](int j, int, int, bool, bool, int) {
          const int b = j & 1;
          // the epilogue must have drained this accumulator (row j - 2)
          if (j >= 2 && !mbar_wait(acc_empty(b), (uint32_t)((j >> 1) - 1) & 1u, p.err_flag)) return false;
          tc_fence_after();
          const uint32_t acc = tmem_base + (uint32_t)(b * 64);
#pragma unroll
          for (int i = 0; i < kStemKBlocks; ++i) {
            if (!mbar_wait(a_full(i), (uint32_t)j & 1u, p.err_flag)) return false;
            tc_fence_after();
            const uint32_t sa = base + S::kAOff + i * S::kABytes, sb = base + S::kWOff + i * S::kWBytes;
#pragma unroll
            for (int k = 0; k < kTcBK / 16; ++k) umma_bf16(acc, umma_desc(sa + k * 32), umma_desc(sb + k * 32), idesc, (uint32_t)((i | k) != 0));
            umma_commit(a_empty(i));   // the gather warps may rebuild this K block for the next output row
          }
          umma_commit(acc_full(b));
          return true;
        });
    }
  } else if (warp < 6) {
    // gather warps: thread r builds row r (output pixel ox = r) of every K block of A
    const int r = (int)threadIdx.x - 64;
    const int ox = min(r, p.Wo - 1);   // rows past Wo repeat the last pixel; the store clips them
    const int e0 = kStemStride * kStemCin * ox - kStemPad * kStemCin - 1;   // image-row element of column 0 of the run (even)
    int box = 0;                                                            // first box that holds the whole run
#pragma unroll
    for (int c = 1; c < kStemBoxes; ++c)
      if (e0 + 2 * kStemRunWords - 1 > (c - 1) * kStemBoxStep - kStemLead + kStemBoxElems - 1) box = c;
    const uint32_t* prow =
        reinterpret_cast<const uint32_t*>(gen + S::kPatchOff + box * kStemBoxBytes) + (e0 - (box * kStemBoxStep - kStemLead)) / 2;
    uint8_t* aline = gen + S::kAOff + r * 128;
    stem_walk<POOL>(p, [&](int j, int, int, bool, bool, int) {
      const int b = j & 1;
      if (!mbar_wait(patch_full(b), (uint32_t)(j >> 1) & 1u, p.err_flag)) return false;
      const uint32_t* pw = prow + b * (kStemPatchBytes / 4);
#pragma unroll
      for (int i = 0; i < kStemKBlocks; ++i) {
        if (!mbar_wait(a_empty(i), ((uint32_t)j & 1u) ^ 1u, p.err_flag)) return false;
        uint32_t w[32];   // the 64 columns of this K block, two per word; all loads issued before the first store
#pragma unroll
        for (int q = 0; q < 32; ++q) {
          const int kw = i * 32 + q, rf = kw / kStemRunWords, jw = kw % kStemRunWords;   // compile-time after unrolling
          if (rf >= kStemKh || jw == kStemRunWords - 1)
            w[q] = 0u;                                          // K padding, columns 22..23
          else if (jw == 0)
            w[q] = pw[rf * (kStemBoxRowBytes / 4)] & 0xFFFF0000u;  // dummy column 0 | first tap
          else
            w[q] = pw[rf * (kStemBoxRowBytes / 4) + jw];
        }
        uint8_t* line = aline + i * S::kABytes;
#pragma unroll
        for (int c = 0; c < 8; ++c)
          *reinterpret_cast<uint4*>(line + ((c ^ (r & 7)) << 4)) = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(a_full(i)) : "memory");
      }
      __syncwarp();   // every lane has read its taps: the patch buffer may be refilled
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(patch_empty(b)) : "memory");
      return true;
    });
  } else {
    // epilogue warps 6..9: TMEM lane quarter = warp % 4
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const int et = (int)threadIdx.x - 192;
    if (et < 64) {
      const bool in = et < p.N;
      s_scale[et] = (p.scale && in) ? p.scale[et] : 1.f;
      s_bias[et] = (p.bias && in) ? p.bias[et] : 0.f;
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");   // once, before the tile loop
    uint8_t* oline = gen + S::kOOff + row * 128;
    bool pending = false;  // the storing lane: a bulk store may still be reading the staging rows
    if constexpr (!POOL) {
      stem_walk<POOL>(p, [&](int j, int, int, bool, bool, int t) {
        const int b = j & 1;
        if (!__all_sync(0xffffffffu, mbar_wait(acc_full(b), (uint32_t)(j >> 1) & 1u, p.err_flag))) return false;
        tc_fence_after();
        const uint32_t acc = tmem_base + (uint32_t)(b * 64) + ((uint32_t)(q * 32) << 16);
        float va[32], vb[32];
        tmem_ld32_issue(acc, va);
        tmem_ld32_issue(acc + 32, vb);
        tmem_ld_wait(va, vb);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acc_empty(b)) : "memory");   // the MMA warp may refill it
          if (pending) {
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            pending = false;
          }
        }
        __syncwarp();
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          float* v = sub ? vb : va;
          scale_bias<32>(v, s_scale + sub * 32, s_bias + sub * 32);
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            Vec16<bf16> o;
#pragma unroll
            for (int e = 0; e < 8; ++e) o.v[e] = apply_act(v[g * 8 + e], p.act);
            o.store(reinterpret_cast<bf16*>(oline + (((sub * 4 + g) ^ (lane & 7)) << 4)));
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          if (q * 32 < p.Wo) tma_store_3d(&tmO, base + S::kOOff + q * 4096, 0, q * 32, t);   // pixels past Wo, channels past Cout: clipped
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          pending = true;
        }
        return true;
      });
    } else {
      // The four epilogue warps meet at barriers when a pooled row goes out, so a warp whose wait ran out must not
      // leave: it raises s_abort and from then on only keeps the barriers' count; the others see the flag at their
      // next row and do the same.
      uint32_t vm[32];   // running maximum over the rows of the open pooled row: this thread's pixel column, 64 channels
#pragma unroll
      for (int i = 0; i < 32; ++i) vm[i] = 0u;
      const int items = p.Wp * 8;   // (pooled pixel, 16-byte channel group) pairs of a pooled row
      bool live = true;
      stem_walk<POOL>(p, [&](int j, int, int, bool fresh, bool emit, int t) {
        const int b = j & 1;
        live = live && !__any_sync(0xffffffffu, *s_abort != 0);
        if (live && !__all_sync(0xffffffffu, mbar_wait(acc_full(b), (uint32_t)(j >> 1) & 1u, p.err_flag))) {
          live = false;
          *s_abort = 1;
        }
        if (emit) {   // the staging tile is about to be rewritten: the store of the pooled row before must have read it
          if (et == 0 && pending) {
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            pending = false;
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        if (live) {
          tc_fence_after();
          const uint32_t acc = tmem_base + (uint32_t)(b * 64) + ((uint32_t)(q * 32) << 16);
#pragma unroll
          for (int sub = 0; sub < 2; ++sub) {
            float v[32];
            tmem_ld32(acc + (uint32_t)(sub * 32), v);
            if (sub == 1) {   // the whole accumulator row is in registers: the MMA warp may refill it
              tc_fence_before();
              __syncwarp();
              if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acc_empty(b)) : "memory");
            }
            scale_bias<32>(v, s_scale + sub * 32, s_bias + sub * 32);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint32_t* m4 = vm + (sub * 4 + g) * 4;
              uint32_t cur[4], top[4];   // this row's values; the maximum including them
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const __nv_bfloat162 h = __floats2bfloat162_rn(apply_act(v[g * 8 + 2 * e], p.act), apply_act(v[g * 8 + 2 * e + 1], p.act));
                cur[e] = *reinterpret_cast<const uint32_t*>(&h);
                top[e] = fresh ? cur[e] : bf16x2_max(m4[e], cur[e]);
                m4[e] = emit ? cur[e] : top[e];   // the last row of a pooled row is the first row of the next one
              }
              if (emit) *reinterpret_cast<uint4*>(oline + (((sub * 4 + g) ^ (lane & 7)) << 4)) = make_uint4(top[0], top[1], top[2], top[3]);
            }
          }
        }
        if (!emit) return true;
        asm volatile("bar.sync 1, 128;" ::: "memory");   // the row of running maxima is staged
        uint4 res[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int idx = et + k * 128;
          res[k] = make_uint4(0u, 0u, 0u, 0u);
          if (idx < items) {
            const int px = idx >> 3, ch = idx & 7;
            const int c1 = 2 * px;   // columns 2px-1 .. 2px+1, clipped to the row
            const uint8_t* stg = gen + S::kOOff;
            uint4 m = *reinterpret_cast<const uint4*>(stg + c1 * 128 + ((ch ^ (c1 & 7)) << 4));
            if (c1 >= 1) {
              const uint4 a = *reinterpret_cast<const uint4*>(stg + (c1 - 1) * 128 + ((ch ^ ((c1 - 1) & 7)) << 4));
              m = make_uint4(bf16x2_max(m.x, a.x), bf16x2_max(m.y, a.y), bf16x2_max(m.z, a.z), bf16x2_max(m.w, a.w));
            }
            if (c1 + 1 < p.Wo) {
              const uint4 a = *reinterpret_cast<const uint4*>(stg + (c1 + 1) * 128 + ((ch ^ ((c1 + 1) & 7)) << 4));
              m = make_uint4(bf16x2_max(m.x, a.x), bf16x2_max(m.y, a.y), bf16x2_max(m.z, a.z), bf16x2_max(m.w, a.w));
            }
            res[k] = m;
          }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");   // every column is read: the pooled row may overwrite the tile's first rows
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int idx = et + k * 128;
          if (idx < items) {
            const int px = idx >> 3, ch = idx & 7;
            *reinterpret_cast<uint4*>(gen + S::kOOff + px * 128 + ((ch ^ (px & 7)) << 4)) = res[k];
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (et == 0 && *s_abort == 0) {
          for (int x0 = 0; x0 < p.Wp; x0 += 32) tma_store_3d(&tmO, base + S::kOOff + x0 * 128, 0, x0, t);   // pixels past Wp: clipped
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          pending = true;
        }
        return true;
      });
    }
    if (pending) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(128) : "memory");
  }
}

// Weight rows [Cout][7][21] into the K layout above: [Cout][7 runs][dummy | 21 taps | 2 zeros], padded to 192 columns.
__global__ void pack_stem_weights_kernel(const bf16* __restrict__ w, bf16* __restrict__ out, int rows) {
  constexpr int run = kStemKw * kStemCin, runp = 2 * kStemRunWords, Kp = kStemKBlocks * kTcBK;
  const long total = (long)rows * Kp;
  for (long idx = (long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
    const int k = (int)(idx % Kp);
    const long co = idx / Kp;
    const int r = k / runp, j = k - r * runp - 1;
    out[idx] = (r < kStemKh && j >= 0 && j < run) ? w[(co * kStemKh + r) * run + j] : __float2bfloat16_rn(0.f);
  }
}

// ----------------------------------------------------------------------------- host side

inline bool stem_supported(const ee_layer_desc_t& d, int in_h, int in_w, int out_w) {
  (void)in_h;
  return d.op == EE_OP_CONV && d.cin == kStemCin && d.kh == kStemKh && d.kw == kStemKw && d.stride == kStemStride && d.pad == kStemPad && d.pad_w == kStemPad &&
         d.cout % 8 == 0 && d.cout <= 64 && in_w % 8 == 0 && out_w <= kStemMaxWo;
}

inline ee_status_t stem_context_init() {
  return cudaFuncSetAttribute(conv_stem7x7_tcgen05_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, StemSmem::kBytes) == cudaSuccess &&
                 cudaFuncSetAttribute(conv_stem7x7_tcgen05_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, StemSmem::kBytes) == cudaSuccess
             ? EE_OK
             : EE_ERR_CUDA;
}

// The pooling layer the stem kernel can take into its epilogue: 3x3 windows, stride 2, one pixel of padding.
inline bool stem_pool_supported(const ee_layer_desc_t& pool) {
  return pool.op == EE_OP_MAXPOOL && pool.kh == 3 && pool.kw == 3 && pool.stride == 2 && pool.pad == 1 && pool.pad_w == 1;
}

// L: the layer's GEMM view planned by tc_plan_layer over the packed weights (tm_w), with the g_* fields holding the
// geometry of the real convolution.  pool: dst is the output of the 3x3 stride-2 pad-1 max-pool behind the convolution,
// [B][(Ho-1)/2+1][(Wo-1)/2+1][Cout].
inline ee_status_t stem_launch(TcContext& c, const TcLayer& L, const void* src, void* dst, int B, const float* scale, const float* bias,
                               int* err_flag, cudaStream_t st, bool pool = false) {
  if (((uintptr_t)src & 15) || ((uintptr_t)dst & 15)) return EE_ERR_INVALID_ARG;
  const CUtensorMap* t = nullptr;
  ee_status_t s = tc_buffer_map(c, L, dst, B, pool ? 5 : 3, &t);
  if (s != EE_OK) return s;
  const CUtensorMap tmO = *t;   // copies: a later lookup may grow the cache and move its entries
  if ((s = tc_buffer_map(c, L, src, B, 2, &t)) != EE_OK) return s;
  const CUtensorMap tmX = *t;
  StemParams p;
  p.tiles = B * L.out_h;
  p.Ho = L.out_h, p.Wo = L.out_w, p.N = L.cout;
  p.act = L.act;
  p.rev = L.rev ? 1 : 0;
  p.Hp = (L.out_h - 1) / 2 + 1, p.Wp = (L.out_w - 1) / 2 + 1, p.rows = B * p.Hp;
  p.scale = scale, p.bias = bias;
  p.err_flag = err_flag;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(std::min(pool ? p.rows : p.tiles, 2 * c.sm_count));   // two persistent CTAs per SM
  cfg.blockDim = dim3(kStemThreads);
  cfg.dynamicSmemBytes = StemSmem::kBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = pool ? cudaLaunchKernelEx(&cfg, conv_stem7x7_tcgen05_kernel<true>, tmX, L.tm_w, tmO, p)
                             : cudaLaunchKernelEx(&cfg, conv_stem7x7_tcgen05_kernel<false>, tmX, L.tm_w, tmO, p);
  return e == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace ee
