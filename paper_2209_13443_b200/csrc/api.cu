// C ABI of the early-exit CNN stage executor: model creation (weight upload, per-layer kernel
// plan, workspace layout), ee_stage_run, ee_batch_refill and the stand-alone head / gather calls.
#include <atomic>
#include <chrono>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"
#include "conv_simt.cuh"
#include "conv_tc.cuh"
#include "conv_stem.cuh"
#include "conv_halo.cuh"
#include "conv_pair.cuh"
#include "conv_dw.cuh"
#include "head.cuh"

using namespace ee;

namespace {

thread_local std::string g_cuda_err;

#define EE_CUDA(expr)                                                                      \
  do {                                                                                     \
    cudaError_t e__ = (expr);                                                              \
    if (e__ != cudaSuccess) {                                                              \
      g_cuda_err = std::string(#expr) + ": " + cudaGetErrorString(e__);                    \
      return EE_ERR_CUDA;                                                                  \
    }                                                                                      \
  } while (0)

constexpr int kBranchMaxBatch = 32;   // shortcut layers run on the branch stream up to this batch size

enum KernelKind { KK_SIMT = 0, KK_TC = 1, KK_DW = 2, KK_POOL = 3, KK_TC_GATHER = 4 };
const char* kKernelNames[] = {"conv_igemm_simt", "conv_igemm_tcgen05", "dwconv", "maxpool", "conv_igemm_tcgen05_gather"};

struct LayerPlan {
  ee_layer_desc_t d;
  int in_h, in_w, out_h, out_w;
  int src_slot;  // -1 = stage input
  int res_slot;  // -2 = none, -1 = stage input
  int out_slot;
  KernelKind kind;
  void* w_dev = nullptr;
  float* scale_dev = nullptr;
  float* bias_dev = nullptr;
  TcLayer tc;  // tensor-core plan (valid iff kind == KK_TC or KK_TC_GATHER)
  // Kernel variant per batch size, index 0..max_batch (TcVariant; empty = TCV_AUTO everywhere).  The analogue of the
  // paper's per-(layer, batch) look-up table that configures the array for the active batch (Section III-C): the
  // variant may change with the batch, the layer's K ranges (tc.splits) may not.
  std::vector<uint8_t> variant;
  // Branch execution: a layer whose output is only ever a residual operand (the projection shortcut of a block) does
  // not depend on the layers between its input and its consumer, so it runs on a side stream beside them.
  // A stem convolution read only by the 3x3 stride-2 pad-1 max-pool right behind it takes that pool into its epilogue
  // inside ee_stage_run (the convolution's own output is then never written); ee_layer_run still runs either alone.
  bool pool_next = false;     // this layer's launch also does the pooling of the next layer
  bool fused_away = false;    // this (pooling) layer's work is done by the launch of the layer before it
  // A projection shortcut (1x1, no padding, read only as the residual operand of one later layer) can be computed inside
  // that layer's launch, on the persistent kernel (see conv_tc.cuh, PROJ).
  int proj_into = -1;         // projection: the layer that can absorb it
  int proj_from = -1;         // absorbing layer: its projection
  bool side = false;          // runs on the model's branch stream
  int wait_for = -1;          // layer index of a side layer whose result this layer consumes
  cudaEvent_t ev_fork = nullptr, ev_done = nullptr;
};

struct StageCallKey {  // everything that distinguishes one ee_stage_run call from another
  ee_stage_in_t in;
  ee_stage_out_t out;
  void* ws;
};
struct StageGraph {
  StageCallKey key;
  cudaGraphExec_t exec;
};
inline bool same_call(const StageCallKey& a, const StageCallKey& b) {  // field by field: the structs have padding
  return a.ws == b.ws && a.in.features == b.in.features && a.in.ids == b.in.ids && a.in.batch == b.in.batch &&
         a.in.logit_shift == b.in.logit_shift && a.in.shift_class == b.in.shift_class &&
         a.out.features_out == b.out.features_out && a.out.conf == b.out.conf && a.out.pred == b.out.pred &&
         a.out.logits == b.out.logits && a.out.exit_mask == b.out.exit_mask && a.out.survivor_idx == b.out.survivor_idx &&
         a.out.ids_out == b.out.ids_out && a.out.n_surv_dev == b.out.n_surv_dev && a.out.n_surv_host == b.out.n_surv_host;
}

struct StagePlan {
  std::vector<LayerPlan> layers;
  std::vector<int> order;          // execution order of the layers (side layers hoisted to where their input is ready)
  // Runs of consecutive layers (positions in `order`) that the CTA-pair kernel can execute in ONE launch, with a grid
  // barrier instead of a kernel boundary between them (see conv_pair.cuh).
  struct Segment {
    int first, n, bn;
  };
  std::vector<Segment> segments;
  std::vector<int> seg_at;         // position -> index into `segments` if a segment starts there, else -1
  std::vector<StageGraph> graphs;  // captured stage executions by call signature
  std::vector<cudaGraphExec_t> retired;   // evicted executables: they may still be in flight, destroyed later
  int in_h, in_w, in_c, out_h, out_w, out_c, out_slot;
  std::vector<size_t> slot_off;  // byte offsets at max_batch
  size_t head_off = 0, ws_bytes = 0, head_bytes = 0;
  size_t split_off = 0, split_bytes = 0;   // split-K partial tiles of the pair kernel, behind the head scratch
  // Pooling partials: when the stage's last layer runs on the persistent tensor-core kernel its epilogue also writes
  // the column sums of every block of gap_g (32 or 16) output rows; the head then pools those block sums instead of
  // reading the feature map again (same bits: see gap_blocks_kernel).  0 = the map's height * width has no such block.
  int out_layer = 0, gap_g = 0;
  size_t gapp_off = 0, gapp_bytes = 0;
  int n_classes = 0;
  void* fc_w = nullptr;
  float* fc_b = nullptr;
  float threshold = 0.f;
  int always_exit = 0;
  bool gap_rev = false, gather_rev = false;   // walk directions of the pooling and gather kernels
  double flops_per_sample = 0;
  // timing of the last run
  std::vector<cudaEvent_t> ev;
  std::vector<const char*> ev_names;
  int ev_used = 0;
};

size_t esize(int dtype) { return dtype == EE_BF16 ? 2 : 4; }

struct HeadLayout {
  size_t off_gap, off_z, off_cnt, bytes;
};

HeadLayout head_layout(int max_batch, int c, int k) {
  HeadLayout h;
  size_t o = 0;
  h.off_cnt = o;
  o = align_up(o + sizeof(unsigned) * ((size_t)max_batch + 1), 256);  // the FC kernel's per-tile counters, then its tile count
  h.off_gap = o;
  o = align_up(o + sizeof(float) * (size_t)max_batch * c, 256);
  h.off_z = o;
  o = align_up(o + sizeof(float) * (size_t)max_batch * k, 256);
  h.bytes = o;
  return h;
}

// Launch with programmatic stream serialization: the kernel may start while its predecessor in the stream drains
// and calls griddepcontrol.wait before it touches that kernel's results.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

}  // namespace

struct ee_model {
  int dtype, in_h, in_w, in_c, max_batch;
  std::vector<StagePlan> stages;
  std::vector<void*> owned;  // device allocations
  int* err_flag = nullptr;   // device word set by kernels whose bounded waits ran out
  unsigned* pair_counters = nullptr;   // arrival counters of the pair kernel's split-K reduction; zero between launches
  unsigned* grid_bar = nullptr;        // arrival counters of the barriers between the layers of a multi-layer launch
  bool stage_kernel = false;           // run eligible layer runs as one launch (measured slower than per-layer launches: off)
  int stage_kernel_max_batch = 1 << 30;
  size_t pair_counter_words = 0;
  unsigned* head_done = nullptr;       // one arrival counter per stage for the one-launch exit head; zero between launches
  int proj_waves = 0;                  // tiles per SM from which a layer absorbs its projection (measured: a gain at every batch)
  bool gap_fusion = true;              // pooling partials from the last layer's epilogue where that applies
  bool proj_fusion = true;             // projection shortcuts computed inside the layer that adds them, where that applies
  bool fused_head = false;             // bf16 models: pool + FC + decision + scan as one cluster kernel where the shape allows (an option)
  long long wait_cycles = kTcWaitCycles;   // limit of the bounded device-side waits of the pair kernel and the self-test
  int device = -1;           // the GPU the model lives on
  bool timing = false;
  bool graphs = true;  // replay stages as CUDA graphs on capturable streams
  TcContext tc;
  // the survivor count travels to the host on a side branch, beside the gather of the survivors' features
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  cudaStream_t branch = nullptr;   // shortcut layers run here, beside the main chain of their block
  cudaStream_t cap = nullptr;      // the bodies of a device-sized stage chain are captured on this stream
  int chain_max_batch = 0;         // ee_run_until_exit runs as ONE graph for batches up to this size (0 = host-sized stages)
  struct ChainGraph {
    int first;
    ee_stage_in_t in;
    void* ws;
    std::vector<ee_stage_out_t> outs;
    cudaGraph_t graph;
    cudaGraphExec_t exec;
  };
  std::vector<ChainGraph> chains;
  bool branches = true;
};

namespace {

template <typename T>
ee_status_t upload(ee_model* m, const T* src, size_t n, int on_device, cudaStream_t st, T** out) {
  *out = nullptr;
  if (!src || n == 0) return EE_OK;
  void* p = nullptr;
  EE_CUDA(cudaMalloc(&p, align_up(n * sizeof(T), 256)));
  m->owned.push_back(p);
  EE_CUDA(cudaMemcpyAsync(p, src, n * sizeof(T), on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, st));
  *out = (T*)p;
  return EE_OK;
}

ee_status_t upload_bytes(ee_model* m, const void* src, size_t bytes, int on_device, cudaStream_t st, void** out) {
  return upload<char>(m, (const char*)src, bytes, on_device, st, (char**)out);
}

void record(ee_model* m, StagePlan& sp, cudaStream_t st, const char* name) {
  if (!m->timing) return;
  if ((int)sp.ev.size() <= sp.ev_used) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return;
    sp.ev.push_back(e);
    sp.ev_names.push_back(name);
  }
  sp.ev_names[sp.ev_used] = name;
  cudaEventRecord(sp.ev[sp.ev_used++], st);
}

// Recomputes the workspace layout of a stage behind its layer slots: head scratch, then the split-K partial tiles of
// the layers that may run on the pair kernel.
void layout_stage_tail(ee_model* m, StagePlan& sp) {
  size_t need = 0;
  for (const LayerPlan& L : sp.layers)
    if (L.kind == KK_TC && !L.tc.gather && !L.tc.halo && L.tc.splits > 1)
      need = std::max(need, std::max(pair_partial_bytes(L.tc, m->max_batch, 256), pair_partial_bytes(L.tc, m->max_batch, 128)));
  sp.split_off = align_up(sp.head_off + sp.head_bytes, 1024);
  sp.split_bytes = need;
  sp.gapp_off = align_up(sp.split_off + need, 1024);
  sp.gapp_bytes = sp.gap_g ? (size_t)m->max_batch * (sp.out_h * sp.out_w / sp.gap_g) * sp.out_c * sizeof(float) : 0;
  sp.ws_bytes = sp.gapp_off + sp.gapp_bytes;
}

template <typename T>
ee_status_t launch_layer(ee_model* m, const LayerPlan& L, const void* src, const void* res, void* dst, int B, float* partial,
                         size_t partial_bytes, cudaStream_t st, bool fuse_pool = false, float* gap_part = nullptr, int gap_g = 0) {
  ConvGeom g{B, L.in_h, L.in_w, L.d.cin, L.out_h, L.out_w, L.d.cout, L.d.kh, L.d.kw, L.d.stride, L.d.pad, L.d.pad_w, L.d.act};
  constexpr int V = Elem<T>::kVec;
  switch (L.kind) {
    case KK_SIMT: {
      dim3 grid(cdiv((long)B * L.out_h * L.out_w, kSimtBM), cdiv(L.d.cout, kSimtBN));
      conv_igemm_simt_kernel<T><<<grid, kSimtThreads, 0, st>>>((const T*)src, (const T*)L.w_dev, L.scale_dev, L.bias_dev,
                                                                 (const T*)res, (T*)dst, g);
      break;
    }
    case KK_TC: {
      const int v = L.variant.empty() ? (int)TCV_AUTO : (int)L.variant[B];
      ee_status_t s = EE_ERR_INTERNAL;
      if constexpr (sizeof(T) == 2) {
        const bool pair_v = v == TCV_PAIR256 || v == TCV_PAIR128;
        const int range_mode = v == TCV_RANGES_CLUSTER ? 1 : v == TCV_RANGES_LOCAL ? 2 : 0;
        if (pair_v && pair_supported(L.tc, v))
          s = pair_launch(m->tc, L.tc, v, src, res, dst, B, L.scale_dev, L.bias_dev, m->err_flag, partial, partial_bytes, m->pair_counters,
                          m->wait_cycles, st);
        else
          s = L.tc.halo ? halo_launch(m->tc, L.tc, src, dst, B, L.scale_dev, L.bias_dev, m->err_flag, st)
                        : tc_launch(m->tc, L.tc, src, res, dst, B, L.scale_dev, L.bias_dev, m->err_flag, st, gap_part, gap_g, range_mode);
      }
      if (s != EE_OK) return s;
      break;
    }
    case KK_TC_GATHER: {
      if constexpr (sizeof(T) == 2) {
        ee_status_t s = L.tc.stem7 ? stem_launch(m->tc, L.tc, src, dst, B, L.scale_dev, L.bias_dev, m->err_flag, st, fuse_pool)
                                   : tc_launch(m->tc, L.tc, src, res, dst, B, L.scale_dev, L.bias_dev, m->err_flag, st);
        if (s != EE_OK) return s;
      } else {
        return EE_ERR_INTERNAL;
      }
      break;
    }
    case KK_DW: {
      if constexpr (sizeof(T) == 2) {
        if (dw_tma_supported(g, src, L.w_dev, dst)) {
          ee_status_t s = dw_tma_launch(m->tc, L.tc, g, src, L.w_dev, L.scale_dev, L.bias_dev, dst, m->err_flag, st);
          if (s != EE_OK) return s;
          break;
        }
        if (dwconv3x3_supported(g, src, L.w_dev, dst)) {
          EE_CUDA(dwconv3x3_launch((const bf16*)src, (const bf16*)L.w_dev, L.scale_dev, L.bias_dev, (bf16*)dst, g, st));
          break;
        }
      }
      const bool vec = L.d.cin % V == 0;
      const long total = (long)B * L.out_h * L.out_w * (vec ? L.d.cin / V : L.d.cin);
      const int grid = (int)std::min<long>(cdiv(total, 256), 148L * 32);
      if (vec)
        dwconv_kernel<T, V><<<grid, 256, 0, st>>>((const T*)src, (const T*)L.w_dev, L.scale_dev, L.bias_dev, (T*)dst, g);
      else
        dwconv_kernel<T, 1><<<grid, 256, 0, st>>>((const T*)src, (const T*)L.w_dev, L.scale_dev, L.bias_dev, (T*)dst, g);
      break;
    }
    case KK_POOL: {
      if constexpr (sizeof(T) == 2) {
        if (dw_tma_supported(g, src, nullptr, dst)) {
          ee_status_t s = dw_tma_launch(m->tc, L.tc, g, src, nullptr, nullptr, nullptr, dst, m->err_flag, st);
          if (s != EE_OK) return s;
          break;
        }
      }
      const bool vec = L.d.cin % V == 0;
      const long total = (long)B * L.out_h * L.out_w * (vec ? L.d.cin / V : L.d.cin);
      const int grid = (int)std::min<long>(cdiv(total, 256), 148L * 32);
      if (vec)
        maxpool_kernel<T, V><<<grid, 256, 0, st>>>((const T*)src, (T*)dst, g);
      else
        maxpool_kernel<T, 1><<<grid, 256, 0, st>>>((const T*)src, (T*)dst, g);
      break;
    }
  }
  EE_CUDA(cudaGetLastError());
  return EE_OK;
}

template <typename T>
ee_status_t launch_head(ee_model* m, StagePlan& sp, const void* x, int B, int hw, const float* shift,
                        const int32_t* shift_cls, char* scratch, const ee_stage_in_t* in_ids, const ee_stage_out_t* out,
                        cudaStream_t st, bool timed, const float* gap_part = nullptr, int gap_g = 0) {
  const int C = sp.out_c, K = sp.n_classes;
  HeadLayout h = head_layout(m->max_batch, C, K);
  unsigned* cnt = (unsigned*)(scratch + h.off_cnt);
  float* gap = (float*)(scratch + h.off_gap);
  float* z = out->logits ? out->logits : (float*)(scratch + h.off_z);
  if constexpr (sizeof(T) == 2) {
    if (m->fused_head && hc_supported(C, K, x, sp.fc_w)) {
      DecideArgs da{shift, shift_cls, sp.threshold, sp.always_exit, out->conf, out->pred, out->exit_mask,
                    in_ids ? in_ids->ids : nullptr, out->survivor_idx, out->ids_out, out->n_surv_dev, nullptr, m->head_done + (&sp - m->stages.data())};
      EE_CUDA(hc_launch((const bf16*)x, hw, C, (const bf16*)sp.fc_w, sp.fc_b, B, K, z, da, st));
      if (timed) record(m, sp, st, "head_gap_fc_softmax_scan");
      return EE_OK;
    }
  }
  constexpr int V = Elem<T>::kVec;
  const bool vec = C % V == 0 && ((uintptr_t)x & 15) == 0;
  const int lanes = gap_lanes(hw);
  const int n_zero = m->max_batch + 1;   // the pooling kernel leaves the FC kernel's counters at zero
  bool pooled = false;
  if constexpr (sizeof(T) == 2) {
    // bf16 maps pool in row blocks (gap_blocks_kernel): over the block sums the last layer's epilogue left, or over the map
    const int sb = sp.gap_rev ? 1 : 0;
    if (gap_part) {
      const int nb = hw / gap_g, bl = gap_block_lanes(nb);
      EE_CUDA(launch_pdl(gap_blocks_kernel<float, 4, 1>, dim3(cdiv(C / 4, bl), B), dim3(kGapThreads), st, gap_part, nb, hw, C, bl, gap, cnt, n_zero, sb));
      pooled = true;
    } else if (vec) {
      const int G = gap_block_rows(hw), nb = hw / G, bl = gap_block_lanes(nb);
      const dim3 bgrid(cdiv(C / V, bl), B);
      auto go = [&](auto kernel) { return launch_pdl(kernel, bgrid, dim3(kGapThreads), st, (const T*)x, nb, hw, C, bl, gap, cnt, n_zero, sb); };
      switch (G) {
        case 32: EE_CUDA(go(gap_blocks_kernel<T, V, 32>)); break;
        case 16: EE_CUDA(go(gap_blocks_kernel<T, V, 16>)); break;
        case 8: EE_CUDA(go(gap_blocks_kernel<T, V, 8>)); break;
        case 4: EE_CUDA(go(gap_blocks_kernel<T, V, 4>)); break;
        case 2: EE_CUDA(go(gap_blocks_kernel<T, V, 2>)); break;
        default: EE_CUDA(go(gap_blocks_kernel<T, V, 1>)); break;
      }
      pooled = true;
    }
  }
  dim3 ggrid(cdiv(vec ? C / V : C, lanes), B);
  if (pooled) {
  } else if (vec)
    EE_CUDA(launch_pdl(gap_kernel<T, V>, ggrid, dim3(kGapThreads), st, (const T*)x, hw, C, lanes, gap, cnt, n_zero, sp.gap_rev ? 1 : 0));
  else
    EE_CUDA(launch_pdl(gap_kernel<T, 1>, ggrid, dim3(kGapThreads), st, (const T*)x, hw, C, lanes, gap, cnt, n_zero, sp.gap_rev ? 1 : 0));
  if (timed) record(m, sp, st, "head_gap");
  DecideArgs da{shift, shift_cls, sp.threshold, sp.always_exit, out->conf, out->pred, out->exit_mask,
                in_ids ? in_ids->ids : nullptr, out->survivor_idx, out->ids_out, out->n_surv_dev, cnt, cnt + m->max_batch};
  const int fs = fc_tile_samples(B);
  dim3 fgrid(cdiv(K, kFcClasses), cdiv(B, fs));
  const bool fal = C % V == 0 && ((uintptr_t)sp.fc_w & 15) == 0;
  auto fc_launch = [&](auto kernel) {
    return launch_pdl(kernel, fgrid, dim3(kFcThreads), st, (const float*)gap, (const T*)sp.fc_w, (const float*)sp.fc_b, B, C, K, z, da);
  };
  if (fs == 4)
    EE_CUDA(fal ? fc_launch(fc_kernel<T, true, 4>) : fc_launch(fc_kernel<T, false, 4>));
  else
    EE_CUDA(fal ? fc_launch(fc_kernel<T, true, 8>) : fc_launch(fc_kernel<T, false, 8>));
  if (timed) record(m, sp, st, "head_fc_softmax_scan");
  return EE_OK;
}

template <typename V>
ee_status_t gather_launch_t(const void* feat, size_t bytes_per_sample, const int32_t* idx, const int32_t* n_dev, int max_rows,
                            void* out, bool rev, cudaStream_t st) {
  const size_t vecs = bytes_per_sample / sizeof(V);
  dim3 grid(cdiv((long)vecs, kCopyThreads * kCopyUnroll), max_rows);
  gather_rows_kernel<V><<<grid, kCopyThreads, 0, st>>>((const V*)feat, vecs, idx, n_dev, (V*)out, rev ? 1 : 0);
  EE_CUDA(cudaGetLastError());
  return EE_OK;
}

// Widest vector that divides the row size and both base addresses.
int copy_width(size_t bytes_per_sample, const void* a, const void* b) {
  const uintptr_t bits = (uintptr_t)bytes_per_sample | (uintptr_t)a | (uintptr_t)b;
  return (bits & 15) == 0 ? 16 : (bits & 3) == 0 ? 4 : (bits & 1) == 0 ? 2 : 1;
}

ee_status_t gather_launch(const void* feat, size_t bytes_per_sample, const int32_t* idx, const int32_t* n_dev, int max_rows,
                          void* out, bool rev, cudaStream_t st) {
  if (max_rows <= 0 || bytes_per_sample == 0) return EE_OK;
  switch (copy_width(bytes_per_sample, feat, out)) {
    case 16: return gather_launch_t<uint4>(feat, bytes_per_sample, idx, n_dev, max_rows, out, rev, st);
    case 4: return gather_launch_t<uint32_t>(feat, bytes_per_sample, idx, n_dev, max_rows, out, rev, st);
    case 2: return gather_launch_t<uint16_t>(feat, bytes_per_sample, idx, n_dev, max_rows, out, rev, st);
    default: return gather_launch_t<uint8_t>(feat, bytes_per_sample, idx, n_dev, max_rows, out, rev, st);
  }
}

template <typename V>
ee_status_t append_launch_t(const void* src, void* dst, size_t bytes, const int32_t* ids_src, int32_t* ids_dst, int n_ids,
                            cudaStream_t st) {
  const size_t vecs = bytes / sizeof(V);
  const int grid = (int)std::min<size_t>((vecs + kCopyThreads - 1) / kCopyThreads, 148 * 16);
  append_rows_kernel<V><<<grid, kCopyThreads, 0, st>>>((const V*)src, (V*)dst, vecs, ids_src, ids_dst, n_ids);
  EE_CUDA(cudaGetLastError());
  return EE_OK;
}

// True when layer `l` of the stage absorbs its projection at batch B: no table entry sends either layer elsewhere.
bool proj_absorbed(const ee_model* m, const StagePlan& sp, int l, int B) {
  const LayerPlan& L = sp.layers[l];
  if (!m->proj_fusion || m->dtype != EE_BF16 || L.proj_from < 0) return false;
  const LayerPlan& P = sp.layers[L.proj_from];
  auto plain = [&](const LayerPlan& q) { return q.variant.empty() || q.variant[B] == (uint8_t)TCV_AUTO; };
  return plain(L) && plain(P) && L.tc.splits == 1 && P.tc.splits == 1 && tc_runs_persistent(m->tc, L.tc, B, m->proj_waves);
}

// True when the stage's last layer writes pooling partials at batch B: it runs on the persistent kernel.
bool gap_partials(const ee_model* m, const StagePlan& sp, int B) {
  if (!m->gap_fusion || m->dtype != EE_BF16 || sp.gap_g == 0 || (m->stage_kernel && !m->timing && !sp.segments.empty() && B <= m->stage_kernel_max_batch))
    return false;
  if (m->fused_head && hc_supported(sp.out_c, sp.n_classes, nullptr, sp.fc_w)) return false;   // that head pools by itself
  const LayerPlan& L = sp.layers[sp.out_layer];
  if (L.kind != KK_TC || L.tc.cin != L.d.cin || L.tc.gather || L.tc.halo) return false;
  if (!(L.variant.empty() || L.variant[B] == (uint8_t)TCV_AUTO)) return false;
  return proj_absorbed(m, sp, sp.out_layer, B) || tc_runs_persistent(m->tc, L.tc, B);
}

bool stage_kernel_active(const ee_model* m, const StagePlan& sp, int B) {
  return m->dtype == EE_BF16 && m->stage_kernel && !m->timing && !sp.segments.empty() && B <= m->stage_kernel_max_batch;
}

// One launch for a run of layers (positions seg.first .. seg.first + seg.n - 1 of the execution order).
ee_status_t launch_segment(ee_model* m, StagePlan& sp, const StagePlan::Segment& seg, const ee_stage_in_t* in, char* ws, int B,
                           cudaStream_t st) {
  static thread_local PairStageArgs args;
  args.n_layers = seg.n;
  for (int j = 0; j < seg.n; ++j) {
    const int i = sp.order[seg.first + j];
    const LayerPlan& L = sp.layers[i];
    const void* src = L.src_slot < 0 ? in->features : ws + sp.slot_off[L.src_slot];
    const void* res = L.res_slot == -2 ? nullptr : (L.res_slot == -1 ? in->features : ws + sp.slot_off[L.res_slot]);
    void* dst = ws + sp.slot_off[L.out_slot];
    // the residual operand is "late" when the layer right before this one in the same launch writes it
    bool res_late = false;
    if (res && j > 0 && L.d.residual_from >= 0) res_late = sp.order[seg.first + j - 1] == L.d.residual_from;
    ee_status_t s = pair_fill_layer(m->tc, L.tc, seg.bn, src, res, dst, B, L.scale_dev, L.bias_dev, (float*)(ws + sp.split_off), sp.split_bytes,
                                    m->pair_counters, res_late, &args, j);
    if (s != EE_OK) return s;
  }
  ee_status_t s = pair_launch_args(m->tc, args, seg.bn, m->err_flag, m->grid_bar, m->wait_cycles, st);
  if (s != EE_OK) return s;
  EE_CUDA(cudaGetLastError());
  return EE_OK;
}

// Everything one stage launches, in stream order (also the body of a captured graph).
ee_status_t enqueue_stage(ee_model* m, StagePlan& sp, const ee_stage_in_t* in, char* ws, const ee_stage_out_t* out, cudaStream_t st) {
  const int B = in->batch;
  sp.ev_used = 0;
  record(m, sp, st, "begin");
  // Timed runs go layer by layer in index order on one stream (so that the events bracket single kernels); otherwise
  // the layers run in execution order with the shortcut layers on the branch stream.
  // Measured on B200 (ResNet-50-shaped model): the overlap gains 8 us per pass at batch 1-4 and costs 6 us at batch 64,
  // where every kernel fills the machine by itself and the two cross-stream edges per shortcut are pure overhead.
  const bool mega = stage_kernel_active(m, sp, B);
  const bool par = m->branches && !m->timing && B <= kBranchMaxBatch && !mega;
  float* gpart = gap_partials(m, sp, B) ? (float*)(ws + sp.gapp_off) : nullptr;   // the last layer's epilogue pools in row blocks
  for (size_t k = 0; k < sp.layers.size(); ++k) {
    if (mega && sp.seg_at[k] >= 0) {
      ee_status_t s = launch_segment(m, sp, sp.segments[sp.seg_at[k]], in, ws, B, st);
      if (s != EE_OK) return s;
      k += sp.segments[sp.seg_at[k]].n - 1;
      continue;
    }
    const size_t i = m->timing ? k : (size_t)sp.order[k];
    const LayerPlan& L = sp.layers[i];
    if (L.fused_away) continue;   // the launch of the convolution before it pools as well
    if (L.proj_into >= 0 && !mega && proj_absorbed(m, sp, L.proj_into, B)) continue;   // computed inside the layer that adds it
    if (L.proj_from >= 0 && !mega && proj_absorbed(m, sp, (int)i, B)) {
      const LayerPlan& P = sp.layers[L.proj_from];
      const void* psrc = P.src_slot < 0 ? in->features : ws + sp.slot_off[P.src_slot];
      const void* lsrc = L.src_slot < 0 ? in->features : ws + sp.slot_off[L.src_slot];
      ee_status_t ps = tc_launch_proj(m->tc, L.tc, P.tc, lsrc, psrc, ws + sp.slot_off[L.out_slot], B, L.scale_dev, L.bias_dev, P.scale_dev,
                                      P.bias_dev, m->err_flag, st, (int)i == sp.out_layer ? gpart : nullptr, sp.gap_g);
      if (ps != EE_OK) return ps;
      record(m, sp, st, kKernelNames[L.kind]);
      continue;
    }
    const void* src = L.src_slot < 0 ? in->features : ws + sp.slot_off[L.src_slot];
    const void* res = L.res_slot == -2 ? nullptr : (L.res_slot == -1 ? in->features : ws + sp.slot_off[L.res_slot]);
    void* dst = ws + sp.slot_off[L.pool_next ? sp.layers[i + 1].out_slot : L.out_slot];
    float* partial = (float*)(ws + sp.split_off);
    cudaStream_t ls = st;
    if (par && L.side) {            // fork: everything enqueued so far (the producer of this layer's input) precedes it
      EE_CUDA(cudaEventRecord(L.ev_fork, st));
      EE_CUDA(cudaStreamWaitEvent(m->branch, L.ev_fork, 0));
      ls = m->branch;
    }
    if (par && L.wait_for >= 0) EE_CUDA(cudaStreamWaitEvent(st, sp.layers[L.wait_for].ev_done, 0));   // join
    ee_status_t s = m->dtype == EE_BF16 ? launch_layer<bf16>(m, L, src, res, dst, B, partial, sp.split_bytes, ls, L.pool_next,
                                                             (int)i == sp.out_layer ? gpart : nullptr, sp.gap_g)
                                        : launch_layer<float>(m, L, src, res, dst, B, partial, sp.split_bytes, ls);
    if (s != EE_OK) return s;
    if (par && L.side) EE_CUDA(cudaEventRecord(L.ev_done, m->branch));
    record(m, sp, st, kKernelNames[L.kind]);
  }
  const void* so = ws + sp.slot_off[sp.out_slot];
  const int hw = sp.out_h * sp.out_w;
  ee_status_t s = m->dtype == EE_BF16
                      ? launch_head<bf16>(m, sp, so, B, hw, in->logit_shift, in->shift_class, ws + sp.head_off, in, out, st, true, gpart, sp.gap_g)
                      : launch_head<float>(m, sp, so, B, hw, in->logit_shift, in->shift_class, ws + sp.head_off, in, out, st, true);
  if (s != EE_OK) return s;
  // B_exit goes to the host as soon as the decisions are taken: the copy runs on a side branch (also when the stage
  // is captured into a graph) while the survivors' features are gathered, and rejoins the stream behind the gather.
  const bool fork = out->n_surv_host && !sp.always_exit;
  if (fork) {
    EE_CUDA(cudaEventRecord(m->ev_fork, st));
    EE_CUDA(cudaStreamWaitEvent(m->side, m->ev_fork, 0));
    EE_CUDA(cudaMemcpyAsync(out->n_surv_host, out->n_surv_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, m->side));
    EE_CUDA(cudaEventRecord(m->ev_join, m->side));
  }
  if (!sp.always_exit) {
    s = gather_launch(so, (size_t)hw * sp.out_c * esize(m->dtype), out->survivor_idx, out->n_surv_dev, B, out->features_out, sp.gather_rev, st);
    if (s != EE_OK) return s;
    record(m, sp, st, "gather_survivors");
  }
  if (fork)
    EE_CUDA(cudaStreamWaitEvent(st, m->ev_join, 0));
  else if (out->n_surv_host)
    EE_CUDA(cudaMemcpyAsync(out->n_surv_host, out->n_surv_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  return EE_OK;
}

// Device-sized stage chain (Section III, steps 3-4: B_exit decides how many samples the next subnet processes).  The
// whole chain from `first` on is ONE graph: the first stage at its batch, and for every later stage a switch node with one
// body per possible survivor count (body b = that stage captured at batch b; count 0 = nothing).  A one-thread kernel in
// front of each switch reads the survivor count the stage before left in device memory and sets the switch: the device
// sizes its own next launch, the host only reads the counts that still travel to its pinned words.
__global__ void chain_select_kernel(cudaGraphConditionalHandle handle, const int32_t* n_surv) {
  const int32_t n = *n_surv;
  cudaGraphSetConditional(handle, n > 0 ? (unsigned)n : 0u);
}

bool same_chain(const ee_model::ChainGraph& c, int first, const ee_stage_in_t* in, void* ws, const ee_stage_out_t* outs, int n_stages) {
  if (c.first != first || c.ws != ws || c.in.features != in->features || c.in.ids != in->ids || c.in.batch != in->batch ||
      c.in.logit_shift != in->logit_shift || c.in.shift_class != in->shift_class)
    return false;
  for (int s = first; s < n_stages; ++s) {
    StageCallKey a, b;
    a.out = c.outs[s];
    b.out = outs[s];
    a.in = b.in = *in;
    a.ws = b.ws = ws;
    if (!same_call(a, b)) return false;
  }
  return true;
}

ee_status_t enqueue_stage(ee_model* m, StagePlan& sp, const ee_stage_in_t* in, char* ws, const ee_stage_out_t* out, cudaStream_t st);

ee_status_t build_chain(ee_model* m, int first, const ee_stage_in_t* in, char* ws, const ee_stage_out_t* outs, ee_model::ChainGraph* out) {
  const int n_stages = (int)m->stages.size();
  cudaGraph_t g = nullptr;
  EE_CUDA(cudaGraphCreate(&g, 0));
  auto fail = [&](ee_status_t s) {
    cudaGraphDestroy(g);
    return s;
  };
  std::vector<cudaGraphNode_t> deps;
  for (int s = first; s < n_stages; ++s) {   // a stage that never runs leaves a zero count behind
    cudaMemsetParams mp = {};
    mp.dst = outs[s].n_surv_dev;
    mp.value = 0;
    mp.elementSize = 4;
    mp.width = 1;
    mp.height = 1;
    mp.pitch = 4;
    cudaGraphNode_t node;
    if (cudaGraphAddMemsetNode(&node, g, nullptr, 0, &mp) != cudaSuccess) return fail(EE_ERR_CUDA);
    deps.push_back(node);
  }
  // the first stage, at the caller's batch
  cudaGraph_t sub = nullptr;
  if (cudaStreamBeginCapture(m->cap, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return fail(EE_ERR_CUDA);
  ee_status_t es = enqueue_stage(m, m->stages[first], in, ws, &outs[first], m->cap);
  cudaError_t ce = cudaStreamEndCapture(m->cap, &sub);
  if (es != EE_OK || ce != cudaSuccess || !sub) {
    if (sub) cudaGraphDestroy(sub);
    return fail(es != EE_OK ? es : EE_ERR_CUDA);
  }
  cudaGraphNode_t prev;
  ce = cudaGraphAddChildGraphNode(&prev, g, deps.data(), deps.size(), sub);
  cudaGraphDestroy(sub);
  if (ce != cudaSuccess) return fail(EE_ERR_CUDA);
  for (int s = first + 1; s < n_stages; ++s) {
    cudaGraphConditionalHandle handle;
    if (cudaGraphConditionalHandleCreate(&handle, g, 0, cudaGraphCondAssignDefault) != cudaSuccess) return fail(EE_ERR_CUDA);
    const int32_t* count = outs[s - 1].n_surv_dev;
    void* kargs[2] = {(void*)&handle, (void*)&count};
    cudaKernelNodeParams kp = {};
    kp.func = (void*)chain_select_kernel;
    kp.gridDim = dim3(1);
    kp.blockDim = dim3(1);
    kp.kernelParams = kargs;
    cudaGraphNode_t sel;
    if (cudaGraphAddKernelNode(&sel, g, &prev, 1, &kp) != cudaSuccess) return fail(EE_ERR_CUDA);
    cudaGraphNodeParams np = {};
    np.type = cudaGraphNodeTypeConditional;
    np.conditional.handle = handle;
    np.conditional.type = cudaGraphCondTypeSwitch;
    np.conditional.size = (unsigned)in->batch + 1;
    cudaGraphNode_t cond;
    if (cudaGraphAddNode(&cond, g, &sel, 1, &np) != cudaSuccess) return fail(EE_ERR_CUDA);
    for (int b = 1; b <= in->batch; ++b) {   // body b: this stage on b survivors of the stage before
      ee_stage_in_t cur = {};
      cur.features = outs[s - 1].features_out;
      cur.ids = (in->ids && outs[s - 1].ids_out) ? outs[s - 1].ids_out : nullptr;
      cur.batch = b;
      cudaGraph_t body = np.conditional.phGraph_out[b];
      if (cudaStreamBeginCaptureToGraph(m->cap, body, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return fail(EE_ERR_CUDA);
      es = enqueue_stage(m, m->stages[s], &cur, ws, &outs[s], m->cap);
      cudaGraph_t ended = nullptr;
      ce = cudaStreamEndCapture(m->cap, &ended);
      if (es != EE_OK || ce != cudaSuccess) return fail(es != EE_OK ? es : EE_ERR_CUDA);
    }
    prev = cond;
  }
  cudaGraphExec_t exec = nullptr;
  if (cudaGraphInstantiate(&exec, g, 0) != cudaSuccess) {
    g_cuda_err = std::string("device-sized stage chain: graph instantiation failed: ") + cudaGetErrorString(cudaGetLastError());
    return fail(EE_ERR_CUDA);
  }
  out->first = first;
  out->in = *in;
  out->ws = ws;
  out->outs.assign(outs, outs + n_stages);
  out->graph = g;
  out->exec = exec;
  return EE_OK;
}

void drop_chains(ee_model* m) {   // whole-chain graphs hold the kernel choices they were captured with
  for (auto& c : m->chains) {
    cudaGraphExecDestroy(c.exec);
    cudaGraphDestroy(c.graph);
  }
  m->chains.clear();
}

// The GPU that is current must be the one the model lives on: kernels launched elsewhere would dereference this
// model's weights from another device.
bool on_model_device(const ee_model* m) {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess && dev == m->device;
}

bool valid_out(const ee_stage_out_t* o, bool need_feat) {
  return o && o->exit_mask && o->survivor_idx && o->n_surv_dev && (!need_feat || o->features_out);
}

}  // namespace

extern "C" {

const char* ee_status_string(ee_status_t s) {
  switch (s) {
    case EE_OK: return "ok";
    case EE_ERR_INVALID_ARG: return "invalid argument";
    case EE_ERR_SHAPE: return "layer shapes do not chain";
    case EE_ERR_CAPACITY: return "batch or workspace capacity exceeded";
    case EE_ERR_STAGE: return "stage index out of range";
    case EE_ERR_UNSUPPORTED: return "unsupported layer geometry";
    case EE_ERR_CUDA: return "CUDA error";
    case EE_ERR_TIMEOUT: return "device-side wait timed out";
    case EE_ERR_INTERNAL: return "internal error";
  }
  return "unknown status";
}

const char* ee_last_cuda_error(void) { return g_cuda_err.c_str(); }

ee_status_t ee_model_destroy(ee_model_t* m) {
  if (!m) return EE_ERR_INVALID_ARG;
  for (auto& sp : m->stages) {
    for (auto e : sp.ev) cudaEventDestroy(e);
    for (auto& g : sp.graphs) cudaGraphExecDestroy(g.exec);
    for (auto e : sp.retired) cudaGraphExecDestroy(e);
  }
  for (void* p : m->owned) cudaFree(p);
  if (m->ev_fork) cudaEventDestroy(m->ev_fork);
  if (m->ev_join) cudaEventDestroy(m->ev_join);
  if (m->side) cudaStreamDestroy(m->side);
  if (m->branch) cudaStreamDestroy(m->branch);
  if (m->cap) cudaStreamDestroy(m->cap);
  for (auto& c : m->chains) {
    cudaGraphExecDestroy(c.exec);
    cudaGraphDestroy(c.graph);
  }
  for (auto& sp : m->stages)
    for (auto& L : sp.layers) {
      if (L.ev_fork) cudaEventDestroy(L.ev_fork);
      if (L.ev_done) cudaEventDestroy(L.ev_done);
    }
  delete m;
  return EE_OK;
}

ee_status_t ee_model_create(const ee_model_desc_t* desc, void* cuda_stream, ee_model_t** out) {
  if (!desc || !out || !desc->stages || desc->n_stages < 1 || desc->max_batch < 1 || desc->in_h < 1 || desc->in_w < 1 ||
      desc->in_c < 1 || (desc->dtype != EE_F32 && desc->dtype != EE_BF16))
    return EE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  ee_model* m = new (std::nothrow) ee_model();
  if (!m) return EE_ERR_INTERNAL;
  m->dtype = desc->dtype;
  m->in_h = desc->in_h;
  m->in_w = desc->in_w;
  m->in_c = desc->in_c;
  m->max_batch = desc->max_batch;
  if (cudaGetDevice(&m->device) != cudaSuccess) {
    delete m;
    return EE_ERR_CUDA;
  }
  const size_t es = esize(desc->dtype);
  const int ondev = desc->weights_on_device;
  ee_status_t rc = EE_OK;
  auto fail = [&](ee_status_t s) {
    cudaStreamSynchronize(st);
    ee_model_destroy(m);
    return s;
  };
  {
    void* p = nullptr;
    if (cudaMalloc(&p, 256) != cudaSuccess) return fail(EE_ERR_CUDA);
    m->owned.push_back(p);
    m->err_flag = (int*)p;
    if (cudaMemsetAsync(p, 0, 256, st) != cudaSuccess) return fail(EE_ERR_CUDA);
  }
  if (cudaStreamCreateWithFlags(&m->cap, cudaStreamNonBlocking) != cudaSuccess ||
      cudaStreamCreateWithFlags(&m->branch, cudaStreamNonBlocking) != cudaSuccess ||
      cudaStreamCreateWithFlags(&m->side, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&m->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&m->ev_join, cudaEventDisableTiming) != cudaSuccess)
    return fail(EE_ERR_CUDA);
  rc = tc_context_init(m->tc);
  if (rc == EE_OK) rc = stem_context_init();
  if (rc == EE_OK) rc = halo_context_init();
  if (rc == EE_OK) rc = pair_context_init();
  if (rc == EE_OK) rc = dw_context_init();
  if (rc == EE_OK && hc_context_init() != cudaSuccess) rc = EE_ERR_CUDA;
  if (rc != EE_OK) return fail(rc);

  int h = desc->in_h, w = desc->in_w, c = desc->in_c;
  bool in_rev = false;   // direction in which the stage input was last walked (by the gather of the stage before)
  m->stages.resize(desc->n_stages);
  for (int s = 0; s < desc->n_stages; ++s) {
    const ee_stage_desc_t& sd = desc->stages[s];
    StagePlan& sp = m->stages[s];
    if (sd.n_layers < 1 || !sd.layers || sd.n_classes < 1 || !sd.fc_weight) return fail(EE_ERR_INVALID_ARG);
    const int out_layer = sd.out_layer < 0 ? sd.n_layers - 1 : sd.out_layer;
    if (out_layer >= sd.n_layers) return fail(EE_ERR_INVALID_ARG);
    sp.in_h = h;
    sp.in_w = w;
    sp.in_c = c;
    sp.layers.resize(sd.n_layers);
    std::vector<int> oh(sd.n_layers), ow(sd.n_layers), oc(sd.n_layers), last_use(sd.n_layers, -1);
    // shapes and liveness
    for (int i = 0; i < sd.n_layers; ++i) {
      const ee_layer_desc_t& d = sd.layers[i];
      LayerPlan& L = sp.layers[i];
      L.d = d;
      if (d.pad_w < EE_PAD_W_SAME) return fail(EE_ERR_INVALID_ARG);
      if (L.d.pad_w == EE_PAD_W_SAME) L.d.pad_w = d.pad;              // from here on pad = rows, pad_w = columns
      if (d.op != EE_OP_CONV && L.d.pad_w != d.pad) return fail(EE_ERR_UNSUPPORTED);
      if (d.op < EE_OP_CONV || d.op > EE_OP_MAXPOOL || d.kh < 1 || d.kw < 1 || d.stride < 1 || d.pad < 0 || d.cin < 1 ||
          d.cout < 1 || d.act < EE_ACT_NONE || d.act > EE_ACT_RELU6 || d.input_from < EE_FROM_STAGE_INPUT ||
          d.input_from >= i || d.residual_from < EE_FROM_STAGE_INPUT || d.residual_from >= i)
        return fail(EE_ERR_INVALID_ARG);
      if (d.op != EE_OP_MAXPOOL && !d.weight) return fail(EE_ERR_INVALID_ARG);
      int ih, iw, ic, src = d.input_from;
      if (src == EE_FROM_STAGE_INPUT || (src == EE_FROM_PREV && i == 0)) {
        ih = h, iw = w, ic = c, src = -1;
      } else {
        if (src == EE_FROM_PREV) src = i - 1;
        ih = oh[src], iw = ow[src], ic = oc[src];
        last_use[src] = i;
      }
      if (ic != d.cin) return fail(EE_ERR_SHAPE);
      if ((d.op == EE_OP_DWCONV || d.op == EE_OP_MAXPOOL) && d.cin != d.cout) return fail(EE_ERR_SHAPE);
      L.in_h = ih;
      L.in_w = iw;
      L.out_h = (ih + 2 * d.pad - d.kh) / d.stride + 1;
      L.out_w = (iw + 2 * L.d.pad_w - d.kw) / d.stride + 1;
      if (ih + 2 * d.pad < d.kh || iw + 2 * L.d.pad_w < d.kw || L.out_h < 1 || L.out_w < 1) return fail(EE_ERR_SHAPE);
      oh[i] = L.out_h, ow[i] = L.out_w, oc[i] = d.cout;
      L.src_slot = src;  // layer index for now; mapped to slots below
      int rs = d.residual_from;
      if (rs == EE_NO_RESIDUAL) {
        L.res_slot = -2;
      } else {
        if (d.op != EE_OP_CONV) return fail(EE_ERR_UNSUPPORTED);
        int rh, rw, rcn;
        if (rs == EE_FROM_STAGE_INPUT) {
          rh = h, rw = w, rcn = c;
          L.res_slot = -1;
        } else {
          rh = oh[rs], rw = ow[rs], rcn = oc[rs];
          L.res_slot = rs;
          last_use[rs] = i;
        }
        if (rh != L.out_h || rw != L.out_w || rcn != d.cout) return fail(EE_ERR_SHAPE);
      }
      if (d.op != EE_OP_MAXPOOL) {
        const int cpg = d.op == EE_OP_DWCONV ? 1 : d.cin;
        sp.flops_per_sample += 2.0 * L.out_h * L.out_w * d.cout * (double)(d.kh * d.kw * cpg);
      }
    }
    // Branch layers: a convolution whose output is used once, as a residual operand, and whose own input was ready
    // some layers earlier (the projection shortcut of a block) is hoisted in the execution order to right behind
    // the producer of its input, and runs on the branch stream beside the layers in between.
    const int n = sd.n_layers;
    std::vector<int> src_of(n), n_in_use(n, 0), n_res_use(n, 0), res_user(n, -1);
    for (int i = 0; i < n; ++i) {
      src_of[i] = sp.layers[i].src_slot;   // still a layer index here (-1 = stage input)
      if (src_of[i] >= 0) ++n_in_use[src_of[i]];
      const int r = sp.layers[i].res_slot;
      if (r >= 0) {
        ++n_res_use[r];
        res_user[r] = i;
      }
    }
    for (int i = 0; i < n; ++i) {
      LayerPlan& L = sp.layers[i];
      L.side = L.d.op == EE_OP_CONV && L.res_slot == -2 && i != out_layer && n_in_use[i] == 0 && n_res_use[i] == 1 &&
               src_of[i] < i - 1 && (src_of[i] < 0 || !sp.layers[src_of[i]].side);
      if (L.side) sp.layers[res_user[i]].wait_for = i;
    }
    sp.order.clear();
    for (int i = 0; i < n; ++i)
      if (sp.layers[i].side && src_of[i] < 0) sp.order.push_back(i);
    for (int i = 0; i < n; ++i) {
      if (sp.layers[i].side) continue;
      sp.order.push_back(i);
      for (int j = i + 2; j < n; ++j)
        if (sp.layers[j].side && src_of[j] == i) sp.order.push_back(j);
    }
    std::vector<int> pos(n);
    for (int k = 0; k < n; ++k) pos[sp.order[k]] = k;
    // liveness in execution order: last position at which a tensor is read
    std::vector<int> last_pos(n, -1);
    for (int i = 0; i < n; ++i) {
      if (src_of[i] >= 0) last_pos[src_of[i]] = std::max(last_pos[src_of[i]], pos[i]);
      if (sp.layers[i].res_slot >= 0) last_pos[sp.layers[i].res_slot] = std::max(last_pos[sp.layers[i].res_slot], pos[i]);
    }
    // a branch layer is only known to have finished (reading its input too) where its consumer joins it
    for (int i = 0; i < n; ++i)
      if (sp.layers[i].side && src_of[i] >= 0) last_pos[src_of[i]] = std::max(last_pos[src_of[i]], pos[res_user[i]]);
    last_pos[out_layer] = n + 1;
    (void)last_use;
    // slot assignment: a slot is reused once every consumer of its tensor has run
    std::vector<size_t> slot_bps;   // bytes per sample of each slot
    std::vector<int> slot_free_at;  // execution position from which the slot is free
    std::vector<int> slot_of(sd.n_layers);
    for (int k = 0; k < n; ++k) {
      const int i = sp.order[k];
      const size_t need = align_up((size_t)oh[i] * ow[i] * oc[i] * es, 256);
      int pick = -1;
      for (size_t q = 0; q < slot_bps.size(); ++q)
        if (slot_free_at[q] <= k && (pick < 0 || slot_bps[q] > slot_bps[pick])) pick = (int)q;
      if (pick < 0) {
        slot_bps.push_back(need);
        slot_free_at.push_back(0);
        pick = (int)slot_bps.size() - 1;
      }
      if (slot_bps[pick] < need) slot_bps[pick] = need;
      // the slot stays busy until after the last consumer; a never-read tensor frees at once
      slot_free_at[pick] = last_pos[i] < 0 ? k + 1 : last_pos[i] + 1;
      slot_of[i] = pick;
    }
    for (int i = 0; i < n; ++i)
      if (sp.layers[i].side) {
        LayerPlan& L = sp.layers[i];
        if (cudaEventCreateWithFlags(&L.ev_fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&L.ev_done, cudaEventDisableTiming) != cudaSuccess)
          return fail(EE_ERR_CUDA);
      }
    size_t off = 0;
    sp.slot_off.resize(slot_bps.size());
    for (size_t k = 0; k < slot_bps.size(); ++k) {
      sp.slot_off[k] = off;
      off += align_up(slot_bps[k] * (size_t)desc->max_batch, 1024);
    }
    for (int i = 0; i < sd.n_layers; ++i) {
      LayerPlan& L = sp.layers[i];
      L.out_slot = slot_of[i];
      if (L.src_slot >= 0) L.src_slot = slot_of[L.src_slot];
      if (L.res_slot >= 0) L.res_slot = slot_of[L.res_slot];
    }
    sp.out_slot = slot_of[out_layer];
    sp.out_layer = out_layer;
    sp.out_h = oh[out_layer];
    sp.out_w = ow[out_layer];
    sp.out_c = oc[out_layer];
    {
      const int g = gap_block_rows(sp.out_h * sp.out_w);
      sp.gap_g = desc->dtype == EE_BF16 && g >= 16 && sp.out_c % 8 == 0 ? g : 0;
    }
    HeadLayout hl = head_layout(desc->max_batch, sp.out_c, sd.n_classes);
    sp.head_off = align_up(off, 1024);
    sp.head_bytes = hl.bytes;
    sp.ws_bytes = sp.head_off + hl.bytes;   // the split-K region is added once the layers are planned
    sp.n_classes = sd.n_classes;
    sp.threshold = sd.threshold;
    sp.always_exit = sd.always_exit;
    // uploads and kernel choice
    for (int i = 0; i < sd.n_layers; ++i) {
      LayerPlan& L = sp.layers[i];
      const ee_layer_desc_t& d = L.d;
      if (d.op == EE_OP_MAXPOOL) {
        L.kind = KK_POOL;
        continue;
      }
      const int cpg = d.op == EE_OP_DWCONV ? 1 : d.cin;
      const size_t wn = (size_t)d.cout * d.kh * d.kw * cpg;
      if ((rc = upload_bytes(m, d.weight, wn * es, ondev, st, &L.w_dev)) != EE_OK) return fail(rc);
      if ((rc = upload<float>(m, d.scale, d.cout, ondev, st, &L.scale_dev)) != EE_OK) return fail(rc);
      if ((rc = upload<float>(m, d.bias, d.cout, ondev, st, &L.bias_dev)) != EE_OK) return fail(rc);
      if (d.op == EE_OP_DWCONV) {
        L.kind = KK_DW;
      } else if (desc->dtype == EE_BF16 && tc_supported(d, L.in_h, L.in_w)) {
        L.kind = KK_TC;
        const int g = pixel_group(d, L.in_h * L.in_w);
        if (g > 1) {   // narrow 1x1 layer: g pixels per row, block-diagonal weights, scale / bias repeated per pixel
          void* wp = nullptr;
          float *sp2 = nullptr, *bp2 = nullptr;
          if (cudaMalloc(&wp, (size_t)g * d.cout * g * d.cin * 2) != cudaSuccess) return fail(EE_ERR_CUDA);
          m->owned.push_back(wp);
          pack_grouped_weights_kernel<<<cdiv((long)g * d.cout * g * d.cin, 256), 256, 0, st>>>((const bf16*)L.w_dev, (bf16*)wp, d.cout, d.cin, g);
          if (L.scale_dev) {
            if (cudaMalloc((void**)&sp2, (size_t)g * d.cout * 4) != cudaSuccess) return fail(EE_ERR_CUDA);
            m->owned.push_back(sp2);
            replicate_kernel<<<cdiv((long)g * d.cout, 256), 256, 0, st>>>(L.scale_dev, sp2, d.cout, g);
            L.scale_dev = sp2;
          }
          if (L.bias_dev) {
            if (cudaMalloc((void**)&bp2, (size_t)g * d.cout * 4) != cudaSuccess) return fail(EE_ERR_CUDA);
            m->owned.push_back(bp2);
            replicate_kernel<<<cdiv((long)g * d.cout, 256), 256, 0, st>>>(L.bias_dev, bp2, d.cout, g);
            L.bias_dev = bp2;
          }
          if (cudaGetLastError() != cudaSuccess) return fail(EE_ERR_CUDA);
          ee_layer_desc_t gd = d;
          gd.cin = g * d.cin, gd.cout = g * d.cout;
          const int rows = L.in_h * L.in_w / g;
          rc = tc_plan_layer(m->tc, gd, 1, rows, 1, rows, desc->max_batch, wp, &L.tc);
        } else {
          rc = tc_plan_layer(m->tc, d, L.in_h, L.in_w, L.out_h, L.out_w, desc->max_batch, L.w_dev, &L.tc);
        }
        if (rc != EE_OK) return fail(rc);
        L.tc.halo = halo_supported(d, L.in_w);
      } else if (desc->dtype == EE_BF16 && d.cout % 8 == 0 && d.kh * d.kw * d.cin <= 1024 && d.pad_w == d.pad) {
        // pixel rows are not 16-byte units (e.g. a 3-channel stem): explicit Toeplitz rows, then the tensor-core GEMM
        L.kind = KK_TC_GATHER;
        const bool stem7 = stem_supported(d, L.in_h, L.in_w, L.out_w) && d.residual_from == EE_NO_RESIDUAL;
        const int run = d.kw * d.cin;
        const int runp = cdiv(run, 8) * 8;
        const int kp = cdiv(d.kh * runp, kTcBK) * kTcBK;
        void* wp = nullptr;
        if (cudaMalloc(&wp, (size_t)d.cout * kp * 2) != cudaSuccess) return fail(EE_ERR_CUDA);
        m->owned.push_back(wp);
        if (stem7)
          pack_stem_weights_kernel<<<cdiv((long)d.cout * kp, 256), 256, 0, st>>>((const bf16*)L.w_dev, (bf16*)wp, d.cout);
        else
          pack_weights_kernel<<<cdiv((long)d.cout * kp, 256), 256, 0, st>>>((const bf16*)L.w_dev, (bf16*)wp, d.cout, d.kh, run, runp, kp);
        if (cudaGetLastError() != cudaSuccess) return fail(EE_ERR_CUDA);
        ee_layer_desc_t g = d;   // the GEMM view: a 1x1 layer over kp packed columns
        g.cin = kp, g.kh = g.kw = 1, g.stride = 1, g.pad = g.pad_w = 0;
        rc = tc_plan_layer(m->tc, g, L.out_h, L.out_w, L.out_h, L.out_w, desc->max_batch, wp, &L.tc);
        if (rc != EE_OK) return fail(rc);
        L.tc.gather = true;
        L.tc.stem7 = stem7;
        L.tc.splits = 1, L.tc.kb_per = kp / kTcBK;
        L.tc.g_h = L.in_h, L.tc.g_w = L.in_w, L.tc.g_cin = d.cin, L.tc.g_kh = d.kh, L.tc.g_kw = d.kw;
        L.tc.g_stride = d.stride, L.tc.g_pad = d.pad, L.tc.g_runp = runp;
      } else {
        L.kind = KK_SIMT;
      }
    }
    for (int i = 0; i + 1 < sd.n_layers; ++i) {
      LayerPlan& L = sp.layers[i];
      LayerPlan& P = sp.layers[i + 1];
      if (L.kind != KK_TC_GATHER || !L.tc.stem7 || !stem_pool_supported(P.d) || i == out_layer) continue;
      if (src_of[i + 1] != i || n_in_use[i] != 1 || n_res_use[i] != 0) continue;   // someone else reads the convolution's output
      if (L.src_slot >= 0 && L.src_slot == P.out_slot) continue;                  // the pooled tensor would overwrite the input
      L.pool_next = true;
      P.fused_away = true;
    }
    for (int i = 0; i < sd.n_layers; ++i) {
      LayerPlan& P = sp.layers[i];
      if (P.kind != KK_TC || P.tc.cin != P.d.cin || i == out_layer || n_in_use[i] != 0 || n_res_use[i] != 1 || P.res_slot != -2) continue;
      LayerPlan& L = sp.layers[res_user[i]];
      if (L.kind != KK_TC || L.tc.cin != L.d.cin || !tc_proj_supported(L.tc, P.tc)) continue;
      if (P.src_slot >= 0 && P.src_slot == L.out_slot) continue;   // the layer's output would overwrite the projection's input
      if (P.src_slot >= 0 && !P.side) continue;   // only a branch layer's input is kept alive until its consumer runs
      P.proj_into = res_user[i];
      L.proj_from = i;
    }
    // Layer runs for the multi-layer launch: consecutive positions of the execution order whose layers the CTA-pair kernel
    // covers with one tile width (256 columns if every layer has more than 128 filters, else 128).
    {
      const int nl = sd.n_layers;
      sp.seg_at.assign(nl, -1);
      auto ok_for = [&](int i, int variant) {
        const LayerPlan& L = sp.layers[i];
        return L.kind == KK_TC && L.tc.cin == L.d.cin && pair_supported(L.tc, variant);
      };
      int k = 0;
      while (k < nl) {
        if (!ok_for(sp.order[k], TCV_PAIR128)) {
          ++k;
          continue;
        }
        int e = k;
        bool all256 = true;
        while (e < nl && e - k < kPairMaxLayers && ok_for(sp.order[e], TCV_PAIR128)) {
          all256 = all256 && ok_for(sp.order[e], TCV_PAIR256);
          ++e;
        }
        if (e - k >= 2) {
          sp.seg_at[k] = (int)sp.segments.size();
          sp.segments.push_back({k, e - k, all256 ? 256 : 128});
        }
        k = e;
      }
    }
    // Walk directions.  Feature maps of a large batch exceed the L2, so a kernel that walks its input from the first
    // row finds the rows its producer wrote first already evicted, and evicts the newest ones before it reaches them.
    // Every kernel therefore walks opposite to the kernel that last touched its largest operand: it starts on the rows
    // that are still cached.  The order of the sums inside a tile does not depend on the direction.
    {
      std::vector<char> slot_rev(sp.slot_off.size(), 0);
      auto dir_of = [&](int slot) { return slot < 0 ? in_rev : slot_rev[slot] != 0; };
      for (int i = 0; i < sd.n_layers; ++i) {
        LayerPlan& L = sp.layers[i];
        const size_t in_sz = (size_t)L.in_h * L.in_w * L.d.cin, res_sz = L.res_slot == -2 ? 0 : (size_t)L.out_h * L.out_w * L.d.cout;
        const bool rev = L.kind != KK_SIMT && !(res_sz > in_sz ? dir_of(L.res_slot) : dir_of(L.src_slot));   // the CUDA-core kernel walks forward
        L.tc.rev = rev;
        if (L.src_slot < 0 || L.res_slot == -1) in_rev = rev;
        if (L.src_slot >= 0) slot_rev[L.src_slot] = rev;
        if (L.res_slot >= 0) slot_rev[L.res_slot] = rev;
        slot_rev[L.out_slot] = rev;
      }
      sp.gap_rev = !slot_rev[sp.out_slot];
      sp.gather_rev = !sp.gap_rev;
      in_rev = sp.gather_rev;
    }
    layout_stage_tail(m, sp);
    for (const LayerPlan& L : sp.layers)
      if (L.kind == KK_TC && !L.tc.gather && !L.tc.halo) m->pair_counter_words = std::max(m->pair_counter_words, pair_counter_words(L.tc, desc->max_batch));
    if ((rc = upload_bytes(m, sd.fc_weight, (size_t)sd.n_classes * sp.out_c * es, ondev, st, &sp.fc_w)) != EE_OK) return fail(rc);
    if ((rc = upload<float>(m, sd.fc_bias, sd.n_classes, ondev, st, &sp.fc_b)) != EE_OK) return fail(rc);
    h = sp.out_h, w = sp.out_w, c = sp.out_c;
  }
  {
    void* p = nullptr;
    if (cudaMalloc(&p, 256) != cudaSuccess) return fail(EE_ERR_CUDA);
    m->owned.push_back(p);
    m->grid_bar = (unsigned*)p;
    if (cudaMemsetAsync(p, 0, 256, st) != cudaSuccess) return fail(EE_ERR_CUDA);
  }
  {
    void* p = nullptr;
    if (cudaMalloc(&p, 256 + m->stages.size() * sizeof(unsigned)) != cudaSuccess) return fail(EE_ERR_CUDA);
    m->owned.push_back(p);
    m->head_done = (unsigned*)p;
    if (cudaMemsetAsync(p, 0, 256 + m->stages.size() * sizeof(unsigned), st) != cudaSuccess) return fail(EE_ERR_CUDA);
  }
  if (m->pair_counter_words) {
    void* p = nullptr;
    if (cudaMalloc(&p, m->pair_counter_words * sizeof(unsigned)) != cudaSuccess) return fail(EE_ERR_CUDA);
    m->owned.push_back(p);
    m->pair_counters = (unsigned*)p;
    if (cudaMemsetAsync(p, 0, m->pair_counter_words * sizeof(unsigned), st) != cudaSuccess) return fail(EE_ERR_CUDA);
  }
  if (cudaStreamSynchronize(st) != cudaSuccess) return fail(EE_ERR_CUDA);
  *out = m;
  return EE_OK;
}

ee_status_t ee_wait_count(const int32_t* n_surv_host, int32_t sentinel, double timeout_s, int32_t* value) {
  if (!n_surv_host || !value || timeout_s < 0) return EE_ERR_INVALID_ARG;
  const volatile int32_t* w = n_surv_host;
  const auto t0 = std::chrono::steady_clock::now();
  for (unsigned spin = 0;; ++spin) {
    const int32_t v = *w;
    if (v != sentinel) {
      *value = v;
      return EE_OK;
    }
#if defined(__x86_64__) || defined(__i386__)
    __builtin_ia32_pause();   // be kind to the sibling hardware thread while spinning
#elif defined(__aarch64__)
    asm volatile("yield" ::: "memory");
#endif
    if ((spin & 1023u) == 1023u && std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count() > timeout_s)
      return EE_ERR_TIMEOUT;
  }
}

ee_status_t ee_run_until_exit(ee_model_t* m, int first_stage, const ee_stage_in_t* in, void* workspace, size_t workspace_bytes,
                              const ee_stage_out_t* outs, int32_t* batch_per_stage, double timeout_s, void* cuda_stream) {
  if (!m || !in || !outs || timeout_s < 0) return EE_ERR_INVALID_ARG;
  const int n_stages = (int)m->stages.size();
  if (first_stage < 0 || first_stage >= n_stages) return EE_ERR_STAGE;
  for (int s = first_stage; s + 1 < n_stages; ++s)
    if (!outs[s].n_surv_host) return EE_ERR_INVALID_ARG;
  if (batch_per_stage)
    for (int s = 0; s < n_stages; ++s) batch_per_stage[s] = 0;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const bool legacy = st == nullptr || st == cudaStreamLegacy || st == cudaStreamPerThread;
  if (in->batch >= 1 && in->batch <= m->chain_max_batch && first_stage + 1 < n_stages && m->graphs && !m->timing && !legacy &&
      in->batch <= m->max_batch && in->features && workspace && !((uintptr_t)workspace & 255) && on_model_device(m)) {
    // Device-sized chain: one graph launch; the host then only collects the counts as they arrive.
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs == cudaStreamCaptureStatusNone) {
      size_t need = 0;
      for (int s = first_stage; s < n_stages; ++s) {
        need = std::max(need, m->stages[s].ws_bytes);
        if (!valid_out(&outs[s], true)) return EE_ERR_INVALID_ARG;
      }
      if (workspace_bytes < need) return EE_ERR_CAPACITY;
      ee_model::ChainGraph* cg = nullptr;
      for (auto& c : m->chains)
        if (same_chain(c, first_stage, in, workspace, outs, n_stages)) cg = &c;
      if (!cg) {
        ee_model::ChainGraph fresh;
        ee_status_t rc = build_chain(m, first_stage, in, (char*)workspace, outs, &fresh);
        if (rc != EE_OK) return rc;
        if (m->chains.size() >= 16) {   // bounded: the oldest chain goes once the stream has passed it
          cudaStreamSynchronize(st);
          cudaGraphExecDestroy(m->chains.front().exec);
          cudaGraphDestroy(m->chains.front().graph);
          m->chains.erase(m->chains.begin());
        }
        m->chains.push_back(std::move(fresh));
        cg = &m->chains.back();
      }
      for (int s = first_stage; s + 1 < n_stages; ++s) *(volatile int32_t*)outs[s].n_surv_host = -1;
      EE_CUDA(cudaGraphLaunch(cg->exec, st));
      int32_t n = in->batch;
      for (int s = first_stage; s < n_stages; ++s) {
        if (batch_per_stage) batch_per_stage[s] = n;
        if (s + 1 == n_stages) break;
        ee_status_t rc = ee_wait_count(outs[s].n_surv_host, -1, timeout_s, &n);
        if (rc != EE_OK) return rc;
        if (n <= 0) break;
      }
      return EE_OK;
    }
  }
  ee_stage_in_t cur = *in;
  for (int s = first_stage; s < n_stages; ++s) {
    const bool last = s + 1 == n_stages;
    if (!last) *(volatile int32_t*)outs[s].n_surv_host = -1;
    ee_status_t rc = ee_stage_run(m, s, &cur, workspace, workspace_bytes, &outs[s], cuda_stream);
    if (rc != EE_OK) return rc;
    if (batch_per_stage) batch_per_stage[s] = cur.batch;
    if (last) break;
    int32_t n = 0;
    if ((rc = ee_wait_count(outs[s].n_surv_host, -1, timeout_s, &n)) != EE_OK) return rc;
    if (n <= 0) break;
    cur.features = outs[s].features_out;
    cur.ids = (in->ids && outs[s].ids_out) ? outs[s].ids_out : nullptr;
    cur.batch = n;
    cur.logit_shift = nullptr;
    cur.shift_class = nullptr;
  }
  return EE_OK;
}

ee_status_t ee_model_query(const ee_model_t* m, int stage, ee_stage_info_t* out) {
  if (!m || !out) return EE_ERR_INVALID_ARG;
  if (stage < 0 || stage >= (int)m->stages.size()) return EE_ERR_STAGE;
  const StagePlan& sp = m->stages[stage];
  const size_t es = esize(m->dtype);
  out->in_h = sp.in_h, out->in_w = sp.in_w, out->in_c = sp.in_c;
  out->out_h = sp.out_h, out->out_w = sp.out_w, out->out_c = sp.out_c;
  out->in_bytes_per_sample = (size_t)sp.in_h * sp.in_w * sp.in_c * es;
  out->out_bytes_per_sample = (size_t)sp.out_h * sp.out_w * sp.out_c * es;
  out->workspace_bytes = sp.ws_bytes;
  out->n_layers = (int)sp.layers.size();
  out->flops_per_sample = sp.flops_per_sample;
  return EE_OK;
}

ee_status_t ee_stage_run(ee_model_t* m, int stage, const ee_stage_in_t* in, void* workspace, size_t workspace_bytes,
                         const ee_stage_out_t* out, void* cuda_stream) {
  if (!m || !in || !valid_out(out, true) || in->batch < 0 || !on_model_device(m)) return EE_ERR_INVALID_ARG;
  if (stage < 0 || stage >= (int)m->stages.size()) return EE_ERR_STAGE;
  if (in->logit_shift && !in->shift_class) return EE_ERR_INVALID_ARG;
  StagePlan& sp = m->stages[stage];
  const int B = in->batch;
  if (B > m->max_batch) return EE_ERR_CAPACITY;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (B == 0) {
    EE_CUDA(cudaMemsetAsync(out->n_surv_dev, 0, sizeof(int32_t), st));
    if (out->n_surv_host) EE_CUDA(cudaMemcpyAsync(out->n_surv_host, out->n_surv_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    return EE_OK;
  }
  if (!in->features || !workspace || ((uintptr_t)workspace & 255)) return EE_ERR_INVALID_ARG;
  if (workspace_bytes < sp.ws_bytes) return EE_ERR_CAPACITY;
  // Replay path: the whole stage (every layer, the head, the gather, the count copy) as one CUDA graph, captured the
  // first time this exact call (same buffers, same batch) is seen on a capturable stream.  It removes the host cost
  // of ~25 launches per stage and most of the launch latency between the small kernels of a small batch.
  const bool legacy = st == nullptr || st == cudaStreamLegacy || st == cudaStreamPerThread;
  if (m->graphs && !m->timing && !legacy) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs == cudaStreamCaptureStatusNone) {
      StageCallKey key;
      key.in = *in;
      key.out = *out;
      key.ws = workspace;
      for (auto& g : sp.graphs)
        if (same_call(g.key, key)) {
          EE_CUDA(cudaGraphLaunch(g.exec, st));
          return EE_OK;
        }
      if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
        ee_status_t es = enqueue_stage(m, sp, in, (char*)workspace, out, st);
        cudaGraph_t graph = nullptr;
        cudaError_t ce = cudaStreamEndCapture(st, &graph);
        cudaGraphExec_t exec = nullptr;
        if (es == EE_OK && ce == cudaSuccess && graph && cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess) {
          cudaGraphDestroy(graph);
          // Bounded cache, sized for a server that keeps two buffer sets and sees every batch size (2 * B_max
          // signatures per stage).  An evicted executable may still be running: it is parked and destroyed once the
          // stream has passed it.
          if (sp.graphs.size() >= (size_t)std::max(96, 2 * m->max_batch + 8)) {
            sp.retired.push_back(sp.graphs.front().exec);
            sp.graphs.erase(sp.graphs.begin());
            if (sp.retired.size() >= 32) {
              cudaStreamSynchronize(st);
              for (auto e : sp.retired) cudaGraphExecDestroy(e);
              sp.retired.clear();
            }
          }
          sp.graphs.push_back({key, exec});
          EE_CUDA(cudaGraphLaunch(exec, st));
          return EE_OK;
        }
        if (graph) cudaGraphDestroy(graph);
        // capture is not available here: plain launches from now on; ee_last_cuda_error() says why
        g_cuda_err = std::string("stage replay switched off, capture failed: ") + cudaGetErrorString(ce != cudaSuccess ? ce : cudaGetLastError());
        cudaGetLastError();
        m->graphs = false;
        if (es != EE_OK) return es;
      }
    }
  }
  return enqueue_stage(m, sp, in, (char*)workspace, out, st);
}

ee_status_t ee_layer_run(ee_model_t* m, int stage, int layer, const void* input, const void* residual, int batch, void* output,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!m || batch < 0 || !on_model_device(m)) return EE_ERR_INVALID_ARG;
  if (stage < 0 || stage >= (int)m->stages.size()) return EE_ERR_STAGE;
  StagePlan& sp = m->stages[stage];
  if (layer < 0 || layer >= (int)sp.layers.size()) return EE_ERR_STAGE;
  if (batch > m->max_batch) return EE_ERR_CAPACITY;
  if (batch == 0) return EE_OK;
  const LayerPlan& L = sp.layers[layer];
  const bool has_res = L.res_slot != -2;
  if (!input || !output || (has_res && !residual) || ((uintptr_t)input & 15) || ((uintptr_t)output & 15) || ((uintptr_t)residual & 15))
    return EE_ERR_INVALID_ARG;
  // the only scratch a layer may need: the split-K partial tiles of the pair kernel, at their place in the stage workspace
  float* partial = nullptr;
  size_t partial_bytes = 0;
  if (workspace && !((uintptr_t)workspace & 255) && workspace_bytes >= sp.split_off + sp.split_bytes) {
    partial = (float*)((char*)workspace + sp.split_off);
    partial_bytes = sp.split_bytes;
  }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  return m->dtype == EE_BF16 ? launch_layer<bf16>(m, L, input, has_res ? residual : nullptr, output, batch, partial, partial_bytes, st)
                             : launch_layer<float>(m, L, input, has_res ? residual : nullptr, output, batch, partial, partial_bytes, st);
}

ee_status_t ee_batch_refill(ee_model_t* m, int boundary, void* batch_feat, int32_t* batch_ids, int n_surv, const void* arr_feat,
                            const int32_t* arr_ids, int n_arr, int* n_accepted, int* n_merged, void* cuda_stream) {
  if (!m || !n_accepted || !n_merged || n_surv < 0 || n_arr < 0 || !on_model_device(m)) return EE_ERR_INVALID_ARG;
  if (boundary < 0 || boundary > (int)m->stages.size() - 1) return EE_ERR_STAGE;
  if (n_surv > m->max_batch) return EE_ERR_CAPACITY;
  if (n_arr > 0 && (!batch_feat || !arr_feat)) return EE_ERR_INVALID_ARG;
  const StagePlan& sp = m->stages[boundary];
  const size_t bps = (size_t)sp.in_h * sp.in_w * sp.in_c * esize(m->dtype);
  const int slack = m->max_batch - n_surv;            // B_slack = B_max - B_rem
  const int n_acc = n_arr < slack ? n_arr : slack;    // B_incr  = min(N_Q, B_slack)
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (n_acc > 0) {
    void* dst = (char*)batch_feat + bps * (size_t)n_surv;
    int32_t* ids_dst = batch_ids ? batch_ids + n_surv : nullptr;
    const size_t bytes = bps * (size_t)n_acc;
    ee_status_t s;
    switch (copy_width(bps, arr_feat, batch_feat)) {
      case 16: s = append_launch_t<uint4>(arr_feat, dst, bytes, arr_ids, ids_dst, n_acc, st); break;
      case 4: s = append_launch_t<uint32_t>(arr_feat, dst, bytes, arr_ids, ids_dst, n_acc, st); break;
      case 2: s = append_launch_t<uint16_t>(arr_feat, dst, bytes, arr_ids, ids_dst, n_acc, st); break;
      default: s = append_launch_t<uint8_t>(arr_feat, dst, bytes, arr_ids, ids_dst, n_acc, st); break;
    }
    if (s != EE_OK) return s;
  }
  *n_accepted = n_acc;
  *n_merged = n_surv + n_acc;                          // B_merged = B_rem + B_incr
  return EE_OK;
}

size_t ee_exit_head_scratch_bytes(const ee_model_t* m, int stage) {
  if (!m || stage < 0 || stage >= (int)m->stages.size()) return 0;
  return m->stages[stage].head_bytes;
}

ee_status_t ee_exit_head(ee_model_t* m, int stage, const void* x, int batch, int hw, const float* logit_shift,
                         const int32_t* shift_class, void* scratch, size_t scratch_bytes, const ee_stage_out_t* out,
                         void* cuda_stream) {
  if (!m || !valid_out(out, false) || batch < 0 || hw < 1 || !on_model_device(m)) return EE_ERR_INVALID_ARG;
  if (stage < 0 || stage >= (int)m->stages.size()) return EE_ERR_STAGE;
  if (logit_shift && !shift_class) return EE_ERR_INVALID_ARG;
  StagePlan& sp = m->stages[stage];
  if (batch > m->max_batch) return EE_ERR_CAPACITY;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (batch == 0) {
    EE_CUDA(cudaMemsetAsync(out->n_surv_dev, 0, sizeof(int32_t), st));
    return EE_OK;
  }
  if (!x || !scratch || ((uintptr_t)scratch & 255)) return EE_ERR_INVALID_ARG;
  HeadLayout hl = head_layout(m->max_batch, sp.out_c, sp.n_classes);
  if (scratch_bytes < hl.bytes) return EE_ERR_CAPACITY;
  return m->dtype == EE_BF16
             ? launch_head<bf16>(m, sp, x, batch, hw, logit_shift, shift_class, (char*)scratch, nullptr, out, st, false)
             : launch_head<float>(m, sp, x, batch, hw, logit_shift, shift_class, (char*)scratch, nullptr, out, st, false);
}

// Scratch of ee_exit_head_static: lives in the library image, so every GPU that loads the library holds these
// bytes until the process exits.  In host code this name is only a handle for the runtime, never a device address.
static __device__ __align__(256) unsigned char g_static_head_scratch[EE_STATIC_HEAD_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::atomic<void*> g_static_head_ptr[kMaxDevices];   // device address of the array, resolved once per device
}  // namespace

ee_status_t ee_exit_head_static(ee_model_t* m, int stage, const void* x, int batch, int hw, const float* logit_shift,
                                const int32_t* shift_class, const ee_stage_out_t* out, void* cuda_stream) {
  if (!m || !valid_out(out, false) || batch < 0 || hw < 1) return EE_ERR_INVALID_ARG;
  if (stage < 0 || stage >= (int)m->stages.size()) return EE_ERR_STAGE;
  if (logit_shift && !shift_class) return EE_ERR_INVALID_ARG;
  StagePlan& sp = m->stages[stage];
  if (batch > m->max_batch) return EE_ERR_CAPACITY;
  HeadLayout hl = head_layout(m->max_batch, sp.out_c, sp.n_classes);
  if (hl.bytes > (size_t)EE_STATIC_HEAD_SCRATCH_BYTES) {
    g_cuda_err = "ee_exit_head_static: this model/shape needs " + std::to_string(hl.bytes) + " scratch bytes, the built-in array holds " +
                 std::to_string((size_t)EE_STATIC_HEAD_SCRATCH_BYTES);
    return EE_ERR_CAPACITY;
  }
  if (!on_model_device(m)) return EE_ERR_INVALID_ARG;   // the array of the model's own GPU is the one to use
  const int dev = m->device;
  if (dev < 0 || dev >= kMaxDevices) return EE_ERR_UNSUPPORTED;
  void* resolved = g_static_head_ptr[dev].load(std::memory_order_acquire);
  if (!resolved) {  // first call on this device (the device is current): ask the runtime where the array lives
    EE_CUDA(cudaGetSymbolAddress(&resolved, g_static_head_scratch));
    if (!resolved) return EE_ERR_INTERNAL;
    g_static_head_ptr[dev].store(resolved, std::memory_order_release);   // every thread resolves the same address
  }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (batch == 0) {
    EE_CUDA(cudaMemsetAsync(out->n_surv_dev, 0, sizeof(int32_t), st));
    return EE_OK;
  }
  if (!x) return EE_ERR_INVALID_ARG;
  char* scratch = (char*)resolved;
  // the pooling kernel zeroes the counters the FC kernel needs; everything else in the array is overwritten before it is read
  return m->dtype == EE_BF16
             ? launch_head<bf16>(m, sp, x, batch, hw, logit_shift, shift_class, scratch, nullptr, out, st, false)
             : launch_head<float>(m, sp, x, batch, hw, logit_shift, shift_class, scratch, nullptr, out, st, false);
}

ee_status_t ee_gather_survivors(const void* feat, size_t bytes_per_sample, const int32_t* survivor_idx, const int32_t* n_surv_dev,
                                int max_rows, void* feat_out, void* cuda_stream) {
  if (!feat || !survivor_idx || !n_surv_dev || !feat_out || max_rows < 0) return EE_ERR_INVALID_ARG;
  return gather_launch(feat, bytes_per_sample, survivor_idx, n_surv_dev, max_rows, feat_out, false, (cudaStream_t)cuda_stream);
}

ee_status_t ee_model_set_graphs(ee_model_t* m, int enabled) {
  if (!m) return EE_ERR_INVALID_ARG;
  m->graphs = enabled != 0;
  return EE_OK;
}

int ee_model_head_launches(const ee_model_t* m, int stage) {
  if (!m || stage < 0 || stage >= (int)m->stages.size()) return 0;
  const StagePlan& sp = m->stages[stage];
  return m->dtype == EE_BF16 && m->fused_head && hc_supported(sp.out_c, sp.n_classes, nullptr, sp.fc_w) ? 1 : 2;
}

int ee_model_gap_partials(const ee_model_t* m, int stage, int batch) {
  if (!m || stage < 0 || stage >= (int)m->stages.size() || batch < 1 || batch > m->max_batch) return 0;
  return gap_partials(m, m->stages[stage], batch) ? m->stages[stage].gap_g : 0;
}

ee_status_t ee_model_set_gap_fusion(ee_model_t* m, int enabled) {
  if (!m) return EE_ERR_INVALID_ARG;
  m->gap_fusion = enabled != 0;
  drop_chains(m);
  for (auto& sp : m->stages) {
    for (auto& g : sp.graphs) sp.retired.push_back(g.exec);
    sp.graphs.clear();
  }
  return EE_OK;
}

ee_status_t ee_model_set_proj_fusion(ee_model_t* m, int enabled) {
  if (!m) return EE_ERR_INVALID_ARG;
  m->proj_fusion = enabled != 0;
  drop_chains(m);
  for (auto& sp : m->stages) {
    for (auto& g : sp.graphs) sp.retired.push_back(g.exec);
    sp.graphs.clear();
  }
  return EE_OK;
}

ee_status_t ee_model_set_fused_head(ee_model_t* m, int enabled) {
  if (!m) return EE_ERR_INVALID_ARG;
  m->fused_head = enabled != 0;
  drop_chains(m);
  for (auto& sp : m->stages) {
    for (auto& g : sp.graphs) sp.retired.push_back(g.exec);
    sp.graphs.clear();
  }
  return EE_OK;
}

ee_status_t ee_model_set_branches(ee_model_t* m, int enabled) {
  if (!m) return EE_ERR_INVALID_ARG;
  m->branches = enabled != 0;
  drop_chains(m);
  for (auto& sp : m->stages) {
    for (auto& g : sp.graphs) sp.retired.push_back(g.exec);
    sp.graphs.clear();
  }
  return EE_OK;
}

ee_status_t ee_model_set_stage_kernel(ee_model_t* m, int enabled, int max_batch) {
  if (!m || max_batch < 0) return EE_ERR_INVALID_ARG;
  m->stage_kernel = enabled != 0;
  m->stage_kernel_max_batch = max_batch == 0 ? (1 << 30) : max_batch;
  drop_chains(m);
  for (auto& sp : m->stages) {
    for (auto& g : sp.graphs) sp.retired.push_back(g.exec);
    sp.graphs.clear();
  }
  return EE_OK;
}

ee_status_t ee_model_set_chain(ee_model_t* m, int max_batch) {
  if (!m || max_batch < 0) return EE_ERR_INVALID_ARG;
  m->chain_max_batch = max_batch;
  return EE_OK;
}

ee_status_t ee_model_set_timing(ee_model_t* m, int enabled) {
  if (!m) return EE_ERR_INVALID_ARG;
  m->timing = enabled != 0;
  return EE_OK;
}

ee_status_t ee_model_get_timing(ee_model_t* m, int stage, int cap, float* ms, const char** names, int* n) {
  if (!m || !ms || !n || cap < 0) return EE_ERR_INVALID_ARG;
  if (stage < 0 || stage >= (int)m->stages.size()) return EE_ERR_STAGE;
  StagePlan& sp = m->stages[stage];
  *n = 0;
  if (sp.ev_used < 2) return EE_OK;
  EE_CUDA(cudaEventSynchronize(sp.ev[sp.ev_used - 1]));
  for (int i = 1; i < sp.ev_used && *n < cap; ++i) {
    float t = 0.f;
    EE_CUDA(cudaEventElapsedTime(&t, sp.ev[i - 1], sp.ev[i]));
    ms[*n] = t;
    if (names) names[*n] = sp.ev_names[i];
    ++*n;
  }
  return EE_OK;
}

ee_status_t ee_model_plan(const ee_model_t* m, int stage, int batch, int cap, ee_layer_plan_t* out, int* n) {
  if (!m || !out || !n || cap < 0 || batch < 0) return EE_ERR_INVALID_ARG;
  if (stage < 0 || stage >= (int)m->stages.size()) return EE_ERR_STAGE;
  const StagePlan& sp = m->stages[stage];
  const double es = (double)esize(m->dtype);
  *n = 0;
  for (size_t i = 0; i < sp.layers.size() && *n < cap; ++i) {
    const LayerPlan& L = sp.layers[i];
    ee_layer_plan_t& p = out[(*n)++];
    const int cpg = L.d.op == EE_OP_CONV ? L.d.cin : 1;
    p.kernel = kKernelNames[L.kind];
    p.m = batch * L.out_h * L.out_w;
    p.n = L.d.cout;
    p.k = L.d.kh * L.d.kw * cpg;
    p.flops = L.d.op == EE_OP_MAXPOOL ? 0.0 : 2.0 * p.m * (double)p.n * p.k;
    const double in_b = (double)batch * L.in_h * L.in_w * L.d.cin * es, out_b = (double)p.m * p.n * es;
    const double w_b = L.d.op == EE_OP_MAXPOOL ? 0.0 : (double)L.d.cout * p.k * es;
    p.bytes = in_b + out_b + w_b + (L.res_slot != -2 ? out_b : 0.0);
    p.launches = 1;
    if (L.pool_next) {   // the launch writes the pooled tensor instead of the convolution's output
      const LayerPlan& P = sp.layers[i + 1];
      p.bytes = in_b + w_b + (double)batch * P.out_h * P.out_w * P.d.cout * es;
    }
    if (L.fused_away) p.bytes = 0.0, p.launches = 0;   // done by the launch of the convolution before it
    if (L.proj_into >= 0 && !stage_kernel_active(m, sp, batch) && proj_absorbed(m, sp, L.proj_into, batch))
      p.bytes = in_b + w_b, p.launches = 0;            // its GEMM runs inside the layer that adds it; its output is never stored
    if (L.proj_from >= 0 && !stage_kernel_active(m, sp, batch) && proj_absorbed(m, sp, (int)i, batch)) p.bytes = in_b + out_b + w_b;
  }
  if (stage_kernel_active(m, sp, batch))   // a run of layers is one launch: its first layer carries it
    for (const auto& seg : sp.segments)
      for (int j = 1; j < seg.n; ++j)
        if (sp.order[seg.first + j] < *n) out[sp.order[seg.first + j]].launches = 0;
  return EE_OK;
}

ee_status_t ee_model_set_layer_variant(ee_model_t* m, int stage, int layer, int batch_lo, int batch_hi, int variant) {
  if (!m || variant < 0 || variant >= TCV_COUNT || batch_lo < 1 || batch_hi < batch_lo) return EE_ERR_INVALID_ARG;
  if (stage < 0 || stage >= (int)m->stages.size()) return EE_ERR_STAGE;
  StagePlan& sp = m->stages[stage];
  if (layer < 0 || layer >= (int)sp.layers.size()) return EE_ERR_STAGE;
  if (batch_hi > m->max_batch) return EE_ERR_CAPACITY;
  LayerPlan& L = sp.layers[layer];
  const bool ranges_v = variant == TCV_RANGES_CLUSTER || variant == TCV_RANGES_LOCAL;
  if (ranges_v && (L.kind != KK_TC || L.tc.gather || L.tc.halo)) return EE_ERR_UNSUPPORTED;
  if (variant != TCV_AUTO && !ranges_v && (L.kind != KK_TC || !pair_supported(L.tc, variant))) return EE_ERR_UNSUPPORTED;
  if (L.variant.empty()) L.variant.assign((size_t)m->max_batch + 1, (uint8_t)TCV_AUTO);
  for (int b = batch_lo; b <= batch_hi; ++b) L.variant[b] = (uint8_t)variant;
  for (auto& g : sp.graphs) cudaGraphExecDestroy(g.exec);   // captured stages hold the old choice
  sp.graphs.clear();
  drop_chains(m);
  return EE_OK;
}

ee_status_t ee_model_set_layer_splits(ee_model_t* m, int stage, int layer, int splits) {
  if (!m) return EE_ERR_INVALID_ARG;
  if (stage < 0 || stage >= (int)m->stages.size()) return EE_ERR_STAGE;
  StagePlan& sp = m->stages[stage];
  if (layer < 0 || layer >= (int)sp.layers.size()) return EE_ERR_STAGE;
  LayerPlan& L = sp.layers[layer];
  if (L.kind != KK_TC || L.tc.gather || L.tc.halo) return EE_ERR_UNSUPPORTED;
  TcLayer trial = L.tc;
  if (!tc_set_splits(trial, splits)) return EE_ERR_INVALID_ARG;
  if (std::max(pair_partial_bytes(trial, m->max_batch, 256), pair_partial_bytes(trial, m->max_batch, 128)) > ((size_t)256 << 20))
    return EE_ERR_CAPACITY;
  L.tc.splits = trial.splits, L.tc.kb_per = trial.kb_per;
  layout_stage_tail(m, sp);
  for (auto& g : sp.graphs) cudaGraphExecDestroy(g.exec);
  sp.graphs.clear();
  drop_chains(m);
  return EE_OK;
}

ee_status_t ee_model_get_layer_config(const ee_model_t* m, int stage, int layer, int batch, int* variant, int* splits, int* tensor_core) {
  if (!m || batch < 0) return EE_ERR_INVALID_ARG;
  if (stage < 0 || stage >= (int)m->stages.size()) return EE_ERR_STAGE;
  const StagePlan& sp = m->stages[stage];
  if (layer < 0 || layer >= (int)sp.layers.size()) return EE_ERR_STAGE;
  if (batch > m->max_batch) return EE_ERR_CAPACITY;
  const LayerPlan& L = sp.layers[layer];
  const bool tc = L.kind == KK_TC && !L.tc.gather && !L.tc.halo;
  if (variant) *variant = L.variant.empty() ? (int)TCV_AUTO : (int)L.variant[batch];
  if (splits) *splits = L.kind == KK_TC ? L.tc.splits : 1;
  if (tensor_core) *tensor_core = tc ? ((pair_supported(L.tc, TCV_PAIR256) ? 1 : 0) | (pair_supported(L.tc, TCV_PAIR128) ? 2 : 0)) : -1;
  return EE_OK;
}

ee_status_t ee_model_set_wait_limit(ee_model_t* m, long long cycles) {
  if (!m || cycles < 1) return EE_ERR_INVALID_ARG;
  m->wait_cycles = cycles;
  return EE_OK;
}

ee_status_t ee_model_selftest_wait(ee_model_t* m, long long limit_cycles, void* cuda_stream) {
  if (!m || limit_cycles < 1 || limit_cycles > 2000000000LL) return EE_ERR_INVALID_ARG;   // at most about a second
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int* end_word = m->err_flag + 1;   // second word of the model's 256-byte status block
  EE_CUDA(cudaMemsetAsync(end_word, 0, sizeof(int), st));
  wait_selftest_kernel<<<1, 32, 0, st>>>(m->err_flag, limit_cycles, end_word);
  EE_CUDA(cudaGetLastError());
  int reached = 0;
  EE_CUDA(cudaMemcpyAsync(&reached, end_word, sizeof(int), cudaMemcpyDeviceToHost, st));
  EE_CUDA(cudaStreamSynchronize(st));
  return reached == 1 ? EE_OK : EE_ERR_INTERNAL;   // the kernel must have returned through the give-up path
}

ee_status_t ee_model_check(ee_model_t* m, void* cuda_stream) {
  if (!m) return EE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int flag = 0;
  EE_CUDA(cudaMemcpyAsync(&flag, m->err_flag, sizeof(int), cudaMemcpyDeviceToHost, st));
  EE_CUDA(cudaStreamSynchronize(st));
  if (flag) {
    // a kernel that gave up may have left arrival counters of a split-K reduction behind
    if (m->pair_counters) EE_CUDA(cudaMemsetAsync(m->pair_counters, 0, m->pair_counter_words * sizeof(unsigned), st));
    if (m->grid_bar) EE_CUDA(cudaMemsetAsync(m->grid_bar, 0, 256, st));
    if (m->head_done) EE_CUDA(cudaMemsetAsync(m->head_done, 0, m->stages.size() * sizeof(unsigned), st));
    EE_CUDA(cudaMemsetAsync(m->err_flag, 0, sizeof(int), st));
    EE_CUDA(cudaStreamSynchronize(st));
    return EE_ERR_TIMEOUT;
  }
  return EE_OK;
}

}  // extern "C"
