/*
 * ee.h - C ABI of the early-exit CNN stage executor for NVIDIA B200 (sm_100a).
 *
 * The library runs an early-exit CNN one subnet ("stage") at a time on a batch whose size
 * changes at every exit: a stage's convolutions, its exit head, the threshold test, the
 * compaction of the samples that stay, and the refill of the batch with new samples before
 * the next stage.  This is the device-side work underneath the serving loop of the paper
 * "Fluid Batching" (Section III overview, steps 2-6; Section III-B; Algorithm 1): the
 * scheduler there calls "process until exit i", learns B_exit, and merges the remaining
 * B_rem samples with B_incr new ones.
 *
 * General rules
 *   - Plain C.  Every function returns an ee_status_t; results only through pointers.
 *     On an error return no output buffer has been written.
 *   - "DEVICE" pointers are CUDA device memory of the current device; "HOST" pointers are
 *     ordinary host memory unless stated to be pinned.  The library never frees or keeps a
 *     caller buffer beyond the call, except the stream-ordered use described per function.
 *   - All work is enqueued on the cuda_stream argument (a cudaStream_t passed as void*;
 *     NULL = the legacy default stream) and is asynchronous with respect to the host unless
 *     stated otherwise.  One stream per model handle at a time.
 *   - Activations are NHWC [B][H][W][C] in the model's dtype (float or bf16).  Convolution
 *     weights are [Cout][kh][kw][Cin/groups], FC weights [n_classes][C], same dtype.
 *     A convolution is executed as the product of the implicit Toeplitz matrix
 *     (M = B*Ho*Wo rows, K = kh*kw*Cin) with the K x Cout weight matrix (Section II-C);
 *     batching appends samples along the row dimension (Section III-A, R-batching).
 *   - Buffers are sized once for max_batch by the caller (Section III-B, Overhead: buffers are
 *     allocated at initialisation for the largest activation at B_max; no run-time allocation).
 *     No entry point below allocates device memory except ee_model_create.
 */
#ifndef EE_H_
#define EE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  EE_OK = 0,
  EE_ERR_INVALID_ARG = 1,  /* NULL where a pointer is required, negative size, bad enum   */
  EE_ERR_SHAPE = 2,        /* layer list does not chain (channel or spatial mismatch)      */
  EE_ERR_CAPACITY = 3,     /* batch > max_batch, workspace too small                       */
  EE_ERR_STAGE = 4,        /* stage / boundary index out of range                          */
  EE_ERR_UNSUPPORTED = 5,  /* geometry no kernel covers; only ever returned at create time */
  EE_ERR_CUDA = 6,         /* a CUDA runtime/driver call failed (see ee_last_cuda_error)   */
  EE_ERR_TIMEOUT = 7,      /* a bounded device-side wait ran out (reported by ee_model_check) */
  EE_ERR_INTERNAL = 8
} ee_status_t;

typedef enum { EE_F32 = 0, EE_BF16 = 1 } ee_dtype_t;
typedef enum { EE_OP_CONV = 0, EE_OP_DWCONV = 1, EE_OP_MAXPOOL = 2 } ee_op_t;
typedef enum { EE_ACT_NONE = 0, EE_ACT_RELU = 1, EE_ACT_RELU6 = 2 } ee_act_t;

/* Sources for ee_layer_desc_t.input_from / residual_from. */
#define EE_FROM_PREV (-1)         /* input_from: output of the previous layer (stage input for layer 0) */
#define EE_FROM_STAGE_INPUT (-2)  /* the stage's input tensor */
#define EE_NO_RESIDUAL (-1)       /* residual_from: no residual operand */
#define EE_PAD_W_SAME (-1)        /* pad_w: the columns are padded like the rows */

/* One layer of a stage.  y = act(scale[c] * conv(x, weight) + bias[c] (+ residual)), stored in
 * the model dtype with one round-to-nearest-even.  BN is folded into scale/bias by the caller.
 * EE_OP_DWCONV is a depthwise convolution (groups = cin = cout, weight [C][kh][kw][1]).
 * EE_OP_MAXPOOL takes the window maximum over in-range taps; weight/scale/bias are ignored. */
typedef struct {
  int op;             /* ee_op_t */
  int cin, cout, kh, kw, stride, pad;
  int act;            /* ee_act_t */
  int input_from;     /* EE_FROM_PREV, EE_FROM_STAGE_INPUT, or index of an earlier layer of this stage */
  int residual_from;  /* EE_NO_RESIDUAL, EE_FROM_STAGE_INPUT, or index of an earlier layer; same shape as y */
  const void* weight; /* HOST or DEVICE (see ee_model_desc_t.weights_on_device); copied at create */
  const float* scale; /* [cout] fp32, may be NULL (= 1) */
  const float* bias;  /* [cout] fp32, may be NULL (= 0) */
  int pad_w;          /* padding of the columns; EE_PAD_W_SAME (-1): `pad` pads rows and columns alike, otherwise `pad`
                         pads the rows only (filters that are not square, such as 1 x 7 and 7 x 1, pad along their own
                         axis); dense convolutions only */
} ee_layer_desc_t;

/* One stage = a subnet followed by its exit head (global average pool, one FC layer, softmax;
 * the largest softmax probability is the confidence: Section II-B; Section IV, Benchmarks).
 * A sample exits iff always_exit or confidence >= threshold (compared in fp32). */
typedef struct {
  int n_layers;
  const ee_layer_desc_t* layers;
  int out_layer;          /* layer whose output leaves the stage; -1 = last */
  int n_classes;
  const void* fc_weight;  /* [n_classes][C] model dtype */
  const float* fc_bias;   /* [n_classes] fp32, may be NULL */
  float threshold;
  int always_exit;        /* 1 for the final exit */
} ee_stage_desc_t;

typedef struct {
  int dtype;              /* ee_dtype_t: EE_F32 computes in fp32 FMA; EE_BF16 stores bf16, accumulates fp32 */
  int in_h, in_w, in_c;
  int n_stages;
  const ee_stage_desc_t* stages;
  int max_batch;          /* B_max */
  int weights_on_device;  /* 0: all weight/scale/bias pointers are HOST; 1: DEVICE */
} ee_model_desc_t;

typedef struct ee_model ee_model_t; /* opaque; owns its device copies of the weights */

typedef struct {
  int in_h, in_w, in_c, out_h, out_w, out_c;
  size_t in_bytes_per_sample, out_bytes_per_sample;
  size_t workspace_bytes; /* what ee_stage_run needs for this stage at max_batch */
  int n_layers;
  double flops_per_sample; /* 2*M*N*K summed over the stage's convolutions, for roofline reports */
} ee_stage_info_t;

/* Validates the description, copies and repacks the weights to the device, and plans each
 * layer's kernel.  Synchronous (returns after the uploads finished).  *out is set only on EE_OK.
 * Errors: INVALID_ARG, SHAPE (layers do not chain), UNSUPPORTED, CUDA. */
ee_status_t ee_model_create(const ee_model_desc_t* desc, void* cuda_stream, ee_model_t** out);

/* Frees everything the model owns.  The caller must have synchronised the streams it used. */
ee_status_t ee_model_destroy(ee_model_t* model);

/* Shapes and sizes of one stage.  Errors: INVALID_ARG, STAGE. */
ee_status_t ee_model_query(const ee_model_t* model, int stage, ee_stage_info_t* out);

/* Inputs of ee_stage_run.  All pointers DEVICE. */
typedef struct {
  const void* features;        /* [batch][in_h][in_w][in_c], model dtype */
  const int32_t* ids;          /* [batch] sample ids (samples finish out of order and are re-associated by id:
                                  Section III-B, Overhead); may be NULL */
  int batch;                   /* B_act, 0 <= batch <= max_batch */
  const float* logit_shift;    /* optional [batch]: added to logit shift_class[b] of sample b before the softmax */
  const int32_t* shift_class;  /* [batch], required iff logit_shift != NULL; entries outside [0, n_classes) are ignored */
} ee_stage_in_t;

/* Outputs of ee_stage_run.  Caller-owned DEVICE buffers sized for max_batch (any may be NULL
 * except features_out, exit_mask, survivor_idx and n_surv_dev). */
typedef struct {
  void* features_out;     /* [n_surv][out_h][out_w][out_c]: the survivors' stage output, compacted, order kept;
                             this is the next stage's input */
  float* conf;            /* [batch] softmax top-1 probability, input order */
  int32_t* pred;          /* [batch] argmax class (lowest index on ties), input order */
  float* logits;          /* [batch][n_classes] fp32, optional */
  uint8_t* exit_mask;     /* [batch] 1 = sample exits here */
  int32_t* survivor_idx;  /* first n_surv entries: ascending positions (in the input batch) of the survivors */
  int32_t* ids_out;       /* first n_surv entries: ids of the survivors (written iff ids given) */
  int32_t* n_surv_dev;    /* [1] B_rem = B_act - B_exit */
  int32_t* n_surv_host;   /* optional PINNED HOST [1]: receives the count by an async copy (the "B_exit is communicated
                             to the scheduler" step).  The copy is issued as soon as the exit decisions are taken,
                             beside the gather of the survivors' features, so the word is valid once the caller has
                             synchronised the stream, or earlier: see ee_wait_count */
} ee_stage_out_t;

/* Runs stage `stage` on a batch: every layer of the subnet (convolutions as implicit GEMM with the
 * bias/BN-fold/activation epilogue fused), the exit head, the threshold test, and the stable
 * compaction + gather of the survivors (Section III, steps 2-4; Algorithm 1 "ProcUntilExit" and
 * B_rem = B_act - B_exit).  `workspace` is DEVICE scratch of at least ee_stage_info_t.workspace_bytes,
 * 256-byte aligned; its contents are undefined afterwards.  features_out must not alias `features`
 * or the workspace.  batch == 0 is legal: only n_surv = 0 is written.
 * Errors: INVALID_ARG, STAGE, CAPACITY (batch > max_batch or workspace too small), CUDA. */
ee_status_t ee_stage_run(ee_model_t* model, int stage, const ee_stage_in_t* in, void* workspace,
                         size_t workspace_bytes, const ee_stage_out_t* out, void* cuda_stream);

/* Merges a halted batch with new samples that stand at the same stage boundary
 * (Section III-B, Preemption Mechanism; Algorithm 1: B_slack = B_max - B_rem,
 * B_incr = min(N_Q, B_slack), B_merged = B_rem + B_incr).  `boundary` 0 = model input,
 * i = output of stage i-1.  batch_feat / batch_ids (DEVICE, sized for max_batch) hold n_surv samples at
 * the front; the first n_accepted = min(n_arr, max_batch - n_surv) arrivals (DEVICE arr_feat / arr_ids) are
 * appended after them in order.  n_accepted and n_merged are HOST ints written before return; arrivals
 * that did not fit stay with the caller.  ids may be NULL on both sides.
 * Errors: INVALID_ARG, STAGE, CAPACITY (n_surv > max_batch), CUDA. */
ee_status_t ee_batch_refill(ee_model_t* model, int boundary, void* batch_feat, int32_t* batch_ids, int n_surv,
                            const void* arr_feat, const int32_t* arr_ids, int n_arr, int* n_accepted,
                            int* n_merged, void* cuda_stream);

/* One layer of a stage alone (the same kernel and launch configuration ee_stage_run uses for it): `input` is
 * the layer's input tensor [batch][in_h][in_w][cin], `residual` its residual operand [batch][out_h][out_w][cout]
 * (required iff the layer has one), `output` [batch][out_h][out_w][cout]; all DEVICE, model dtype, 16-byte aligned,
 * caller-owned.  `workspace` is reserved (no layer kernel needs scratch today; pass the stage workspace or NULL).  For per-layer parity checks and
 * micro-benchmarks.  Errors: INVALID_ARG, STAGE (stage or layer out of range), CAPACITY, CUDA. */
ee_status_t ee_layer_run(ee_model_t* model, int stage, int layer, const void* input, const void* residual, int batch,
                         void* output, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Exit head alone on a feature map (same kernels ee_stage_run uses): GAP, FC, softmax top-1,
 * threshold, and the stable scan that yields survivor_idx / n_surv (no feature gather).
 * x DEVICE [batch][hw][c] model dtype; `out` as in ee_stage_run with features_out ignored;
 * `scratch` DEVICE, at least ee_exit_head_scratch_bytes(model, stage) bytes, 256-byte aligned.
 * Errors: INVALID_ARG, STAGE, CAPACITY, CUDA. */
ee_status_t ee_exit_head(ee_model_t* model, int stage, const void* x, int batch, int hw,
                         const float* logit_shift, const int32_t* shift_class, void* scratch, size_t scratch_bytes,
                         const ee_stage_out_t* out, void* cuda_stream);
size_t ee_exit_head_scratch_bytes(const ee_model_t* model, int stage);

/* ee_exit_head without any caller scratch and without any allocation.  The paper has no counterpart: this is
 * a convenience of this library.  It is for callers that may not allocate device memory when they need an exit
 * decision: code living inside a host application that hands out all device memory at start-up and forbids
 * later cudaMalloc calls (inference-server plug-ins, engines running under a fixed memory budget), and latency-bound
 * serving threads, for which an allocation's implicit synchronisation and unpredictable duration are not
 * acceptable.  Same arguments, results and errors as ee_exit_head, minus `scratch`: the pooled vectors,
 * logits (when out->logits is NULL) and counters go to an array of EE_STATIC_HEAD_SCRATCH_BYTES bytes that is part of
 * the library image (each GPU that loads the library holds it until the process exits).
 *   - A model/shape whose head needs more than EE_STATIC_HEAD_SCRATCH_BYTES (what ee_exit_head_scratch_bytes reports
 *     for the stage) is refused with EE_ERR_CAPACITY and an explanatory ee_last_cuda_error() text.
 *   - The first call on a device resolves the array's device address; make that first call outside any stream
 *     capture.  As for every call, the calling thread's current device must be the one the model lives on
 *     (EE_ERR_INVALID_ARG otherwise: another GPU's copy of the array must not be paired with this model's weights).
 *   - No cudaMalloc / cudaFree or allocating library routine is called.
 *   - All calls, from every model and stream, share the one array and it keeps the previous call's contents; the call
 *     clears what has to start at zero.  Two calls whose kernels overlap on the GPU race on it: serialise them
 *     (same stream, or an event between streams). */
#define EE_STATIC_HEAD_SCRATCH_BYTES (8u << 20)
ee_status_t ee_exit_head_static(ee_model_t* model, int stage, const void* x, int batch, int hw,
                                const float* logit_shift, const int32_t* shift_class, const ee_stage_out_t* out,
                                void* cuda_stream);

/* Stable compaction + gather alone: feat_out[j] = feat[survivor_idx[j]] for j < *n_surv_dev
 * (both read from DEVICE memory, no host round trip).  Rows move as 16-byte vectors when bytes_per_sample
 * and both base addresses are multiples of 16, in narrower units otherwise.
 * Errors: INVALID_ARG, CUDA. */
ee_status_t ee_gather_survivors(const void* feat, size_t bytes_per_sample, const int32_t* survivor_idx,
                                const int32_t* n_surv_dev, int max_rows, void* feat_out, void* cuda_stream);

/* Stage replay.  On by default: the first ee_stage_run with a given signature (stage, every pointer of in/out, the
 * workspace, the batch) on a capturable stream (not the legacy default stream, not a stream the caller is already
 * capturing) records the stage's launches into a CUDA graph; later calls with the same signature replay it.  A server
 * that keeps its buffers (Section III-B, Overhead: buffers are allocated once at initialisation) therefore pays the
 * launch cost of a stage once per batch size.  Results are identical either way.  Disabled while per-layer timing is on.
 * Errors: INVALID_ARG. */
ee_status_t ee_model_set_graphs(ee_model_t* model, int enabled);

/* Projection shortcuts inside the layer that adds them.  On by default.  A 1x1 convolution without padding whose output
 * is read only as the residual operand of one later 1x1 layer (the projection shortcut of the first block of a stage)
 * is computed by that layer's launch (the persistent tensor-core kernel) into a second accumulator, provided both
 * layers have one K range and no table entry: the epilogue rounds
 * the projection to bf16 exactly as the projection layer would have stored it and adds it, so results are bit-identical
 * to the two launches, and the projection's output is neither written nor read back.  ee_model_plan reports such a
 * projection with 0 launches.  ee_layer_run always runs a layer alone.  Errors: INVALID_ARG. */
ee_status_t ee_model_set_proj_fusion(ee_model_t* model, int enabled);

/* Pooling partials from the last layer's epilogue.  On by default.  bf16 models pool a stage's output (Section II-B: the
 * exit head's global average) in blocks of G consecutive rows, G the largest power of two up to 32 that divides
 * height * width: pairwise tree inside a block, blocks in a fixed order.  When G is 32 or 16 and the stage's last layer
 * runs on the persistent tensor-core kernel at the batch at hand, that kernel's epilogue writes the block sums of the
 * tiles it stores (a warp holds 32 rows: one or two blocks) and the head pools those instead of reading the feature map
 * again; the logits are the same bits either way, and the same as ee_exit_head computes on the stored map.
 * ee_model_gap_partials returns G when ee_stage_run takes that route for (stage, batch), else 0.  Errors: INVALID_ARG. */
ee_status_t ee_model_set_gap_fusion(ee_model_t* model, int enabled);
int ee_model_gap_partials(const ee_model_t* model, int stage, int batch);

/* One-launch exit head.  Off by default.  For bf16 models whose head has C % 8 == 0, C <= 2048 and K <= 1024 (16-byte
 * aligned features and FC weights) global average pool, FC, softmax top-1, threshold and the survivor scan (Section II-B;
 * Section III-B steps 2-3) can run as one kernel of 8-CTA thread-block clusters, one cluster per tile of 1, 2 or 4
 * samples, that exchange the pooled vectors and the softmax partials through distributed shared memory.  Otherwise, and
 * for other shapes and fp32 models: a pooling kernel and an FC + decision kernel.  Both orders of summation are fixed by
 * the head's shape, so either way a sample's logits do not depend on its batch; between the two ways logits differ by
 * the fp32 rounding of differently grouped sums.  Measured on B200 the cluster kernel wins only on large maps at batch 1
 * (10 us against 14 us at 56x56x256): a cluster per sample tile leaves the pooling with one CTA per SM and eight SMs per
 * tile to pull the FC weights, where the two kernels spread both over the whole GPU (54 against 32 us at batch 64 on
 * 56x56x256, 25 against 20 us at batch 27 on 7x7x2048), hence the default.
 * Applies to ee_stage_run, ee_exit_head and ee_exit_head_static alike.  Errors: INVALID_ARG. */
ee_status_t ee_model_set_fused_head(ee_model_t* model, int enabled);
/* Kernels the exit head of `stage` launches on 16-byte aligned features: 1 (one-launch head) or 2; 0 for a bad argument. */
int ee_model_head_launches(const ee_model_t* model, int stage);

/* Branch execution.  On by default for batches of up to 32 samples: a layer whose output is only a residual operand of a later layer (the projection
 * shortcut of a residual block) runs on a stream of the model's own, beside the layers between its input and its
 * consumer, forked from and joined to the caller's stream by events (also inside captured stages).  Results are
 * identical either way: the layers and their kernels are the same, only their order in time changes.
 * Errors: INVALID_ARG. */
ee_status_t ee_model_set_branches(ee_model_t* model, int enabled);

/* Multi-layer launches.  Off by default: a run of consecutive layers that the CTA-pair kernel covers (dense convolutions
 * with more than 64 filters) can execute as ONE persistent kernel with a grid-wide barrier between layers in place of a
 * kernel boundary; the layers' arithmetic, K ranges and results are those of the per-layer kernels, bit for bit.
 * Measured on B200 the barrier (output stores complete, release, acquire on every SM, first activation tiles) costs more
 * than a kernel boundary under programmatic dependent launch at every batch size, hence the default.
 * `max_batch` > 0 restricts it to batches of at most that size (0 = no limit).  Per-layer timing switches it off.
 * Errors: INVALID_ARG. */
ee_status_t ee_model_set_stage_kernel(ee_model_t* model, int enabled, int max_batch);

/* Per-layer device timing.  When enabled, ee_stage_run brackets every kernel with CUDA events on the
 * stream it launches on.  ee_model_get_timing synchronises those events and writes, for the last run
 * of `stage`, up to `cap` entries: the layers that launch a kernel (ee_layer_plan_t.launches > 0) in order, then the
 * head and the gather kernels.
 * names[i] points at a static string.  Errors: INVALID_ARG, STAGE, CUDA. */
ee_status_t ee_model_set_timing(ee_model_t* model, int enabled);
ee_status_t ee_model_get_timing(ee_model_t* model, int stage, int cap, float* ms, const char** names, int* n);

/* Per-layer plan of a stage at a batch size: kernel family chosen, GEMM M/N/K, FLOPs and the
 * algorithmic bytes (inputs + outputs + weights, each once).  Up to `cap` entries. */
typedef struct {
  const char* kernel;
  int m, n, k;
  double flops, bytes;
  int launches; /* kernels this layer launches at this batch size; 0: an earlier layer's launch does its work (a layer
                 * inside a multi-layer launch; a 3x3 stride-2 pad-1 max-pool read only from the 7x7 stride-2 3-channel
                 * bf16 convolution right before it, which pools in its epilogue and never stores its own output) */
} ee_layer_plan_t;
ee_status_t ee_model_plan(const ee_model_t* model, int stage, int batch, int cap, ee_layer_plan_t* out, int* n);

/* Per-(layer, batch) kernel table.  The paper's NPU looks up, for every (layer, active batch size), how to map the batch
 * onto its array (Section III-A Eq. 1; Section III-C: an L x B_max table addressed by (l, B_act)) and fills the table
 * offline by an exhaustive search over the design space (Section III-D Eq. 2).  Here the table holds, for every
 * tensor-core layer and every batch size 1..max_batch, which kernel variant runs the layer:
 *   0  one-CTA tiles (128 x 128 or 128 x 64; one-tile, persistent or cluster split-K kernels chosen from the grid),
 *   1  CTA pairs, 256 x 256 tiles (tcgen05 cta_group::2, persistent (tile, K-range) units),
 *   2  CTA pairs, 256 x 128 tiles,
 *   3  one-CTA tiles, the layer's K ranges as a cluster of CTAs per tile (reduce-scatter over distributed shared memory),
 *   4  one-CTA tiles, the K ranges inside ONE CTA per tile, an accumulator in tensor memory per range (ranges x tile
 *      width <= 512 columns, else as 3); variant 0 picks 3 while tiles x ranges stays within 1.25 waves of SMs, else 4.
 * The number of K ranges of a layer (`splits`) is one value per layer for all batch sizes and all variants, and the
 * partial sums of the ranges are always added in ascending order, so a sample's result is bit-identical whichever
 * variant the table picks for the batch it rides in.  Both setters drop the stage's captured graphs.
 * ee_model_set_layer_splits may change ee_stage_info_t.workspace_bytes: query again before the next run.
 * ee_model_get_layer_config: tensor_core = -1 (not a tensor-core layer with a table), else a bit mask of the pair
 * variants the layer supports (bit 0: variant 1, bit 1: variant 2).  Errors: INVALID_ARG, STAGE, CAPACITY (batch range beyond max_batch; partial tiles of more than 256 MB),
 * UNSUPPORTED (the layer cannot run as that variant). */
ee_status_t ee_model_set_layer_variant(ee_model_t* model, int stage, int layer, int batch_lo, int batch_hi, int variant);
ee_status_t ee_model_set_layer_splits(ee_model_t* model, int stage, int layer, int splits);
ee_status_t ee_model_get_layer_config(const ee_model_t* model, int stage, int layer, int batch, int* variant, int* splits,
                                      int* tensor_core);

/* Limit, in SM clock cycles, of the bounded device-side waits (default about 2 s).  Errors: INVALID_ARG. */
ee_status_t ee_model_set_wait_limit(ee_model_t* model, long long cycles);

/* Self-test of the device-side time-out path (no counterpart in the paper; the kernels' waits on barriers are
 * bounded so that a fault of the pipeline shows up as an error code, never as a hung GPU).  Launches one thread that
 * waits, with the given limit in SM clock cycles (at most 2e9), on a barrier that nothing signals, and synchronises
 * the stream.  Returns EE_OK when the wait ran out and the kernel returned normally; afterwards ee_model_check
 * reports EE_ERR_TIMEOUT once (and clears it).  Errors: INVALID_ARG, CUDA, INTERNAL (the wait did not give up). */
ee_status_t ee_model_selftest_wait(ee_model_t* model, long long limit_cycles, void* cuda_stream);

/* Runs a batch from stage `first_stage` on until it is empty or the last stage has been launched: ee_stage_run for a
 * stage, the host's wait for its survivor count (the protocol of ee_wait_count on outs[s].n_surv_host, which must be
 * a pinned host word for every stage but the last), then the next stage on the survivors (features_out / ids_out of
 * the stage before).  This is Algorithm 1's "ProcUntilExit" chain without preemption, kept inside the library so that
 * a stage boundary costs one poll and one launch and no trip through the caller's language runtime.
 * `in` describes the batch at `first_stage`; its logit_shift applies to that stage only.  `outs` holds one
 * ee_stage_out_t per stage of the model, indexed by stage (entries below first_stage are ignored).
 * batch_per_stage (HOST, optional, n_stages ints) receives the batch every stage ran on, 0 for stages not reached.
 * The last stage is launched but not waited for: its results are ordered on the stream like any other call's.
 * Errors: those of ee_stage_run; INVALID_ARG when a needed n_surv_host is NULL; TIMEOUT when a count does not arrive
 * within `timeout_s` seconds. */
ee_status_t ee_run_until_exit(ee_model_t* model, int first_stage, const ee_stage_in_t* in, void* workspace,
                              size_t workspace_bytes, const ee_stage_out_t* outs, int32_t* batch_per_stage,
                              double timeout_s, void* cuda_stream);

/* Device-sized stage chain.  With max_batch > 0, ee_run_until_exit on a batch of up to max_batch samples runs as ONE CUDA
 * graph: the first stage at the caller's batch, then for every later stage a switch node with one body per possible
 * survivor count (body b = that stage at batch b, count 0 = nothing), selected on the device from the count the stage
 * before left in n_surv_dev (Section III, steps 3-4: B_exit sizes the next launch -- here without the host in the loop).
 * The counts still travel to the pinned words, so ee_run_until_exit returns the same batch_per_stage; results are
 * identical to the host-sized chain.  The graph of a (first stage, buffers, batch) signature is built at its first use
 * (one capture per stage and possible count: tens of milliseconds at batch 64) and cached (16 signatures).  Needs a
 * capturable stream and stage replay on; otherwise, and for larger batches, the host sizes every stage as before.
 * max_batch = 0 (the default) switches it off.  Errors: INVALID_ARG. */
ee_status_t ee_model_set_chain(ee_model_t* model, int max_batch);

/* Host-side wait for a survivor count without synchronising the stream (Section III, step 4: the scheduler needs
 * B_exit, not the features, to size its next launch).  Protocol: the caller stores `sentinel` (a negative value) in
 * its pinned word, passes the word as n_surv_host to ee_stage_run, then calls this: it polls the word until it differs
 * from the sentinel and returns the value in *value.  Work enqueued on the stream afterwards is still ordered behind
 * the stage by the stream.  Errors: INVALID_ARG; TIMEOUT when `timeout_s` seconds pass first (*value untouched). */
ee_status_t ee_wait_count(const int32_t* n_surv_host, int32_t sentinel, double timeout_s, int32_t* value);

/* Synchronises the stream and reports device-side faults the kernels recorded instead of hanging:
 * EE_ERR_TIMEOUT when a bounded wait on a barrier ran out.  The flag is cleared by the call. */
ee_status_t ee_model_check(ee_model_t* model, void* cuda_stream);

const char* ee_status_string(ee_status_t s);
const char* ee_last_cuda_error(void); /* text of the last CUDA error seen by this thread, "" if none */

#ifdef __cplusplus
}
#endif
#endif /* EE_H_ */
