/*
 * sti.h - C ABI of the shard-elastic transformer execution path (STI, arXiv 2207.05022).
 *
 * The library executes a plan that the caller supplies: for every layer, which shard units
 * are kept, at which bitwidth each is stored, and whether it sits in the preload buffer or is
 * streamed while earlier layers compute.  Choosing the plan (the paper's two-stage planner,
 * Section 5) is the caller's business; the paper's engine likewise only loads and runs the
 * shards its planning stage picked (Section 3.2).
 *
 * Vocabulary (Section 4.2, Table 1).  A layer with hidden size d, M heads of width 64 and
 * d_ff FFN neurons is cut into vertical slices.  Here the attention part and the FFN part of a
 * slice are separate *shard units*:
 *   attention unit h : Q_h, K_h, V_h  [64 x d]   and  O_h [d x 64]
 *   FFN unit j       : F1_j [f x d]              and  F2_j [d x f],   f = d_ff / n_ffn_slices
 * All matrices are out-features x in-features, row-major (y = x W^T).  The paper's shard i is
 * the pair (attention unit i, FFN unit i) with equal keep/bits.
 *
 * Shard blob format (upload).  Bitwidth k in {2,3,4,5,6}: every weight is a k-bit index into
 * the unit's table of 2^k fp32 centroids.  Index i of a matrix (row-major flat order) occupies
 * bits [i*k, i*k+k) of a bit stream, least-significant bit first, stored as little-endian
 * 32-bit words; the unit's matrices follow each other in the order Q,K,V,O (attention) or
 * F1,F2 (FFN), each starting on a 16-byte boundary (automatic for the shapes accepted here).
 * Outliers (Section 6) are (flat offset within the unit, fp32 value) pairs, offsets ascending;
 * their slot in the index stream holds an arbitrary valid index.  Bitwidth 32 is the
 * uncompressed version: `codes` holds the raw fp32 weights in the same order, no table.
 *
 * Shape limits: head_dim == 64, hidden % 128 == 0, (ffn / n_ffn_slices) % 128 == 0,
 * max_seq <= 512.
 *
 * Threading/streams: a context owns one compute stream (or borrows the caller's) and one copy
 * stream.  Forward calls are asynchronous on the compute stream; sti_sync waits for them and
 * returns the first error a kernel reported.  A context is not thread-safe.
 *
 * Errors: every call returns a status and never aborts; out-parameters are left untouched on
 * error.  Device-side waits are bounded: a kernel that gives up sets a status word that
 * sti_sync reports as STI_ERR_TIMEOUT, and the context stays usable.
 */
#ifndef STI_H_
#define STI_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default)   /* the library is built with hidden visibility otherwise */
#endif

typedef struct sti_ctx sti_ctx;    /* device, streams, dense parameters, activation scratch */
typedef struct sti_plan sti_plan;  /* which shard units, at which bits, where they live     */

typedef enum {
  STI_OK = 0,
  STI_ERR_ARG = 1,           /* null pointer, index out of range                      */
  STI_ERR_BITS = 2,          /* bitwidth not in {2..6, 32} or blob/plan mismatch       */
  STI_ERR_SHAPE = 3,         /* model shape outside the limits above, batch*seq too big */
  STI_ERR_SIZE = 4,          /* blob size does not match the unit's shape              */
  STI_ERR_STATE = 5,         /* call not allowed in this state (e.g. upload after use) */
  STI_ERR_SHARD_MISSING = 6, /* a kept unit was never uploaded                         */
  STI_ERR_OOM = 7,           /* device or pinned-host allocation failed                */
  STI_ERR_CUDA = 8,          /* CUDA runtime error                                     */
  STI_ERR_TIMEOUT = 9        /* a bounded device-side wait ran out                     */
} sti_status;

typedef enum { STI_ATTN = 0, STI_FFN = 1 } sti_kind;
typedef enum { STI_F32 = 0, STI_BF16 = 1 } sti_dtype;

typedef struct {
  int32_t n_layers;
  int32_t hidden;        /* d                                         */
  int32_t n_heads;       /* M                                         */
  int32_t head_dim;      /* must be 64                                */
  int32_t ffn;           /* d_ff                                      */
  int32_t n_ffn_slices;  /* M_f                                       */
  int32_t max_batch;
  int32_t max_seq;       /* <= 512                                    */
  int32_t act_dtype;     /* sti_dtype of x and y                      */
  float ln_eps;          /* LayerNorm epsilon (BERT: 1e-12)           */
} sti_model_desc;

typedef struct {
  uint8_t keep;      /* 0 = dropped: contributes exactly zero (Section 4.2)      */
  uint8_t bits;      /* 2..6, or 32 = uncompressed fp32                          */
  uint8_t resident;  /* 1 = preload buffer in device memory, 0 = streamed         */
} sti_shard_cfg;

typedef struct {
  int32_t bits;
  const uint32_t* codes;        /* host; index stream (or raw fp32 when bits == 32)      */
  size_t n_code_words;          /* must equal the unit's weight count * bits / 32         */
  const float* centroids;       /* host; 2^bits entries; NULL when bits == 32            */
  const uint32_t* outlier_off;  /* host; flat offsets within the unit, strictly ascending */
  const float* outlier_val;     /* host                                                   */
  size_t n_outliers;
} sti_shard_blob;

typedef struct {
  /* filled by sti_get_stats for the most recent sti_model_forward on the plan */
  int32_t n_layers;
  float compute_us[64];   /* per layer: first kernel start to last kernel end              */
  float copy_us[64];      /* per layer: duration of its host-to-device shard copy (0 if none) */
  float stall_us[64];     /* per layer: time compute waited for the copy beyond the previous layer's end */
  uint64_t streamed_bytes[64];
  uint64_t resident_bytes[64];
  float total_us;         /* first operation of the forward to its last                    */
  /* kernel-level profiling only (sti_plan_set_profiling(plan, 2)); intervals between events recorded
   * around each kernel, so each includes the launch gap before the kernel */
  float gemm_us[64];      /* per layer: the four dequant-GEMM launches (QKV, O, FFN1, FFN2)   */
  float attn_us[64];      /* per layer: the attention kernel                                  */
  float ln_us[64];        /* per layer: the two residual+LayerNorm kernels                    */
  int32_t gemm_launches;  /* dequant-GEMM launches in the forward                             */
} sti_stats;

/* Section 3.1 (the system model: a library the app links; one model per context).
 * Creates streams and scratch sized for max_batch*max_seq tokens on `device`.
 * `compute_stream` is a cudaStream_t to borrow, or NULL to create one. */
sti_status sti_ctx_create(const sti_model_desc* desc, int device, void* compute_stream, sti_ctx** out);

/* Section 6: biases and LayerNorm parameters are not quantized; they stay in memory as fp32.
 * Host arrays, copied before return: bq,bk,bv [n_heads*64]; bo [d]; b1 [ffn]; b2 [d];
 * ln1_g, ln1_b, ln2_g, ln2_b [d]. */
sti_status sti_ctx_set_layer_params(sti_ctx* ctx, int layer,
                                    const float* bq, const float* bk, const float* bv, const float* bo,
                                    const float* b1, const float* b2,
                                    const float* ln1_g, const float* ln1_b,
                                    const float* ln2_g, const float* ln2_b);

/* Section 3.2 / 5.4: a plan is the submodel with one version and one residency per shard.
 * attn has n_layers*n_heads entries (layer-major), ffn has n_layers*n_ffn_slices.
 * ring_slots >= 2 is the number of streamed-layer buffers in device memory. */
sti_status sti_plan_create(sti_ctx* ctx, const sti_shard_cfg* attn, const sti_shard_cfg* ffn,
                           int ring_slots, sti_plan** out);

/* Section 4.2 (each shard is stored once per fidelity version): hands one unit's blob to the plan.  Host pointers
 * are only read during the call.  The blob's bits must equal the plan's.  Not allowed after
 * the plan has been finalized. */
sti_status sti_shard_upload(sti_plan* plan, int layer, sti_kind kind, int index, const sti_shard_blob* blob);

/* Section 3.1: fills the preload buffer (resident units -> device memory) and lays every
 * streamed layer out as one contiguous pinned-host blob ("one layer ... as a single IO job").
 * Called implicitly by the first forward.  STI_ERR_SHARD_MISSING if a kept unit has no blob. */
sti_status sti_plan_finalize(sti_plan* plan);

/* Section 2.1 / 4.2: one layer over its kept units.  x_dev, y_dev: device, [batch, seq, hidden]
 * contiguous in act_dtype, caller-owned; x_dev == y_dev allowed.  seq_lens_dev: device int32
 * [batch] of valid lengths (padded keys get probability 0) or NULL.  A streamed layer is
 * copied first (not overlapped).  Asynchronous. */
sti_status sti_layer_forward(sti_plan* plan, int layer, const void* x_dev, void* y_dev,
                             int batch, int seq, const int32_t* seq_lens_dev);

/* Section 5.5: layers 0..n-1 in order; layer l's shard copy overlaps the compute of earlier
 * layers, a layer starts only when its own shards have arrived, and a ring slot is reused only
 * after its layer has finished.  Asynchronous. */
sti_status sti_model_forward(sti_plan* plan, const void* x_dev, void* y_dev,
                             int batch, int seq, const int32_t* seq_lens_dev);

/* Same with host buffers: x_host/y_host are [batch, seq, hidden] in act_dtype (pinned memory
 * makes the copies asynchronous), seq_lens_host int32 [batch] or NULL.  The input copy, the
 * forward and the output copy are enqueued in order; call sti_sync before reading y_host. */
sti_status sti_model_forward_host(sti_plan* plan, const void* x_host, void* y_host,
                                  int batch, int seq, const int32_t* seq_lens_host);

/* Waits for everything enqueued on the context; returns the first asynchronous error. */
sti_status sti_sync(sti_ctx* ctx);

/* Section 4.2 (decompression replaces every index by its centroid and then writes the outliers
 * over their positions): decodes one matrix of an uploaded unit for inspection.  matrix: 0..3 = Q,K,V,O
 * or 0..1 = F1,F2.  Any of the outputs may be NULL: w_dev fp32 [rows*cols] exact table values
 * with outliers patched, codes_dev one byte per index, wbf16_dev the bf16 (round-to-nearest-
 * even) operand values the GEMMs use.  Device pointers, caller-owned.  Asynchronous. */
sti_status sti_shard_decode(sti_plan* plan, int layer, sti_kind kind, int index, int matrix,
                            float* w_dev, uint8_t* codes_dev, uint16_t* wbf16_dev);

/* Section 4.2 (decompression feeds the layer's linear maps directly): runs ONE of a layer's four fused
 * dequant-GEMMs by itself, on activations the caller supplies, with the tile tables, the decode routine and
 * the kernel that a forward uses: out = x W^T, no bias, no activation function.  It is the parity hook for
 * the decode that lives inside the GEMM: with x = the identity matrix the output holds, bit for bit, the
 * bf16 (round-to-nearest-even) dequantized weights the tensor cores were given (each output element is one
 * exact product 1 * w).
 *   gemm       : 0 = QKV, 1 = O projection, 2 = FFN1, 3 = FFN2, over the layer's kept units in index order
 *   x_bf16_dev : DEVICE, [tokens, K] bf16 row-major, 16-byte aligned; K = hidden (QKV, FFN1),
 *                64 * kept heads (O), f * kept slices (FFN2); tokens need not respect max_batch * max_seq
 *   out_dev    : DEVICE, 16-byte aligned, caller-owned:
 *                QKV  bf16 [(kept head * 3 + {Q,K,V})][tokens][64]
 *                FFN1 bf16 [tokens][kept slices * f]
 *                O, FFN2  fp32 [n_partials][tokens][hidden]: the K range is split over n_partials groups of
 *                         units, each group writes its own partial sum (the caller adds them up)
 *   out_capacity_bytes : size of out_dev; STI_ERR_SIZE when the result would not fit
 *   variant    : 0 = the kernel a forward would choose for this token count, 1 = the one-CTA kernel,
 *                2 = the two-CTA (cta_group::2) kernel, STI_ERR_STATE when the tiling does not allow it,
 *                3 = (gemm 3 only) the K-accumulating two-CTA kernel that forwards of many tokens use for FFN2:
 *                all K groups summed in tensor memory, ONE complete plane written (n_partials = 1);
 *                STI_ERR_STATE when the plan was not made for that many tokens
 *   n_partials : optional out
 * STI_ERR_STATE when no kept unit feeds the GEMM.  A streamed layer is copied first.  Asynchronous. */
sti_status sti_gemm_probe(sti_plan* plan, int layer, int gemm, const void* x_bf16_dev, int tokens, void* out_dev,
                          size_t out_capacity_bytes, int variant, int32_t* n_partials);

/* Section 4.2 decompression at its steady-state rate: ONE launch of the fused dequant-GEMM over the FFN1 tiles of
 * ALL layers (every kept FFN slice's F1 matrix, hundreds of tiles for a 24-layer model), on few tokens, so that the
 * launch is long enough for the decode's throughput to show instead of one layer's launch and fill latencies.  Used by
 * the benchmark to report packed-weight GB/s against the HBM roof.  out = x F1^T per layer, no bias, no GELU.
 *   x_bf16_dev : DEVICE, [tokens, hidden] bf16, 16-byte aligned; tokens <= 128
 *   out_dev    : DEVICE, bf16 [tokens][n_layers * ffn] (layer l, kept slice number j of that layer at columns
 *                l * ffn + j * f ...), 16-byte aligned; out_capacity_bytes >= tokens * n_layers * ffn * 2
 *   packed_bytes, n_tiles : optional outs - index-stream and table bytes the launch reads, weight tiles (CTAs) it runs
 * Every kept shard must be resident (STI_ERR_STATE otherwise, also when no FFN slice is kept).  Asynchronous. */
sti_status sti_decode_rate_probe(sti_plan* plan, const void* x_bf16_dev, int tokens, void* out_dev,
                                 size_t out_capacity_bytes, uint64_t* packed_bytes, int32_t* n_tiles);

/* Section 5.2 (profiling of IO and compute delays): per-layer timings of the last
 * sti_model_forward.  Enable with sti_plan_set_profiling before that forward: level 0 = off,
 * 1 = per-layer events, 2 = additionally events around every kernel (slightly slower; levels 1 and 2 launch
 * the kernels one by one instead of replaying a CUDA graph), 3 = device-timer stamps written by the kernels
 * themselves (read with sti_get_kernel_stamps; sti_get_stats has nothing to report at this level). */
sti_status sti_plan_set_profiling(sti_plan* plan, int level);
sti_status sti_get_stats(sti_plan* plan, sti_stats* out);

/* Section 5.2, kernel by kernel and in the execution mode that is timed: with profiling level 3 a forward runs as
 * usual (CUDA graph replay, kernels launched ahead of their predecessors' end) and every kernel additionally
 * stamps the device's nanosecond timer into a record of its own.  sti_get_kernel_stamps waits for the context and
 * copies the records of the last such forward to `out` (HOST): [layer][kernel][word], STI_STAMP_KERNELS kernels per
 * layer in execution order (fp32->bf16 cast of the model input, QKV, attention, O projection, LayerNorm 1, FFN1,
 * FFN2, LayerNorm 2), STI_STAMP_WORDS words per kernel, times in ns on the device timer, 0 = not stamped (the
 * kernel did not run: dropped units, LayerNorm merged into the preceding GEMM):
 *   word 0 first CTA started          1 first CTA past the wait for the preceding kernel   2 last CTA finished
 *   word 3 last weight tile decoded   4 last CTA started      5 accumulators complete      6 row statistics exchanged
 *   (3: dequant-GEMMs only; 5, 6: dequant-GEMMs with the LayerNorm epilogue only; 7 unused)
 * capacity_words must be at least n_layers * STI_STAMP_KERNELS * STI_STAMP_WORDS (STI_ERR_SIZE otherwise). */
#define STI_STAMP_KERNELS 8
#define STI_STAMP_WORDS 8
sti_status sti_get_kernel_stamps(sti_plan* plan, uint64_t* out, size_t capacity_words, int32_t* n_layers);

/* Section 7.1 (the Load&Exec baseline: the whole model is loaded first, then executed): with overlap = 0 a model
 * forward first copies every streamed layer into its ring slot and only then starts layer 0, so IO and
 * compute delays add up; overlap = 1 (the default) is the layerwise pipeline of Section 3.1.  Results are
 * identical.  overlap = 0 needs one ring slot per streamed layer (STI_ERR_STATE otherwise: a slot could
 * only be reused after a layer that has not started).  Takes effect at the next forward. */
sti_status sti_plan_set_overlap(sti_plan* plan, int overlap);

/* Section 3.2 (executions that follow one another: shards a run loaded stay cached, and the next plan spends the freed IO time
 * on the others) and Section 5.5 (after a run, loaded shards are evicted from the top layer down until the rest fits
 * the preload buffer).  Which shards stay is the planner's decision (sti_preload_after_run); these calls keep them in
 * DEVICE memory across plans, so that the next plan uploads nothing it already holds.
 *
 * sti_plan_retain: attn_keep [n_layers*n_heads] and ffn_keep [n_layers*n_ffn_slices] (host, 0/1) mark the kept units
 * of `plan` that must stay on the device after its next run.  Preloaded units are there already; for the streamed
 * ones the call allocates a retained arena of their size (*retained_bytes) and the NEXT sti_model_forward on the plan
 * - launched kernel by kernel once, not as a graph replay - copies each of them device-to-device out of its ring slot
 * right after the layer that used it.  Marking a unit the plan dropped is STI_ERR_ARG; one retained set per plan
 * (STI_ERR_STATE on a second call).
 *
 * sti_shard_adopt: instead of sti_shard_upload - the unit (layer, kind, index) of the not yet finalized `plan` takes
 * over the unit that `from` (same context, finalized, still alive until `plan` is finalized) holds in device memory:
 * preloaded there, or retained and the retaining forward already enqueued.  Same bitwidth in both plans
 * (STI_ERR_BITS otherwise: a shard is cached at the version it was loaded with), resident in `plan` (STI_ERR_STATE
 * otherwise, also when `from` does not hold the unit on the device).  sti_plan_finalize then fills that part of the
 * preload buffer with a device-to-device copy.
 *
 * sti_plan_fill_stats: bytes sti_plan_finalize uploaded from the host into the preload buffer, bytes it took over on
 * the device, bytes of the retained arena (any pointer may be NULL). */
sti_status sti_plan_retain(sti_plan* plan, const uint8_t* attn_keep, const uint8_t* ffn_keep, uint64_t* retained_bytes);
sti_status sti_shard_adopt(sti_plan* plan, const sti_plan* from, int layer, sti_kind kind, int index);
sti_status sti_plan_fill_stats(sti_plan* plan, uint64_t* uploaded_bytes, uint64_t* adopted_bytes, uint64_t* retained_bytes);

/* Host-made faults for testing the pipeline's accounting and error paths (no counterpart in the paper, whose
 * only fault is the operating system reclaiming memory, Section 2.2).  Nothing here touches the device.
 *   STI_INJECT_SLOW_COPY            : the host sleeps `value` microseconds (<= 1 s) before it enqueues the shard
 *                                     copy of `layer` in forwards that are launched kernel by kernel (profiling
 *                                     level 1 or 2); the layer then starts late and its stall_us shows the wait.
 *                                     Results do not change.
 *   STI_INJECT_PINNED_ALLOC_FAILURE : with value != 0 the pinned-host allocation of sti_plan_finalize is treated as
 *                                     failed (STI_ERR_OOM); the plan cannot be used afterwards but can be destroyed.
 *                                     Only before the plan is finalized (STI_ERR_STATE otherwise); layer is ignored.
 *   STI_INJECT_NONE                 : clears both. */
typedef enum { STI_INJECT_NONE = 0, STI_INJECT_SLOW_COPY = 1, STI_INJECT_PINNED_ALLOC_FAILURE = 2 } sti_inject;
sti_status sti_plan_inject(sti_plan* plan, int what, int layer, unsigned value);

/* Bytes the plan holds: preload buffer in device memory, pinned host arena, ring slots. */
sti_status sti_plan_memory(sti_plan* plan, uint64_t* preload_bytes, uint64_t* pinned_bytes, uint64_t* ring_bytes);

/* Debugging aid (no counterpart in the paper): the preload buffer and every ring slot of the working buffer are
 * followed (and the buffers preceded) by 256 guard bytes of a fixed pattern that nothing may write - only the upload
 * and the per-layer copies write those buffers, each with the size the plan computed.  Waits for the plan's work on
 * both streams, reads the guards back and returns in *damaged how many of them no longer hold the pattern (0 = intact).
 * Together with sti_plan_inject's delayed copies this is the stream-order check of the pipeline: results and guards
 * must not depend on when a copy reaches the copy engine.  ring_bytes of sti_plan_memory includes the guards. */
sti_status sti_plan_check_guards(sti_plan* plan, int32_t* damaged);

/* Host-only utility: re-tiles one matrix's canonical index stream (rows x cols indexes of `bits`
 * bits) into the order the device holds it (see the upload format above; the size is unchanged).
 * For every group of 32 rows (64 rows when cols == 64) and every 128-column chunk, the `bits`
 * 16-byte planes of the 32 rows' 128-index runs are stored plane-major, 512 bytes per plane.
 * Exposed so that the layout can be inspected and tested without a device. */
sti_status sti_host_retile(const uint8_t* src, uint8_t* dst, uint32_t rows, uint32_t cols, uint32_t bits);

/* (The paper has no counterpart to this call; it exists for callers that cannot allocate.)
 * Decodes one matrix of a shard like sti_shard_decode, but without a context or a plan and without
 * allocating anything, on the host or on the device.  It is meant for callers that must not call
 * cudaMalloc: code running inside a process whose framework allocator already owns the device memory,
 * integrity checks of shard files under an enforced memory budget, sections where the allocator's
 * implicit device synchronisation is unwelcome.  The kernel's working copy of the shard (re-tiled
 * index stream, centroid table, outlier lists) lives in a fixed array of STI_NOALLOC_SCRATCH_BYTES
 * bytes inside the library image; each GPU that loads the library holds that array until exit.
 *   device, stream : where to run; stream is a cudaStream_t or NULL for the default stream
 *   bits           : 2..6                      rows, cols: the matrix shape, cols == 64 with rows % 64 == 0,
 *                    or cols % 128 == 0 with rows % 32 == 0
 *   codes          : HOST, the matrix's canonical index stream (rows*cols*bits/32 words)
 *   centroids      : HOST, 2^bits entries
 *   outlier_off/val: HOST, n_outliers pairs, offsets within the matrix, strictly ascending
 *   w_dev, codes_dev, wbf16_dev : DEVICE outputs as in sti_shard_decode, caller-owned, any may be NULL
 * Limits: rows*cols*bits/8 <= STI_NOALLOC_MAX_STREAM_BYTES and n_outliers <= STI_NOALLOC_MAX_OUTLIERS
 * (every matrix of BERT-base and BERT-large at up to 6 bits fits); anything larger returns STI_ERR_SIZE
 * and nothing runs.  Host inputs are copied into library-owned staging buffers before the call returns
 * (pinned or pageable alike: the caller may reuse or free them at once); the kernel runs asynchronously
 * on `stream`.  The caller's current device is the same after the call as before it.  The first call on a
 * device looks up the array's device address; make that first call before starting any stream capture.
 * A call on a stream that is being captured is refused with STI_ERR_STATE, because its copies would read
 * the shared staging buffers only when the captured work runs.  All calls share the one array, which keeps the last call's
 * contents (each call overwrites everything its kernel reads): calls on the same stream are ordered,
 * calls whose GPU work can overlap (different streams or threads) race on it and must be serialised
 * by the caller. */
#define STI_NOALLOC_MAX_STREAM_BYTES 262144u
#define STI_NOALLOC_MAX_OUTLIERS 4096u
#define STI_NOALLOC_SCRATCH_BYTES (262144u + 256u + 2u * 4u * 4096u)
sti_status sti_matrix_decode_noalloc(int device, void* stream, int bits, uint32_t rows, uint32_t cols,
                                     const uint32_t* codes, const float* centroids,
                                     const uint32_t* outlier_off, const float* outlier_val, size_t n_outliers,
                                     float* w_dev, uint8_t* codes_dev, uint16_t* wbf16_dev);

/* Kernel launches issued by the library on this context since creation (for accounting). */
uint64_t sti_ctx_launch_count(sti_ctx* ctx);

void sti_plan_destroy(sti_plan* plan);
void sti_ctx_destroy(sti_ctx* ctx);
const char* sti_strerror(sti_status s);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* STI_H_ */
