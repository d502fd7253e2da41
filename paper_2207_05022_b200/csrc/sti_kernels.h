// Internal interface between the host runtime (api.cu) and the sm_100a kernels.
// Nothing here is part of the public ABI.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sti {

// One contiguous run of a unit matrix's rows feeding a weight tile.
// Index streams are held re-tiled (see retile.h): for every group of 32 rows (64 when the
// matrix has 64 in-features) and every 128-column chunk, the k 16-byte planes of the 32
// per-lane quanta are stored plane-major, so that a warp reads each plane as one coalesced
// 512-byte line and every lane ends up with 128 consecutive indexes of one row.
struct Seg {
  const uint4* codes;       // device; first plane of the tile's first row group (raw fp32 rows when bits == 32)
  const float* table;       // device; 2^bits fp32 centroids (unused when bits == 32)
  const uint32_t* out_off;  // device; outliers whose flat offset falls inside this tile
  const float* out_val;
  uint32_t n_out;
  uint32_t flat_base;       // flat offset, within the unit, of the tile's first weight
  uint32_t bits;            // 2..6 or 32
  uint32_t kc;              // in-features (row length) of the source matrix
  uint32_t koff;            // where this segment starts in the job's K range
  uint32_t pad_;
};

// One weight-stationary tile: n_rows output features x k_total input features.
struct Job {
  uint32_t seg_begin, n_seg;
  uint32_t n_rows;          // 32, 64 or 128 (multiple of 64 when segments have kc == 64)
  uint32_t k_total;         // multiple of 64
  uint32_t x_koff;          // first column of the activation operand
  uint32_t out_mat;         // output element (t, c) goes to out[(out_mat*T + t)*ldo + out_col + c]
  uint32_t out_col;
  int32_t bias_off;         // index of the tile's first bias element, -1 = no bias
};

enum GemmKind : int {
  GEMM_BF16_TO_BF16 = 1,      // bf16 in, bf16 out (+bias)                     : QKV
  GEMM_BF16_TO_BF16_GELU = 2, // bf16 in, bf16 out, +bias, erf-GELU            : FFN1
  GEMM_BF16_TO_F32 = 3        // bf16 in, fp32 partial sums out, no bias       : O projection, FFN2
};

struct GemmLaunch {
  const Job* jobs;
  const Seg* segs;
  int n_jobs;
  int m_ctas;               // CTAs along the token dimension (each loops over its M tiles)
  CUtensorMap xmap;         // TMA descriptor of x: [T rows, ldx columns] bf16, box 64 x 128, 128-byte swizzle
  const void* x;            // [T, ldx] bf16
  int ldx;
  int T;
  void* out;
  int ldo;
  const float* bias;
  int* err;                 // device status word
  size_t smem_bytes;        // header + w_bytes + n_stages activation stages
  uint32_t n_stages;        // stages in the activation ring
  uint32_t bps;             // 16 KB boxes (64 columns) per stage: 1, 2 or 4
  uint32_t w_bytes;         // shared memory reserved for the weight tile (largest job)
  uint32_t hdr_bytes;       // barriers + bias + per-warp centroid tables
  uint32_t seg_stride;      // the segments of job j start at segs[j * seg_stride]
  const uint8_t* pf_ptr[4]; // what the next layer reads first (packed shards, tile descriptors, dense parameters):
  uint32_t pf_bytes[4];     // pulled into L2 by this launch's idle warps
  bool simt_debug;          // compute the products on the plain ALUs instead of the tensor cores
  bool pdl;                 // launch with programmatic dependent launch
  bool pair;                // two-CTA clusters (cta_group::2): jobs 2i and 2i+1 share one M=256 x N=128 MMA
};

size_t gemm_weight_bytes(uint32_t n_rows, uint32_t k_total);
uint32_t gemm_header_bytes();
bool gemm_pick_ring(uint32_t w_bytes, uint32_t k_total, uint32_t hdr_bytes, uint32_t* n_stages, uint32_t* bps);   // false: does not fit
size_t gemm_smem_bytes(uint32_t w_bytes, uint32_t n_stages, uint32_t bps, uint32_t hdr_bytes);
cudaError_t gemm_configure();   // opt in to large dynamic shared memory (once per device)
cudaError_t launch_gemm(GemmKind kind, const GemmLaunch& p, cudaStream_t s);

// Per-head attention over kept heads.  qkv: [(kept*3 + which)][T][64] bf16; out: [T][n_kept*64] bf16.
cudaError_t attention_configure();
cudaError_t launch_attention(const uint16_t* qkv, uint16_t* out, int n_kept, int batch, int seq,
                             const int32_t* seq_lens, cudaStream_t s, bool pdl);

// out = LayerNorm(sum_p partial[p] + bias + resid) * gamma + beta, one warp per token row.
struct LnLaunch {
  const float* partial;     // [n_partial][T][d]
  int n_partial;
  const float* bias;        // [d]
  const void* resid;        // [T][d], fp32 or bf16
  int resid_bf16;
  const float* gamma;
  const float* beta;
  float eps;
  int T, d;
  float* out_f32;           // optional
  uint16_t* out_bf16;       // optional
  int ctas_hint;            // > 0: pack rows so that about this many CTAs are launched (few tokens); 0: one row per CTA
};
cudaError_t launch_layernorm(const LnLaunch& p, cudaStream_t s, bool pdl);

// fp32 -> bf16 (round-to-nearest-even) copy of the activations the first GEMM reads.
cudaError_t launch_cast_bf16(const float* in, uint16_t* out, size_t n, cudaStream_t s, bool pdl);

// Stand-alone decode of one matrix (inspection / parity).
struct DecodeLaunch {
  const uint4* codes;       // re-tiled stream of the matrix (raw fp32 when bits == 32)
  const float* table;
  const uint32_t* out_off;  // the unit's outliers restricted to this matrix
  const float* out_val;
  uint32_t n_out;
  uint32_t flat_base;       // flat offset of the matrix inside the unit
  uint32_t bits, rows, kc;
  float* w;                 // optional outputs
  uint8_t* codes_out;
  uint16_t* wbf16;
};
cudaError_t launch_decode(const DecodeLaunch& p, cudaStream_t s);

// ---------------------------------------------------------------------------------------
// Whole-layer kernel for few tokens (one launch per layer instead of seven).
// A grid of at most one CTA per SM runs the layer's seven steps one after the other - QKV GEMM,
// attention, O projection, residual + LayerNorm, FFN1 + GELU, FFN2, residual + LayerNorm - with a
// grid-wide barrier between steps.  Between arriving at a barrier and waiting on it a CTA decodes the
// weight tile of its next GEMM step (weights depend on no activation), so shard decode never sits on
// the critical path, and the barriers replace the kernel boundaries.
// ---------------------------------------------------------------------------------------
struct FusedGemm {
  CUtensorMap xmap;         // activation operand of this step: [T, ld] bf16, box 64 x 128, 128-byte swizzle
  const Job* jobs;
  const Seg* segs;          // the segments of job j start at segs[j * seg_stride]
  void* out;
  const float* bias;
  int n_jobs;
  int m_ctas;               // CTAs per job along the token dimension; n_jobs * m_ctas <= grid
  int ldo;
  int kind;                 // GemmKind
  uint32_t n_stages, bps;   // activation ring: stages, 16 KB boxes per stage
  uint32_t w_bytes;         // shared memory of the largest weight tile of this step
  uint32_t seg_stride;
  uint32_t ahead;           // 1: the tile is decoded before the preceding barrier wait (its shared memory is free then)
};

struct FusedLayerParams {
  FusedGemm g[4];           // QKV, O projection, FFN1, FFN2
  LnLaunch ln[2];           // after the O projection, after FFN2
  const uint16_t* qkv;      // attention operands / result, as in launch_attention
  uint16_t* attn_out;
  const int32_t* seq_lens;
  int n_kept_heads, batch, seq, T;
  unsigned int* barrier;    // one counter per launch, zero when the kernel starts
  const uint8_t* pf_ptr[4]; // the next layer's packed shards, tile descriptors and dense parameters,
  uint32_t pf_bytes[4];     // pulled into L2 while this layer computes
  int* err;
};

constexpr int kFusedMaxCtas = 148;
cudaError_t fused_configure();
// Shared memory the attention step needs for sequences of `seq` tokens, counted from the start of the
// activation area; the O-projection tile may be decoded ahead only if it fits above that.
size_t fused_attention_bytes(int seq);
size_t fused_smem_total();      // dynamic shared memory of the kernel
size_t fused_low_offset();      // where the activation stages / attention buffers start
cudaError_t launch_fused_layer(const FusedLayerParams& p, int grid, cudaStream_t s, bool pdl);

// Launch with or without the programmatic-dependent-launch attribute (every kernel of the layer calls
// pdl_wait before it reads what its predecessor wrote, so consecutive kernels may overlap their prologues).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool pdl,
                                 Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

constexpr int ERR_NONE = 0;
constexpr int ERR_WAIT_TIMEOUT = 1;   // a bounded mbarrier wait ran out
constexpr int ERR_BAD_JOB = 2;        // a job descriptor failed the kernel's own checks

}  // namespace sti
