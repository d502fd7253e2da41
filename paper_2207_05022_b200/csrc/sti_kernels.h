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
  unsigned long long* stamps;   // this launch's profiling record (see sti_device.cuh), or null
};

size_t gemm_weight_bytes(uint32_t n_rows, uint32_t k_total);
uint32_t gemm_header_bytes();
bool gemm_pick_ring(uint32_t w_bytes, uint32_t k_total, uint32_t hdr_bytes, uint32_t* n_stages, uint32_t* bps);   // false: does not fit
size_t gemm_smem_bytes(uint32_t w_bytes, uint32_t n_stages, uint32_t bps, uint32_t hdr_bytes);
cudaError_t gemm_configure();   // opt in to large dynamic shared memory (once per device)
cudaError_t launch_gemm(GemmKind kind, const GemmLaunch& p, cudaStream_t s);

// K-accumulating two-CTA dequant-GEMM (fp32 output written once, all K groups summed in tensor memory).
// jobs: n_groups x n_cols64 tile jobs of 64 rows and at most k_group columns, job (g, c) at index g * n_cols64 + c,
// segments at the fixed stride; out: [T][ldo] fp32, tile c writes columns [64 c, 64 c + 64).
struct KaccLaunch {
  const Job* jobs;
  const Seg* segs;
  int n_groups, n_cols64, m_ctas;
  CUtensorMap xmap;         // x: [T rows, ldx columns] bf16, box 64 x 128, 128-byte swizzle
  const void* x;            // the same operand as a plain pointer: idle warps prefetch it into L2; null = no prefetch
  int ldx;
  int T;
  float* out;
  int ldo;
  int* err;
  uint32_t n_stages, bps, hdr_bytes, seg_stride;   // ring: n_stages stages of bps boxes (1 or 2; K groups are multiples of 64 * bps)
  uint32_t k_group;         // columns of the widest K group (a multiple of 64): the size of the two weight buffers
  bool pdl;
  unsigned long long* stamps;
};
cudaError_t gemm_kacc_configure();
uint32_t gemm_kacc_stages(uint32_t hdr_bytes, uint32_t k_group, uint32_t bps, size_t smem_limit);
size_t gemm_kacc_smem_bytes(uint32_t hdr_bytes, uint32_t n_stages, uint32_t bps, uint32_t k_group);
cudaError_t launch_gemm_kacc(const KaccLaunch& p, cudaStream_t s);

// Per-head attention over kept heads.  qkv: [(kept*3 + which)][T][64] bf16; out: [T][n_kept*64] bf16.
// sm_count (the device's multiprocessor count) picks the CTA shape: large query tiles once they fill the GPU.
cudaError_t attention_configure();
cudaError_t launch_attention(const uint16_t* qkv, uint16_t* out, int n_kept, int batch, int seq,
                             const int32_t* seq_lens, int sm_count, cudaStream_t s, bool pdl,
                             unsigned long long* stamps);

// The same attention on the tcgen05 tensor cores, one CTA per (sequence, kept head) with two query tiles in flight, for
// many tokens (attention_tc.cu).
// `qkv_map`: TMA view of qkv as [3 * n_kept * T rows, 64 columns] bf16, boxes of 128 rows x 64 columns, 128-byte swizzle.
cudaError_t attention_tc_configure();
cudaError_t launch_attention_tc(const CUtensorMap& qkv_map, uint16_t* out, int n_kept, int batch, int seq,
                                const int32_t* seq_lens, int* err, cudaStream_t s, bool pdl, unsigned long long* stamps);


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
  unsigned long long* stamps;   // profiling record or null
};
cudaError_t launch_layernorm(const LnLaunch& p, cudaStream_t s, bool pdl);

// fp32 -> bf16 (round-to-nearest-even) copy of the activations the first GEMM reads.
cudaError_t launch_cast_bf16(const float* in, uint16_t* out, size_t n, cudaStream_t s, bool pdl, unsigned long long* stamps);

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

// Launch with or without the programmatic-dependent-launch attribute (every kernel of the layer calls
// pdl_wait before it reads what its predecessor wrote, so consecutive kernels may overlap their prologues).
// `cluster_x` > 1 groups that many consecutive CTAs along x into one thread-block cluster.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                         bool pdl, unsigned cluster_x, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster_x; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool pdl,
                                 Args... args) {
  return launch_kernel_cluster(kernel, grid, block, smem, s, pdl, 1u, args...);
}

constexpr int ERR_NONE = 0;
constexpr int ERR_WAIT_TIMEOUT = 1;   // a bounded mbarrier wait ran out
constexpr int ERR_BAD_JOB = 2;        // a job descriptor failed the kernel's own checks

}  // namespace sti
