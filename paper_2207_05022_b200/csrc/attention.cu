// Per-head scaled-dot-product attention over the kept heads (Section 2.1: each attention head
// independently contributes one representation; Section 4.2: any subset of heads executes).
//
// One CTA = (64-query tile, kept head, sequence); 4 warps x 16 query rows.  K and V of the whole
// sequence (<= 512 keys) are brought into shared memory with cp.async (row-major, padded rows; the
// value fragments are read with ldmatrix.trans); scores and the probability-value product run on
// mma.sync m16n8k16 bf16 with fp32 accumulation, softmax is done in registers with warp shuffles
// over the four lanes that share a row (online max/sum over 64-key blocks).
// Attention is ~3 % of a layer's FLOPs at seq 128; the dense projections use tcgen05 (dqgemm.cu).
#include <cuda_bf16.h>

#include "attention_device.cuh"
#include "sti_kernels.h"

namespace sti {
namespace {

constexpr int kHeadDim = 64;
constexpr int kKStride = kAttnKStride;

template <int WARPS>      // 16 query rows per warp; K and V of the sequence are shared by the CTA's warps
__global__ void __launch_bounds__(32 * WARPS)
attention_kernel(const uint16_t* __restrict__ qkv, uint16_t* __restrict__ out, int n_kept, int batch, int L,
                 const int32_t* __restrict__ seq_lens, unsigned long long* stamps) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int qt = blockIdx.x, hi = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int T = batch * L;
  const int Lpad = (L + 63) / 64 * 64;
  uint16_t* Ks = reinterpret_cast<uint16_t*>(smem);                       // [Lpad][72]
  uint16_t* Vs = Ks + static_cast<size_t>(Lpad) * kKStride;               // [Lpad][72]

  const uint16_t* Qg = qkv + (static_cast<size_t>(hi * 3 + 0) * T + static_cast<size_t>(b) * L) * kHeadDim;
  const uint16_t* Kg = qkv + (static_cast<size_t>(hi * 3 + 1) * T + static_cast<size_t>(b) * L) * kHeadDim;
  const uint16_t* Vg = qkv + (static_cast<size_t>(hi * 3 + 2) * T + static_cast<size_t>(b) * L) * kHeadDim;

  pdl_launch_dependents();
  if (tid == 0) { stamp_min(stamps, STAMP_FIRST_START); stamp_max(stamps, STAMP_LAST_START); }
  pdl_wait();          // q, k, v (and possibly seq_lens) come from the preceding kernels
  if (tid == 0) stamp_min(stamps, STAMP_RELEASE);
  int valid = L;
  if (seq_lens != nullptr) {
    valid = seq_lens[b];
    valid = valid < 0 ? 0 : (valid > L ? L : valid);
  }

  // K and V rows: every 16-byte piece is its own cp.async, all in flight at once; rows past L are zero
  const uint32_t ks_addr = smem_addr(Ks), vs_addr = smem_addr(Vs);
  for (int idx = tid; idx < Lpad * 8; idx += 32 * WARPS) {
    const int key = idx >> 3, piece = idx & 7;
    const bool ok = key < L;
    const size_t goff = static_cast<size_t>(ok ? key : 0) * kHeadDim + piece * 8;
    const uint32_t soff = static_cast<uint32_t>(key * kKStride + piece * 8) * 2;
    cp_async16(ks_addr + soff, Kg + goff, ok ? 16u : 0u);
    cp_async16(vs_addr + soff, Vg + goff, ok ? 16u : 0u);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");

  // query fragments of this warp's 16 rows
  const int q0 = qt * (16 * WARPS) + warp * 16;
  uint32_t qa[4][4];
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
    const int r0 = q0 + g, r1 = q0 + g + 8;
    const int c = kk * 16 + 2 * t4;
    qa[kk][0] = r0 < L ? __ldg(reinterpret_cast<const uint32_t*>(Qg + static_cast<size_t>(r0) * kHeadDim + c)) : 0u;
    qa[kk][1] = r1 < L ? __ldg(reinterpret_cast<const uint32_t*>(Qg + static_cast<size_t>(r1) * kHeadDim + c)) : 0u;
    qa[kk][2] = r0 < L ? __ldg(reinterpret_cast<const uint32_t*>(Qg + static_cast<size_t>(r0) * kHeadDim + c + 8)) : 0u;
    qa[kk][3] = r1 < L ? __ldg(reinterpret_cast<const uint32_t*>(Qg + static_cast<size_t>(r1) * kHeadDim + c + 8)) : 0u;
  }

  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  const float scale_log2 = 0.125f * 1.4426950408889634f;     // 1/sqrt(64) * log2(e)
  float o[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};

  const int n_kblocks = (valid + 63) / 64;
  for (int kb = 0; kb < n_kblocks; ++kb) {
    float s[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint16_t* krow = Ks + static_cast<size_t>(kb * 64 + j * 8 + g) * kKStride + 2 * t4;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(krow + kk * 16);
        const uint32_t b1 = *reinterpret_cast<const uint32_t*>(krow + kk * 16 + 8);
        mma_bf16_16816(s[j], qa[kk], b0, b1);
      }
    }
    float mblk[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int key = kb * 64 + j * 8 + 2 * t4;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float v = (key + (c & 1) < valid) ? s[j][c] * scale_log2 : -INFINITY;
        s[j][c] = v;
        mblk[c >> 1] = fmaxf(mblk[c >> 1], v);
      }
    }
    float alpha[2], m_use[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mblk[r] = fmaxf(mblk[r], __shfl_xor_sync(0xffffffffu, mblk[r], 1));
      mblk[r] = fmaxf(mblk[r], __shfl_xor_sync(0xffffffffu, mblk[r], 2));
      const float m_new = fmaxf(m_run[r], mblk[r]);
      m_use[r] = (m_new == -INFINITY) ? 0.f : m_new;
      alpha[r] = exp2f(m_run[r] - m_use[r]);
      m_run[r] = m_new;
      l_run[r] *= alpha[r];
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float p = exp2f(s[j][c] - m_use[c >> 1]);
        s[j][c] = p;
        l_run[c >> 1] += p;
        o[j][c] *= alpha[c >> 1];
      }
    }
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      uint32_t pa[4];
      pa[0] = pack_bf16x2(s[2 * kk][0], s[2 * kk][1]);
      pa[1] = pack_bf16x2(s[2 * kk][2], s[2 * kk][3]);
      pa[2] = pack_bf16x2(s[2 * kk + 1][0], s[2 * kk + 1][1]);
      pa[3] = pack_bf16x2(s[2 * kk + 1][2], s[2 * kk + 1][3]);
      // lanes 0-15 address the 16 key rows of this k-step (8 rows per 8x8 matrix)
      const uint32_t vrow = vs_addr + static_cast<uint32_t>((kb * 64 + kk * 16 + (lane & 15)) * kKStride) * 2;
#pragma unroll
      for (int jd = 0; jd < 8; ++jd) {
        uint32_t b0, b1;
        ldmatrix_x2_trans(vrow + jd * 16, b0, b1);
        mma_bf16_16816(o[jd], pa, b0, b1);
      }
    }
  }

  float inv[2];
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    float l = l_run[r];
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    inv[r] = l > 0.f ? 1.f / l : 0.f;
  }
  const int ldo = n_kept * kHeadDim;
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int row = q0 + g + 8 * r;
    if (row < L) {
      uint16_t* dst = out + (static_cast<size_t>(b) * L + row) * ldo + hi * kHeadDim + 2 * t4;
#pragma unroll
      for (int jd = 0; jd < 8; ++jd)
        *reinterpret_cast<uint32_t*>(dst + jd * 8) = pack_bf16x2(o[jd][2 * r] * inv[r], o[jd][2 * r + 1] * inv[r]);
    }
  }
  if (stamps != nullptr) {
    __syncthreads();
    if (tid == 0) stamp_max(stamps, STAMP_LAST_END);
  }
}

// Few tokens: one CTA of 16 warps per (64-query tile, kept head, sequence), keys split four ways inside the
// CTA - a quarter of the serial key loop of the kernel above, at the price of one merge through shared memory.
__global__ void __launch_bounds__(kAttnThreads)
attention_split_kernel(AttnArgs p) {
  extern __shared__ __align__(16) uint8_t smem[];
  pdl_launch_dependents();
  if (threadIdx.x == 0) { stamp_min(p.stamps, STAMP_FIRST_START); stamp_max(p.stamps, STAMP_LAST_START); }
  pdl_wait();          // q, k, v (and possibly seq_lens) come from the preceding kernels
  if (threadIdx.x == 0) stamp_min(p.stamps, STAMP_RELEASE);
  attention_step(p, blockIdx.x, gridDim.x, smem, threadIdx.x);
  if (p.stamps != nullptr) {
    __syncthreads();
    if (threadIdx.x == 0) stamp_max(p.stamps, STAMP_LAST_END);
  }
}

size_t attn_split_smem_bytes(int L) {
  const int Lpad = (L + 63) / 64 * 64;
  return static_cast<size_t>(Lpad) * kAttnKStride * 2 * 2 + kAttnMergeBytes;
}

size_t attn_smem_bytes(int L) {
  const int Lpad = (L + 63) / 64 * 64;
  return static_cast<size_t>(Lpad) * kKStride * 2 * 2;      // K and V, padded rows
}

}  // namespace

cudaError_t attention_configure() {
  cudaError_t e = cudaFuncSetAttribute(attention_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(attn_smem_bytes(512)));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attention_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           static_cast<int>(attn_smem_bytes(512)));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(attention_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(attn_split_smem_bytes(512)));
}

cudaError_t launch_attention(const uint16_t* qkv, uint16_t* out, int n_kept, int batch, int seq,
                             const int32_t* seq_lens, int sm_count, cudaStream_t s, bool pdl,
                             unsigned long long* stamps) {
  if (n_kept <= 0) return cudaSuccess;
  // 128-query CTAs when there are enough of them to fill the GPU (fewer K/V re-reads per head), 64 otherwise
  const long ctas128 = static_cast<long>((seq + 127) / 128) * n_kept * batch;
  if (seq >= 128 && ctas128 >= sm_count) {
    dim3 grid((seq + 127) / 128, n_kept, batch);
    return launch_kernel(attention_kernel<8>, grid, dim3(256), attn_smem_bytes(seq), s, pdl, qkv, out, n_kept, batch,
                         seq, seq_lens, stamps);
  }
  const long items = static_cast<long>((seq + 63) / 64) * n_kept * batch;
  if (items <= 2 * sm_count && seq > 64) {          // too few CTAs to fill the GPU: shorten each CTA's key loop instead
    AttnArgs a{qkv, out, seq_lens, n_kept, batch, seq, batch * seq, stamps};
    return launch_kernel(attention_split_kernel, dim3(static_cast<unsigned>(items)), dim3(kAttnThreads),
                         attn_split_smem_bytes(seq), s, pdl, a);
  }
  dim3 grid((seq + 63) / 64, n_kept, batch);
  return launch_kernel(attention_kernel<4>, grid, dim3(128), attn_smem_bytes(seq), s, pdl, qkv, out, n_kept, batch, seq,
                       seq_lens, stamps);
}

}  // namespace sti
