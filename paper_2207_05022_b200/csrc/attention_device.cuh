// Key-split attention over the kept heads, shared by the stand-alone attention kernel for few tokens and
// by the whole-layer kernel (Section 2.1: each head contributes independently; Section 4.2: any subset).
#pragma once
#include <cuda_bf16.h>

#include "sti_device.cuh"

namespace sti {
namespace {

constexpr int kAttnThreads = 512;                        // 4 query groups x 4 key splits
constexpr int kAttnKStride = 64 + 8;                     // bf16 per K / V row in shared memory (conflict-free fragment reads)
constexpr uint32_t kAttnMergeBytes = 3 * 4 * 32 * 36 * 4;   // three key-split partners x four query groups

struct AttnArgs {
  const uint16_t* qkv;      // [(kept head * 3 + {Q,K,V})][T][64] bf16
  uint16_t* out;            // [T][n_kept * 64] bf16
  const int32_t* seq_lens;  // optional, per sequence
  int n_kept, batch, seq, T;
  unsigned long long* stamps;   // profiling record or null
};

// ---------------------------------------------------------------------------------------
// Attention step (Section 2.1; kept heads only).  Work item = (64-query tile, kept head, sequence).
// The CTA's 16 warps form 4 query groups (16 rows each) x 4 key splits: warp (qg, ks) walks the 64-key
// blocks kb = ks, ks + 4, ... with mma.sync m16n8k16 and an online softmax in registers; the four
// partial (max, sum, output) triples of a query group are merged through shared memory.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t addr, uint32_t& r0, uint32_t& r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}

// `buf`: shared memory for K, V ([Lpad][72] bf16 each) and the merge buffer (kAttnMergeBytes); 512 threads.
__device__ __forceinline__ void attention_step(const AttnArgs& p, uint32_t cta, uint32_t n_ctas, uint8_t* buf, uint32_t tid) {
  const int L = p.seq, T = p.T, n_kept = p.n_kept;
  const int lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int qg = warp & 3, ks = warp >> 2;
  const int Lpad = (L + 63) / 64 * 64;
  const int q_tiles = (L + 63) / 64;
  const int n_items = q_tiles * n_kept * p.batch;
  uint16_t* Ks = reinterpret_cast<uint16_t*>(buf);
  uint16_t* Vs = Ks + static_cast<size_t>(Lpad) * kAttnKStride;
  float* merge = reinterpret_cast<float*>(Vs + static_cast<size_t>(Lpad) * kAttnKStride);   // [3][4][36][32]
  const uint32_t ks_addr = smem_addr(Ks), vs_addr = smem_addr(Vs);
  const float scale_log2 = 0.125f * 1.4426950408889634f;     // 1/sqrt(64) * log2(e)

  for (int item = cta; item < n_items; item += n_ctas) {
    const int qt = item % q_tiles, hi = (item / q_tiles) % n_kept, b = item / (q_tiles * n_kept);
    const uint16_t* Qg = p.qkv + (static_cast<size_t>(hi * 3 + 0) * T + static_cast<size_t>(b) * L) * 64;
    const uint16_t* Kg = p.qkv + (static_cast<size_t>(hi * 3 + 1) * T + static_cast<size_t>(b) * L) * 64;
    const uint16_t* Vg = p.qkv + (static_cast<size_t>(hi * 3 + 2) * T + static_cast<size_t>(b) * L) * 64;
    int valid = L;
    if (p.seq_lens != nullptr) {
      valid = p.seq_lens[b];
      valid = valid < 0 ? 0 : (valid > L ? L : valid);
    }
    for (int idx = tid; idx < Lpad * 8; idx += kAttnThreads) {
      const int key = idx >> 3, piece = idx & 7;
      const bool ok = key < L;
      const size_t goff = static_cast<size_t>(ok ? key : 0) * 64 + piece * 8;
      const uint32_t soff = static_cast<uint32_t>(key * kAttnKStride + piece * 8) * 2;
      cp_async16(ks_addr + soff, Kg + goff, ok ? 16u : 0u);
      cp_async16(vs_addr + soff, Vg + goff, ok ? 16u : 0u);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");

    const int q0 = qt * 64 + qg * 16;
    uint32_t qa[4][4];
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      const int r0 = q0 + g, r1 = q0 + g + 8;
      const int c = kk * 16 + 2 * t4;
      qa[kk][0] = r0 < L ? *reinterpret_cast<const uint32_t*>(Qg + static_cast<size_t>(r0) * 64 + c) : 0u;
      qa[kk][1] = r1 < L ? *reinterpret_cast<const uint32_t*>(Qg + static_cast<size_t>(r1) * 64 + c) : 0u;
      qa[kk][2] = r0 < L ? *reinterpret_cast<const uint32_t*>(Qg + static_cast<size_t>(r0) * 64 + c + 8) : 0u;
      qa[kk][3] = r1 < L ? *reinterpret_cast<const uint32_t*>(Qg + static_cast<size_t>(r1) * 64 + c + 8) : 0u;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

    float o[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};
    const int n_kblocks = (valid + 63) / 64;
    for (int kb = ks; kb < n_kblocks; kb += 4) {
      float s[8][4];
#pragma unroll
      for (int j = 0; j < 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint16_t* krow = Ks + static_cast<size_t>(kb * 64 + j * 8 + g) * kAttnKStride + 2 * t4;
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
          const float pr = exp2f(s[j][c] - m_use[c >> 1]);
          s[j][c] = pr;
          l_run[c >> 1] += pr;
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
        const uint32_t vrow = vs_addr + static_cast<uint32_t>((kb * 64 + kk * 16 + (lane & 15)) * kAttnKStride) * 2;
#pragma unroll
        for (int jd = 0; jd < 8; ++jd) {
          uint32_t b0, b1;
          ldmatrix_x2_trans(vrow + jd * 16, b0, b1);
          mma_bf16_16816(o[jd], pa, b0, b1);
        }
      }
    }
    // the four lanes of a row hold disjoint keys: complete the row sums before merging
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
      l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    }
    // key splits 1..3 hand their partial result to split 0 of the same query group
    if (ks > 0) {
      float* dst = merge + (static_cast<size_t>(ks - 1) * 4 + qg) * 36 * 32 + lane;
      dst[0 * 32] = m_run[0]; dst[1 * 32] = m_run[1]; dst[2 * 32] = l_run[0]; dst[3 * 32] = l_run[1];
#pragma unroll
      for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int c = 0; c < 4; ++c) dst[(4 + j * 4 + c) * 32] = o[j][c];
    }
    __syncthreads();
    if (ks == 0) {
#pragma unroll 1
      for (int part = 0; part < 3; ++part) {
        const float* src = merge + (static_cast<size_t>(part) * 4 + qg) * 36 * 32 + lane;
        float f_old[2], f_new[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const float m_o = src[r * 32], l_o = src[(2 + r) * 32];
          const float m_new = fmaxf(m_run[r], m_o);
          const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
          f_old[r] = exp2f(m_run[r] - m_use);
          f_new[r] = exp2f(m_o - m_use);
          l_run[r] = l_run[r] * f_old[r] + l_o * f_new[r];
          m_run[r] = m_new;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
          for (int c = 0; c < 4; ++c)
            o[j][c] = o[j][c] * f_old[c >> 1] + src[(4 + j * 4 + c) * 32] * f_new[c >> 1];
      }
      const int ldo = n_kept * 64;
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const float inv = l_run[r] > 0.f ? 1.f / l_run[r] : 0.f;
        const int row = q0 + g + 8 * r;
        if (row < L) {
          uint16_t* dst = p.out + (static_cast<size_t>(b) * L + row) * ldo + hi * 64 + 2 * t4;
#pragma unroll
          for (int jd = 0; jd < 8; ++jd)
            *reinterpret_cast<uint32_t*>(dst + jd * 8) = pack_bf16x2(o[jd][2 * r] * inv, o[jd][2 * r + 1] * inv);
        }
      }
    }
    __syncthreads();        // K, V and the merge buffer are reused by the CTA's next item
  }
}

}  // namespace
}  // namespace sti
