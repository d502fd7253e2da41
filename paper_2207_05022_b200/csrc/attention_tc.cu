// Per-head attention on the 5th-generation tensor cores, for many tokens (Section 2.1: each attention head
// independently contributes one representation; Section 4.2: only the kept heads exist).
//
// One CTA per (sequence, kept head): the sequence's K and V (at most 512 keys x 64) are brought into shared
// memory once by TMA (128-byte swizzle, 128-key boxes) and stay there while the CTA walks the sequence's
// 128-query tiles.  Per query tile and 128-key chunk:
//   S = Q K^T      tcgen05.mma, M = 128 queries, N = 128 keys, K = 64        -> tensor memory
//   softmax        two threads per query row (64 keys each; they exchange their maxima through shared memory):
//                  tcgen05.ld S, running maximum and sum (online softmax), probabilities rounded to bf16 and
//                  written to shared memory in the operand layout
//   O_c = P V      tcgen05.mma, M = 128, N = 64 (head width), K = 128 keys; V is used as it lies in shared
//                  memory (keys x 64: the "MN-major" form of the B operand)   -> tensor memory
//   o = o * exp2(m_old - m_new) + O_c in the row's registers.
// Scores, probabilities and O_c are double-buffered by chunk parity: while the tensor core multiplies chunk c's
// probabilities with V and computes chunk c + 2's scores, the softmax warps are already on chunk c + 1.
// Warp 8 issues the TMA copies, warp 9 the MMAs (one elected lane), warps 0-7 are the softmax rows (warp w and
// w + 4 share the rows of tensor-memory lane quadrant w % 4; each keeps 32 of the 64 output columns).
// Every wait is bounded.
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_device.cuh"
#include "sti_kernels.h"

namespace sti {
namespace {

constexpr int kTcSoftmaxWarps = 8;                            // 4 lane quadrants x 2 threads per row
constexpr int kTcProducerWarp = kTcSoftmaxWarps, kTcMmaWarp = kTcSoftmaxWarps + 1;
constexpr int kTcThreads = 32 * (kTcSoftmaxWarps + 2);
constexpr int kTcQTile = 128, kTcChunk = 128, kTcHead = 64;
constexpr int kTcMaxSeq = 512;
constexpr uint32_t kTcBox = kTcChunk * kTcHead * 2;           // 16 KB: 128 rows x 64 bf16, one TMA box
constexpr uint32_t kTcOffXchg = 1024;                         // [softmax warps][32] row maxima, the same for row sums
constexpr uint32_t kTcOffQ = kTcOffXchg + 2 * kTcSoftmaxWarps * 32 * 4;   // 3072: after the barrier block and the exchange area
constexpr uint32_t kTcOffK = kTcOffQ + kTcBox;
constexpr uint32_t kTcOffV = kTcOffK + 4 * kTcBox;
constexpr uint32_t kTcOffP = kTcOffV + 4 * kTcBox;            // probabilities: two buffers of two boxes (128 rows x 64 keys)
constexpr uint32_t kTcSmem = kTcOffP + 4 * kTcBox;
static_assert(kTcOffQ % 1024 == 0 && kTcSmem <= 227 * 1024, "shared-memory layout");
constexpr uint32_t kTcTmemCols = 512;                         // S buffers at columns 0 and 128, O buffers at 256 and 320
constexpr uint32_t kTcColS = 0, kTcColO = 256;

struct TcBarriers {
  uint64_t kv_full;        // K and V of the sequence have landed
  uint64_t q_full;         // the query tile has landed
  uint64_t q_empty;        // the MMAs that read the query tile have completed
  uint64_t s_full[2];      // a score chunk is complete in tensor memory (buffer = chunk parity, here and below)
  uint64_t s_empty[2];     // ... and has been read by all softmax warps
  uint64_t p_full[2];      // a chunk's probabilities are in shared memory
  uint64_t o_full[2];      // a chunk's O_c is complete in tensor memory
  uint32_t tmem_base;
  volatile uint32_t abort;
};

// K-major operand with 128-byte swizzle is built by gemm_device.cuh's umma_smem_desc_sw128.  The same bytes read
// as an MN-major operand (V: rows are keys = the K dimension of P V, the 64 head features are contiguous): eight
// keys form one 1024-byte swizzle pattern, consecutive patterns follow each other (stride byte offset 1024); the
// 64 features are exactly one pattern wide, so the leading byte offset is never used.
__device__ __forceinline__ uint64_t umma_smem_desc_sw128_mn(uint32_t saddr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

// bf16 x bf16 -> fp32, M = 128; `b_mn_major`: the B operand's N dimension is the contiguous one.
__device__ __forceinline__ uint32_t umma_idesc_bf16_m128_b(uint32_t n, bool b_mn_major) {
  return umma_idesc_bf16_m128(n) | (b_mn_major ? (1u << 16) : 0u);
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// One lane polls, the warp takes its result (keeps the barrier word free of a warp's worth of pollers).  The poll
// does not sleep: these waits sit on the per-chunk critical path and are short.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, uint32_t lane) {
  uint32_t ok = 1;
  if (lane == 0) ok = mbar_wait_bounded(bar, parity) ? 1u : 0u;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

__global__ void __launch_bounds__(kTcThreads, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap qkv_map, uint16_t* __restrict__ out,
                    const int32_t* __restrict__ seq_lens, int n_kept, int batch, int L, int* __restrict__ err,
                    unsigned long long* stamps) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int hi = blockIdx.x, b = blockIdx.y;
  const int T = batch * L;
  if (tid == 0) { stamp_min(stamps, STAMP_FIRST_START); stamp_max(stamps, STAMP_LAST_START); }
  TcBarriers* bar = reinterpret_cast<TcBarriers*>(smem);
  const uint32_t sbase = smem_addr(smem);
  if ((sbase & 1023u) != 0 || L < 1 || L > kTcMaxSeq) {          // refuse rather than touch memory wrongly
    if (tid == 0) atomicCAS(err, ERR_NONE, ERR_BAD_JOB);
    return;
  }
  if (tid == 0) {
    mbar_init(smem_addr(&bar->kv_full), 1);
    mbar_init(smem_addr(&bar->q_full), 1);
    mbar_init(smem_addr(&bar->q_empty), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_addr(&bar->s_full[i]), 1);
      mbar_init(smem_addr(&bar->s_empty[i]), kTcSoftmaxWarps);   // one arrival per softmax warp
      mbar_init(smem_addr(&bar->p_full[i]), kTcSoftmaxWarps);
      mbar_init(smem_addr(&bar->o_full[i]), 1);
    }
    bar->abort = 0;
    mbar_fence_init();
    fence_proxy_async_smem();
  }
  if (warp == kTcProducerWarp) {
    tmem_alloc(smem_addr(&bar->tmem_base), kTcTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bar->tmem_base;
  pdl_launch_dependents();
  pdl_wait();                       // q, k, v (and possibly seq_lens) come from the preceding kernels
  if (tid == 0) stamp_min(stamps, STAMP_RELEASE);

  int valid = L;
  if (seq_lens != nullptr) {
    valid = seq_lens[b];
    valid = valid < 0 ? 0 : (valid > L ? L : valid);
  }
  const int n_qt = (L + kTcQTile - 1) / kTcQTile;
  const int nc = (valid + kTcChunk - 1) / kTcChunk;            // key chunks that hold at least one valid key
  const int q_row = (hi * 3 + 0) * T + b * L, k_row = (hi * 3 + 1) * T + b * L, v_row = (hi * 3 + 2) * T + b * L;
  const uint32_t q_sm = sbase + kTcOffQ, k_sm = sbase + kTcOffK, v_sm = sbase + kTcOffV, p_sm = sbase + kTcOffP;
  bool failed = false;

  if (warp == kTcProducerWarp) {
    // ---- producer: K and V of the sequence once, then one query tile at a time
    if (lane == 0 && nc > 0) {
      mbar_expect_tx(smem_addr(&bar->kv_full), 2u * nc * kTcBox);
      for (int c = 0; c < nc; ++c) {
        tma_load_2d(k_sm + c * kTcBox, &qkv_map, 0, k_row + c * kTcChunk, smem_addr(&bar->kv_full));
        tma_load_2d(v_sm + c * kTcBox, &qkv_map, 0, v_row + c * kTcChunk, smem_addr(&bar->kv_full));
      }
      for (int qt = 0; qt < n_qt; ++qt) {
        if (qt > 0 && !mbar_wait_bounded_relaxed(smem_addr(&bar->q_empty), (qt - 1) & 1)) { failed = true; break; }
        mbar_expect_tx(smem_addr(&bar->q_full), kTcBox);
        tma_load_2d(q_sm, &qkv_map, 0, q_row + qt * kTcQTile, smem_addr(&bar->q_full));
      }
    }
    __syncwarp();
  } else if (warp == kTcMmaWarp) {
    // ---- MMA issuer: the warp runs converged, one elected lane issues.  Buffers go by chunk parity; `used[]`
    // counts how often each has been used, which gives the barrier phases.
    if (nc > 0) {
      const uint32_t idesc_s = umma_idesc_bf16_m128_b(kTcChunk, false);
      const uint32_t idesc_o = umma_idesc_bf16_m128_b(kTcHead, true);
      const uint64_t q_desc = umma_smem_desc_sw128(q_sm), k_desc0 = umma_smem_desc_sw128(k_sm);
      const uint64_t p_desc0 = umma_smem_desc_sw128(p_sm), v_desc0 = umma_smem_desc_sw128_mn(v_sm);
      uint32_t used_s[2] = {0, 0}, used_p[2] = {0, 0};
      auto issue_scores = [&](int c) -> bool {                   // S = Q K_c^T into the score buffer of c's parity
        const uint32_t bi = c & 1;
        if (used_s[bi] > 0 && !warp_wait(smem_addr(&bar->s_empty[bi]), (used_s[bi] - 1) & 1, lane)) return false;
        tc_fence_after_sync();
        if (elect_one()) {
          umma_bf16_ss_x4(tmem + kTcColS + bi * kTcChunk, q_desc, k_desc0 + c * (kTcBox >> 4), 2, 2, idesc_s, 0u);
          umma_commit(smem_addr(&bar->s_full[bi]));
        }
        __syncwarp();
        ++used_s[bi];
        return true;
      };
      bool ok = warp_wait(smem_addr(&bar->kv_full), 0, lane);
      for (int qt = 0; ok && qt < n_qt; ++qt) {
        ok = warp_wait(smem_addr(&bar->q_full), qt & 1, lane);
        if (!ok) break;
        ok = issue_scores(0);
        for (int c = 0; ok && c < nc; ++c) {
          if (c + 1 < nc) ok = issue_scores(c + 1);              // the next chunk's scores run under this chunk's softmax
          if (!ok) break;
          if (c + 1 == nc) {                                     // all of this tile's score MMAs are issued: Q may go
            if (elect_one()) umma_commit(smem_addr(&bar->q_empty));
            __syncwarp();
          }
          const uint32_t bi = c & 1;
          ok = warp_wait(smem_addr(&bar->p_full[bi]), used_p[bi] & 1, lane);
          if (!ok) break;
          tc_fence_after_sync();
          if (elect_one()) {
            // O_c = P V_c: two boxes of 64 keys; per K = 16 step P moves 32 bytes in its swizzled row, V 16 rows
            const uint64_t vd = v_desc0 + c * (kTcBox >> 4), pd = p_desc0 + bi * (2 * kTcBox >> 4);
            const uint32_t od = tmem + kTcColO + bi * kTcHead;
            umma_bf16_ss_x4(od, pd, vd, 2, 2048 >> 4, idesc_o, 0u);
            umma_bf16_ss_x4(od, pd + (kTcBox >> 4), vd + (8192 >> 4), 2, 2048 >> 4, idesc_o, 1u);
            umma_commit(smem_addr(&bar->o_full[bi]));
          }
          __syncwarp();
          ++used_p[bi];
        }
      }
      if (!ok) failed = true;
    }
  } else {
    // ---- softmax rows: two threads per query row (TMEM lane), 64 keys and 32 output columns each
    const uint32_t quad = warp & 3, half = warp >> 2;
    const uint32_t row = quad * 32 + lane;
    const uint32_t t_lane = (quad * 32) << 16;
    const float scale = 0.125f * 1.4426950408889634f;            // 1/sqrt(64) * log2(e)
    const int ldo = n_kept * kTcHead;
    float* xmax = reinterpret_cast<float*>(smem + kTcOffXchg);   // [softmax warps][32]
    float* xsum = xmax + kTcSoftmaxWarps * 32;
    constexpr int kKeys = kTcChunk / 2, kCols = kTcHead / 2;
    const uint32_t partner = warp ^ 4;                           // the other half of the row
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1u + quad) : "memory"); };
    uint32_t used[2] = {0, 0};                                   // how often each buffer has been used (barrier phases)
    // A wait that runs out sets `failed` and is not repeated, but the loops run on to their end: the two warps of a
    // quadrant meet at a named barrier every chunk, and neither may leave the other waiting there.
    for (int qt = 0; qt < n_qt; ++qt) {
      float m = -INFINITY, l = 0.f, alpha_prev = 0.f;
      float o[kCols];
#pragma unroll
      for (int i = 0; i < kCols; ++i) o[i] = 0.f;
      // o = o * alpha + O_c of the chunk whose buffer is bi (the buffer's latest use)
      auto take_output = [&](uint32_t bi, float alpha) {
        if (!failed && !warp_wait(smem_addr(&bar->o_full[bi]), (used[bi] - 1) & 1, lane)) failed = true;
        tc_fence_after_sync();
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem + t_lane + kTcColO + bi * kTcHead + half * kCols, r);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < kCols; ++i) o[i] = fmaf(o[i], alpha, __uint_as_float(r[i]));
      };
      for (int c = 0; c < nc; ++c) {
        const uint32_t bi = c & 1;
        if (!failed && !warp_wait(smem_addr(&bar->s_full[bi]), used[bi] & 1, lane)) failed = true;
        tc_fence_after_sync();
        const uint32_t s_addr = tmem + t_lane + kTcColS + bi * kTcChunk + half * kKeys;
        // this thread's 64 scores of the row into registers (one pass over tensor memory)
        float sc[kKeys];
#pragma unroll
        for (int pc = 0; pc < 2; ++pc) {
          uint32_t r[32];
          tmem_ld_32x32b_x32(s_addr + pc * 32, r);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) sc[pc * 32 + i] = __uint_as_float(r[i]);
        }
        const int n_valid = valid - (c * kTcChunk + static_cast<int>(half) * kKeys);   // keys at and past it are padding
        if (n_valid < kKeys) {
#pragma unroll
          for (int i = 0; i < kKeys; ++i)
            if (i >= n_valid) sc[i] = -INFINITY;                 // exp2(-inf) = 0: padded keys get probability exactly 0
        }
        float mx4[4] = {sc[0], sc[1], sc[2], sc[3]};              // four independent chains
#pragma unroll
        for (int i = 4; i < kKeys; i += 4) {
          mx4[0] = fmaxf(mx4[0], sc[i]); mx4[1] = fmaxf(mx4[1], sc[i + 1]);
          mx4[2] = fmaxf(mx4[2], sc[i + 2]); mx4[3] = fmaxf(mx4[3], sc[i + 3]);
        }
        float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        // the row's other half: write, meet, read, meet (the second meeting frees the slot for the next chunk)
        xmax[warp * 32 + lane] = mx;
        pair_sync();
        mx = fmaxf(mx, xmax[partner * 32 + lane]);
        pair_sync();
        const float m_new = fmaxf(m, mx * scale);              // finite: the chunk holds at least one valid key
        const float alpha = fast_exp2(m - m_new);              // 0 for the first chunk (m = -inf)
        // probabilities (bf16) into shared memory, K-major with 128-byte swizzle: this thread's 64 keys are its own
        // box of the chunk's buffer (the MMAs that read the buffer two chunks ago are done: their O_c has been taken)
        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
        uint8_t* box = smem + kTcOffP + (bi * 2 + half) * kTcBox + row * 128;
#pragma unroll
        for (int q = 0; q < 8; ++q) {                          // eight keys = one 16-byte piece
          uint32_t pk[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int i = q * 8 + 2 * e;
            const float p0 = fast_exp2(fmaf(sc[i], scale, -m_new));
            const float p1 = fast_exp2(fmaf(sc[i + 1], scale, -m_new));
            sum4[e] += p0 + p1;
            pk[e] = pack_bf16x2(p0, p1);
          }
          *reinterpret_cast<uint4*>(box + ((static_cast<uint32_t>(q) ^ (row & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
        l = fmaf(l, alpha, (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));     // this thread's half of the row sum
        m = m_new;
        tc_fence_before_sync();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(smem_addr(&bar->s_empty[bi]));
          mbar_arrive(smem_addr(&bar->p_full[bi]));
        }
        ++used[bi];
        // the previous chunk's O_c (its P V product ran while this chunk's softmax did)
        if (c > 0) take_output(bi ^ 1, alpha_prev);
        alpha_prev = alpha;
      }
      if (nc > 0) take_output((nc - 1) & 1, alpha_prev);
      // the two halves of the row sum meet
      xsum[warp * 32 + lane] = l;
      pair_sync();
      l += xsum[partner * 32 + lane];
      pair_sync();                                             // the slot is free again for the next query tile
      const int qi = qt * kTcQTile + static_cast<int>(row);
      if (qi < L) {
        const float inv = l > 0.f ? 1.0f / l : 0.f;
        uint16_t* dst = out + (static_cast<size_t>(b) * L + qi) * ldo + hi * kTcHead + half * kCols;
#pragma unroll
        for (int i = 0; i < kCols; i += 8)
          *reinterpret_cast<uint4*>(dst + i) = make_uint4(pack_bf16x2(o[i] * inv, o[i + 1] * inv), pack_bf16x2(o[i + 2] * inv, o[i + 3] * inv),
                                                          pack_bf16x2(o[i + 4] * inv, o[i + 5] * inv), pack_bf16x2(o[i + 6] * inv, o[i + 7] * inv));
      }
    }
  }
  if (failed) {
    bar->abort = 1;
    if (lane == 0) atomicCAS(err, ERR_NONE, ERR_WAIT_TIMEOUT);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kTcProducerWarp) tmem_dealloc(tmem, kTcTmemCols);
  if (tid == 0) stamp_max(stamps, STAMP_LAST_END);
}

}  // namespace

cudaError_t attention_tc_configure() {
  return cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kTcSmem));
}

// `qkv_map`: TMA view of qkv as [3 * n_kept * T rows, 64 columns] bf16, boxes of 128 rows, 128-byte swizzle.
cudaError_t launch_attention_tc(const CUtensorMap& qkv_map, uint16_t* out, int n_kept, int batch, int seq,
                                const int32_t* seq_lens, int* err, cudaStream_t s, bool pdl, unsigned long long* stamps) {
  if (n_kept <= 0 || batch <= 0) return cudaSuccess;
  if (seq < 1 || seq > kTcMaxSeq) return cudaErrorInvalidValue;
  return launch_kernel(attention_tc_kernel, dim3(n_kept, batch), dim3(kTcThreads), kTcSmem, s, pdl, qkv_map, out, seq_lens,
                       n_kept, batch, seq, err, stamps);
}

}  // namespace sti
