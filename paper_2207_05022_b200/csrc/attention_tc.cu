// Per-head attention on the tcgen05 tensor cores with TWO query tiles in flight per CTA (Section 2.1: softmax(Q K^T /
// sqrt 64) V per kept head; padded keys get probability exactly 0).
//
// One CTA per (sequence, kept head): K and V of the sequence (at most 512 keys) stay in shared memory.  Two groups of
// four softmax warps each own one 128-query tile at a time (tiles g, g + 2, ... for group g) with ONE thread per query
// row, so a row's maximum and sum never leave the thread.  The MMA warp serves the groups in turn: while one group is
// busy with its exponentials the other's S = Q K^T or O_c = P V runs, and a group that waits for the tensor core
// leaves the issue slots to the other.
//
//   warps 0-3, 4-7  softmax group 0 / 1: thread = query row = tensor-memory lane.  Per 128-key chunk: pass 1 reads
//                   the scores (tcgen05.ld) for the row maximum; then the previous chunk's O_c is folded into the
//                   register accumulator (which also says that the probability buffer is free); pass 2 reads the
//                   scores again, exponentiates, sums, and writes the bf16 probabilities into shared memory in the
//                   swizzled K-major layout the second MMA reads
//   warp 8          TMA: K and V once (a barrier per 128-key chunk, so the first scores start after 16 KB of K have
//                   landed, not after the sequence's 128 KB), query tiles into the two slots
//   warp 9          MMA issuer: for each group in turn  S(next chunk)  and  O_c = P V(this chunk)
//
// Tensor memory: S of group g at columns 128 g, O_c of group g at 256 + 64 g.  Every barrier has one class of
// waiters that meets every phase in order.  Waits are bounded; a role that gives up sets the abort flag and the
// status word, the others run out of their own waits.
#include <cuda_bf16.h>

#include "gemm_device.cuh"
#include "sti_kernels.h"

namespace sti {
namespace {

constexpr int kTcGroupWarps = 4, kTcGroups = 2;
constexpr int kTcProducerWarp = kTcGroupWarps * kTcGroups, kTcMmaWarp = kTcProducerWarp + 1;
constexpr int kTcThreads = 32 * (kTcMmaWarp + 1);
constexpr int kTcQTile = 128, kTcChunk = 128, kTcHead = 64;
constexpr int kTcMaxSeq = 512;
constexpr uint32_t kTcBox = kTcChunk * kTcHead * 2;              // 16 KB: 128 rows x 64 bf16, one TMA box
constexpr uint32_t kTcOffQ = 3072;                               // two query slots
constexpr uint32_t kTcOffK = kTcOffQ + 2 * kTcBox;
constexpr uint32_t kTcOffV = kTcOffK + 4 * kTcBox;
constexpr uint32_t kTcOffP = kTcOffV + 4 * kTcBox;               // probabilities: per group two boxes (128 rows x 64 keys)
constexpr uint32_t kTcSmem = kTcOffP + 4 * kTcBox;
static_assert(kTcOffQ % 1024 == 0 && kTcSmem <= 227 * 1024, "shared-memory layout");
constexpr uint32_t kTcTmemCols = 512;
constexpr uint32_t kTcColS = 0, kTcColO = 256;

struct TcBarriers {
  uint64_t k_full[4];      // key chunk c has landed (one phase each: K and V are loaded once per CTA)
  uint64_t v_full[4];      // value chunk c has landed
  uint64_t q_full[2];      // a query tile has landed in the group's slot
  uint64_t q_empty[2];     // the score MMAs of the slot's tile have completed
  uint64_t s_full[2];      // the group's score chunk is complete in tensor memory
  uint64_t s_empty[2];     // the group has read its score chunk for the last time (the chunk's last tcgen05.ld is complete)
  uint64_t p_full[2];      // the group's probabilities are in shared memory
  uint64_t o_full[2];      // the group's O_c is complete in tensor memory (and its probabilities have been read)
  uint32_t tmem_base;
  volatile uint32_t abort;
};

__device__ __forceinline__ uint64_t umma_smem_desc_sw128_mn(uint32_t saddr) {    // V: keys are rows, the 64 features contiguous
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// tcgen05.wait::ld that names the registers of one earlier 32-column load as read-write operands: the compiler then
// keeps those values where the load put them until here and orders every later use after the wait, so the load may
// stay in flight while the thread works on other registers.
__device__ __forceinline__ void tmem_wait_ld_x32(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                 "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                 "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}

__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, uint32_t lane, volatile uint32_t* abort) {
  uint32_t ok = 1;
  if (lane == 0) ok = *abort ? 0u : (mbar_wait_bounded(bar, parity) ? 1u : 0u);
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
  if ((sbase & 1023u) != 0 || L < 1 || L > kTcMaxSeq) {
    if (tid == 0) atomicCAS(err, ERR_NONE, ERR_BAD_JOB);
    return;
  }
  if (tid == 0) {
    for (int c = 0; c < 4; ++c) { mbar_init(smem_addr(&bar->k_full[c]), 1); mbar_init(smem_addr(&bar->v_full[c]), 1); }
    for (int g = 0; g < 2; ++g) {
      mbar_init(smem_addr(&bar->q_full[g]), 1);
      mbar_init(smem_addr(&bar->q_empty[g]), 1);
      mbar_init(smem_addr(&bar->s_full[g]), 1);
      mbar_init(smem_addr(&bar->s_empty[g]), kTcGroupWarps);
      mbar_init(smem_addr(&bar->p_full[g]), kTcGroupWarps);
      mbar_init(smem_addr(&bar->o_full[g]), 1);
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
  pdl_wait();
  if (tid == 0) stamp_min(stamps, STAMP_RELEASE);

  int valid = L;
  if (seq_lens != nullptr) {
    valid = seq_lens[b];
    valid = valid < 0 ? 0 : (valid > L ? L : valid);
  }
  const int n_qt = (L + kTcQTile - 1) / kTcQTile;
  const int nc = (valid + kTcChunk - 1) / kTcChunk;              // key chunks with at least one valid key
  const int q_row = (hi * 3 + 0) * T + b * L, k_row = (hi * 3 + 1) * T + b * L, v_row = (hi * 3 + 2) * T + b * L;
  const uint32_t q_sm = sbase + kTcOffQ, k_sm = sbase + kTcOffK, v_sm = sbase + kTcOffV, p_sm = sbase + kTcOffP;
  // tiles of group g: g, g + 2, ...; steps of a group = (its tile number i, chunk c) in order
  auto tiles_of = [&](int g) { return n_qt > g ? (n_qt - g + 1) / 2 : 0; };
  bool failed = false;

  if (warp == kTcProducerWarp) {
    if (lane == 0 && nc > 0) {
      // in the order the MMA warp needs them: the first key chunk, the first two query tiles, then V and K chunk by chunk
      auto load_k = [&](int c) {
        mbar_expect_tx(smem_addr(&bar->k_full[c]), kTcBox);
        tma_load_2d(k_sm + c * kTcBox, &qkv_map, 0, k_row + c * kTcChunk, smem_addr(&bar->k_full[c]));
      };
      auto load_v = [&](int c) {
        mbar_expect_tx(smem_addr(&bar->v_full[c]), kTcBox);
        tma_load_2d(v_sm + c * kTcBox, &qkv_map, 0, v_row + c * kTcChunk, smem_addr(&bar->v_full[c]));
      };
      auto load_q = [&](int qt) {
        const uint32_t g = qt & 1;
        mbar_expect_tx(smem_addr(&bar->q_full[g]), kTcBox);
        tma_load_2d(q_sm + g * kTcBox, &qkv_map, 0, q_row + qt * kTcQTile, smem_addr(&bar->q_full[g]));
      };
      load_k(0);
      for (int qt = 0; qt < n_qt && qt < 2; ++qt) load_q(qt);
      load_v(0);
      for (int c = 1; c < nc; ++c) { load_k(c); load_v(c); }
      for (int qt = 2; qt < n_qt; ++qt) {
        const uint32_t g = qt & 1, i = qt >> 1;                  // the group's i-th tile
        if (!mbar_wait_bounded_relaxed(smem_addr(&bar->q_empty[g]), (i - 1) & 1)) { failed = true; break; }
        load_q(qt);
      }
    }
    __syncwarp();
  } else if (warp == kTcMmaWarp) {
    if (nc > 0) {
      const uint32_t idesc_s = umma_idesc_bf16_m128(kTcChunk);
      const uint32_t idesc_o = umma_idesc_bf16_m128(kTcHead) | (1u << 16);       // B (V) is MN-major
      const uint64_t q_desc0 = umma_smem_desc_sw128(q_sm), k_desc0 = umma_smem_desc_sw128(k_sm);
      const uint64_t p_desc0 = umma_smem_desc_sw128(p_sm), v_desc0 = umma_smem_desc_sw128_mn(v_sm);
      const int steps[2] = {tiles_of(0) * nc, tiles_of(1) * nc};
      // S of step n of group g into the group's score columns; a new tile first waits for its queries
      auto issue_scores = [&](int g, int n) -> bool {
        const int i = n / nc, c = n - i * nc;
        if (c == 0 && !warp_wait(smem_addr(&bar->q_full[g]), i & 1, lane, &bar->abort)) return false;
        if (i == 0 && !warp_wait(smem_addr(&bar->k_full[c]), 0, lane, &bar->abort)) return false;   // later tiles: long landed
        tc_fence_after_sync();
        if (elect_one()) {
          umma_bf16_ss_x4(tmem + kTcColS + g * kTcChunk, q_desc0 + g * (kTcBox >> 4), k_desc0 + c * (kTcBox >> 4), 2, 2,
                          idesc_s, 0u);
          umma_commit(smem_addr(&bar->s_full[g]));
          if (c + 1 == nc && i + 1 < tiles_of(g)) umma_commit(smem_addr(&bar->q_empty[g]));   // the slot's next tile may land
        }
        __syncwarp();
        return true;
      };
      bool ok = true;
      for (int g = 0; ok && g < 2; ++g)
        if (steps[g] > 0) ok = issue_scores(g, 0);
      // Serve whichever group has something ready: its scores read for the last time -> the next chunk's S; its
      // probabilities in shared memory -> O_c = P V.  Neither group waits for the other's softmax.
      int next_s[2] = {1, 1}, next_pv[2] = {0, 0};               // S of step 0 is issued above
      uint64_t t_idle = global_timer_ns();
      while (ok && (next_pv[0] < steps[0] || next_pv[1] < steps[1])) {
        bool progressed = false;
        for (int g = 0; ok && g < 2; ++g) {
          if (next_s[g] < steps[g]) {                            // S(next_s) needs the reads of step next_s - 1 done
            uint32_t ready = 0;
            if (lane == 0) ready = mbar_try_wait(smem_addr(&bar->s_empty[g]), (next_s[g] - 1) & 1);
            if (__shfl_sync(0xffffffffu, ready, 0)) {
              ok = issue_scores(g, next_s[g]);
              if (!ok) break;
              ++next_s[g];
              progressed = true;
            }
          }
          const int n = next_pv[g];
          if (n < steps[g]) {
            uint32_t ready = 0;
            if (lane == 0) ready = mbar_try_wait(smem_addr(&bar->p_full[g]), n & 1);
            if (__shfl_sync(0xffffffffu, ready, 0)) {
              const int c = n % nc;
              if (n < nc && !warp_wait(smem_addr(&bar->v_full[c]), 0, lane, &bar->abort)) { ok = false; break; }
              tc_fence_after_sync();
              if (elect_one()) {
                // O_c = P V_c: two boxes of 64 keys; per K = 16 step P moves 32 bytes in its swizzled row, V 16 rows
                const uint64_t vd = v_desc0 + c * (kTcBox >> 4), pd = p_desc0 + g * (2 * kTcBox >> 4);
                const uint32_t od = tmem + kTcColO + g * kTcHead;
                umma_bf16_ss_x4(od, pd, vd, 2, 2048 >> 4, idesc_o, 0u);
                umma_bf16_ss_x4(od, pd + (kTcBox >> 4), vd + (8192 >> 4), 2, 2048 >> 4, idesc_o, 1u);
                umma_commit(smem_addr(&bar->o_full[g]));
              }
              __syncwarp();
              next_pv[g] = n + 1;
              progressed = true;
            }
          }
        }
        if (progressed) {
          t_idle = global_timer_ns();
        } else {
          uint32_t give_up = 0;
          if (lane == 0) give_up = (bar->abort || global_timer_ns() - t_idle > 2000000000ull) ? 1u : 0u;
          if (__shfl_sync(0xffffffffu, give_up, 0)) ok = false;
        }
      }
      if (!ok) failed = true;
    }
  } else {
    // ---- softmax group g: thread = query row
    const uint32_t g = warp >> 2, quad = warp & 3;
    const uint32_t row = quad * 32 + lane;
    const uint32_t t_lane = (quad * 32) << 16;
    const float scale = 0.125f * 1.4426950408889634f;            // 1/sqrt(64) * log2(e)
    const int ldo = n_kept * kTcHead;
    const int my_tiles = tiles_of(static_cast<int>(g));
    const uint32_t s_addr = tmem + t_lane + kTcColS + g * kTcChunk;
    const uint32_t o_addr = tmem + t_lane + kTcColO + g * kTcHead;
    uint8_t* prow = smem + kTcOffP + g * 2 * kTcBox + row * 128;   // this row inside the group's first probability box
    uint32_t n = 0;                                              // the group's step number (barrier phases)
    for (int i = 0; i < my_tiles && nc > 0; ++i) {
      const int qt = 2 * i + static_cast<int>(g);
      float m = -INFINITY, l = 0.f, alpha_prev = 0.f;
      float o[kTcHead];
#pragma unroll
      for (int k = 0; k < kTcHead; ++k) o[k] = 0.f;
      // o = o * alpha + O_c of the previous step (its P V product is complete: the probability buffer is free too)
      auto take_output = [&](uint32_t step, float alpha) {
        if (!failed && !warp_wait(smem_addr(&bar->o_full[g]), step & 1, lane, &bar->abort)) failed = true;
        tc_fence_after_sync();
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint32_t r[32];
          tmem_ld_32x32b_x32(o_addr + h * 32, r);
          tc_wait_ld();
#pragma unroll
          for (int k = 0; k < 32; ++k) o[h * 32 + k] = fmaf(o[h * 32 + k], alpha, __uint_as_float(r[k]));
        }
      };
      for (int c = 0; c < nc; ++c, ++n) {
        if (!failed && !warp_wait(smem_addr(&bar->s_full[g]), n & 1, lane, &bar->abort)) failed = true;
        tc_fence_after_sync();
        const int n_valid = valid - c * kTcChunk;                // keys of this chunk at and past it are padding
        // pass 1: the row maximum
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        uint32_t rr[2][32];                                      // the next 32 scores load while these are worked on
        tmem_ld_32x32b_x32(s_addr, rr[0]);
#pragma unroll
        for (int pc = 0; pc < 4; ++pc) {
          uint32_t (&r)[32] = rr[pc & 1];
          tmem_wait_ld_x32(r);
          if (pc + 1 < 4) tmem_ld_32x32b_x32(s_addr + (pc + 1) * 32, rr[(pc + 1) & 1]);
          if (n_valid < (pc + 1) * 32) {
#pragma unroll
            for (int k = 0; k < 32; ++k)
              if (pc * 32 + k >= n_valid) r[k] = 0xff800000u;    // -inf
          }
#pragma unroll
          for (int k = 0; k < 32; k += 4) {
            mx4[0] = fmaxf(mx4[0], __uint_as_float(r[k])); mx4[1] = fmaxf(mx4[1], __uint_as_float(r[k + 1]));
            mx4[2] = fmaxf(mx4[2], __uint_as_float(r[k + 2])); mx4[3] = fmaxf(mx4[3], __uint_as_float(r[k + 3]));
          }
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        const float m_new = fmaxf(m, mx * scale);                // finite: the chunk holds at least one valid key
        const float alpha = fast_exp2(m - m_new);                  // 0 for the tile's first chunk (m = -inf)
        // the previous chunk's O_c; after this the probability buffer may be overwritten
        if (c > 0) take_output(n - 1, alpha_prev);
        alpha_prev = alpha;
        // pass 2: probabilities (bf16) into shared memory, K-major with 128-byte swizzle, two boxes of 64 keys
        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
        tmem_ld_32x32b_x32(s_addr, rr[0]);
#pragma unroll
        for (int pc = 0; pc < 4; ++pc) {
          uint32_t (&r)[32] = rr[pc & 1];
          tmem_wait_ld_x32(r);
          if (pc + 1 < 4) {
            tmem_ld_32x32b_x32(s_addr + (pc + 1) * 32, rr[(pc + 1) & 1]);
          } else {                                               // the scores are in registers: their buffer may be refilled
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_addr(&bar->s_empty[g]));
          }
          if (n_valid < (pc + 1) * 32) {
#pragma unroll
            for (int k = 0; k < 32; ++k)
              if (pc * 32 + k >= n_valid) r[k] = 0xff800000u;
          }
          uint8_t* box = prow + (pc >> 1) * kTcBox;
#pragma unroll
          for (int q = 0; q < 4; ++q) {                          // eight keys = one 16-byte piece
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float p0 = fast_exp2(fmaf(__uint_as_float(r[q * 8 + 2 * e]), scale, -m_new));
              const float p1 = fast_exp2(fmaf(__uint_as_float(r[q * 8 + 2 * e + 1]), scale, -m_new));
              sum4[e] += p0 + p1;
              pk[e] = pack_bf16x2(p0, p1);
            }
            const uint32_t piece = static_cast<uint32_t>((pc & 1) * 4 + q);
            *reinterpret_cast<uint4*>(box + ((piece ^ (row & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
        l = fmaf(l, alpha, (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));
        m = m_new;
        tc_fence_before_sync();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_addr(&bar->p_full[g]));
      }
      take_output(n - 1, alpha_prev);
      const int qi = qt * kTcQTile + static_cast<int>(row);
      if (qi < L) {
        const float inv = l > 0.f ? 1.0f / l : 0.f;
        uint16_t* dst = out + (static_cast<size_t>(b) * L + qi) * ldo + hi * kTcHead;
#pragma unroll
        for (int k = 0; k < kTcHead; k += 8)
          *reinterpret_cast<uint4*>(dst + k) = make_uint4(pack_bf16x2(o[k] * inv, o[k + 1] * inv), pack_bf16x2(o[k + 2] * inv, o[k + 3] * inv),
                                                          pack_bf16x2(o[k + 4] * inv, o[k + 5] * inv), pack_bf16x2(o[k + 6] * inv, o[k + 7] * inv));
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
