// Whole-layer kernel for sm_100a: the seven steps of one transformer layer over the kept shards
// (Section 2.1 layer maths, Section 4.2 shard decode) in ONE launch, for the few-token regime where
// a layer is a chain of latencies rather than a bandwidth or tensor problem.
//
// A grid of G <= 148 CTAs (one per SM, 512 threads) walks the steps in order:
//   QKV GEMM -> attention -> O projection -> residual+LayerNorm -> FFN1+GELU -> FFN2 -> residual+LayerNorm
// Every GEMM step is the weight-stationary fused dequant-GEMM of dqgemm.cu (same decode, same TMA ring,
// same tcgen05/TMEM pipeline, same epilogues) with CTA i taking tile-job i of the step.  Steps are
// separated by a grid-wide barrier (one atomic counter per launch).  The barrier is split: a CTA
// arrives, then decodes the weight tile of its NEXT GEMM step into the shared memory its finished
// step no longer needs, and only then waits - so index unpack, table lookup and the DRAM latency of
// the packed shards overlap the other CTAs' tails instead of following them.
//
// Shared memory map (offsets from the 1024-aligned base):
//   [0, 256)      mbarriers, TMEM base, abort flag          [256, 512)  LayerNorm reduction scratch
//   [512, 3072)   header slot 0: bias (512 B) + 16 segment tables (128 B each)
//   [3072, 5632)  header slot 1 (consecutive GEMM steps alternate, so a tile can be decoded ahead)
//   [6144, ...)   activation ring of the running GEMM step / K, V and merge buffers of attention
//   [..., top)    weight tile of the running or the next GEMM step, placed at the top end
// Every wait (mbarrier or grid barrier) is bounded; a CTA that gives up sets the status word, skips
// the rest of its work, frees its tensor memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "gemm_device.cuh"

namespace sti {
namespace {

constexpr uint32_t kSlotOff0 = 512, kSlotBytes = 2560, kSlotOff1 = kSlotOff0 + kSlotBytes;
constexpr uint32_t kLowOff = 6144;                       // 1024-aligned start of the activation area
constexpr uint32_t kFusedTotal = 226 * 1024;             // usable bytes after the alignment slack
constexpr uint32_t kFusedTmemCols = 256;                 // two accumulators of up to 128 columns
constexpr int kAttnKStride = 64 + 8;                     // bf16 per K / V row in shared memory
constexpr uint32_t kAttnMergeBytes = 3 * 4 * 32 * 36 * 4;   // three key-split partners x four query groups

struct FusedScratch {                // lives at offset 256
  float red[2][16];                  // LayerNorm: per row group, one partial per warp
  uint32_t skip[4];                  // GEMM step g has no valid job on this CTA
  uint32_t where;                    // first wait that ran out: (step << 4) | kind, for the status word
};

// ---------------------------------------------------------------------------------------
// Grid-wide barrier, split into arrive and wait.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void grid_arrive(unsigned int* ctr, uint32_t tid) {
  __syncthreads();                                       // the CTA's writes of this step are done
  if (tid == 0) {
    __threadfence();
    atomicAdd(ctr, 1u);
  }
}
// false: the wait ran out (about three seconds) or the CTA had already given up
__device__ __forceinline__ bool grid_wait(unsigned int* ctr, unsigned int target, SmemHeader* hdr, uint32_t* where,
                                          uint32_t code, uint32_t tid) {
  if (tid == 0 && hdr->abort == 0) {
    bool ok = false;
    const uint64_t t0 = global_timer_ns();
    for (;;) {
      unsigned int v = 0;
#pragma unroll 1
      for (int i = 0; i < 64 && !ok; ++i) {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
        ok = v >= target;
      }
      if (ok || global_timer_ns() - t0 > 3000000000ull) break;     // longer than the mbarrier waits inside a step
    }
    if (!ok) { hdr->abort = 1; atomicCAS(where, 0u, code); }
    // what other CTAs wrote with ordinary stores is read next through TMA (async proxy) as well
    asm volatile("fence.proxy.async;" ::: "memory");
  }
  __syncthreads();
  return hdr->abort == 0;
}

// ---------------------------------------------------------------------------------------
// GEMM step, part 1: tables, bias and the decoded weight tile of this CTA's job.
// Reads only weights, descriptors and parameters - may run before the data dependency is met.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void gemm_prologue(const FusedGemm& g, int gi, uint32_t cta, uint8_t* smem, uint32_t slot_off,
                                              int* err, uint32_t tid) {
  FusedScratch* sc = reinterpret_cast<FusedScratch*>(smem + 256);
  const uint32_t n_items = static_cast<uint32_t>(g.n_jobs) * static_cast<uint32_t>(g.m_ctas);
  if (cta >= n_items) return;                            // uniform over the CTA
  const Job job = g.jobs[cta % static_cast<uint32_t>(g.n_jobs)];
  const uint32_t n_rows = job.n_rows, k_total = job.k_total;
  const bool bad = job.n_seg == 0 || job.n_seg > kMaxSegs || (n_rows != 32 && n_rows != 64 && n_rows != 128) ||
                   (k_total % kChunkK) != 0 || k_total == 0 || n_rows * k_total * 2 > g.w_bytes ||
                   g.n_stages < 2 || g.n_stages > kMaxStages || (g.bps != 1 && g.bps != 2 && g.bps != 4) ||
                   kLowOff + g.n_stages * g.bps * kBoxBytes + g.w_bytes > kFusedTotal;
  if (tid == 0) sc->skip[gi] = bad ? 1u : 0u;
  if (bad) {
    if (tid == 0) atomicCAS(err, ERR_NONE, ERR_BAD_JOB);
    return;
  }
  float* bias_sm = reinterpret_cast<float*>(smem + slot_off);
  uint16_t* tables = reinterpret_cast<uint16_t*>(smem + slot_off + 512);
  load_tables(job, g.segs, tables, tid);
  if (tid < n_rows) bias_sm[tid] = job.bias_off >= 0 ? __ldg(g.bias + job.bias_off + tid) : 0.f;
  __syncthreads();
  decode_weight_tile(job, g.segs, tables, smem + kFusedTotal - g.w_bytes, tid);
}

// ---------------------------------------------------------------------------------------
// GEMM step, part 2: activation tiles through the TMA ring, tcgen05 MMAs into TMEM, epilogue.
// ---------------------------------------------------------------------------------------
template <typename OutT, bool GELU>
__device__ __forceinline__ void drain_tile(uint32_t taddr, uint32_t col0, uint32_t col1, const float* bias_sm, OutT* drow,
                                           bool row_ok) {
  for (uint32_t col = col0; col < col1; col += 16) {
    uint32_t r[16];
    tmem_ld_32x32b_x16(taddr + col, r);
    tc_wait_ld();
    if (row_ok) {
      float v[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const float a = __uint_as_float(r[i]) + bias_sm[col + i];
        v[i] = GELU ? gelu_erf(a) : a;
      }
      store_row16<OutT>(drow + col, v);
    }
  }
}

// Returns false when a bounded wait ran out.
__device__ __forceinline__ bool gemm_main(const FusedGemm& g, int gi, uint32_t cta, int T, uint8_t* smem, uint32_t slot_off,
                                          uint32_t tmem_base, uint32_t tid) {
  SmemHeader* hdr = reinterpret_cast<SmemHeader*>(smem);
  FusedScratch* sc = reinterpret_cast<FusedScratch*>(smem + 256);
  const uint32_t lane = tid & 31, warp = tid >> 5;
  const uint32_t n_items = static_cast<uint32_t>(g.n_jobs) * static_cast<uint32_t>(g.m_ctas);
  if (cta >= n_items) return true;
  __syncthreads();
  if (sc->skip[gi]) return true;
  // fresh barriers for this step: the previous step on this CTA has drained completely
  if (tid == 0) {
    for (uint32_t s = 0; s < g.n_stages; ++s) {
      mbar_init(smem_addr(&hdr->full[s]), 1);
      mbar_init(smem_addr(&hdr->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_addr(&hdr->acc_full[b]), 1);
      mbar_init(smem_addr(&hdr->acc_empty[b]), kEpilogueWarps);
    }
    mbar_init(smem_addr(&hdr->drain), 1);
    mbar_fence_init();
    fence_proxy_async_smem();
  }
  __syncthreads();

  const uint32_t job_i = cta % static_cast<uint32_t>(g.n_jobs), my = cta / static_cast<uint32_t>(g.n_jobs);
  const uint32_t m_ctas = static_cast<uint32_t>(g.m_ctas);
  const Job job = g.jobs[job_i];
  const uint32_t n_rows = job.n_rows, k_total = job.k_total;
  const float* bias_sm = reinterpret_cast<const float*>(smem + slot_off);
  uint8_t* xsm = smem + kLowOff;
  uint8_t* wsm = smem + kFusedTotal - g.w_bytes;
  const uint32_t n_stages = g.n_stages, bps = g.bps;
  const uint32_t stage_bytes = bps * kBoxBytes;
  const int n_mtiles = (T + kTileM - 1) / kTileM;
  const uint32_t n_boxes = k_total / kChunkK;
  const uint32_t n_chunks = (n_boxes + bps - 1) / bps;
  const uint32_t my_mtiles = my < static_cast<uint32_t>(n_mtiles) ? (n_mtiles - my + m_ctas - 1) / m_ctas : 0;
  const uint32_t total = my_mtiles * n_chunks;
  const uint32_t xsm_addr = smem_addr(xsm);
  const uint32_t rot = job_i % n_chunks;       // CTAs walk K in rotated order (L2 lines are not hit together)
  bool failed = false;

  if (warp == 0) {
    // ---- producer
    if (lane == 0) {
      uint32_t c = 0, stage = 0, phase = 0, kcr = rot, kc = 0, ti = 0;
      for (; c < total; ++c) {
        if (c >= n_stages) {
          if (!mbar_wait_bounded_relaxed(smem_addr(&hdr->empty[stage]), phase)) {
            failed = true; atomicCAS(&sc->where, 0u, (static_cast<uint32_t>(gi) << 4) | 2u); break;
          }
        }
        const uint32_t bar = smem_addr(&hdr->full[stage]);
        const uint32_t box0 = kcr * bps;
        const uint32_t nb = n_boxes - box0 < bps ? n_boxes - box0 : bps;
        mbar_expect_tx(bar, nb * kBoxBytes);
        for (uint32_t b = 0; b < nb; ++b)
          tma_load_2d(xsm_addr + stage * stage_bytes + b * kBoxBytes, &g.xmap,
                      static_cast<int>(job.x_koff + (box0 + b) * kChunkK),
                      static_cast<int>((my + ti * m_ctas) * kTileM), bar);
        if (++stage == n_stages) { stage = 0; if (c >= n_stages) phase ^= 1; }
        if (++kcr == n_chunks) kcr = 0;
        if (++kc == n_chunks) { kc = 0; ++ti; }
      }
      if (failed) {
        // give every copy this CTA requested a bounded chance to land before it moves on
        const uint32_t first = c > n_stages ? c - n_stages : 0;
        for (uint32_t q = first; q < c; ++q)
          (void)mbar_wait_bounded(smem_addr(&hdr->full[q % n_stages]), (q / n_stages) & 1);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- MMA issuer: converged warp, one elected lane issues
    const uint32_t idesc = umma_idesc_bf16_m128(n_rows);
    const uint32_t w_lbo = n_rows * 16;
    const uint64_t a_desc0 = umma_smem_desc_sw128(xsm_addr);
    const uint64_t b_desc0 = umma_smem_desc(smem_addr(wsm), w_lbo, 128);
    const uint32_t a_stage_step = stage_bytes >> 4, a_box_step = kBoxBytes >> 4;
    const uint32_t b_ks_step = (2 * w_lbo) >> 4, b_chunk_step = 4 * b_ks_step;
    uint32_t stage = 0, phase = 0, kc = 0, kcr = rot, ti = 0, issued = 0;
    for (uint32_t c = 0; c < total; ++c) {
      const uint32_t buf = ti & 1;
      bool ok = true;
      if (kc == 0 && ti >= 2)
        ok = __all_sync(0xffffffffu, mbar_wait_bounded(smem_addr(&hdr->acc_empty[buf]), ((ti >> 1) - 1) & 1));
      if (!ok && lane == 0) atomicCAS(&sc->where, 0u, (static_cast<uint32_t>(gi) << 4) | 4u);
      if (ok) {
        ok = __all_sync(0xffffffffu, mbar_wait_bounded(smem_addr(&hdr->full[stage]), phase));
        if (!ok && lane == 0) atomicCAS(&sc->where, 0u, (static_cast<uint32_t>(gi) << 4) | 3u);
      }
      if (!ok) { failed = true; break; }
      tc_fence_after_sync();
      const uint32_t box0 = kcr * bps;
      const uint32_t nb = n_boxes - box0 < bps ? n_boxes - box0 : bps;
      const uint64_t da0 = a_desc0 + stage * a_stage_step;
      const uint64_t db0 = b_desc0 + box0 * b_chunk_step;
      const uint32_t d_addr = tmem_base + buf * n_rows;
      if (elect_one()) {
        uint64_t da = da0, db = db0;
        umma_bf16_ss_x4(d_addr, da, db, 2, b_ks_step, idesc, kc != 0 ? 1u : 0u);
        for (uint32_t b = 1; b < nb; ++b) {
          da += a_box_step;
          db += b_chunk_step;
          umma_bf16_ss_x4(d_addr, da, db, 2, b_ks_step, idesc, 1u);
        }
        if (c + n_stages < total) umma_commit(smem_addr(&hdr->empty[stage]));
        if (kc + 1 == n_chunks) umma_commit(smem_addr(&hdr->acc_full[buf]));
      }
      __syncwarp();
      issued = c + 1;
      if (++stage == n_stages) { stage = 0; phase ^= 1; }
      if (++kcr == n_chunks) kcr = 0;
      if (++kc == n_chunks) { kc = 0; ++ti; }
    }
    if (failed && issued > 0) {
      if (elect_one()) umma_commit(smem_addr(&hdr->drain));
      __syncwarp();
      (void)mbar_wait_bounded(smem_addr(&hdr->drain), 0);
    }
  } else if (warp >= kEpilogueWarp0 && warp < kEpilogueWarp0 + kEpilogueWarps) {
    // ---- epilogue: warp w owns TMEM lanes 32*(w%4).. (token rows) and one half of the columns
    const uint32_t q = warp & 3, half = (warp - kEpilogueWarp0) >> 2, ncol = n_rows / 2;
    for (uint32_t ti = 0; ti < my_mtiles; ++ti) {
      const uint32_t buf = ti & 1;
      uint32_t ok = 1;
      if (lane == 0) ok = mbar_wait_bounded_relaxed(smem_addr(&hdr->acc_full[buf]), (ti >> 1) & 1) ? 1u : 0u;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) {
        failed = true;
        if (lane == 0) atomicCAS(&sc->where, 0u, (static_cast<uint32_t>(gi) << 4) | 5u);
        break;
      }
      tc_fence_after_sync();
      const int t = static_cast<int>((my + ti * m_ctas) * kTileM + q * 32 + lane);
      const size_t row_off = (static_cast<size_t>(job.out_mat) * T + (t < T ? t : 0)) * g.ldo + job.out_col;
      const uint32_t taddr = tmem_base + ((q * 32) << 16) + buf * n_rows;
      const uint32_t c0 = half * ncol, c1 = (half + 1) * ncol;
      if (g.kind == GEMM_BF16_TO_F32)
        drain_tile<float, false>(taddr, c0, c1, bias_sm, static_cast<float*>(g.out) + row_off, t < T);
      else if (g.kind == GEMM_BF16_TO_BF16_GELU)
        drain_tile<__nv_bfloat16, true>(taddr, c0, c1, bias_sm, static_cast<__nv_bfloat16*>(g.out) + row_off, t < T);
      else
        drain_tile<__nv_bfloat16, false>(taddr, c0, c1, bias_sm, static_cast<__nv_bfloat16*>(g.out) + row_off, t < T);
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_addr(&hdr->acc_empty[buf]));
    }
  }
  if (failed) hdr->abort = 1;
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  // the step has drained: retire its barriers, the next GEMM step initialises them afresh
  if (tid == 0) {
    for (uint32_t s = 0; s < n_stages; ++s) {
      mbar_inval(smem_addr(&hdr->full[s]));
      mbar_inval(smem_addr(&hdr->empty[s]));
    }
    for (int b = 0; b < 2; ++b) {
      mbar_inval(smem_addr(&hdr->acc_full[b]));
      mbar_inval(smem_addr(&hdr->acc_empty[b]));
    }
    mbar_inval(smem_addr(&hdr->drain));
  }
  return hdr->abort == 0;
}

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

__device__ __forceinline__ void attention_step(const FusedLayerParams& p, uint32_t cta, uint32_t n_ctas, uint8_t* smem,
                                               uint32_t tid) {
  const int L = p.seq, T = p.T, n_kept = p.n_kept_heads;
  const int lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int qg = warp & 3, ks = warp >> 2;
  const int Lpad = (L + 63) / 64 * 64;
  const int q_tiles = (L + 63) / 64;
  const int n_items = q_tiles * n_kept * p.batch;
  uint16_t* Ks = reinterpret_cast<uint16_t*>(smem + kLowOff);
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
    for (int idx = tid; idx < Lpad * 8; idx += kThreads) {
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
          uint16_t* dst = p.attn_out + (static_cast<size_t>(b) * L + row) * ldo + hi * 64 + 2 * t4;
#pragma unroll
          for (int jd = 0; jd < 8; ++jd)
            *reinterpret_cast<uint32_t*>(dst + jd * 8) = pack_bf16x2(o[jd][2 * r] * inv, o[jd][2 * r + 1] * inv);
        }
      }
    }
    __syncthreads();        // K, V and the merge buffer are reused by the CTA's next item
  }
}

// ---------------------------------------------------------------------------------------
// Residual + bias + LayerNorm step over split-K partial sums (same arithmetic and summation order as
// layernorm_kernel).  hidden / 4 threads per token row, one float4 each; a CTA works on 512 / (hidden / 4)
// rows at a time, each row group with its own named barrier.  Partial sums and the residual were written
// by other CTAs of this launch: they are read through L2 (ld.global.cg), never through the read-only path.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float group_sum(float v, float* red, int gt, int n_warps, int bar_id, int n_threads) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((gt & 31) == 0) red[gt >> 5] = v;
  asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(n_threads) : "memory");
  float t = 0.f;
  for (int w = 0; w < n_warps; ++w) t += red[w];
  asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(n_threads) : "memory");
  return t;
}

__device__ __forceinline__ void layernorm_step(const LnLaunch& p, uint32_t cta, uint32_t n_ctas, uint8_t* smem, uint32_t tid) {
  FusedScratch* sc = reinterpret_cast<FusedScratch*>(smem + 256);
  const int tpr = p.d / 4;                               // threads per row (a multiple of 32)
  const int groups = kThreads / tpr >= 2 ? 2 : 1;        // row groups per CTA
  const int grp = static_cast<int>(tid) / tpr, gt = static_cast<int>(tid) % tpr;
  if (grp >= groups) return;
  const int n_warps = tpr >> 5;
  const int c = gt * 4;
  float* red = sc->red[grp];
  const float4 bias = __ldg(reinterpret_cast<const float4*>(p.bias + c));
  const float4 gm = __ldg(reinterpret_cast<const float4*>(p.gamma + c));
  const float4 bt = __ldg(reinterpret_cast<const float4*>(p.beta + c));
  const size_t pstride = static_cast<size_t>(p.T) * p.d;
  for (int r = static_cast<int>(cta) * groups + grp; r < p.T; r += static_cast<int>(n_ctas) * groups) {
    const size_t row = static_cast<size_t>(r) * p.d;
    float4 a = bias;
    if (p.resid_bf16) {
      const uint2 rr = __ldcg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.resid) + row + c));
      a.x += __uint_as_float(rr.x << 16); a.y += __uint_as_float(rr.x & 0xffff0000u);
      a.z += __uint_as_float(rr.y << 16); a.w += __uint_as_float(rr.y & 0xffff0000u);
    } else {
      const float4 rr = __ldcg(reinterpret_cast<const float4*>(static_cast<const float*>(p.resid) + row + c));
      a.x += rr.x; a.y += rr.y; a.z += rr.z; a.w += rr.w;
    }
    int q = 0;
    for (; q + 4 <= p.n_partial; q += 4) {
      const float4 s0 = __ldcg(reinterpret_cast<const float4*>(p.partial + (q + 0) * pstride + row + c));
      const float4 s1 = __ldcg(reinterpret_cast<const float4*>(p.partial + (q + 1) * pstride + row + c));
      const float4 s2 = __ldcg(reinterpret_cast<const float4*>(p.partial + (q + 2) * pstride + row + c));
      const float4 s3 = __ldcg(reinterpret_cast<const float4*>(p.partial + (q + 3) * pstride + row + c));
      a.x += (s0.x + s1.x) + (s2.x + s3.x); a.y += (s0.y + s1.y) + (s2.y + s3.y);
      a.z += (s0.z + s1.z) + (s2.z + s3.z); a.w += (s0.w + s1.w) + (s2.w + s3.w);
    }
    for (; q < p.n_partial; ++q) {
      const float4 s = __ldcg(reinterpret_cast<const float4*>(p.partial + q * pstride + row + c));
      a.x += s.x; a.y += s.y; a.z += s.z; a.w += s.w;
    }
    const float mean = group_sum(a.x + a.y + a.z + a.w, red, gt, n_warps, 1 + grp, tpr) / static_cast<float>(p.d);
    const float dx = a.x - mean, dy = a.y - mean, dz = a.z - mean, dw = a.w - mean;
    const float var = group_sum(dx * dx + dy * dy + dz * dz + dw * dw, red, gt, n_warps, 1 + grp, tpr) /
                      static_cast<float>(p.d);
    const float rstd = rsqrtf(var + p.eps);
    float4 y;
    y.x = dx * rstd * gm.x + bt.x; y.y = dy * rstd * gm.y + bt.y;
    y.z = dz * rstd * gm.z + bt.z; y.w = dw * rstd * gm.w + bt.w;
    if (p.out_f32) *reinterpret_cast<float4*>(p.out_f32 + row + c) = y;
    if (p.out_bf16)
      *reinterpret_cast<uint2*>(p.out_bf16 + row + c) = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
  }
}

// ---------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1)
fused_layer_kernel(const __grid_constant__ FusedLayerParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  const uint32_t tid = threadIdx.x, warp = tid >> 5;
  const uint32_t cta = blockIdx.x, G = gridDim.x;
  SmemHeader* hdr = reinterpret_cast<SmemHeader*>(smem);
  FusedScratch* sc = reinterpret_cast<FusedScratch*>(smem + 256);
  if (tid == 0) { hdr->abort = 0; sc->where = 0; }
  if (warp == 1) {
    tmem_alloc(smem_addr(&hdr->tmem_base), kFusedTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = hdr->tmem_base;
  pdl_launch_dependents();          // this CTA owns its tensor memory: a successor can never starve it

  unsigned int passed = 0;          // grid barriers completed
  bool alive = true;
  // between arriving at a barrier and waiting on it: decode the next GEMM step's tile if its memory is free
  auto barrier = [&](int next_gemm, uint32_t next_slot) {
    if (!alive) return;
    grid_arrive(p.barrier, tid);
    if (next_gemm >= 0 && p.g[next_gemm].ahead) gemm_prologue(p.g[next_gemm], next_gemm, cta, smem, next_slot, p.err, tid);
    ++passed;
    alive = grid_wait(p.barrier, passed * G, hdr, &sc->where, (passed << 4) | 1u, tid);
  };

  gemm_prologue(p.g[0], 0, cta, smem, kSlotOff0, p.err, tid);
  pdl_wait();                       // from here on: the previous kernel's output (the layer input)
  alive = gemm_main(p.g[0], 0, cta, p.T, smem, kSlotOff0, tmem_base, tid);
  barrier(1, kSlotOff1);
  if (alive) attention_step(p, cta, G, smem, tid);
  barrier(-1, 0);
  if (alive) {
    if (!p.g[1].ahead) gemm_prologue(p.g[1], 1, cta, smem, kSlotOff1, p.err, tid);
    alive = gemm_main(p.g[1], 1, cta, p.T, smem, kSlotOff1, tmem_base, tid);
  }
  barrier(2, kSlotOff0);
  if (alive) layernorm_step(p.ln[0], cta, G, smem, tid);
  barrier(-1, 0);
  if (alive) {
    if (!p.g[2].ahead) gemm_prologue(p.g[2], 2, cta, smem, kSlotOff0, p.err, tid);
    alive = gemm_main(p.g[2], 2, cta, p.T, smem, kSlotOff0, tmem_base, tid);
  }
  barrier(3, kSlotOff1);
  if (alive) {
    if (!p.g[3].ahead) gemm_prologue(p.g[3], 3, cta, smem, kSlotOff1, p.err, tid);
    alive = gemm_main(p.g[3], 3, cta, p.T, smem, kSlotOff1, tmem_base, tid);
  }
  barrier(-1, 0);
  if (alive) layernorm_step(p.ln[1], cta, G, smem, tid);

  // status word: low byte = what went wrong; for a timeout the next bytes say which wait (step, kind) and which CTA
  if (!alive && tid == 0) atomicCAS(p.err, ERR_NONE, ERR_WAIT_TIMEOUT | static_cast<int>(sc->where << 8) | static_cast<int>(cta << 20));
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kFusedTmemCols);
}

}  // namespace

size_t fused_attention_bytes(int seq) {
  const int Lpad = (seq + 63) / 64 * 64;
  return static_cast<size_t>(Lpad) * kAttnKStride * 2 * 2 + kAttnMergeBytes;
}
size_t fused_smem_total() { return kFusedTotal + kAlignSlack; }
size_t fused_low_offset() { return kLowOff; }

cudaError_t fused_configure() {
  return cudaFuncSetAttribute(fused_layer_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(fused_smem_total()));
}

cudaError_t launch_fused_layer(const FusedLayerParams& p, int grid, cudaStream_t s, bool pdl) {
  if (grid < 1 || grid > kFusedMaxCtas) return cudaErrorInvalidValue;
  return launch_kernel(fused_layer_kernel, dim3(grid), dim3(kThreads), fused_smem_total(), s, pdl, p);
}

}  // namespace sti
