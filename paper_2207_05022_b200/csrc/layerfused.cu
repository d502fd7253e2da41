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
//   [512, 3072)   header slot 0: bias (512 B) + one 128-byte centroid table per warp
//   [3072, 5632)  header slot 1 (consecutive GEMM steps alternate, so a tile can be decoded ahead)
//   [6144, ...)   activation ring of the running GEMM step / K, V and merge buffers of attention
//   [..., top)    weight tile of the running or the next GEMM step, placed at the top end
// Every wait (mbarrier or grid barrier) is bounded; a CTA that gives up sets the status word, skips
// the rest of its work, frees its tensor memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "attention_device.cuh"
#include "gemm_device.cuh"

namespace sti {
namespace {

constexpr uint32_t kSlotOff0 = 512, kSlotBytes = 2560, kSlotOff1 = kSlotOff0 + kSlotBytes;
constexpr uint32_t kLowOff = 6144;                       // 1024-aligned start of the activation area
constexpr uint32_t kFusedTotal = 227 * 1024;             // dynamic shared memory of the kernel
constexpr uint32_t kFusedTmemCols = 256;                 // two accumulators of up to 128 columns

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
__device__ __noinline__ void gemm_prologue(const FusedGemm& g, int gi, uint32_t cta, uint8_t* smem, uint32_t slot_off,
                                              int* err, uint32_t tid) {
  FusedScratch* sc = reinterpret_cast<FusedScratch*>(smem + 256);
  const uint32_t n_items = static_cast<uint32_t>(g.n_jobs) * static_cast<uint32_t>(g.m_ctas);
  if (cta >= n_items) return;                            // uniform over the CTA
  const uint32_t job_i = cta % static_cast<uint32_t>(g.n_jobs);
  const Job job = g.jobs[job_i];
  const Seg* my_segs = g.segs + static_cast<size_t>(job_i) * g.seg_stride;      // independent of the job load
  const uint32_t n_rows = job.n_rows, k_total = job.k_total;
  const bool bad = job.seg_begin != job_i * g.seg_stride || job.n_seg > g.seg_stride || job.n_seg == 0 || job.n_seg > kMaxSegs || (n_rows != 32 && n_rows != 64 && n_rows != 128) ||
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
  if (tid < n_rows) bias_sm[tid] = job.bias_off >= 0 ? __ldg(g.bias + job.bias_off + tid) : 0.f;
  decode_weight_tile(job, my_segs, tables, smem + kFusedTotal - g.w_bytes, tid);
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
__device__ __noinline__ bool gemm_main(const FusedGemm& g, int gi, uint32_t cta, int T, uint8_t* smem, uint32_t slot_off,
                                          uint32_t tmem_base, uint32_t tid, const FusedLayerParams* pf = nullptr) {
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
  } else if ((warp == 2 || warp == 3) && pf != nullptr) {
    // ---- otherwise idle: pull the next layer's packed shards into L2
    for (int r = 0; r < 4; ++r) prefetch_range_l2(pf->pf_ptr[r], pf->pf_bytes[r], cta * 64 + (tid - 64), n_items * 64);
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

__device__ __noinline__ void layernorm_step(const LnLaunch& p, uint32_t cta, uint32_t n_ctas, uint8_t* smem, uint32_t tid) {
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
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = smem_raw;
  const uint32_t tid = threadIdx.x, warp = tid >> 5;
  const uint32_t cta = blockIdx.x, G = gridDim.x;
  if ((smem_addr(smem_raw) & 1023u) != 0) {            // the swizzled TMA stages need this alignment
    if (tid == 0) atomicCAS(p.err, ERR_NONE, ERR_BAD_JOB);
    return;
  }
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
  alive = gemm_main(p.g[0], 0, cta, p.T, smem, kSlotOff0, tmem_base, tid, &p);
  barrier(1, kSlotOff1);
  if (alive) {
    AttnArgs aa{p.qkv, p.attn_out, p.seq_lens, p.n_kept_heads, p.batch, p.seq, p.T};
    attention_step(aa, cta, G, smem + kLowOff, tid);
  }
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
size_t fused_smem_total() { return kFusedTotal; }
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
