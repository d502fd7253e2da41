// Fused dequant-GEMM for sm_100a (Section 4.2 decompression + Section 2.1 linear layers).
//
// Y[T, N] = X[T, K] * W[N, K]^T where W only exists as bit-packed k-bit dictionary indexes.
// One CTA owns a weight tile (n_rows output features x k_total input features), decodes it ONCE
// into shared memory as bf16 (index unpack in registers -> per-unit centroid table in shared
// memory -> outlier patch), and then streams 128-token activation tiles past it.  After the decode
// the CTA is warp-specialised, with no CTA-wide barrier in the main loop:
//   warp 0  producer : TMA (cp.async.bulk.tensor, 128-byte swizzle) brings [128 x 64] bf16 activation
//                      chunks into a ring of stages; the first stages are requested before the decode
//   warp 1  MMA      : waits for a chunk, issues tcgen05.mma (M = 128 tokens, N = n_rows, K = 16) into
//                      one of two TMEM accumulators, tcgen05.commit frees the stage / publishes the tile
//   warps 4-7 epilogue: tcgen05.ld -> bias / erf-GELU -> global, while the next tile accumulates
//
// Weight tile layout in shared memory: element (row, k) at ((k / 8) * rows + row) * 16 + (k % 8) * 2,
// the no-swizzle K-major core-matrix layout (SBO = 128 B, LBO = rows * 16 B): lanes holding consecutive
// rows write consecutive 16-byte pieces, so decode stores are conflict-free.  Activation stages use the
// 128-byte-swizzled K-major layout that TMA writes (SBO = 1024 B).  Every wait is bounded.
#include <cuda.h>
#include <cuda_bf16.h>

#include <type_traits>

#include "gemm_device.cuh"

namespace sti {

namespace {

// ---------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------
// One accumulator tile's columns [half * ncol, (half + 1) * ncol) of this warp's 32 token rows: TMEM -> bias / erf-GELU -> global.
// FEW (at most two token tiles per CTA): eight columns per step in a rolled loop - the epilogue then runs once or twice
// per CTA, its instructions are fetched cold, and the kernel's code size is what it costs.  Otherwise 32 columns per step,
// unrolled (each thread writes 128 or 64 contiguous bytes of its row).
template <typename OutT, bool GELU, bool FEW>
__device__ __forceinline__ void epilogue_tile(uint32_t taddr, uint32_t half, uint32_t ncol, const float* bias_sm, OutT* drow,
                                              bool row_ok) {
  if constexpr (FEW) {
#pragma unroll 1
    for (uint32_t col = half * ncol; col < (half + 1) * ncol; col += 8) {
      uint32_t r[8];
      tmem_ld_32x32b_x8(taddr + col, r);
      tc_wait_ld();
      float v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float a = __uint_as_float(r[i]) + bias_sm[col + i];
        v[i] = GELU ? gelu_erf(a) : a;
      }
      if constexpr (sizeof(OutT) == 2) {
        const uint4 o = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]),
                                   pack_bf16x2(v[6], v[7]));
        if (row_ok) *reinterpret_cast<uint4*>(drow + col) = o;
      } else {
        if (row_ok) {
          reinterpret_cast<float4*>(drow + col)[0] = make_float4(v[0], v[1], v[2], v[3]);
          reinterpret_cast<float4*>(drow + col)[1] = make_float4(v[4], v[5], v[6], v[7]);
        }
      }
    }
  } else {
    for (uint32_t col = half * ncol; col < (half + 1) * ncol; col += 32) {
      if (col + 32 > (half + 1) * ncol) {            // 16-column tail of 32-row tiles
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
        break;
      }
      uint32_t r[32];
      tmem_ld_32x32b_x32(taddr + col, r);
      tc_wait_ld();
      if (row_ok) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float v[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float a = __uint_as_float(r[h * 16 + i]) + bias_sm[col + h * 16 + i];
            v[i] = GELU ? gelu_erf(a) : a;
          }
          store_row16<OutT>(drow + col + h * 16, v);
        }
      }
    }
  }
}


template <typename OutT, bool GELU, bool SIMT, bool FEW>
__global__ void __launch_bounds__(kThreads, 1)
dqgemm_kernel(const __grid_constant__ CUtensorMap xmap, const Job* __restrict__ jobs, const Seg* __restrict__ segs,
              const __nv_bfloat16* __restrict__ x, int ldx, int T, OutT* __restrict__ out, int ldo,
              const float* __restrict__ bias, int* __restrict__ err, uint32_t n_stages, uint32_t bps,
              uint32_t w_bytes, uint32_t hdr_bytes, uint32_t seg_stride, PrefetchRanges pf, int kind,
              unsigned long long* stamps) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = smem_raw;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { stamp_min(stamps, STAMP_FIRST_START); stamp_max(stamps, STAMP_LAST_START); }
  const Job job = jobs[blockIdx.x];
  const Seg* my_segs = segs + static_cast<size_t>(blockIdx.x) * seg_stride;     // independent of the job load
  const uint32_t n_rows = job.n_rows, k_total = job.k_total;

  SmemHeader* hdr = reinterpret_cast<SmemHeader*>(smem);
  float* bias_sm = reinterpret_cast<float*>(smem + 256);                            // [n_rows <= 128]
  uint16_t* tables = reinterpret_cast<uint16_t*>(smem + 768);                       // [warp][64]
  uint8_t* xsm = smem + hdr_bytes;                                                   // stages, 1024-aligned
  const uint32_t stage_bytes = bps * kBoxBytes;          // bps boxes of 64 columns per stage
  uint8_t* wsm = xsm + n_stages * stage_bytes;

  // the kernel's own checks of the descriptor: refuse rather than touch memory out of bounds
  const bool bad = job.n_seg == 0 || job.n_seg > kMaxSegs || (n_rows != 32 && n_rows != 64 && n_rows != 128) ||
                   (k_total % kChunkK) != 0 || k_total == 0 || n_rows * k_total * 2 > w_bytes ||
                   n_stages < 2 || n_stages > kMaxStages || (bps != 1 && bps != 2 && bps != 4) ||
                   768 + kWarps * kTableStride * 2 > hdr_bytes || (hdr_bytes & 1023) != 0 ||
                   (smem_addr(smem_raw) & 1023u) != 0 || job.seg_begin != blockIdx.x * seg_stride || job.n_seg > seg_stride;
  if (bad) {
    if (tid == 0) atomicCAS(err, ERR_NONE, ERR_BAD_JOB);
    return;
  }

  const int n_mtiles = (T + kTileM - 1) / kTileM;
  const uint32_t n_boxes = k_total / kChunkK;
  const uint32_t n_chunks = (n_boxes + bps - 1) / bps;  // pipeline steps per token tile
  const uint32_t my_mtiles = blockIdx.y < static_cast<uint32_t>(n_mtiles)
                                 ? (n_mtiles - blockIdx.y + gridDim.y - 1) / gridDim.y : 0;
  const uint32_t total = my_mtiles * n_chunks;          // activation chunks this CTA consumes
  const uint32_t xsm_addr = smem_addr(xsm);
  // CTAs walk the K range in rotated order so that they do not all ask L2 for the same lines at once
  const uint32_t rot = blockIdx.x % n_chunks;
  // one thread: chunk `kcr` (rotated K index) of this CTA's token tile `ti` into ring stage `stage`
  auto request_chunk = [&](uint32_t stage, uint32_t kcr, uint32_t ti) {
    const uint32_t bar = smem_addr(&hdr->full[stage]);
    const uint32_t box0 = kcr * bps;
    const uint32_t nb = n_boxes - box0 < bps ? n_boxes - box0 : bps;
    mbar_expect_tx(bar, nb * kBoxBytes);
    for (uint32_t b = 0; b < nb; ++b)
      tma_load_2d(xsm_addr + stage * stage_bytes + b * kBoxBytes, &xmap,
                  static_cast<int>(job.x_koff + (box0 + b) * kChunkK),
                  static_cast<int>((blockIdx.y + ti * gridDim.y) * kTileM), bar);
  };
  // running position of the producer: next chunk to request
  uint32_t p_c = 0, p_stage = 0, p_kcr = rot, p_kc = 0, p_ti = 0;
  auto producer_advance = [&]() {
    ++p_c;
    if (++p_stage == n_stages) p_stage = 0;
    if (++p_kcr == n_chunks) p_kcr = 0;
    if (++p_kc == n_chunks) { p_kc = 0; ++p_ti; }
  };

  uint32_t tmem_cols = 32;
  while (tmem_cols < 2 * n_rows) tmem_cols <<= 1;       // two accumulators
  if constexpr (!SIMT) {
    if (tid == 0) {
      for (uint32_t s = 0; s < n_stages; ++s) {
        mbar_init(smem_addr(&hdr->full[s]), 1);
        mbar_init(smem_addr(&hdr->empty[s]), 1);
      }
      for (int b = 0; b < 2; ++b) {
        mbar_init(smem_addr(&hdr->acc_full[b]), 1);
        mbar_init(smem_addr(&hdr->acc_empty[b]), kEpilogueWarps);     // one arrival per epilogue warp
      }
      mbar_init(smem_addr(&hdr->drain), 1);
      hdr->abort = 0;
      mbar_fence_init();
      fence_proxy_async_smem();
    }
    if (warp == 1) {
      tmem_alloc(smem_addr(&hdr->tmem_base), tmem_cols);
      tmem_relinquish();
    }
  }
  if (tid < n_rows) bias_sm[tid] = job.bias_off >= 0 ? __ldg(bias + job.bias_off + tid) : 0.f;
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = SIMT ? 0u : hdr->tmem_base;
  // Only now may the next kernel's CTAs start (and decode their weights while this kernel runs): this CTA
  // already owns its tensor memory, so a successor that allocates and then waits for this kernel to finish
  // can never starve it of columns.
  pdl_launch_dependents();

  decode_weight_tile(job, my_segs, tables, wsm, tid);
  if (tid == 0) stamp_max(stamps, STAMP_DECODED);
  // Everything above read only weights, descriptors and parameters.  The activations are the previous
  // kernel's output: from here on this kernel depends on it.
  pdl_wait();
  if (tid == 0) stamp_min(stamps, STAMP_RELEASE);

  if constexpr (SIMT) {
    // Debug path: the decoded tile multiplied on the plain ALUs, activations straight from global memory.
    for (int mt = blockIdx.y; mt < n_mtiles; mt += gridDim.y) {
      const uint32_t row = tid & 127, chalf = (tid >> 7) & 1, ncol = n_rows / 2;   // threads 0..255 work
      const int t = mt * kTileM + static_cast<int>(row);
      float acc[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) acc[c] = 0.f;
      if (t < T && tid < 256) {
        for (uint32_t kg = 0; kg < k_total; ++kg) {
          const float a = __bfloat162float(x[static_cast<size_t>(t) * ldx + job.x_koff + kg]);
#pragma unroll
          for (int c = 0; c < 64; ++c) {
            if (static_cast<uint32_t>(c) < ncol) {
              const float b = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(
                  wsm)[(static_cast<size_t>(kg >> 3) * n_rows + chalf * ncol + c) * 8 + (kg & 7)]);
              acc[c] = fmaf(a, b, acc[c]);
            }
          }
        }
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          if (static_cast<uint32_t>(cb * 16) < ncol) {
            float v[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) {
              const float a = acc[cb * 16 + c] + bias_sm[chalf * ncol + cb * 16 + c];
              v[c] = GELU ? gelu_erf(a) : a;
            }
            OutT* dst = out + (static_cast<size_t>(job.out_mat) * T + t) * ldo + job.out_col + chalf * ncol + cb * 16;
            store_row16<OutT>(dst, v);
          }
        }
      }
    }
  } else {
    bool failed = false;
    if (warp == 0) {
      // ---- producer: fill the ring, then refill a stage as soon as the MMAs that read it have completed
      if (lane == 0) {
        while (p_c < n_stages && p_c < total) { request_chunk(p_stage, p_kcr, p_ti); producer_advance(); }
        uint32_t p_phase = 0;                 // parity of the `empty` completion being waited for
        while (p_c < total) {
          if (!mbar_wait_bounded_relaxed(smem_addr(&hdr->empty[p_stage]), p_phase)) { failed = true; break; }
          request_chunk(p_stage, p_kcr, p_ti);
          if (p_stage + 1 == n_stages) p_phase ^= 1;
          producer_advance();
        }
        if (failed) {
          // give every copy this CTA requested a bounded chance to land before the CTA exits
          const uint32_t first = p_c > n_stages ? p_c - n_stages : 0;
          for (uint32_t c = first; c < p_c; ++c)
            (void)mbar_wait_bounded(smem_addr(&hdr->full[c % n_stages]), (c / n_stages) & 1);
        }
      }
      __syncwarp();
    } else if (warp == 1) {
      // ---- MMA issuer.  Descriptors are built once; per instruction only their start address moves.
      const uint32_t idesc = umma_idesc_bf16_m128(n_rows);
      const uint32_t w_lbo = n_rows * 16;
      const uint64_t a_desc0 = umma_smem_desc_sw128(xsm_addr);
      const uint64_t b_desc0 = umma_smem_desc(smem_addr(wsm), w_lbo, 128);
      const uint32_t a_stage_step = stage_bytes >> 4;          // next ring stage
      const uint32_t a_box_step = kBoxBytes >> 4;              // next 64-column box inside a stage
      const uint32_t b_ks_step = (2 * w_lbo) >> 4;             // next 16 columns of the weight tile
      const uint32_t b_chunk_step = 4 * b_ks_step;             // next 64 columns
      // The whole warp runs the loop converged; one elected lane issues.
      uint32_t stage = 0, phase = 0, kc = 0, kcr = rot, ti = 0, issued = 0;
      for (uint32_t c = 0; c < total; ++c) {
        const uint32_t buf = ti & 1;
        bool ok = true;
        if (kc == 0 && ti >= 2)        // the epilogue must have drained this accumulator
          ok = __all_sync(0xffffffffu, mbar_wait_bounded(smem_addr(&hdr->acc_empty[buf]), ((ti >> 1) - 1) & 1));
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait_bounded(smem_addr(&hdr->full[stage]), phase));
        if (!ok) { failed = true; break; }
        tc_fence_after_sync();
        const uint32_t box0 = kcr * bps;
        const uint32_t nb = n_boxes - box0 < bps ? n_boxes - box0 : bps;
        const uint64_t da0 = a_desc0 + stage * a_stage_step;
        const uint64_t db0 = b_desc0 + box0 * b_chunk_step;
        const uint32_t d_addr = tmem_base + buf * n_rows;
        if (elect_one()) {
          uint64_t da = da0, db = db0;
          // per box: four K = 16 steps, +32 bytes inside the swizzled activation row, +2 core-matrix columns of W
          umma_bf16_ss_x4(d_addr, da, db, 2, b_ks_step, idesc, kc != 0 ? 1u : 0u);
          for (uint32_t b = 1; b < nb; ++b) {
            da += a_box_step;
            db += b_chunk_step;
            umma_bf16_ss_x4(d_addr, da, db, 2, b_ks_step, idesc, 1u);
          }
          if (c + n_stages < total) umma_commit(smem_addr(&hdr->empty[stage]));   // only if the stage is refilled
          if (kc + 1 == n_chunks) umma_commit(smem_addr(&hdr->acc_full[buf]));
        }
        __syncwarp();
        issued = c + 1;
        if (++stage == n_stages) { stage = 0; phase ^= 1; }
        if (++kcr == n_chunks) kcr = 0;
        if (++kc == n_chunks) { kc = 0; ++ti; }
      }
      if (failed && issued > 0) {
        // outstanding MMAs: a commit of its own and one more bounded chance before TMEM is freed
        if (elect_one()) umma_commit(smem_addr(&hdr->drain));
        __syncwarp();
        (void)mbar_wait_bounded(smem_addr(&hdr->drain), 0);
      }
    } else if (warp == 2 || warp == 3) {
      // ---- otherwise idle: pull the packed shards of a later launch into L2
      const uint32_t n_cta = gridDim.x * gridDim.y, me = (blockIdx.y * gridDim.x + blockIdx.x) * 64 + (tid - 64);
      for (int r = 0; r < 4; ++r) prefetch_range_l2(pf.ptr[r], pf.bytes[r], me, n_cta * 64);
    } else if (warp >= kEpilogueWarp0 && warp < kEpilogueWarp0 + kEpilogueWarps) {
      // ---- epilogue: warp w owns TMEM lanes 32*(w%4).. (token rows) and one half of the columns
      const uint32_t q = warp & 3, half = (warp - kEpilogueWarp0) >> 2, ncol = n_rows / 2;
      for (uint32_t ti = 0; ti < my_mtiles; ++ti) {
        const uint32_t buf = ti & 1;
        // one lane polls (a whole CTA's worth of pollers on one barrier word slows the MMA warp's own
        // barrier traffic down); the warp then re-converges before it touches tensor memory
        uint32_t ok = 1;
        if (lane == 0) ok = mbar_wait_bounded_relaxed(smem_addr(&hdr->acc_full[buf]), (ti >> 1) & 1) ? 1u : 0u;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) { failed = true; break; }
        tc_fence_after_sync();
        const int t = static_cast<int>((blockIdx.y + ti * gridDim.y) * kTileM + q * 32 + lane);
        const size_t row_off = (static_cast<size_t>(job.out_mat) * T + (t < T ? t : 0)) * ldo + job.out_col;
        const uint32_t taddr = tmem_base + ((q * 32) << 16) + buf * n_rows;
        if constexpr (std::is_void<OutT>::value) {
          // one kernel for every GEMM of a layer: the output kind is a launch parameter, the code stays in the
          // instruction caches from launch to launch
          if (kind == GEMM_BF16_TO_F32)
            epilogue_tile<float, false, FEW>(taddr, half, ncol, bias_sm, static_cast<float*>(out) + row_off, t < T);
          else if (kind == GEMM_BF16_TO_BF16_GELU)
            epilogue_tile<__nv_bfloat16, true, FEW>(taddr, half, ncol, bias_sm, static_cast<__nv_bfloat16*>(out) + row_off, t < T);
          else
            epilogue_tile<__nv_bfloat16, false, FEW>(taddr, half, ncol, bias_sm, static_cast<__nv_bfloat16*>(out) + row_off, t < T);
        } else {
          epilogue_tile<OutT, GELU, FEW>(taddr, half, ncol, bias_sm, out + row_off, t < T);
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_addr(&hdr->acc_empty[buf]));
      }
    }
    if (failed) {
      hdr->abort = 1;
      if (lane == 0) atomicCAS(err, ERR_NONE, ERR_WAIT_TIMEOUT);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);
  }
  if (tid == 0) stamp_max(stamps, STAMP_LAST_END);
}

// ---------------------------------------------------------------------------------------
// Two-CTA variant (cta_group::2) for many tokens.
//
// A cluster of two CTAs shares one MMA: M = 256 (each CTA contributes its own 128-token activation tile),
// N = 128 (each CTA contributes the 64 decoded weight rows of its own job).  Per instruction the pair does
// twice the work of the one-CTA kernel per SM for the same issue cost, and every activation byte brought in
// from L2 is used against 128 instead of 64 output features - the one-CTA kernel is bound by exactly these
// two things once there are thousands of tokens.  CTA 0 issues; tcgen05.commit multicasts completions to both
// CTAs; both CTAs' TMA loads report to CTA 0's `full` barriers; each CTA drains its own accumulator rows
// (its 128 tokens x all 128 features) and reports to CTA 0's `acc_empty`.
// ---------------------------------------------------------------------------------------
template <typename OutT, bool GELU>
__global__ void __launch_bounds__(kThreads, 1)
dqgemm_pair_kernel(const __grid_constant__ CUtensorMap xmap, const Job* __restrict__ jobs, const Seg* __restrict__ segs,
                   int T, OutT* __restrict__ out, int ldo, const float* __restrict__ bias, int* __restrict__ err,
                   uint32_t n_stages, uint32_t bps, uint32_t w_bytes, uint32_t hdr_bytes, uint32_t seg_stride,
                   unsigned long long* stamps) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = smem_raw;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { stamp_min(stamps, STAMP_FIRST_START); stamp_max(stamps, STAMP_LAST_START); }
  const uint32_t rank = cluster_ctarank();                 // 0 issues the MMAs
  const uint32_t pair_base = blockIdx.x & ~1u;
  const Job job = jobs[blockIdx.x];                        // the 64 weight rows this CTA decodes
  const Job job0 = jobs[pair_base], job1 = jobs[pair_base + 1];   // columns 0-63 / 64-127 of the accumulator
  const uint32_t k_total = job.k_total;

  SmemHeader* hdr = reinterpret_cast<SmemHeader*>(smem);
  float* bias_sm = reinterpret_cast<float*>(smem + 256);            // [128]
  uint16_t* tables = reinterpret_cast<uint16_t*>(smem + 768);       // [warp][64]
  const Seg* my_segs = segs + static_cast<size_t>(blockIdx.x) * seg_stride;
  uint8_t* xsm = smem + hdr_bytes;
  const uint32_t stage_bytes = bps * kBoxBytes;
  uint8_t* wsm = xsm + n_stages * stage_bytes;

  // both CTAs evaluate the same conditions, so a refused pair leaves together
  const bool bad = job0.n_rows != 64 || job1.n_rows != 64 || job0.k_total != job1.k_total || job0.x_koff != job1.x_koff ||
                   job0.n_seg == 0 || job0.n_seg > kMaxSegs || job1.n_seg == 0 || job1.n_seg > kMaxSegs ||
                   (k_total % kChunkK) != 0 || k_total == 0 || 64 * k_total * 2 > w_bytes || n_stages < 2 ||
                   n_stages > kMaxStages || (bps != 1 && bps != 2 && bps != 4) ||
                   768 + kWarps * kTableStride * 2 > hdr_bytes || (hdr_bytes & 1023) != 0 || (gridDim.x & 1) != 0 ||
                   (smem_addr(smem_raw) & 1023u) != 0 || job0.n_seg > seg_stride || job1.n_seg > seg_stride ||
                   job0.seg_begin != pair_base * seg_stride || job1.seg_begin != (pair_base + 1) * seg_stride;
  if (bad) {
    if (tid == 0) atomicCAS(err, ERR_NONE, ERR_BAD_JOB);
    return;
  }

  const int n_mtiles = (T + kTileM - 1) / kTileM;
  const uint32_t n_mpairs = (n_mtiles + 1) / 2;           // the pair takes token tiles 2p (CTA 0) and 2p + 1 (CTA 1)
  const uint32_t n_boxes = k_total / kChunkK;
  const uint32_t n_chunks = (n_boxes + bps - 1) / bps;
  const uint32_t my_pairs = blockIdx.y < n_mpairs ? (n_mpairs - blockIdx.y + gridDim.y - 1) / gridDim.y : 0;
  const uint32_t total = my_pairs * n_chunks;
  const uint32_t xsm_addr = smem_addr(xsm);
  const uint32_t rot = (blockIdx.x >> 1) % n_chunks;      // both CTAs of a pair walk K in the same order
  auto tile_row0 = [&](uint32_t ti) { return static_cast<int>((2 * (blockIdx.y + ti * gridDim.y) + rank) * kTileM); };

  constexpr uint32_t kAccCols = 128, kTmemCols = 256;      // two accumulators of 128 columns
  if (tid == 0) {
    for (uint32_t s = 0; s < n_stages; ++s) {
      mbar_init(smem_addr(&hdr->full[s]), 1);              // used in CTA 0 only
      mbar_init(smem_addr(&hdr->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_addr(&hdr->acc_full[b]), 1);
      mbar_init(smem_addr(&hdr->acc_empty[b]), 2 * kPairEpilogueWarps);   // CTA 0 only: both CTAs' epilogue warps
    }
    mbar_init(smem_addr(&hdr->drain), 1);
    hdr->abort = 0;
    mbar_fence_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_addr(&hdr->tmem_base), kTmemCols);
    tmem_relinquish_pair();
  }
  if (tid < 128) {
    const Job& jb = tid < 64 ? job0 : job1;
    bias_sm[tid] = jb.bias_off >= 0 ? __ldg(bias + jb.bias_off + (tid & 63)) : 0.f;
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = hdr->tmem_base;
  pdl_launch_dependents();          // this CTA owns its tensor memory now (see the one-CTA kernel)

  decode_weight_tile(job, my_segs, tables, wsm, tid);
  if (tid == 0) stamp_max(stamps, STAMP_DECODED);
  cluster_sync_all();               // both halves of the weight tile are in place, all barriers initialised
  pdl_wait();                       // from here on: the previous kernel's output
  if (tid == 0) stamp_min(stamps, STAMP_RELEASE);

  bool failed = false;
  if (warp == 0) {
    // ---- producer (one in each CTA): own token tile into own ring, completion reported to CTA 0
    if (lane == 0) {
      uint32_t c = 0, stage = 0, phase = 0, kcr = rot, kc = 0, ti = 0;
      for (; c < total; ++c) {
        if (c >= n_stages) {
          if (!mbar_wait_bounded_relaxed(smem_addr(&hdr->empty[stage]), phase)) { failed = true; break; }
        }
        const uint32_t box0 = kcr * bps;
        const uint32_t nb = n_boxes - box0 < bps ? n_boxes - box0 : bps;
        if (rank == 0) mbar_expect_tx(smem_addr(&hdr->full[stage]), 2 * nb * kBoxBytes);    // both CTAs' bytes
        const uint32_t bar = map_to_cta(smem_addr(&hdr->full[stage]), 0);
        for (uint32_t b = 0; b < nb; ++b)
          tma_load_2d_pair(xsm_addr + stage * stage_bytes + b * kBoxBytes, &xmap,
                           static_cast<int>(job.x_koff + (box0 + b) * kChunkK), tile_row0(ti), bar);
        if (++stage == n_stages) { stage = 0; if (c >= n_stages) phase ^= 1; }
        if (++kcr == n_chunks) kcr = 0;
        if (++kc == n_chunks) { kc = 0; ++ti; }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (rank == 0) {
      // ---- MMA issuer of the pair
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((256u >> 4) << 24);
      const uint32_t w_lbo = 64 * 16;
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
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait_bounded(smem_addr(&hdr->full[stage]), phase));
        if (!ok) { failed = true; break; }
        tc_fence_after_sync();
        const uint32_t box0 = kcr * bps;
        const uint32_t nb = n_boxes - box0 < bps ? n_boxes - box0 : bps;
        const uint64_t da0 = a_desc0 + stage * a_stage_step;
        const uint64_t db0 = b_desc0 + box0 * b_chunk_step;
        const uint32_t d_addr = tmem_base + buf * kAccCols;
        if (elect_one()) {
          uint64_t da = da0, db = db0;
          umma_bf16_ss_x4_pair(d_addr, da, db, 2, b_ks_step, idesc, kc != 0 ? 1u : 0u);
          for (uint32_t b = 1; b < nb; ++b) {
            da += a_box_step;
            db += b_chunk_step;
            umma_bf16_ss_x4_pair(d_addr, da, db, 2, b_ks_step, idesc, 1u);
          }
          if (c + n_stages < total) umma_commit_pair(smem_addr(&hdr->empty[stage]));
          if (kc + 1 == n_chunks) umma_commit_pair(smem_addr(&hdr->acc_full[buf]));
        }
        __syncwarp();
        issued = c + 1;
        if (++stage == n_stages) { stage = 0; phase ^= 1; }
        if (++kcr == n_chunks) kcr = 0;
        if (++kc == n_chunks) { kc = 0; ++ti; }
      }
      if (failed && issued > 0) {
        if (elect_one()) umma_commit_pair(smem_addr(&hdr->drain));
        __syncwarp();
        (void)mbar_wait_bounded(smem_addr(&hdr->drain), 0);
      }
    }
  } else if (warp >= kEpilogueWarp0 && warp < kEpilogueWarp0 + kPairEpilogueWarps) {
    // ---- epilogue: this CTA's 128 token rows x 128 features.  Twelve warps, three per tensor-memory lane quadrant
    // (a warp reads only the 32 lanes of quadrant warp % 4); the three share the eight 16-column chunks 3 + 3 + 2.
    const uint32_t q = warp & 3, part = (warp - kEpilogueWarp0) >> 2;
    const uint32_t chunk0 = part * 3, chunk1 = part == 2 ? 8 : chunk0 + 3;
    for (uint32_t ti = 0; ti < my_pairs; ++ti) {
      const uint32_t buf = ti & 1;
      uint32_t ok = 1;
      if (lane == 0) ok = mbar_wait_bounded_relaxed(smem_addr(&hdr->acc_full[buf]), (ti >> 1) & 1) ? 1u : 0u;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) { failed = true; break; }
      tc_fence_after_sync();
      const int t = tile_row0(ti) + static_cast<int>(q * 32 + lane);
      const size_t trow = static_cast<size_t>(t < T ? t : 0);
      OutT* drow0 = out + (static_cast<size_t>(job0.out_mat) * T + trow) * ldo + job0.out_col;
      OutT* drow1 = out + (static_cast<size_t>(job1.out_mat) * T + trow) * ldo + job1.out_col;
      const uint32_t taddr = tmem_base + ((q * 32) << 16) + buf * kAccCols;
      uint32_t r[3][16];
#pragma unroll
      for (uint32_t c = 0; c < 3; ++c)
        if (chunk0 + c < chunk1) tmem_ld_32x32b_x16(taddr + (chunk0 + c) * 16, r[c]);
      tc_wait_ld();
      if (t < T) {
#pragma unroll
        for (uint32_t c = 0; c < 3; ++c) {
          if (chunk0 + c < chunk1) {
            const uint32_t col = (chunk0 + c) * 16;            // 0..127: the first 64 are job 0's features
            float v[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float a = __uint_as_float(r[c][i]) + bias_sm[col + i];
              v[i] = GELU ? gelu_erf(a) : a;
            }
            store_row16<OutT>((col < 64 ? drow0 : drow1) + (col & 63), v);
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster_cta_scope(map_to_cta(smem_addr(&hdr->acc_empty[buf]), 0));
    }
  }
  if (failed) {
    hdr->abort = 1;
    if (lane == 0) atomicCAS(err, ERR_NONE, ERR_WAIT_TIMEOUT);
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();      // neither CTA frees tensor memory or exits while the pair's MMAs may still use it
  if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
  if (tid == 0) stamp_max(stamps, STAMP_LAST_END);
}

template <typename OutT, bool GELU>
cudaError_t launch_t(const GemmLaunch& p, cudaStream_t s) {
  const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(p.x);
  if (p.pair && !p.simt_debug) {
    // clusters of two CTAs along x (consecutive jobs = the two halves of a 128-feature tile)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.n_jobs, p.m_ctas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.pdl ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, dqgemm_pair_kernel<OutT, GELU>, p.xmap, p.jobs, p.segs, p.T, static_cast<OutT*>(p.out),
                              p.ldo, p.bias, p.err, p.n_stages, p.bps, p.w_bytes, p.hdr_bytes, p.seg_stride, p.stamps);
  }
  dim3 grid(p.n_jobs, p.m_ctas), block(kThreads);
  PrefetchRanges pf;
  for (int r = 0; r < 4; ++r) { pf.ptr[r] = p.pf_ptr[r]; pf.bytes[r] = p.pf_bytes[r]; }
  const int kind = sizeof(OutT) == 4 ? GEMM_BF16_TO_F32 : (GELU ? GEMM_BF16_TO_BF16_GELU : GEMM_BF16_TO_BF16);
  if (p.simt_debug) {
    return launch_kernel(dqgemm_kernel<OutT, GELU, true, false>, grid, block, p.smem_bytes, s, p.pdl, p.xmap, p.jobs, p.segs, x, p.ldx,
                         p.T, static_cast<OutT*>(p.out), p.ldo, p.bias, p.err, p.n_stages, p.bps, p.w_bytes, p.hdr_bytes,
                         p.seg_stride, pf, kind, p.stamps);
  }
  // every output kind runs the same kernel (the kind is a parameter): one copy of the code for a layer's four GEMMs;
  // two builds of it, for few and for many token tiles per CTA (they differ in the epilogue's shape)
  const int n_mtiles = (p.T + kTileM - 1) / kTileM;
  const bool few = (n_mtiles + p.m_ctas - 1) / p.m_ctas <= 2;
  if (few)
    return launch_kernel(dqgemm_kernel<void, false, false, true>, grid, block, p.smem_bytes, s, p.pdl, p.xmap,
                                 p.jobs, p.segs, x, p.ldx, p.T, p.out, p.ldo, p.bias, p.err, p.n_stages, p.bps, p.w_bytes,
                                 p.hdr_bytes, p.seg_stride, pf, kind, p.stamps);
  return launch_kernel(dqgemm_kernel<void, false, false, false>, grid, block, p.smem_bytes, s, p.pdl, p.xmap,
                               p.jobs, p.segs, x, p.ldx, p.T, p.out, p.ldo, p.bias, p.err, p.n_stages, p.bps, p.w_bytes,
                               p.hdr_bytes, p.seg_stride, pf, kind, p.stamps);
}

template <typename K>
cudaError_t set_smem(K kernel) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

}  // namespace

size_t gemm_weight_bytes(uint32_t n_rows, uint32_t k_total) { return static_cast<size_t>(n_rows) * k_total * 2; }

uint32_t gemm_header_bytes() { return kHeaderBytes; }

size_t gemm_smem_bytes(uint32_t w_bytes, uint32_t n_stages, uint32_t bps, uint32_t hdr_bytes) {
  return hdr_bytes + static_cast<size_t>(w_bytes) + static_cast<size_t>(n_stages) * bps * kBoxBytes;
}

// Ring shape for a weight tile of `w_bytes` and a K range of `k_total`: boxes per stage and stages.
// Fewer, larger stages mean fewer waits for the MMA-issuing warp; at least ~64 KB stay in flight.
bool gemm_pick_ring(uint32_t w_bytes, uint32_t k_total, uint32_t hdr_bytes, uint32_t* n_stages, uint32_t* bps) {
  const long room = 227L * 1024 - static_cast<long>(hdr_bytes) - static_cast<long>(w_bytes);
  if (room < 3L * kBoxBytes) return false;           // the tile does not fit
  const uint32_t n_boxes = k_total / kChunkK;
  if (n_boxes <= 8 && room >= 2L * 4 * kBoxBytes) { *bps = 4; *n_stages = 2; return true; }   // a tile's K in <= 2 stages
  if (room >= 3L * 2 * kBoxBytes) { *bps = 2; *n_stages = static_cast<uint32_t>(room / (2 * kBoxBytes) > 4 ? 4 : room / (2 * kBoxBytes)); return true; }
  *bps = 1;
  *n_stages = static_cast<uint32_t>(room / kBoxBytes > 6 ? 6 : room / kBoxBytes);
  return true;
}

cudaError_t gemm_configure() {
  cudaError_t e;
#define STI_SET(OutT, G)                                                  \
  if ((e = set_smem(dqgemm_kernel<OutT, G, true, false>)) != cudaSuccess) return e;  \
  if ((e = set_smem(dqgemm_pair_kernel<OutT, G>)) != cudaSuccess) return e;
  if ((e = set_smem(dqgemm_kernel<void, false, false, true>)) != cudaSuccess) return e;
  if ((e = set_smem(dqgemm_kernel<void, false, false, false>)) != cudaSuccess) return e;
  STI_SET(__nv_bfloat16, false)
  STI_SET(__nv_bfloat16, true)
  STI_SET(float, false)
#undef STI_SET
  return cudaSuccess;
}

cudaError_t launch_gemm(GemmKind kind, const GemmLaunch& p, cudaStream_t s) {
  switch (kind) {
    case GEMM_BF16_TO_BF16: return launch_t<__nv_bfloat16, false>(p, s);
    case GEMM_BF16_TO_BF16_GELU: return launch_t<__nv_bfloat16, true>(p, s);
    case GEMM_BF16_TO_F32: return launch_t<float, false>(p, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace sti
