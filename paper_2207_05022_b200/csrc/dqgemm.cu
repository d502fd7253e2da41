// Fused dequant-GEMM for sm_100a (Section 4.2 decompression + Section 2.1 linear layers).
//
// Y[T, N] = X[T, K] * W[N, K]^T where W only exists as bit-packed k-bit dictionary indexes.
// One CTA owns a weight tile (n_rows output features x k_total input features), decodes it ONCE
// into shared memory as bf16 (index unpack in registers -> per-unit centroid table in shared
// memory -> outlier patch), and then streams 128-token activation tiles past it:
//   activation chunk [128 x 64] bf16 -> shared memory with cp.async, several chunks in flight
//   (K-major core-matrix layout), issued before the decode so that their latency hides behind it
//   tcgen05.mma (M = 128 tokens, N = n_rows, K = 16 per instruction), fp32 accumulator in TMEM
//   epilogue: tcgen05.ld -> bias / GELU -> global.
//
// Shared-memory operand layout (both operands): element (row, k) lives at
//   ((k / 8) * rows + row) * 16 + (k % 8) * 2   bytes,
// i.e. 8x8 core matrices, 8-row groups contiguous (SBO = 128 B), K-adjacent core matrices
// `rows * 16` bytes apart (LBO).  This is the no-swizzle K-major canonical layout; lanes that
// hold consecutive rows write consecutive 16-byte pieces, so decode stores are conflict-free.
#include <cuda_bf16.h>

#include "sti_device.cuh"
#include "sti_kernels.h"

namespace sti {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kTileM = 128;                 // tokens per MMA tile
constexpr int kChunkK = 64;                 // activation K per pipeline stage
constexpr int kMaxStages = 8;
constexpr int kStageBytes = kTileM * kChunkK * 2;   // 16 KB
constexpr int kHeaderBytes = 3072;          // barriers + segment tables
constexpr int kRefillLag = 2;               // a stage is refilled two chunks after its MMAs were issued
constexpr int kMaxSegs = 16;
constexpr int kTableStride = 64;            // bf16 entries per segment table

struct SmemHeader {
  uint64_t mma_done[kMaxStages];
  uint64_t acc_full;
  uint32_t tmem_base;
  uint32_t pad;
};

// ---------------------------------------------------------------------------------------
// Weight-tile decode
// ---------------------------------------------------------------------------------------
template <int BITS>
__device__ __forceinline__ void decode_task(const Seg& sg, const uint16_t* __restrict__ tab, uint8_t* wsm,
                                            uint32_t n_rows, uint32_t task, uint32_t lane) {
  // task = (row group, 128-column chunk); the k planes of the group are contiguous.
  const uint32_t chunks = sg.kc >= 128 ? sg.kc / 128 : 1;
  const uint32_t g = task / chunks, j = task % chunks;
  const uint4* src = sg.codes + (static_cast<size_t>(g) * chunks + j) * (BITS * 32) + lane;
  uint32_t w[4 * BITS];
#pragma unroll
  for (int p = 0; p < BITS; ++p) {
    const uint4 v = __ldg(src + p * 32);
    w[4 * p + 0] = v.x; w[4 * p + 1] = v.y; w[4 * p + 2] = v.z; w[4 * p + 3] = v.w;
  }
  const bool narrow = sg.kc < 128;     // 64 in-features: the quantum is rows (l, l + 32) of a 64-row group
  const uint32_t row0 = narrow ? g * 64 + lane : g * 32 + lane;
  const uint32_t kcore0 = (sg.koff + (narrow ? 0 : j * 128)) >> 3;
#pragma unroll
  for (int s = 0; s < 16; ++s) {
    uint32_t pk[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint32_t c0 = extract_index<BITS>(w, 8 * s + 2 * e);
      const uint32_t c1 = extract_index<BITS>(w, 8 * s + 2 * e + 1);
      pk[e] = static_cast<uint32_t>(tab[c0]) | (static_cast<uint32_t>(tab[c1]) << 16);
    }
    const uint32_t row = narrow ? row0 + 32 * (s >> 3) : row0;
    const uint32_t kcore = narrow ? kcore0 + (s & 7) : kcore0 + s;
    *reinterpret_cast<uint4*>(wsm + (static_cast<size_t>(kcore) * n_rows + row) * 16) =
        make_uint4(pk[0], pk[1], pk[2], pk[3]);
  }
}

// Uncompressed (32-bit) version of a unit: rows are plain fp32, converted to bf16 on the way in.
__device__ __forceinline__ void decode_raw(const Seg& sg, uint8_t* wsm, uint32_t n_rows, uint32_t tid) {
  const float* src = reinterpret_cast<const float*>(sg.codes);
  const uint32_t pieces_per_row = sg.kc / 8;
  const uint32_t total = n_rows * pieces_per_row;
  for (uint32_t idx = tid; idx < total; idx += kThreads) {
    const uint32_t row = idx % n_rows, piece = idx / n_rows;
    const float4 a = __ldg(reinterpret_cast<const float4*>(src + static_cast<size_t>(row) * sg.kc + piece * 8));
    const float4 b = __ldg(reinterpret_cast<const float4*>(src + static_cast<size_t>(row) * sg.kc + piece * 8 + 4));
    const uint32_t kcore = (sg.koff >> 3) + piece;
    *reinterpret_cast<uint4*>(wsm + (static_cast<size_t>(kcore) * n_rows + row) * 16) =
        make_uint4(pack_bf16x2(a.x, a.y), pack_bf16x2(a.z, a.w), pack_bf16x2(b.x, b.y), pack_bf16x2(b.z, b.w));
  }
}

// ---------------------------------------------------------------------------------------
// Activation chunk: rows [m0, m0+128) x columns [k0, k0+64) -> stage buffer
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Asynchronous version: 4 x 16 bytes per thread, rows past T are zero-filled.  Within a quarter warp
// the lanes hold 8 consecutive rows of one 16-byte column piece = 128 contiguous bytes of the stage.
__device__ __forceinline__ void load_x_chunk_async(const __nv_bfloat16* __restrict__ x, int ldx, int T, int m0, int k0,
                                                   uint32_t stage_addr, uint32_t tid) {
  const uint32_t lane = tid & 31;
#pragma unroll
  for (int i = 0; i < (kTileM * (kChunkK / 8)) / kThreads; ++i) {
    const uint32_t u = (i * kThreads + tid) >> 5;          // warp-level unit, 0..31
    const uint32_t row = (u & 15) * 8 + (lane & 7);
    const uint32_t piece = (u >> 4) * 4 + (lane >> 3);
    const int t = m0 + static_cast<int>(row);
    const bool ok = t < T;
    const __nv_bfloat16* src = ok ? x + static_cast<size_t>(t) * ldx + k0 + piece * 8 : x;
    cp_async16_zfill(stage_addr + piece * (kTileM * 16) + row * 16, src, ok ? 16u : 0u);
  }
}

// Synchronous version (debug path).
__device__ __forceinline__ void load_x_chunk(const __nv_bfloat16* __restrict__ x, int ldx, int T, int m0, int k0,
                                             uint8_t* stage, uint32_t tid) {
  const uint32_t lane = tid & 31;
#pragma unroll
  for (int i = 0; i < (kTileM * (kChunkK / 8)) / kThreads; ++i) {
    const uint32_t u = (i * kThreads + tid) >> 5;
    const uint32_t row = (u & 15) * 8 + (lane & 7);
    const uint32_t piece = (u >> 4) * 4 + (lane >> 3);
    uint4 v = make_uint4(0, 0, 0, 0);
    const int t = m0 + static_cast<int>(row);
    if (t < T) v = __ldg(reinterpret_cast<const uint4*>(x + static_cast<size_t>(t) * ldx + k0 + piece * 8));
    *reinterpret_cast<uint4*>(stage + piece * (kTileM * 16) + row * 16) = v;
  }
}

__device__ __forceinline__ float gelu_erf(float v) { return 0.5f * v * (1.0f + erff(v * 0.70710678118654752440f)); }

template <typename OutT>
__device__ __forceinline__ void store_row16(OutT* dst, const float (&v)[16]) {
  if constexpr (sizeof(OutT) == 2) {
    uint32_t p[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) p[i] = pack_bf16x2(v[2 * i], v[2 * i + 1]);
    reinterpret_cast<uint4*>(dst)[0] = make_uint4(p[0], p[1], p[2], p[3]);
    reinterpret_cast<uint4*>(dst)[1] = make_uint4(p[4], p[5], p[6], p[7]);
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i)
      reinterpret_cast<float4*>(dst)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
  }
}

// ---------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------
template <typename OutT, bool GELU, bool SIMT>
__global__ void __launch_bounds__(kThreads, 1)
dqgemm_kernel(const Job* __restrict__ jobs, const Seg* __restrict__ segs, const __nv_bfloat16* __restrict__ x, int ldx,
              int T, OutT* __restrict__ out, int ldo, const float* __restrict__ bias, int* __restrict__ err,
              uint32_t n_stages, uint32_t w_bytes) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const Job job = jobs[blockIdx.x];
  const uint32_t n_rows = job.n_rows, k_total = job.k_total;

  SmemHeader* hdr = reinterpret_cast<SmemHeader*>(smem);
  uint16_t* tables = reinterpret_cast<uint16_t*>(smem + 256);                       // [kMaxSegs][64]
  uint8_t* wsm = smem + kHeaderBytes;
  uint8_t* xsm = wsm + w_bytes;                                                      // n_stages x 16 KB

  // the kernel's own checks of the descriptor: refuse rather than touch memory out of bounds
  const bool bad = job.n_seg == 0 || job.n_seg > kMaxSegs || (n_rows != 32 && n_rows != 64 && n_rows != 128) ||
                   (k_total % kChunkK) != 0 || k_total == 0 || n_rows * k_total * 2 > w_bytes ||
                   n_stages < kRefillLag + 1 || n_stages > kMaxStages;
  if (bad) {
    if (tid == 0) atomicCAS(err, ERR_NONE, ERR_BAD_JOB);
    return;
  }

  const int n_mtiles = (T + kTileM - 1) / kTileM;
  const uint32_t n_chunks = k_total / kChunkK;
  const uint32_t my_mtiles = blockIdx.y < static_cast<uint32_t>(n_mtiles)
                                 ? (n_mtiles - blockIdx.y + gridDim.y - 1) / gridDim.y : 0;
  const uint32_t total = my_mtiles * n_chunks;          // activation chunks this CTA consumes
  const uint32_t xsm_addr = smem_addr(xsm);
  auto issue_chunk = [&](uint32_t c) {
    const int m0 = (blockIdx.y + (c / n_chunks) * gridDim.y) * kTileM;
    load_x_chunk_async(x, ldx, T, m0, job.x_koff + (c % n_chunks) * kChunkK,
                       xsm_addr + (c % n_stages) * kStageBytes, tid);
  };

  uint32_t tmem_cols = 32;
  while (tmem_cols < n_rows) tmem_cols <<= 1;
  if constexpr (!SIMT) {
    // activations first: n_stages - kRefillLag chunks in flight while the weights are decoded
    for (uint32_t c = 0; c < n_stages - kRefillLag; ++c) {
      if (c < total) issue_chunk(c);
      cp_async_commit();
    }
    if (warp == 0) {
      tmem_alloc(smem_addr(&hdr->tmem_base), tmem_cols);
      tmem_relinquish();
    }
    if (tid == 0) {
      for (uint32_t s = 0; s < n_stages; ++s) mbar_init(smem_addr(&hdr->mma_done[s]), 1);
      mbar_init(smem_addr(&hdr->acc_full), 1);
      mbar_fence_init();
    }
  }
  // centroid tables, rounded once to bf16 (round-to-nearest-even)
  for (uint32_t i = tid; i < job.n_seg * kTableStride; i += kThreads) {
    const Seg& sg = segs[job.seg_begin + i / kTableStride];
    const uint32_t e = i % kTableStride;
    tables[i] = (sg.bits <= 6 && e < (1u << sg.bits)) ? bf16_bits(__ldg(sg.table + e)) : 0;
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = SIMT ? 0u : hdr->tmem_base;

  // ---- decode the weight tile once
  {
    const Seg& s0 = segs[job.seg_begin];
    const uint32_t rows_per_group = s0.kc >= 128 ? 32 : 64;
    const uint32_t chunks = s0.kc >= 128 ? s0.kc / 128 : 1;
    const uint32_t tasks_per_seg = (n_rows / rows_per_group) * chunks;
    const uint32_t n_tasks = tasks_per_seg * job.n_seg;
    for (uint32_t t = warp; t < n_tasks; t += kWarps) {
      const uint32_t si = t / tasks_per_seg, task = t % tasks_per_seg;
      const Seg& sg = segs[job.seg_begin + si];
      const uint16_t* tab = tables + si * kTableStride;
      switch (sg.bits) {
        case 2: decode_task<2>(sg, tab, wsm, n_rows, task, lane); break;
        case 3: decode_task<3>(sg, tab, wsm, n_rows, task, lane); break;
        case 4: decode_task<4>(sg, tab, wsm, n_rows, task, lane); break;
        case 5: decode_task<5>(sg, tab, wsm, n_rows, task, lane); break;
        case 6: decode_task<6>(sg, tab, wsm, n_rows, task, lane); break;
        default: break;
      }
    }
    for (uint32_t si = 0; si < job.n_seg; ++si) {
      const Seg& sg = segs[job.seg_begin + si];
      if (sg.bits == 32) decode_raw(sg, wsm, n_rows, tid);
    }
    __syncthreads();
    // outliers keep their original value (Section 6): overwrite their slot
    for (uint32_t si = 0; si < job.n_seg; ++si) {
      const Seg& sg = segs[job.seg_begin + si];
      for (uint32_t o = tid; o < sg.n_out; o += kThreads) {
        const uint32_t local = __ldg(sg.out_off + o) - sg.flat_base;
        const uint32_t row = local / sg.kc, kk = sg.koff + local % sg.kc;
        if (row < n_rows && kk < k_total)
          reinterpret_cast<uint16_t*>(wsm)[(static_cast<size_t>(kk >> 3) * n_rows + row) * 8 + (kk & 7)] =
              bf16_bits(__ldg(sg.out_val + o));
      }
    }
    fence_proxy_async_smem();
    __syncthreads();
  }

  if constexpr (SIMT) {
    // Debug path: the same shared-memory tiles multiplied on the plain ALUs.
    for (int mt = blockIdx.y; mt < n_mtiles; mt += gridDim.y) {
      const int m0 = mt * kTileM;
      const uint32_t row = tid & 127, chalf = tid >> 7, ncol = n_rows / 2;
      float acc[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) acc[c] = 0.f;
      for (uint32_t kc = 0; kc < n_chunks; ++kc) {
        __syncthreads();
        load_x_chunk(x, ldx, T, m0, job.x_koff + kc * kChunkK, xsm, tid);
        __syncthreads();
        for (uint32_t kk = 0; kk < kChunkK; ++kk) {
          const float a = __bfloat162float(
              reinterpret_cast<const __nv_bfloat16*>(xsm)[((kk >> 3) * kTileM + row) * 8 + (kk & 7)]);
          const uint32_t kg = kc * kChunkK + kk;
#pragma unroll
          for (int c = 0; c < 64; ++c) {
            if (static_cast<uint32_t>(c) < ncol) {
              const float b = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(
                  wsm)[(static_cast<size_t>(kg >> 3) * n_rows + chalf * ncol + c) * 8 + (kg & 7)]);
              acc[c] = fmaf(a, b, acc[c]);
            }
          }
        }
      }
      const int t = m0 + static_cast<int>(row);
      if (t < T) {
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          if (static_cast<uint32_t>(cb * 16) < ncol) {
            float v[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) {
              float a = acc[cb * 16 + c];
              if (job.bias_off >= 0) a += __ldg(bias + job.bias_off + chalf * ncol + cb * 16 + c);
              v[c] = GELU ? gelu_erf(a) : a;
            }
            OutT* dst = out + (static_cast<size_t>(job.out_mat) * T + t) * ldo + job.out_col + chalf * ncol + cb * 16;
            store_row16<OutT>(dst, v);
          }
        }
      }
    }
  } else {
    const uint32_t idesc = umma_idesc_bf16_m128(n_rows);
    const uint32_t w_lbo = n_rows * 16;
    const uint32_t wsm_addr = smem_addr(wsm);
    uint32_t acc_phase = 0;
    uint32_t issued = 0;       // chunks whose MMAs have been issued
    bool failed = false;
    for (uint32_t c = 0; c < total; ++c) {
      const uint32_t kc = c % n_chunks;
      // refill: chunk c + S - L goes into the stage that chunk c - L used; its MMAs were issued L iterations ago
      const uint32_t nxt = c + n_stages - kRefillLag;
      if (nxt < total && c >= kRefillLag && !failed) {
        const uint32_t prev = c - kRefillLag;
        if (!mbar_wait_bounded(smem_addr(&hdr->mma_done[prev % n_stages]), (prev / n_stages) & 1)) failed = true;
      }
      if (nxt < total && !failed) issue_chunk(nxt);
      cp_async_commit();
      // chunk c is complete once at most (n_stages - kRefillLag) newer groups are pending
      switch (n_stages - kRefillLag) {
        case 1: cp_async_wait<1>(); break;
        case 2: cp_async_wait<2>(); break;
        case 3: cp_async_wait<3>(); break;
        case 4: cp_async_wait<4>(); break;
        case 5: cp_async_wait<5>(); break;
        default: cp_async_wait<6>(); break;
      }
      fence_proxy_async_smem();
      if (__syncthreads_or(failed)) { failed = true; break; }
      if (tid == 0) {
        tc_fence_after_sync();
        const uint32_t a_base = xsm_addr + (c % n_stages) * kStageBytes;
        const uint32_t b_base = wsm_addr + (kc * (kChunkK / 8)) * w_lbo;
#pragma unroll
        for (int ks = 0; ks < kChunkK / 16; ++ks) {
          const uint64_t da = umma_smem_desc(a_base + ks * 2 * (kTileM * 16), kTileM * 16, 128);
          const uint64_t db = umma_smem_desc(b_base + ks * 2 * w_lbo, w_lbo, 128);
          umma_bf16_ss(tmem_base, da, db, idesc, (kc | ks) != 0 ? 1u : 0u);
        }
        umma_commit(smem_addr(&hdr->mma_done[c % n_stages]));
        if (kc + 1 == n_chunks) umma_commit(smem_addr(&hdr->acc_full));
      }
      issued = c + 1;
      if (kc + 1 != n_chunks) continue;
      // ---- epilogue of this token tile: accumulator -> registers -> global
      if (!mbar_wait_bounded(smem_addr(&hdr->acc_full), acc_phase)) failed = true;
      acc_phase ^= 1;
      if (__syncthreads_or(failed)) { failed = true; break; }
      tc_fence_after_sync();
      const int m0 = (blockIdx.y + (c / n_chunks) * gridDim.y) * kTileM;
      const uint32_t q = warp & 3, chalf = warp >> 2, ncol = n_rows / 2;
      const int t = m0 + static_cast<int>(q * 32 + lane);
      for (uint32_t c0 = 0; c0 < ncol; c0 += 16) {
        uint32_t r[16];
        const uint32_t col = chalf * ncol + c0;
        tmem_ld_32x32b_x16(tmem_base + ((q * 32) << 16) + col, r);
        tc_wait_ld();
        if (t < T) {
          float v[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            float a = __uint_as_float(r[i]);
            if (job.bias_off >= 0) a += __ldg(bias + job.bias_off + col + i);
            v[i] = GELU ? gelu_erf(a) : a;
          }
          OutT* dst = out + (static_cast<size_t>(job.out_mat) * T + t) * ldo + job.out_col + col;
          store_row16<OutT>(dst, v);
        }
      }
      tc_fence_before_sync();
      __syncthreads();        // all accumulator reads done before the next tile's first MMA overwrites it
    }
    cp_async_wait<0>();       // no copy of this CTA may still be in flight when it exits
    if (failed && tid == 0) atomicCAS(err, ERR_NONE, ERR_WAIT_TIMEOUT);
    // Every MMA this CTA issued has completed (acc_full was waited for after the last tile) unless a
    // wait ran out; in that case give outstanding MMAs one more bounded chance before freeing TMEM.
    if (failed && issued > 0) {
      const uint32_t last = issued - 1;
      (void)mbar_wait_bounded(smem_addr(&hdr->mma_done[last % n_stages]), (last / n_stages) & 1);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, tmem_cols);
  }
}

template <typename OutT, bool GELU>
cudaError_t launch_t(const GemmLaunch& p, cudaStream_t s) {
  dim3 grid(p.n_jobs, p.m_ctas), block(kThreads);
  const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(p.x);
  if (p.simt_debug)
    dqgemm_kernel<OutT, GELU, true><<<grid, block, p.smem_bytes, s>>>(
        p.jobs, p.segs, x, p.ldx, p.T, static_cast<OutT*>(p.out), p.ldo, p.bias, p.err, p.n_stages, p.w_bytes);
  else
    dqgemm_kernel<OutT, GELU, false><<<grid, block, p.smem_bytes, s>>>(
        p.jobs, p.segs, x, p.ldx, p.T, static_cast<OutT*>(p.out), p.ldo, p.bias, p.err, p.n_stages, p.w_bytes);
  return cudaGetLastError();
}

template <typename K>
cudaError_t set_smem(K kernel) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

}  // namespace

size_t gemm_weight_bytes(uint32_t n_rows, uint32_t k_total) { return static_cast<size_t>(n_rows) * k_total * 2; }

size_t gemm_smem_bytes(uint32_t w_bytes, uint32_t n_stages) {
  return kHeaderBytes + static_cast<size_t>(w_bytes) + static_cast<size_t>(n_stages) * kStageBytes;
}

uint32_t gemm_pick_stages(uint32_t w_bytes) {
  const size_t room = 227 * 1024 - kHeaderBytes - static_cast<size_t>(w_bytes);
  const size_t s = room / kStageBytes;
  return static_cast<uint32_t>(s > 6 ? 6 : s);       // fewer than 3 means the tile does not fit
}

cudaError_t gemm_configure() {
  cudaError_t e;
#define STI_SET(OutT, G)                                                  \
  if ((e = set_smem(dqgemm_kernel<OutT, G, false>)) != cudaSuccess) return e; \
  if ((e = set_smem(dqgemm_kernel<OutT, G, true>)) != cudaSuccess) return e;
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
