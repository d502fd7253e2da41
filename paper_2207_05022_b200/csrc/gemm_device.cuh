// Device-side pieces of the fused dequant-GEMM that more than one kernel uses: tile constants, the
// shared-memory header with the mbarriers, the weight-tile decode (Section 4.2 decompression: index
// unpack -> per-unit centroid table -> outlier patch), TMA / descriptor helpers and the epilogue maths.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "sti_device.cuh"
#include "sti_kernels.h"

namespace sti {
namespace {

constexpr int kThreads = 512;               // warp 0: TMA producer, warp 1: MMA issuer, warps 4-7: epilogue; all 16 decode
constexpr int kWarps = kThreads / 32;
constexpr int kTileM = 128;                 // tokens per MMA tile
constexpr int kChunkK = 64;                 // one TMA box = 64 columns = one 128-byte swizzle row; a stage holds 1, 2 or 4 boxes
constexpr int kMaxStages = 8;
constexpr int kBoxBytes = kTileM * kChunkK * 2;     // 16 KB
// header = barriers (256 B) + bias (512 B) + one 128-byte centroid table per warp; stages start 1024-aligned after it
constexpr int kHeaderBytes = 3072;
constexpr int kMaxSegs = 16;
constexpr int kTableStride = 64;            // bf16 entries per segment table
constexpr int kEpilogueWarp0 = 4;             // epilogue warps 4..11: two per TMEM lane quadrant
constexpr int kEpilogueWarps = 8;
constexpr int kPairEpilogueWarps = 12;        // the two-CTA kernel drains with warps 4..15: three per lane quadrant

struct SmemHeader {
  uint64_t full[kMaxStages];     // activation chunk landed (TMA transaction bytes)
  uint64_t empty[kMaxStages];    // the MMAs that read the chunk have completed
  uint64_t acc_full[2];          // accumulator buffer complete
  uint64_t acc_empty[2];         // accumulator buffer drained by the epilogue warps
  uint64_t drain;                // failure path only: all issued MMAs have completed
  uint32_t tmem_base;
  volatile uint32_t abort;       // a bounded wait ran out somewhere in the CTA
};

// ---------------------------------------------------------------------------------------
// Weight-tile decode
// ---------------------------------------------------------------------------------------
// The k index planes of one task = (row group, 128-column chunk), one coalesced 128-bit load per plane.
// `bits` is only known at run time here, so that the loads can be issued before anything else of the
// task is ready.  All six loads are issued back to back and unconditionally - a plane number beyond `bits`
// re-reads the last plane (a cache hit) - so that the task pays one memory round trip: with a load under
// `if (p < bits)` each plane's load waited for the one before it.
__device__ __forceinline__ void load_planes(const Seg& sg, uint32_t task, uint32_t lane, uint32_t (&w)[24]) {
  const uint32_t bits = sg.bits;
  const uint32_t chunks = sg.kc >= 128 ? sg.kc / 128 : 1;
  const uint32_t g = task / chunks, j = task % chunks;
  const uint4* src = sg.codes + (static_cast<size_t>(g) * chunks + j) * (bits * 32) + lane;
  uint4 v[6];
#pragma unroll
  for (int p = 0; p < 6; ++p) v[p] = __ldg(src + (static_cast<uint32_t>(p) < bits ? p : (bits ? bits - 1 : 0)) * 32);
#pragma unroll
  for (int p = 0; p < 6; ++p) { w[4 * p + 0] = v[p].x; w[4 * p + 1] = v[p].y; w[4 * p + 2] = v[p].z; w[4 * p + 3] = v[p].w; }
}

// Which outlier of the tile a thread patches: outlier number `t` in the order of the tile's segments.  The segments'
// counts are read in one go (lane s reads segment s: one memory round trip for up to kMaxSegs descriptors instead of
// one per segment) and handed round by shuffles.  Returns the total; `seg` stays 0xffffffff when t is beyond it.
__device__ __forceinline__ uint32_t find_outlier_slot(const Seg* __restrict__ segs, uint32_t n_seg, uint32_t t, uint32_t lane,
                                                      uint32_t& seg, uint32_t& index) {
  const uint32_t mine = lane < n_seg ? segs[lane].n_out : 0u;
  uint32_t before = 0;
  seg = 0xffffffffu;
  index = 0;
#pragma unroll 1
  for (uint32_t si = 0; si < n_seg; ++si) {
    const uint32_t n = __shfl_sync(0xffffffffu, mine, static_cast<int>(si));
    if (seg == 0xffffffffu && t >= before && t - before < n) { seg = si; index = t - before; }
    before += n;
  }
  return before;
}

// Index unpack in registers -> bf16 table lookup in shared memory -> 16-byte stores into the K-major
// core-matrix layout.  Each lane holds 128 consecutive indexes of its own row.
// `half`: 0 = the whole quantum (four index groups), 1 / 2 = its first / second two groups only (two warps share a
// task when a tile has fewer tasks than the CTA has warps; both hold the task's planes).
template <int BITS>
__device__ __forceinline__ void unpack_task(const uint32_t (&planes)[24], const Seg& sg, const uint16_t* __restrict__ tab,
                                            uint8_t* wsm, uint32_t n_rows, uint32_t task, uint32_t lane, uint32_t half = 0) {
  uint32_t w[4 * BITS];
#pragma unroll
  for (int i = 0; i < 4 * BITS; ++i) w[i] = planes[i];
  if (half == 2) {
#pragma unroll
    for (int i = 0; i < 2 * BITS; ++i) w[i] = planes[i + 2 * BITS];
  }
  const int grp0 = half == 2 ? 2 : 0, grp1 = half == 1 ? 2 : 4;
  const uint32_t chunks = sg.kc >= 128 ? sg.kc / 128 : 1;
  const uint32_t g = task / chunks, j = task % chunks;
  const bool narrow = sg.kc < 128;     // 64 in-features: the quantum is rows (l, l + 32) of a 64-row group
  const uint32_t row0 = narrow ? g * 64 + lane : g * 32 + lane;
  const uint32_t kcore0 = (sg.koff + (narrow ? 0 : j * 128)) >> 3;
  // 32 indexes = exactly BITS words, whatever BITS is: the loop below is rolled over the four such groups
  // of the quantum and always reads w[0 .. BITS), the words moving down by BITS after each group.  A
  // quarter of the instructions of the fully unrolled form: the decode runs once per CTA, so its code is
  // fetched cold and its size is what it costs.
#pragma unroll 1
  for (int grp = grp0; grp < grp1; ++grp) {
    uint32_t lo[BITS];
#pragma unroll
    for (int i = 0; i < BITS; ++i) lo[i] = w[i];
#pragma unroll
    for (int ss = 0; ss < 4; ++ss) {
      uint32_t pk[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t c0 = extract_index_words<BITS>(lo, 8 * ss + 2 * e);
        const uint32_t c1 = extract_index_words<BITS>(lo, 8 * ss + 2 * e + 1);
        pk[e] = static_cast<uint32_t>(tab[c0]) | (static_cast<uint32_t>(tab[c1]) << 16);
      }
      const uint32_t sidx = 4 * grp + ss;
      const uint32_t row = narrow ? row0 + 32 * (sidx >> 3) : row0;
      const uint32_t kcore = narrow ? kcore0 + (sidx & 7) : kcore0 + sidx;
      *reinterpret_cast<uint4*>(wsm + (static_cast<size_t>(kcore) * n_rows + row) * 16) =
          make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
#pragma unroll
    for (int i = 0; i + BITS < 4 * BITS; ++i) w[i] = w[i + BITS];
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
// TMA / mbarrier helpers local to this kernel
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// [128 rows x 64 columns] box at (column k0, row m0); rows past the tensor's extent arrive as zeros.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int k0, int m0, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(k0), "r"(m0), "r"(bar)
      : "memory");
}
// K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;                 // leading byte offset: unused for this layout
  d |= static_cast<uint64_t>(1024 >> 4) << 32;         // stride byte offset
  d |= static_cast<uint64_t>(1) << 46;                 // descriptor version for sm_100
  d |= static_cast<uint64_t>(2) << 61;                 // layout type: 128-byte swizzle
  return d;
}

// ---------------------------------------------------------------------------------------
// Thread-block clusters: rank, barrier, distributed shared memory
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {     // every thread of both CTAs
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {   // same offset in CTA `rank`
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// The same arrival with release semantics at CTA scope only: enough where the arrival hands over tensor memory
// (ordered by the tcgen05 fences), and it does not wait for the thread's earlier global stores to reach the
// cluster's point of coherence, which the cluster-scope form does.
__device__ __forceinline__ void mbar_arrive_cluster_cta_scope(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t cluster_nctas() {      // CTAs in this cluster (1 without a cluster launch)
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_arrive_release() {  // every thread of every CTA in the cluster
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait_acquire() {
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float4 ld_dsmem_f4(uint32_t cluster_addr) {   // 16 bytes of any CTA of the cluster
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(cluster_addr) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t ld_acquire_gpu(const unsigned int* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// erf-GELU.  erf through the rational approximation 7.1.26 of Abramowitz & Stegun (absolute error
// below 1.5e-7, three orders of magnitude under the bf16 rounding of the result) with the hardware
// exponential; the epilogue runs it for every element of the FFN1 output.
__device__ __forceinline__ float gelu_erf(float v) {
  // gelu(v) = v/2 + |v|/2 * erf(|v| / sqrt 2), erf(x) = 1 - poly(t) t exp(-x^2), t = 1 / (1 + p x)
  const float x = fabsf(v) * 0.70710678118654752440f;
  float t;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f, x, 1.0f)));
  float poly = fmaf(1.061405429f, t, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  float e;                                                   // exp(-x^2) = 2^(v^2 * (-log2(e) / 2))
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"((v * v) * -0.72134752044448170368f));
  const float erf_abs = fmaf(-(poly * t), e, 1.0f);
  const float h = 0.5f * v;
  return fmaf(fabsf(h), erf_abs, h);
}

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

struct PrefetchRanges {
  const uint8_t* ptr[4];
  uint32_t bytes[4];
};

// Pulls [ptr, ptr + bytes) into L2, one 128-byte line per instruction, the range shared out over
// `n_threads` threads of which this is number `t`.  Packed shards are read once per forward, so without
// this every decode starts with address translation and DRAM latency on its critical path.
__device__ __forceinline__ void prefetch_range_l2(const uint8_t* ptr, uint32_t bytes, uint32_t t, uint32_t n_threads) {
  // plain loads whose values are dropped: unlike a prefetch hint they also bring the translation in
  uint32_t sink = 0;
  for (uint32_t off = t * 128u; off < bytes; off += n_threads * 128u) {
    uint32_t v;
    asm volatile("ld.global.cg.b32 %0, [%1];" : "=r"(v) : "l"(ptr + off) : "memory");
    sink |= v;
  }
  asm volatile("" ::"r"(sink));
}

// ---------------------------------------------------------------------------------------
// Decode of one job's weight tile (shared by every GEMM kernel)
// ---------------------------------------------------------------------------------------
// One outlier (Section 6: outliers keep their original value) into its slot of the decoded tile.
__device__ __forceinline__ void patch_outlier(const Seg& sg, uint32_t off, float val, uint8_t* wsm, uint32_t n_rows,
                                              uint32_t k_total) {
  const uint32_t local = off - sg.flat_base;
  const uint32_t row = local / sg.kc, kk = sg.koff + local % sg.kc;
  if (row < n_rows && kk < k_total)
    reinterpret_cast<uint16_t*>(wsm)[(static_cast<size_t>(kk >> 3) * n_rows + row) * 8 + (kk & 7)] = bf16_bits(val);
}

// Decodes the job's weight tile into `wsm` (all threads of the CTA; ends with the tile visible to the tensor
// core: proxy fence + CTA barrier).  `segs` are the job's own segments.  The whole prologue is two memory
// round trips: the segment descriptors, then - issued together - the index planes, the centroid table and
// the outliers.  A warp keeps the table of the segment it works on (rounded once to bf16, round-to-nearest-
// even) in its own 128 bytes of `warp_tables`, so no CTA-wide barrier sits between the loads and the unpack.
__device__ __forceinline__ void decode_weight_tile(const Job& job, const Seg* __restrict__ segs, uint16_t* warp_tables,
                                                   uint8_t* wsm, uint32_t tid) {
  const uint32_t lane = tid & 31, warp = tid >> 5;
  const uint32_t n_rows = job.n_rows, k_total = job.k_total;
  const Seg& s0 = segs[0];
  const uint32_t rows_per_group = s0.kc >= 128 ? 32 : 64;
  const uint32_t chunks = s0.kc >= 128 ? s0.kc / 128 : 1;
  const uint32_t tasks_per_seg = (n_rows / rows_per_group) * chunks;
  const uint32_t n_tasks = tasks_per_seg * job.n_seg;
  // outlier number `tid` of the tile (segments in order): fetched now, applied once the tile is written
  uint32_t o_seg, o_idx, o_off = 0;
  float o_val = 0.f;
  const uint32_t n_out_total = find_outlier_slot(segs, job.n_seg, tid, lane, o_seg, o_idx);
  if (o_seg != 0xffffffffu) {
    o_off = __ldg(segs[o_seg].out_off + o_idx);
    o_val = __ldg(segs[o_seg].out_val + o_idx);
  }
  uint16_t* tab = warp_tables + warp * kTableStride;
  // a tile with at most half as many tasks as the CTA has warps: two warps share a task (half the decode latency)
  const bool split = 2 * n_tasks <= kWarps;
  const uint32_t n_units = split ? 2 * n_tasks : n_tasks;
  for (uint32_t u = warp; u < n_units; u += kWarps) {
    const uint32_t t = split ? u >> 1 : u, half = split ? 1 + (u & 1) : 0;
    const uint32_t si = t / tasks_per_seg, task = t % tasks_per_seg;
    const Seg& sg = segs[si];
    const uint32_t bits = sg.bits;
    if (bits > 6) continue;            // raw fp32 segments are handled below
    const uint32_t n_entries = 1u << bits;
    const float c0 = lane < n_entries ? __ldg(sg.table + lane) : 0.f;
    const float c1 = lane + 32 < n_entries ? __ldg(sg.table + lane + 32) : 0.f;
    uint32_t planes[24];
    load_planes(sg, task, lane, planes);
    tab[lane] = bf16_bits(c0);
    tab[lane + 32] = bf16_bits(c1);
    __syncwarp();
    switch (bits) {
      case 2: unpack_task<2>(planes, sg, tab, wsm, n_rows, task, lane, half); break;
      case 3: unpack_task<3>(planes, sg, tab, wsm, n_rows, task, lane, half); break;
      case 4: unpack_task<4>(planes, sg, tab, wsm, n_rows, task, lane, half); break;
      case 5: unpack_task<5>(planes, sg, tab, wsm, n_rows, task, lane, half); break;
      case 6: unpack_task<6>(planes, sg, tab, wsm, n_rows, task, lane, half); break;
      default: break;
    }
    __syncwarp();                      // the table is overwritten by the warp's next task
  }
  for (uint32_t si = 0; si < job.n_seg; ++si) {
    const Seg& sg = segs[si];
    if (sg.bits == 32) decode_raw(sg, wsm, n_rows, tid);
  }
  __syncthreads();
  if (o_seg != 0xffffffffu) patch_outlier(segs[o_seg], o_off, o_val, wsm, n_rows, k_total);
  if (n_out_total > kThreads) {        // more outliers than threads: the rest, one pass per 512
    uint32_t base = 0;
    for (uint32_t si = 0; si < job.n_seg; ++si) {
      const Seg& sg = segs[si];
      for (uint32_t o = tid; o < sg.n_out; o += kThreads)
        if (base + o >= kThreads) patch_outlier(sg, __ldg(sg.out_off + o), __ldg(sg.out_val + o), wsm, n_rows, k_total);
      base += sg.n_out;
    }
  }
  fence_proxy_async_smem();
  __syncthreads();
}

// ---------------------------------------------------------------------------------------
// Two-CTA (cta_group::2) forms of the tensor-memory, TMA and MMA helpers
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t n_cols) {     // one warp in each CTA
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(n_cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t n_cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(n_cols) : "memory");
}
// Own tile into own shared memory, completion bytes credited to the barrier at `bar_cluster_addr` (CTA 0's).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int k0, int m0,
                                                 uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(k0), "r"(m0), "r"(bar_cluster_addr)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_ss_x4_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t a_step,
                                                     uint32_t b_step, uint32_t idesc, uint32_t accumulate_first) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 a1, a2, a3, b1, b2, b3, as, bs;\n\t"
      "setp.ne.b32 p0, %6, 0;\n\t"
      "setp.eq.b32 p1, 0, 0;\n\t"
      "cvt.u64.u32 as, %3;\n\t"
      "cvt.u64.u32 bs, %4;\n\t"
      "add.u64 a1, %1, as;\n\tadd.u64 a2, a1, as;\n\tadd.u64 a3, a2, as;\n\t"
      "add.u64 b1, %2, bs;\n\tadd.u64 b2, b1, bs;\n\tadd.u64 b3, b2, bs;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %5, p0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a1, b1, %5, p1;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a2, b2, %5, p1;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a3, b3, %5, p1;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(a_step), "r"(b_step), "r"(idesc), "r"(accumulate_first)
      : "memory");
}
// Completion of all MMAs issued so far -> the barrier at this offset in both CTAs.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(static_cast<uint16_t>(3)) : "memory");
}


// ---------------------------------------------------------------------------------------
// The same decode run by a group of NWARPS warps of the CTA (the others do something else meanwhile):
// `gtid` is the thread's index inside the group, `warp_tables` the group's first centroid table, `bar_id`
// a named barrier reserved for the group.  Ends with the tile visible to the tensor core (proxy fence +
// group barrier).  Every thread of the group must call it the same number of times.
// ---------------------------------------------------------------------------------------
template <int NWARPS>
__device__ __forceinline__ void group_barrier(uint32_t bar_id) {
  asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(NWARPS * 32) : "memory");
}

// SPLIT: every task is shared by two warps (unit u = 2 * task + half), for tiles with fewer tasks than warps.
template <int NWARPS, bool SPLIT = false>
__device__ __forceinline__ void decode_weight_tile_group(const Job& job, const Seg* __restrict__ segs,
                                                         uint16_t* warp_tables, uint8_t* wsm, uint32_t gtid,
                                                         uint32_t bar_id) {
  constexpr uint32_t kGroupThreads = NWARPS * 32;
  const uint32_t lane = gtid & 31, warp = gtid >> 5;
  const uint32_t n_rows = job.n_rows, k_total = job.k_total;
  const Seg& s0 = segs[0];
  const uint32_t rows_per_group = s0.kc >= 128 ? 32 : 64;
  const uint32_t chunks = s0.kc >= 128 ? s0.kc / 128 : 1;
  const uint32_t tasks_per_seg = (n_rows / rows_per_group) * chunks;
  const uint32_t n_tasks = tasks_per_seg * job.n_seg;
  uint32_t o_seg, o_idx, o_off = 0;
  float o_val = 0.f;
  const uint32_t n_out_total = find_outlier_slot(segs, job.n_seg, gtid, lane, o_seg, o_idx);
  if (o_seg != 0xffffffffu) {
    o_off = __ldg(segs[o_seg].out_off + o_idx);
    o_val = __ldg(segs[o_seg].out_val + o_idx);
  }
  uint16_t* tab = warp_tables + warp * kTableStride;
  for (uint32_t u = warp; u < (SPLIT ? 2 * n_tasks : n_tasks); u += NWARPS) {
    const uint32_t t = SPLIT ? u >> 1 : u;
    const uint32_t si = t / tasks_per_seg, task = t % tasks_per_seg;
    const Seg& sg = segs[si];
    const uint32_t bits = sg.bits;
    if (bits > 6) continue;
    const uint32_t n_entries = 1u << bits;
    const float c0 = lane < n_entries ? __ldg(sg.table + lane) : 0.f;
    const float c1 = lane + 32 < n_entries ? __ldg(sg.table + lane + 32) : 0.f;
    uint32_t planes[24];
    load_planes(sg, task, lane, planes);
    tab[lane] = bf16_bits(c0);
    tab[lane + 32] = bf16_bits(c1);
    __syncwarp();
    if (SPLIT) {
      switch (bits) {
        case 2: unpack_task<2>(planes, sg, tab, wsm, n_rows, task, lane, 1 + (u & 1)); break;
        case 3: unpack_task<3>(planes, sg, tab, wsm, n_rows, task, lane, 1 + (u & 1)); break;
        case 4: unpack_task<4>(planes, sg, tab, wsm, n_rows, task, lane, 1 + (u & 1)); break;
        case 5: unpack_task<5>(planes, sg, tab, wsm, n_rows, task, lane, 1 + (u & 1)); break;
        case 6: unpack_task<6>(planes, sg, tab, wsm, n_rows, task, lane, 1 + (u & 1)); break;
        default: break;
      }
    } else {
    switch (bits) {
      case 2: unpack_task<2>(planes, sg, tab, wsm, n_rows, task, lane); break;
      case 3: unpack_task<3>(planes, sg, tab, wsm, n_rows, task, lane); break;
      case 4: unpack_task<4>(planes, sg, tab, wsm, n_rows, task, lane); break;
      case 5: unpack_task<5>(planes, sg, tab, wsm, n_rows, task, lane); break;
      case 6: unpack_task<6>(planes, sg, tab, wsm, n_rows, task, lane); break;
      default: break;
    }
    }
    __syncwarp();
  }
  for (uint32_t si = 0; si < job.n_seg; ++si) {
    const Seg& sg = segs[si];
    if (sg.bits == 32) {             // uncompressed version: fp32 rows, rounded to bf16 on the way in
      const float* src = reinterpret_cast<const float*>(sg.codes);
      const uint32_t pieces_per_row = sg.kc / 8;
      const uint32_t total = n_rows * pieces_per_row;
      for (uint32_t idx = gtid; idx < total; idx += kGroupThreads) {
        const uint32_t row = idx % n_rows, piece = idx / n_rows;
        const float4 a = __ldg(reinterpret_cast<const float4*>(src + static_cast<size_t>(row) * sg.kc + piece * 8));
        const float4 b = __ldg(reinterpret_cast<const float4*>(src + static_cast<size_t>(row) * sg.kc + piece * 8 + 4));
        const uint32_t kcore = (sg.koff >> 3) + piece;
        *reinterpret_cast<uint4*>(wsm + (static_cast<size_t>(kcore) * n_rows + row) * 16) =
            make_uint4(pack_bf16x2(a.x, a.y), pack_bf16x2(a.z, a.w), pack_bf16x2(b.x, b.y), pack_bf16x2(b.z, b.w));
      }
    }
  }
  group_barrier<NWARPS>(bar_id);
  if (o_seg != 0xffffffffu) patch_outlier(segs[o_seg], o_off, o_val, wsm, n_rows, k_total);
  if (n_out_total > kGroupThreads) {
    uint32_t base = 0;
    for (uint32_t si = 0; si < job.n_seg; ++si) {
      const Seg& sg = segs[si];
      for (uint32_t o = gtid; o < sg.n_out; o += kGroupThreads)
        if (base + o >= kGroupThreads) patch_outlier(sg, __ldg(sg.out_off + o), __ldg(sg.out_val + o), wsm, n_rows, k_total);
      base += sg.n_out;
    }
  }
  fence_proxy_async_smem();
  group_barrier<NWARPS>(bar_id);
}

}  // namespace
}  // namespace sti
