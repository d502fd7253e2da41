// K-accumulating form of the fused dequant-GEMM for many tokens (FFN2: out = u F2^T, K = all kept FFN neurons).
//
// The ordinary kernels keep one decoded weight tile per CTA, so a GEMM whose K does not fit one tile is cut into
// K groups that each write their own fp32 plane of partial sums, which the LayerNorm kernel then adds up.  With
// thousands of tokens those planes are most of the traffic of the layer's second half.  Here a pair of CTAs
// (cta_group::2, M = 256 tokens, N = 128 features) keeps the accumulators of up to four token-tile pairs in tensor
// memory (4 x 128 columns = all of it) and walks ALL K groups over them, so the result is written once, complete.
// The price is that the pair's weight tile changes with every K group: the tiles are small (64 rows x <= 512
// columns, 64 KB), two of them sit in shared memory, and eight warps decode K group g + 1 (Section 4.2
// decompression, the same routine as everywhere) while the tensor core works on K group g.  The same eight
// warps drain the accumulators, tile pair by tile pair, when a block's last K group is through.
//
//   warp 0      TMA producer: activation boxes [128 tokens x 64] of (block, K group, tile, box) into a ring
//   warp 1      MMA issuer (CTA 0 of the pair): tcgen05.mma.cta_group::2, commits free ring stages / weight buffers
//   warps 4-11  decode weight tiles into the two buffers; epilogue (tcgen05.ld -> fp32 rows in global memory)
//   warps 12-15 L2 prefetch of the activations of the step after next, when the operand does not fit L2
//
// An mbarrier parity wait only tells "the phase of this parity has completed": every waiter here meets every phase
// of the barriers it waits on, in order (a waiter that skipped a phase would take the one two back for its own).
//
// Every wait is bounded; a role that gives up raises the CTA's abort flag, the others stop waiting but keep
// walking their loops (the decode group meets at named barriers), and the status word reports the timeout.
#include <algorithm>

#include "gemm_device.cuh"

namespace sti {
namespace {

constexpr uint32_t kKaccTiles = 4;                    // token-tile pairs whose accumulators are live at once
constexpr uint32_t kKaccAccCols = 128;                // columns of one accumulator (N of the pair's MMA)
constexpr uint32_t kKaccTmemCols = kKaccTiles * kKaccAccCols;
constexpr int kKaccMaxStages = 12;
constexpr int kKaccGroupWarp0 = 4, kKaccGroupWarps = 8;
constexpr int kKaccPrefetchWarp0 = 12;               // warps 12-15: L2 prefetch of the activation stream
constexpr uint32_t kKaccGroupBarrier = 1;

struct KaccHeader {
  uint64_t full[kKaccMaxStages];   // CTA 0: both CTAs' activation boxes of the stage have landed
  uint64_t empty[kKaccMaxStages];  // both CTAs: the MMAs that read the stage have completed
  uint64_t w_full[2];            // CTA 0: both CTAs' halves of the weight tile in this buffer are decoded (2 arrivals)
  uint64_t w_empty[2];           // both CTAs: the MMAs that read the buffer have completed
  uint64_t acc_full[kKaccTiles];   // both CTAs: this tile pair's accumulator is complete (all K groups)
  uint64_t acc_empty[kKaccTiles];  // CTA 0: both CTAs' epilogue warps have read it (2 x 8 arrivals)
  uint64_t drain;                // failure path only
  uint32_t tmem_base;
  volatile uint32_t abort;
};
static_assert(sizeof(KaccHeader) <= 320, "barriers must fit the first 320 bytes of the header");

// What the roles need to know about a K group, kept in shared memory (bytes 320..768 of the header) so that no role
// has a global-memory round trip on its path at every step; the CTA's own segment descriptors sit in the upper
// half of the table area (bytes 1792..2816, the tables of warps that do not decode here) when they fit.
struct KaccGroup {
  uint16_t n_boxes;        // K range of the group in 64-column boxes
  uint16_t n_seg;          // segments of this CTA's job
  uint32_t x_koff;         // first activation column
};
constexpr int kKaccMaxGroups = 56;
constexpr uint32_t kKaccSegArea = 1024;

__device__ __forceinline__ void fence_acq_rel_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }

// SPLIT: two warps share a decode task (weight buffers of at most 64 x 256: four tasks for the eight warps).
template <bool SPLIT>
__global__ void __launch_bounds__(kThreads, 1)
dqgemm_kacc_kernel(const __grid_constant__ CUtensorMap xmap, const Job* __restrict__ jobs, const Seg* __restrict__ segs,
                   const __nv_bfloat16* __restrict__ x, int ldx, int n_groups, int T, float* __restrict__ out, int ldo,
                   int* __restrict__ err, uint32_t n_stages,
                   uint32_t bps, uint32_t w_buf_bytes, uint32_t hdr_bytes, uint32_t seg_stride,
                   unsigned long long* stamps) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = smem_raw;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { stamp_min(stamps, STAMP_FIRST_START); stamp_max(stamps, STAMP_LAST_START); }
  const uint32_t rank = cluster_ctarank();
  const uint32_t pair_base = blockIdx.x & ~1u;
  const uint32_t n_cols64 = gridDim.x;                 // 64-feature tiles: job (g, c) = jobs[g * n_cols64 + c]

  KaccHeader* hdr = reinterpret_cast<KaccHeader*>(smem);
  KaccGroup* ginfo = reinterpret_cast<KaccGroup*>(smem + 320);
  uint16_t* tables = reinterpret_cast<uint16_t*>(smem + 768);
  Seg* seg_sm = reinterpret_cast<Seg*>(smem + 1792);
  const bool segs_in_smem = static_cast<uint32_t>(n_groups) * seg_stride * sizeof(Seg) <= kKaccSegArea;
  uint8_t* xsm = smem + hdr_bytes;
  const uint32_t stage_bytes = bps * kBoxBytes;         // a ring stage holds `bps` boxes of 64 columns
  uint8_t* wsm = xsm + n_stages * stage_bytes;          // two buffers of w_buf_bytes
  const uint32_t k_max = w_buf_bytes / (64 * 2);        // columns a buffer holds

  // both CTAs look at both halves of every K group, so a refused pair leaves together
  bool bad = n_groups < 1 || n_groups > kKaccMaxGroups || n_stages < 2 || n_stages > kKaccMaxStages || (w_buf_bytes & 1023) != 0 || (bps != 1 && bps != 2) || (gridDim.x & 1) != 0 || (hdr_bytes & 1023) != 0 ||
             768 + kWarps * kTableStride * 2 > hdr_bytes || (smem_addr(smem_raw) & 1023u) != 0;
  for (int g = 0; g < n_groups; ++g) {      // no early exit: the loads of all groups are in flight together
    const uint32_t i0 = g * n_cols64 + pair_base;
    const Job a = jobs[i0], b = jobs[i0 + 1];
    bad |= a.n_rows != 64 || b.n_rows != 64 || a.k_total != b.k_total || a.x_koff != b.x_koff || a.k_total == 0 ||
          a.k_total > k_max || (a.k_total % (kChunkK * bps)) != 0 || a.n_seg == 0 || b.n_seg == 0 || a.n_seg > seg_stride ||
          b.n_seg > seg_stride || a.n_seg > kMaxSegs || b.n_seg > kMaxSegs || a.seg_begin != i0 * seg_stride ||
          b.seg_begin != (i0 + 1) * seg_stride || a.out_col != pair_base * 64 || b.out_col != (pair_base + 1) * 64;
  }
  if (bad) {
    if (tid == 0) atomicCAS(err, ERR_NONE, ERR_BAD_JOB);
    return;
  }

  const int n_mtiles = (T + kTileM - 1) / kTileM;
  const uint32_t n_mpairs = (n_mtiles + 1) / 2;
  const uint32_t my_pairs = blockIdx.y < n_mpairs ? (n_mpairs - blockIdx.y + gridDim.y - 1) / gridDim.y : 0;
  const uint32_t n_blocks = (my_pairs + kKaccTiles - 1) / kKaccTiles;
  const uint32_t n_steps = n_blocks * static_cast<uint32_t>(n_groups);       // (block, K group) steps of this pair
  const uint32_t xsm_addr = smem_addr(xsm);
  auto tile_row0 = [&](uint32_t ti) { return static_cast<int>((2 * (blockIdx.y + ti * gridDim.y) + rank) * kTileM); };
  auto tiles_in = [&](uint32_t blk) { return my_pairs - blk * kKaccTiles < kKaccTiles ? my_pairs - blk * kKaccTiles : kKaccTiles; };

  if (tid < static_cast<uint32_t>(n_groups)) {
    const Job j = jobs[tid * n_cols64 + blockIdx.x];
    ginfo[tid].n_boxes = static_cast<uint16_t>(j.k_total / kChunkK);
    ginfo[tid].n_seg = static_cast<uint16_t>(j.n_seg);
    ginfo[tid].x_koff = j.x_koff;
  }
  if (segs_in_smem) {
    constexpr uint32_t kSegWords = sizeof(Seg) / 4;
    const uint32_t per_group = seg_stride * kSegWords, n_words = static_cast<uint32_t>(n_groups) * per_group;
    const uint32_t* src = reinterpret_cast<const uint32_t*>(segs);
    uint32_t* dst = reinterpret_cast<uint32_t*>(seg_sm);
    for (uint32_t w = tid; w < n_words; w += kThreads) {
      const uint32_t g = w / per_group, k = w % per_group;
      dst[w] = __ldg(src + (static_cast<size_t>(g) * n_cols64 + blockIdx.x) * per_group + k);
    }
  }
  if (tid == 0) {
    for (uint32_t s = 0; s < n_stages; ++s) {
      mbar_init(smem_addr(&hdr->full[s]), 1);
      mbar_init(smem_addr(&hdr->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_addr(&hdr->w_full[b]), 2);
      mbar_init(smem_addr(&hdr->w_empty[b]), 1);
    }
    for (uint32_t t = 0; t < kKaccTiles; ++t) {
      mbar_init(smem_addr(&hdr->acc_full[t]), 1);
      mbar_init(smem_addr(&hdr->acc_empty[t]), 2 * kKaccGroupWarps);
    }
    mbar_init(smem_addr(&hdr->drain), 1);
    hdr->abort = 0;
    mbar_fence_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_addr(&hdr->tmem_base), kKaccTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = hdr->tmem_base;
  // activation boxes the pair brings in over the whole launch (for the "does anybody still wait" rule of the commits)
  uint32_t boxes_per_tile = 0;
  for (int g = 0; g < n_groups; ++g) boxes_per_tile += ginfo[g].n_boxes;
  const uint32_t total_chunks = my_pairs * boxes_per_tile / bps;      // ring stages filled over the whole launch
  cluster_sync_all();               // the partner's barriers are initialised before anything arrives on them
  pdl_launch_dependents();

  bool failed = false;
  if (warp == 0) {
    // ---- producer (one in each CTA): own token tile into own ring, bytes credited to CTA 0's barrier
    if (lane == 0) {
      pdl_wait();                   // the activations are the previous kernel's output
      stamp_min(stamps, STAMP_RELEASE);
      uint32_t c = 0, stage = 0, round = 0;
      for (uint32_t blk = 0; blk < n_blocks && !failed; ++blk) {
        const uint32_t nt = tiles_in(blk);
        for (int g = 0; g < n_groups && !failed; ++g) {
          const uint32_t nc = ginfo[g].n_boxes / bps, x_koff = ginfo[g].x_koff, rot = (blockIdx.x >> 1) % nc;
          for (uint32_t t = 0; t < nt && !failed; ++t) {
            const int row0 = tile_row0(blk * kKaccTiles + t);
            for (uint32_t ci = 0; ci < nc; ++ci, ++c) {
              if (round > 0 && !mbar_wait_bounded_relaxed(smem_addr(&hdr->empty[stage]), (round - 1) & 1)) {
                failed = true;
                break;
              }
              const uint32_t ch = ci + rot < nc ? ci + rot : ci + rot - nc;
              if (rank == 0) mbar_expect_tx(smem_addr(&hdr->full[stage]), 2 * stage_bytes);
              const uint32_t bar = map_to_cta(smem_addr(&hdr->full[stage]), 0);
              for (uint32_t b = 0; b < bps; ++b)
                tma_load_2d_pair(xsm_addr + stage * stage_bytes + b * kBoxBytes, &xmap,
                                 static_cast<int>(x_koff + (ch * bps + b) * kChunkK), row0, bar);
              if (++stage == n_stages) { stage = 0; ++round; }
            }
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (rank == 0) {
      // ---- MMA issuer of the pair
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((256u >> 4) << 24);
      const uint32_t w_lbo = 64 * 16;
      const uint64_t a_desc0 = umma_smem_desc_sw128(xsm_addr);
      const uint64_t b_desc_buf[2] = {umma_smem_desc(smem_addr(wsm), w_lbo, 128),
                                      umma_smem_desc(smem_addr(wsm + w_buf_bytes), w_lbo, 128)};
      const uint32_t a_stage_step = stage_bytes >> 4, a_box_step = kBoxBytes >> 4;
      const uint32_t b_ks_step = (2 * w_lbo) >> 4, b_chunk_step = 4 * b_ks_step;
      uint32_t c = 0, stage = 0, round = 0, step = 0, issued = 0;
      long long wait_w = 0, wait_x = 0, wait_acc = 0;      // SM cycles the issuer spent waiting: weights, activations, drain
      for (uint32_t blk = 0; blk < n_blocks && !failed; ++blk) {
        const uint32_t nt = tiles_in(blk);
        for (int g = 0; g < n_groups && !failed; ++g, ++step) {
          const uint32_t wb = step & 1;
          const uint32_t nc = ginfo[g].n_boxes / bps, rot = (blockIdx.x >> 1) % nc;
          const long long tw0 = clock64();
          if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_addr(&hdr->w_full[wb]), (step >> 1) & 1))) {
            failed = true;
            break;
          }
          wait_w += clock64() - tw0;
          fence_acq_rel_cluster();      // the other CTA's half of the tile was written by the other CTA's threads
          tc_fence_after_sync();
          for (uint32_t t = 0; t < nt && !failed; ++t) {
            const uint32_t d_addr = tmem_base + t * kKaccAccCols;
            if (g == 0 && blk > 0) {      // the previous block's sums of this tile slot have been read
              const long long ta0 = clock64();
              if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_addr(&hdr->acc_empty[t]), (blk - 1) & 1))) {
                failed = true;
                break;
              }
              wait_acc += clock64() - ta0;
              tc_fence_after_sync();
            }
            for (uint32_t ci = 0; ci < nc; ++ci, ++c) {
              const long long tx0 = clock64();
              if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_addr(&hdr->full[stage]), round & 1))) {
                failed = true;
                break;
              }
              wait_x += clock64() - tx0;
              tc_fence_after_sync();
              const uint32_t ch = ci + rot < nc ? ci + rot : ci + rot - nc;
              if (elect_one()) {
                uint64_t da = a_desc0 + stage * a_stage_step, db = b_desc_buf[wb] + ch * bps * b_chunk_step;
                umma_bf16_ss_x4_pair(d_addr, da, db, 2, b_ks_step, idesc, (g != 0 || ci != 0) ? 1u : 0u);
                for (uint32_t b = 1; b < bps; ++b) {
                  da += a_box_step;
                  db += b_chunk_step;
                  umma_bf16_ss_x4_pair(d_addr, da, db, 2, b_ks_step, idesc, 1u);
                }
                if (c + n_stages < total_chunks) umma_commit_pair(smem_addr(&hdr->empty[stage]));
              }
              __syncwarp();
              issued = c + 1;
              if (++stage == n_stages) { stage = 0; ++round; }
            }
            if (!failed && g + 1 == n_groups) {      // last K group: this tile is complete, its drain may start
              if (elect_one()) umma_commit_pair(smem_addr(&hdr->acc_full[t]));
              __syncwarp();
            }
          }
          if (!failed && step + 2 < n_steps) {
            if (elect_one()) umma_commit_pair(smem_addr(&hdr->w_empty[wb]));
            __syncwarp();
          }
        }
      }
      if (lane == 0 && stamps != nullptr) {      // maxima over the launch's pairs, stored complemented like the time stamps
        atomicMin(stamps + STAMP_ACC, ~static_cast<unsigned long long>(wait_w));
        atomicMin(stamps + STAMP_EXCHANGED, ~static_cast<unsigned long long>(wait_x));
        atomicMin(stamps + 7, ~static_cast<unsigned long long>(wait_acc));
      }
      if (failed && issued > 0) {
        if (elect_one()) umma_commit_pair(smem_addr(&hdr->drain));
        __syncwarp();
        (void)mbar_wait_bounded(smem_addr(&hdr->drain), 0);
      }
    }
  } else if (warp >= kKaccPrefetchWarp0 && x != nullptr) {
    // ---- otherwise idle: pull the activations of the step after next into L2 (the host passes x only when the
    // operand is larger than L2: 16,384 tokens x 4096 columns of bf16 are 134 MB).  Without this every box's first
    // reader - and the seven other column pairs
    // that ask for the same lines at the same moment - waits for DRAM.  The column pairs share the work: pair p
    // takes the boxes p, p + n_pairs, ... of a K group, each thread one 128-byte line of one token row.  Paced by the
    // same barrier as the decode (a weight buffer is free = the step two back has been computed).
    pdl_wait();
    const uint32_t n_pairs = gridDim.x >> 1, pair = blockIdx.x >> 1;
    const uint32_t r_in_tile = (warp - kKaccPrefetchWarp0) * 32 + lane;        // 0..127: the CTA's rows of a tile
    uint32_t step = 0;
    for (uint32_t blk = 0; blk < n_blocks && !failed; ++blk) {
      const uint32_t nt = tiles_in(blk);
      for (int g = 0; g < n_groups; ++g, ++step) {
        if (step >= 2) {
          uint32_t ok = 1;
          if (lane == 0) ok = hdr->abort ? 0u : (mbar_wait_bounded_relaxed(smem_addr(&hdr->w_empty[step & 1]), ((step >> 1) - 1) & 1) ? 1u : 0u);
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) { failed = true; break; }
        }
        const uint32_t nb = ginfo[g].n_boxes, x_koff = ginfo[g].x_koff;
        for (uint32_t t = 0; t < nt; ++t) {
          const int row = tile_row0(blk * kKaccTiles + t) + static_cast<int>(r_in_tile);
          if (row < T) {
            const __nv_bfloat16* line = x + static_cast<size_t>(row) * ldx + x_koff;
            for (uint32_t b = pair; b < nb; b += n_pairs)
              asm volatile("prefetch.global.L2 [%0];" ::"l"(line + b * kChunkK));
          }
        }
      }
    }
  } else if (warp >= kKaccGroupWarp0 && warp < kKaccGroupWarp0 + kKaccGroupWarps) {
    // ---- decode group / epilogue.  No early exit: the group meets at named barriers inside the decode.
    const uint32_t gtid = tid - kKaccGroupWarp0 * 32;
    const uint32_t q = warp & 3, half = (warp - kKaccGroupWarp0) >> 2;
    bool released = false;
    // lane 0 polls and the warp takes its result; once the CTA has given up nobody waits any more
    auto wait_uniform = [&](uint32_t bar, uint32_t parity) {
      uint32_t ok = 1;
      if (lane == 0) ok = (failed || hdr->abort) ? 0u : (mbar_wait_bounded(bar, parity) ? 1u : 0u);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) {
        failed = true;
        if (lane == 0) hdr->abort = 1;
      }
    };
    auto epilogue = [&](uint32_t blk) {
      if (!released) { pdl_wait(); released = true; }               // `out` may still be read by an earlier kernel
      const uint32_t nt = tiles_in(blk);
      for (uint32_t t = 0; t < nt; ++t) {
        wait_uniform(smem_addr(&hdr->acc_full[t]), blk & 1);
        tc_fence_after_sync();
        const int row = tile_row0(blk * kKaccTiles + t) + static_cast<int>(q * 32 + lane);
        float* drow = out + static_cast<size_t>(row < T ? row : 0) * ldo + pair_base * 64 + half * 64;
        const uint32_t taddr = tmem_base + ((q * 32) << 16) + t * kKaccAccCols + half * 64;
#pragma unroll
        for (uint32_t col = 0; col < 64; col += 32) {
          uint32_t r[32];
          tmem_ld_32x32b_x32(taddr + col, r);
          tc_wait_ld();
          if (row < T) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              float v[16];
#pragma unroll
              for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[h * 16 + i]);
              store_row16<float>(drow + col + h * 16, v);
            }
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster_cta_scope(map_to_cta(smem_addr(&hdr->acc_empty[t]), 0));
      }
    };
    uint32_t step = 0;
    for (uint32_t blk = 0; blk < n_blocks; ++blk) {
      for (int g = 0; g < n_groups; ++g, ++step) {
        const uint32_t wb = step & 1;
        if (step >= 2) wait_uniform(smem_addr(&hdr->w_empty[wb]), ((step >> 1) - 1) & 1);
        Job job{};
        job.n_rows = 64; job.k_total = ginfo[g].n_boxes * kChunkK; job.n_seg = ginfo[g].n_seg;
        const Seg* my_segs = segs_in_smem ? seg_sm + static_cast<size_t>(g) * seg_stride
                                          : segs + (static_cast<size_t>(g) * n_cols64 + blockIdx.x) * seg_stride;
        decode_weight_tile_group<kKaccGroupWarps, SPLIT>(job, my_segs, tables, wsm + wb * w_buf_bytes, gtid,
                                                         kKaccGroupBarrier);
        if (gtid == 0) {
          if (step == 0) stamp_max(stamps, STAMP_DECODED);
          mbar_arrive_cluster(map_to_cta(smem_addr(&hdr->w_full[wb]), 0));
        }
        // the previous block is drained after this block's first tile is decoded: that decode ran under the
        // previous block's last MMAs
        if (g == 0 && blk > 0) epilogue(blk - 1);
      }
    }
    if (n_blocks > 0) epilogue(n_blocks - 1);
  }
  if (failed) {
    hdr->abort = 1;
    if (lane == 0) atomicCAS(err, ERR_NONE, ERR_WAIT_TIMEOUT);
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();      // neither CTA frees tensor memory or exits while the pair's MMAs may still use it
  if (warp == 1) tmem_dealloc_pair(tmem_base, kKaccTmemCols);
  if (tid == 0) stamp_max(stamps, STAMP_LAST_END);
}

}  // namespace

// Ring stages that fit beside two weight buffers of 64 rows x k_group columns.
uint32_t gemm_kacc_stages(uint32_t hdr_bytes, uint32_t k_group, uint32_t bps, size_t smem_limit) {
  const size_t w = 2 * static_cast<size_t>(64) * k_group * 2, stage = static_cast<size_t>(bps) * kBoxBytes;
  if (smem_limit < hdr_bytes + w + 2 * stage) return 0;
  return static_cast<uint32_t>(std::min<size_t>(kKaccMaxStages, (smem_limit - hdr_bytes - w) / stage));
}

size_t gemm_kacc_smem_bytes(uint32_t hdr_bytes, uint32_t n_stages, uint32_t bps, uint32_t k_group) {
  return static_cast<size_t>(hdr_bytes) + static_cast<size_t>(n_stages) * bps * kBoxBytes +
         2 * static_cast<size_t>(64) * k_group * 2;
}

cudaError_t gemm_kacc_configure() {
  cudaError_t e = cudaFuncSetAttribute(dqgemm_kacc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(dqgemm_kacc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
}

cudaError_t launch_gemm_kacc(const KaccLaunch& p, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.n_cols64, p.m_ctas);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = gemm_kacc_smem_bytes(p.hdr_bytes, p.n_stages, p.bps, p.k_group);
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.pdl ? 2 : 1;
  const uint32_t w_buf_bytes = 64u * p.k_group * 2u;
  if (p.k_group <= 256)      // at most four decode tasks per weight tile: two warps share each
    return cudaLaunchKernelEx(&cfg, dqgemm_kacc_kernel<true>, p.xmap, p.jobs, p.segs, static_cast<const __nv_bfloat16*>(p.x), p.ldx, p.n_groups, p.T, p.out, p.ldo, p.err,
                              p.n_stages, p.bps, w_buf_bytes, p.hdr_bytes, p.seg_stride, p.stamps);
  return cudaLaunchKernelEx(&cfg, dqgemm_kacc_kernel<false>, p.xmap, p.jobs, p.segs, static_cast<const __nv_bfloat16*>(p.x), p.ldx, p.n_groups, p.T, p.out, p.ldo, p.err,
                            p.n_stages, p.bps, w_buf_bytes, p.hdr_bytes, p.seg_stride, p.stamps);
}

}  // namespace sti
