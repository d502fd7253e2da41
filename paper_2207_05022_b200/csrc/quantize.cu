// Shard quantizer on the device (Section 6: Gaussian outlier-aware dictionary quantization).
//
// Two kernels produce the same output.  quantize_select_kernel (further down, the default) never sorts: the
// clusters are equal-population slices of the sorted order, so all it needs are the 2^k - 1 elements that sit at
// the slice boundaries, which it finds by rank selection.  Units it cannot handle (zero variance, more than
// kSelMaxSeg weights in one selection bin) are marked and done by quantize_units_kernel, the sorting kernel:
//
// One CTA of 1024 threads per shard unit runs the paper's steps in order on the unit's flat fp32 array:
//   1. maximum-likelihood fit of one Gaussian (mean, 1/n variance; fp64 block reductions);
//   2. outliers = weights whose log-likelihood is below -4: their (offset, value) pairs are written in
//      ascending offset order by a stable compaction; the other weights become (sortable key, offset) pairs;
//   3. a least-significant-digit radix sort (4 passes of 8 bits, stable, so equal weights keep their
//      original order) of the pairs between two workspace buffers, 4096 elements per step: every thread
//      holds one element of each of four consecutive 1024-element stripes, ranks come from warp match
//      masks plus a per-(stripe, warp, digit) count table in shared memory;
//   4. 2^k clusters of equal population over the sorted order, cluster c = [floor(c n'/2^k), floor((c+1) n'/2^k)),
//      centroid = arithmetic mean (fp64 sum, rounded once to fp32);
//   5. every weight gets its cluster's k-bit index; an outlier's slot gets the nearest centroid's index
//      (lower index on a tie);
//   6. the indexes are packed into the upload format: index i at stream bits [i k, i k + k), LSB first.
// All decisions that yield integers (outlier test, sort order, cluster of a rank, nearest centroid) are taken
// in fp64 / exact integer arithmetic.  Units are independent: the grid is the number of units.
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/sti_quantize.h"

namespace {

constexpr int kQThreads = 1024;
constexpr int kQWarps = kQThreads / 32;

constexpr int kItems = 4;             // elements per thread and chunk; a chunk is 4 stripes of 1024 consecutive elements
constexpr int kSlots = kItems * kQWarps;   // (stripe, warp) pairs of a chunk, in element order

struct QuantShared {
  double red[kQWarps];
  uint32_t hist[256];
  uint32_t base[2][256];
  uint8_t wcount[kSlots][256];       // per chunk: elements of digit d held by (stripe, warp) slot q
  uint16_t woff[kSlots][256];        // per chunk: elements of digit d held by the slots before q
  uint32_t wcnt_in[kSlots], wcnt_out[kSlots];
  uint32_t tot_in, tot_out;
  uint16_t stripe_tot[kItems][256];  // per chunk: elements of digit d in stripe j
  uint32_t bounds[65];
  float cents[64];
};

__device__ __forceinline__ double block_sum(double v, double* red, int tid) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((tid & 31) == 0) red[tid >> 5] = v;
  __syncthreads();
  double t = 0.0;
  for (int w = 0; w < kQWarps; ++w) t += red[w];
  __syncthreads();
  return t;
}

// Maximum-likelihood mean and 1/n variance in fp64 (n is a multiple of 4; four 16-byte loads in flight per thread).
__device__ __forceinline__ void fit_gaussian(const float* w, uint32_t n, double* red, int tid, double& mu, double& var) {
  double s = 0.0;
  for (uint32_t i0 = 4u * tid; i0 < n; i0 += 16u * kQThreads) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t i = i0 + u * 4u * kQThreads;
      v[u] = i < n ? *reinterpret_cast<const float4*>(w + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      s += (static_cast<double>(v[u].x) + static_cast<double>(v[u].y)) + (static_cast<double>(v[u].z) + static_cast<double>(v[u].w));
  }
  mu = block_sum(s, red, tid) / static_cast<double>(n);
  double q = 0.0;
  for (uint32_t i0 = 4u * tid; i0 < n; i0 += 16u * kQThreads) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t i = i0 + u * 4u * kQThreads;
      v[u] = i < n ? *reinterpret_cast<const float4*>(w + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (i0 + u * 4u * kQThreads >= n) continue;
      const double d0 = static_cast<double>(v[u].x) - mu, d1 = static_cast<double>(v[u].y) - mu;
      const double d2 = static_cast<double>(v[u].z) - mu, d3 = static_cast<double>(v[u].w) - mu;
      q += (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
    }
  }
  var = block_sum(q, red, tid) / static_cast<double>(n);
}

// Order-preserving map of an fp32 bit pattern to an unsigned key (-0 sorts as +0).
__device__ __forceinline__ uint32_t sort_key(float x) {
  uint32_t u = __float_as_uint(x);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_value(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
// Lanes of the warp that hold the same 8-bit digit (valid lanes only): eight ballots, a fixed cost whatever
// the number of distinct digits (a hardware match instruction walks the distinct values one by one).
__device__ __forceinline__ uint32_t same_digit_lanes(uint32_t d, bool valid) {
  uint32_t peers = __ballot_sync(0xffffffffu, valid);
#pragma unroll
  for (int b = 0; b < 8; ++b) {
    const bool bit = (d >> b) & 1u;
    const uint32_t bal = __ballot_sync(0xffffffffu, bit);
    peers &= bit ? bal : ~bal;
  }
  return peers;
}
// inv2var = 1 / (2 var); with zero variance c0 is +inf and 0 * inf is NaN, which compares false: no outliers
__device__ __forceinline__ bool is_outlier(float x, double mu, double inv2var, double c0) {
  const double d = static_cast<double>(x) - mu;
  const double ll = c0 - d * d * inv2var;
  return ll < -4.0;
}

__global__ void __launch_bounds__(kQThreads, 1)
quantize_units_kernel(const float* w_all, uint32_t n, int bits, uint32_t* codes_all, float* cent_all, uint32_t* ooff_all,
                      float* oval_all, uint32_t max_out, uint32_t* n_out_all, uint8_t* ws_all, size_t ws_per_unit,
                      const uint8_t* only_marked) {
  extern __shared__ __align__(16) uint8_t q_smem[];
  QuantShared& sm = *reinterpret_cast<QuantShared*>(q_smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t unit = blockIdx.x;
  if (only_marked != nullptr && only_marked[unit] == 0) return;      // the selection kernel has done this unit
  const uint32_t K = 1u << bits;
  const float* w = w_all + static_cast<size_t>(unit) * n;
  uint32_t* codes = codes_all + static_cast<size_t>(unit) * (static_cast<size_t>(n) * bits / 32);
  float* cent = cent_all + static_cast<size_t>(unit) * K;
  uint32_t* ooff = ooff_all + static_cast<size_t>(unit) * max_out;
  float* oval = oval_all + static_cast<size_t>(unit) * max_out;
  uint8_t* ws = ws_all + static_cast<size_t>(unit) * ws_per_unit;
  uint32_t* key[2] = {reinterpret_cast<uint32_t*>(ws), reinterpret_cast<uint32_t*>(ws) + 2 * static_cast<size_t>(n)};
  uint32_t* idx[2] = {key[0] + n, key[1] + n};
  uint8_t* codes8 = ws + 16 * static_cast<size_t>(n);

  // ---- 1. Gaussian fit
  double mu, var;
  fit_gaussian(w, n, sm.red, tid, mu, var);
  const double c0 = -0.5 * log(2.0 * 3.14159265358979323846 * var);
  const double inv2var = 1.0 / (2.0 * var);

  // ---- 2. outliers out (ascending offsets), the rest as (key, offset) pairs, both by stable compaction
  uint32_t n_in = 0, n_out = 0;
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (uint32_t start = 0; start < n; start += kItems * kQThreads) {
    float x[kItems];
    bool in[kItems], out[kItems];
    uint32_t m_in[kItems], m_out[kItems];
#pragma unroll
    for (int j = 0; j < kItems; ++j) {
      const uint32_t i = start + j * kQThreads + tid;
      x[j] = i < n ? w[i] : 0.f;
    }
#pragma unroll
    for (int j = 0; j < kItems; ++j) {
      const uint32_t i = start + j * kQThreads + tid;
      out[j] = i < n && is_outlier(x[j], mu, inv2var, c0);
      in[j] = i < n && !out[j];
      m_in[j] = __ballot_sync(0xffffffffu, in[j]);
      m_out[j] = __ballot_sync(0xffffffffu, out[j]);
      if (lane == 0) { sm.wcnt_in[j * kQWarps + warp] = __popc(m_in[j]); sm.wcnt_out[j * kQWarps + warp] = __popc(m_out[j]); }
    }
    __syncthreads();
    // exclusive prefix of the 128 slot counts in element order: warp 0, four slots per lane, one shuffle scan
    if (warp == 0) {
      uint32_t a[4], b[4], sa = 0, sb = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) { a[e] = sm.wcnt_in[4 * lane + e]; b[e] = sm.wcnt_out[4 * lane + e]; sa += a[e]; sb += b[e]; }
      uint32_t ia = sa, ib = sb;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t ta = __shfl_up_sync(0xffffffffu, ia, o), tb = __shfl_up_sync(0xffffffffu, ib, o);
        if (lane >= o) { ia += ta; ib += tb; }
      }
      uint32_t ea = ia - sa, eb = ib - sb;
#pragma unroll
      for (int e = 0; e < 4; ++e) { sm.wcnt_in[4 * lane + e] = ea; sm.wcnt_out[4 * lane + e] = eb; ea += a[e]; eb += b[e]; }
      if (lane == 31) { sm.tot_in = ia; sm.tot_out = ib; }
    }
    __syncthreads();
    const uint32_t run_in = sm.tot_in, run_out = sm.tot_out;
    uint32_t pre_in[kItems], pre_out[kItems];
#pragma unroll
    for (int j = 0; j < kItems; ++j) { pre_in[j] = sm.wcnt_in[j * kQWarps + warp]; pre_out[j] = sm.wcnt_out[j * kQWarps + warp]; }
#pragma unroll
    for (int j = 0; j < kItems; ++j) {
      const uint32_t i = start + j * kQThreads + tid;
      if (in[j]) {
        const uint32_t dst = n_in + pre_in[j] + __popc(m_in[j] & lt_mask);
        key[0][dst] = sort_key(x[j]);
        idx[0][dst] = i;
      }
      if (out[j]) {
        const uint32_t dst = n_out + pre_out[j] + __popc(m_out[j] & lt_mask);
        if (dst < max_out) { ooff[dst] = i; oval[dst] = x[j]; }
      }
    }
    n_in += run_in;
    n_out += run_out;
    __syncthreads();
  }
  if (tid == 0) n_out_all[unit] = n_out;

  // ---- 3. stable LSD radix sort of the n_in pairs, 8 bits per pass
  int cur = 0;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 8 * pass;
    const uint32_t* ksrc = key[cur];
    const uint32_t* isrc = idx[cur];
    uint32_t* kdst = key[cur ^ 1];
    uint32_t* idst = idx[cur ^ 1];
    if (tid < 256) sm.hist[tid] = 0;
    __syncthreads();
    // one shared-memory atomic per distinct digit of a warp (the high digits of weights fall into a few bins)
    const uint32_t n_in_up = (n_in + 31u) & ~31u;          // whole warps take every iteration (match is warp-wide)
    for (uint32_t i0 = tid; i0 < n_in_up; i0 += 8 * kQThreads) {
      uint32_t kv[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) { const uint32_t i = i0 + u * kQThreads; kv[u] = i < n_in ? ksrc[i] : 0u; }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint32_t i = i0 + u * kQThreads;
        const uint32_t dg = (kv[u] >> shift) & 255u;
        const uint32_t pm = same_digit_lanes(dg, i < n_in);
        if (i < n_in && (pm & lt_mask) == 0) atomicAdd(&sm.hist[dg], static_cast<uint32_t>(__popc(pm)));
      }
    }
    __syncthreads();
    // exclusive prefix of the histogram -> first destination of every digit
    if (tid < 256) sm.base[0][tid] = sm.hist[tid];
    __syncthreads();
    for (int o = 1; o < 256; o <<= 1) {
      uint32_t v = 0;
      if (tid < 256 && tid >= o) v = sm.base[0][tid - o];
      __syncthreads();
      if (tid < 256) sm.base[0][tid] += v;
      __syncthreads();
    }
    if (tid < 256) sm.base[0][tid] -= sm.hist[tid];
    __syncthreads();
    int bsel = 0;
    for (uint32_t start = 0; start < n_in; start += kItems * kQThreads) {
      uint32_t kk[kItems], ii[kItems], d[kItems], peers[kItems];
      bool valid[kItems];
#pragma unroll
      for (int j = 0; j < kItems; ++j) {
        const uint32_t i = start + j * kQThreads + tid;
        valid[j] = i < n_in;
        kk[j] = valid[j] ? ksrc[i] : 0u;
        ii[j] = valid[j] ? isrc[i] : 0u;
      }
      for (int z = tid; z < kSlots * 256 / 4; z += kQThreads) reinterpret_cast<uint32_t*>(&sm.wcount[0][0])[z] = 0u;
#pragma unroll
      for (int j = 0; j < kItems; ++j) {
        d[j] = (kk[j] >> shift) & 255u;
        peers[j] = same_digit_lanes(d[j], valid[j]);
      }
      __syncthreads();
#pragma unroll
      for (int j = 0; j < kItems; ++j)
        if (valid[j] && (peers[j] & lt_mask) == 0) sm.wcount[j * kQWarps + warp][d[j]] = static_cast<uint8_t>(__popc(peers[j]));
      __syncthreads();
      {
        // thread (stripe sj, digit sd): prefix over the stripe's 32 warps; the four stripes run side by side
        const int sj = tid >> 8, sd = tid & 255;
        uint32_t pre = 0;
        for (int ww = 0; ww < kQWarps; ++ww) {
          sm.woff[sj * kQWarps + ww][sd] = static_cast<uint16_t>(pre);
          pre += sm.wcount[sj * kQWarps + ww][sd];
        }
        sm.stripe_tot[sj][sd] = static_cast<uint16_t>(pre);
      }
      __syncthreads();
      if (tid < 256) {
        uint32_t t = 0;
#pragma unroll
        for (int j = 0; j < kItems; ++j) t += sm.stripe_tot[j][tid];
        sm.base[bsel ^ 1][tid] = sm.base[bsel][tid] + t;
      }
#pragma unroll
      for (int j = 0; j < kItems; ++j) {
        if (valid[j]) {
          uint32_t dst = sm.base[bsel][d[j]] + sm.woff[j * kQWarps + warp][d[j]] + __popc(peers[j] & lt_mask);
#pragma unroll
          for (int jj = 0; jj < kItems; ++jj)
            if (jj < j) dst += sm.stripe_tot[jj][d[j]];
          kdst[dst] = kk[j];
          idst[dst] = ii[j];
        }
      }
      bsel ^= 1;
      __syncthreads();
    }
    cur ^= 1;
  }
  const uint32_t* ks = key[cur];
  const uint32_t* is = idx[cur];

  // ---- 4. equal-population clusters, centroid = mean
  if (tid <= static_cast<int>(K))
    sm.bounds[tid] = static_cast<uint32_t>(static_cast<uint64_t>(tid) * n_in / K);
  __syncthreads();
  for (uint32_t c = warp; c < K; c += kQWarps) {
    const uint32_t lo = sm.bounds[c], hi = sm.bounds[c + 1];
    double acc = 0.0;
    for (uint32_t r = lo + lane; r < hi; r += 32) acc += static_cast<double>(key_value(ks[r]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) {
      const float m = hi > lo ? static_cast<float>(acc / static_cast<double>(hi - lo)) : 0.f;
      sm.cents[c] = m;
      cent[c] = m;
    }
  }
  __syncthreads();

  // ---- 5. indexes: the cluster of a weight's rank; for an outlier the nearest centroid
  for (uint32_t r0 = tid; r0 < n_in; r0 += 8 * kQThreads) {
    uint32_t dst[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) { const uint32_t r = r0 + u * kQThreads; dst[u] = r < n_in ? is[r] : 0u; }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const uint32_t r = r0 + u * kQThreads;
      if (r >= n_in) continue;
      uint32_t c = r * K / n_in;             // r < 2^26 and K <= 2^6: the product fits 32 bits
      while (c + 1 < K && sm.bounds[c + 1] <= r) ++c;
      while (c > 0 && sm.bounds[c] > r) --c;
      codes8[dst[u]] = static_cast<uint8_t>(c);
    }
  }
  if (n_out > 0) {
    for (uint32_t i0 = tid; i0 < n; i0 += 8 * kQThreads) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) { const uint32_t i = i0 + u * kQThreads; v[u] = i < n ? w[i] : 0.f; }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint32_t i = i0 + u * kQThreads;
        if (i >= n || !is_outlier(v[u], mu, inv2var, c0)) continue;
        uint32_t best = 0;
        double bd = fabs(static_cast<double>(v[u]) - static_cast<double>(sm.cents[0]));
        for (uint32_t c = 1; c < K; ++c) {
          const double dd = fabs(static_cast<double>(v[u]) - static_cast<double>(sm.cents[c]));
          if (dd < bd) { bd = dd; best = c; }
        }
        codes8[i] = static_cast<uint8_t>(best);
      }
    }
  }
  __syncthreads();

  // ---- 6. the index stream: 32 consecutive indexes are exactly `bits` words; a thread reads them as two 16-byte
  //         loads and shifts them into a 64-bit window, emitting a word whenever 32 bits are complete
  const uint32_t n_groups = n / 32;
  for (uint32_t gidx = tid; gidx < n_groups; gidx += kQThreads) {
    const uint4 a = *reinterpret_cast<const uint4*>(codes8 + static_cast<size_t>(gidx) * 32);
    const uint4 b = *reinterpret_cast<const uint4*>(codes8 + static_cast<size_t>(gidx) * 32 + 16);
    const uint32_t src[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint64_t window = 0;
    uint32_t fill = 0, out_w = gidx * bits;
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      const uint32_t code = (src[e >> 2] >> (8 * (e & 3))) & 255u;
      window |= static_cast<uint64_t>(code) << fill;
      fill += bits;
      if (fill >= 32u) {
        codes[out_w++] = static_cast<uint32_t>(window);
        window >>= 32;
        fill -= 32u;
      }
    }
  }
}


// ---------------------------------------------------------------------------------------------------------------
// Selection kernel.  The stable sorted order of the inliers is the lexicographic order of (key, offset) pairs, and
// cluster c starts at sorted rank floor(c n'/2^k).  So a weight's index is the number of boundary elements (the
// elements at those ranks, c = 1 .. 2^k - 1) whose pair is not above its own - no sort needed once the boundary
// elements are known.  They are found in two levels: a histogram of the inliers over kSelBins equal-width value
// bins between the two outlier thresholds (the bin is a monotone function of the value, so bins partition the
// sorted order), then, for the few bins that hold a boundary rank, their members are gathered and the member with
// the wanted number of smaller pairs is picked by counting.  One CTA per unit; every warp owns one contiguous
// 1/32 of the unit in all passes (a lane reads four consecutive weights at a time), so outlier lists come out in
// ascending offsets from per-warp counts alone.  Cluster sums are plain fp64 additions in a fixed order (every cell
// of a shared-memory table has one writing thread, the columns are then added in a fixed tree), so the output is
// deterministic.
//
// The fp64 outlier test is taken only where it can matter: a weight whose bin is neither the first nor the last
// lies at least half a bin (3e-5 of the threshold distance) inside the thresholds, far more than the rounding of
// the bin's fp32 arithmetic (about 1e-6 bins while |mean| < 10 threshold distances; otherwise every weight is
// tested), so it is an inlier.

constexpr int kSelBins = 16384;
constexpr int kSelMaxSeg = 1024;           // members of one boundary bin the counting selection accepts
constexpr int kSelGroups = 4;              // groups of 128 consecutive weights (four per lane) a warp classifies per step
constexpr int kSelStep = kSelGroups * 128; // weights of one step of one warp
constexpr int kAccCells = 16384;           // fp64 cells of the cluster-sum table: 2^k clusters x columns

struct SelShared {
  double red[kQWarps];
  unsigned long long bnd_pair[64];         // (key << 32 | offset) of the element at the boundary rank
  uint32_t warp_out[kQWarps];              // outliers of each warp's part -> their exclusive prefix
  uint32_t scan[kQWarps];
  uint32_t n_out, fallback;
  uint32_t bounds[65];
  uint32_t bnd_bin[64], bnd_rho[64], seg_start[64], seg_len[64], seg_fill[64];
  float cents[64];
  uint8_t binfo[kSelBins];                 // boundaries in lower bins (6 bits) | 0x80 when the bin holds a boundary rank
  alignas(16) uint32_t stage[kQWarps][kSelStep / 4];   // a step's indexes of one warp, a byte each, in element order
  union {
    uint32_t hist[kSelBins];               // first the inlier histogram, in place its exclusive prefix
    double acc[kAccCells];                 // later the cluster sums
  } u;
};
static_assert(offsetof(SelShared, stage) % 16 == 0 && offsetof(SelShared, u) % 8 == 0 && offsetof(SelShared, bnd_pair) % 8 == 0,
              "vector and 64-bit accesses into the shared layout");
static_assert(sizeof(SelShared) <= 227 * 1024, "shared memory of one CTA");

// Nearest integer of x inv_w + off, clamped to the bins: monotone in x, and no conversion instructions (a float in
// [0, 2^23) plus 2^23 has its integer value in the low mantissa bits).  NaN goes to bin 0.
__device__ __forceinline__ int value_bin(float x, float inv_w, float off) {
  const float t = fminf(fmaxf(fmaf(x, inv_w, off), 0.f), static_cast<float>(kSelBins - 1));
  return __float_as_int(t + 8388608.0f) - 0x4B000000;
}
__device__ __forceinline__ bool edge_bin(int b) { return static_cast<unsigned>(b - 1) >= static_cast<unsigned>(kSelBins - 2); }

struct SelUnit {                           // what every pass needs to classify a weight
  double mu, inv2var, c0;
  float inv_w, off;
  bool test_all;                           // the bins' arithmetic is too coarse to clear weights of inner bins
  // bins of the lane's four weights; bit j of the result: weight j is an outlier
  __device__ __forceinline__ uint32_t classify(const float4& x, int (&b)[4]) const {
    b[0] = value_bin(x.x, inv_w, off); b[1] = value_bin(x.y, inv_w, off);
    b[2] = value_bin(x.z, inv_w, off); b[3] = value_bin(x.w, inv_w, off);
    uint32_t om = 0;
    if (test_all || edge_bin(b[0]) || edge_bin(b[1]) || edge_bin(b[2]) || edge_bin(b[3])) {
      const float v[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if ((test_all || edge_bin(b[j])) && is_outlier(v[j], mu, inv2var, c0)) om |= 1u << j;
    }
    return om;
  }
};

__device__ __forceinline__ float4 load4(const float* w, uint32_t i, uint32_t n) {
  return i < n ? *reinterpret_cast<const float4*>(w + i) : make_float4(0.f, 0.f, 0.f, 0.f);
}

template <int BITS>      // the index width is a compile-time constant: the packing and the table addressing unroll to immediates
__global__ void __launch_bounds__(kQThreads, 1)
quantize_select_kernel(const float* w_all, uint32_t n, uint32_t* codes_all, float* cent_all, uint32_t* ooff_all,
                       float* oval_all, uint32_t max_out, uint32_t* n_out_all, uint8_t* ws_all, size_t ws_per_unit,
                       uint8_t* marks) {
  extern __shared__ __align__(16) uint8_t q_smem[];
  SelShared& sm = *reinterpret_cast<SelShared*>(q_smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t unit = blockIdx.x;
  constexpr uint32_t bits = BITS, K = 1u << BITS;
  const float* w = w_all + static_cast<size_t>(unit) * n;
  uint32_t* codes = codes_all + static_cast<size_t>(unit) * (static_cast<size_t>(n) * bits / 32);
  float* cent = cent_all + static_cast<size_t>(unit) * K;
  uint32_t* ooff = ooff_all + static_cast<size_t>(unit) * max_out;
  float* oval = oval_all + static_cast<size_t>(unit) * max_out;
  unsigned long long* cand = reinterpret_cast<unsigned long long*>(ws_all + static_cast<size_t>(unit) * ws_per_unit);
  const uint32_t lt_mask = (1u << lane) - 1u;

  // ---- 1. Gaussian fit (shared with the sorting kernel, so both take the same outlier decisions)
  double mu, var;
  fit_gaussian(w, n, sm.red, tid, mu, var);
  SelUnit un;
  un.mu = mu;
  un.c0 = -0.5 * log(2.0 * 3.14159265358979323846 * var);
  un.inv2var = 1.0 / (2.0 * var);
  // inliers satisfy (x - mu)^2 <= 2 var (c0 + 4): the bins span that interval, values outside are clamped
  const double radius = sqrt(2.0 * var * (un.c0 + 4.0));
  un.inv_w = static_cast<float>(static_cast<double>(kSelBins - 1) / (2.0 * radius));
  un.off = -static_cast<float>(mu - radius) * un.inv_w;
  un.test_all = !(fabs(mu) < 10.0 * radius);
  if (!(var > 0.0) || !(radius > 0.0) || !(un.inv_w > 0.f) || !(un.inv_w < 3.0e38f) || !(fabsf(un.off) < 3.0e38f)) {
    if (tid == 0) marks[unit] = 1;                                   // every thread sees the same values: all leave
    return;
  }

  // the warp's part: whole steps
  const uint32_t part = (((n + kQWarps - 1u) / kQWarps + kSelStep - 1u) / kSelStep) * kSelStep;
  const uint32_t base = static_cast<uint32_t>(warp) * part + 4u * lane;     // the lane's first weight

  // ---- 2. outliers counted per warp, inliers into the histogram
  for (int i = tid; i < kSelBins; i += kQThreads) sm.u.hist[i] = 0u;
  if (tid < 64) { sm.bnd_pair[tid] = ~0ull; sm.seg_fill[tid] = 0u; sm.seg_len[tid] = 0u; sm.seg_start[tid] = 0u; }
  __syncthreads();
  uint32_t my_out = 0;
  for (uint32_t e0 = 0; e0 < part; e0 += kSelStep) {
    float4 x[kSelGroups];
#pragma unroll
    for (int u = 0; u < kSelGroups; ++u) x[u] = load4(w, base + e0 + u * 128u, n);
#pragma unroll
    for (int u = 0; u < kSelGroups; ++u) {
      const bool valid = base + e0 + u * 128u < n;
      int b[4];
      const uint32_t om = valid ? un.classify(x[u], b) : 0xfu;
      if (__any_sync(0xffffffffu, valid && om != 0u)) my_out += __reduce_add_sync(0xffffffffu, valid ? __popc(om) : 0u);
      if (valid) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (!((om >> j) & 1u)) atomicAdd(&sm.u.hist[b[j]], 1u);
      }
    }
  }
  if (lane == 0) sm.warp_out[warp] = my_out;
  __syncthreads();
  if (warp == 0) {
    const uint32_t mine = sm.warp_out[lane];
    uint32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
    sm.warp_out[lane] = inc - mine;
    if (lane == 31) sm.n_out = inc;
  }
  // exclusive prefix of the histogram, in place: thread t owns bins 16 t .. 16 t + 15
  {
    uint32_t c[16], tot = 0;
#pragma unroll
    for (int e = 0; e < 16; ++e) { c[e] = sm.u.hist[16 * tid + e]; tot += c[e]; }
    uint32_t inc = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
    if (lane == 31) sm.scan[warp] = inc;
    __syncthreads();
    uint32_t before = inc - tot;
    for (int ww = 0; ww < warp; ++ww) before += sm.scan[ww];
#pragma unroll
    for (int e = 0; e < 16; ++e) { sm.u.hist[16 * tid + e] = before; before += c[e]; }
  }
  __syncthreads();
  const uint32_t n_out = sm.n_out, n_in = n - n_out;

  // ---- 3. the boundary ranks: their bin, their rank inside it, the bin's population
  if (tid <= static_cast<int>(K)) {
    const uint32_t r = static_cast<uint32_t>(static_cast<uint64_t>(tid) * n_in / K);
    sm.bounds[tid] = r;
    if (tid >= 1 && tid < static_cast<int>(K)) {
      int lo = 0, hi = kSelBins - 1;                                  // the last bin whose prefix is <= r holds rank r
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (sm.u.hist[mid] <= r) lo = mid; else hi = mid - 1;
      }
      sm.bnd_bin[tid] = static_cast<uint32_t>(lo);
      sm.bnd_rho[tid] = r - sm.u.hist[lo];
      sm.seg_len[tid] = (lo + 1 < kSelBins ? sm.u.hist[lo + 1] : n_in) - sm.u.hist[lo];
    }
  }
  __syncthreads();
  if (tid == 0) {
    uint32_t start = 0, longest = 0;
    for (uint32_t c = 1; c < K; ++c) {
      if (c == 1 || sm.bnd_bin[c] != sm.bnd_bin[c - 1]) {             // the first boundary of a bin owns its member list
        sm.seg_start[c] = start;
        start += sm.seg_len[c];
        longest = longest > sm.seg_len[c] ? longest : sm.seg_len[c];
      } else {
        sm.seg_start[c] = sm.seg_start[c - 1];
      }
    }
    sm.fallback = longest > static_cast<uint32_t>(kSelMaxSeg) ? 1u : 0u;
  }
  __syncthreads();
  if (sm.fallback) {
    if (tid == 0) marks[unit] = 1;
    return;
  }
  for (int b = tid; b < kSelBins; b += kQThreads) {
    uint32_t below = 0;                                              // boundaries 1 .. below sit in lower bins (their bins ascend)
    for (uint32_t step = K >> 1; step > 0; step >>= 1)
      if (below + step < K && sm.bnd_bin[below + step] < static_cast<uint32_t>(b)) below += step;
    const uint32_t here = (below + 1 < K && sm.bnd_bin[below + 1] == static_cast<uint32_t>(b)) ? 0x80u : 0u;
    sm.binfo[b] = static_cast<uint8_t>(below | here);
  }
  __syncthreads();

  // ---- 4. the members of the boundary bins, as (key, offset) pairs, in any order
  for (uint32_t e0 = 0; e0 < part; e0 += kSelStep) {
    float4 x[kSelGroups];
#pragma unroll
    for (int u = 0; u < kSelGroups; ++u) x[u] = load4(w, base + e0 + u * 128u, n);
#pragma unroll
    for (int u = 0; u < kSelGroups; ++u) {
      const uint32_t i0 = base + e0 + u * 128u;
      if (i0 >= n) continue;
      const float v[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int b = value_bin(v[j], un.inv_w, un.off);
        const uint32_t info = sm.binfo[b];
        if (info & 0x80u) {
          if ((un.test_all || edge_bin(b)) && is_outlier(v[j], un.mu, un.inv2var, un.c0)) continue;
          const uint32_t owner = (info & 63u) + 1u;
          const uint32_t pos = atomicAdd(&sm.seg_fill[owner], 1u);
          cand[sm.seg_start[owner] + pos] = (static_cast<unsigned long long>(sort_key(v[j])) << 32) | (i0 + j);
        }
      }
    }
  }
  __syncthreads();
  // the member with exactly rho smaller members is the boundary element (all pairs are distinct)
  for (uint32_t c = 1 + warp; c < K; c += kQWarps) {
    const uint32_t m = sm.seg_len[c], rho = sm.bnd_rho[c];
    const unsigned long long* seg = cand + sm.seg_start[c];
    for (uint32_t j = lane; j < m; j += 32) {
      const unsigned long long pj = seg[j];
      uint32_t smaller = 0;
      for (uint32_t t = 0; t < m; ++t) smaller += seg[t] < pj ? 1u : 0u;
      if (smaller == rho) sm.bnd_pair[c] = pj;
    }
  }
  for (int i = tid; i < kAccCells; i += kQThreads) sm.u.acc[i] = 0.0;
  __syncthreads();

  // ---- 5. indexes, outlier lists, cluster sums, the packed stream
  // The cluster-sum table has one column per `share` neighbouring lanes (1, 2 or 4: 2^k columns of 1024 cells do not
  // fit above 16 clusters); the lanes of such a group add one after the other, so every cell sees a fixed order of
  // additions.
  constexpr uint32_t acc_cols = (kAccCells >> BITS) < kQThreads ? (kAccCells >> BITS) : kQThreads;
  constexpr uint32_t share = kQThreads / acc_cols;
  const uint32_t col = static_cast<uint32_t>(tid) / share;
  uint32_t run_out = sm.warp_out[warp];
  for (uint32_t e0 = 0; e0 < part; e0 += kSelStep) {
    float4 x[kSelGroups];
#pragma unroll
    for (int u = 0; u < kSelGroups; ++u) x[u] = load4(w, base + e0 + u * 128u, n);
#pragma unroll
    for (int u = 0; u < kSelGroups; ++u) {
      const uint32_t i0 = base + e0 + u * 128u;
      const bool valid = i0 < n;
      const float v[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
      int b[4];
      const uint32_t om = valid ? un.classify(x[u], b) : 0u;
      uint32_t cw = 0xffffffffu;                                     // the four indexes, a byte each; 255 = nothing to add
      if (valid) {
        cw = 0u;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint32_t code = 255u;
          if (!((om >> j) & 1u)) {
            const uint32_t info = sm.binfo[b[j]];
            code = info & 63u;
            if (info & 0x80u) {
              const unsigned long long pair = (static_cast<unsigned long long>(sort_key(v[j])) << 32) | (i0 + j);
              while (code + 1u < K && sm.bnd_pair[code + 1u] <= pair) ++code;
            }
          }
          cw |= code << (8 * j);
        }
      }
      if (__any_sync(0xffffffffu, om != 0u)) {                       // outliers in this group of 128: in ascending offsets
        uint32_t before = 0, total = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t bj = __ballot_sync(0xffffffffu, (om >> j) & 1u);
          before += __popc(bj & lt_mask);
          total += __popc(bj);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if ((om >> j) & 1u) {
            const uint32_t dst = run_out + before + __popc(om & ((1u << j) - 1u));
            if (dst < max_out) { ooff[dst] = i0 + j; oval[dst] = v[j]; }
          }
        }
        run_out += total;
      }
      // cluster sums: the lanes that share a column add in turns
#pragma unroll
      for (uint32_t q = 0; q < share; ++q) {
        if ((lane & (share - 1u)) == q) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t code = (cw >> (8 * j)) & 255u;
            if (code != 255u) sm.u.acc[code * acc_cols + col] += static_cast<double>(v[j]);
          }
        }
        if (share > 1u) __syncwarp();
      }
      // an outlier's index is set in step 6: its bits stay zero here
      sm.stage[warp][u * 32 + lane] = cw & ~(((cw & 0x80808080u) >> 7) * 255u);
    }
    __syncwarp();
    // 32 consecutive indexes are exactly `bits` words: lane r packs the r-th 32 weights of the step
    if (lane < kSelStep / 32 && static_cast<uint32_t>(warp) * part + e0 + lane * 32u < n) {
      const uint4 a = *reinterpret_cast<const uint4*>(&sm.stage[warp][lane * 8]);
      const uint4 c = *reinterpret_cast<const uint4*>(&sm.stage[warp][lane * 8 + 4]);
      const uint32_t src[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
      unsigned long long window = 0;
      uint32_t fill = 0, out_w = ((static_cast<uint32_t>(warp) * part + e0) / 32u + lane) * bits;
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        const uint32_t code = (src[e >> 2] >> (8 * (e & 3))) & 255u;
        window |= static_cast<unsigned long long>(code) << fill;
        fill += bits;
        if (fill >= 32u) {
          codes[out_w++] = static_cast<uint32_t>(window);
          window >>= 32;
          fill -= 32u;
        }
      }
    }
    __syncwarp();
  }
  __syncthreads();
  // centroids: the columns of a cluster added in a fixed order
  for (uint32_t c = warp; c < K; c += kQWarps) {
    double acc = 0.0;
    for (uint32_t t = lane; t < acc_cols; t += 32) acc += sm.u.acc[c * acc_cols + t];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) {
      const uint32_t members = sm.bounds[c + 1] - sm.bounds[c];
      const float m = members > 0 ? static_cast<float>(acc / static_cast<double>(members)) : 0.f;
      sm.cents[c] = m;
      cent[c] = m;
    }
  }
  if (tid == 0) { n_out_all[unit] = n_out; marks[unit] = 0; }
  __syncthreads();

  // ---- 6. an outlier's slot gets the nearest centroid's index (its bits in the stream are still zero)
  if (n_out > 0) {
    const bool listed = n_out <= max_out;                             // else the lists were cut short: scan the unit again
    const uint32_t count = listed ? n_out : n;
    for (uint32_t j = tid; j < count; j += kQThreads) {
      uint32_t i = j;
      float x;
      if (listed) { i = ooff[j]; x = oval[j]; }
      else { x = w[j]; if (!is_outlier(x, un.mu, un.inv2var, un.c0)) continue; }
      uint32_t best = 0;
      double bd = fabs(static_cast<double>(x) - static_cast<double>(sm.cents[0]));
      for (uint32_t c = 1; c < K; ++c) {
        const double dd = fabs(static_cast<double>(x) - static_cast<double>(sm.cents[c]));
        if (dd < bd) { bd = dd; best = c; }
      }
      const uint64_t bit = static_cast<uint64_t>(i) * bits;
      const uint32_t sh = static_cast<uint32_t>(bit & 31u);
      atomicOr(&codes[bit >> 5], best << sh);
      if (sh + bits > 32u) atomicOr(&codes[(bit >> 5) + 1], best >> (32u - sh));
    }
  }
}

template <int BITS>
bool select_configure_one() {
  return cudaFuncSetAttribute(quantize_select_kernel<BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(sizeof(SelShared))) == cudaSuccess;
}
bool select_configure(int bits) {
  switch (bits) {
    case 2: return select_configure_one<2>();
    case 3: return select_configure_one<3>();
    case 4: return select_configure_one<4>();
    case 5: return select_configure_one<5>();
    default: return select_configure_one<6>();
  }
}
template <typename... Args>
void launch_select(int bits, uint32_t n_units, cudaStream_t cs, Args... args) {
  switch (bits) {
    case 2: quantize_select_kernel<2><<<n_units, kQThreads, sizeof(SelShared), cs>>>(args...); break;
    case 3: quantize_select_kernel<3><<<n_units, kQThreads, sizeof(SelShared), cs>>>(args...); break;
    case 4: quantize_select_kernel<4><<<n_units, kQThreads, sizeof(SelShared), cs>>>(args...); break;
    case 5: quantize_select_kernel<5><<<n_units, kQThreads, sizeof(SelShared), cs>>>(args...); break;
    default: quantize_select_kernel<6><<<n_units, kQThreads, sizeof(SelShared), cs>>>(args...); break;
  }
}

size_t ws_per_unit_bytes(uint32_t n) { return (17 * static_cast<size_t>(n) + 255) & ~static_cast<size_t>(255); }
size_t marks_bytes(uint32_t n_units) { return (static_cast<size_t>(n_units) + 255) & ~static_cast<size_t>(255); }

}  // namespace

extern "C" {

size_t sti_quantize_workspace_bytes(uint32_t n_units, uint32_t n_weights) {
  return static_cast<size_t>(n_units) * ws_per_unit_bytes(n_weights) + marks_bytes(n_units);
}

sti_status sti_quantize_units_by(int device, void* stream, const float* w_dev, uint32_t n_units, uint32_t n_weights, int bits,
                                 uint32_t* codes_dev, float* centroids_dev, uint32_t* outlier_off_dev, float* outlier_val_dev,
                                 uint32_t max_outliers, uint32_t* n_outliers_dev, void* workspace_dev, size_t workspace_bytes,
                                 int method, uint8_t* sorted_units_dev) {
  if (!w_dev || !codes_dev || !centroids_dev || !outlier_off_dev || !outlier_val_dev || !n_outliers_dev || !workspace_dev)
    return STI_ERR_ARG;
  if (method != STI_QUANTIZE_SELECT && method != STI_QUANTIZE_SORT) return STI_ERR_ARG;
  if (bits < 2 || bits > 6) return STI_ERR_BITS;
  if (n_units == 0 || n_units > 65535 || n_weights == 0 || n_weights % 32 != 0 || n_weights > (1u << 26) || max_outliers == 0)
    return STI_ERR_SHAPE;
  if (workspace_bytes < sti_quantize_workspace_bytes(n_units, n_weights)) return STI_ERR_SIZE;
  if ((reinterpret_cast<uintptr_t>(workspace_dev) & 15) != 0 || (reinterpret_cast<uintptr_t>(w_dev) & 15) != 0) return STI_ERR_ARG;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) {
    (void)cudaGetLastError();
    return STI_ERR_CUDA;
  }
  int prev = 0;
  if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(device) != cudaSuccess) return STI_ERR_CUDA;
  sti_status st = STI_OK;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace_dev);
  const size_t per_unit = ws_per_unit_bytes(n_weights);
  uint8_t* marks = ws + static_cast<size_t>(n_units) * per_unit;
  if (cudaFuncSetAttribute(quantize_units_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           static_cast<int>(sizeof(QuantShared))) != cudaSuccess ||
      !select_configure(bits))
    st = STI_ERR_CUDA;
  if (st == STI_OK) {
    if (method == STI_QUANTIZE_SELECT) {
      launch_select(bits, n_units, cs, w_dev, n_weights, codes_dev, centroids_dev, outlier_off_dev, outlier_val_dev,
                    max_outliers, n_outliers_dev, ws, per_unit, marks);
    } else if (cudaMemsetAsync(marks, 1, n_units, cs) != cudaSuccess) {
      st = STI_ERR_CUDA;
    }
  }
  if (st == STI_OK) {
    quantize_units_kernel<<<n_units, kQThreads, sizeof(QuantShared), cs>>>(
        w_dev, n_weights, bits, codes_dev, centroids_dev, outlier_off_dev, outlier_val_dev, max_outliers, n_outliers_dev,
        ws, per_unit, marks);
    if (cudaGetLastError() != cudaSuccess) st = STI_ERR_CUDA;
  }
  if (st == STI_OK && sorted_units_dev != nullptr &&
      cudaMemcpyAsync(sorted_units_dev, marks, n_units, cudaMemcpyDeviceToDevice, cs) != cudaSuccess)
    st = STI_ERR_CUDA;
  (void)cudaSetDevice(prev);
  return st;
}

sti_status sti_quantize_units(int device, void* stream, const float* w_dev, uint32_t n_units, uint32_t n_weights, int bits,
                              uint32_t* codes_dev, float* centroids_dev, uint32_t* outlier_off_dev, float* outlier_val_dev,
                              uint32_t max_outliers, uint32_t* n_outliers_dev, void* workspace_dev, size_t workspace_bytes) {
  return sti_quantize_units_by(device, stream, w_dev, n_units, n_weights, bits, codes_dev, centroids_dev, outlier_off_dev,
                               outlier_val_dev, max_outliers, n_outliers_dev, workspace_dev, workspace_bytes,
                               STI_QUANTIZE_SELECT, nullptr);
}

}  // extern "C"
