// Shard quantizer on the device (Section 6: Gaussian outlier-aware dictionary quantization).
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

__device__ __forceinline__ double block_sum(double v, QuantShared& sm, int tid) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((tid & 31) == 0) sm.red[tid >> 5] = v;
  __syncthreads();
  double t = 0.0;
  for (int w = 0; w < kQWarps; ++w) t += sm.red[w];
  __syncthreads();
  return t;
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
                      float* oval_all, uint32_t max_out, uint32_t* n_out_all, uint8_t* ws_all, size_t ws_per_unit) {
  extern __shared__ __align__(16) uint8_t q_smem[];
  QuantShared& sm = *reinterpret_cast<QuantShared*>(q_smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t unit = blockIdx.x;
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

  // ---- 1. Gaussian fit (eight independent loads in flight per thread: a single CTA has little else to hide latency)
  double s = 0.0;
  for (uint32_t i0 = tid; i0 < n; i0 += 8 * kQThreads) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) { const uint32_t i = i0 + u * kQThreads; v[u] = i < n ? w[i] : 0.f; }
#pragma unroll
    for (int u = 0; u < 8; ++u) s += static_cast<double>(v[u]);
  }
  const double mu = block_sum(s, sm, tid) / static_cast<double>(n);
  double q = 0.0;
  for (uint32_t i0 = tid; i0 < n; i0 += 8 * kQThreads) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) { const uint32_t i = i0 + u * kQThreads; v[u] = i < n ? w[i] : 0.f; }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const double d = static_cast<double>(v[u]) - mu;
      if (i0 + u * kQThreads < n) q += d * d;
    }
  }
  const double var = block_sum(q, sm, tid) / static_cast<double>(n);
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

size_t ws_per_unit_bytes(uint32_t n) { return (17 * static_cast<size_t>(n) + 255) & ~static_cast<size_t>(255); }

}  // namespace

extern "C" {

size_t sti_quantize_workspace_bytes(uint32_t n_units, uint32_t n_weights) {
  return static_cast<size_t>(n_units) * ws_per_unit_bytes(n_weights);
}

sti_status sti_quantize_units(int device, void* stream, const float* w_dev, uint32_t n_units, uint32_t n_weights, int bits,
                              uint32_t* codes_dev, float* centroids_dev, uint32_t* outlier_off_dev, float* outlier_val_dev,
                              uint32_t max_outliers, uint32_t* n_outliers_dev, void* workspace_dev, size_t workspace_bytes) {
  if (!w_dev || !codes_dev || !centroids_dev || !outlier_off_dev || !outlier_val_dev || !n_outliers_dev || !workspace_dev)
    return STI_ERR_ARG;
  if (bits < 2 || bits > 6) return STI_ERR_BITS;
  if (n_units == 0 || n_units > 65535 || n_weights == 0 || n_weights % 32 != 0 || n_weights > (1u << 26) || max_outliers == 0)
    return STI_ERR_SHAPE;
  if (workspace_bytes < sti_quantize_workspace_bytes(n_units, n_weights)) return STI_ERR_SIZE;
  if ((reinterpret_cast<uintptr_t>(workspace_dev) & 15) != 0) return STI_ERR_ARG;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) {
    (void)cudaGetLastError();
    return STI_ERR_CUDA;
  }
  if (cudaSetDevice(device) != cudaSuccess) return STI_ERR_CUDA;
  if (cudaFuncSetAttribute(quantize_units_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           static_cast<int>(sizeof(QuantShared))) != cudaSuccess)
    return STI_ERR_CUDA;
  quantize_units_kernel<<<n_units, kQThreads, sizeof(QuantShared), static_cast<cudaStream_t>(stream)>>>(
      w_dev, n_weights, bits, codes_dev, centroids_dev, outlier_off_dev, outlier_val_dev, max_outliers, n_outliers_dev,
      static_cast<uint8_t*>(workspace_dev), ws_per_unit_bytes(n_weights));
  return cudaGetLastError() == cudaSuccess ? STI_OK : STI_ERR_CUDA;
}

}  // extern "C"
