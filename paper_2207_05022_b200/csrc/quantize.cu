// Shard quantizer on the device (Section 6: Gaussian outlier-aware dictionary quantization).
//
// One CTA of 1024 threads per shard unit runs the paper's steps in order on the unit's flat fp32 array:
//   1. maximum-likelihood fit of one Gaussian (mean, 1/n variance; fp64 block reductions);
//   2. outliers = weights whose log-likelihood is below -4: their (offset, value) pairs are written in
//      ascending offset order by a stable compaction; the other weights become (sortable key, offset) pairs;
//   3. a least-significant-digit radix sort (4 passes of 8 bits, stable, so equal weights keep their
//      original order) of the pairs between two workspace buffers;
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

struct QuantShared {
  double red[kQWarps];
  uint32_t hist[256];
  uint32_t base[2][256];
  uint8_t wcount[kQWarps][256];      // per chunk: elements of digit d held by warp w
  uint16_t woff[kQWarps][256];       // per chunk: elements of digit d held by warps before w
  uint32_t wcnt_in[kQWarps], wcnt_out[kQWarps];
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
__device__ __forceinline__ bool is_outlier(float x, double mu, double var, double c0) {
  const double d = static_cast<double>(x) - mu;
  const double ll = c0 - d * d / (2.0 * var);        // NaN when the variance is zero: compares false
  return ll < -4.0;
}

__global__ void __launch_bounds__(kQThreads, 1)
quantize_units_kernel(const float* w_all, uint32_t n, int bits, uint32_t* codes_all, float* cent_all, uint32_t* ooff_all,
                      float* oval_all, uint32_t max_out, uint32_t* n_out_all, uint8_t* ws_all, size_t ws_per_unit) {
  __shared__ QuantShared sm;
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

  // ---- 1. Gaussian fit
  double s = 0.0;
  for (uint32_t i = tid; i < n; i += kQThreads) s += static_cast<double>(w[i]);
  const double mu = block_sum(s, sm, tid) / static_cast<double>(n);
  double q = 0.0;
  for (uint32_t i = tid; i < n; i += kQThreads) {
    const double d = static_cast<double>(w[i]) - mu;
    q += d * d;
  }
  const double var = block_sum(q, sm, tid) / static_cast<double>(n);
  const double c0 = -0.5 * log(2.0 * 3.14159265358979323846 * var);

  // ---- 2. outliers out (ascending offsets), the rest as (key, offset) pairs, both by stable compaction
  uint32_t n_in = 0, n_out = 0;
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (uint32_t start = 0; start < n; start += kQThreads) {
    const uint32_t i = start + tid;
    const bool valid = i < n;
    const float x = valid ? w[i] : 0.f;
    const bool out = valid && is_outlier(x, mu, var, c0);
    const bool in = valid && !out;
    const uint32_t m_in = __ballot_sync(0xffffffffu, in), m_out = __ballot_sync(0xffffffffu, out);
    if (lane == 0) { sm.wcnt_in[warp] = __popc(m_in); sm.wcnt_out[warp] = __popc(m_out); }
    __syncthreads();
    uint32_t pre_in = 0, pre_out = 0, tot_in = 0, tot_out = 0;
    for (int ww = 0; ww < kQWarps; ++ww) {
      const uint32_t a = sm.wcnt_in[ww], b = sm.wcnt_out[ww];
      if (ww < warp) { pre_in += a; pre_out += b; }
      tot_in += a; tot_out += b;
    }
    if (in) {
      const uint32_t dst = n_in + pre_in + __popc(m_in & lt_mask);
      key[0][dst] = sort_key(x);
      idx[0][dst] = i;
    }
    if (out) {
      const uint32_t dst = n_out + pre_out + __popc(m_out & lt_mask);
      if (dst < max_out) { ooff[dst] = i; oval[dst] = x; }
    }
    n_in += tot_in;
    n_out += tot_out;
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
    for (uint32_t i = tid; i < n_in; i += kQThreads) atomicAdd(&sm.hist[(ksrc[i] >> shift) & 255u], 1u);
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
    for (uint32_t start = 0; start < n_in; start += kQThreads) {
      const uint32_t i = start + tid;
      const bool valid = i < n_in;
      const uint32_t kk = valid ? ksrc[i] : 0u;
      const uint32_t ii = valid ? isrc[i] : 0u;
      const uint32_t d = (kk >> shift) & 255u;
      // lanes holding the same digit; lanes past the end get a value of their own
      const uint32_t peers = __match_any_sync(0xffffffffu, valid ? d : (256u + lane));
      const uint32_t rank_w = __popc(peers & lt_mask);
      reinterpret_cast<uint32_t*>(&sm.wcount[0][0])[tid] = 0u;
      reinterpret_cast<uint32_t*>(&sm.wcount[0][0])[tid + kQThreads] = 0u;
      __syncthreads();
      if (valid && rank_w == 0) sm.wcount[warp][d] = static_cast<uint8_t>(__popc(peers));
      __syncthreads();
      if (tid < 256) {
        uint32_t pre = 0;
        for (int ww = 0; ww < kQWarps; ++ww) {
          sm.woff[ww][tid] = static_cast<uint16_t>(pre);
          pre += sm.wcount[ww][tid];
        }
        sm.base[bsel ^ 1][tid] = sm.base[bsel][tid] + pre;
      }
      __syncthreads();
      if (valid) {
        const uint32_t dst = sm.base[bsel][d] + sm.woff[warp][d] + rank_w;
        kdst[dst] = kk;
        idst[dst] = ii;
      }
      bsel ^= 1;
      // the next chunk's zeroing of wcount is ordered after these reads by its own barrier below the zeroing
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
  for (uint32_t r = tid; r < n_in; r += kQThreads) {
    uint32_t c = static_cast<uint32_t>(static_cast<uint64_t>(r) * K / n_in);
    while (c + 1 < K && sm.bounds[c + 1] <= r) ++c;
    while (c > 0 && sm.bounds[c] > r) --c;
    codes8[is[r]] = static_cast<uint8_t>(c);
  }
  if (n_out > 0) {
    for (uint32_t i = tid; i < n; i += kQThreads) {
      const float x = w[i];
      if (!is_outlier(x, mu, var, c0)) continue;
      uint32_t best = 0;
      double bd = fabs(static_cast<double>(x) - static_cast<double>(sm.cents[0]));
      for (uint32_t c = 1; c < K; ++c) {
        const double dd = fabs(static_cast<double>(x) - static_cast<double>(sm.cents[c]));
        if (dd < bd) { bd = dd; best = c; }
      }
      codes8[i] = static_cast<uint8_t>(best);
    }
  }
  __syncthreads();

  // ---- 6. the index stream: word j holds stream bits [32 j, 32 j + 32)
  const uint32_t n_words = static_cast<uint32_t>(static_cast<uint64_t>(n) * bits / 32);
  for (uint32_t j = tid; j < n_words; j += kQThreads) {
    const uint32_t bit0 = 32u * j;
    uint32_t i = bit0 / bits;
    const uint32_t used = bit0 - i * bits;             // bits of index i that belong to the previous word
    uint32_t word = static_cast<uint32_t>(codes8[i]) >> used;
    uint32_t pos = bits - used;
    ++i;
    while (pos < 32u) {
      word |= static_cast<uint32_t>(codes8[i]) << pos;
      pos += bits;
      ++i;
    }
    codes[j] = word;
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
  quantize_units_kernel<<<n_units, kQThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      w_dev, n_weights, bits, codes_dev, centroids_dev, outlier_off_dev, outlier_val_dev, max_outliers, n_outliers_dev,
      static_cast<uint8_t*>(workspace_dev), ws_per_unit_bytes(n_weights));
  return cudaGetLastError() == cudaSuccess ? STI_OK : STI_ERR_CUDA;
}

}  // extern "C"
