// Stand-alone shard decompression (Section 4.2: every k-bit index is replaced by its centroid, and the
// outlier list then overwrites its positions), used for inspection and parity checks.  It reads the same
// re-tiled plane layout as the GEMM (one quantum of 128 indexes per lane) but extracts each index by its
// bit offset (extract_index); the GEMM's own plane-wise unpack is a separate routine (gemm_device.cuh),
// checked bit for bit through sti_gemm_probe.
#include <cuda_bf16.h>

#include "sti_device.cuh"
#include "sti_kernels.h"

namespace sti {
namespace {

template <int BITS>
__device__ __forceinline__ void decode_quantum(const DecodeLaunch& p, const float* tab, uint32_t task, uint32_t lane) {
  const bool narrow = p.kc < 128;
  const uint32_t chunks = narrow ? 1 : p.kc / 128;
  const uint32_t g = task / chunks, j = task % chunks;
  const uint4* src = p.codes + (static_cast<size_t>(g) * chunks + j) * (BITS * 32) + lane;
  uint32_t w[4 * BITS];
#pragma unroll
  for (int q = 0; q < BITS; ++q) {
    const uint4 v = __ldg(src + q * 32);
    w[4 * q + 0] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
  }
#pragma unroll
  for (int s = 0; s < 16; ++s) {
    uint32_t c[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) c[e] = extract_index<BITS>(w, 8 * s + e);
    const uint32_t row = narrow ? g * 64 + lane + 32 * (s >> 3) : g * 32 + lane;
    const uint32_t col = narrow ? (s & 7) * 8 : j * 128 + s * 8;
    const size_t at = static_cast<size_t>(row) * p.kc + col;
    if (p.codes_out) {
      const uint32_t lo = c[0] | (c[1] << 8) | (c[2] << 16) | (c[3] << 24);
      const uint32_t hi = c[4] | (c[5] << 8) | (c[6] << 16) | (c[7] << 24);
      *reinterpret_cast<uint2*>(p.codes_out + at) = make_uint2(lo, hi);
    }
    if (p.w) {
      *reinterpret_cast<float4*>(p.w + at) = make_float4(tab[c[0]], tab[c[1]], tab[c[2]], tab[c[3]]);
      *reinterpret_cast<float4*>(p.w + at + 4) = make_float4(tab[c[4]], tab[c[5]], tab[c[6]], tab[c[7]]);
    }
    if (p.wbf16) {
      *reinterpret_cast<uint4*>(p.wbf16 + at) =
          make_uint4(pack_bf16x2(tab[c[0]], tab[c[1]]), pack_bf16x2(tab[c[2]], tab[c[3]]),
                     pack_bf16x2(tab[c[4]], tab[c[5]]), pack_bf16x2(tab[c[6]], tab[c[7]]));
    }
  }
}

__global__ void __launch_bounds__(128)
decode_kernel(DecodeLaunch p, uint32_t n_tasks) {
  __shared__ float tab[64];
  if (threadIdx.x < 64) tab[threadIdx.x] = threadIdx.x < (1u << p.bits) ? p.table[threadIdx.x] : 0.f;
  __syncthreads();
  const uint32_t task = blockIdx.x * 4 + (threadIdx.x >> 5);
  const uint32_t lane = threadIdx.x & 31;
  if (task >= n_tasks) return;
  switch (p.bits) {
    case 2: decode_quantum<2>(p, tab, task, lane); break;
    case 3: decode_quantum<3>(p, tab, task, lane); break;
    case 4: decode_quantum<4>(p, tab, task, lane); break;
    case 5: decode_quantum<5>(p, tab, task, lane); break;
    case 6: decode_quantum<6>(p, tab, task, lane); break;
    default: break;
  }
}

__global__ void raw_copy_kernel(DecodeLaunch p, uint32_t n) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float v = reinterpret_cast<const float*>(p.codes)[i];
  if (p.w) p.w[i] = v;
  if (p.wbf16) p.wbf16[i] = bf16_bits(v);
}

__global__ void patch_outliers_kernel(DecodeLaunch p) {
  const uint32_t o = blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= p.n_out) return;
  const uint32_t local = p.out_off[o] - p.flat_base;
  if (local >= p.rows * p.kc) return;
  const float v = p.out_val[o];
  if (p.w) p.w[local] = v;
  if (p.wbf16) p.wbf16[local] = bf16_bits(v);
}

}  // namespace

cudaError_t launch_decode(const DecodeLaunch& p, cudaStream_t s) {
  if (p.bits == 32) {
    const uint32_t n = p.rows * p.kc;
    raw_copy_kernel<<<(n + 255) / 256, 256, 0, s>>>(p, n);
    return cudaGetLastError();
  }
  const uint32_t n_tasks = p.kc >= 128 ? (p.rows / 32) * (p.kc / 128) : p.rows / 64;
  decode_kernel<<<(n_tasks + 3) / 4, 128, 0, s>>>(p, n_tasks);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (p.n_out) {
    patch_outliers_kernel<<<(p.n_out + 127) / 128, 128, 0, s>>>(p);
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace sti
