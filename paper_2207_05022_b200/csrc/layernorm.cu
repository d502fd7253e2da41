// Residual + bias + LayerNorm over the split-K partial sums of the O projection and of FFN2
// (Section 2.1; Section 6: biases and layernorm parameters stay in fp32).
// One warp per token row; the row lives in registers, mean and variance are two-pass.
#include <cuda_bf16.h>

#include "sti_device.cuh"
#include "sti_kernels.h"

namespace sti {
namespace {

constexpr int kMaxVec = 16;   // float4 per lane: hidden <= 16 * 128 = 2048

__global__ void __launch_bounds__(256)
layernorm_kernel(LnLaunch p) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= p.T) return;
  const int nvec = p.d / 128;
  const size_t row = static_cast<size_t>(warp) * p.d;
  float4 v[kMaxVec];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    if (i < nvec) {
      const int c = (i * 32 + lane) * 4;
      float4 a = __ldg(reinterpret_cast<const float4*>(p.bias + c));
      if (p.resid_bf16) {
        const uint2 r = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.resid) + row + c));
        a.x += __uint_as_float(r.x << 16); a.y += __uint_as_float(r.x & 0xffff0000u);
        a.z += __uint_as_float(r.y << 16); a.w += __uint_as_float(r.y & 0xffff0000u);
      } else {
        const float4 r = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(p.resid) + row + c));
        a.x += r.x; a.y += r.y; a.z += r.z; a.w += r.w;
      }
      for (int q = 0; q < p.n_partial; ++q) {
        const float4 s = __ldg(reinterpret_cast<const float4*>(p.partial + static_cast<size_t>(q) * p.T * p.d + row + c));
        a.x += s.x; a.y += s.y; a.z += s.z; a.w += s.w;
      }
      v[i] = a;
      sum += a.x + a.y + a.z + a.w;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float mean = sum / static_cast<float>(p.d);
  float sq = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    if (i < nvec) {
      const float dx = v[i].x - mean, dy = v[i].y - mean, dz = v[i].z - mean, dw = v[i].w - mean;
      sq += dx * dx + dy * dy + dz * dz + dw * dw;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  const float rstd = rsqrtf(sq / static_cast<float>(p.d) + p.eps);
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    if (i < nvec) {
      const int c = (i * 32 + lane) * 4;
      const float4 g = __ldg(reinterpret_cast<const float4*>(p.gamma + c));
      const float4 b = __ldg(reinterpret_cast<const float4*>(p.beta + c));
      float4 y;
      y.x = (v[i].x - mean) * rstd * g.x + b.x;
      y.y = (v[i].y - mean) * rstd * g.y + b.y;
      y.z = (v[i].z - mean) * rstd * g.z + b.z;
      y.w = (v[i].w - mean) * rstd * g.w + b.w;
      if (p.out_f32) *reinterpret_cast<float4*>(p.out_f32 + row + c) = y;
      if (p.out_bf16)
        *reinterpret_cast<uint2*>(p.out_bf16 + row + c) = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
    }
  }
}

}  // namespace

cudaError_t launch_layernorm(const LnLaunch& p, cudaStream_t s) {
  if (p.T <= 0) return cudaSuccess;
  if (p.d % 128 != 0 || p.d / 128 > kMaxVec) return cudaErrorInvalidValue;
  const int warps_per_block = 8;
  const int blocks = (p.T + warps_per_block - 1) / warps_per_block;
  layernorm_kernel<<<blocks, warps_per_block * 32, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace sti
