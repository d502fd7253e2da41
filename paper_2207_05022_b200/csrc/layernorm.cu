// Residual + bias + LayerNorm over the split-K partial sums of the O projection and of FFN2
// (Section 2.1; Section 6: biases and layernorm parameters stay in fp32).
// One CTA per token row, one float4 per thread (hidden / 4 threads): every load of a row is in
// flight at once; mean and variance are two-pass over registers with a block reduction.
#include <algorithm>

#include <cuda_bf16.h>

#include "sti_device.cuh"
#include "sti_kernels.h"

namespace sti {
namespace {

__device__ __forceinline__ float block_sum(float v, float* red, int tid, int n_warps) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((tid & 31) == 0) red[tid >> 5] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll 1
  for (int w = 0; w < n_warps; ++w) t += red[w];
  __syncthreads();
  return t;
}

__global__ void __launch_bounds__(512)
layernorm_kernel(LnLaunch p) {
  __shared__ float red[16];
  const int tid = threadIdx.x;
  const int n_warps = blockDim.x >> 5;
  const size_t row = static_cast<size_t>(blockIdx.x) * p.d;
  const int c = tid * 4;
  pdl_launch_dependents();
  if (tid == 0) { stamp_min(p.stamps, STAMP_FIRST_START); stamp_max(p.stamps, STAMP_LAST_START); }
  float4 a = __ldg(reinterpret_cast<const float4*>(p.bias + c));      // parameters: not written by any kernel
  const float4 g = __ldg(reinterpret_cast<const float4*>(p.gamma + c));
  const float4 b = __ldg(reinterpret_cast<const float4*>(p.beta + c));
  pdl_wait();                                                          // residual and partial sums are
  if (tid == 0) stamp_min(p.stamps, STAMP_RELEASE);                    // the preceding kernels' output
  if (p.resid_bf16) {
    const uint2 r = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.resid) + row + c));
    a.x += __uint_as_float(r.x << 16); a.y += __uint_as_float(r.x & 0xffff0000u);
    a.z += __uint_as_float(r.y << 16); a.w += __uint_as_float(r.y & 0xffff0000u);
  } else {
    const float4 r = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(p.resid) + row + c));
    a.x += r.x; a.y += r.y; a.z += r.z; a.w += r.w;
  }
  const size_t pstride = static_cast<size_t>(p.T) * p.d;
  int q = 0;
#pragma unroll 1
  for (; q + 4 <= p.n_partial; q += 4) {          // four independent loads at a time
    const float4 s0 = __ldg(reinterpret_cast<const float4*>(p.partial + (q + 0) * pstride + row + c));
    const float4 s1 = __ldg(reinterpret_cast<const float4*>(p.partial + (q + 1) * pstride + row + c));
    const float4 s2 = __ldg(reinterpret_cast<const float4*>(p.partial + (q + 2) * pstride + row + c));
    const float4 s3 = __ldg(reinterpret_cast<const float4*>(p.partial + (q + 3) * pstride + row + c));
    a.x += (s0.x + s1.x) + (s2.x + s3.x); a.y += (s0.y + s1.y) + (s2.y + s3.y);
    a.z += (s0.z + s1.z) + (s2.z + s3.z); a.w += (s0.w + s1.w) + (s2.w + s3.w);
  }
#pragma unroll 1
  for (; q < p.n_partial; ++q) {
    const float4 s = __ldg(reinterpret_cast<const float4*>(p.partial + q * pstride + row + c));
    a.x += s.x; a.y += s.y; a.z += s.z; a.w += s.w;
  }
  const float mean = block_sum(a.x + a.y + a.z + a.w, red, tid, n_warps) / static_cast<float>(p.d);
  const float dx = a.x - mean, dy = a.y - mean, dz = a.z - mean, dw = a.w - mean;
  const float var = block_sum(dx * dx + dy * dy + dz * dz + dw * dw, red, tid, n_warps) / static_cast<float>(p.d);
  const float rstd = rsqrtf(var + p.eps);
  float4 y;
  y.x = dx * rstd * g.x + b.x; y.y = dy * rstd * g.y + b.y;
  y.z = dz * rstd * g.z + b.z; y.w = dw * rstd * g.w + b.w;
  if (p.out_f32) *reinterpret_cast<float4*>(p.out_f32 + row + c) = y;
  if (p.out_bf16)
    *reinterpret_cast<uint2*>(p.out_bf16 + row + c) = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
  if (p.stamps != nullptr) {
    __syncthreads();
    if (tid == 0) stamp_max(p.stamps, STAMP_LAST_END);
  }
}

// Few tokens: the same arithmetic with several rows per CTA and several float4 per thread, so that the kernel
// sits on a handful of SMs only.  A GEMM CTA needs a whole SM; the CTAs of the GEMM that follows are launched while
// this kernel runs (programmatic dependent launch) and decode their weights meanwhile - but only on SMs that hold
// none of this kernel's CTAs.  A row is handled by `wpr` warps (named barrier = row slot, 0..15; the kernel uses
// no CTA-wide barrier), thread t of the row holds float4 number t, t + tpr, ... of it.
constexpr int kLnMaxV = 4;
template <int V>
__global__ void __launch_bounds__(1024)
layernorm_rows_kernel(LnLaunch p, int tpr, int rows_per_cta) {
  __shared__ float red_all[16][16];
  const int slot = threadIdx.x / tpr, tid = threadIdx.x % tpr;
  const int n_warps = tpr >> 5;
  const int r = blockIdx.x * rows_per_cta + slot;
  pdl_launch_dependents();
  if (threadIdx.x == 0) { stamp_min(p.stamps, STAMP_FIRST_START); stamp_max(p.stamps, STAMP_LAST_START); }
  if (slot >= rows_per_cta || r >= p.T) {      // whole warps: tpr is a multiple of 32
    pdl_wait();
    return;
  }
  float* red = red_all[slot];
  const size_t row = static_cast<size_t>(r) * p.d;
  float4 a[V];
#pragma unroll
  for (int v = 0; v < V; ++v) a[v] = __ldg(reinterpret_cast<const float4*>(p.bias + (tid + v * tpr) * 4));
  pdl_wait();
  if (tid == 0) stamp_min(p.stamps, STAMP_RELEASE);
  const size_t pstride = static_cast<size_t>(p.T) * p.d;
#pragma unroll
  for (int v = 0; v < V; ++v) {
    {
      const int c = (tid + v * tpr) * 4;
      if (p.resid_bf16) {
        const uint2 rr = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.resid) + row + c));
        a[v].x += __uint_as_float(rr.x << 16); a[v].y += __uint_as_float(rr.x & 0xffff0000u);
        a[v].z += __uint_as_float(rr.y << 16); a[v].w += __uint_as_float(rr.y & 0xffff0000u);
      } else {
        const float4 rr = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(p.resid) + row + c));
        a[v].x += rr.x; a[v].y += rr.y; a[v].z += rr.z; a[v].w += rr.w;
      }
      int q = 0;
#pragma unroll 1
      for (; q + 4 <= p.n_partial; q += 4) {          // same grouping of the partial sums as the one-row kernel
        const float4 s0 = __ldg(reinterpret_cast<const float4*>(p.partial + (q + 0) * pstride + row + c));
        const float4 s1 = __ldg(reinterpret_cast<const float4*>(p.partial + (q + 1) * pstride + row + c));
        const float4 s2 = __ldg(reinterpret_cast<const float4*>(p.partial + (q + 2) * pstride + row + c));
        const float4 s3 = __ldg(reinterpret_cast<const float4*>(p.partial + (q + 3) * pstride + row + c));
        a[v].x += (s0.x + s1.x) + (s2.x + s3.x); a[v].y += (s0.y + s1.y) + (s2.y + s3.y);
        a[v].z += (s0.z + s1.z) + (s2.z + s3.z); a[v].w += (s0.w + s1.w) + (s2.w + s3.w);
      }
#pragma unroll 1
      for (; q < p.n_partial; ++q) {
        const float4 s = __ldg(reinterpret_cast<const float4*>(p.partial + q * pstride + row + c));
        a[v].x += s.x; a[v].y += s.y; a[v].z += s.z; a[v].w += s.w;
      }
    }
  }
  auto row_sum = [&](float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((tid & 31) == 0) red[tid >> 5] = v;
    asm volatile("bar.sync %0, %1;" ::"r"(slot), "r"(tpr) : "memory");
    float t = 0.f;
#pragma unroll 1
    for (int w = 0; w < n_warps; ++w) t += red[w];
    asm volatile("bar.sync %0, %1;" ::"r"(slot), "r"(tpr) : "memory");
    return t;
  };
  float part = 0.f;
#pragma unroll
  for (int v = 0; v < V; ++v) part += a[v].x + a[v].y + a[v].z + a[v].w;
  const float mean = row_sum(part) / static_cast<float>(p.d);
  part = 0.f;
#pragma unroll
  for (int v = 0; v < V; ++v) {
    {
      a[v].x -= mean; a[v].y -= mean; a[v].z -= mean; a[v].w -= mean;
      part += a[v].x * a[v].x + a[v].y * a[v].y + a[v].z * a[v].z + a[v].w * a[v].w;
    }
  }
  const float var = row_sum(part) / static_cast<float>(p.d);
  const float rstd = rsqrtf(var + p.eps);
#pragma unroll
  for (int v = 0; v < V; ++v) {
    {
      const int c = (tid + v * tpr) * 4;
      const float4 g = __ldg(reinterpret_cast<const float4*>(p.gamma + c));
      const float4 b = __ldg(reinterpret_cast<const float4*>(p.beta + c));
      float4 y;
      y.x = a[v].x * rstd * g.x + b.x; y.y = a[v].y * rstd * g.y + b.y;
      y.z = a[v].z * rstd * g.z + b.z; y.w = a[v].w * rstd * g.w + b.w;
      if (p.out_f32) *reinterpret_cast<float4*>(p.out_f32 + row + c) = y;
      if (p.out_bf16)
        *reinterpret_cast<uint2*>(p.out_bf16 + row + c) = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
    }
  }
  if (p.stamps != nullptr) {
    asm volatile("bar.sync %0, %1;" ::"r"(slot), "r"(tpr) : "memory");
    if (tid == 0) stamp_max(p.stamps, STAMP_LAST_END);
  }
}

// Many tokens: a warp per row, lane l holding float4 number l, l + 32, ... of it (V = d / 128 of them).  Every load of
// a row - residual and one partial-sum plane at a time - is issued before the first use, 8 rows per CTA, and the two
// reductions are warp shuffles: no barrier, and enough bytes in flight per SM to keep the memory system busy.
constexpr int kLnWarpRows = 8;
constexpr int kLnWarpMinRows = 2048;
template <int V>
__global__ void __launch_bounds__(kLnWarpRows * 32)
layernorm_warp_kernel(LnLaunch p) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int r = blockIdx.x * kLnWarpRows + warp;
  pdl_launch_dependents();
  if (threadIdx.x == 0) { stamp_min(p.stamps, STAMP_FIRST_START); stamp_max(p.stamps, STAMP_LAST_START); }
  float4 a[V];
#pragma unroll
  for (int v = 0; v < V; ++v) a[v] = __ldg(reinterpret_cast<const float4*>(p.bias + (lane + v * 32) * 4));
  pdl_wait();
  if (threadIdx.x == 0) stamp_min(p.stamps, STAMP_RELEASE);
  if (r < p.T) {
    const size_t row = static_cast<size_t>(r) * p.d;
    if (p.resid_bf16) {
      uint2 rr[V];
#pragma unroll
      for (int v = 0; v < V; ++v)
        rr[v] = __ldg(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(p.resid) + row + (lane + v * 32) * 4));
#pragma unroll
      for (int v = 0; v < V; ++v) {
        a[v].x += __uint_as_float(rr[v].x << 16); a[v].y += __uint_as_float(rr[v].x & 0xffff0000u);
        a[v].z += __uint_as_float(rr[v].y << 16); a[v].w += __uint_as_float(rr[v].y & 0xffff0000u);
      }
    } else {
      float4 rr[V];
#pragma unroll
      for (int v = 0; v < V; ++v)
        rr[v] = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(p.resid) + row + (lane + v * 32) * 4));
#pragma unroll
      for (int v = 0; v < V; ++v) { a[v].x += rr[v].x; a[v].y += rr[v].y; a[v].z += rr[v].z; a[v].w += rr[v].w; }
    }
    const size_t pstride = static_cast<size_t>(p.T) * p.d;
#pragma unroll 1
    for (int q = 0; q < p.n_partial; ++q) {
      float4 s[V];
#pragma unroll
      for (int v = 0; v < V; ++v)
        s[v] = __ldg(reinterpret_cast<const float4*>(p.partial + q * pstride + row + (lane + v * 32) * 4));
#pragma unroll
      for (int v = 0; v < V; ++v) { a[v].x += s[v].x; a[v].y += s[v].y; a[v].z += s[v].z; a[v].w += s[v].w; }
    }
    float part = 0.f;
#pragma unroll
    for (int v = 0; v < V; ++v) part += (a[v].x + a[v].y) + (a[v].z + a[v].w);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    const float mean = part / static_cast<float>(p.d);
    part = 0.f;
#pragma unroll
    for (int v = 0; v < V; ++v) {
      a[v].x -= mean; a[v].y -= mean; a[v].z -= mean; a[v].w -= mean;
      part += (a[v].x * a[v].x + a[v].y * a[v].y) + (a[v].z * a[v].z + a[v].w * a[v].w);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    const float rstd = rsqrtf(part / static_cast<float>(p.d) + p.eps);
#pragma unroll
    for (int v = 0; v < V; ++v) {
      const int c = (lane + v * 32) * 4;
      const float4 g = __ldg(reinterpret_cast<const float4*>(p.gamma + c));
      const float4 b = __ldg(reinterpret_cast<const float4*>(p.beta + c));
      float4 y;
      y.x = a[v].x * rstd * g.x + b.x; y.y = a[v].y * rstd * g.y + b.y;
      y.z = a[v].z * rstd * g.z + b.z; y.w = a[v].w * rstd * g.w + b.w;
      if (p.out_f32) *reinterpret_cast<float4*>(p.out_f32 + row + c) = y;
      if (p.out_bf16)
        *reinterpret_cast<uint2*>(p.out_bf16 + row + c) = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
    }
  }
  if (p.stamps != nullptr) {
    __syncthreads();
    if (threadIdx.x == 0) stamp_max(p.stamps, STAMP_LAST_END);
  }
}

__global__ void cast_bf16_kernel(const float* __restrict__ in, uint16_t* __restrict__ out, size_t n4,
                                 unsigned long long* stamps) {
  const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  pdl_launch_dependents();
  if (threadIdx.x == 0) { stamp_min(stamps, STAMP_FIRST_START); stamp_max(stamps, STAMP_LAST_START); }
  pdl_wait();
  if (threadIdx.x == 0) stamp_min(stamps, STAMP_RELEASE);
  if (i < n4) {
    const float4 v = __ldg(reinterpret_cast<const float4*>(in) + i);
    reinterpret_cast<uint2*>(out)[i] = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
  }
  if (stamps != nullptr) {
    __syncthreads();
    if (threadIdx.x == 0) stamp_max(stamps, STAMP_LAST_END);
  }
}

}  // namespace

cudaError_t launch_layernorm(const LnLaunch& p, cudaStream_t s, bool pdl) {
  if (p.T <= 0) return cudaSuccess;
  if (p.d % 128 != 0 || p.d > 2048) return cudaErrorInvalidValue;     // d / 4 threads, whole warps
  if (p.ctas_hint > 0 && p.ctas_hint < p.T) {
    // the widest row group (fewest float4 per thread) whose CTA count stays within the hint
    const int n4 = p.d / 4;
    int tpr = 0;
    for (int cand = n4; cand >= 32; cand -= 32) {
      if (n4 % cand != 0 || (n4 / cand != 1 && n4 / cand != 2 && n4 / cand != 4)) continue;
      const int rows = std::min(16, 1024 / cand);
      tpr = cand;
      if ((p.T + rows - 1) / rows <= p.ctas_hint) break;
    }
    if (tpr > 0) {
      const int rows = std::min(16, 1024 / tpr);
      const dim3 grid((p.T + rows - 1) / rows), block(rows * tpr);
      switch (n4 / tpr) {
        case 1: return launch_kernel(layernorm_rows_kernel<1>, grid, block, 0, s, pdl, p, tpr, rows);
        case 2: return launch_kernel(layernorm_rows_kernel<2>, grid, block, 0, s, pdl, p, tpr, rows);
        case 4: return launch_kernel(layernorm_rows_kernel<4>, grid, block, 0, s, pdl, p, tpr, rows);
        default: break;
      }
    }
  }
  if (p.T >= kLnWarpMinRows && p.d <= 1024) {      // thousands of rows: a warp per row
    const dim3 grid((p.T + kLnWarpRows - 1) / kLnWarpRows), block(kLnWarpRows * 32);
    switch (p.d / 128) {
      case 1: return launch_kernel(layernorm_warp_kernel<1>, grid, block, 0, s, pdl, p);
      case 2: return launch_kernel(layernorm_warp_kernel<2>, grid, block, 0, s, pdl, p);
      case 3: return launch_kernel(layernorm_warp_kernel<3>, grid, block, 0, s, pdl, p);
      case 4: return launch_kernel(layernorm_warp_kernel<4>, grid, block, 0, s, pdl, p);
      case 5: return launch_kernel(layernorm_warp_kernel<5>, grid, block, 0, s, pdl, p);
      case 6: return launch_kernel(layernorm_warp_kernel<6>, grid, block, 0, s, pdl, p);
      case 7: return launch_kernel(layernorm_warp_kernel<7>, grid, block, 0, s, pdl, p);
      case 8: return launch_kernel(layernorm_warp_kernel<8>, grid, block, 0, s, pdl, p);
      default: break;
    }
  }
  return launch_kernel(layernorm_kernel, dim3(p.T), dim3(p.d / 4), 0, s, pdl, p);
}

cudaError_t launch_cast_bf16(const float* in, uint16_t* out, size_t n, cudaStream_t s, bool pdl, unsigned long long* stamps) {
  if (n == 0) return cudaSuccess;
  if (n % 4) return cudaErrorInvalidValue;
  const size_t n4 = n / 4;
  return launch_kernel(cast_bf16_kernel, dim3(static_cast<unsigned>((n4 + 255) / 256)), dim3(256), 0, s, pdl, in, out, n4, stamps);
}

}  // namespace sti
