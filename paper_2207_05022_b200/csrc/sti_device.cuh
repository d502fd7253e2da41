// Device-side building blocks shared by the sm_100a kernels: k-bit index extraction,
// bf16 conversion, mbarrier and tcgen05 wrappers (inline PTX).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sti {

// ---------------------------------------------------------------------------------------
// k-bit index extraction.  `w` holds one quantum: 128 consecutive indexes of a row as
// 4*BITS little-endian words, index i at stream bits [i*BITS, i*BITS+BITS), LSB first.
// `i` must be a compile-time constant after unrolling so that w[] stays in registers.
// ---------------------------------------------------------------------------------------
template <int BITS>
__device__ __forceinline__ uint32_t extract_index(const uint32_t (&w)[4 * BITS], int i) {
  const int b = i * BITS;
  const int word = b >> 5;
  const int s = b & 31;
  uint32_t v = w[word] >> s;
  if (s + BITS > 32) v |= w[word + 1] << (32 - s);
  return v & ((1u << BITS) - 1u);
}

// Same extraction from the first BITS words of a quantum (32 indexes).
template <int BITS>
__device__ __forceinline__ uint32_t extract_index_words(const uint32_t (&w)[BITS], int i) {
  const int b = i * BITS;
  const int word = b >> 5;
  const int s = b & 31;
  uint32_t v = w[word] >> s;
  if (s + BITS > 32) v |= w[word + 1] << (32 - s);
  return v & ((1u << BITS) - 1u);
}

__device__ __forceinline__ uint16_t bf16_bits(float f) {
  return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// ---------------------------------------------------------------------------------------
// Profiling stamps (Section 5.2: the delays the planner works with are measured on the device in use).
// One record of kStampWords 64-bit words per kernel launch, every word 0xff..ff before the forward.  A slot that
// holds a minimum over the launch's CTAs stores the time, a slot that holds a maximum stores its complement, so
// both are one atomicMin.  One thread per CTA stamps; a null record switches stamping off.
// ---------------------------------------------------------------------------------------
constexpr int kStampWords = 8;
enum StampSlot : int {
  STAMP_FIRST_START = 0,   // min: the launch's first CTA starts
  STAMP_RELEASE = 1,       // min: first CTA past the wait for the preceding kernel
  STAMP_LAST_END = 2,      // max: the last CTA is done
  STAMP_DECODED = 3,       // max: weight tiles decoded (dequant-GEMM)
  STAMP_LAST_START = 4,    // max: the launch's last CTA starts
  STAMP_ACC = 5,           // max: accumulators complete (dequant-GEMM with the LayerNorm epilogue)
  STAMP_EXCHANGED = 6      // max: row statistics of all column tiles have arrived (same)
};
__device__ __forceinline__ void stamp_min(unsigned long long* rec, int slot) {
  if (rec != nullptr) atomicMin(rec + slot, static_cast<unsigned long long>(global_timer_ns()));
}
__device__ __forceinline__ void stamp_max(unsigned long long* rec, int slot) {
  if (rec != nullptr) atomicMin(rec + slot, ~static_cast<unsigned long long>(global_timer_ns()));
}

// ---------------------------------------------------------------------------------------
// mbarrier
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_inval(uint32_t bar) {
  asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// Bounded wait: gives up after about two seconds and returns false.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_timer_ns() - t0 > 2000000000ull) return false;
  }
}

// Same bound, but the waiting thread sleeps between polls so that it does not take issue slots from
// the warp that shares its scheduler (used by the roles that wait long: producer, epilogue).
__device__ __forceinline__ bool mbar_wait_bounded_relaxed(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      __nanosleep(64);
      if (mbar_try_wait(bar, parity)) return true;
    }
    if (global_timer_ns() - t0 > 2000000000ull) return false;
  }
}

// Programmatic dependent launch: a kernel launched with the attribute may start while its predecessor
// on the stream still runs.  `pdl_wait` blocks until the predecessor has completed and its writes are
// visible - everything before it may only touch data no kernel writes (weights, descriptors, parameters);
// `pdl_launch_dependents` lets the successor start launching.  Both are no-ops for ordinary launches.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Make generic-proxy shared-memory writes visible to the async proxy (tensor core reads).
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------------------------------
// tcgen05: tensor memory and the 5th-generation MMA
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t n_cols) {   // whole warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(n_cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {                                // whole warp
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t n_cols) {    // whole warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(n_cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// One lane of a converged warp.  Issuing tcgen05.mma under this predicate from an otherwise converged
// warp keeps the descriptor arithmetic in the uniform datapath (about 25 % faster issue than a loop that
// only lane 0 runs).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}

// Shared-memory matrix descriptor, K-major, no swizzle: 8-row x 16-byte core matrices;
// `lbo` = byte distance between core matrices adjacent in K, `sbo` = between 8-row groups.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>((sbo >> 4) & 0x3FFFu) << 32;
  d |= static_cast<uint64_t>(1) << 46;   // descriptor version for sm_100
  return d;                              // base offset 0, layout type 0 (no swizzle)
}

// Instruction descriptor for kind::f16: bf16 x bf16 -> fp32, both operands K-major, M = 128.
__device__ __forceinline__ uint32_t umma_idesc_bf16_m128(uint32_t n) {
  return (1u << 4)            // D format fp32
         | (1u << 7)          // A format bf16
         | (1u << 10)         // B format bf16
         | ((n >> 3) << 17)   // N
         | ((128u >> 4) << 24);  // M
}

// D[tmem] (+)= A[smem] * B[smem]^T, issued by one thread.
__device__ __forceinline__ void umma_bf16_ss(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Four consecutive K = 16 steps of one 64-column box in a single instruction group: the A descriptor
// advances by `a_step`, the B descriptor by `b_step` (both in 16-byte units) per step; only the first
// step may overwrite the accumulator.  One predicate set-up for the four instructions.
__device__ __forceinline__ void umma_bf16_ss_x4(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t a_step,
                                                uint32_t b_step, uint32_t idesc, uint32_t accumulate_first) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 a1, a2, a3, b1, b2, b3, as, bs;\n\t"
      "setp.ne.b32 p0, %6, 0;\n\t"
      "setp.eq.b32 p1, 0, 0;\n\t"
      "cvt.u64.u32 as, %3;\n\t"
      "cvt.u64.u32 bs, %4;\n\t"
      "add.u64 a1, %1, as;\n\tadd.u64 a2, a1, as;\n\tadd.u64 a3, a2, as;\n\t"
      "add.u64 b1, %2, bs;\n\tadd.u64 b2, b1, bs;\n\tadd.u64 b3, b2, bs;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %5, p0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a1, b1, %5, p1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a2, b2, %5, p1;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a3, b3, %5, p1;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(a_step), "r"(b_step), "r"(idesc), "r"(accumulate_first)
      : "memory");
}

// Arrive on an mbarrier once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 16 consecutive fp32 columns: thread i of the warp gets TMEM lane (base lane + i).
__device__ __forceinline__ void tmem_ld_32x32b_x16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

// Same, 8 consecutive columns.
__device__ __forceinline__ void tmem_ld_32x32b_x8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
      : "r"(taddr)
      : "memory");
}

// Same, 32 consecutive columns.
__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}

}  // namespace sti
