// Device helpers shared by the expert-streaming kernels: mbarrier primitives with bounded waits,
// the bulk asynchronous global->shared copy (TMA, non-tensor form, one CTA's own shared memory) and the decoding
// of 16-byte groups of stored weights to float.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

namespace remoe {
namespace ring {

constexpr unsigned kSpinLimit = 1u << 20;      // polls of one bounded wait before it gives up
constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the phase did not complete within the spin limit.  A parity wait cannot
// tell "phase k done" from "phase k-2 done", so a waiter must never be a whole phase ahead of the
// barrier: every kernel here lets a stage be consumed by the same agent every time.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned limit = kSpinLimit) {
  for (unsigned it = 0; it < limit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// dst and src 16-byte aligned, bytes a multiple of 16; completion is counted on `bar`.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst)),
      "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
// Barrier over the 256 consumer threads (named barrier 1; the producer warp never joins it).
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// Same barrier, also ORing a flag: every thread learns whether any of them failed, so that they
// leave a loop containing barriers together.
__device__ __forceinline__ bool consumer_bar_any(bool flag) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, 1, 256, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out)
      : "r"((uint32_t)flag)
      : "memory");
  return out != 0;
}

// Elems<bytes per element>: sixteen stored bytes -> kVec floats.
template <int WB>
struct Elems;
template <>
struct Elems<4> {
  static constexpr int kVec = 4;
  __device__ static __forceinline__ void load(const char* p, float* f) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
};
template <>
struct Elems<2> {                                   // bfloat16: the upper half of a float
  static constexpr int kVec = 8;
  __device__ static __forceinline__ void load(const char* p, float* f) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
  }
};
// FP8 E4M3: a stored byte q stands for q * 2^-8 (the stack-wide power-of-two scale is applied to
// the dot products, not per element).  Decoding is cvt.e4m3x2 -> f16x2 -> f32; an integer-pipe bit
// construction and packed fp32 FMAs were measured and are no faster: with several issuing producer
// lanes the FP8 stream runs at the HBM rate, so the decode is not what bounds it.
template <>
struct Elems<1> {
  static constexpr int kVec = 16;
  __device__ static __forceinline__ void pair(uint32_t two_bytes, float& lo, float& hi) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((unsigned short)two_bytes));
    const __half2 v = *reinterpret_cast<const __half2*>(&h2);
    lo = __low2float(v);
    hi = __high2float(v);
  }
  __device__ static __forceinline__ void load(const char* p, float* f) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    pair(v.x & 0xffffu, f[0], f[1]);   pair(v.x >> 16, f[2], f[3]);
    pair(v.y & 0xffffu, f[4], f[5]);   pair(v.y >> 16, f[6], f[7]);
    pair(v.z & 0xffffu, f[8], f[9]);   pair(v.z >> 16, f[10], f[11]);
    pair(v.w & 0xffffu, f[12], f[13]); pair(v.w >> 16, f[14], f[15]);
  }
};
// 4-bit grouped format (tag 0): sixteen stored bytes are one group of 32 codes, element 2i in the low and element
// 2i+1 in the high half of byte i; a code c stands for (c - 8) * the group's scale, the scales (bfloat16) follow
// the codes of a row.  load() yields the 32 numbers c + 128 as floats: 128 + c is the float with bit pattern
// 0x43000000 | (c << 16), so a code costs one shift and one logic operation (the code that already sits at
// bits 16-19 only the latter).  The caller removes the offset kBias = 136 once per group, from the finished
// partial sum (sum_j (c_j + 128) h_j - 136 sum_j h_j), and multiplies by the group's scale.
template <>
struct Elems<0> {
  static constexpr int kVec = 32;
  static constexpr float kBias = 136.f;
  __device__ static __forceinline__ float code(uint32_t at_bit16) {
    return __uint_as_float((at_bit16 & 0x000f0000u) | 0x43000000u);
  }
  __device__ static __forceinline__ void word(uint32_t w, float* f) {
    f[0] = code(w << 16); f[1] = code(w << 12); f[2] = code(w << 8); f[3] = code(w << 4);
    f[4] = code(w);       f[5] = code(w >> 4);  f[6] = code(w >> 8); f[7] = code(w >> 12);
  }
  __device__ static __forceinline__ void load(const char* p, float* f) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    word(v.x, f); word(v.y, f + 8); word(v.z, f + 16); word(v.w, f + 24);
  }
  // scale of 16-byte piece `piece` of the row starting at `row` (H elements)
  __device__ static __forceinline__ float scale(const char* row, int H, int piece) {
    return __uint_as_float((uint32_t)*reinterpret_cast<const unsigned short*>(row + H / 2 + 2 * piece) << 16);
  }
};
// kDot rescales a finished dot product to its true value, kAct multiplies the activation before
// the AXPY (FP8 weights are stored without their factor 2^-8).
template <int WB>
struct WScale {
  static constexpr float kDot = 1.f, kAct = 1.f;
};
template <>
struct WScale<1> {
  static constexpr float kDot = 1.f / 256.f, kAct = 1.f / 256.f;
};

}  // namespace ring
}  // namespace remoe
