// Shared device helpers: mbarrier / bulk-copy (TMA) wrappers with bounded waits, element loads.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace fa {

constexpr int kStTimeout = 16;                       // FA_ST_TIMEOUT
constexpr long long kWaitCycles = 4000000000LL;      // ~2 s at B200 clocks: limit of any device wait

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
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

// Non-blocking test of a phase (try_wait above may suspend the thread for a system-dependent time).
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

constexpr long long kShortWaitCycles = 1000000;      // limits below this poll without suspending

// Wait for a phase with a cycle limit.  Returns false when the limit ran out (the caller then
// records FA_ST_TIMEOUT and winds down); never spins unbounded.  `limit` is the caller's primary
// limit (a launch parameter where a test shortens it); waits that only let copies already in
// flight land before a block exits always use the long default.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, long long limit = kWaitCycles) {
  if (limit < kShortWaitCycles) {      // a deliberately short limit: the suspending form could outlast it
    const long long t0 = clock64();
    do {
      if (mbar_test_wait(bar, parity)) return true;
    } while (clock64() - t0 <= limit);
    return false;
  }
  if (mbar_try_wait(bar, parity)) return true;
  long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > limit) return false;
  }
  return true;
}

// One-dimensional bulk copy global -> shared, completion counted in bytes on `bar`.
// src and dst must be 16-byte aligned and bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst)),
      "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Butterfly reduce-scatter of NACCP values per lane across the warp: afterwards lane l holds the
// warp sums of elements [l*NACCP/32, (l+1)*NACCP/32) in x[0 .. NACCP/32).  NACCP is a multiple of 32.
template <int NACCP, int L, int MASK>
__device__ __forceinline__ void butterfly_step(float (&x)[NACCP], int lane) {
  if constexpr (MASK >= 1) {
    constexpr int H = L / 2;
    const bool up = (lane & MASK) != 0;
#pragma unroll
    for (int k = 0; k < H; ++k) {
      float lo = x[k], hi = x[H + k];
      float send = up ? lo : hi;
      float keep = up ? hi : lo;
      x[k] = keep + __shfl_xor_sync(0xffffffffu, send, MASK);
    }
    butterfly_step<NACCP, H, MASK / 2>(x, lane);
  }
}

template <int NACCP>
__device__ __forceinline__ void flush(float (&acc)[NACCP], double (&dacc)[NACCP / 32], int lane) {
  butterfly_step<NACCP, NACCP, 16>(acc, lane);
#pragma unroll
  for (int k = 0; k < NACCP / 32; ++k) dacc[k] += static_cast<double>(acc[k]);
#pragma unroll
  for (int k = 0; k < NACCP; ++k) acc[k] = 0.f;
}

// ---- element access: V consecutive elements at a V-element-aligned shared address -> floats
template <typename T, int V>
struct SmemVec;

template <>
struct SmemVec<float, 1> {
  static __device__ __forceinline__ void load(const char* p, float (&v)[1]) { v[0] = *reinterpret_cast<const float*>(p); }
};
template <>
struct SmemVec<float, 2> {
  static __device__ __forceinline__ void load(const char* p, float (&v)[2]) {
    float2 t = *reinterpret_cast<const float2*>(p);
    v[0] = t.x; v[1] = t.y;
  }
};
template <>
struct SmemVec<float, 4> {
  static __device__ __forceinline__ void load(const char* p, float (&v)[4]) {
    float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
};
template <>
struct SmemVec<__nv_bfloat16, 1> {
  static __device__ __forceinline__ void load(const char* p, float (&v)[1]) {
    v[0] = __uint_as_float(static_cast<uint32_t>(*reinterpret_cast<const uint16_t*>(p)) << 16);
  }
};
template <>
struct SmemVec<__nv_bfloat16, 2> {
  static __device__ __forceinline__ void load(const char* p, float (&v)[2]) {
    uint32_t u = *reinterpret_cast<const uint32_t*>(p);
    v[0] = __uint_as_float(u << 16); v[1] = __uint_as_float(u & 0xffff0000u);
  }
};
template <>
struct SmemVec<__nv_bfloat16, 4> {
  static __device__ __forceinline__ void load(const char* p, float (&v)[4]) {
    uint2 u = *reinterpret_cast<const uint2*>(p);
    v[0] = __uint_as_float(u.x << 16); v[1] = __uint_as_float(u.x & 0xffff0000u);
    v[2] = __uint_as_float(u.y << 16); v[3] = __uint_as_float(u.y & 0xffff0000u);
  }
};

}  // namespace fa
