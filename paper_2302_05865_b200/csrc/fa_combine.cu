// Output pass: out[j] = sum_i c_i G[i][j]  (Algorithm 1, direction step d = (1/p) Y Y^T G 1, in the
// right-multiplied form of the appendix's optimality conditions: Y Y^T G 1 / p = G c).
// Pure streaming: p coalesced loads per output element, fp32 FMA, one store.  Column groups are
// walked from the END of the rows backwards, so the part of G that the Gram pass read last and
// that still sits in L2 is consumed first.
#include <cuda_bf16.h>
#include <stdint.h>

#include "fa_kernels.h"

namespace fa {
namespace combine {

constexpr int kThreads = 256;

template <typename T, int V> struct Vec;
template <> struct Vec<float, 1> { using type = float; };
template <> struct Vec<float, 2> { using type = float2; };
template <> struct Vec<float, 4> { using type = float4; };
template <> struct Vec<__nv_bfloat16, 1> { using type = uint16_t; };
template <> struct Vec<__nv_bfloat16, 2> { using type = uint32_t; };
template <> struct Vec<__nv_bfloat16, 4> { using type = uint2; };
template <> struct Vec<__nv_bfloat16, 8> { using type = uint4; };

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

template <int V> __device__ __forceinline__ void unpack(float v, float (&x)[V]) { x[0] = v; }
template <int V> __device__ __forceinline__ void unpack(float2 v, float (&x)[V]) { x[0] = v.x; x[1] = v.y; }
template <int V> __device__ __forceinline__ void unpack(float4 v, float (&x)[V]) { x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w; }
template <int V> __device__ __forceinline__ void unpack(uint16_t v, float (&x)[V]) { x[0] = __uint_as_float((uint32_t)v << 16); }
template <int V> __device__ __forceinline__ void unpack(uint32_t v, float (&x)[V]) { x[0] = bf_lo(v); x[1] = bf_hi(v); }
template <int V> __device__ __forceinline__ void unpack(uint2 v, float (&x)[V]) { x[0] = bf_lo(v.x); x[1] = bf_hi(v.x); x[2] = bf_lo(v.y); x[3] = bf_hi(v.y); }
template <int V> __device__ __forceinline__ void unpack(uint4 v, float (&x)[V]) {
  x[0] = bf_lo(v.x); x[1] = bf_hi(v.x); x[2] = bf_lo(v.y); x[3] = bf_hi(v.y);
  x[4] = bf_lo(v.z); x[5] = bf_hi(v.z); x[6] = bf_lo(v.w); x[7] = bf_hi(v.w);
}

// Each thread owns V consecutive columns (all rows are V-element aligned there); n % V == 0.
template <typename T, int V>
__global__ void __launch_bounds__(kThreads) combine_kernel(const T* __restrict__ G, int p, long long n,
                                                          const float* __restrict__ c, float* __restrict__ out) {
  using VT = typename Vec<T, V>::type;
  __shared__ float cs[64];
  float mine = 0.f;
  if (threadIdx.x < 64) { mine = threadIdx.x < p ? c[threadIdx.x] : 0.f; cs[threadIdx.x] = mine; }
  const int any = __syncthreads_or(mine != 0.f);
  const long long groups = n / V;
  const long long g = groups - 1 - ((long long)blockIdx.x * kThreads + threadIdx.x);
  if (g < 0) return;
  if (!any) {   // c = 0 (rejected or all-zero input): the result is exactly zero whatever G holds
#pragma unroll
    for (int e = 0; e < V; ++e) out[g * V + e] = 0.f;
    return;
  }
  const T* col = G + g * V;
  float acc[V];
#pragma unroll
  for (int e = 0; e < V; ++e) acc[e] = 0.f;
  int i = 0;
  for (; i + 8 <= p; i += 8) {
    VT v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = __ldcs(reinterpret_cast<const VT*>(col + (size_t)(i + k) * n));
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      float x[V];
      unpack<V>(v[k], x);
      const float ck = cs[i + k];
#pragma unroll
      for (int e = 0; e < V; ++e) acc[e] = fmaf(ck, x[e], acc[e]);
    }
  }
  for (; i < p; ++i) {
    float x[V];
    unpack<V>(__ldcs(reinterpret_cast<const VT*>(col + (size_t)i * n)), x);
    const float ck = cs[i];
#pragma unroll
    for (int e = 0; e < V; ++e) acc[e] = fmaf(ck, x[e], acc[e]);
  }
  float* o = out + g * V;
  // `out` is only guaranteed element-aligned: store element-wise unless the vector store is aligned
  if (V > 1 && (reinterpret_cast<uintptr_t>(o) % (V * sizeof(float))) == 0) {
    if constexpr (V == 2) __stcs(reinterpret_cast<float2*>(o), make_float2(acc[0], acc[1]));
    else if constexpr (V == 4) __stcs(reinterpret_cast<float4*>(o), make_float4(acc[0], acc[1], acc[2], acc[3]));
    else if constexpr (V == 8) {
      __stcs(reinterpret_cast<float4*>(o), make_float4(acc[0], acc[1], acc[2], acc[3]));
      __stcs(reinterpret_cast<float4*>(o) + 1, make_float4(acc[4], acc[5], acc[6], acc[7]));
    }
  } else {
#pragma unroll
    for (int e = 0; e < V; ++e) __stcs(o + e, acc[e]);
  }
}

// fp32 rows that start on 8-byte but not all on 16-byte boundaries (n even with n % 4 = 2, or a base
// that is 8 modulo 16): every row is still read with 16-byte loads.  A thread owns columns 4g..4g+3.
// From a row whose start is 8 modulo 16 ("shifted") it loads the aligned vector at columns
// 4g-2..4g+1: the upper half belongs to its own columns 0 and 1, the lower half to columns 2 and 3
// of the thread that owns the group before (g - 1), for which it keeps a second pair of sums.  At
// the end the pair is handed over with one shuffle.  Groups are walked from the end of the rows
// backwards (see the kernel above), so group g - 1 sits in the next lane; the first lane of a warp
// has no lane to receive from and reads its columns 2 and 3 of the shifted rows itself (8-byte
// loads, 1/32 of the threads).  The thread of group 0 must not read before the matrix, and the last
// two columns (n % 4 = 2) form a half group: both use 8-byte loads where a vector would leave the row.
__global__ void __launch_bounds__(kThreads) combine_shifted_kernel(const float* __restrict__ G, int p, long long n,
                                                                  const float* __restrict__ c, float* __restrict__ out,
                                                                  int shift0, int nmod) {
  __shared__ float cs[64];
  float mine = 0.f;
  if (threadIdx.x < 64) { mine = threadIdx.x < p ? c[threadIdx.x] : 0.f; cs[threadIdx.x] = mine; }
  const int any = __syncthreads_or(mine != 0.f);
  const long long full = n / 4;                         // whole groups; a half group of two columns may follow
  const long long groups = full + ((n & 3) ? 1 : 0);
  const long long g = groups - 1 - ((long long)blockIdx.x * kThreads + threadIdx.x);
  const bool live = g >= 0;
  const bool half = live && g == full;                  // the two columns n-2, n-1
  const long long col = (live ? g : 0) * 4;
  if (!any) {   // c = 0 (rejected or all-zero input): the result is exactly zero whatever G holds
    if (live) for (int e = 0; e < (half ? 2 : 4); ++e) out[col + e] = 0.f;
    return;
  }
  const int lane = threadIdx.x & 31;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;         // own columns
  float b0 = 0.f, b1 = 0.f;                             // columns 2, 3 of group g - 1, from shifted rows
  float e0 = 0.f, e1 = 0.f;                             // own columns 2, 3 from shifted rows, first lane only
  if (live) {
    for (int i0 = 0; i0 < p; i0 += 8) {
      float4 v[8];
      float2 w[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int i = i0 + k;
        v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        w[k] = make_float2(0.f, 0.f);
        if (i < p) {
          const float* row = G + (size_t)i * n + col;
          const bool shifted = ((shift0 + i * nmod) & 3) != 0;
          if (!shifted) {
            if (!half) v[k] = __ldcs(reinterpret_cast<const float4*>(row));
            else { const float2 t = __ldcs(reinterpret_cast<const float2*>(row)); v[k].x = t.x; v[k].y = t.y; }
          } else {
            if (g > 0) v[k] = __ldcs(reinterpret_cast<const float4*>(row - 2));            // columns 4g-2 .. 4g+1
            else { const float2 t = __ldcs(reinterpret_cast<const float2*>(row)); v[k].z = t.x; v[k].w = t.y; }
            if (lane == 0 && !half) w[k] = __ldcs(reinterpret_cast<const float2*>(row + 2));
          }
        }
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int i = i0 + k;
        const float ck = i < p ? cs[i] : 0.f;
        const bool shifted = ((shift0 + i * nmod) & 3) != 0;
        if (!shifted) {
          a0 = fmaf(ck, v[k].x, a0); a1 = fmaf(ck, v[k].y, a1); a2 = fmaf(ck, v[k].z, a2); a3 = fmaf(ck, v[k].w, a3);
        } else {
          b0 = fmaf(ck, v[k].x, b0); b1 = fmaf(ck, v[k].y, b1); a0 = fmaf(ck, v[k].z, a0); a1 = fmaf(ck, v[k].w, a1);
          e0 = fmaf(ck, w[k].x, e0); e1 = fmaf(ck, w[k].y, e1);
        }
      }
    }
  }
  // columns 2, 3 of this group from the shifted rows: summed by the thread of group g + 1 (previous lane)
  const float r0 = __shfl_up_sync(0xffffffffu, b0, 1), r1 = __shfl_up_sync(0xffffffffu, b1, 1);
  if (!live) return;
  a2 += (lane == 0) ? e0 : r0;
  a3 += (lane == 0) ? e1 : r1;
  float* o = out + col;
  if (half) { __stcs(o, a0); __stcs(o + 1, a1); return; }
  if ((reinterpret_cast<uintptr_t>(o) % 16) == 0) __stcs(reinterpret_cast<float4*>(o), make_float4(a0, a1, a2, a3));
  else { __stcs(o, a0); __stcs(o + 1, a1); __stcs(o + 2, a2); __stcs(o + 3, a3); }
}

template <typename T, int V>
static cudaError_t run(const void* G, int p, long long n, const float* c, float* out, cudaStream_t st) {
  const long long groups = n / V;
  const long long blocks = (groups + kThreads - 1) / kThreads;
  combine_kernel<T, V><<<(unsigned)blocks, kThreads, 0, st>>>(static_cast<const T*>(G), p, n, c, out);
  return cudaGetLastError();
}

}  // namespace combine

cudaError_t launch_combine(const void* G, int dtype, int p, long long n, const float* c, float* out,
                           cudaStream_t st) {
  const uintptr_t a = reinterpret_cast<uintptr_t>(G);
  if (dtype == 0) {
    if (n % 4 == 0 && a % 16 == 0) return combine::run<float, 4>(G, p, n, c, out, st);
    if (n % 2 == 0 && a % 8 == 0 && n >= 8) {            // every row on an 8-byte boundary: 16-byte loads with a hand-over
      const long long groups = n / 4 + ((n & 3) ? 1 : 0);
      const long long blocks = (groups + combine::kThreads - 1) / combine::kThreads;
      combine::combine_shifted_kernel<<<(unsigned)blocks, combine::kThreads, 0, st>>>(
          static_cast<const float*>(G), p, n, c, out, (int)((a % 16) / 4), (int)(n % 4));
      return cudaGetLastError();
    }
    if (n % 2 == 0 && a % 8 == 0) return combine::run<float, 2>(G, p, n, c, out, st);
    return combine::run<float, 1>(G, p, n, c, out, st);
  }
  if (n % 8 == 0 && a % 16 == 0) return combine::run<__nv_bfloat16, 8>(G, p, n, c, out, st);
  if (n % 4 == 0 && a % 8 == 0) return combine::run<__nv_bfloat16, 4>(G, p, n, c, out, st);
  if (n % 2 == 0 && a % 4 == 0) return combine::run<__nv_bfloat16, 2>(G, p, n, c, out, st);
  return combine::run<__nv_bfloat16, 1>(G, p, n, c, out, st);
}

}  // namespace fa
