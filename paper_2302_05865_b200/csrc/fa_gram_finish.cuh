// Tail shared by the Gram kernels: per-block partial sums -> K, by the last block to finish.
#pragma once
#include <cuda_runtime.h>

namespace fa {
namespace gram {

// Position of (i, j), i <= j, in the row-major upper triangle of a p x p matrix.
__host__ __device__ inline int canon_index(int i, int j, int p) {
  return i * p - (i * (i - 1)) / 2 + (j - i);
}

// Called by every thread of a block after it has written its entries of `partials`.  The last
// block to arrive (atomic counter) adds up all blocks' entries and writes the symmetric K.  Each
// entry is summed by one warp: lane l takes blocks l, l+32, ... in order, then a fixed shuffle
// tree -- the order does not depend on which block happens to be last, so K is bit-reproducible.
__device__ __forceinline__ void finish_gram(double* partials, unsigned int* counter, double* K, int p, int* smem_flag) {
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned int done = atomicAdd(counter, 1u);
    *smem_flag = (done == gridDim.x - 1) ? 1 : 0;
  }
  __syncthreads();
  if (!*smem_flag) return;
  __threadfence();
  const int ntri = p * (p + 1) / 2;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int nb = gridDim.x;
  constexpr int E = 10;                          // entries a warp sums at once
  for (int c0 = warp * E; c0 < ntri; c0 += nwarps * E) {
    double sum[E];
#pragma unroll
    for (int e = 0; e < E; ++e) sum[e] = 0.0;
    // The first 160 blocks: every load of the lane goes out before the first add -- the loads are
    // unconditional (clamped indices, masked afterwards) so that nothing keeps them from being issued
    // back to back; a round then costs one trip to L2 (about 0.7 us here) instead of five.  The adds
    // keep their order (blocks lane, lane + 32, ...), so the sums are the same bits as before.
    constexpr int kUnrolled = 5;
    double v[kUnrolled][E];
#pragma unroll
    for (int k = 0; k < kUnrolled; ++k) {
      const int b = min(lane + 32 * k, nb - 1);
#pragma unroll
      for (int e = 0; e < E; ++e) v[k][e] = __ldcg(partials + (size_t)min(c0 + e, ntri - 1) * nb + b);
    }
#pragma unroll
    for (int k = 0; k < kUnrolled; ++k) {
      const bool ok = lane + 32 * k < nb;
#pragma unroll
      for (int e = 0; e < E; ++e) sum[e] += ok ? v[k][e] : 0.0;
    }
    for (int b = lane + 32 * kUnrolled; b < nb; b += 32) {
#pragma unroll
      for (int e = 0; e < E; ++e)
        if (c0 + e < ntri) sum[e] += __ldcg(partials + (size_t)(c0 + e) * nb + b);
    }
#pragma unroll
    for (int e = 0; e < E; ++e) {
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) sum[e] += __shfl_xor_sync(0xffffffffu, sum[e], off);
    }
    if (lane == 0) {
#pragma unroll
      for (int e = 0; e < E; ++e) {
        const int c = c0 + e;
        if (c < ntri) {
          int i = 0, r = c;
          while (r >= p - i) { r -= p - i; ++i; }
          const int j = i + r;
          K[i * p + j] = sum[e];
          K[j * p + i] = sum[e];
        }
      }
    }
  }
  if (threadIdx.x == 0) *counter = 0u;     // leave the counter ready for the next launch
}

}  // namespace gram
}  // namespace fa
