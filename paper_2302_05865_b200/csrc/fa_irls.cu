// Persistent single-block kernel around the p-dimensional IRLS (Algorithm 1, IRLS step): every
// round -- ratios, Beta-likelihood weights, pairwise regulariser, Jacobi eigensolve -- runs out
// of shared memory; global memory is touched only to read K and write A, c, w, objective.
#include "fa_irls_core.cuh"
#include "fa_kernels.h"

namespace fa {

template <int NT, int LD, bool kPlain>
__global__ void __launch_bounds__(NT, 1) irls_kernel(IrlsArgs a) {
  extern __shared__ __align__(16) unsigned char irls_smem[];
  fa_irls::Ctx ctx{(int)threadIdx.x, (int)blockDim.x};
  const double* K = a.K;
  fa_irls::Smem s;
  fa_irls::carve(s, irls_smem, a.p, ctx.nt);
  fa_irls::Outputs o{a.A, a.c, a.w, a.obj, a.S, a.status, a.rounds};
  const int st = fa_irls::run<LD, kPlain>(ctx, s, K, a.p, a.m, a.lambda, a.a, a.iters, a.start_from_A, a.A0, a.tol, o,
                                           a.workers, a.counts, a.cb, a.ca);
  if (st && a.status && ctx.tid == 0) atomicOr(a.status, st);
}

template <int NT, int LD, bool kPlain>
static cudaError_t launch_kernel(const IrlsArgs& a, cudaStream_t st) {
  const size_t smem = fa_irls::smem_bytes(a.p, NT);
  cudaError_t e = cudaFuncSetAttribute(irls_kernel<NT, LD, kPlain>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  irls_kernel<NT, LD, kPlain><<<1, NT, smem, st>>>(a);
  return cudaGetLastError();
}

// The default terms of the paper (a = 2, Beta(1, 1/2), one gradient per worker) have a kernel of their own with
// everything else compiled out; the arithmetic is the same statements either way.
template <int NT, int LD>
static cudaError_t launch_nt(const IrlsArgs& a, cudaStream_t st) {
  const bool plain = a.a == 2.0 && a.cb == 1.0 && a.ca == 0.0 && a.workers == 0;
  return plain ? launch_kernel<NT, LD, true>(a, st) : launch_kernel<NT, LD, false>(a, st);
}

// One thread per Jacobi work item where the block size allows it: (p/2)^2 2x2 blocks plus
// p * p/2 eigenvector row pairs.
cudaError_t launch_irls(const IrlsArgs& a, cudaStream_t st) {
  // 256 threads up to 16 gradients, 512 above: the matrix phases hand out 8 x 8 tiles to a power-of-two
  // number of warps, and the Jacobi sweeps want one thread per work item where the block size allows it
  if (a.p <= 16) return launch_nt<256, 20>(a, st);
  if (a.p <= 32) return launch_nt<512, 36>(a, st);
  return launch_nt<512, 68>(a, st);
}

}  // namespace fa
