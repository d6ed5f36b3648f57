// Internal launch interface between the C ABI (fa_api.cu) and the kernels.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

namespace fa {

int sm_count();   // SMs of the current device (cached per device)

// Gram pass -> per-block partial triangles in `partials` (gram_partials_bytes() bytes).
int gram_num_blocks(int p, long long n, int dtype);
size_t gram_partials_bytes(int p, long long n, int dtype);
cudaError_t launch_gram_partials(const void* G, int dtype, int p, long long n, double* partials, int* status,
                                 cudaStream_t st, int* nblocks_out);
cudaError_t launch_reduce_partials(const double* partials, int nblocks, int p, double* K, cudaStream_t st);

// Persistent single-block IRLS.  If `partials` is non-null the block first sums the Gram slots
// into Kbuf (p*p doubles) and uses that; otherwise it reads K.
struct IrlsArgs {
  const double* K;
  const double* partials;
  int nblocks;
  double* Kbuf;
  int p, m, iters;
  double lambda;
  int start_from_A;
  double* A;
  float* c;
  double* w;
  double* obj;
  int* status;
};
cudaError_t launch_irls(const IrlsArgs& a, cudaStream_t st);

// out[j] = sum_i c[i] G[i][j]
cudaError_t launch_combine(const void* G, int dtype, int p, long long n, const float* c, float* out,
                           cudaStream_t st);

}  // namespace fa
