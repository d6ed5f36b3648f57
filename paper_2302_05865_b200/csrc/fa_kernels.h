// Internal launch interface between the C ABI (fa_api.cu) and the kernels.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

namespace fa {

int sm_count();   // SMs of the current device (cached per device)

// Gram pass.  `partials` (gram_partials_bytes() bytes) and `counter` are scratch; K (p x p) is
// written by the last block to finish.
int gram_num_blocks(int p, long long n, int dtype);
size_t gram_partials_bytes(int p, long long n, int dtype);
cudaError_t launch_gram(const void* G, int dtype, int p, long long n, double* partials, unsigned int* counter,
                        double* K, int* status, cudaStream_t st);

// Tensor-core Gram pass (bf16, 16 < p <= 64, 16-byte aligned rows); same scratch and output.
bool gram_tc_eligible(const void* G, int dtype, int p, long long n);
cudaError_t launch_gram_tc(const void* G, int p, long long n, double* partials, unsigned int* counter, double* K,
                           int* status, cudaStream_t st);

// Gram pass fed by tensor loads (matrix on a 16-byte boundary, p <= 16); same scratch and output.
bool gram_tm_eligible(const void* G, int dtype, int p, long long n);
cudaError_t launch_gram_tm(const void* G, int dtype, int p, long long n, double* partials, unsigned int* counter,
                           double* K, int* status, cudaStream_t st);

// Tensor-fed Gram pass for fp32 with 16 < p <= 32 and rows on 16-byte boundaries.
bool gram_tm32_eligible(const void* G, int dtype, int p, long long n);
cudaError_t launch_gram_tm32(const void* G, int p, long long n, double* partials, unsigned int* counter, double* K,
                             int* status, cudaStream_t st);

// The same for fp32 with 32 < p <= 64: three launches (two triangles of 32 rows and the rectangle between them).
bool gram_tm64_eligible(const void* G, int dtype, int p, long long n);
cudaError_t launch_gram_tm64(const void* G, int p, long long n, double* partials, unsigned int* counter, double* K,
                             int* status, cudaStream_t st);

// Persistent single-block IRLS on K (p x p).
struct IrlsArgs {
  const double* K;
  int p, m, iters;
  double lambda;
  double a;          // surrogate constant of Eq. (4); 2 = the paper's square roots
  double cb, ca;     // data term cb (1-v)^(1/a) + ca v^(1/a): 2(1-beta), 2(1-alpha) of a Beta likelihood; 1, 0 = Eq. (1)
  int start_from_A;  // 0 uniform first round; 1 start from A0 (orthonormal image); 2 start from any A0
  const double* A0;  // p x m, read before A is written (may alias A)
  double tol;        // >= 0: stop once the objective moved by <= tol; < 0: run all rounds
  int* rounds;       // rounds run, or null
  double* A;
  float* c;
  double* w;
  double* obj;
  double* S;         // p x p selection matrix or null
  int* status;
  int workers;               // > 0: the p rows belong to this many workers, counts[i] consecutive rows each
  unsigned char counts[64];  //      (w then has `workers` entries); 0: one gradient per worker
};
cudaError_t launch_irls(const IrlsArgs& a, cudaStream_t st);

// out[j] = sum_i c[i] G[i][j]
cudaError_t launch_combine(const void* G, int dtype, int p, long long n, const float* c, float* out,
                           cudaStream_t st);

}  // namespace fa
