// Test helper: the p-dimensional IRLS of csrc/fa_irls_core.cuh compiled for the host with one
// "thread" (FA_IRLS_HOST), so that its arithmetic can be compared with the CPU oracle on machines
// without a GPU.  The device build runs the same phases with the loops spread over a thread block.
#define FA_IRLS_HOST 1
#include <stdlib.h>
#include <string.h>

#include "../paper_2302_05865_b200/csrc/fa_irls_core.cuh"

extern "C" int irls_host(const double* K, int p, int m, double lambda, double a, int iters, int start,
                         const double* A0, double tol, double* A, float* c, double* w, double* obj, double* S,
                         int* rounds, int workers, const unsigned char* counts, double cb, double ca,
                         int* sweeps_out, int* refinements_out, int* sweeps_f32_out) {
  const size_t bytes = fa_irls::smem_bytes(p, 1);
  void* mem = calloc(bytes, 1);
  fa_irls::Ctx ctx{0, 1};
  fa_irls::Smem s;
  fa_irls::carve(s, mem, p, 1);
  fa_irls::Outputs o{A, c, w, obj, S, nullptr, rounds};
  int st;
  if (p <= 16) st = fa_irls::run<20>(ctx, s, K, p, m, lambda, a, iters, start, A0, tol, o, workers, counts, cb, ca);
  else if (p <= 32) st = fa_irls::run<36>(ctx, s, K, p, m, lambda, a, iters, start, A0, tol, o, workers, counts, cb, ca);
  else st = fa_irls::run<68>(ctx, s, K, p, m, lambda, a, iters, start, A0, tol, o, workers, counts, cb, ca);
  if (sweeps_out) *sweeps_out = s.count_sweeps;
  if (refinements_out) *refinements_out = s.count_refinements;
  if (sweeps_f32_out) *sweeps_f32_out = s.count_sweeps_f32;
  free(mem);
  return st;
}
