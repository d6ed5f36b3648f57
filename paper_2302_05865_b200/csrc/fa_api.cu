// C ABI of the library (declared in include/fa.h): argument checks, workspace carving, launches.
// Nothing here allocates, frees or synchronises.
#include <math.h>
#include <stdint.h>

#include <atomic>

#include "../../include/fa.h"
#include "fa_kernels.h"

namespace fa {

int sm_count() {
  static std::atomic<int> cached[64];                  // zero-initialised; a slot is published once, whole
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
  int v = cached[dev].load(std::memory_order_acquire);
  if (v == 0) {
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    cached[dev].store(v, std::memory_order_release);   // concurrent first calls store the same value
  }
  return v;
}

namespace {

constexpr size_t kAlign = 256;
inline size_t round_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct Workspace {
  double* partials;
  double* Kbuf;
  float* c;
  unsigned int* counter;
  size_t total;
};

Workspace carve_ws(void* ws, int p, long long n, int dtype) {
  Workspace w{};
  size_t off = 0;
  char* base = static_cast<char*>(ws);
  w.partials = reinterpret_cast<double*>(base + off);
  off += round_up(gram_partials_bytes(p, n, dtype));
  w.Kbuf = reinterpret_cast<double*>(base + off);
  off += round_up((size_t)p * p * sizeof(double));
  w.c = reinterpret_cast<float*>(base + off);
  off += round_up(FA_MAX_P * sizeof(float));
  w.counter = reinterpret_cast<unsigned int*>(base + off);
  off += kAlign;
  w.total = off;
  return w;
}

bool shape_ok(int p, long long n, int dtype) {
  return p >= 1 && p <= FA_MAX_P && n >= 1 && (dtype == FA_F32 || dtype == FA_BF16);
}

bool aligned(const void* ptr, size_t a) { return (reinterpret_cast<uintptr_t>(ptr) % a) == 0; }

// counts (host): `workers` positive entries that add up to `rows`
bool counts_ok(const int* counts, int workers, int rows) {
  if (!counts || workers < 1 || workers > rows) return false;
  long long total = 0;
  for (int i = 0; i < workers; ++i) {
    if (counts[i] < 1 || counts[i] > rows) return false;
    total += counts[i];
  }
  return total == rows;
}

}  // namespace
}  // namespace fa

extern "C" {

const char* fa_error_string(int code) {
  switch (code) {
    case FA_OK: return "ok";
    case FA_ERR_ARG: return "invalid argument";
    case FA_ERR_ALIGN: return "misaligned pointer";
    case FA_ERR_WORKSPACE: return "workspace too small";
    case FA_ERR_CUDA: return "CUDA launch failed";
    case FA_ERR_STATIC_LIMIT: return "shape exceeds the built-in scratch array of fa_gram_static (p <= 32, <= 160 blocks)";
    default: return "unknown error code";
  }
}

int fa_workspace_bytes(int p, long long n, int m, int dtype, size_t* bytes) {
  (void)m;
  if (!bytes || !fa::shape_ok(p, n, dtype)) return FA_ERR_ARG;
  *bytes = fa::carve_ws(nullptr, p, n, dtype).total;
  return FA_OK;
}

int fa_gram(const void* G, int dtype, int p, long long n, double* K, void* ws, size_t ws_bytes, void* stream) {
  if (!G || !K || !ws || !fa::shape_ok(p, n, dtype)) return FA_ERR_ARG;
  if (!fa::aligned(G, dtype == FA_F32 ? 4 : 2) || !fa::aligned(K, 8) || !fa::aligned(ws, 16)) return FA_ERR_ALIGN;
  fa::Workspace w = fa::carve_ws(ws, p, n, dtype);
  if (ws_bytes < w.total) return FA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (fa::launch_gram(G, dtype, p, n, w.partials, w.counter, K, nullptr, st) != cudaSuccess) return FA_ERR_CUDA;
  return FA_OK;
}

int fa_irls_step(const double* K, int p, int m, double lambda, int first, double* A, double* w, double* objective,
                 int* status, void* stream) {
  if (!K || !A || !w || p < 1 || p > FA_MAX_P || m < 1 || m > p || !(lambda >= 0.0) || isinf(lambda)) return FA_ERR_ARG;
  if (!fa::aligned(K, 8) || !fa::aligned(A, 8) || !fa::aligned(w, 8) || (objective && !fa::aligned(objective, 8)) ||
      (status && !fa::aligned(status, 4)))
    return FA_ERR_ALIGN;
  fa::IrlsArgs a{};
  a.cb = 1.0; a.ca = 0.0;
  a.K = K; a.p = p; a.m = m; a.iters = 1; a.lambda = lambda; a.a = 2.0; a.start_from_A = first ? 0 : 1;
  a.A0 = A; a.tol = -1.0;
  a.A = A; a.w = w; a.obj = objective; a.status = status;
  return fa::launch_irls(a, static_cast<cudaStream_t>(stream)) == cudaSuccess ? FA_OK : FA_ERR_CUDA;
}

static int irls_common(const double* K, int p, int m, double lambda, double a, int iters, double tol, const double* A0,
                       double* A_out, float* c_out, double* S_out, double* w_out, double* obj_out, int* rounds_out,
                       int* status, void* stream, double alpha = 1.0, double beta = 0.5) {
  if (!(alpha > 0.0 && alpha <= 1.0 && beta > 0.0 && beta <= 1.0)) return FA_ERR_ARG;
  if (!K || !c_out || p < 1 || p > FA_MAX_P || m < 1 || m > p || iters < 1 || !(lambda >= 0.0) || isinf(lambda) ||
      !(a > 1.0) || isinf(a) || isnan(tol))
    return FA_ERR_ARG;
  if (!fa::aligned(K, 8) || (A_out && !fa::aligned(A_out, 8)) || !fa::aligned(c_out, 4) ||
      (A0 && !fa::aligned(A0, 8)) || (S_out && !fa::aligned(S_out, 8)) || (w_out && !fa::aligned(w_out, 8)) ||
      (obj_out && !fa::aligned(obj_out, 8)) || (rounds_out && !fa::aligned(rounds_out, 4)) ||
      (status && !fa::aligned(status, 4)))
    return FA_ERR_ALIGN;
  fa::IrlsArgs args{};
  args.cb = 1.0; args.ca = 0.0;
  args.K = K; args.p = p; args.m = m; args.iters = iters; args.lambda = lambda; args.a = a;
  args.start_from_A = A0 ? 2 : 0; args.A0 = A0; args.tol = tol; args.rounds = rounds_out;
  if (!(alpha == 1.0 && beta == 0.5)) { args.cb = 2.0 * (1.0 - beta); args.ca = 2.0 * (1.0 - alpha); }
  args.A = A_out; args.c = c_out; args.S = S_out; args.w = w_out; args.obj = obj_out; args.status = status;
  return fa::launch_irls(args, static_cast<cudaStream_t>(stream)) == cudaSuccess ? FA_OK : FA_ERR_CUDA;
}

int fa_irls_ex(const double* K, int p, int m, double lambda, double a, int iters, double* A_out, float* c_out,
               double* S_out, double* w_out, double* obj_out, int* status, void* stream) {
  return irls_common(K, p, m, lambda, a, iters, -1.0, nullptr, A_out, c_out, S_out, w_out, obj_out, nullptr, status,
                     stream);
}

int fa_irls_beta(const double* K, int p, int m, double lambda, double a, double alpha, double beta, int iters,
                 double* A_out, float* c_out, double* w_out, double* obj_out, int* status, void* stream) {
  return irls_common(K, p, m, lambda, a, iters, -1.0, nullptr, A_out, c_out, nullptr, w_out, obj_out, nullptr, status,
                     stream, alpha, beta);
}

int fa_irls_warm(const double* K, int p, int m, double lambda, double a, int iters, double tol, const double* A0,
                 double* A_out, float* c_out, double* w_out, double* obj_out, int* rounds_out, int* status,
                 void* stream) {
  return irls_common(K, p, m, lambda, a, iters, tol, A0, A_out, c_out, nullptr, w_out, obj_out, rounds_out, status,
                     stream);
}

int fa_irls(const double* K, int p, int m, double lambda, int iters, double* A_out, float* c_out, double* w_out,
            double* obj_out, int* status, void* stream) {
  return fa_irls_ex(K, p, m, lambda, 2.0, iters, A_out, c_out, nullptr, w_out, obj_out, status, stream);
}

int fa_combine(const void* G, int dtype, int p, long long n, const float* c, float* out, void* stream) {
  if (!G || !c || !out || !fa::shape_ok(p, n, dtype)) return FA_ERR_ARG;
  if (!fa::aligned(G, dtype == FA_F32 ? 4 : 2) || !fa::aligned(c, 4) || !fa::aligned(out, 4)) return FA_ERR_ALIGN;
  return fa::launch_combine(G, dtype, p, n, c, out, static_cast<cudaStream_t>(stream)) == cudaSuccess ? FA_OK
                                                                                                       : FA_ERR_CUDA;
}

int fa_aggregate_ex(const void* G, int dtype, int p, long long n, int m, double lambda, double a, int iters,
                    float* out, double* A_out, double* S_out, void* ws, size_t ws_bytes, int* status, void* stream) {
  if (!G || !out || !ws || !fa::shape_ok(p, n, dtype) || m < 1 || m > p || iters < 1 || !(lambda >= 0.0) ||
      isinf(lambda) || !(a > 1.0) || isinf(a))
    return FA_ERR_ARG;
  if (!fa::aligned(G, dtype == FA_F32 ? 4 : 2) || !fa::aligned(out, 4) || (A_out && !fa::aligned(A_out, 8)) ||
      (S_out && !fa::aligned(S_out, 8)) || !fa::aligned(ws, 16) || (status && !fa::aligned(status, 4)))
    return FA_ERR_ALIGN;
  fa::Workspace w = fa::carve_ws(ws, p, n, dtype);
  if (ws_bytes < w.total) return FA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (status && cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return FA_ERR_CUDA;
  if (fa::launch_gram(G, dtype, p, n, w.partials, w.counter, w.Kbuf, status, st) != cudaSuccess) return FA_ERR_CUDA;
  fa::IrlsArgs args{};
  args.cb = 1.0; args.ca = 0.0;
  args.K = w.Kbuf;
  args.p = p; args.m = m; args.iters = iters; args.lambda = lambda; args.a = a; args.start_from_A = 0;
  args.tol = -1.0;
  args.A = A_out; args.c = w.c; args.S = S_out; args.status = status;
  if (fa::launch_irls(args, st) != cudaSuccess) return FA_ERR_CUDA;
  if (fa::launch_combine(G, dtype, p, n, w.c, out, st) != cudaSuccess) return FA_ERR_CUDA;
  return FA_OK;
}

int fa_irls_multi(const double* K, int rows, const int* counts, int workers, int m, double lambda, double a, int iters,
                  double* A_out, float* c_out, double* S_out, double* w_out, double* obj_out, int* status,
                  void* stream) {
  if (!K || !c_out || rows < 1 || rows > FA_MAX_P || !fa::counts_ok(counts, workers, rows) || m < 1 || m > rows ||
      iters < 1 || !(lambda >= 0.0) || isinf(lambda) || !(a > 1.0) || isinf(a))
    return FA_ERR_ARG;
  if (!fa::aligned(K, 8) || (A_out && !fa::aligned(A_out, 8)) || !fa::aligned(c_out, 4) ||
      (S_out && !fa::aligned(S_out, 8)) || (w_out && !fa::aligned(w_out, 8)) || (obj_out && !fa::aligned(obj_out, 8)) ||
      (status && !fa::aligned(status, 4)))
    return FA_ERR_ALIGN;
  fa::IrlsArgs args{};
  args.cb = 1.0; args.ca = 0.0;
  args.K = K; args.p = rows; args.m = m; args.iters = iters; args.lambda = lambda; args.a = a; args.start_from_A = 0;
  args.tol = -1.0;
  args.A = A_out; args.c = c_out; args.S = S_out; args.w = w_out; args.obj = obj_out; args.status = status;
  args.workers = workers;
  for (int i = 0; i < workers; ++i) args.counts[i] = (unsigned char)counts[i];
  return fa::launch_irls(args, static_cast<cudaStream_t>(stream)) == cudaSuccess ? FA_OK : FA_ERR_CUDA;
}

int fa_aggregate_multi(const void* G, int dtype, int rows, long long n, const int* counts, int workers, int m,
                       double lambda, double a, int iters, float* out, double* A_out, double* w_out, void* ws,
                       size_t ws_bytes, int* status, void* stream) {
  if (!G || !out || !ws || !fa::shape_ok(rows, n, dtype) || !fa::counts_ok(counts, workers, rows) || m < 1 ||
      m > rows || iters < 1 || !(lambda >= 0.0) || isinf(lambda) || !(a > 1.0) || isinf(a))
    return FA_ERR_ARG;
  if (!fa::aligned(G, dtype == FA_F32 ? 4 : 2) || !fa::aligned(out, 4) || (A_out && !fa::aligned(A_out, 8)) ||
      (w_out && !fa::aligned(w_out, 8)) || !fa::aligned(ws, 16) || (status && !fa::aligned(status, 4)))
    return FA_ERR_ALIGN;
  fa::Workspace w = fa::carve_ws(ws, rows, n, dtype);
  if (ws_bytes < w.total) return FA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (status && cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return FA_ERR_CUDA;
  if (fa::launch_gram(G, dtype, rows, n, w.partials, w.counter, w.Kbuf, status, st) != cudaSuccess) return FA_ERR_CUDA;
  int rc = fa_irls_multi(w.Kbuf, rows, counts, workers, m, lambda, a, iters, A_out, w.c, nullptr, w_out, nullptr, status,
                         stream);
  if (rc != FA_OK) return rc;
  if (fa::launch_combine(G, dtype, rows, n, w.c, out, st) != cudaSuccess) return FA_ERR_CUDA;
  return FA_OK;
}

int fa_aggregate_beta(const void* G, int dtype, int p, long long n, int m, double lambda, double a, double alpha,
                      double beta, int iters, float* out, double* A_out, void* ws, size_t ws_bytes, int* status,
                      void* stream) {
  if (!G || !out || !ws || !fa::shape_ok(p, n, dtype)) return FA_ERR_ARG;
  if (m < 1 || m > p || iters < 1 || !(lambda >= 0.0) || isinf(lambda) || !(a > 1.0) || isinf(a) ||
      !(alpha > 0.0 && alpha <= 1.0 && beta > 0.0 && beta <= 1.0))
    return FA_ERR_ARG;
  if (!fa::aligned(G, dtype == FA_F32 ? 4 : 2) || !fa::aligned(out, 4) || !fa::aligned(ws, 16) ||
      (A_out && !fa::aligned(A_out, 8)) || (status && !fa::aligned(status, 4)))
    return FA_ERR_ALIGN;
  fa::Workspace w = fa::carve_ws(ws, p, n, dtype);
  if (ws_bytes < w.total) return FA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (status && cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return FA_ERR_CUDA;
  if (fa::launch_gram(G, dtype, p, n, w.partials, w.counter, w.Kbuf, status, st) != cudaSuccess) return FA_ERR_CUDA;
  int rc = irls_common(w.Kbuf, p, m, lambda, a, iters, -1.0, nullptr, A_out, w.c, nullptr, nullptr, nullptr, nullptr,
                       status, stream, alpha, beta);
  if (rc != FA_OK) return rc;
  if (fa::launch_combine(G, dtype, p, n, w.c, out, st) != cudaSuccess) return FA_ERR_CUDA;
  return FA_OK;
}

int fa_aggregate_warm(const void* G, int dtype, int p, long long n, int m, double lambda, double a, int iters,
                      double tol, const double* A0, float* out, double* A_out, int* rounds_out, void* ws,
                      size_t ws_bytes, int* status, void* stream) {
  if (!G || !out || !ws || !fa::shape_ok(p, n, dtype)) return FA_ERR_ARG;
  if (m < 1 || m > p || iters < 1 || !(lambda >= 0.0) || isinf(lambda) || !(a > 1.0) || isinf(a) || isnan(tol))
    return FA_ERR_ARG;
  if (!fa::aligned(G, dtype == FA_F32 ? 4 : 2) || !fa::aligned(out, 4) || !fa::aligned(ws, 16) ||
      (A0 && !fa::aligned(A0, 8)) || (A_out && !fa::aligned(A_out, 8)) ||
      (rounds_out && !fa::aligned(rounds_out, 4)) || (status && !fa::aligned(status, 4)))
    return FA_ERR_ALIGN;
  fa::Workspace w = fa::carve_ws(ws, p, n, dtype);
  if (ws_bytes < w.total) return FA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (status && cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return FA_ERR_CUDA;
  if (fa::launch_gram(G, dtype, p, n, w.partials, w.counter, w.Kbuf, status, st) != cudaSuccess) return FA_ERR_CUDA;
  int rc = irls_common(w.Kbuf, p, m, lambda, a, iters, tol, A0, A_out, w.c, nullptr, nullptr, nullptr, rounds_out,
                       status, stream);
  if (rc != FA_OK) return rc;
  if (fa::launch_combine(G, dtype, p, n, w.c, out, st) != cudaSuccess) return FA_ERR_CUDA;
  return FA_OK;
}

int fa_aggregate(const void* G, int dtype, int p, long long n, int m, double lambda, int iters, float* out,
                 double* A_out, void* ws, size_t ws_bytes, int* status, void* stream) {
  return fa_aggregate_ex(G, dtype, p, n, m, lambda, 2.0, iters, out, A_out, nullptr, ws, ws_bytes, status, stream);
}

int fa_aggregate_host(const void* G_host, int dtype, int p, long long n, int m, double lambda, int iters,
                      float* out_host, int* status_host, void* G_dev, float* out_dev, void* ws, size_t ws_bytes,
                      int* status_dev, void* stream) {
  if (!G_host || !out_host || !G_dev || !out_dev || !fa::shape_ok(p, n, dtype)) return FA_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t gbytes = (size_t)p * (size_t)n * (dtype == FA_F32 ? 4 : 2);
  // validate everything else before the first copy is enqueued
  if (!ws || m < 1 || m > p || iters < 1 || !(lambda >= 0.0) || isinf(lambda)) return FA_ERR_ARG;
  if (!fa::aligned(G_dev, dtype == FA_F32 ? 4 : 2) || !fa::aligned(out_dev, 4) || !fa::aligned(ws, 16) ||
      (status_dev && !fa::aligned(status_dev, 4)))
    return FA_ERR_ALIGN;
  if (ws_bytes < fa::carve_ws(ws, p, n, dtype).total) return FA_ERR_WORKSPACE;
  if (cudaMemcpyAsync(G_dev, G_host, gbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return FA_ERR_CUDA;
  int rc = fa_aggregate(G_dev, dtype, p, n, m, lambda, iters, out_dev, nullptr, ws, ws_bytes, status_dev, stream);
  if (rc != FA_OK) return rc;
  if (cudaMemcpyAsync(out_host, out_dev, (size_t)n * sizeof(float), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return FA_ERR_CUDA;
  if (status_host && status_dev &&
      cudaMemcpyAsync(status_host, status_dev, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return FA_ERR_CUDA;
  return FA_OK;
}

}  // extern "C"
