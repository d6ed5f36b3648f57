// IRLS of the Flag Aggregator carried out in p-dimensional coordinates by ONE thread block.
//
// Input is only K (p x p inner products of the gradients).  The n-dimensional problem of
// Algorithm 1 / Eq. (5) is mapped isometrically to R^r, r = rank(K):
//   * Kt = D^-1 K D^-1 with D = diag(sqrt(K_ii))  (unit diagonal, so the truncation of null
//     directions below does not depend on the scale of any single worker);
//   * Kt = V L V^T by cyclic Jacobi; the r eigenpairs with L_k > RANK_REL * L_1 are kept;
//   * f_i = L^(1/2) V^T D e_i in R^r satisfies <f_i, f_j> = K_ij, and Q = G D^-1 V L^(-1/2)
//     (n x r) has orthonormal columns with Q^T g_i = f_i.
// A subspace Y = Q Z is represented by Z (r x m); in gradient coordinates Y = G A with
// A = D^-1 V L^(-1/2) Z.  Each round forms T = sum w_i f_i f_i^T + sum w_ij (f_i-f_j)(f_i-f_j)^T
// = F M F^T in the previous round's eigenbasis and diagonalises it: cyclic Jacobi sweeps while T is
// far from diagonal, then a matrix-product refinement of the eigenvectors that squares the error
// per step at about a tenth of the cost of a sweep (refine_eig below).  The m leading eigenvectors
// are kept and the terms under the square roots of Eq. (5) are evaluated as squared residual norms,
// i.e. as sums of squares over the discarded eigen-directions -- no "1 - x" cancellation.
//
// The code is written as phases separated by block barriers, every phase a strided loop over
// independent items, so that it also compiles for the host with one "thread" (FA_IRLS_HOST): the
// CPU test suite runs that build against the CPU reference implementation.
#pragma once

#include <math.h>
#include <stdint.h>

#ifndef FA_IRLS_HOST
#define FA_FN __device__ __forceinline__
#define FA_HD __host__ __device__ inline
// A function that is called from several places and is large, or that only rare arguments reach: one copy,
// out of line.  The kernels' code does not fit the instruction cache (stalls for instruction fetch were
// a fifth of all stall cycles at 15 gradients), so every copy that is not needed is paid for in time.
#define FA_FN_SHARED __device__ __noinline__
#else
#define FA_FN static inline
#define FA_HD static inline
#define FA_FN_SHARED static
#endif

#ifndef FA_IRLS_HOST
// 1/sqrt(x) for normal positive x: hardware approximation (about 22 bits) and two Newton steps.
__device__ __forceinline__ double fa_fast_rsqrt(double x) {
  double y;
  asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
  const double hx = 0.5 * x;
  y = y * fma(-hx * y, y, 1.5);
  y = y * fma(-hx * y, y, 1.5);
  return y;
}
// The bare hardware approximation (relative error about 2^-22).
__device__ __forceinline__ double fa_approx_rsqrt(double x) {
  double y;
  asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
  return y;
}
#define FA_RSQRT(x) fa_fast_rsqrt(x)
#define FA_RSQRT_APPROX(x) fa_approx_rsqrt(x)
#else
#define FA_RSQRT(x) (1.0 / sqrt(x))
#define FA_RSQRT_APPROX(x) (1.0 / sqrt(x))
#endif

namespace fa_irls {

constexpr double kEps = 1e-6;          // floor on sqrt(term) inside a weight
constexpr double kZeroNormRel = 1e-30; // K_ii <= this * max K_kk: zero gradient
constexpr double kSamePairRel = 1e-12; // D_ij^2 <= this * (K_ii + K_jj): identical pair
constexpr double kRankRel = 1e-12;     // eigenvalue <= this * largest: direction dropped
constexpr double kJacobiTol = 1e-17;   // rotate when |a_pq| > tol * sqrt(|a_pp a_qq|)
constexpr double kJacobiBig = 1e-6;    // sweep again while some rotated |a_pq| exceeded this (relative)
constexpr int kMaxSweeps = 40;
// The refinement is tried when every |T_ij| <= theta * |T_jj - T_ii|, has converged when a step's largest
// correction is below kRefineStop, and is given up when a step's largest correction is not below
// `contract` times the one before.  Up to 32 gradients a declined attempt is cheap next to a sweep, so the
// reach is set wide (measured on the workloads' spectra: 13 sweeps + 51 steps instead of 16 + 45 at p = 15,
// 20 + 90 instead of 26 + 82 at p = 31); above, a failed attempt costs a quarter of a sweep and the tighter
// pair is faster (p = 63 at its full size: 2.9 ms per call against 3.8 ms).
template <int LD> struct RefineLimits {
  static constexpr double theta = LD > 36 ? 0.3 : 0.5;
  static constexpr double contract = LD > 36 ? 0.5 : 0.7;
};
constexpr double kRefineStop = 1e-8;
constexpr int kMaxRefine = 8;          // steps after which a refinement that has not converged is given up
constexpr int kMaxSweepsF32 = 12;      // fp32 sweeps per round before the fp64 sweeps take over
constexpr int kMaxP = 64;

constexpr int ST_NONFINITE = 1, ST_RANK0 = 2, ST_RANK_LT_M = 4, ST_EIG_SWEEPS = 8;

struct Ctx {
  int tid, nt;
#ifndef FA_IRLS_HOST
  FA_FN void sync() const { __syncthreads(); }
#else
  void sync() const {}
#endif
};

// x / d for 0 <= x < 65536 and 1 <= d <= 64 without an integer division (a division by a run-time
// value has a latency of about 75 cycles on this GPU, which is a fifth of a whole phase here): with
// mul = ceil(2^32 / d) the high word of x * mul is the quotient exactly for these ranges.
struct FastDiv { unsigned mul; int d; };
FA_HD FastDiv make_div(int d) {
  FastDiv f;
  f.d = d < 1 ? 1 : d;
  f.mul = f.d == 1 ? 0u : (unsigned)((0x100000000ULL + (unsigned long long)f.d - 1ULL) / (unsigned long long)f.d);
  return f;
}
FA_FN int fast_div(int x, const FastDiv& f) {
#ifndef FA_IRLS_HOST
  return f.d == 1 ? x : (int)__umulhi((unsigned)x, f.mul);
#else
  return x / f.d;
#endif
}

// Leading dimension of every matrix buffer: a compile-time constant per kernel instantiation (20, 36
// or 68 doubles for up to 16, 32, 64 rows), which turns the element offsets of the unrolled inner
// loops into immediates.  It is 4 modulo 16: the sixteen lanes of a half-warp that load a tensor-core
// fragment (4 rows x 4 consecutive elements, or the transpose) then hit sixteen different bank pairs.
constexpr int kLdPad = 4;
FA_HD int leading_dim(int p) { return (p <= 16 ? 16 : (p <= 32 ? 32 : 64)) + kLdPad; }

// Shared-memory image.  Matrices are (ld - kLdPad) x ld doubles.
struct Smem {
  double *T, *J, *P, *M, *Aacc, *tmp;   // six matrix buffers, rotated by pointer swaps
  double *V0, *V1;                       // up to 32 gradients: two more, for T X of the refinement (null above)
  double *kd, *dinv, *fn, *u, *w, *wused, *ev, *red;
  double *lam, *rdiag;                   // refinement: eigenvalue estimates, diagonal of I - X^T X
  double *rc, *rs;                       // rotation cos / sin per pair
  int *ra, *rb, *ord;                    // rotation indices per pair, sort order
  int *piv;                              // pivot column of every step of the factorisation
  unsigned short* pairs;                 // (i << 8) | j of the q-th worker pair i < j (see tri_pair)
  int *flags;                            // [0],[3] rotated-this-sweep (by sweep parity), [1] scratch
  // several gradients per worker (nw > 0): per-worker trace, value, weight, weight in use, 1/k_i;
  // grp[row] = worker of a row, first[i] = first row of worker i
  double *gtr, *gu, *gw, *gwused, *ginv;
  int *grp, *first;
  int nw;
  int ld;
  int count_sweeps, count_sweeps_f32, count_refinements;   // work done by the eigensolver in this call (diagnostics)
  FastDiv div_r, div_p, div_tr, div_tp;  // by the rank r, by p, by their numbers of 8-wide tiles
  int max_calls, sum_calls;              // block_max / block_sum calls so far (parity picks the exchange slots)
};

FA_HD size_t smem_bytes(int p, int nt) {
  int ld = leading_dim(p);
  int pp = ld - kLdPad;
  size_t doubles = (size_t)(ld <= 36 ? 8 : 6) * pp * ld + (size_t)14 * pp + (nt < 128 ? 128 : nt) + 2 * (pp / 2 + 1);
  size_t ints = (size_t)2 * (pp / 2 + 1) + 4 * pp + 8 + (size_t)(pp * (pp - 1) / 2 + 1) / 2;
  return doubles * sizeof(double) + ints * sizeof(int) + 64;
}

FA_FN void carve(Smem& s, void* base, int p, int nt) {
  int ld = leading_dim(p);
  int pp = ld - kLdPad;
  double* d = reinterpret_cast<double*>(base);
  s.ld = ld;
  s.T = d; d += (size_t)pp * ld;
  s.J = d; d += (size_t)pp * ld;
  s.P = d; d += (size_t)pp * ld;
  s.M = d; d += (size_t)pp * ld;
  s.Aacc = d; d += (size_t)pp * ld;
  s.tmp = d; d += (size_t)pp * ld;
  s.V0 = s.V1 = nullptr;
  if (ld <= 36) { s.V0 = d; d += (size_t)pp * ld; s.V1 = d; d += (size_t)pp * ld; }
  s.kd = d; d += pp; s.dinv = d; d += pp; s.fn = d; d += pp; s.u = d; d += pp;
  s.w = d; d += pp; s.wused = d; d += pp; s.ev = d; d += pp;
  s.gtr = d; d += pp; s.gu = d; d += pp; s.gw = d; d += pp; s.gwused = d; d += pp; s.ginv = d; d += pp;
  s.lam = d; d += pp; s.rdiag = d; d += pp;
  s.red = d; d += (nt < 128 ? 128 : nt);
  s.rc = d; d += pp / 2 + 1; s.rs = d; d += pp / 2 + 1;
  int* q = reinterpret_cast<int*>(d);
  s.ra = q; q += pp / 2 + 1; s.rb = q; q += pp / 2 + 1; s.ord = q; q += pp; s.grp = q; q += pp;
  s.first = q; q += pp; s.piv = q; q += pp; s.flags = q; q += 8;
  s.pairs = reinterpret_cast<unsigned short*>(q);
  s.nw = 0;
  s.count_sweeps = 0; s.count_sweeps_f32 = 0; s.count_refinements = 0;
  s.div_r = s.div_p = s.div_tr = s.div_tp = make_div(1);
  s.max_calls = 0; s.sum_calls = 0;
}

// Deterministic block-wide sum; every thread gets the result.  One barrier: the exchange slots
// alternate between calls (see block_max), and every thread adds the warps' sums in the same order.
FA_FN double block_sum(const Ctx& c, Smem& s, double v) {
#ifndef FA_IRLS_HOST
  for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
  double* slots = s.red + 64 + ((s.sum_calls++ & 1) ? 32 : 0);
  if ((c.tid & 31) == 0) slots[c.tid >> 5] = v;
  c.sync();
  double tot = 0.0;
  const int nw = c.nt >> 5;
  for (int k = 0; k < nw; ++k) tot += slots[k];
  return tot;
#else
  (void)c; (void)s;
  return v;
#endif
}

// Block-wide maximum of non-negative finite values; every thread gets the result, truncated to the
// upper 32 bits of the double (about six digits) -- it only feeds threshold decisions, and every
// thread takes the same ones.  Non-negative doubles order like their upper words, so the reduction
// runs on integers: one warp reduction, one shared-memory exchange, one barrier (the exchange slots
// alternate between calls, which keeps a slow warp's reads apart from the next call's writes).
FA_FN double block_max(const Ctx& c, Smem& s, double v) {
#ifndef FA_IRLS_HOST
  const unsigned hi = __reduce_max_sync(0xffffffffu, (unsigned)__double2hiint(v));
  unsigned* slots = reinterpret_cast<unsigned*>(s.red) + ((s.max_calls++ & 1) ? 32 : 0);
  if ((c.tid & 31) == 0) slots[c.tid >> 5] = hi;
  c.sync();
  unsigned m = 0u;
  const int nw = c.nt >> 5;
  for (int k = 0; k < nw; ++k) m = max(m, slots[k]);
  return __hiloint2double((int)m, 0);
#else
  (void)c; (void)s;
  return v;
#endif
}

// sum_k a[k * SA] * b[k * SB] over k < n <= NMAX.  The phases of this kernel are latency-bound (few
// warps on one SM: a shared-memory load takes about 29 cycles, a dependent fp64 FMA 8), so the
// operands of eight terms are loaded before the first product and two running sums are kept.  The
// strides are compile-time constants (1 or the leading dimension): the loads of a chunk are one
// base register plus immediates.  Up to 16 terms the chunks are unrolled and the loads predicated.
template <int SA, int SB, int NMAX>
FA_FN double dot(const double* a, const double* b, int n) {
  constexpr int CH = 8;
  double acc0 = 0.0, acc1 = 0.0;
  if (NMAX <= 16) {
#pragma unroll
    for (int k0 = 0; k0 < NMAX; k0 += CH) {
      double x[CH], y[CH];
#pragma unroll
      for (int u = 0; u < CH; ++u) {
        const bool ok = k0 + u < n;
        x[u] = ok ? a[(k0 + u) * SA] : 0.0; y[u] = ok ? b[(k0 + u) * SB] : 0.0;
      }
#pragma unroll
      for (int u = 0; u < CH; u += 2) { acc0 = fma(x[u], y[u], acc0); acc1 = fma(x[u + 1], y[u + 1], acc1); }
    }
  } else {
#pragma unroll 1
    for (int k0 = 0; k0 < n; k0 += CH, a += CH * SA, b += CH * SB) {
      double x[CH], y[CH];
#pragma unroll
      for (int u = 0; u < CH; ++u) {
        const bool ok = k0 + u < n;
        x[u] = ok ? a[u * SA] : 0.0; y[u] = ok ? b[u * SB] : 0.0;
      }
#pragma unroll
      for (int u = 0; u < CH; u += 2) { acc0 = fma(x[u], y[u], acc0); acc1 = fma(x[u + 1], y[u + 1], acc1); }
    }
  }
  return acc0 + acc1;
}

// sum_k w[k] * a[k * SA] * b[k * SB] over k < n (same scheme).
template <int SA, int SB, int NMAX>
FA_FN double dot_weighted(const double* w, const double* a, const double* b, int n) {
  constexpr int CH = 8;
  double acc0 = 0.0, acc1 = 0.0;
#pragma unroll 1
  for (int k0 = 0; k0 < n; k0 += CH, w += CH, a += CH * SA, b += CH * SB) {
    double x[CH], y[CH];
#pragma unroll
    for (int u = 0; u < CH; ++u) {
      const bool ok = k0 + u < n;
      x[u] = ok ? w[u] * a[u * SA] : 0.0; y[u] = ok ? b[u * SB] : 0.0;
    }
#pragma unroll
    for (int u = 0; u < CH; u += 2) { acc0 = fma(x[u], y[u], acc0); acc1 = fma(x[u + 1], y[u + 1], acc1); }
  }
  return acc0 + acc1;
}

// sum_k (a[k * ST] - b[k * ST])^2 over k in [0, n) and over k in [k0, n): squared distance of two
// columns of a coordinate matrix, and of their parts in the discarded directions.
template <int ST>
FA_FN void diff_sq(const double* a, const double* b, int k0, int n, double& all, double& tail) {
  constexpr int CH = 8;
  double s0 = 0.0, s1 = 0.0, t0 = 0.0, t1 = 0.0;
#pragma unroll 1
  for (int kb = 0; kb < n; kb += CH, a += CH * ST, b += CH * ST) {
    double v[CH];
#pragma unroll
    for (int u = 0; u < CH; ++u) v[u] = (kb + u < n) ? a[u * ST] - b[u * ST] : 0.0;
#pragma unroll
    for (int u = 0; u < CH; u += 2) {
      const double q0 = v[u] * v[u], q1 = v[u + 1] * v[u + 1];
      s0 += q0; s1 += q1;
      t0 += (kb + u >= k0) ? q0 : 0.0; t1 += (kb + u + 1 >= k0) ? q1 : 0.0;
    }
  }
  all = s0 + s1; tail = t0 + t1;
}

// C = A B for small fp64 matrices (M x K times K x N) held in shared memory, on the fp64 tensor-core
// instruction mma.m8n8k4: one warp per 8 x 8 tile of C, 256 multiply-adds per instruction with one
// element of A and one of B per lane.  With one output element per thread every multiply-add needs
// two shared-memory loads, and a 64-bit load instruction occupies the shared-memory pipe for two
// cycles whatever its addresses: a 49 x 49 x 49 product took 16,500 cycles that way and takes about
// a third of it this way (14 x 14 x 14: 690 -> below 400).
//   A_ik = A[imap(i) * SAI + k * SAK],  B_kj = B[k * SBK + jmap(j) * SBJ]  (strides are 1 or the leading
//   dimension, compile-time; imap / jmap are optional index lists, e.g. a sort order, null = identity)
//   epi(i, j, v)  : consumes C_ij; called once per element in range
//   dtn           : FastDiv by the number of column tiles, (N + 7) / 8
//   first_warp    : the tiles go to warps first_warp, first_warp + 1, ... (mod the warp count), so
//                   that two products of one phase use different warps
// Fragments are loaded without bounds checks and masked afterwards: every index they can reach
// (below the next multiple of 8 of M and N, of 16 of K) lies inside the (ld - kLdPad) x ld buffers.
// All threads of the block must call it (whole warps execute the instruction); the number of warps
// is a power of two.  The host build runs the plain triple loop.
#ifndef FA_IRLS_HOST
__device__ __forceinline__ void fa_dmma(double& d0, double& d1, double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(d0), "+d"(d1) : "d"(a), "d"(b));
}
#endif

template <int SAI, int SAK, int SBK, int SBJ, class EP>
FA_FN void matmul(const Ctx& c, int M, int N, int K, const FastDiv& dtn, const double* A, const double* B, EP epi,
                  int first_warp = 0, const int* imap = nullptr, const int* jmap = nullptr) {
#ifndef FA_IRLS_HOST
  const int lane = c.tid & 31, nwarp = c.nt >> 5;
  const int warp = ((c.tid >> 5) - first_warp) & (nwarp - 1);
  const int tn = (N + 7) >> 3, tiles = ((M + 7) >> 3) * tn;
  const int fr = lane >> 2, fk = lane & 3;          // fragment coordinates: A (row fr, k fk), B (k fk, column fr)
#pragma unroll 1
  for (int t = warp; t < tiles; t += nwarp) {
    const int ti = fast_div(t, dtn);
    const int i0 = ti * 8, j0 = (t - ti * tn) * 8;
    const int i = i0 + fr, j = j0 + fr;
    const bool iok = i < M, jok = j < N;
    const int ia = imap ? imap[iok ? i : 0] : i, jb = jmap ? jmap[jok ? j : 0] : j;
    const double* ap = A + ia * SAI + fk * SAK;
    const double* bp = B + fk * SBK + jb * SBJ;
    double d0 = 0.0, d1 = 0.0, e0 = 0.0, e1 = 0.0;  // two chains of dependent instructions, added at the end
#pragma unroll 1
    for (int k0 = 0; k0 < K; k0 += 16, ap += 16 * SAK, bp += 16 * SBK) {
      double a[4], b[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { a[u] = ap[4 * u * SAK]; b[u] = bp[4 * u * SBK]; }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const bool kok = k0 + 4 * u + fk < K;
        a[u] = (iok && kok) ? a[u] : 0.0;
        b[u] = (jok && kok) ? b[u] : 0.0;
      }
      fa_dmma(d0, d1, a[0], b[0]);
      fa_dmma(e0, e1, a[1], b[1]);
      if (k0 + 8 < K) {                              // uniform in the warp
        fa_dmma(d0, d1, a[2], b[2]);
        fa_dmma(e0, e1, a[3], b[3]);
      }
    }
    const int jc = j0 + 2 * fk;
    if (iok) {
      if (jc < N) epi(i, jc, d0 + e0);
      if (jc + 1 < N) epi(i, jc + 1, d1 + e1);
    }
  }
#else
  (void)first_warp; (void)dtn;
#pragma unroll 1
  for (int idx = c.tid; idx < M * N; idx += c.nt) {
    const int i = idx / N, j = idx - i * N;
    const int ia = imap ? imap[i] : i, jb = jmap ? jmap[j] : j;
    double acc = 0.0;
    for (int k = 0; k < K; ++k) acc += A[ia * SAI + k * SAK] * B[k * SBK + jb * SBJ];
    epi(i, j, acc);
  }
#endif
}

// The q-th pair (i, j), i <= j, in the order (0,0) (0,1) (1,1) (0,2) (1,2) (2,2) ...: q = j (j + 1) / 2 + i.
// The numbering does not depend on the matrix size.
FA_FN void tri_pair(int q, int& i, int& j) {
  int jj = (int)((sqrtf(8.0f * (float)q + 1.0f) - 1.0f) * 0.5f);   // within one of the answer; fixed up below
  while (jj * (jj + 1) / 2 > q) --jj;
  while ((jj + 1) * (jj + 2) / 2 <= q) ++jj;
  j = jj; i = q - jj * (jj + 1) / 2;
}

#ifndef FA_IRLS_HOST
// 1 / x for normal x: hardware approximation and two Newton steps (relative error ~1e-15 at best;
// it scales corrections that are themselves iterated on).
__device__ __forceinline__ double fa_fast_rcp(double x) {
  double y;
  asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
  y = fma(y, fma(-x, y, 1.0), y);
  y = fma(y, fma(-x, y, 1.0), y);
  return y;
}
#define FA_RCP(x) fa_fast_rcp(x)
#else
#define FA_RCP(x) (1.0 / (x))
#endif

// Rotation (cs, sn) for a pair with diagonal entries app, aqq and off-diagonal entry apq; identity
// for entries at rounding level.  From the double angle, without division:
//   d = a_qq - a_pp, h = 2 a_pq, cos 2phi = |d| / sqrt(d^2 + h^2),
//   c = sqrt((1 + cos 2phi) / 2), s = sign(d) * h / (2 c sqrt(d^2 + h^2)).
// The reciprocal square roots start from the hardware approximation (22 bits).  The first gets one
// Newton step (44 bits): it alone fixes the angle, s / c = hr / x, and an angle that is off by
// 1e-13 relative leaves 1e-13 of the entry it was meant to annihilate.  The second only scales c
// and s together, and a Jacobi rotation has to be ORTHOGONAL to full accuracy for the similarity
// transform to be exact; so (c, s) is scaled onto the unit circle at the end:
// c^2 + s^2 = 1 + e with |e| ~ 1e-6, factor 1 - e/2 + 3 e^2 / 8, error e^3.  This keeps the chain of
// dependent fp64 operations (8 cycles each, the unit of cost in this kernel) short; there is no
// branch, so two rotations worked out by one thread overlap.
// Returns true when the entry was "large" (above kJacobiBig relative to its diagonal).
FA_FN bool rotation_of(double app, double aqq, double apq, double& cs, double& sn) {
  const double m2 = apq * apq, ref2 = fabs(app * aqq);
  const bool ok = (m2 > (kJacobiTol * kJacobiTol) * ref2) && (m2 > 1e-280);
  const double d = aqq - app, h = 2.0 * apq;
  const double q = fma(d, d, h * h);
  const double qs = ok ? q : 1.0;
  double rinv = FA_RSQRT_APPROX(qs);
  rinv = rinv * fma((-0.5 * qs) * rinv, rinv, 1.5);      // one Newton step: the angle (s / c = hr / x) depends on rinv only
  const double hr = (0.5 * h) * rinv;
  const double x = fma(0.5 * fabs(d), rinv, 0.5);        // cos^2 phi, in [1/2, 1]
  const double cinv = FA_RSQRT_APPROX(x);
  double c = x * cinv, sv = hr * cinv;
  const double e = fma(c, c, fma(sv, sv, -1.0));
  const double f = fma(e, fma(e, 0.375, -0.5), 1.0);
  c *= f;
  sv *= f;
  cs = ok ? c : 1.0;
  sn = ok ? (d < 0.0 ? -sv : sv) : 0.0;
  return ok && (m2 > (kJacobiBig * kJacobiBig) * ref2);
}

// The same rotation in fp32, for sweeps whose only job is to bring T close enough to diagonal form for
// the fp64 refinement to take over (which also repairs the orthogonality the fp32 products lose): the
// chain of dependent operations is less than half as long (fp32 FMA 4 cycles, hardware rsqrt).
// Entries are expected scaled to order one.
FA_FN bool rotation_of(float app, float aqq, float apq, float& cs, float& sn) {
  constexpr float kTol = 3e-8f, kBig = 1e-3f;
  const float m2 = apq * apq, ref2 = fabsf(app * aqq);
  const bool ok = (m2 > (kTol * kTol) * ref2) && (m2 > 1e-30f);
  const float d = aqq - app, h = 2.0f * apq;
  const float q = fmaf(d, d, h * h);
  const float qs = ok ? q : 1.0f;
#ifndef FA_IRLS_HOST
  const float rinv = rsqrtf(qs);
#else
  const float rinv = 1.0f / sqrtf(qs);
#endif
  const float hr = (0.5f * h) * rinv;
  const float x = fmaf(0.5f * fabsf(d), rinv, 0.5f);           // cos^2 phi, in [1/2, 1]
#ifndef FA_IRLS_HOST
  const float cinv = rsqrtf(x);
#else
  const float cinv = 1.0f / sqrtf(x);
#endif
  float c = x * cinv, sv = hr * cinv;
  const float e = fmaf(c, c, fmaf(sv, sv, -1.0f));
  const float f = fmaf(e, -0.5f, 1.0f);
  c *= f;
  sv *= f;
  cs = ok ? c : 1.0f;
  sn = ok ? (d < 0.0f ? -sv : sv) : 0.0f;
  return ok && (m2 > (kBig * kBig) * ref2);
}

// Systolic (Brent-Luk) arrangement of np pairs: pair k sits at positions (k, np + k) -- "top" entries
// in the first half, "bottom" entries in the second, so that threads with consecutive pair numbers
// touch consecutive shared-memory words.  After a round top_0 stays, the other top entries move one
// pair up, the bottom entries one pair down, and the two ends cross over (bottom_0 -> top_1,
// top_{np-1} -> bottom_{np-1}).  pp - 1 rounds pair every two indices exactly once and bring every
// index back to where it started.  Returns where the content of position x goes.
FA_FN int systolic_next(int x, int np) {
  if (x == 0) return 0;
  if (x < np) return x == np - 1 ? 2 * np - 1 : x + 1;      // top_k, k >= 1
  return x == np ? (np > 1 ? 1 : np) : x - 1;                // bottom_k
}

// Cyclic Jacobi, all pairs of a round in parallel.  T (dim x dim, symmetric, both halves stored, rows
// and columns dim..pp-1 zero) is driven towards diagonal form; J accumulates the rotations (J <- J * R).
// A pair is rotated whenever its off-diagonal entry is above rounding level.  At most `max_sweeps`
// sweeps are made; sweeping also stops after the first sweep in which no rotated entry exceeded
// kJacobiBig relative to its diagonal: that sweep's rotations leave entries of the order of its
// square (quadratic convergence of the cyclic method), i.e. below rounding level.  *big_out tells
// whether the last sweep made still saw such an entry (T is then not yet diagonal).
//
// The data MOVES instead of the pairing (Brent-Luk systolic arrangement): a round rotates the pairs
// at the fixed positions (k, np + k) and stores rows and columns (and the columns of J) at their
// systolic_next() positions, from T / J into Talt / Jalt and back.  So every thread owns the same
// 2x2 blocks of T and (row, pair) items of J for the whole solve, all its offsets are worked out
// once before the first sweep, and all its loads go out together at the top of a round -- what a
// round costs here is the number of dependent instructions a warp has to issue.
//   * up to 8 pairs (dim <= 16): one item per thread; each lane works out the rotation of its
//     column pair itself and gets the one of its row pair from another lane of its warp by a
//     shuffle: one barrier per round and nothing else between threads;
//   * more pairs (jacobi_large): several items per thread; every warp works out all rotations
//     (lane q: pair q) and the items fetch theirs by shuffles -- still one barrier per round; or
//     (kOnce, used up to 16 pairs in fp64) the first warp alone works them out and a second barrier
//     publishes them: sixteen warps repeating the fp64 divisions and square roots kept the fp64
//     pipe busier than the extra barrier costs.
// A full sweep (pp - 1 rounds) returns every index to its own position, and sweeps are never cut
// short.  On return *Tio / *Jio point at the buffers that hold the results.  Returns the sweeps made.
// Up to 8 pairs on the device; any size on the host.
template <int LD, typename R>
FA_FN int jacobi_small(const Ctx& c, const Smem& s, R** Tio, R** Taltio, R** Jio, R** Jaltio,
                       int dim, int jrows, int max_sweeps, int* big_out) {
  constexpr int ld = LD;
  const int pp = (dim + 1) & ~1;
  const int np = pp >> 1;
  R* T = *Tio;
  R* Tn = *Taltio;
  R* J = *Jio;
  R* Jn = *Jaltio;
  const int nb2 = np * np, total2 = nb2 + jrows * np;
  // the item this thread owns for the whole solve (element offsets into T / J)
  struct Item { int kind, diag, ksrc, kaa, kbb, kab, laa, lbb, lab, x0, x1, x2, x3, z0, z1, z2, z3; } it;
  it.kind = 0; it.ksrc = -1; it.laa = it.lbb = it.lab = 0;
  {
    const int idx = c.tid;
    if (idx < nb2) {
      const int k = idx / np, l = idx - k * np;
      const int a = k, b = np + k, cc = l, d = np + l;
      const int pa = systolic_next(a, np), pb = systolic_next(b, np), pc = systolic_next(cc, np), pd = systolic_next(d, np);
      it.kind = 1; it.diag = (k == l);
      it.kaa = a * ld + a; it.kbb = b * ld + b; it.kab = a * ld + b;
      it.laa = cc * ld + cc; it.lbb = d * ld + d; it.lab = cc * ld + d;
      it.x0 = a * ld + cc; it.x1 = a * ld + d; it.x2 = b * ld + cc; it.x3 = b * ld + d;
      it.z0 = pa * ld + pc; it.z1 = pa * ld + pd; it.z2 = pb * ld + pc; it.z3 = pb * ld + pd;
#ifndef FA_IRLS_HOST
      // a lane of this warp whose own (column) pair is k hands over the row rotation: the item with
      // number o has column pair o mod np (nb2 is a multiple of np), so the first such lane is
      const int w0 = idx & ~31;
      const int j = (k - w0 % np + np) % np;
      if (j < 32 && w0 + j < total2) it.ksrc = j;
#endif
    } else if (idx < total2) {
      const int q = idx - nb2;
      const int x = q / np, l = q - x * np;
      const int cc = l, d = np + l;
      it.kind = 2; it.diag = 0;
      it.laa = cc * ld + cc; it.lbb = d * ld + d; it.lab = cc * ld + d;
      it.x0 = x * ld + cc; it.x1 = x * ld + d;
      it.z0 = x * ld + systolic_next(cc, np); it.z1 = x * ld + systolic_next(d, np);
      it.kaa = it.kbb = it.kab = it.x2 = it.x3 = it.z2 = it.z3 = 0;
    }
  }
  int sweep = 0, again = 0;
  // "large rotation in this sweep" flag, double-buffered by sweep parity (slots 0 and 3)
  if (c.tid == 0) { s.flags[0] = 0; s.flags[3] = 0; }
  c.sync();
  for (; sweep < max_sweeps; ++sweep) {
    int* big = &s.flags[(sweep & 1) ? 3 : 0];
    if (c.tid == 0) s.flags[(sweep & 1) ? 0 : 3] = 0;
    for (int rd = 0; rd < pp - 1; ++rd) {
#ifndef FA_IRLS_HOST
      {
        // every lane with an item works out the rotation of its column pair l; a block of T gets
        // its row rotation from the lane `ksrc` of its warp (worked out here only if there is none)
        R cl = 1.0, sl = 0.0;
        bool bigl = false;
        R xac = 0.0, xad = 0.0, xbc = 0.0, xbd = 0.0;
        if (it.kind != 0) {
          const R laa = T[it.laa], lbb = T[it.lbb], lab = T[it.lab];
          if (it.kind == 1) { xac = T[it.x0]; xad = T[it.x1]; xbc = T[it.x2]; xbd = T[it.x3]; }
          else { xac = J[it.x0]; xad = J[it.x1]; }
          bigl = rotation_of(laa, lbb, lab, cl, sl);
        }
        const int src = it.ksrc < 0 ? 0 : it.ksrc;
        R ck = __shfl_sync(0xffffffffu, cl, src), sk = __shfl_sync(0xffffffffu, sl, src);
        if (it.kind == 1) {
          if (it.ksrc < 0) (void)rotation_of(T[it.kaa], T[it.kbb], T[it.kab], ck, sk);
          if (it.diag && bigl) *big = 1;
          const R yac = ck * xac - sk * xbc, yad = ck * xad - sk * xbd;
          const R ybc = sk * xac + ck * xbc, ybd = sk * xad + ck * xbd;
          Tn[it.z0] = cl * yac - sl * yad; Tn[it.z1] = sl * yac + cl * yad;
          Tn[it.z2] = cl * ybc - sl * ybd; Tn[it.z3] = sl * ybc + cl * ybd;
        } else if (it.kind == 2) {
          Jn[it.z0] = cl * xac - sl * xad;
          Jn[it.z1] = sl * xac + cl * xad;
        }
      }
#else
      if (it.kind == 1) {
        const R kaa = T[it.kaa], kbb = T[it.kbb], kab = T[it.kab];
        const R laa = T[it.laa], lbb = T[it.lbb], lab = T[it.lab];
        const R xac = T[it.x0], xad = T[it.x1], xbc = T[it.x2], xbd = T[it.x3];
        R ck, sk, cl, sl;
        const bool bigk = rotation_of(kaa, kbb, kab, ck, sk);
        (void)rotation_of(laa, lbb, lab, cl, sl);
        if (it.diag && bigk) *big = 1;
        const R yac = ck * xac - sk * xbc, yad = ck * xad - sk * xbd;
        const R ybc = sk * xac + ck * xbc, ybd = sk * xad + ck * xbd;
        Tn[it.z0] = cl * yac - sl * yad; Tn[it.z1] = sl * yac + cl * yad;
        Tn[it.z2] = cl * ybc - sl * ybd; Tn[it.z3] = sl * ybc + cl * ybd;
      } else if (it.kind == 2) {
        const R laa = T[it.laa], lbb = T[it.lbb], lab = T[it.lab];
        const R va = J[it.x0], vb = J[it.x1];
        R cl, sl;
        (void)rotation_of(laa, lbb, lab, cl, sl);
        Jn[it.z0] = cl * va - sl * vb;
        Jn[it.z1] = sl * va + cl * vb;
      }
#endif
      // further items (fewer threads than items): offsets on the fly
#pragma unroll 1
      for (int idx = c.tid + c.nt; idx < total2; idx += c.nt) {
        if (idx < nb2) {
          const int k = idx / np, l = idx - k * np;
          const int a = k, b = np + k, cc = l, d = np + l;
          const R kaa = T[a * ld + a], kbb = T[b * ld + b], kab = T[a * ld + b];
          const R laa = T[cc * ld + cc], lbb = T[d * ld + d], lab = T[cc * ld + d];
          const R xac = T[a * ld + cc], xad = T[a * ld + d], xbc = T[b * ld + cc], xbd = T[b * ld + d];
          R ck, sk, cl, sl;
          const bool bigk = rotation_of(kaa, kbb, kab, ck, sk);
          (void)rotation_of(laa, lbb, lab, cl, sl);
          if (k == l && bigk) *big = 1;
          const R yac = ck * xac - sk * xbc, yad = ck * xad - sk * xbd;
          const R ybc = sk * xac + ck * xbc, ybd = sk * xad + ck * xbd;
          const int pa = systolic_next(a, np), pb = systolic_next(b, np);
          const int pc = systolic_next(cc, np), pd = systolic_next(d, np);
          Tn[pa * ld + pc] = cl * yac - sl * yad; Tn[pa * ld + pd] = sl * yac + cl * yad;
          Tn[pb * ld + pc] = cl * ybc - sl * ybd; Tn[pb * ld + pd] = sl * ybc + cl * ybd;
        } else {
          const int q = idx - nb2;
          const int x = q / np, l = q - x * np;
          const int cc = l, d = np + l;
          const R laa = T[cc * ld + cc], lbb = T[d * ld + d], lab = T[cc * ld + d];
          const R va = J[x * ld + cc], vb = J[x * ld + d];
          R cl, sl;
          (void)rotation_of(laa, lbb, lab, cl, sl);
          Jn[x * ld + systolic_next(cc, np)] = cl * va - sl * vb;
          Jn[x * ld + systolic_next(d, np)] = sl * va + cl * vb;
        }
      }
      c.sync();
      { R* t = T; T = Tn; Tn = t; }
      { R* t = J; J = Jn; Jn = t; }
    }
    again = *big;
    c.sync();
    if (!again) { ++sweep; break; }
  }
  *Tio = T; *Taltio = Tn; *Jio = J; *Jaltio = Jn;
  *big_out = again;
  return sweep;
}

#ifndef FA_IRLS_HOST
// More than 8 pairs, at most 32 (device only).  This thread's items are tid + u * nt: 2x2 blocks of T (kMT of
// them) and (row, pair) items of J (kMJ).  Per item: the offset of its first element, the offsets
// its results are stored at, and the pairs whose rotations it needs; offsets are below 2^16
// (matrices of at most 64 x 65 doubles) and are kept two to a register.
template <int LD, int kMT, int kMJ, typename R, bool kOnce = false>
FA_FN int jacobi_large(const Ctx& c, const Smem& s, R** Tio, R** Taltio, R** Jio, R** Jaltio,
                       int dim, int jrows, int max_sweeps, int* big_out) {
  constexpr int ld = LD;
  const int pp = (dim + 1) & ~1;
  const int np = pp >> 1;
  R* T = *Tio;
  R* Tn = *Taltio;
  R* J = *Jio;
  R* Jn = *Jaltio;
  unsigned tdesc0[kMT], tdesc1[kMT], tdesc2[kMT], jdesc0[kMJ], jdesc1[kMJ];
  bool tv[kMT], jv[kMJ];
#pragma unroll
  for (int u = 0; u < kMT; ++u) {
    const int idx = c.tid + u * c.nt;
    tv[u] = idx < np * np;
    const int k = tv[u] ? idx / np : 0, l = tv[u] ? idx - k * np : 0;
    const int pa = systolic_next(k, np) * ld, pb = systolic_next(np + k, np) * ld;
    const int pc = systolic_next(l, np), pd = systolic_next(np + l, np);
    tdesc0[u] = (unsigned)(k * ld + l) | ((unsigned)k << 16) | ((unsigned)l << 24);
    tdesc1[u] = (unsigned)(pa + pc) | ((unsigned)(pa + pd) << 16);
    tdesc2[u] = (unsigned)(pb + pc) | ((unsigned)(pb + pd) << 16);
  }
#pragma unroll
  for (int u = 0; u < kMJ; ++u) {
    const int idx = c.tid + u * c.nt;
    jv[u] = idx < jrows * np;
    const int x = jv[u] ? idx / np : 0, l = jv[u] ? idx - x * np : 0;
    jdesc0[u] = (unsigned)(x * ld + l) | ((unsigned)l << 16);
    jdesc1[u] = (unsigned)(x * ld + systolic_next(l, np)) | ((unsigned)(x * ld + systolic_next(np + l, np)) << 16);
  }
  int sweep = 0, again = 0;
  if (c.tid == 0) { s.flags[0] = 0; s.flags[3] = 0; }
  c.sync();
  for (; sweep < max_sweeps; ++sweep) {
    int* big = &s.flags[(sweep & 1) ? 3 : 0];
    if (c.tid == 0) s.flags[(sweep & 1) ? 0 : 3] = 0;
    for (int rd = 0; rd < pp - 1; ++rd) {
      // every warp works out all np <= 32 rotations itself, lane q the one of pair q; the items then
      // fetch the two (one) they need with shuffles: no second barrier, no waiting for one warp
      const int lane = c.tid & 31;
      R x0[kMT], x1[kMT], x2[kMT], x3[kMT], v0[kMJ], v1[kMJ];
#pragma unroll
      for (int u = 0; u < kMT; ++u) {
        if (tv[u]) {
          const int tb = tdesc0[u] & 0xffffu;
          x0[u] = T[tb]; x1[u] = T[tb + np]; x2[u] = T[tb + np * ld]; x3[u] = T[tb + np * ld + np];
        }
      }
#pragma unroll
      for (int u = 0; u < kMJ; ++u) {
        if (jv[u]) { const int jb = jdesc0[u] & 0xffffu; v0[u] = J[jb]; v1[u] = J[jb + np]; }
      }
      R cq = 1.0, sq = 0.0;
      if (kOnce) {
        // the first warp alone works out the rotations and leaves them in shared memory: a second barrier,
        // but the other warps' arithmetic pipes stay free of fifteen more copies of the same work
        if (c.tid < np) {
          const int o = c.tid * (ld + 1);
          if (rotation_of(T[o], T[o + np * (ld + 1)], T[o + np], cq, sq)) *big = 1;
          s.rc[c.tid] = (double)cq; s.rs[c.tid] = (double)sq;
        }
        c.sync();
      } else if (lane < np) {
        const int o = lane * (ld + 1);
        if (rotation_of(T[o], T[o + np * (ld + 1)], T[o + np], cq, sq) && c.tid < np) *big = 1;
      }
#pragma unroll
      for (int u = 0; u < kMT; ++u) {
        const int tk = (tdesc0[u] >> 16) & 0xffu, tl = tdesc0[u] >> 24;
        R ck, sk, cl, sl;
        if (kOnce) { ck = (R)s.rc[tk]; sk = (R)s.rs[tk]; cl = (R)s.rc[tl]; sl = (R)s.rs[tl]; }
        else {
          ck = __shfl_sync(0xffffffffu, cq, tk); sk = __shfl_sync(0xffffffffu, sq, tk);
          cl = __shfl_sync(0xffffffffu, cq, tl); sl = __shfl_sync(0xffffffffu, sq, tl);
        }
        if (tv[u]) {
          const R yac = ck * x0[u] - sk * x2[u], yad = ck * x1[u] - sk * x3[u];
          const R ybc = sk * x0[u] + ck * x2[u], ybd = sk * x1[u] + ck * x3[u];
          Tn[tdesc1[u] & 0xffffu] = cl * yac - sl * yad; Tn[tdesc1[u] >> 16] = sl * yac + cl * yad;
          Tn[tdesc2[u] & 0xffffu] = cl * ybc - sl * ybd; Tn[tdesc2[u] >> 16] = sl * ybc + cl * ybd;
        }
      }
#pragma unroll
      for (int u = 0; u < kMJ; ++u) {
        const int jl = jdesc0[u] >> 16;
        R cl, sl;
        if (kOnce) { cl = (R)s.rc[jl]; sl = (R)s.rs[jl]; }
        else { cl = __shfl_sync(0xffffffffu, cq, jl); sl = __shfl_sync(0xffffffffu, sq, jl); }
        if (jv[u]) {
          Jn[jdesc1[u] & 0xffffu] = cl * v0[u] - sl * v1[u];
          Jn[jdesc1[u] >> 16] = sl * v0[u] + cl * v1[u];
        }
      }
      if (!kOnce && lane < np) { s.rc[lane] = (double)cq; s.rs[lane] = (double)sq; }     // same values from every warp: for the loops below
      // items beyond the per-thread lists (a smaller block than expected): offsets on the fly
      if (!kOnce && (kMT * c.nt < np * np || kMJ * c.nt < jrows * np)) c.sync();
#pragma unroll 1
      for (int idx = c.tid + kMT * c.nt; idx < np * np; idx += c.nt) {
        const int k = idx / np, l = idx - k * np;
        const int a = k, b = np + k, cc = l, d = np + l;
        const R ck = (R)s.rc[k], sk = (R)s.rs[k], cl = (R)s.rc[l], sl = (R)s.rs[l];
        const R xac = T[a * ld + cc], xad = T[a * ld + d], xbc = T[b * ld + cc], xbd = T[b * ld + d];
        const R yac = ck * xac - sk * xbc, yad = ck * xad - sk * xbd;
        const R ybc = sk * xac + ck * xbc, ybd = sk * xad + ck * xbd;
        const int pa = systolic_next(a, np), pb = systolic_next(b, np);
        const int pc = systolic_next(cc, np), pd = systolic_next(d, np);
        Tn[pa * ld + pc] = cl * yac - sl * yad; Tn[pa * ld + pd] = sl * yac + cl * yad;
        Tn[pb * ld + pc] = cl * ybc - sl * ybd; Tn[pb * ld + pd] = sl * ybc + cl * ybd;
      }
#pragma unroll 1
      for (int idx = c.tid + kMJ * c.nt; idx < jrows * np; idx += c.nt) {
        const int x = idx / np, l = idx - x * np;
        const int cc = l, d = np + l;
        const R cl = (R)s.rc[l], sl = (R)s.rs[l];
        const R va = J[x * ld + cc], vb = J[x * ld + d];
        Jn[x * ld + systolic_next(cc, np)] = cl * va - sl * vb;
        Jn[x * ld + systolic_next(d, np)] = sl * va + cl * vb;
      }
      c.sync();
      { R* t = T; T = Tn; Tn = t; }
      { R* t = J; J = Jn; Jn = t; }
    }
    again = *big;
    c.sync();
    if (!again) { ++sweep; break; }
  }
  *Tio = T; *Taltio = Tn; *Jio = J; *Jaltio = Jn;
  *big_out = again;
  return sweep;
}
#endif

template <int LD, typename R>
FA_FN int jacobi(const Ctx& c, const Smem& s, R** Tio, R** Taltio, R** Jio, R** Jaltio, int dim,
                 int jrows, int max_sweeps, int* big_out) {
  *big_out = 0;
  if (dim < 2) return 0;
#ifndef FA_IRLS_HOST
  // item slots per thread are compile-time (slots without an item still cost their instructions):
  // one of each up to 16 pairs with 512 threads, two blocks and three or four J items up to 32 pairs
  const int np = (dim + 1) >> 1;
  if constexpr (LD > 20) {
    // Only the variants a kernel needs are compiled into it -- every further one costs it registers (the
    // 512-thread kernels have 128 each: with all variants inlined the p = 31 call was 10 % slower).  So
    // the kernels for more than 16 gradients run every size, a small rank included, through jacobi_large.
    // Up to 32 gradients (512 threads) one item of each kind always suffices.  Above, the fp32 sweeps
    // (the ones that normally run) come with three or four J items; the fp64 fallback with four.
    if constexpr (LD <= 36) {
      return jacobi_large<LD, 1, 1, R, true>(c, s, Tio, Taltio, Jio, Jaltio, dim, jrows, max_sweeps, big_out);
    } else if constexpr (sizeof(R) == 4) {
      if (np * np <= 2 * c.nt && jrows * np <= 3 * c.nt)    // e.g. 49 indices after 15 identical gradients of 63
        return jacobi_large<LD, 2, 3, R>(c, s, Tio, Taltio, Jio, Jaltio, dim, jrows, max_sweeps, big_out);
      return jacobi_large<LD, 2, 4, R>(c, s, Tio, Taltio, Jio, Jaltio, dim, jrows, max_sweeps, big_out);
    } else {
      return jacobi_large<LD, 2, 4, R>(c, s, Tio, Taltio, Jio, Jaltio, dim, jrows, max_sweeps, big_out);
    }
  } else {
    return jacobi_small<LD, R>(c, s, Tio, Taltio, Jio, Jaltio, dim, jrows, max_sweeps, big_out);
  }
#else
  return jacobi_small<LD, R>(c, s, Tio, Taltio, Jio, Jaltio, dim, jrows, max_sweeps, big_out);
#endif
}

// Refinement of approximate eigenvectors by matrix products (the iterative refinement for the
// symmetric eigenvalue decomposition of Ogita and Aishima, Japan J. Indust. Appl. Math. 35 (2018)):
// for X (r x r, nearly orthogonal) with X^T T X nearly diagonal,
//     Rm = I - X^T X,  S = X^T T X,  lam_i = S_ii / (1 - Rm_ii),
//     E_ij = (S_ij + lam_j Rm_ij) / (lam_j - lam_i)  (i != j),  E_ii = Rm_ii / 2,   X <- X + X E
// squares the distance of X from the exact orthogonal eigenvector matrix.  A step is four r x r
// products (length-r dot products, independent of each other) against 2 (r - 1) dependent rotation
// rounds for a Jacobi sweep.  It only converges from close by: |E_ij| must be well below one, which
// near-equal eigenvalues with a sizeable coupling entry violate -- those stay with the Jacobi sweeps.
//
// Starts from X = I, i.e. in the basis T is given in -- the first step then needs no products
// (S = T, Rm = 0) -- or, with from_x, from the matrix in s.J (the eigenvectors the fp32 sweeps found).
// Returns 1 with X in s.J and the eigenvalue estimates on the diagonal of T when the corrections
// went below kRefineStop; 0 (T untouched but for nothing) when the first corrections are above
// the reach (RefineLimits), the steps stop contracting or kMaxRefine steps are not enough.  Uses s.J, s.tmp and
// s.M as scratch (pointers may come back swapped).
template <int LD>
FA_FN int refine_eig(const Ctx& c, Smem& s, int r, bool from_x = false) {
  constexpr int ld = LD;
  const double* T = s.T;
  double* X = s.J;       // current eigenvector estimate
  double* E = s.tmp;     // T X, then the correction E
  double* SR = s.M;      // S on and above the diagonal, Rm below it; becomes the next X
  constexpr double kRefineTheta = RefineLimits<LD>::theta, kRefineContract = RefineLimits<LD>::contract;
  double part = 0.0, emax = kRefineTheta / kRefineContract;   // from_x: the first full step must come out below kRefineTheta
  int steps = 0;
  if (!from_x) {
    // ---- first step from X = I
#pragma unroll 1
    for (int idx = c.tid; idx < r * r; idx += c.nt) {
      const int i = fast_div(idx, s.div_r), j = idx - i * r;
      double e = 0.0;
      if (i != j) {
        const double tij = T[i * ld + j], tii = T[i * ld + i], tjj = T[j * ld + j];
        if (tij * tij > (kJacobiTol * kJacobiTol) * fabs(tii * tjj) && tij * tij > 1e-280) {
          e = tij * FA_RCP(tjj - tii);                 // equal diagonal entries: Inf, refused below
          part = fmax(part, fabs(e) <= 1.7e308 ? fabs(e) : 1.7e308);
        }
      }
      X[i * ld + j] = (i == j) ? 1.0 : e;
    }
    emax = block_max(c, s, part);                      // its barrier also publishes X
    if (!(emax <= kRefineTheta)) return 0;
#pragma unroll 1
    for (int k = c.tid; k < r; k += c.nt) s.lam[k] = T[k * ld + k];
    steps = 1;
  }
  // V = T X.  Up to 32 gradients it has buffers of its own and is carried along (T (X + X E) = V + V E: the
  // product by E that updates X updates V in the same phase, on other warps); above, there is no room
  // and it is formed afresh in every step, in E's buffer.
  double* V = s.V0;
  double* Vn = s.V1;
  constexpr bool carry = LD <= 36;               // (= the kernels whose shared memory holds V0 and V1)
  if (carry && emax >= kRefineStop) {
    matmul<LD, 1, LD, 1>(c, r, r, r, s.div_tr, T, X, [&](int i, int j, double v) { V[i * ld + j] = v; });
    c.sync();
  }
  while (emax >= kRefineStop) {
    if (steps > kMaxRefine) return 0;
    const double prev = emax;
    if (!carry) {
      V = E;
      matmul<LD, 1, LD, 1>(c, r, r, r, s.div_tr, T, X, [&](int i, int j, double v) { V[i * ld + j] = v; });
      c.sync();
    }
    // ---- S = X^T (T X) on and above the diagonal, Rm = I - X^T X below it (its diagonal -> rdiag)
    matmul<1, LD, LD, 1>(c, r, r, r, s.div_tr, X, V, [&](int i, int j, double v) { if (i <= j) SR[i * ld + j] = v; });
    matmul<1, LD, LD, 1>(c, r, r, r, s.div_tr, X, X,
                         [&](int i, int j, double v) { if (i == j) s.rdiag[i] = 1.0 - v; else if (i > j) SR[i * ld + j] = -v; },
                         ((r + 7) >> 3) * ((r + 7) >> 3));
    c.sync();
    // ---- the correction.  lam_i = S_ii / (1 - Rm_ii) with the quotient expanded to second order:
    // Rm_ii is of the order of the last correction squared.
    part = 0.0;
#pragma unroll 1
    for (int idx = c.tid; idx < r * r; idx += c.nt) {
      const int i = fast_div(idx, s.div_r), j = idx - i * r;
      const double rii = s.rdiag[i];
      const double li = SR[i * ld + i] * fma(rii, 1.0 + rii, 1.0);
      double e;
      if (i == j) { e = 0.5 * rii; s.lam[i] = li; }
      else {
        const double rjj = s.rdiag[j];
        const double lj = SR[j * ld + j] * fma(rjj, 1.0 + rjj, 1.0);
        const double sij = (i < j) ? SR[i * ld + j] : SR[j * ld + i];
        const double rij = (i < j) ? SR[j * ld + i] : SR[i * ld + j];
        const double num = fma(lj, rij, sij);
        if (num * num > (kJacobiTol * kJacobiTol) * fabs(li * lj) && num * num > 1e-280) {
          e = num * FA_RCP(lj - li);
          part = fmax(part, fabs(e) <= 1.7e308 ? fabs(e) : 1.7e308);
        } else {
          e = 0.5 * rij;                             // nothing to rotate: keep the pair orthogonal
        }
      }
      E[i * ld + j] = e;
    }
    emax = block_max(c, s, part);                    // its barrier: every thread is done with SR, E is published
    if (!(emax <= kRefineContract * prev) && emax > 1e-12) return 0;
    // ---- X <- X + X E  (into SR's buffer, which then changes roles with X's), and V <- V + V E
    matmul<LD, 1, LD, 1>(c, r, r, r, s.div_tr, X, E, [&](int i, int j, double v) { SR[i * ld + j] = X[i * ld + j] + v; });
    if (carry && emax >= kRefineStop)          // (the last step's V would not be used)
      matmul<LD, 1, LD, 1>(c, r, r, r, s.div_tr, V, E, [&](int i, int j, double v) { Vn[i * ld + j] = V[i * ld + j] + v; },
                           ((r + 7) >> 3) * ((r + 7) >> 3));
    c.sync();
    if (carry) { double* t = V; V = Vn; Vn = t; }
    { double* t = X; X = SR; SR = t; }
    ++steps;
  }
  c.sync();
#pragma unroll 1
  for (int k = c.tid; k < r; k += c.nt) s.T[k * ld + k] = s.lam[k];
  s.J = X; s.M = SR;
  s.count_refinements += steps;
  c.sync();
  return 1;
}

// Jacobi sweeps in fp32 on a copy of T (scaled to order one), for a round whose T is too far from
// diagonal form for the refinement: sweeps until every |T_ij| is below half of the refinement's reach times
// |T_jj - T_ii| in the swept copy (or the sweeps have converged as far as fp32 goes), then the
// accumulated rotations are widened into s.J as the refinement's starting point.  A rotation round
// costs about a third of the fp64 one when the block is latency-bound (up to 16 indices) and about
// half when it is bound by shared-memory traffic (64 indices); what fp32 loses -- eigenvectors good
// to 1e-6, orthogonal to 1e-6 -- the refinement restores in two of its steps.  s.T is only read.
// The fp32 matrices live in s.tmp (T and its alternate) and s.M (J and its alternate).
template <int LD>
FA_FN void sweeps_fp32(const Ctx& c, Smem& s, int r) {
  constexpr int ld = LD;
  const int ppr = (r + 1) & ~1;
  float* Tf = reinterpret_cast<float*>(s.tmp);
  float* Ta = Tf + (LD - kLdPad) * LD;
  float* Jf = reinterpret_cast<float*>(s.M);
  float* Ja = Jf + (LD - kLdPad) * LD;
  double part = 0.0;
#pragma unroll 1
  for (int k = c.tid; k < r; k += c.nt) part = fmax(part, fmin(fabs(s.T[k * ld + k]), 1.7e308));
  const double dmax = block_max(c, s, part);
  const double scale = dmax > 0.0 ? 1.0 / dmax : 1.0;
#pragma unroll 1
  for (int idx = c.tid; idx < ppr * ld; idx += c.nt) {
    const int a = idx / ld, b = idx - a * ld;          // ld is a compile-time constant
    Tf[idx] = (a < r && b < r) ? (float)(s.T[idx] * scale) : 0.0f;
    Jf[idx] = (a == b) ? 1.0f : 0.0f;
  }
  c.sync();
  for (int sweep = 0; sweep < kMaxSweepsF32; ++sweep) {
    int big = 0;
    s.count_sweeps_f32 += jacobi<LD, float>(c, s, &Tf, &Ta, &Jf, &Ja, r, r, 1, &big);
    if (!big) break;
    part = 0.0;
#pragma unroll 1
    for (int idx = c.tid; idx < r * r; idx += c.nt) {
      const int i = fast_div(idx, s.div_r), j = idx - i * r;
      if (i != j) {
        const float tij = Tf[i * ld + j], tii = Tf[i * ld + i], tjj = Tf[j * ld + j];
        if (tij * tij > 1e-14f * fabsf(tii * tjj) && tij * tij > 1e-30f) {
          const float th = fabsf(tij) / fabsf(tjj - tii);              // Inf for equal diagonal entries
          part = fmax(part, th <= 3.0e38f ? (double)th : 1.7e308);
        }
      }
    }
    if (block_max(c, s, part) <= 0.5 * RefineLimits<LD>::theta) break;
  }
#pragma unroll 1
  for (int idx = c.tid; idx < r * r; idx += c.nt) {
    const int i = fast_div(idx, s.div_r), j = idx - i * r;
    s.J[i * ld + j] = (double)Jf[i * ld + j];
  }
  c.sync();
}

// ev[k] = T[k][k]; ord[q] = index of the q-th largest (ties by index).  All threads return
// the number of eigenvalues > kRankRel * largest among the first `limit` in that order.
// One phase: the thread of index k reads the whole diagonal, so it knows the rank of its own
// entry and the largest one; the count is taken by the barrier that publishes ord and ev.
template <int LD>
FA_FN int sort_eigs(const Ctx& c, const Smem& s, const double* T, int dim, int limit) {
  constexpr int ld = LD;
  const int lim = limit < dim ? limit : dim;
  int mine = 0;
#ifdef FA_IRLS_HOST
  int keep = 0;
#endif
#pragma unroll 1
  for (int k = c.tid; k < dim; k += c.nt) {
    const double e = T[k * ld + k];
    double top = e;
    int rank = 0;
    for (int l = 0; l < dim; ++l) {
      const double o = T[l * ld + l];
      rank += (o > e || (o == e && l < k)) ? 1 : 0;
      top = fmax(top, o);
    }
    s.ord[rank] = k;
    s.ev[k] = e;
    mine = (rank < lim && top > 0.0 && e > kRankRel * top) ? 1 : 0;
#ifdef FA_IRLS_HOST
    keep += mine;
#endif
  }
#ifndef FA_IRLS_HOST
  return __syncthreads_count(mine);
#else
  return keep;
#endif
}

// One term of the objective with value u (the quantity under the root in Eq. (5)): its
// contribution u^(1/a) and the factor max(u^(1 - 1/a), eps) of its reweighting (Eq. (4) with
// constant a; a = 2 gives the square roots of Eq. (5) and takes the sqrt fast path).
FA_FN_SHARED void term_of_general(double u, double a, double& contrib, double& denom) {
  if (u <= 0.0) { contrib = 0.0; denom = kEps; }
  else { contrib = pow(u, 1.0 / a); denom = fmax(pow(u, 1.0 - 1.0 / a), kEps); }
}
FA_FN void term_of(double u, double a, double& contrib, double& denom) {
  if (a == 2.0) { contrib = sqrt(u); denom = fmax(contrib, kEps); }
  else term_of_general(u, a, contrib, denom);
}

// From residual coordinates Res (rows k0..r-1 are the part of f_i outside the subspace) and the
// full coordinates P: u_i, next data weights w_i, the matrix M of the next weighted PCA and the
// value of Eq. (5).  `uniform` builds the round-one weights instead (u is not needed then).
//
// cb, ca: the data term of worker i is cb (1 - v_i)^(1/a) + ca v_i^(1/a) -- a Beta(alpha, beta)
// likelihood of the values with cb = 2 (1 - beta), ca = 2 (1 - alpha); Eq. (1) has alpha = 1,
// beta = 1/2, i.e. cb = 1, ca = 0.  With ca > 0 a weight can be negative.
template <int LD>
FA_FN double weights_and_objective(const Ctx& c, Smem& s, const double* Res, int k0, int r, int p,
                                   double coef, bool uniform, double a, double cb = 1.0, double ca = 0.0,
                                   bool want_objective = true) {
  constexpr int ld = LD;
  double part = 0.0;
#pragma unroll 1
  for (int i = c.tid; i < p; i += c.nt) {
    double ui = 0.0, wi = 0.0;
    if (s.dinv[i] != 0.0) {
      if (uniform) wi = 1.0;
      else {
        const double acc = dot<LD, LD, LD - kLdPad>(Res + k0 * ld + i, Res + k0 * ld + i, r - k0);
        if (a == 2.0 && cb == 1.0 && ca == 0.0) {
          // the paper's square roots without a division or a square root: with y = 1/sqrt(acc fn),
          // sqrt(u) = acc y and 1/(fn sqrt(u)) = y
          const double fni = s.fn[i];
          const double y = acc > 0.0 ? FA_RSQRT(acc * fni) : 0.0;
          const double contrib = acc * y;
          part += contrib;
          wi = contrib >= kEps ? y : 1.0 / (fni * kEps);
          ui = contrib * contrib;
          s.u[i] = ui;
          s.w[i] = wi;
          continue;
        }
        ui = acc / s.fn[i];
        double contrib, denom;
        term_of(ui, a, contrib, denom);
        if (cb == 1.0 && ca == 0.0) {
          part += contrib;
          wi = 1.0 / (s.fn[i] * denom);
        } else {
          // explained part: the leading coordinates when Res is the coordinate matrix itself
          double vi;
          if (Res == s.P) {
            double e = 0.0;
            for (int k = 0; k < k0; ++k) { double v = s.P[k * ld + i]; e += v * v; }
            vi = e / s.fn[i];
          } else {
            vi = fmax(1.0 - ui, 0.0);
          }
          double contrib_v, denom_v;
          term_of(vi, a, contrib_v, denom_v);
          part += cb * contrib + ca * contrib_v;
          wi = (cb / denom - ca / denom_v) / s.fn[i];
        }
      }
    }
    s.u[i] = ui;
    s.w[i] = wi;
  }
  c.sync();
  if (coef > 0.0) {
    // off-diagonal entries M_ij = M_ji = -2 w_ij (ordered pairs: each unordered pair counted twice, and
    // twice in the objective); one item per unordered pair i < j
#pragma unroll 1
    for (int idx = c.tid; idx < p * (p - 1) / 2; idx += c.nt) {
      const int i = s.pairs[idx] >> 8, j = s.pairs[idx] & 255;
      double d2, res2;
      diff_sq<LD>(s.P + i, s.P + j, (Res == s.P) ? k0 : r, r, d2, res2);
      double wij = 0.0;
      if (d2 > kSamePairRel * (s.fn[i] + s.fn[j])) {
        if (uniform) wij = coef;
        else {
          if (Res != s.P) { double all; diff_sq<LD>(Res + i, Res + j, k0, r, all, res2); }
          if (a == 2.0) {
            const double y = res2 > 0.0 ? FA_RSQRT(res2 * d2) : 0.0;     // sqrt(u) = res2 y, 1/(d2 sqrt(u)) = y
            const double contrib = res2 * y;
            part += 2.0 * coef * contrib;
            wij = contrib >= kEps ? coef * y : coef / (d2 * kEps);
          } else {
            double contrib, denom;
            term_of(res2 / d2, a, contrib, denom);
            part += 2.0 * coef * contrib;
            wij = coef / (d2 * denom);
          }
        }
      }
      s.M[i * ld + j] = -2.0 * wij;
      s.M[j * ld + i] = -2.0 * wij;
    }
    c.sync();
#pragma unroll 1
    for (int i = c.tid; i < p; i += c.nt) {
      double acc = 0.0;
      for (int j = 0; j < p; ++j) acc -= (j != i) ? s.M[i * ld + j] : 0.0;
      s.M[i * ld + i] = s.w[i] + acc;
    }
  }
  if (!want_objective) {                 // nobody asked for the value of Eq. (5): the sum over the block is skipped
    c.sync();                            // publishes M and w
    return 0.0;
  }
  return block_sum(c, s, part);          // its barrier also publishes M and w
}

// The same for workers that hold several gradients each (rows of one worker are consecutive):
// the value of worker i is 1 - tr(Y^T g_i g_i^T Y) / tr(g_i^T g_i) (appendix restatement of Eq. (5)),
// one weight per worker multiplies all of its rows, and the pair terms of the regulariser are taken
// between the workers' mean gradients.  `p` is the number of rows.  s.T and s.J are scratch here
// (mean coordinates of every worker: all of them, and the residual part).
template <int LD>
FA_FN double weights_and_objective_grouped(const Ctx& c, Smem& s, const double* Res, int k0, int r, int p,
                                           double coef, bool uniform, double a) {
  constexpr int ld = LD;
  const int nw = s.nw;
  double* Fm = s.T;
  double* Rm = s.J;
  double part = 0.0;
  double gmax = 0.0;
  for (int i = 0; i < nw; ++i) gmax = fmax(gmax, s.gtr[i]);
#pragma unroll 1
  for (int i = c.tid; i < nw; i += c.nt) {
    double ui = 0.0, wi = 0.0;
    if (s.gtr[i] > kZeroNormRel * gmax) {
      if (uniform) wi = 1.0;
      else {
        const int r0 = s.first[i], r1 = (i + 1 < nw) ? s.first[i + 1] : p;
        double acc = 0.0;
        for (int row = r0; row < r1; ++row)
          for (int k = k0; k < r; ++k) { double v = Res[k * ld + row]; acc += v * v; }
        ui = acc / s.gtr[i];
        double contrib, denom;
        term_of(ui, a, contrib, denom);
        part += contrib;
        wi = 1.0 / (s.gtr[i] * denom);
      }
    }
    s.gu[i] = ui;
    s.gw[i] = wi;
  }
  if (coef > 0.0) {
#pragma unroll 1
    for (int idx = c.tid; idx < r * nw; idx += c.nt) {
      const int k = idx / nw, i = idx - k * nw;
      const int r0 = s.first[i], r1 = (i + 1 < nw) ? s.first[i + 1] : p;
      double fm = 0.0, rm = 0.0;
      for (int row = r0; row < r1; ++row) { fm += s.P[k * ld + row]; rm += Res[k * ld + row]; }
      Fm[k * ld + i] = fm * s.ginv[i];
      Rm[k * ld + i] = (k >= k0) ? rm * s.ginv[i] : 0.0;
    }
  }
  c.sync();
#pragma unroll 1
  for (int row = c.tid; row < p; row += c.nt) { s.w[row] = s.gw[s.grp[row]]; s.u[row] = s.gu[s.grp[row]]; }
  if (coef > 0.0) {
    // rows of different workers i != j: M = -2 w_ij / (k_i k_j)  (ordered pairs: each pair twice)
#pragma unroll 1
    for (int idx = c.tid; idx < p * p; idx += c.nt) {
      const int ra = idx / p, rb = idx - ra * p;
      const int i = s.grp[ra], j = s.grp[rb];
      if (i == j) continue;
      double d2 = 0.0, ni = 0.0, nj = 0.0, res2 = 0.0;
      for (int k = 0; k < r; ++k) {
        const double x = Fm[k * ld + i], y = Fm[k * ld + j];
        d2 += (x - y) * (x - y); ni += x * x; nj += y * y;
      }
      double wij = 0.0;
      if (d2 > kSamePairRel * (ni + nj)) {
        if (uniform) wij = coef;
        else {
          for (int k = k0; k < r; ++k) { double v = Rm[k * ld + i] - Rm[k * ld + j]; res2 += v * v; }
          double contrib, denom;
          term_of(res2 / d2, a, contrib, denom);
          if (ra == s.first[i] && rb == s.first[j]) part += coef * contrib;   // once per ordered pair
          wij = coef / (d2 * denom);
        }
      }
      s.M[ra * ld + rb] = -2.0 * wij * s.ginv[i] * s.ginv[j];
    }
    c.sync();
    // rows of one worker: what makes the pair part's row sums vanish, plus the data weight
#pragma unroll 1
    for (int idx = c.tid; idx < p * p; idx += c.nt) {
      const int ra = idx / p, rb = idx - ra * p;
      const int i = s.grp[ra];
      if (s.grp[rb] != i) continue;
      double acc = 0.0;
      for (int q = 0; q < p; ++q) if (s.grp[q] != i) acc -= s.M[ra * ld + q];
      s.M[ra * ld + rb] = acc * s.ginv[i] + ((ra == rb) ? s.w[ra] : 0.0);
    }
  }
  return block_sum(c, s, part);
}

struct Outputs {
  double* A;          // p x m or null
  float* c;           // p or null
  double* w;          // p or null
  double* obj;        // iters (or 1) or null
  double* S;          // p x p selection matrix or null
  int* status;        // or null
  int* rounds;        // rounds actually run, or null
};

FA_FN void write_zero_outputs(const Ctx& c, const Outputs& o, int p, int m, int iters, int nweights) {
#pragma unroll 1
  for (int i = c.tid; i < p * m; i += c.nt) if (o.A) o.A[i] = 0.0;
#pragma unroll 1
  for (int i = c.tid; i < p; i += c.nt) if (o.c) o.c[i] = 0.f;
#pragma unroll 1
  for (int i = c.tid; i < nweights; i += c.nt) if (o.w) o.w[i] = 0.0;
#pragma unroll 1
  for (int i = c.tid; i < iters; i += c.nt) if (o.obj) o.obj[i] = 0.0;
#pragma unroll 1
  for (int i = c.tid; i < p * p; i += c.nt) if (o.S) o.S[i] = 0.0;
  if (o.rounds && c.tid == 0) *o.rounds = 0;
}

// K: p x p inner products (global or shared memory).  start: 0 = round one is uniform; 1 = take the
// subspace spanned by G^T A0 as the current one for the first reweighting, A0 being the A of an
// earlier round on the same K (its image is orthonormal already: single-step interface); 2 = the
// same for any A0 (p x m), e.g. the A of the previous training step: its image is orthonormalised
// first, and a rank-deficient one falls back to the uniform round.  tol >= 0: stop after round
// t >= 2 once the objective moved by <= tol (remaining entries of o.obj repeat the last value).  nw > 0: the p rows belong to nw workers, cnt[i] consecutive rows each (o.w then has nw
// entries); nw = 0: one gradient per worker.  Returns the status bits (same value in every thread).
// kPlain: the caller promises the paper's default terms (a = 2, Beta(1, 1/2), one gradient per worker).  The
// arguments are then replaced by those constants, the compiler drops every other branch, and the code of
// a round shrinks to what this case executes -- the kernels are bound by instruction fetch as much as by
// anything else (their code does not fit the instruction cache).
template <int LD, bool kPlain = false>
FA_FN int run(const Ctx& c, Smem& s, const double* K, int p, int m, double lambda, double a, int iters,
              int start, const double* A0, double tol, const Outputs& o, int nw = 0,
              const unsigned char* cnt = nullptr, double cb = 1.0, double ca = 0.0) {
  if (kPlain) { a = 2.0; nw = 0; cnt = nullptr; cb = 1.0; ca = 0.0; }
  constexpr int ld = LD;
  const int pp = (p + 1) & ~1;
  int status = 0;

  // ---- load K, reject non-finite input
  if (c.tid == 0) { s.flags[1] = 0; }
  s.div_p = make_div(p);
  c.sync();
#pragma unroll 1
  for (int idx = c.tid; idx < pp * ld; idx += c.nt) { s.T[idx] = 0.0; s.J[idx] = 0.0; s.Aacc[idx] = 0.0; s.P[idx] = 0.0; s.M[idx] = 0.0; s.tmp[idx] = 0.0; }
  c.sync();
#pragma unroll 1
  for (int idx = c.tid; idx < p * p; idx += c.nt) {
    const int i = fast_div(idx, s.div_p), j = idx - i * p;
    double v = K[idx];
    if (!(fabs(v) <= 1.7e308)) s.flags[1] = 1;
    s.T[i * ld + j] = v;
  }
  c.sync();
  if (s.flags[1]) {
    write_zero_outputs(c, o, p, m, iters, nw > 0 ? nw : p);
    return ST_NONFINITE;
  }
  double kmax = 0.0;
  for (int i = 0; i < p; ++i) kmax = fmax(kmax, s.T[i * ld + i]);
  if (!(kmax > 0.0)) {
    write_zero_outputs(c, o, p, m, iters, nw > 0 ? nw : p);
    return ST_RANK0;
  }
#pragma unroll 1
  for (int idx = c.tid; idx < p * (p - 1) / 2; idx += c.nt) {
    int i, jm;
    tri_pair(idx, i, jm);                         // i <= jm over p - 1 columns: the pair (i, jm + 1)
    s.pairs[idx] = (unsigned short)((i << 8) | (jm + 1));
  }
  // kd = ||g_i||^2, dinv = 1 / ||g_i|| (0 for a zero gradient), fn (for now) = ||g_i||
#pragma unroll 1
  for (int i = c.tid; i < p; i += c.nt) {
    const double kii = s.T[i * ld + i];
    const bool zero = kii <= kZeroNormRel * kmax;
    const double nrm = zero ? 0.0 : sqrt(kii);
    s.kd[i] = kii; s.fn[i] = nrm; s.dinv[i] = zero ? 0.0 : 1.0 / nrm;
  }
  c.sync();

  // ---- Kt = D^-1 K D^-1 (symmetrised, unit diagonal) -> tmp
#pragma unroll 1
  for (int idx = c.tid; idx < p * (p + 1) / 2; idx += c.nt) {
    int i, j;
    tri_pair(idx, i, j);
    double v = (i == j) ? (s.dinv[i] != 0.0 ? 1.0 : 0.0)
                        : 0.5 * (s.T[i * ld + j] + s.T[j * ld + i]) * s.dinv[i] * s.dinv[j];
    s.tmp[i * ld + j] = v; s.tmp[j * ld + i] = v;
  }
  // remaining diagonal of the factorisation -> u (and, on alternate steps, w: see below); ord[j] = 0
  // while column j has not been a pivot, else 1 + the step at which it was
#pragma unroll 1
  for (int i = c.tid; i < p; i += c.nt) { s.u[i] = (s.dinv[i] != 0.0) ? 1.0 : 0.0; s.ord[i] = 0; }
  c.sync();

  // ---- Cholesky with complete pivoting, Kt = R^T R, R (r x p) kept in P with the original column
  // order: column i of R is the image f_i / ||g_i|| of worker i in R^r.  Stops when the largest
  // remaining diagonal entry is <= kRankRel (the diagonal of Kt is 1), which fixes the rank r.
  // One barrier per step: the pivot is found by every warp for itself (a reduction on the upper
  // words of the remaining diagonal -- values closer than six digits count as tied and the lowest
  // index wins), and the thread of column j updates the column and its remaining diagonal entry.
  // What a step writes must not be seen by a warp that is still searching in the same step: the
  // remaining diagonal alternates between two arrays, and a pivot mark counts from the next step on.
  int r = 0;
  for (int k = 0; k < p; ++k) {
    const double* ucur = (k & 1) ? s.w : s.u;
    double* unext = (k & 1) ? s.u : s.w;
    int piv = -1;
#ifndef FA_IRLS_HOST
    {
      const int lane = c.tid & 31;
      const int m0 = lane < p ? s.ord[lane] : 1, m1 = lane + 32 < p ? s.ord[lane + 32] : 1;
      const double u0 = (m0 == 0 || m0 > k) ? ucur[lane < p ? lane : 0] : 0.0;
      const double u1 = (m1 == 0 || m1 > k) ? ucur[lane + 32 < p ? lane + 32 : 0] : 0.0;
      const unsigned h0 = (lane < p) ? (unsigned)__double2hiint(u0) : 0u;
      const unsigned h1 = (lane + 32 < p) ? (unsigned)__double2hiint(u1) : 0u;
      const unsigned best = __reduce_max_sync(0xffffffffu, max(h0, h1));
      const unsigned cand = (h0 == best && lane < p) ? (unsigned)lane
                                                     : ((h1 == best && lane + 32 < p) ? (unsigned)(lane + 32) : 64u);
      const unsigned at = __reduce_min_sync(0xffffffffu, cand);
      if (best > (unsigned)__double2hiint(kRankRel) && at < 64u) piv = (int)at;
    }
#else
    {
      double dmax = kRankRel;
      for (int j = 0; j < p; ++j) {               // ties go to the lowest index
        const double dj = ucur[j];
        if (s.ord[j] == 0 && dj > dmax) { dmax = dj; piv = j; }
      }
    }
#endif
    if (piv < 0) break;
    const double dpiv = ucur[piv];
    if (!(dpiv > kRankRel)) break;                // (the upper-word test lets a value just below the cut through)
    const double rinv = FA_RSQRT(dpiv), rkk = dpiv * rinv;   // dpiv in (1e-12, 1]: a normal number
#pragma unroll 1
    for (int j = c.tid; j < p; j += c.nt) {
      const int mark = s.ord[j];
      const bool done = mark != 0 && mark <= k;   // a pivot of an earlier step
      double v, left = 0.0;
      if (j == piv) { v = rkk; s.ord[j] = k + 1; s.piv[k] = piv; s.lam[k] = rinv; }
      else if (done) v = 0.0;
      else {
        v = (s.tmp[piv * ld + j] - dot<LD, LD, LD - kLdPad>(s.P + piv, s.P + j, k)) * rinv;
        left = fmax(ucur[j] - v * v, 0.0);
      }
      s.P[k * ld + j] = v;
      unext[j] = left;
    }
    c.sync();
    r = k + 1;
  }
  s.div_r = make_div(r);
  s.div_tr = make_div((r + 7) >> 3); s.div_tp = make_div((p + 7) >> 3);

  // ---- U = R11^-1 (R11 = pivot columns of R, upper triangular) by back substitution, one column
  // per thread -> J buffer.  Q = G D^-1 X with X[piv_a][:] = U[a][:] has orthonormal columns and
  // Q^T g_i = f_i, so Aacc starts as D^-1 X (p x r).  First the pivot columns are gathered (-> M),
  // so that the sums below run over consecutive elements; 1 / R11_aa is the rinv of step a.
#pragma unroll 1
  for (int idx = c.tid; idx < r * r; idx += c.nt) {
    const int a = fast_div(idx, s.div_r), l = idx - a * r;
    s.M[a * ld + l] = s.P[a * ld + s.piv[l]];
  }
  c.sync();
#pragma unroll 1
  for (int bcol = c.tid; bcol < r; bcol += c.nt) {
    for (int a = bcol; a >= 0; --a) {
      const double sum = dot<1, LD, LD - kLdPad>(s.M + a * ld + a + 1, s.J + (a + 1) * ld + bcol, bcol - a);
      s.J[a * ld + bcol] = (((a == bcol) ? 1.0 : 0.0) - sum) * s.lam[a];
    }
  }
  c.sync();
#pragma unroll 1
  for (int idx = c.tid; idx < r * r; idx += c.nt) {
    const int a = fast_div(idx, s.div_r), bcol = idx - a * r;
    if (bcol >= a) {
      const int pa = s.piv[a];
      s.Aacc[pa * ld + bcol] = s.dinv[pa] * s.J[a * ld + bcol];
    }
  }
  // ---- P = F: scale column i of R back by ||g_i||; fn = ||f_i||^2
#pragma unroll 1
  for (int i = c.tid; i < p; i += c.nt) {
    const double nrm = s.fn[i];
    double acc = 0.0;
    for (int k = 0; k < r; ++k) { const double v = s.P[k * ld + i] * nrm; s.P[k * ld + i] = v; acc = fma(v, v, acc); }
    s.fn[i] = acc;
  }
#pragma unroll 1
  for (int idx = c.tid; idx < pp * ld; idx += c.nt) s.M[idx] = 0.0;     // M held the gathered columns
  c.sync();
  int sw = 0;

  s.div_r = make_div(r); s.div_p = make_div(p);
  s.div_tr = make_div((r + 7) >> 3); s.div_tp = make_div((p + 7) >> 3);
  const bool grouped = nw > 0;
  const int workers = grouped ? nw : p;
  if (grouped) {
    if (c.tid == 0) {
      int row = 0;
      for (int i = 0; i < nw; ++i) {
        s.first[i] = row;
        s.ginv[i] = 1.0 / (double)cnt[i];
        for (int q = 0; q < (int)cnt[i]; ++q) s.grp[row++] = i;
      }
    }
    c.sync();
#pragma unroll 1
    for (int i = c.tid; i < nw; i += c.nt) {
      const int r0 = s.first[i], r1 = (i + 1 < nw) ? s.first[i + 1] : p;
      double acc = 0.0;
      for (int row = r0; row < r1; ++row) acc += s.fn[row];
      s.gtr[i] = acc;
    }
    c.sync();
    s.nw = nw;
  }
  const double coef = (lambda > 0.0 && workers > 1) ? lambda / (double)(workers - 1) : 0.0;

  // ---- weights of the first round
  if (start != 0) {
    // Z0 = F A0 (r x m) -> J buffer
#pragma unroll 1
    for (int idx = c.tid; idx < r * m; idx += c.nt) {
      int k = idx / m, q = idx - k * m;
      double acc = 0.0;
      for (int i = 0; i < p; ++i) acc += s.P[k * ld + i] * A0[i * m + q];
      s.J[k * ld + q] = acc;
    }
    c.sync();
    if (start == 2) {
      // W = Z0^T Z0 -> T; Cholesky W = L L^T by one thread; Z = Z0 L^-T row by row
#pragma unroll 1
      for (int idx = c.tid; idx < m * m; idx += c.nt) {
        int q = idx / m, l = idx - q * m;
        double acc = 0.0;
        for (int k = 0; k < r; ++k) acc += s.J[k * ld + q] * s.J[k * ld + l];
        s.T[q * ld + l] = acc;
      }
      c.sync();
      if (c.tid == 0) {
        double dmin = 1.7e308, dmax = 0.0;
        bool ok = true;
        for (int q = 0; q < m && ok; ++q) {
          double d = s.T[q * ld + q];
          for (int l = 0; l < q; ++l) d -= s.T[q * ld + l] * s.T[q * ld + l];
          if (!(d > 0.0)) { ok = false; break; }
          const double lqq = sqrt(d);
          s.T[q * ld + q] = lqq;
          dmin = fmin(dmin, lqq); dmax = fmax(dmax, lqq);
          for (int i = q + 1; i < m; ++i) {
            double v = s.T[i * ld + q];
            for (int l = 0; l < q; ++l) v -= s.T[i * ld + l] * s.T[q * ld + l];
            s.T[i * ld + q] = v / lqq;
          }
        }
        s.flags[1] = (ok && dmin > 1e-12 * dmax) ? 1 : 0;
      }
      c.sync();
      if (s.flags[1] == 0) start = 0;
      else {
#pragma unroll 1
        for (int k = c.tid; k < r; k += c.nt) {
          for (int q = 0; q < m; ++q) {
            double v = s.J[k * ld + q];
            for (int l = 0; l < q; ++l) v -= s.J[k * ld + l] * s.T[q * ld + l];
            s.J[k * ld + q] = v / s.T[q * ld + q];
          }
        }
      }
      c.sync();
    }
  }
  if (start == 0) {
    if (grouped) (void)weights_and_objective_grouped<LD>(c, s, s.P, 0, r, p, coef, true, a);
    else (void)weights_and_objective<LD>(c, s, s.P, 0, r, p, coef, true, a, cb, ca);
  } else {
    // C = Z0^T F (m x p) -> T buffer; Res = F - Z0 C -> tmp
#pragma unroll 1
    for (int idx = c.tid; idx < m * p; idx += c.nt) {
      int q = idx / p, i = idx - q * p;
      double acc = 0.0;
      for (int k = 0; k < r; ++k) acc += s.J[k * ld + q] * s.P[k * ld + i];
      s.T[q * ld + i] = acc;
    }
    c.sync();
#pragma unroll 1
    for (int idx = c.tid; idx < r * p; idx += c.nt) {
      int k = idx / p, i = idx - k * p;
      double acc = s.P[k * ld + i];
      for (int q = 0; q < m; ++q) acc -= s.J[k * ld + q] * s.T[q * ld + i];
      s.tmp[k * ld + i] = acc;
    }
    c.sync();
    if (grouped) (void)weights_and_objective_grouped<LD>(c, s, s.tmp, 0, r, p, coef, false, a);
    else (void)weights_and_objective<LD>(c, s, s.tmp, 0, r, p, coef, false, a, cb, ca);
  }

  int m_eff = 0, rounds = iters;
  double prev_obj = 0.0;
  for (int t = 0; t < iters; ++t) {
    sw = 0;
#pragma unroll 1
    for (int i = c.tid; i < p; i += c.nt) s.wused[i] = s.w[i];
    if (grouped) for (int i = c.tid; i < nw; i += c.nt) s.gwused[i] = s.gw[i];
    // ---- T = P M P^T (current basis); only one triangle is taken from the product, so that T is
    // symmetric to the last bit
    if (coef > 0.0) {
      matmul<LD, 1, 1, LD>(c, p, r, p, s.div_tr, s.M, s.P, [&](int i, int a, double v) { s.tmp[i * ld + a] = v; });   // tmp = M P^T
      c.sync();
      matmul<LD, 1, LD, 1>(c, r, r, p, s.div_tr, s.P, s.tmp,
                           [&](int a, int b, double v) { if (a <= b) { s.T[a * ld + b] = v; s.T[b * ld + a] = v; } });
    } else {
#pragma unroll 1
      for (int idx = c.tid; idx < r * p; idx += c.nt) {                                   // tmp = P diag(w)
        const int a = fast_div(idx, s.div_p), i = idx - a * p;
        s.tmp[a * ld + i] = s.w[i] * s.P[a * ld + i];
      }
      c.sync();
      matmul<LD, 1, 1, LD>(c, r, r, p, s.div_tr, s.tmp, s.P,
                           [&](int a, int b, double v) { if (a <= b) { s.T[a * ld + b] = v; s.T[b * ld + a] = v; } });
    }
    c.sync();
    // ---- eigenvectors of T.  From the second round on T is close to diagonal here (the basis is the
    // previous round's eigenbasis), the closer the further the rounds have converged: the refinement
    // is tried first, and each time it declines one Jacobi sweep is made, the coordinates are taken
    // to the swept basis and T is looked at again.
    bool f32_tried = false;
    for (;;) {
      if (refine_eig<LD>(c, s, r)) break;
      // far from diagonal: fp32 sweeps, then the refinement from what they found.  Only where a rotation
      // round is bound by shared-memory traffic (more than 32 gradients: a quarter faster in fp32); with
      // fewer the round costs the same in either precision and the extra refinement steps are a loss.
      if (LD > 36 && !f32_tried) {
        f32_tried = true;
        sweeps_fp32<LD>(c, s, r);
        if (refine_eig<LD>(c, s, r, true)) break;
      }
      const int ppr = (r + 1) & ~1;                       // the sweeps work on an even number of indices
#pragma unroll 1
      for (int idx = c.tid; idx < ppr * ld; idx += c.nt) s.J[idx] = 0.0;
      if (ppr > r) for (int b = c.tid; b < ppr; b += c.nt) { s.T[r * ld + b] = 0.0; s.T[b * ld + r] = 0.0; }
      c.sync();
#pragma unroll 1
      for (int a = c.tid; a < ppr; a += c.nt) s.J[a * (ld + 1)] = 1.0;
      c.sync();
      int big = 0;
      sw += jacobi<LD, double>(c, s, &s.T, &s.tmp, &s.J, &s.M, r, r, 1, &big);   // M is free until the next weights
      const bool last = !big || sw >= kMaxSweeps;
      if (big && last) status |= ST_EIG_SWEEPS;
      if (last) break;           // diagonal to rounding level (or given up): J holds the eigenvectors
      matmul<1, LD, LD, 1>(c, r, p, r, s.div_tp, s.J, s.P, [&](int k, int i, double v) { s.tmp[k * ld + i] = v; });   // P <- J^T P
      matmul<LD, 1, LD, 1>(c, p, r, r, s.div_tr, s.Aacc, s.J, [&](int i, int k, double v) { s.M[i * ld + k] = v; },
                           ((r + 7) >> 3) * ((p + 7) >> 3));                                                        // Aacc <- Aacc J
      c.sync();
      { double* x = s.P; s.P = s.tmp; s.tmp = x; }
      { double* x = s.Aacc; s.Aacc = s.M; s.M = x; }
    }
    s.count_sweeps += sw;
    m_eff = sort_eigs<LD>(c, s, s.T, r, m);

    // ---- rotate into the new (sorted) eigenbasis: P <- J^T P, Aacc <- Aacc J
    matmul<1, LD, LD, 1>(c, r, p, r, s.div_tp, s.J, s.P, [&](int k, int i, double v) { s.tmp[k * ld + i] = v; }, 0, s.ord, nullptr);
    matmul<LD, 1, LD, 1>(c, p, r, r, s.div_tr, s.Aacc, s.J, [&](int i, int k, double v) { s.M[i * ld + k] = v; },
                         ((r + 7) >> 3) * ((p + 7) >> 3), nullptr, s.ord);
    c.sync();
    { double* x = s.P; s.P = s.tmp; s.tmp = x; }
    { double* x = s.Aacc; s.Aacc = s.M; s.M = x; }

    // ---- terms of Eq. (5) at the new subspace, and the next round's weights
    const bool want_obj = o.obj != nullptr || tol >= 0.0;
    double obj = grouped ? weights_and_objective_grouped<LD>(c, s, s.P, m_eff, r, p, coef, false, a)
                         : weights_and_objective<LD>(c, s, s.P, m_eff, r, p, coef, false, a, cb, ca, want_obj);
    if (o.obj && c.tid == 0) o.obj[t] = obj;
    if (tol >= 0.0 && t >= 1 && fabs(prev_obj - obj) <= tol) {      // same value in every thread
      rounds = t + 1;
      if (o.obj) for (int q = t + 1 + c.tid; q < iters; q += c.nt) o.obj[q] = obj;
      break;
    }
    prev_obj = obj;
  }
  if (o.rounds && c.tid == 0) *o.rounds = rounds;
  if (m_eff < m) status |= ST_RANK_LT_M;

  // ---- outputs
  if (o.A) {
#pragma unroll 1
    for (int idx = c.tid; idx < p * m; idx += c.nt) {
      int i = idx / m, q = idx - i * m;
      o.A[idx] = (q < m_eff) ? s.Aacc[i * ld + q] : 0.0;
    }
  }
  if (o.w) {
    if (grouped) for (int i = c.tid; i < nw; i += c.nt) o.w[i] = s.gwused[i];
    else for (int i = c.tid; i < p; i += c.nt) o.w[i] = s.wused[i];
  }
  if (o.S) {   // Y Y^T G = G S with S = A (A^T K): (A^T K) e_j are the leading coordinates of f_j
#pragma unroll 1
    for (int idx = c.tid; idx < p * p; idx += c.nt) {
      const int i = idx / p, j = idx - i * p;
      double acc = 0.0;
      for (int k = 0; k < m_eff; ++k) acc += s.Aacc[i * ld + k] * s.P[k * ld + j];
      o.S[idx] = acc;
    }
  }
  if (o.c) {
#pragma unroll 1
    for (int k = c.tid; k < m_eff; k += c.nt) {        // s_k = sum_j P[k][j]  (Z^T F 1)
      double acc = 0.0;
      if (grouped) for (int j = 0; j < p; ++j) acc += s.P[k * ld + j] * s.ginv[s.grp[j]];   // sum of worker means
      else for (int j = 0; j < p; ++j) acc += s.P[k * ld + j];
      s.ev[k] = acc;
    }
    c.sync();
#pragma unroll 1
    for (int i = c.tid; i < p; i += c.nt) {
      double acc = 0.0;
      for (int k = 0; k < m_eff; ++k) acc += s.Aacc[i * ld + k] * s.ev[k];
      o.c[i] = (float)(acc / (double)workers);
    }
  }
  return status;
}

}  // namespace fa_irls
