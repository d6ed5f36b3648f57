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
// = F M F^T, diagonalises it by Jacobi (started in the previous round's eigenbasis, where T is
// already nearly diagonal), keeps the m leading eigenvectors and evaluates the terms under the
// square roots of Eq. (5) as squared residual norms, i.e. as sums of squares over the discarded
// eigen-directions -- no "1 - x" cancellation.
//
// The code is written as phases separated by block barriers, every phase a strided loop over
// independent items, so that it can also be compiled for the host with one "thread" (used to
// debug the arithmetic without a GPU).
#pragma once

#include <math.h>
#include <stdint.h>

#ifndef FA_IRLS_HOST
#define FA_FN __device__ __forceinline__
#define FA_HD __host__ __device__ inline
#else
#define FA_FN static inline
#define FA_HD static inline
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

// Shared-memory image.  Matrices are (pp x ld) doubles, pp = p rounded up to even, ld odd.
struct Smem {
  double *T, *J, *P, *M, *Aacc, *tmp;   // six matrix buffers, rotated by pointer swaps
  double *kd, *dinv, *fn, *u, *w, *wused, *ev, *red;
  double *rc, *rs;                       // rotation cos / sin per pair
  int *ra, *rb, *ord;                    // rotation indices per pair, sort order
  int *flags;                            // [0],[3] rotated-this-sweep (by sweep parity), [1] scratch
  // several gradients per worker (nw > 0): per-worker trace, value, weight, weight in use, 1/k_i;
  // grp[row] = worker of a row, first[i] = first row of worker i
  double *gtr, *gu, *gw, *gwused, *ginv;
  int *grp, *first;
  int nw;
  int ld;
};

FA_HD size_t smem_bytes(int p, int nt) {
  int pp = (p + 1) & ~1;
  int ld = pp + 1;
  size_t doubles = (size_t)6 * pp * ld + (size_t)12 * pp + nt + 2 * (pp / 2 + 1);
  size_t ints = (size_t)2 * (pp / 2 + 1) + 3 * pp + 8;
  return doubles * sizeof(double) + ints * sizeof(int) + 64;
}

FA_FN void carve(Smem& s, void* base, int p, int nt) {
  int pp = (p + 1) & ~1;
  int ld = pp + 1;
  double* d = reinterpret_cast<double*>(base);
  s.ld = ld;
  s.T = d; d += (size_t)pp * ld;
  s.J = d; d += (size_t)pp * ld;
  s.P = d; d += (size_t)pp * ld;
  s.M = d; d += (size_t)pp * ld;
  s.Aacc = d; d += (size_t)pp * ld;
  s.tmp = d; d += (size_t)pp * ld;
  s.kd = d; d += pp; s.dinv = d; d += pp; s.fn = d; d += pp; s.u = d; d += pp;
  s.w = d; d += pp; s.wused = d; d += pp; s.ev = d; d += pp;
  s.gtr = d; d += pp; s.gu = d; d += pp; s.gw = d; d += pp; s.gwused = d; d += pp; s.ginv = d; d += pp;
  s.red = d; d += nt;
  s.rc = d; d += pp / 2 + 1; s.rs = d; d += pp / 2 + 1;
  int* q = reinterpret_cast<int*>(d);
  s.ra = q; q += pp / 2 + 1; s.rb = q; q += pp / 2 + 1; s.ord = q; q += pp; s.grp = q; q += pp;
  s.first = q; q += pp; s.flags = q;
  s.nw = 0;
}

// Deterministic block-wide sum; every thread gets the result.
FA_FN double block_sum(const Ctx& c, const Smem& s, double v) {
#ifndef FA_IRLS_HOST
  for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
  c.sync();                                // s.red may still be read from a previous call
  if ((c.tid & 31) == 0) s.red[c.tid >> 5] = v;
  c.sync();
  double tot = 0.0;
  int nw = (c.nt + 31) >> 5;
  for (int k = 0; k < nw; ++k) tot += s.red[k];
  return tot;
#else
  (void)c; (void)s;
  return v;
#endif
}

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

FA_FN bool rotation(const double* T, int ld, int a, int b, int dim, double& cs, double& sn) {
  if (b >= dim) { cs = 1.0; sn = 0.0; return false; }
  return rotation_of(T[a * ld + a], T[b * ld + b], T[a * ld + b], cs, sn);
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
// and columns dim..pp-1 zero) is driven to diagonal form; J accumulates the rotations (J <- J * R).
// A pair is rotated whenever its off-diagonal entry is above rounding level; sweeping stops after
// the first sweep in which no rotated entry exceeded kJacobiBig relative to its diagonal: that
// sweep's rotations leave entries of the order of its square (quadratic convergence of the cyclic
// method), i.e. below rounding level.
//
// The data MOVES instead of the pairing (Brent-Luk systolic arrangement): a round rotates the pairs
// at the fixed positions (k, np + k) and stores rows and columns (and the columns of J) at their
// systolic_next() positions, from T / J into Talt / Jalt and back.  So every thread owns the same
// 2x2 blocks of T and (row, pair) items of J for the whole solve, all its offsets are worked out
// once before the first sweep, and all its loads go out together at the top of a round -- what a
// round costs here is the number of dependent instructions a warp has to issue.
//   * up to 8 pairs (dim <= 16): one item per thread; each thread works out the one or two
//     rotations it needs itself: one barrier per round and nothing else between threads;
//   * more pairs: several items per thread; the rotations are worked out once by the first np
//     threads and published in shared memory (a second barrier per round).
// A full sweep (pp - 1 rounds) returns every index to its own position, and sweeps are never cut
// short.  On return *Tio / *Jio point at the buffers that hold the results.  Returns the sweeps made.
// Up to 8 pairs on the device; any size on the host.
FA_FN int jacobi_small(const Ctx& c, const Smem& s, double** Tio, double** Taltio, double** Jio, double** Jaltio,
                       int dim, int jrows) {
  const int ld = s.ld;
  const int pp = (dim + 1) & ~1;
  const int np = pp >> 1;
  double* T = *Tio;
  double* Tn = *Taltio;
  double* J = *Jio;
  double* Jn = *Jaltio;
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
      // a lane of this warp whose own (column) pair is k hands over the row rotation
      const int w0 = idx & ~31;
      for (int j = 0; j < 32; ++j) {
        const int o = w0 + j;
        if (o < total2 && (o < nb2 ? o % np : (o - nb2) % np) == k) { it.ksrc = j; break; }
      }
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
  int sweep = 0;
  // "large rotation in this sweep" flag, double-buffered by sweep parity (slots 0 and 3)
  if (c.tid == 0) { s.flags[0] = 0; s.flags[3] = 0; }
  c.sync();
  for (; sweep < kMaxSweeps; ++sweep) {
    int* big = &s.flags[(sweep & 1) ? 3 : 0];
    if (c.tid == 0) s.flags[(sweep & 1) ? 0 : 3] = 0;
    for (int rd = 0; rd < pp - 1; ++rd) {
#ifndef FA_IRLS_HOST
      {
        // every lane with an item works out the rotation of its column pair l; a block of T gets
        // its row rotation from the lane `ksrc` of its warp (worked out here only if there is none)
        double cl = 1.0, sl = 0.0;
        bool bigl = false;
        double xac = 0.0, xad = 0.0, xbc = 0.0, xbd = 0.0;
        if (it.kind != 0) {
          const double laa = T[it.laa], lbb = T[it.lbb], lab = T[it.lab];
          if (it.kind == 1) { xac = T[it.x0]; xad = T[it.x1]; xbc = T[it.x2]; xbd = T[it.x3]; }
          else { xac = J[it.x0]; xad = J[it.x1]; }
          bigl = rotation_of(laa, lbb, lab, cl, sl);
        }
        const int src = it.ksrc < 0 ? 0 : it.ksrc;
        double ck = __shfl_sync(0xffffffffu, cl, src), sk = __shfl_sync(0xffffffffu, sl, src);
        if (it.kind == 1) {
          if (it.ksrc < 0) (void)rotation_of(T[it.kaa], T[it.kbb], T[it.kab], ck, sk);
          if (it.diag && bigl) *big = 1;
          const double yac = ck * xac - sk * xbc, yad = ck * xad - sk * xbd;
          const double ybc = sk * xac + ck * xbc, ybd = sk * xad + ck * xbd;
          Tn[it.z0] = cl * yac - sl * yad; Tn[it.z1] = sl * yac + cl * yad;
          Tn[it.z2] = cl * ybc - sl * ybd; Tn[it.z3] = sl * ybc + cl * ybd;
        } else if (it.kind == 2) {
          Jn[it.z0] = cl * xac - sl * xad;
          Jn[it.z1] = sl * xac + cl * xad;
        }
      }
#else
      if (it.kind == 1) {
        const double kaa = T[it.kaa], kbb = T[it.kbb], kab = T[it.kab];
        const double laa = T[it.laa], lbb = T[it.lbb], lab = T[it.lab];
        const double xac = T[it.x0], xad = T[it.x1], xbc = T[it.x2], xbd = T[it.x3];
        double ck, sk, cl, sl;
        const bool bigk = rotation_of(kaa, kbb, kab, ck, sk);
        (void)rotation_of(laa, lbb, lab, cl, sl);
        if (it.diag && bigk) *big = 1;
        const double yac = ck * xac - sk * xbc, yad = ck * xad - sk * xbd;
        const double ybc = sk * xac + ck * xbc, ybd = sk * xad + ck * xbd;
        Tn[it.z0] = cl * yac - sl * yad; Tn[it.z1] = sl * yac + cl * yad;
        Tn[it.z2] = cl * ybc - sl * ybd; Tn[it.z3] = sl * ybc + cl * ybd;
      } else if (it.kind == 2) {
        const double laa = T[it.laa], lbb = T[it.lbb], lab = T[it.lab];
        const double va = J[it.x0], vb = J[it.x1];
        double cl, sl;
        (void)rotation_of(laa, lbb, lab, cl, sl);
        Jn[it.z0] = cl * va - sl * vb;
        Jn[it.z1] = sl * va + cl * vb;
      }
#endif
      // further items (fewer threads than items): offsets on the fly
      for (int idx = c.tid + c.nt; idx < total2; idx += c.nt) {
        if (idx < nb2) {
          const int k = idx / np, l = idx - k * np;
          const int a = k, b = np + k, cc = l, d = np + l;
          const double kaa = T[a * ld + a], kbb = T[b * ld + b], kab = T[a * ld + b];
          const double laa = T[cc * ld + cc], lbb = T[d * ld + d], lab = T[cc * ld + d];
          const double xac = T[a * ld + cc], xad = T[a * ld + d], xbc = T[b * ld + cc], xbd = T[b * ld + d];
          double ck, sk, cl, sl;
          const bool bigk = rotation_of(kaa, kbb, kab, ck, sk);
          (void)rotation_of(laa, lbb, lab, cl, sl);
          if (k == l && bigk) *big = 1;
          const double yac = ck * xac - sk * xbc, yad = ck * xad - sk * xbd;
          const double ybc = sk * xac + ck * xbc, ybd = sk * xad + ck * xbd;
          const int pa = systolic_next(a, np), pb = systolic_next(b, np);
          const int pc = systolic_next(cc, np), pd = systolic_next(d, np);
          Tn[pa * ld + pc] = cl * yac - sl * yad; Tn[pa * ld + pd] = sl * yac + cl * yad;
          Tn[pb * ld + pc] = cl * ybc - sl * ybd; Tn[pb * ld + pd] = sl * ybc + cl * ybd;
        } else {
          const int q = idx - nb2;
          const int x = q / np, l = q - x * np;
          const int cc = l, d = np + l;
          const double laa = T[cc * ld + cc], lbb = T[d * ld + d], lab = T[cc * ld + d];
          const double va = J[x * ld + cc], vb = J[x * ld + d];
          double cl, sl;
          (void)rotation_of(laa, lbb, lab, cl, sl);
          Jn[x * ld + systolic_next(cc, np)] = cl * va - sl * vb;
          Jn[x * ld + systolic_next(d, np)] = sl * va + cl * vb;
        }
      }
      c.sync();
      { double* t = T; T = Tn; Tn = t; }
      { double* t = J; J = Jn; Jn = t; }
    }
    const int again = *big;
    c.sync();
    if (!again) { ++sweep; break; }
  }
  *Tio = T; *Taltio = Tn; *Jio = J; *Jaltio = Jn;
  return sweep;
}

#ifndef FA_IRLS_HOST
// More than 8 pairs, at most 32 (device only).  This thread's items are tid + u * nt: 2x2 blocks of T (kMT of
// them) and (row, pair) items of J (kMJ).  Per item: the offset of its first element, the offsets
// its results are stored at, and the pairs whose rotations it needs; offsets are below 2^16
// (matrices of at most 64 x 65 doubles) and are kept two to a register.
template <int kMT, int kMJ>
FA_FN int jacobi_large(const Ctx& c, const Smem& s, double** Tio, double** Taltio, double** Jio, double** Jaltio,
                       int dim, int jrows) {
  const int ld = s.ld;
  const int pp = (dim + 1) & ~1;
  const int np = pp >> 1;
  double* T = *Tio;
  double* Tn = *Taltio;
  double* J = *Jio;
  double* Jn = *Jaltio;
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
  int sweep = 0;
  if (c.tid == 0) { s.flags[0] = 0; s.flags[3] = 0; }
  c.sync();
  for (; sweep < kMaxSweeps; ++sweep) {
    int* big = &s.flags[(sweep & 1) ? 3 : 0];
    if (c.tid == 0) s.flags[(sweep & 1) ? 0 : 3] = 0;
    for (int rd = 0; rd < pp - 1; ++rd) {
      // every warp works out all np <= 32 rotations itself, lane q the one of pair q; the items then
      // fetch the two (one) they need with shuffles: no second barrier, no waiting for one warp
      const int lane = c.tid & 31;
      double x0[kMT], x1[kMT], x2[kMT], x3[kMT], v0[kMJ], v1[kMJ];
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
      double cq = 1.0, sq = 0.0;
      if (lane < np) {
        const int o = lane * (ld + 1);
        if (rotation_of(T[o], T[o + np * (ld + 1)], T[o + np], cq, sq) && c.tid < np) *big = 1;
      }
#pragma unroll
      for (int u = 0; u < kMT; ++u) {
        const int tk = (tdesc0[u] >> 16) & 0xffu, tl = tdesc0[u] >> 24;
        const double ck = __shfl_sync(0xffffffffu, cq, tk), sk = __shfl_sync(0xffffffffu, sq, tk);
        const double cl = __shfl_sync(0xffffffffu, cq, tl), sl = __shfl_sync(0xffffffffu, sq, tl);
        if (tv[u]) {
          const double yac = ck * x0[u] - sk * x2[u], yad = ck * x1[u] - sk * x3[u];
          const double ybc = sk * x0[u] + ck * x2[u], ybd = sk * x1[u] + ck * x3[u];
          Tn[tdesc1[u] & 0xffffu] = cl * yac - sl * yad; Tn[tdesc1[u] >> 16] = sl * yac + cl * yad;
          Tn[tdesc2[u] & 0xffffu] = cl * ybc - sl * ybd; Tn[tdesc2[u] >> 16] = sl * ybc + cl * ybd;
        }
      }
#pragma unroll
      for (int u = 0; u < kMJ; ++u) {
        const int jl = jdesc0[u] >> 16;
        const double cl = __shfl_sync(0xffffffffu, cq, jl), sl = __shfl_sync(0xffffffffu, sq, jl);
        if (jv[u]) {
          Jn[jdesc1[u] & 0xffffu] = cl * v0[u] - sl * v1[u];
          Jn[jdesc1[u] >> 16] = sl * v0[u] + cl * v1[u];
        }
      }
      if (lane < np) { s.rc[lane] = cq; s.rs[lane] = sq; }     // same values from every warp: for the loops below
      // items beyond the per-thread lists (a smaller block than expected): offsets on the fly
      if (kMT * c.nt < np * np || kMJ * c.nt < jrows * np) c.sync();
      for (int idx = c.tid + kMT * c.nt; idx < np * np; idx += c.nt) {
        const int k = idx / np, l = idx - k * np;
        const int a = k, b = np + k, cc = l, d = np + l;
        const double ck = s.rc[k], sk = s.rs[k], cl = s.rc[l], sl = s.rs[l];
        const double xac = T[a * ld + cc], xad = T[a * ld + d], xbc = T[b * ld + cc], xbd = T[b * ld + d];
        const double yac = ck * xac - sk * xbc, yad = ck * xad - sk * xbd;
        const double ybc = sk * xac + ck * xbc, ybd = sk * xad + ck * xbd;
        const int pa = systolic_next(a, np), pb = systolic_next(b, np);
        const int pc = systolic_next(cc, np), pd = systolic_next(d, np);
        Tn[pa * ld + pc] = cl * yac - sl * yad; Tn[pa * ld + pd] = sl * yac + cl * yad;
        Tn[pb * ld + pc] = cl * ybc - sl * ybd; Tn[pb * ld + pd] = sl * ybc + cl * ybd;
      }
      for (int idx = c.tid + kMJ * c.nt; idx < jrows * np; idx += c.nt) {
        const int x = idx / np, l = idx - x * np;
        const int cc = l, d = np + l;
        const double cl = s.rc[l], sl = s.rs[l];
        const double va = J[x * ld + cc], vb = J[x * ld + d];
        Jn[x * ld + systolic_next(cc, np)] = cl * va - sl * vb;
        Jn[x * ld + systolic_next(d, np)] = sl * va + cl * vb;
      }
      c.sync();
      { double* t = T; T = Tn; Tn = t; }
      { double* t = J; J = Jn; Jn = t; }
    }
    const int again = *big;
    c.sync();
    if (!again) { ++sweep; break; }
  }
  *Tio = T; *Taltio = Tn; *Jio = J; *Jaltio = Jn;
  return sweep;
}
#endif

template <bool LARGE>
FA_FN int jacobi(const Ctx& c, const Smem& s, double** Tio, double** Taltio, double** Jio, double** Jaltio, int dim,
                 int jrows) {
  if (dim < 2) return 0;
#ifndef FA_IRLS_HOST
  // item slots per thread are compile-time (slots without an item still cost their instructions):
  // one of each up to 16 pairs with 512 threads, two blocks and four J items up to 32 pairs
  const int np = (dim + 1) >> 1;
  if (LARGE && np > 8) {
    if (np * np <= c.nt && jrows * np <= c.nt) return jacobi_large<1, 1>(c, s, Tio, Taltio, Jio, Jaltio, dim, jrows);
    return jacobi_large<2, 4>(c, s, Tio, Taltio, Jio, Jaltio, dim, jrows);
  }
#endif
  return jacobi_small(c, s, Tio, Taltio, Jio, Jaltio, dim, jrows);
}

// ev[k] = T[k][k]; ord[q] = index of the q-th largest (ties by index).  All threads return
// the number of eigenvalues > kRankRel * largest among the first `limit` in that order.
FA_FN int sort_eigs(const Ctx& c, const Smem& s, const double* T, int dim, int limit) {
  const int ld = s.ld;
  for (int k = c.tid; k < dim; k += c.nt) s.ev[k] = T[k * ld + k];
  c.sync();
  for (int k = c.tid; k < dim; k += c.nt) {
    double e = s.ev[k];
    int rank = 0;
    for (int l = 0; l < dim; ++l) {
      double o = s.ev[l];
      rank += (o > e || (o == e && l < k)) ? 1 : 0;
    }
    s.ord[rank] = k;
  }
  c.sync();
  double top = s.ev[s.ord[0]];
  int keep = 0;
  if (top > 0.0) {
    int lim = limit < dim ? limit : dim;
    for (int q = 0; q < lim; ++q) keep += (s.ev[s.ord[q]] > kRankRel * top) ? 1 : 0;
  }
  return keep;
}

// One term of the objective with value u (the quantity under the root in Eq. (5)): its
// contribution u^(1/a) and the factor max(u^(1 - 1/a), eps) of its reweighting (Eq. (4) with
// constant a; a = 2 gives the square roots of Eq. (5) and takes the sqrt fast path).
FA_FN void term_of(double u, double a, double& contrib, double& denom) {
  if (a == 2.0) { contrib = sqrt(u); denom = fmax(contrib, kEps); }
  else if (u <= 0.0) { contrib = 0.0; denom = kEps; }
  else { contrib = pow(u, 1.0 / a); denom = fmax(pow(u, 1.0 - 1.0 / a), kEps); }
}

// From residual coordinates Res (rows k0..r-1 are the part of f_i outside the subspace) and the
// full coordinates P: u_i, next data weights w_i, the matrix M of the next weighted PCA and the
// value of Eq. (5).  `uniform` builds the round-one weights instead (u is not needed then).
//
// cb, ca: the data term of worker i is cb (1 - v_i)^(1/a) + ca v_i^(1/a) -- a Beta(alpha, beta)
// likelihood of the values with cb = 2 (1 - beta), ca = 2 (1 - alpha); Eq. (1) has alpha = 1,
// beta = 1/2, i.e. cb = 1, ca = 0.  With ca > 0 a weight can be negative.
FA_FN double weights_and_objective(const Ctx& c, Smem& s, const double* Res, int k0, int r, int p,
                                   double coef, bool uniform, double a, double cb = 1.0, double ca = 0.0) {
  const int ld = s.ld;
  double part = 0.0;
  for (int i = c.tid; i < p; i += c.nt) {
    double ui = 0.0, wi = 0.0;
    if (s.dinv[i] != 0.0) {
      if (uniform) wi = 1.0;
      else {
        double acc = 0.0;
        for (int k = k0; k < r; ++k) { double v = Res[k * ld + i]; acc += v * v; }
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
    // off-diagonal entries M_ij = -2 w_ij (ordered pairs: each unordered pair counted twice)
    for (int idx = c.tid; idx < p * p; idx += c.nt) {
      int i = idx / p, j = idx - i * p;
      if (i == j) continue;
      double d2 = 0.0, res2 = 0.0;
      for (int k = 0; k < r; ++k) { double v = s.P[k * ld + i] - s.P[k * ld + j]; d2 += v * v; }
      double wij = 0.0;
      if (d2 > kSamePairRel * (s.fn[i] + s.fn[j])) {
        if (uniform) wij = coef;
        else {
          for (int k = k0; k < r; ++k) { double v = Res[k * ld + i] - Res[k * ld + j]; res2 += v * v; }
          if (a == 2.0) {
            const double y = res2 > 0.0 ? FA_RSQRT(res2 * d2) : 0.0;     // sqrt(u) = res2 y, 1/(d2 sqrt(u)) = y
            const double contrib = res2 * y;
            part += coef * contrib;
            wij = contrib >= kEps ? coef * y : coef / (d2 * kEps);
          } else {
            double contrib, denom;
            term_of(res2 / d2, a, contrib, denom);
            part += coef * contrib;
            wij = coef / (d2 * denom);
          }
        }
      }
      s.M[i * ld + j] = -2.0 * wij;
    }
    c.sync();
    for (int i = c.tid; i < p; i += c.nt) {
      double acc = 0.0;
      for (int j = 0; j < p; ++j) if (j != i) acc -= s.M[i * ld + j];
      s.M[i * ld + i] = s.w[i] + acc;
    }
  }
  double obj = block_sum(c, s, part);   // contains the barriers that publish M and w
  return obj;
}

// The same for workers that hold several gradients each (rows of one worker are consecutive):
// the value of worker i is 1 - tr(Y^T g_i g_i^T Y) / tr(g_i^T g_i) (appendix restatement of Eq. (5)),
// one weight per worker multiplies all of its rows, and the pair terms of the regulariser are taken
// between the workers' mean gradients.  `p` is the number of rows.  s.T and s.J are scratch here
// (mean coordinates of every worker: all of them, and the residual part).
FA_FN double weights_and_objective_grouped(const Ctx& c, Smem& s, const double* Res, int k0, int r, int p,
                                           double coef, bool uniform, double a) {
  const int ld = s.ld, nw = s.nw;
  double* Fm = s.T;
  double* Rm = s.J;
  double part = 0.0;
  double gmax = 0.0;
  for (int i = 0; i < nw; ++i) gmax = fmax(gmax, s.gtr[i]);
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
  for (int row = c.tid; row < p; row += c.nt) { s.w[row] = s.gw[s.grp[row]]; s.u[row] = s.gu[s.grp[row]]; }
  if (coef > 0.0) {
    // rows of different workers i != j: M = -2 w_ij / (k_i k_j)  (ordered pairs: each pair twice)
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
  for (int i = c.tid; i < p * m; i += c.nt) if (o.A) o.A[i] = 0.0;
  for (int i = c.tid; i < p; i += c.nt) if (o.c) o.c[i] = 0.f;
  for (int i = c.tid; i < nweights; i += c.nt) if (o.w) o.w[i] = 0.0;
  for (int i = c.tid; i < iters; i += c.nt) if (o.obj) o.obj[i] = 0.0;
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
template <bool LARGE>
FA_FN int run(const Ctx& c, Smem& s, const double* K, int p, int m, double lambda, double a, int iters,
              int start, const double* A0, double tol, const Outputs& o, int nw = 0,
              const unsigned char* cnt = nullptr, double cb = 1.0, double ca = 0.0) {
  const int ld = s.ld;
  const int pp = (p + 1) & ~1;
  int status = 0;

  // ---- load K, reject non-finite input
  if (c.tid == 0) { s.flags[1] = 0; }
  c.sync();
  for (int idx = c.tid; idx < pp * ld; idx += c.nt) { s.T[idx] = 0.0; s.J[idx] = 0.0; s.Aacc[idx] = 0.0; s.P[idx] = 0.0; s.M[idx] = 0.0; s.tmp[idx] = 0.0; }
  c.sync();
  for (int idx = c.tid; idx < p * p; idx += c.nt) {
    int i = idx / p, j = idx - i * p;
    double v = K[idx];
    if (!(fabs(v) <= 1.7e308)) s.flags[1] = 1;
    s.T[i * ld + j] = v;
  }
  c.sync();
  if (s.flags[1]) {
    write_zero_outputs(c, o, p, m, iters, nw > 0 ? nw : p);
    return ST_NONFINITE;
  }
  for (int i = c.tid; i < p; i += c.nt) s.kd[i] = s.T[i * ld + i];
  c.sync();
  double kmax = 0.0;
  for (int i = 0; i < p; ++i) kmax = fmax(kmax, s.kd[i]);
  if (!(kmax > 0.0)) {
    write_zero_outputs(c, o, p, m, iters, nw > 0 ? nw : p);
    return ST_RANK0;
  }
  for (int i = c.tid; i < p; i += c.nt)
    s.dinv[i] = (s.kd[i] <= kZeroNormRel * kmax) ? 0.0 : 1.0 / sqrt(s.kd[i]);
  c.sync();

  // ---- Kt = D^-1 K D^-1 (symmetrised, unit diagonal) -> tmp
  for (int idx = c.tid; idx < p * p; idx += c.nt) {
    int i = idx / p, j = idx - i * p;
    if (j < i) continue;
    double v = (i == j) ? (s.dinv[i] != 0.0 ? 1.0 : 0.0)
                        : 0.5 * (s.T[i * ld + j] + s.T[j * ld + i]) * s.dinv[i] * s.dinv[j];
    s.tmp[i * ld + j] = v; s.tmp[j * ld + i] = v;
  }
  // remaining diagonal of the factorisation -> u; "already a pivot" marks -> ord (as flags)
  for (int i = c.tid; i < p; i += c.nt) { s.u[i] = (s.dinv[i] != 0.0) ? 1.0 : 0.0; s.ord[i] = 0; }
  c.sync();

  // ---- Cholesky with complete pivoting, Kt = R^T R, R (r x p) kept in P with the original column
  // order: column i of R is the image f_i / ||g_i|| of worker i in R^r.  Stops when the largest
  // remaining diagonal entry is <= kRankRel (the diagonal of Kt is 1), which fixes the rank r.
  int r = 0;
  for (int k = 0; k < p; ++k) {
    int piv = -1;
    double dmax = kRankRel;
#ifndef FA_IRLS_HOST
    if (p > 32) {
      // every warp finds the pivot itself (two candidates per lane, butterfly); ties go to the lowest index
      for (int j = (c.tid & 31); j < p; j += 32) {
        const double dj = s.u[j];
        if (s.ord[j] == 0 && dj > dmax) { dmax = dj; piv = j; }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const double od = __shfl_xor_sync(0xffffffffu, dmax, off);
        const int oi = __shfl_xor_sync(0xffffffffu, piv, off);
        if (od > dmax || (od == dmax && oi >= 0 && (piv < 0 || oi < piv))) { dmax = od; piv = oi; }
      }
    } else
#endif
    {
      for (int j = 0; j < p; ++j) {               // every thread scans; ties go to the lowest index
        const double dj = s.u[j];
        if (s.ord[j] == 0 && dj > dmax) { dmax = dj; piv = j; }
      }
    }
    if (piv < 0) break;
    const double rinv = FA_RSQRT(dmax), rkk = dmax * rinv;   // dmax in (1e-12, 1]: a normal number
    for (int j = c.tid; j < p; j += c.nt) {
      double v;
      if (j == piv) v = rkk;
      else if (s.ord[j] != 0) v = 0.0;
      else {
        double acc = s.tmp[piv * ld + j];
        for (int l = 0; l < k; ++l) acc -= s.P[l * ld + piv] * s.P[l * ld + j];
        v = acc * rinv;
      }
      s.P[k * ld + j] = v;
    }
    if (c.tid == 0) s.wused[k] = (double)piv;     // pivot order (exact small integers)
    c.sync();
    for (int j = c.tid; j < p; j += c.nt) {
      if (j == piv) { s.ord[j] = 1; s.u[j] = 0.0; }
      else if (s.ord[j] == 0) { const double v = s.P[k * ld + j]; s.u[j] = fmax(s.u[j] - v * v, 0.0); }
    }
    c.sync();
    r = k + 1;
  }

  // ---- U = R11^-1 (R11 = pivot columns of R, upper triangular) by back substitution, one column
  // per thread -> J buffer.  Q = G D^-1 X with X[piv_a][:] = U[a][:] has orthonormal columns and
  // Q^T g_i = f_i, so Aacc starts as D^-1 X (p x r).
  for (int bcol = c.tid; bcol < r; bcol += c.nt) {
    for (int a = bcol; a >= 0; --a) {
      const int pa = (int)s.wused[a];
      double acc = (a == bcol) ? 1.0 : 0.0;
      for (int l = a + 1; l <= bcol; ++l) acc -= s.P[a * ld + (int)s.wused[l]] * s.J[l * ld + bcol];
      s.J[a * ld + bcol] = acc / s.P[a * ld + pa];
    }
  }
  c.sync();
  for (int idx = c.tid; idx < r * r; idx += c.nt) {
    const int a = idx / r, bcol = idx - a * r;
    if (bcol >= a) {
      const int pa = (int)s.wused[a];
      s.Aacc[pa * ld + bcol] = s.dinv[pa] * s.J[a * ld + bcol];
    }
  }
  // ---- P = F: scale column i of R back by ||g_i||
  for (int idx = c.tid; idx < r * p; idx += c.nt) {
    const int k = idx / p, i = idx - k * p;
    s.P[k * ld + i] = (s.dinv[i] != 0.0) ? s.P[k * ld + i] / s.dinv[i] : 0.0;
  }
  c.sync();
  int sw = 0;
  for (int i = c.tid; i < p; i += c.nt) {
    double acc = 0.0;
    for (int k = 0; k < r; ++k) { double v = s.P[k * ld + i]; acc += v * v; }
    s.fn[i] = acc;
  }
  c.sync();

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
    for (int idx = c.tid; idx < r * m; idx += c.nt) {
      int k = idx / m, q = idx - k * m;
      double acc = 0.0;
      for (int i = 0; i < p; ++i) acc += s.P[k * ld + i] * A0[i * m + q];
      s.J[k * ld + q] = acc;
    }
    c.sync();
    if (start == 2) {
      // W = Z0^T Z0 -> T; Cholesky W = L L^T by one thread; Z = Z0 L^-T row by row
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
    if (grouped) (void)weights_and_objective_grouped(c, s, s.P, 0, r, p, coef, true, a);
    else (void)weights_and_objective(c, s, s.P, 0, r, p, coef, true, a, cb, ca);
  } else {
    // C = Z0^T F (m x p) -> T buffer; Res = F - Z0 C -> tmp
    for (int idx = c.tid; idx < m * p; idx += c.nt) {
      int q = idx / p, i = idx - q * p;
      double acc = 0.0;
      for (int k = 0; k < r; ++k) acc += s.J[k * ld + q] * s.P[k * ld + i];
      s.T[q * ld + i] = acc;
    }
    c.sync();
    for (int idx = c.tid; idx < r * p; idx += c.nt) {
      int k = idx / p, i = idx - k * p;
      double acc = s.P[k * ld + i];
      for (int q = 0; q < m; ++q) acc -= s.J[k * ld + q] * s.T[q * ld + i];
      s.tmp[k * ld + i] = acc;
    }
    c.sync();
    if (grouped) (void)weights_and_objective_grouped(c, s, s.tmp, 0, r, p, coef, false, a);
    else (void)weights_and_objective(c, s, s.tmp, 0, r, p, coef, false, a, cb, ca);
  }

  int m_eff = 0, rounds = iters;
  double prev_obj = 0.0;
  for (int t = 0; t < iters; ++t) {
    for (int i = c.tid; i < p; i += c.nt) s.wused[i] = s.w[i];
    if (grouped) for (int i = c.tid; i < nw; i += c.nt) s.gwused[i] = s.gw[i];
    // ---- T = P M P^T (current basis)
    if (coef > 0.0) {
      for (int idx = c.tid; idx < p * r; idx += c.nt) {       // tmp[i][a] = sum_j M[i][j] P[a][j]
        int i = idx / r, a = idx - i * r;
        double acc = 0.0;
        for (int j = 0; j < p; ++j) acc += s.M[i * ld + j] * s.P[a * ld + j];
        s.tmp[i * ld + a] = acc;
      }
      c.sync();
      for (int idx = c.tid; idx < r * r; idx += c.nt) {
        int a = idx / r, b = idx - a * r;
        if (b < a) continue;
        double acc = 0.0;
        for (int i = 0; i < p; ++i) acc += s.P[a * ld + i] * s.tmp[i * ld + b];
        s.T[a * ld + b] = acc; s.T[b * ld + a] = acc;
      }
    } else {
      for (int idx = c.tid; idx < r * r; idx += c.nt) {
        int a = idx / r, b = idx - a * r;
        if (b < a) continue;
        double acc = 0.0;
        for (int i = 0; i < p; ++i) acc += s.w[i] * s.P[a * ld + i] * s.P[b * ld + i];
        s.T[a * ld + b] = acc; s.T[b * ld + a] = acc;
      }
    }
    for (int idx = c.tid; idx < pp * pp; idx += c.nt) {
      int a = idx / pp, b = idx - a * pp;
      s.J[a * ld + b] = (a == b) ? 1.0 : 0.0;
      if (a >= r || b >= r) s.T[a * ld + b] = 0.0;
    }
    c.sync();
    sw = jacobi<LARGE>(c, s, &s.T, &s.tmp, &s.J, &s.M, r, r);   // M is free until the next weights
    if (sw >= kMaxSweeps) status |= ST_EIG_SWEEPS;
    m_eff = sort_eigs(c, s, s.T, r, m);

    // ---- rotate into the new (sorted) eigenbasis: P <- J^T P, Aacc <- Aacc J
    for (int idx = c.tid; idx < r * p; idx += c.nt) {
      int k = idx / p, i = idx - k * p;
      int col = s.ord[k];
      double acc = 0.0;
      for (int l = 0; l < r; ++l) acc += s.J[l * ld + col] * s.P[l * ld + i];
      s.tmp[k * ld + i] = acc;
    }
    for (int idx = c.tid; idx < p * r; idx += c.nt) {
      int i = idx / r, k = idx - i * r;
      int col = s.ord[k];
      double acc = 0.0;
      for (int l = 0; l < r; ++l) acc += s.Aacc[i * ld + l] * s.J[l * ld + col];
      s.M[i * ld + k] = acc;
    }
    c.sync();
    { double* x = s.P; s.P = s.tmp; s.tmp = x; }
    { double* x = s.Aacc; s.Aacc = s.M; s.M = x; }

    // ---- terms of Eq. (5) at the new subspace, and the next round's weights
    double obj = grouped ? weights_and_objective_grouped(c, s, s.P, m_eff, r, p, coef, false, a)
                         : weights_and_objective(c, s, s.P, m_eff, r, p, coef, false, a, cb, ca);
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
    for (int idx = c.tid; idx < p * p; idx += c.nt) {
      const int i = idx / p, j = idx - i * p;
      double acc = 0.0;
      for (int k = 0; k < m_eff; ++k) acc += s.Aacc[i * ld + k] * s.P[k * ld + j];
      o.S[idx] = acc;
    }
  }
  if (o.c) {
    for (int k = c.tid; k < m_eff; k += c.nt) {        // s_k = sum_j P[k][j]  (Z^T F 1)
      double acc = 0.0;
      if (grouped) for (int j = 0; j < p; ++j) acc += s.P[k * ld + j] * s.ginv[s.grp[j]];   // sum of worker means
      else for (int j = 0; j < p; ++j) acc += s.P[k * ld + j];
      s.ev[k] = acc;
    }
    c.sync();
    for (int i = c.tid; i < p; i += c.nt) {
      double acc = 0.0;
      for (int k = 0; k < m_eff; ++k) acc += s.Aacc[i * ld + k] * s.ev[k];
      o.c[i] = (float)(acc / (double)workers);
    }
  }
  return status;
}

}  // namespace fa_irls
