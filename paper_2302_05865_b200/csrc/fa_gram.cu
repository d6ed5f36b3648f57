// Gram pass: K_ij = <g_i, g_j> in one streaming read of the worker-major gradient matrix
// (Section 2.1: ||g_i||^2 = K_ii; Section 2.3: D_ij^2 = K_ii + K_jj - 2 K_ij).
//
// One persistent block per SM.  A producer warp stages column tiles of all p rows in shared
// memory with one 1-D bulk copy (TMA) per row and tile, through a ring of mbarrier-guarded
// stages; rows may start at any element-aligned address, so each row is copied from its
// 16-byte-aligned start and read back with a per-row byte skew.  Eight consumer warps form the
// products in fp32 (exact for bf16 inputs, correctly rounded for fp32 inputs), keep fp32 running
// sums over at most kFlushCols columns, then fold them with a warp butterfly into fp64 lane
// accumulators.  Block totals go to the workspace; the last block to finish adds them up in a
// fixed order and writes K, so the result is bit-reproducible and no second launch is needed.
#include "fa_common.cuh"
#include "fa_gram_finish.cuh"
#include "fa_kernels.h"

namespace fa {
namespace gram {

constexpr int kConsumerWarps = 8;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kThreads = kConsumers + 32;   // + producer warp
constexpr int kStages = 3;
constexpr int kFlushCols = 64;              // fp32 running sums cover at most this many columns
constexpr int kTriWarps = 11;               // consumer warps of the p <= 16 kernel (384 threads with the producer)

struct Params {
  const char* G;
  long long n;
  int p;
  int tile_cols;       // columns per tile
  int row_stride;      // bytes between staged rows
  long long num_tiles;
  double* partials;    // [p(p+1)/2][gridDim.x]: entry c (canonical upper-triangle order) of block b at c*gridDim.x + b
  unsigned int* counter;   // blocks finished so far (zero at launch)
  double* K;           // out: p x p, written by the last block to finish
  int* status;
};

struct Ring {
  uint64_t* full;
  uint64_t* empty;
  int* abort;
};

// ---- producer: runs in warp kConsumerWarps, all 32 lanes
template <int S>
__device__ __forceinline__ void producer(const Params& prm, char* stages, int stage_bytes, Ring ring, int lane) {
  const char* Gend = prm.G + (size_t)prm.p * (size_t)prm.n * S;
  long long use = 0;
  bool ok = true;
  for (long long t = blockIdx.x; t < prm.num_tiles && ok; t += gridDim.x, ++use) {
    const int s = static_cast<int>(use % kStages);
    const uint32_t par = static_cast<uint32_t>((use / kStages) & 1);
    if (!mbar_wait(&ring.empty[s], par ^ 1u)) { ok = false; break; }
    if (*reinterpret_cast<volatile int*>(ring.abort)) { ok = false; break; }
    const long long j0 = t * (long long)prm.tile_cols;
    const int tc = static_cast<int>(min((long long)prm.tile_cols, prm.n - j0));
    char* sbase = stages + (size_t)s * stage_bytes;
    uint32_t mybytes = 0;
    // rows whose aligned span would leave the matrix are staged with plain loads
    for (int i = lane; i < prm.p; i += 32) {
      const char* addr = prm.G + ((size_t)i * (size_t)prm.n + (size_t)j0) * S;
      const uint32_t skew = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(addr) & 15u);
      const char* src = addr - skew;
      const uint32_t bytes = (skew + (uint32_t)tc * S + 15u) & ~15u;
      if (src < prm.G || src + bytes > Gend) {
        char* dst = sbase + (size_t)i * prm.row_stride + skew;
        for (int c = 0; c < tc * S; ++c) dst[c] = addr[c];
        fence_proxy_async();      // later bulk copies into this row are ordered after these stores
      } else {
        mybytes += bytes;
      }
    }
    uint32_t total = mybytes;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) total += __shfl_xor_sync(0xffffffffu, total, off);
    __syncwarp();
    if (lane == 0) mbar_arrive_expect_tx(&ring.full[s], total);
    __syncwarp();
    for (int i = lane; i < prm.p; i += 32) {
      const char* addr = prm.G + ((size_t)i * (size_t)prm.n + (size_t)j0) * S;
      const uint32_t skew = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(addr) & 15u);
      const char* src = addr - skew;
      const uint32_t bytes = (skew + (uint32_t)tc * S + 15u) & ~15u;
      if (!(src < prm.G || src + bytes > Gend))
        bulk_g2s(sbase + (size_t)i * prm.row_stride, src, bytes, &ring.full[s]);
    }
  }
  if (!ok) {
    if (lane == 0) {
      *ring.abort = 1;
      if (prm.status) atomicOr(prm.status, kStTimeout);
      // let copies already in flight land before the block can exit
      long long first = use > kStages ? use - kStages : 0;
      for (long long u = first; u < use; ++u)
        (void)mbar_wait(&ring.full[u % kStages], static_cast<uint32_t>((u / kStages) & 1));
    }
  }
}

// ---- consumers, p <= 16: every thread keeps the whole upper triangle for its columns
template <typename T, int V, int PB, int CW>
__device__ __forceinline__ void consume_tri(const Params& prm, const char* stages, int stage_bytes, Ring ring,
                                            double* totals, int ctid) {
  constexpr int S = sizeof(T);
  constexpr int NACC = PB * (PB + 1) / 2;
  constexpr int NACCP = (NACC + 31) / 32 * 32;
  const int lane = ctid & 31, warp = ctid >> 5;
  float acc[NACCP];
  double dacc[NACCP / 32];
#pragma unroll
  for (int k = 0; k < NACCP; ++k) acc[k] = 0.f;
#pragma unroll
  for (int k = 0; k < NACCP / 32; ++k) dacc[k] = 0.0;
  int rowoff[PB];
#pragma unroll
  for (int i = 0; i < PB; ++i) {
    const int ii = i < prm.p ? i : 0;     // rows >= p read row 0's skew; their stage rows are zero
    rowoff[i] = i * prm.row_stride +
                static_cast<int>(reinterpret_cast<uintptr_t>(prm.G + (size_t)ii * (size_t)prm.n * S) & 15u);
  }
  int since = 0;
  long long use = 0;
  for (long long t = blockIdx.x; t < prm.num_tiles; t += gridDim.x, ++use) {
    const int s = static_cast<int>(use % kStages);
    if (!mbar_wait(&ring.full[s], static_cast<uint32_t>((use / kStages) & 1))) {
      if (lane == 0) { *ring.abort = 1; if (prm.status) atomicOr(prm.status, kStTimeout); }
      break;
    }
    const long long j0 = t * (long long)prm.tile_cols;
    const int tc = static_cast<int>(min((long long)prm.tile_cols, prm.n - j0));
    const char* sbase = stages + (size_t)s * stage_bytes;
    const int ncg = (tc + V - 1) / V;
    const bool ragged = (tc % V) != 0;
    for (int cg = ctid; cg < ncg; cg += CW * 32) {
      float x[PB][V];
#pragma unroll
      for (int i = 0; i < PB; ++i) SmemVec<T, V>::load(sbase + rowoff[i] + cg * (V * S), x[i]);
      if (ragged && cg == ncg - 1) {
#pragma unroll
        for (int e = 0; e < V; ++e)
          if (cg * V + e >= tc) {
#pragma unroll
            for (int i = 0; i < PB; ++i) x[i][e] = 0.f;
          }
      }
      int idx = 0;
#pragma unroll
      for (int i = 0; i < PB; ++i)
#pragma unroll
        for (int j = i; j < PB; ++j) {
#pragma unroll
          for (int e = 0; e < V; ++e) acc[idx] = fmaf(x[i][e], x[j][e], acc[idx]);
          ++idx;
        }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&ring.empty[s]);
    since += (prm.tile_cols / V + CW * 32 - 1) / (CW * 32) * V;
    if (since >= kFlushCols) { flush<NACCP>(acc, dacc, lane); since = 0; }
  }
  flush<NACCP>(acc, dacc, lane);
#pragma unroll
  for (int k = 0; k < NACCP / 32; ++k) totals[warp * NACCP + lane * (NACCP / 32) + k] = dacc[k];
}

template <typename T, int V, int PB, int CW>
__global__ void __launch_bounds__((CW + 1) * 32, 1) gram_tri_kernel(Params prm) {
  constexpr int kThreads = (CW + 1) * 32;
  constexpr int kConsumers = CW * 32;
  constexpr int kConsumerWarps = CW;
  constexpr int S = sizeof(T);
  constexpr int NACC = PB * (PB + 1) / 2;
  constexpr int NACCP = (NACC + 31) / 32 * 32;
  extern __shared__ __align__(128) char smem[];
  const int stage_bytes = PB * prm.row_stride;
  char* stages = smem;
  double* totals = reinterpret_cast<double*>(smem + (size_t)kStages * stage_bytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(totals + kConsumerWarps * NACCP);
  Ring ring{bars, bars + kStages, reinterpret_cast<int*>(bars + 2 * kStages)};
  const int tid = threadIdx.x;

  // rows >= p of every stage must read as zero; nothing ever writes them again
  for (int i = tid * 16; i < kStages * stage_bytes; i += kThreads * 16)
    *reinterpret_cast<uint4*>(stages + i) = make_uint4(0, 0, 0, 0);
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&ring.full[s], 1); mbar_init(&ring.empty[s], kConsumerWarps); }
    *ring.abort = 0;
  }
  fence_proxy_async();
  __syncthreads();

  if (tid >= kConsumers) producer<S>(prm, stages, stage_bytes, ring, tid - kConsumers);
  else consume_tri<T, V, PB, CW>(prm, stages, stage_bytes, ring, totals, tid);
  __syncthreads();

  // block total (fixed warp order) -> this block's entries, then the last block forms K
  for (int e = tid; e < NACC; e += kThreads) {
    int i = 0, r = e;
    while (r >= PB - i) { r -= PB - i; ++i; }
    const int j = i + r;
    if (j < prm.p) {
      double sum = 0.0;
      for (int w = 0; w < kConsumerWarps; ++w) sum += totals[w * NACCP + e];
      prm.partials[(size_t)canon_index(i, j, prm.p) * gridDim.x + blockIdx.x] = sum;
    }
  }
  finish_gram(prm.partials, prm.counter, prm.K, prm.p, ring.abort);
}

// ---- consumers, 16 < p <= 64: rows are cut into blocks of 16; a work item is the triangle of
// one block (136 sums) or an 8 x 16 rectangle between two blocks (128 sums).  NB*NB items.
constexpr int kItemAcc = 160;   // 136 rounded up to a multiple of 32

template <int NB>
__device__ __forceinline__ void item_rows(int item, bool& tri, int& i0, int& j0) {
  if (item < NB) { tri = true; i0 = j0 = 16 * item; return; }
  tri = false;
  int q = item - NB;            // (a, b, half) with a < b
  const int half = q & 1; q >>= 1;
  int a = 0;
  while (q >= NB - 1 - a) { q -= NB - 1 - a; ++a; }
  const int b = a + 1 + q;
  i0 = 16 * a + 8 * half;
  j0 = 16 * b;
}

template <typename T>
__device__ __forceinline__ void item_accumulate(bool tri, const char* sbase, const int* rowoff_s, int i0, int j0,
                                                int col, float (&acc)[kItemAcc]) {
  constexpr int S = sizeof(T);
  if (tri) {
    float x[16][1];
#pragma unroll
    for (int i = 0; i < 16; ++i) SmemVec<T, 1>::load(sbase + rowoff_s[i0 + i] + col * S, x[i]);
    int idx = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i)
#pragma unroll
      for (int j = i; j < 16; ++j) { acc[idx] = fmaf(x[i][0], x[j][0], acc[idx]); ++idx; }
  } else {
    float a[8][1], b[16][1];
#pragma unroll
    for (int i = 0; i < 8; ++i) SmemVec<T, 1>::load(sbase + rowoff_s[i0 + i] + col * S, a[i]);
#pragma unroll
    for (int j = 0; j < 16; ++j) SmemVec<T, 1>::load(sbase + rowoff_s[j0 + j] + col * S, b[j]);
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 16; ++j) acc[i * 16 + j] = fmaf(a[i][0], b[j][0], acc[i * 16 + j]);
  }
}

template <typename T, int NB>
__device__ __forceinline__ void consume_blocks(const Params& prm, const char* stages, int stage_bytes, Ring ring,
                                               double* totals, const int* rowoff_s, int ctid) {
  constexpr int W = NB * NB;                                   // work items
  constexpr int WPI = (W <= kConsumerWarps) ? kConsumerWarps / W : 1;   // warps per item
  constexpr int IPW = (W <= kConsumerWarps) ? 1 : W / kConsumerWarps;   // items per warp
  const int lane = ctid & 31, warp = ctid >> 5;
  float acc[kItemAcc];
  double dacc[IPW][kItemAcc / 32];
#pragma unroll
  for (int k = 0; k < kItemAcc; ++k) acc[k] = 0.f;
#pragma unroll
  for (int q = 0; q < IPW; ++q)
#pragma unroll
    for (int k = 0; k < kItemAcc / 32; ++k) dacc[q][k] = 0.0;
  int since = 0;
  long long use = 0;
  for (long long t = blockIdx.x; t < prm.num_tiles; t += gridDim.x, ++use) {
    const int s = static_cast<int>(use % kStages);
    if (!mbar_wait(&ring.full[s], static_cast<uint32_t>((use / kStages) & 1))) {
      if (lane == 0) { *ring.abort = 1; if (prm.status) atomicOr(prm.status, kStTimeout); }
      break;
    }
    const long long c0 = t * (long long)prm.tile_cols;
    const int tc = static_cast<int>(min((long long)prm.tile_cols, prm.n - c0));
    const char* sbase = stages + (size_t)s * stage_bytes;
    if constexpr (IPW == 1) {
      bool tri; int i0, j0;
      item_rows<NB>(warp % W, tri, i0, j0);
      const int sub = warp / W;
      for (int col = sub * 32 + lane; col < tc; col += 32 * WPI) item_accumulate<T>(tri, sbase, rowoff_s, i0, j0, col, acc);
      since += (prm.tile_cols + 32 * WPI - 1) / (32 * WPI);
      if (since >= kFlushCols) { flush<kItemAcc>(acc, dacc[0], lane); since = 0; }
    } else {
#pragma unroll
      for (int q = 0; q < IPW; ++q) {
        bool tri; int i0, j0;
        item_rows<NB>(warp + kConsumerWarps * q, tri, i0, j0);
        for (int col = lane; col < tc; col += 32) item_accumulate<T>(tri, sbase, rowoff_s, i0, j0, col, acc);
        flush<kItemAcc>(acc, dacc[q], lane);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&ring.empty[s]);
  }
  if constexpr (IPW == 1) flush<kItemAcc>(acc, dacc[0], lane);
#pragma unroll
  for (int q = 0; q < IPW; ++q)
#pragma unroll
    for (int k = 0; k < kItemAcc / 32; ++k)
      totals[(warp * IPW + q) * kItemAcc + lane * (kItemAcc / 32) + k] = dacc[q][k];
}

template <typename T, int NB>
__global__ void __launch_bounds__(kThreads, 1) gram_blocks_kernel(Params prm) {
  constexpr int S = sizeof(T);
  constexpr int ROWS = 16 * NB;
  constexpr int W = NB * NB;
  constexpr int WPI = (W <= kConsumerWarps) ? kConsumerWarps / W : 1;
  constexpr int IPW = (W <= kConsumerWarps) ? 1 : W / kConsumerWarps;
  extern __shared__ __align__(128) char smem[];
  const int stage_bytes = ROWS * prm.row_stride;
  char* stages = smem;
  double* totals = reinterpret_cast<double*>(smem + (size_t)kStages * stage_bytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(totals + kConsumerWarps * IPW * kItemAcc);
  Ring ring{bars, bars + kStages, reinterpret_cast<int*>(bars + 2 * kStages)};
  int* rowoff_s = reinterpret_cast<int*>(bars + 2 * kStages + 1);
  const int tid = threadIdx.x;

  for (int i = tid * 16; i < kStages * stage_bytes; i += kThreads * 16)
    *reinterpret_cast<uint4*>(stages + i) = make_uint4(0, 0, 0, 0);
  for (int i = tid; i < ROWS; i += kThreads) {
    const int ii = i < prm.p ? i : 0;
    rowoff_s[i] = i * prm.row_stride +
                  static_cast<int>(reinterpret_cast<uintptr_t>(prm.G + (size_t)ii * (size_t)prm.n * S) & 15u);
  }
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&ring.full[s], 1); mbar_init(&ring.empty[s], kConsumerWarps); }
    *ring.abort = 0;
  }
  fence_proxy_async();
  __syncthreads();

  if (tid >= kConsumers) producer<S>(prm, stages, stage_bytes, ring, tid - kConsumers);
  else consume_blocks<T, NB>(prm, stages, stage_bytes, ring, totals, rowoff_s, tid);
  __syncthreads();

  for (int idx = tid; idx < W * kItemAcc; idx += kThreads) {
    const int item = idx / kItemAcc, e = idx - item * kItemAcc;
    bool tri; int i0, j0;
    item_rows<NB>(item, tri, i0, j0);
    int gi, gj;
    if (tri) {
      if (e >= 136) continue;
      int i = 0, r = e;
      while (r >= 16 - i) { r -= 16 - i; ++i; }
      gi = i0 + i; gj = i0 + i + r;
    } else {
      if (e >= 128) continue;
      gi = i0 + e / 16; gj = j0 + e % 16;
    }
    if (gi >= prm.p || gj >= prm.p) continue;
    double sum = 0.0;
    if constexpr (IPW == 1) {
      for (int sub = 0; sub < WPI; ++sub) sum += totals[(size_t)(sub * W + item) * kItemAcc + e];
    } else {
      const int w = item % kConsumerWarps, q = item / kConsumerWarps;
      sum = totals[(size_t)(w * IPW + q) * kItemAcc + e];
    }
    prm.partials[(size_t)canon_index(gi, gj, prm.p) * gridDim.x + blockIdx.x] = sum;
  }
  finish_gram(prm.partials, prm.counter, prm.K, prm.p, ring.abort);
}

// ---- host side
struct Shape {
  int kind;        // 0: tri kernel with PB rows, 1: block kernel with NB blocks
  int pb_or_nb;
  int rows;        // staged rows
  int row_bytes;   // payload bytes per staged row and tile
  int naccp;       // doubles per warp slot in `totals`
  int ipw;
};

static Shape pick_shape(int p) {
  Shape s{};
  if (p <= 16) {
    int pb = p <= 4 ? 4 : p <= 8 ? 8 : p <= 12 ? 12 : p <= 15 ? 15 : 16;
    s.kind = 0; s.pb_or_nb = pb; s.rows = pb; s.row_bytes = 4096;
    s.naccp = (pb * (pb + 1) / 2 + 31) / 32 * 32; s.ipw = 1;
  } else if (p <= 32) {
    s.kind = 1; s.pb_or_nb = 2; s.rows = 32; s.row_bytes = 2048; s.naccp = kItemAcc; s.ipw = 1;
  } else {
    s.kind = 1; s.pb_or_nb = 4; s.rows = 64; s.row_bytes = 1024; s.naccp = kItemAcc; s.ipw = 2;
  }
  return s;
}

static size_t smem_bytes(const Shape& s) {
  const int row_stride = s.row_bytes + 16;
  const int warps = s.kind == 0 ? kTriWarps : kConsumerWarps;
  return (size_t)kStages * s.rows * row_stride + (size_t)warps * s.ipw * s.naccp * sizeof(double) +
         (2 * kStages + 1) * sizeof(uint64_t) + 64 * sizeof(int) + 128;
}

template <typename K>
static cudaError_t launch(K kernel, const Params& prm, int grid, int threads, size_t smem, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kernel<<<grid, threads, smem, st>>>(prm);
  return cudaGetLastError();
}

template <typename T>
static cudaError_t dispatch(const Shape& sh, int vec, const Params& prm, int grid, size_t smem, cudaStream_t st) {
  if (sh.kind == 1) {
    if (sh.pb_or_nb == 2) return launch(gram_blocks_kernel<T, 2>, prm, grid, kThreads, smem, st);
    return launch(gram_blocks_kernel<T, 4>, prm, grid, kThreads, smem, st);
  }
#define FA_TRI_CASE(PB)                                                            \
  case PB:                                                                         \
    return vec == 2 ? launch(gram_tri_kernel<T, 2, PB, kTriWarps>, prm, grid, (kTriWarps + 1) * 32, smem, st) \
                    : launch(gram_tri_kernel<T, 1, PB, kTriWarps>, prm, grid, (kTriWarps + 1) * 32, smem, st);
  switch (sh.pb_or_nb) {
    FA_TRI_CASE(4)
    FA_TRI_CASE(8)
    FA_TRI_CASE(12)
    FA_TRI_CASE(15)
    FA_TRI_CASE(16)
  }
#undef FA_TRI_CASE
  return cudaErrorInvalidValue;
}

}  // namespace gram

// Upper bound on the blocks any Gram kernel launches for this shape (one per SM at most); it
// sizes the per-block partial sums in the workspace.
int gram_num_blocks(int p, long long n, int dtype) {
  (void)p; (void)dtype;
  const int sms = sm_count();
  return (int)(n < sms ? n : sms);
}

size_t gram_partials_bytes(int p, long long n, int dtype) {
  return (size_t)gram_num_blocks(p, n, dtype) * (size_t)(p * (p + 1) / 2) * sizeof(double);
}

cudaError_t launch_gram(const void* G, int dtype, int p, long long n, double* partials, unsigned int* counter,
                        double* K, int* status, cudaStream_t st) {
  if (gram_tc_eligible(G, dtype, p, n)) return launch_gram_tc(G, p, n, partials, counter, K, status, st);
  if (gram_tm_eligible(G, dtype, p, n)) return launch_gram_tm(G, dtype, p, n, partials, counter, K, status, st);
  if (gram_tm32_eligible(G, dtype, p, n)) return launch_gram_tm32(G, p, n, partials, counter, K, status, st);
  if (gram_tm64_eligible(G, dtype, p, n)) return launch_gram_tm64(G, p, n, partials, counter, K, status, st);
  const gram::Shape sh = gram::pick_shape(p);
  const int S = dtype == 0 ? 4 : 2;
  gram::Params prm{};
  prm.G = static_cast<const char*>(G);
  prm.n = n;
  prm.p = p;
  prm.tile_cols = sh.row_bytes / S;
  prm.row_stride = sh.row_bytes + 16;
  prm.num_tiles = (n + prm.tile_cols - 1) / prm.tile_cols;
  prm.partials = partials;
  prm.counter = counter;
  prm.K = K;
  prm.status = status;
  const int sms = sm_count();
  const int grid = (int)(prm.num_tiles < sms ? prm.num_tiles : sms);
  cudaError_t e = cudaMemsetAsync(counter, 0, sizeof(unsigned int), st);
  if (e != cudaSuccess) return e;
  // two elements per shared load when every row starts on an even element
  const bool even = (n % 2 == 0) && ((reinterpret_cast<uintptr_t>(G) % (2 * S)) == 0);
  const int vec = even ? 2 : 1;
  const size_t smem = gram::smem_bytes(sh);
  if (dtype == 0) return gram::dispatch<float>(sh, vec, prm, grid, smem, st);
  return gram::dispatch<__nv_bfloat16>(sh, vec, prm, grid, smem, st);
}

}  // namespace fa
