// Gram pass fed by TMA TENSOR loads (K_ij = <g_i, g_j>, Section 2.1) -- the fast path of fa_gram
// whenever the matrix starts on a 16-byte boundary.
//
// One tensor-map load brings a 256-column tile of ALL rows of a row class into shared memory
// (15-64 KB per instruction).  Measured on B200 this feed sustains about 24.7 bytes per clock and SM
// (7.2 TB/s), against 19.5 for one 1-D bulk copy of 4 KB per row (fa_gram.cu) -- the tensor unit
// pays its fixed cost per ROW of a box, and 1 KB rows are long enough.
//
// Row classes.  A tensor map wants every row to start on a 16-byte boundary (base and strides are
// multiples of 16 bytes), and n * sizeof(T) need not be one.  So the rows are split into q classes
// i mod q (q = 1, 2 or 4: the smallest with q * n * sizeof(T) a multiple of 16); class c gets its own
// map over the rows c, c + q, ... with stride q * n, based at the 16-byte boundary at or before the
// start of row c.  Row c therefore begins `shift_c` elements into its map's rows, the tile of a
// class is read back with that shift, and consecutive tiles advance by 256 - 16/sizeof(T) columns
// instead of 256 so that every class holds all the columns of a tile (1.6 % re-read; none when
// q = 1).  Columns past the end of a row are outside the map's extent and arrive as zeros, so
// there is no ragged tile; the few elements before row c that the shift drags in belong to row
// c - 1 and are never read back.
//
// p <= 16: every warp takes whole tiles (tile u of a block goes to warp u mod 12) and loads them
// itself; every thread keeps the upper triangle for its columns, as in fa_gram.cu; products in
// fp32, runs of at most 64 columns, warp butterfly into fp64.  Block totals and the last-block reduction are
// the ones of fa_gram.cu (bit-reproducible, single launch).  fp32 with 16 < p <= 32 and one row class has a
// kernel of its own below (teams of four warps), and 32 < p <= 64 is put together from three launches by
// row blocks of 32 (launch_gram_tm64).
#include <atomic>

#include "fa_gram_tm.cuh"
#include "fa_gram_finish.cuh"
#include "fa_kernels.h"

namespace fa {
namespace gramtm {

struct Params {
  int p;                       // rows of the matrix this launch reads
  int row0;                    // their position among the `ptotal` rows of K (a launch on a block of rows)
  int ptotal;                  // rows of K
  int finish;                  // the last block forms K from all blocks' sums (the last launch of a pass)
  long long num_tiles;
  double* partials;            // [p(p+1)/2][gridDim.x]
  unsigned int* counter;
  double* K;
  int* status;
  long long wait_cycles;       // limit of a wait for a tile (kWaitCycles unless a test shortened it)
};

// p <= 16.  No producer: every warp owns `depth` stages and keeps them loaded itself -- lane 0 issues
// the tensor loads of the warp's next tile into the stage the warp has just finished with.  (One
// issuing thread for the whole block could not keep up: a tile costs it about 500 cycles, and a
// stage must in any case be consumed by the warp that waited for its previous phases -- a parity
// wait cannot tell "two phases behind" from "done".)  Tile u of a block (global tile
// blockIdx.x + u * gridDim.x) goes to warp u mod 12.
template <typename T, int V, int PB>
__global__ void __launch_bounds__(kTriWarps * 32, 1)
gram_tri_tm_kernel(const __grid_constant__ Maps maps, const Params prm, const Layout lay) {
  constexpr int S = sizeof(T);
  constexpr int kThreads = kTriWarps * 32;
  constexpr int NACC = PB * (PB + 1) / 2;
  constexpr int NACCP = (NACC + 31) / 32 * 32;
  extern __shared__ __align__(1024) char smem[];
  const int stage_bytes = prm.p * kTileCols * S;
  const int depth = lay.depth;
  char* stages = smem;
  double* totals = reinterpret_cast<double*>(smem + (size_t)kTriWarps * depth * stage_bytes);
  uint64_t* full = reinterpret_cast<uint64_t*>(totals + kTriWarps * NACCP);
  int* flag = reinterpret_cast<int*>(full + kTriWarps * kMaxDepth);      // last-block flag
  int* aborted = flag + 1;                                               // a warp of this block gave up on a tile
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int s = 0; s < kTriWarps * kMaxDepth; ++s) mbar_init(&full[s], 1);
    *aborted = 0;
  }
  fence_proxy_async();
  __syncthreads();

  float acc[NACCP];
  double dacc[NACCP / 32];
#pragma unroll
  for (int k = 0; k < NACCP; ++k) acc[k] = 0.f;
#pragma unroll
  for (int k = 0; k < NACCP / 32; ++k) dacc[k] = 0.0;
  int rowoff[PB];
#pragma unroll
  for (int i = 0; i < PB; ++i) {
    const int ii = i < prm.p ? i : 0;
    const int cidx = ii % lay.q;
    rowoff[i] = (lay.rowbase[cidx] + ii / lay.q) * (kTileCols * S) + lay.shift[cidx] * S;
  }
  char* mystages = stages + (size_t)warp * depth * stage_bytes;
  uint64_t* mybars = full + warp * kMaxDepth;

  // this warp's tiles: global tiles blockIdx.x + (warp + 12 v) * gridDim.x, v = 0, 1, ..., in stage
  // v mod depth; tile numbers fit 32 bits, stage and phase are stepped along with the tile
  const int ntiles = static_cast<int>(prm.num_tiles);
  const int tstride = kTriWarps * static_cast<int>(gridDim.x);
  const int tfirst = static_cast<int>(blockIdx.x) + warp * static_cast<int>(gridDim.x);
  auto issue = [&](int t, int s) {       // lane 0 only
    if (t >= ntiles) return;
    mbar_arrive_expect_tx(&mybars[s], static_cast<uint32_t>(stage_bytes));
    char* sbase = mystages + (size_t)s * stage_bytes;
    const int x0 = t * lay.step;
    for (int cidx = 0; cidx < lay.q; ++cidx)
      if (lay.rows[cidx] > 0)
        tma_load_2d(sbase + (size_t)lay.rowbase[cidx] * kTileCols * S, &maps.map[cidx], x0, 0, &mybars[s]);
  };
  if (lane == 0)
    for (int v = 0; v < depth; ++v) issue(tfirst + v * tstride, v);

  const int groups = lay.step / V;
  const int per_tile = (groups + 31) / 32 * V;      // columns a thread takes from one tile
  int since = 0;
  int s = 0;
  uint32_t phase = 0;
  for (int t = tfirst; t < ntiles; t += tstride) {
    // the lanes poll on their own; once any of them has seen the phase complete, it is complete
    if (!__any_sync(0xffffffffu, mbar_wait(&mybars[s], phase, prm.wait_cycles))) {
      if (lane == 0) {
        if (prm.status) atomicOr(prm.status, kStTimeout);
        *reinterpret_cast<volatile int*>(aborted) = 1;
        // every load of this warp that is in flight -- the one it gave up on and those of the stages
        // after it -- must land before the block can exit: these waits keep the long limit
        int s2 = s;
        uint32_t ph2 = phase;
        for (int k = 0; k < depth; ++k) {
          if (t + k * tstride < ntiles) (void)mbar_wait(&mybars[s2], ph2);
          if (++s2 == depth) { s2 = 0; ph2 ^= 1u; }
        }
      }
      break;
    }
    const char* sbase = mystages + (size_t)s * stage_bytes;
    for (int cg = lane; cg < groups; cg += 32) {
      float x[PB][V];
#pragma unroll
      for (int i = 0; i < PB; ++i) {
        if constexpr (S == 4 && V == 2 && PB > 12) {
          // two columns half a tile apart, one 4-byte load each: an 8-byte load of neighbours would put both
          // factors of every product into the same register bank (every other FMA then takes a second
          // dispatch cycle).  Up to 12 rows the pass is bound by the loads of the tiles and the fewer, wider
          // shared loads are the better choice.
          x[i][0] = *reinterpret_cast<const float*>(sbase + rowoff[i] + cg * 4);
          x[i][1] = *reinterpret_cast<const float*>(sbase + rowoff[i] + (cg + groups) * 4);
        } else {
          SmemVec<T, V>::load(sbase + rowoff[i] + cg * (V * S), x[i]);
        }
        if (i >= prm.p) {
#pragma unroll
          for (int e = 0; e < V; ++e) x[i][e] = 0.f;
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
    if (lane == 0) {
      fence_proxy_async();          // the warp's reads of this stage come before the next load's writes
      issue(t + depth * tstride, s);
    }
    if (++s == depth) { s = 0; phase ^= 1u; }
    since += per_tile;
    if (since + per_tile > kFlushCols) { flush<NACCP>(acc, dacc, lane); since = 0; }
  }
  flush<NACCP>(acc, dacc, lane);
#pragma unroll
  for (int k = 0; k < NACCP / 32; ++k) totals[warp * NACCP + lane * (NACCP / 32) + k] = dacc[k];
  __syncthreads();

  // block total (fixed warp order) -> this block's entries, then the last block forms K
  for (int e = tid; e < NACC; e += kThreads) {
    int i = 0, r = e;
    while (r >= PB - i) { r -= PB - i; ++i; }
    const int j = i + r;
    if (j < prm.p) {
      double sum = 0.0;
      for (int w = 0; w < kTriWarps; ++w) sum += totals[w * NACCP + e];
      // a block that gave up has incomplete sums: NaN, so that K comes out non-finite and whoever
      // reads it (the IRLS kernel sets FA_ST_NONFINITE and writes zeros) sees the failure
      if (*reinterpret_cast<volatile int*>(aborted)) sum = __longlong_as_double(0x7ff8000000000000LL);
      prm.partials[(size_t)gram::canon_index(prm.row0 + i, prm.row0 + j, prm.ptotal) * gridDim.x + blockIdx.x] = sum;
    }
  }
  if (prm.finish) gram::finish_gram(prm.partials, prm.counter, prm.K, prm.ptotal, flag);
}

// ---- 16 < p <= 32, one row class (rows on 16-byte boundaries), fp32.
// The 32 x 32 triangle is cut into four parts of at most 136 sums -- the triangles of rows 0-15 and
// 16-31 and the two 8 x 16 halves of the rectangle between them -- and a TEAM of four warps, one per
// part, works through a tile together; the block's two teams take alternate tiles, each with its
// own stages, and the first lane of a team re-issues the team's next load once the four warps have
// met at the team's barrier.  Eight warps (two per scheduler) leave 255 registers per thread: the
// sums, two columns of operands and nothing spilled.  A lane's two columns are 32 apart and are
// fetched with 4-byte loads, not as one 8-byte load of neighbouring columns: an 8-byte load puts
// every row's first column in an even register and its second in an odd one, so both factors of a
// product always come from the same register bank and, with one running sum per entry serving both
// columns, every other FMA took a second dispatch cycle (0.58 FMA per clock and scheduler against
// 0.69 with 4-byte loads, on the 16-row triangle alone).  Staged rows are exactly 1 KB apart, so
// every shared load is one base register plus an immediate; rows p..31 of a stage are zeroed once
// and never written.
constexpr int kQuadWarps = 8;
constexpr int kQuadDepth = 3;                // stages per team: 2 x 3 x 32 KB
constexpr int kQuadAcc = 160;                // 136 rounded up to a multiple of 32
constexpr int kQuadFlushCols = 128;          // fp32 running sums cover at most this many columns here

__device__ __forceinline__ void team_barrier(int team) {
  asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "r"(128) : "memory");
}

__global__ void __launch_bounds__(kQuadWarps * 32, 1)
gram_quad_tm_kernel(const __grid_constant__ Maps maps, const Params prm) {
  constexpr int kThreads = kQuadWarps * 32;
  constexpr int kRowBytes = kTileCols * 4;
  constexpr int kStageBytes = 32 * kRowBytes;
  extern __shared__ __align__(1024) char smem[];
  char* stages = smem;
  double* totals = reinterpret_cast<double*>(smem + (size_t)2 * kQuadDepth * kStageBytes);
  uint64_t* full = reinterpret_cast<uint64_t*>(totals + kQuadWarps * kQuadAcc);
  int* flag = reinterpret_cast<int*>(full + 2 * kQuadDepth);
  int* aborted = flag + 1;                   // [team]: a warp of the team gave up on a tile
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int team = warp >> 2, role = warp & 3;
  if (tid == 0) { aborted[0] = 0; aborted[1] = 0; }

  for (int i = tid * 16; i < 2 * kQuadDepth * kStageBytes; i += kThreads * 16)
    *reinterpret_cast<uint4*>(stages + i) = make_uint4(0, 0, 0, 0);
  if (tid == 0)
    for (int s = 0; s < 2 * kQuadDepth; ++s) mbar_init(&full[s], 1);
  fence_proxy_async();
  __syncthreads();

  char* mystages = stages + (size_t)team * kQuadDepth * kStageBytes;
  uint64_t* mybars = full + team * kQuadDepth;
  const uint32_t tile_bytes = static_cast<uint32_t>(prm.p * kRowBytes);
  // the team's tiles: global tiles blockIdx.x + (2 v + team) * gridDim.x, v = 0, 1, ...; tile numbers
  // fit 32 bits (n < 2^31), and stage and phase are stepped along with the tile instead of being
  // worked out from v (64-bit divisions by the depth were a visible part of the per-tile cost)
  const int ntiles = static_cast<int>(prm.num_tiles);
  const int tstride = 2 * static_cast<int>(gridDim.x);
  const int tfirst = static_cast<int>(blockIdx.x) + team * static_cast<int>(gridDim.x);
  auto issue = [&](int t, int s) {       // first lane of the team only
    if (t >= ntiles) return;
    mbar_arrive_expect_tx(&mybars[s], tile_bytes);
    tma_load_2d(mystages + (size_t)s * kStageBytes, &maps.map[0], t * kTileCols, 0, &mybars[s]);
  };
  const bool issuer = role == 0 && lane == 0;
  if (issuer)
    for (int v = 0; v < kQuadDepth; ++v) issue(tfirst + v * tstride, v);
  // the team's loads in flight when it gives up at tile t (stage s0, phase ph0) -- this stage's and the
  // following ones' -- must land before the block can exit: these waits keep the long limit
  auto drain = [&](int t, int s0, uint32_t ph0) {
    if (!issuer) return;
    for (int k = 0; k < kQuadDepth; ++k) {
      if (t + k * tstride < ntiles) (void)mbar_wait(&mybars[s0], ph0);
      if (++s0 == kQuadDepth) { s0 = 0; ph0 ^= 1u; }
    }
  };

  float acc[kQuadAcc];
  double dacc[kQuadAcc / 32];
#pragma unroll
  for (int k = 0; k < kQuadAcc; ++k) acc[k] = 0.f;
#pragma unroll
  for (int k = 0; k < kQuadAcc / 32; ++k) dacc[k] = 0.0;
  const int rowbase = (role < 2 ? 16 * role : 8 * (role - 2)) * kRowBytes;   // first row of the part (rectangle: its a-rows)
  int since = 0;
  int s = 0;
  uint32_t phase = 0;
  for (int t = tfirst; t < ntiles; t += tstride) {
    // Giving up must be a decision of the whole team: its four warps meet at the team's barrier after
    // every tile, so a warp whose wait ran out raises the team's flag and still goes to that barrier;
    // behind it all four read the flag and leave together.  (The lanes of a warp poll on their own;
    // once any of them has seen the phase complete, it is complete.)
    if (!__any_sync(0xffffffffu, mbar_wait(&mybars[s], phase, prm.wait_cycles))) {
      if (lane == 0) {
        if (prm.status) atomicOr(prm.status, kStTimeout);
        *reinterpret_cast<volatile int*>(&aborted[team]) = 1;
      }
      team_barrier(team);
      drain(t, s, phase);
      break;
    }
    const char* sbase = mystages + (size_t)s * kStageBytes;
    if (role < 2) {
#pragma unroll 1
      for (int cg = lane; cg < kTileCols; cg += 64) {
        const char* ptr = sbase + rowbase + cg * 4;
        float x[16][2];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          x[i][0] = *reinterpret_cast<const float*>(ptr + i * kRowBytes);
          x[i][1] = *reinterpret_cast<const float*>(ptr + i * kRowBytes + 128);
        }
        int idx = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i)
#pragma unroll
          for (int j = i; j < 16; ++j) {
            acc[idx] = fmaf(x[i][0], x[j][0], acc[idx]);
            acc[idx] = fmaf(x[i][1], x[j][1], acc[idx]);
            ++idx;
          }
      }
    } else {
#pragma unroll 1
      for (int cg = lane; cg < kTileCols; cg += 64) {
        const char* pa = sbase + rowbase + cg * 4;
        const char* pb = sbase + 16 * kRowBytes + cg * 4;
        float a[8][2], b[16][2];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          a[i][0] = *reinterpret_cast<const float*>(pa + i * kRowBytes);
          a[i][1] = *reinterpret_cast<const float*>(pa + i * kRowBytes + 128);
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          b[j][0] = *reinterpret_cast<const float*>(pb + j * kRowBytes);
          b[j][1] = *reinterpret_cast<const float*>(pb + j * kRowBytes + 128);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            acc[i * 16 + j] = fmaf(a[i][0], b[j][0], acc[i * 16 + j]);
            acc[i * 16 + j] = fmaf(a[i][1], b[j][1], acc[i * 16 + j]);
          }
      }
    }
    team_barrier(team);                  // all four parts are done with the stage
    if (*reinterpret_cast<volatile int*>(&aborted[team])) {      // another warp of the team gave up on this tile
      drain(t, s, phase);
      break;
    }
    if (issuer) {
      fence_proxy_async();
      issue(t + kQuadDepth * tstride, s);
    }
    if (++s == kQuadDepth) { s = 0; phase ^= 1u; }
    since += 8;
    if (since + 8 > kQuadFlushCols) { flush<kQuadAcc>(acc, dacc, lane); since = 0; }
  }
  flush<kQuadAcc>(acc, dacc, lane);
#pragma unroll
  for (int k = 0; k < kQuadAcc / 32; ++k) totals[warp * kQuadAcc + lane * (kQuadAcc / 32) + k] = dacc[k];
  __syncthreads();

  // block totals: the two teams' sums of every part, in a fixed order
  for (int idx = tid; idx < 4 * kQuadAcc; idx += kThreads) {
    const int part = idx / kQuadAcc, e = idx - part * kQuadAcc;
    int gi, gj;
    if (part < 2) {
      if (e >= 136) continue;
      int i = 0, r = e;
      while (r >= 16 - i) { r -= 16 - i; ++i; }
      gi = 16 * part + i; gj = 16 * part + i + r;
    } else {
      if (e >= 128) continue;
      gi = 8 * (part - 2) + e / 16; gj = 16 + e % 16;
    }
    if (gi >= prm.p || gj >= prm.p) continue;
    double sum = totals[(size_t)part * kQuadAcc + e] + totals[(size_t)(4 + part) * kQuadAcc + e];
    if (*reinterpret_cast<volatile int*>(&aborted[0]) | *reinterpret_cast<volatile int*>(&aborted[1]))
      sum = __longlong_as_double(0x7ff8000000000000LL);     // incomplete sums must not pass for inner products
    prm.partials[(size_t)gram::canon_index(prm.row0 + gi, prm.row0 + gj, prm.ptotal) * gridDim.x + blockIdx.x] = sum;
  }
  if (prm.finish) gram::finish_gram(prm.partials, prm.counter, prm.K, prm.ptotal, flag);
}

// ---- 32 < p <= 64, one row class, fp32: the rectangle between rows 0-31 and rows 32..p-1.
// K is put together from three launches over the same column tiles: the triangle kernel above on
// rows 0-31, the same on rows 32..p-1, and this kernel for the 32 x (p - 32) entries between the two
// blocks of rows -- the matrix is read twice, which is what 255 registers per thread allow (2080 sums
// per column do not fit one block's registers, and sums have to stay in registers from tile to tile).
// One tile holds all p rows (64 KB); the rectangle is cut into eight parts of 8 x 16 sums, one per
// warp (a-rows 8 (w mod 4) .., b-rows 32 + 16 (w / 4) ..), operands by 4-byte loads of columns 32
// apart as above.  All eight warps work on the same tile; the first thread re-issues a stage's load
// behind the block's barrier.  This launch comes last and its last block forms K.
constexpr int kCrossWarps = 8;
constexpr int kCrossDepth = 3;               // stages of 64 KB
constexpr int kCrossAcc = 128;

__global__ void __launch_bounds__(kCrossWarps * 32, 1)
gram_cross_tm_kernel(const __grid_constant__ Maps maps, const Params prm) {
  constexpr int kThreads = kCrossWarps * 32;
  constexpr int kRowBytes = kTileCols * 4;
  constexpr int kStageBytes = 64 * kRowBytes;
  extern __shared__ __align__(1024) char smem[];
  char* stages = smem;
  double* totals = reinterpret_cast<double*>(smem + (size_t)kCrossDepth * kStageBytes);
  uint64_t* full = reinterpret_cast<uint64_t*>(totals + kCrossWarps * kCrossAcc);
  int* flag = reinterpret_cast<int*>(full + kCrossDepth);
  int* aborted = flag + 1;                   // a warp gave up on a tile
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) *aborted = 0;

  for (int i = tid * 16; i < kCrossDepth * kStageBytes; i += kThreads * 16)
    *reinterpret_cast<uint4*>(stages + i) = make_uint4(0, 0, 0, 0);
  if (tid == 0)
    for (int s = 0; s < kCrossDepth; ++s) mbar_init(&full[s], 1);
  fence_proxy_async();
  __syncthreads();

  const uint32_t tile_bytes = static_cast<uint32_t>(prm.p * kRowBytes);
  const int ntiles = static_cast<int>(prm.num_tiles);
  const int tstride = static_cast<int>(gridDim.x);
  const int tfirst = static_cast<int>(blockIdx.x);
  auto issue = [&](int t, int s) {       // first thread of the block only
    if (t >= ntiles) return;
    mbar_arrive_expect_tx(&full[s], tile_bytes);
    tma_load_2d(stages + (size_t)s * kStageBytes, &maps.map[0], t * kTileCols, 0, &full[s]);
  };
  const bool issuer = tid == 0;
  if (issuer)
    for (int v = 0; v < kCrossDepth; ++v) issue(tfirst + v * tstride, v);
  // the loads in flight when the block gives up at tile t (stage s0, phase ph0) must land before it can
  // exit: these waits keep the long limit
  auto drain = [&](int t, int s0, uint32_t ph0) {
    if (!issuer) return;
    for (int k = 0; k < kCrossDepth; ++k) {
      if (t + k * tstride < ntiles) (void)mbar_wait(&full[s0], ph0);
      if (++s0 == kCrossDepth) { s0 = 0; ph0 ^= 1u; }
    }
  };

  float acc[kCrossAcc];
  double dacc[kCrossAcc / 32];
#pragma unroll
  for (int k = 0; k < kCrossAcc; ++k) acc[k] = 0.f;
#pragma unroll
  for (int k = 0; k < kCrossAcc / 32; ++k) dacc[k] = 0.0;
  const int abase = 8 * (warp & 3) * kRowBytes;
  const int bbase = (32 + 16 * (warp >> 2)) * kRowBytes;
  const bool active = 32 + 16 * (warp >> 2) < prm.p;       // up to 48 rows the second half of the warps has no entries
  int since = 0;
  int s = 0;
  uint32_t phase = 0;
  for (int t = tfirst; t < ntiles; t += tstride) {
    // giving up is a decision of the whole block, taken behind the barrier that ends the tile (as in the
    // kernel above, with the block in the place of a team)
    if (!__any_sync(0xffffffffu, mbar_wait(&full[s], phase, prm.wait_cycles))) {
      if (lane == 0) {
        if (prm.status) atomicOr(prm.status, kStTimeout);
        *reinterpret_cast<volatile int*>(aborted) = 1;
      }
      __syncthreads();
      drain(t, s, phase);
      break;
    }
    const char* sbase = stages + (size_t)s * kStageBytes;
#pragma unroll 1
    for (int cg = active ? lane : kTileCols; cg < kTileCols; cg += 64) {
      const char* pa = sbase + abase + cg * 4;
      const char* pb = sbase + bbase + cg * 4;
      float a[8][2], b[16][2];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        a[i][0] = *reinterpret_cast<const float*>(pa + i * kRowBytes);
        a[i][1] = *reinterpret_cast<const float*>(pa + i * kRowBytes + 128);
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        b[j][0] = *reinterpret_cast<const float*>(pb + j * kRowBytes);
        b[j][1] = *reinterpret_cast<const float*>(pb + j * kRowBytes + 128);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          acc[i * 16 + j] = fmaf(a[i][0], b[j][0], acc[i * 16 + j]);
          acc[i * 16 + j] = fmaf(a[i][1], b[j][1], acc[i * 16 + j]);
        }
    }
    __syncthreads();                     // all eight parts are done with the stage
    if (*reinterpret_cast<volatile int*>(aborted)) {      // another warp gave up on this tile
      drain(t, s, phase);
      break;
    }
    if (issuer) {
      fence_proxy_async();
      issue(t + kCrossDepth * tstride, s);
    }
    if (++s == kCrossDepth) { s = 0; phase ^= 1u; }
    since += 8;
    if (since + 8 > kQuadFlushCols) { flush<kCrossAcc>(acc, dacc, lane); since = 0; }
  }
  flush<kCrossAcc>(acc, dacc, lane);
#pragma unroll
  for (int k = 0; k < kCrossAcc / 32; ++k) totals[warp * kCrossAcc + lane * (kCrossAcc / 32) + k] = dacc[k];
  __syncthreads();

  for (int idx = tid; idx < kCrossWarps * kCrossAcc; idx += kThreads) {
    const int part = idx / kCrossAcc, e = idx - part * kCrossAcc;
    const int gi = 8 * (part & 3) + e / 16, gj = 32 + 16 * (part >> 2) + e % 16;
    if (gj >= prm.p) continue;
    double sum = totals[idx];
    if (*reinterpret_cast<volatile int*>(aborted))
      sum = __longlong_as_double(0x7ff8000000000000LL);     // incomplete sums must not pass for inner products
    prm.partials[(size_t)gram::canon_index(gi, gj, prm.p) * gridDim.x + blockIdx.x] = sum;
  }
  if (prm.finish) gram::finish_gram(prm.partials, prm.counter, prm.K, prm.p, flag);
}

namespace {

// Row classes of a p x n matrix of S-byte elements: 0 when more than kMaxClasses would be needed.
int class_count(long long n, int S) {
  for (int q = 1; q <= kMaxClasses; q *= 2)
    if ((static_cast<unsigned long long>(q) * static_cast<unsigned long long>(n) * S) % 16 == 0) return q;
  return 0;
}

}  // namespace

bool build(const void* G, int dtype, int p, long long n, Maps& maps, Layout& lay) {
  EncodeTiledFn enc = encode_tiled();
  const int S = dtype == 0 ? 4 : 2;
  const int q = class_count(n, S);
  if (!enc || q == 0) return false;
  lay.q = q;
  lay.step = q == 1 ? kTileCols : kTileCols - 16 / S;
  int base = 0;
  for (int c = 0; c < kMaxClasses; ++c) { lay.rows[c] = 0; lay.rowbase[c] = 0; lay.shift[c] = 0; }
  for (int c = 0; c < q; ++c) {
    const int rows = c < p ? (p - c + q - 1) / q : 0;
    lay.rows[c] = rows;
    lay.rowbase[c] = base;
    base += rows;
    if (rows == 0) continue;
    const unsigned long long off = static_cast<unsigned long long>(c) * static_cast<unsigned long long>(n) * S;   // bytes
    const int skew = static_cast<int>(off % 16);
    lay.shift[c] = skew / S;
    const char* start = static_cast<const char*>(G) + off - skew;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(n) + static_cast<cuuint64_t>(lay.shift[c]),
                                static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(q) * static_cast<cuuint64_t>(n) * S};
    const cuuint32_t box[2] = {kTileCols, static_cast<cuuint32_t>(rows)};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&maps.map[c], dtype == 0 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            const_cast<char*>(start), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  return true;
}

bool available(const void* G, int dtype, long long n) {
  return (reinterpret_cast<uintptr_t>(G) % 16) == 0 && n >= 4096 && n < (1LL << 31) - 4096 &&
         class_count(n, dtype == 0 ? 4 : 2) != 0 && encode_tiled() != nullptr;
}

namespace {

template <typename K>
cudaError_t launch(K kernel, const Maps& maps, const Params& prm, const Layout& lay, int grid, int threads,
                   size_t smem, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kernel<<<grid, threads, smem, st>>>(maps, prm, lay);
  return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch_tri(int pb, int vec, const Maps& maps, const Params& prm, const Layout& lay, int grid, size_t smem,
                         cudaStream_t st) {
#define FA_TM_CASE(PB)                                                                                       \
  case PB:                                                                                                   \
    return vec == 2 ? launch(gram_tri_tm_kernel<T, 2, PB>, maps, prm, lay, grid, kTriWarps * 32, smem, st) \
                    : launch(gram_tri_tm_kernel<T, 1, PB>, maps, prm, lay, grid, kTriWarps * 32, smem, st);
  switch (pb) {
    FA_TM_CASE(4)
    FA_TM_CASE(8)
    FA_TM_CASE(12)
    FA_TM_CASE(15)
    FA_TM_CASE(16)
  }
#undef FA_TM_CASE
  return cudaErrorInvalidValue;
}

}  // namespace
}  // namespace gramtm

// Tensor-load feed: matrix on a 16-byte boundary, at most four row classes, enough columns for a
// few tiles per block, column coordinates within the 32-bit range of the copy instruction.
bool gram_tm_eligible(const void* G, int dtype, int p, long long n) {
  return p >= 1 && p <= 16 && gramtm::available(G, dtype, n);
}

bool gram_tm32_eligible(const void* G, int dtype, int p, long long n) {
  return dtype == 0 && p > 16 && p <= 32 && gramtm::available(G, dtype, n) && (n % 4) == 0;
}

bool gram_tm64_eligible(const void* G, int dtype, int p, long long n) {
  return dtype == 0 && p > 32 && p <= 64 && gramtm::available(G, dtype, n) && (n % 4) == 0;
}

namespace {
// Limit of the kernels' waits for a tile, in cycles.  Always kWaitCycles in normal use.
std::atomic<long long> g_tile_wait_cycles{kWaitCycles};
}  // namespace

}  // namespace fa

// Test hook (exported, but deliberately not declared in include/fa.h): shortens the tile waits of
// the tensor-fed Gram kernels so that a test can watch a wait run out on a launch that is otherwise
// correct -- the kernel gives up, lets its loads land (those waits keep the long limit), reports
// FA_ST_TIMEOUT and returns.  cycles <= 0 restores the default.
extern "C" void fa_test_set_gram_wait_cycles(long long cycles) {
  fa::g_tile_wait_cycles.store(cycles > 0 ? cycles : fa::kWaitCycles);
}

namespace fa {

cudaError_t launch_gram_tm32(const void* G, int p, long long n, double* partials, unsigned int* counter, double* K,
                             int* status, cudaStream_t st) {
  gramtm::Maps maps;
  gramtm::Layout lay;
  if (!gramtm::build(G, 0, p, n, maps, lay) || lay.q != 1) return cudaErrorInvalidValue;
  gramtm::Params prm{};
  prm.p = p;
  prm.row0 = 0;
  prm.ptotal = p;
  prm.finish = 1;
  prm.num_tiles = (n + gramtm::kTileCols - 1) / gramtm::kTileCols;
  prm.partials = partials;
  prm.counter = counter;
  prm.K = K;
  prm.status = status;
  prm.wait_cycles = g_tile_wait_cycles.load();
  const int sms = sm_count();
  const int grid = (int)(prm.num_tiles < sms ? prm.num_tiles : sms);
  cudaError_t e = cudaMemsetAsync(counter, 0, sizeof(unsigned int), st);
  if (e != cudaSuccess) return e;
  const size_t smem = (size_t)2 * gramtm::kQuadDepth * 32 * gramtm::kTileCols * 4 +
                      (size_t)gramtm::kQuadWarps * gramtm::kQuadAcc * sizeof(double) +
                      2 * gramtm::kQuadDepth * sizeof(uint64_t) + 64;
  e = cudaFuncSetAttribute(gramtm::gram_quad_tm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  gramtm::gram_quad_tm_kernel<<<grid, gramtm::kQuadWarps * 32, smem, st>>>(maps, prm);
  return cudaGetLastError();
}

namespace {
// The p <= 16 kernel on the p rows at G; prm carries everything but p, the tile count and the wait limit.
cudaError_t launch_tri_rows(const void* G, int dtype, int p, long long n, gramtm::Params prm, cudaStream_t st);
}  // namespace

cudaError_t launch_gram_tm64(const void* G, int p, long long n, double* partials, unsigned int* counter, double* K,
                             int* status, cudaStream_t st) {
  const float* g = static_cast<const float*>(G);
  const int rows2 = p - 32;
  gramtm::Maps maps1, maps2, maps3;
  gramtm::Layout lay;
  if (!gramtm::build(g, 0, 32, n, maps1, lay) || lay.q != 1) return cudaErrorInvalidValue;
  if (!gramtm::build(g + (size_t)32 * (size_t)n, 0, rows2, n, maps2, lay) || lay.q != 1) return cudaErrorInvalidValue;
  if (!gramtm::build(g, 0, p, n, maps3, lay) || lay.q != 1) return cudaErrorInvalidValue;
  gramtm::Params prm{};
  prm.ptotal = p;
  prm.num_tiles = (n + gramtm::kTileCols - 1) / gramtm::kTileCols;
  prm.partials = partials;
  prm.counter = counter;
  prm.K = K;
  prm.status = status;
  prm.wait_cycles = g_tile_wait_cycles.load();
  const int sms = sm_count();
  const int grid = (int)(prm.num_tiles < sms ? prm.num_tiles : sms);     // the same for all three: one slot per block
  const size_t smem_quad = (size_t)2 * gramtm::kQuadDepth * 32 * gramtm::kTileCols * 4 +
                           (size_t)gramtm::kQuadWarps * gramtm::kQuadAcc * sizeof(double) +
                           2 * gramtm::kQuadDepth * sizeof(uint64_t) + 64;
  const size_t smem_cross = (size_t)gramtm::kCrossDepth * 64 * gramtm::kTileCols * 4 +
                            (size_t)gramtm::kCrossWarps * gramtm::kCrossAcc * sizeof(double) +
                            gramtm::kCrossDepth * sizeof(uint64_t) + 64;
  cudaError_t e = cudaFuncSetAttribute(gramtm::gram_quad_tm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_quad);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gramtm::gram_cross_tm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_cross);
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(counter, 0, sizeof(unsigned int), st);
  if (e != cudaSuccess) return e;
  prm.p = 32; prm.row0 = 0; prm.finish = 0;
  gramtm::gram_quad_tm_kernel<<<grid, gramtm::kQuadWarps * 32, smem_quad, st>>>(maps1, prm);
  prm.p = rows2; prm.row0 = 32;
  if (rows2 <= 16) {                    // a block of at most 16 rows goes through the faster kernel for such blocks
    e = launch_tri_rows(g + (size_t)32 * (size_t)n, 0, rows2, n, prm, st);
    if (e != cudaSuccess) return e;
  } else {
    gramtm::gram_quad_tm_kernel<<<grid, gramtm::kQuadWarps * 32, smem_quad, st>>>(maps2, prm);
  }
  prm.p = p; prm.row0 = 0; prm.finish = 1;
  gramtm::gram_cross_tm_kernel<<<grid, gramtm::kCrossWarps * 32, smem_cross, st>>>(maps3, prm);
  return cudaGetLastError();
}

cudaError_t launch_gram_tm(const void* G, int dtype, int p, long long n, double* partials, unsigned int* counter,
                           double* K, int* status, cudaStream_t st) {
  gramtm::Params prm{};
  prm.row0 = 0;
  prm.ptotal = p;
  prm.finish = 1;
  prm.partials = partials;
  prm.counter = counter;
  prm.K = K;
  prm.status = status;
  cudaError_t e = cudaMemsetAsync(counter, 0, sizeof(unsigned int), st);
  if (e != cudaSuccess) return e;
  return launch_tri_rows(G, dtype, p, n, prm, st);
}

namespace {
cudaError_t launch_tri_rows(const void* G, int dtype, int p, long long n, gramtm::Params prm, cudaStream_t st) {
  gramtm::Maps maps;
  gramtm::Layout lay;
  if (!gramtm::build(G, dtype, p, n, maps, lay)) return cudaErrorInvalidValue;
  const int S = dtype == 0 ? 4 : 2;
  prm.p = p;
  prm.num_tiles = (n + lay.step - 1) / lay.step;
  prm.wait_cycles = g_tile_wait_cycles.load();
  const int sms = sm_count();
  const int grid = (int)(prm.num_tiles < sms ? prm.num_tiles : sms);
  const int pb = p <= 4 ? 4 : p <= 8 ? 8 : p <= 12 ? 12 : p <= 15 ? 15 : 16;
  const int naccp = (pb * (pb + 1) / 2 + 31) / 32 * 32;
  // two elements per shared load when every class's shift is even
  bool even = true;
  for (int c = 0; c < lay.q; ++c) even = even && (lay.shift[c] % 2 == 0);
  const int vec = even ? 2 : 1;
  const size_t stage_bytes = (size_t)p * gramtm::kTileCols * S;
  int depth = (int)(gramtm::kStageBudget / (gramtm::kTriWarps * stage_bytes));
  depth = depth < 1 ? 1 : depth > gramtm::kMaxDepth ? gramtm::kMaxDepth : depth;
  lay.depth = depth;
  const size_t smem = (size_t)gramtm::kTriWarps * depth * stage_bytes + (size_t)gramtm::kTriWarps * naccp * sizeof(double) +
                      (size_t)gramtm::kTriWarps * gramtm::kMaxDepth * sizeof(uint64_t) + 64;
  if (dtype == 0) return gramtm::dispatch_tri<float>(pb, vec, maps, prm, lay, grid, smem, st);
  return gramtm::dispatch_tri<__nv_bfloat16>(pb, vec, maps, prm, lay, grid, smem, st);
}
}  // namespace

}  // namespace fa
