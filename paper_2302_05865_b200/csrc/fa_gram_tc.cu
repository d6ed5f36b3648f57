// Gram pass on the 5th-generation tensor cores, for bf16 gradients with 16 < p <= 64 workers
// (K = G G^T needs 16 FMA per byte at p = 63, far beyond the fp32 pipes at HBM speed).
//
// One persistent block per SM (352 threads), four roles:
//   warp 0   : TMA producer.  The gradient matrix is a 2-D tensor (n columns x p rows, row stride n);
//              a box of 64 columns x 64 rows (rows >= p and columns >= n read as zero) lands in
//              shared memory in the 128-byte-swizzled K-major layout the MMA unit reads.  The
//              tensor-load unit delivers about 14 bytes per clock and SM for such 128-byte rows,
//              less than HBM supplies, so it fills three of the six stages only (the even tiles).
//   warps 6-9: loaders.  The other three stages (the odd tiles) are filled with 16-byte cp.async
//              copies written straight into the same swizzled layout, three tiles in flight.
//   warps 1, 10: MMA issuers.  One thread each issues tcgen05.mma (kind::f16, bf16 x bf16 -> fp32)
//              with the SAME shared-memory tile as A and B operand: D[64 x 64] += T T^T, 16 columns
//              per instruction, accumulator in tensor memory (eight accumulators used in turn).
//              Warp 1 takes the even tiles, warp 10 the odd ones: sixteen small instructions per
//              tile from one thread were slower than the feed.  tcgen05.commit frees the stage.
//   warps 2-5: read-out.  After every stage (256 columns) the fp32 accumulator (products are exact,
//              the running sum is fp32) is read out of tensor memory with tcgen05.ld and added into
//              fp32 registers; every eighth run these are folded into fp64 sums in shared memory.
// Block totals then go through the same last-block reduction as the fp32-pipe kernels.
// Needs 16-byte aligned rows (n % 8 == 0, base % 16 == 0); other shapes use the fp32-pipe kernel.
#include <cuda.h>
#include <cuda_bf16.h>

#include "fa_common.cuh"
#include "fa_tensor_map.cuh"
#include "fa_gram_finish.cuh"
#include "fa_kernels.h"

namespace fa {
namespace gramtc {

constexpr int kBoxCols = 64;                    // 128 bytes of bf16: one swizzle atom along K
constexpr int kBoxRows = 64;
constexpr int kBoxBytes = kBoxCols * kBoxRows * 2;   // 8 KiB
constexpr int kBoxesPerStage = 4;               // 256 columns per stage
constexpr int kStageBytes = kBoxBytes * kBoxesPerStage;
constexpr int kStages = 6;                      // 192 KiB of staging
constexpr int kFlushStages = 1;                 // 256 columns per fp32 accumulation run
constexpr int kFold = 8;                        // runs added in fp32 registers before the fp64 fold
constexpr int kLoaderWarps = 4;                 // warps 6..9 fill the loader stages with cp.async copies
constexpr int kMmaWarp2 = 6 + kLoaderWarps;       // second MMA issuer (odd tiles); warp 1 takes the even ones
constexpr int kThreads = 192 + 32 * kLoaderWarps + 32;
constexpr int kAccs = 8;               // 64-column accumulators in tensor memory, used in turn
constexpr int kTmemCols = 64 * kAccs;
static_assert(kAccs == 2 || kAccs == 4 || kAccs == 8, "tensor-memory allocations are powers of two");
constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + 256 + 64 * 64 * sizeof(double);

// Stages whose bit is set in kLoaderMask are filled by the loader warps, the others by the
// tensor-load thread; tile u goes to stage u mod kStages.
constexpr uint32_t kLoaderMask = 0x2A;
constexpr int kLoaderDepth = ((kLoaderMask >> 0) & 1) + ((kLoaderMask >> 1) & 1) + ((kLoaderMask >> 2) & 1) +
                             ((kLoaderMask >> 3) & 1) + ((kLoaderMask >> 4) & 1) + ((kLoaderMask >> 5) & 1);
static_assert(kLoaderDepth >= 1 && kLoaderDepth <= 3 && kLoaderMask < (1u << kStages), "loader stages");
__device__ __forceinline__ bool loader_stage(int s) { return (kLoaderMask >> s) & 1u; }
__device__ __forceinline__ bool loader_tile(long long u) { return loader_stage(static_cast<int>(u % kStages)); }
__device__ __forceinline__ long long next_loader_tile(long long u) {
  do { ++u; } while (!loader_tile(u));
  return u;
}

struct Params {
  int p;
  const uint4* G;            // the matrix as 16-byte chunks (rows start on 16-byte boundaries)
  long long n;
  long long num_tiles;       // stages' worth of columns in the whole matrix
  double* partials;
  unsigned int* counter;
  double* K;
  int* status;
};

// kind::f16 instruction descriptor: D fp32, A and B bf16, both K-major, N = 64, M = 64.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((64u >> 4) << 24);

// Shared-memory matrix descriptor for a K-major, 128-byte-swizzled tile: 8-row groups 1024 bytes
// apart (stride byte offset), leading byte offset unused (1), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

struct Bars {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t acc_full[kAccs];
  uint64_t acc_empty[kAccs];
  uint32_t tmem_base;
  int abort;
};

__device__ __forceinline__ void give_up(Bars* b, int* status) {
  b->abort = 1;
  if (status) atomicOr(status, kStTimeout);
}

__global__ void __launch_bounds__(kThreads, 1) gram_tc_kernel(const __grid_constant__ CUtensorMap tmap, Params prm) {
  extern __shared__ unsigned char smem_raw[];
  // stage buffers must sit on 1024-byte boundaries (swizzle atom = 8 rows x 128 bytes)
  unsigned char* stages =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  Bars* bars = reinterpret_cast<Bars*>(stages + (size_t)kStages * kStageBytes);
  double* dsum = reinterpret_cast<double*>(stages + (size_t)kStages * kStageBytes + 256);   // 64 x 64 fp64 sums
  static_assert(sizeof(Bars) <= 256, "barrier block");
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->full[s], loader_stage(s) ? kLoaderWarps : 1);
      mbar_init(&bars->empty[s], 1);
    }
    for (int a = 0; a < kAccs; ++a) { mbar_init(&bars->acc_full[a], 1); mbar_init(&bars->acc_empty[a], 4); }
    bars->abort = 0;
    fence_proxy_async();
  }
  if (warp == 1) {   // tensor memory: kTmemCols columns for this block (the only block on the SM)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int i = tid; i < 64 * 64; i += kThreads) dsum[i] = 0.0;
  if (warp >= 6 && warp < 6 + kLoaderWarps) {   // rows p..63 of the stages the loader warps fill are zeroed once and never written
    for (int s = 0; s < kStages; ++s)
      if (loader_stage(s))
      for (int i = (tid - 192) * 16; i < kStageBytes; i += 32 * kLoaderWarps * 16)
        *reinterpret_cast<uint4*>(stages + (size_t)s * kStageBytes + i) = make_uint4(0, 0, 0, 0);
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

  // tiles of this block: t = blockIdx.x, blockIdx.x + gridDim.x, ...
  const long long my_tiles = (prm.num_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x;
  const long long periods = (my_tiles + kFlushStages - 1) / kFlushStages;

  if (warp == 0) {
    // ---------------- TMA producer
    if (lane == 0) {
      long long issued = 0;
      bool ok = true;
      for (long long u = 0; u < my_tiles; ++u) {
        if (loader_tile(u)) continue;
        const int s = static_cast<int>(u % kStages);
        if (!mbar_wait(&bars->empty[s], static_cast<uint32_t>(((u / kStages) & 1) ^ 1)) ||
            *reinterpret_cast<volatile int*>(&bars->abort)) { ok = false; break; }
        const long long t = blockIdx.x + u * (long long)gridDim.x;
        mbar_arrive_expect_tx(&bars->full[s], kStageBytes);
        for (int q = 0; q < kBoxesPerStage; ++q)
          tma_load_2d(stages + (size_t)s * kStageBytes + (size_t)q * kBoxBytes, &tmap,
                      static_cast<int>(t * (kBoxesPerStage * kBoxCols) + q * kBoxCols), 0, &bars->full[s]);
        issued = u + 1;
      }
      if (!ok) {
        give_up(bars, prm.status);
        const long long first = issued > kStages ? issued - kStages : 0;   // copies still in flight must land
        for (long long u = first; u < issued; ++u)
          if (!loader_tile(u)) (void)mbar_wait(&bars->full[u % kStages], static_cast<uint32_t>((u / kStages) & 1));
      }
    }
  } else if (warp == 1 || warp == kMmaWarp2) {
    // ---------------- MMA issuers: one thread each, tiles of one parity (its own accumulators: tile u
    // uses accumulator u mod kAccs, and kAccs is even); a commit covers the issuing thread's MMAs
    static_assert(kFlushStages == 1 && kAccs % 2 == 0, "tiles alternate between the two issuers");
    if (lane == 0) {
      for (long long u = (warp == 1 ? 0 : 1); u < my_tiles; u += 2) {
        const int s = static_cast<int>(u % kStages);
        const long long period = u / kFlushStages;
        const int ab = static_cast<int>(period % kAccs);
        const bool first_of_period = (u % kFlushStages) == 0;
        if (first_of_period && period >= kAccs) {     // the epilogue must have drained this accumulator
          if (!mbar_wait(&bars->acc_empty[ab], static_cast<uint32_t>(((period / kAccs) - 1) & 1))) { give_up(bars, prm.status); break; }
        }
        if (!mbar_wait(&bars->full[s], static_cast<uint32_t>((u / kStages) & 1))) { give_up(bars, prm.status); break; }
        if (*reinterpret_cast<volatile int*>(&bars->abort)) break;
        tc_fence_after();
        const uint32_t sbase = smem_u32(stages + (size_t)s * kStageBytes);
        const uint32_t d = tmem_base + static_cast<uint32_t>(ab * 64);
#pragma unroll
        for (int q = 0; q < kBoxesPerStage; ++q) {
#pragma unroll
          for (int k = 0; k < kBoxCols / 16; ++k) {
            const uint64_t desc = smem_desc(sbase + q * kBoxBytes + k * 32);   // 16 bf16 = 32 bytes along K
            umma_bf16(d, desc, desc, (first_of_period && q == 0 && k == 0) ? 0u : 1u);
          }
        }
        umma_commit(&bars->empty[s]);             // stage reusable once these MMAs have read it
        if ((u % kFlushStages) == kFlushStages - 1 || u == my_tiles - 1) umma_commit(&bars->acc_full[ab]);
      }
    }
  } else if (warp >= 6 && warp < 6 + kLoaderWarps) {
    // ---------------- loader warps: the tensor-load unit delivers about 14 bytes per clock for boxes
    // with 128-byte rows, well below what HBM can supply, so every other tile comes in through the
    // load/store path instead: 16-byte asynchronous copies (cp.async; a warp covers the 512 contiguous
    // bytes of one row of the tile) straight into the layout the 128-byte swizzled tensor load would
    // have produced -- box q = 64 columns, row r at r * 128 bytes, 16-byte chunk c at position
    // c ^ (r mod 8).  As many tiles are in flight as there are loader stages; a tile is handed to the tensor
    // core once every thread's copies have landed and a proxy fence has made them visible to it.
    const int lt = tid - 192;
    const int chunks = prm.p * 32;                        // 16-byte chunks of a tile: p rows x 512 bytes
    const long long row_chunks = prm.n / 8;
    constexpr int kPer = 2048 / (32 * kLoaderWarps);      // chunks per thread and tile
    bool ok = true;
    auto fill = [&](long long u) {                        // wait for the stage of tile u, start its copies
      const int s = static_cast<int>(u % kStages);
      ok = mbar_wait(&bars->empty[s], static_cast<uint32_t>(((u / kStages) & 1) ^ 1)) &&
           !*reinterpret_cast<volatile int*>(&bars->abort);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      const long long t = blockIdx.x + u * (long long)gridDim.x;
      const long long chunk0 = t * (kBoxesPerStage * kBoxCols / 8);   // first chunk of the tile within a row
      const uint32_t sbase = smem_u32(stages + (size_t)s * kStageBytes);
#pragma unroll
      for (int k = 0; k < kPer; ++k) {
        const int idx = lt + k * 32 * kLoaderWarps;
        const int r = idx >> 5, ch = idx & 31;
        if (idx < chunks) {
          const bool inside = chunk0 + ch < row_chunks;   // chunks past the end of the row are zero-filled
          const uint4* src = inside ? prm.G + (size_t)r * row_chunks + chunk0 + ch : prm.G;
          const uint32_t dst = sbase + (ch >> 3) * kBoxBytes + r * 128 + (((ch & 7) ^ (r & 7)) << 4);
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(inside ? 16 : 0)
                       : "memory");
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // loader tiles in order; `head` is the next one to start, `tail` the next one to hand over;
    // kLoaderDepth of them (one per loader stage) are in flight
    long long head = next_loader_tile(-1), tail = head;
    for (int i = 0; i < kLoaderDepth - 1 && head < my_tiles && ok; ++i) {
      fill(head);
      head = next_loader_tile(head);
    }
    while (tail < my_tiles && ok) {
      const bool more = head < my_tiles;
      if (more) {
        fill(head);
        head = next_loader_tile(head);
        if (!ok) break;
      }
      // copy groups complete in order: with kLoaderDepth groups committed the oldest has landed when
      // at most kLoaderDepth - 1 are pending; near the end simply wait for all of them
      if (more && kLoaderDepth == 3) asm volatile("cp.async.wait_group 2;" ::: "memory");
      else if (more && kLoaderDepth == 2) asm volatile("cp.async.wait_group 1;" ::: "memory");
      else asm volatile("cp.async.wait_group 0;" ::: "memory");
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->full[static_cast<int>(tail % kStages)]);
      tail = next_loader_tile(tail);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");   // nothing of this thread's is in flight at exit
    if (!ok && lane == 0) give_up(bars, prm.status);
  } else if (warp < 6) {
    // ---------------- epilogue: warp w reads TMEM lanes 32*(w%4) .. +31; with M = 64 only the first
    // 16 lanes of each quarter carry rows: row = 16*(w%4) + lane
    const int quarter = warp & 3;
    const int row = 16 * quarter + (lane & 15);
    // Read-out per 256-column run: the fp32 values are added into fp32 registers (round to nearest;
    // kFold runs), and only every kFold-th run are these folded into the fp64 sums, which live in
    // shared memory (entry (row, j) at j * 64 + row: the rows of a warp are neighbours).  Converting
    // and adding all 64 values in fp64 after every run made the read-out the slowest stage of the
    // pipeline (2300 cycles per run).
    float facc[64];
#pragma unroll
    for (int j = 0; j < 64; ++j) facc[j] = 0.f;
    int in_fold = 0;
    bool first_fold = true;
    auto fold = [&]() {
      if (lane < 16) {
#pragma unroll
        for (int j = 0; j < 64; ++j) dsum[j * 64 + row] += static_cast<double>(facc[j]);
      }
#pragma unroll
      for (int j = 0; j < 64; ++j) facc[j] = 0.f;
      first_fold = false;
      in_fold = 0;
    };
    bool ok = true;
    for (long long period = 0; period < periods && ok; ++period) {
      const int ab = static_cast<int>(period % kAccs);
      if (!mbar_wait(&bars->acc_full[ab], static_cast<uint32_t>((period / kAccs) & 1))) {
        if (lane == 0) give_up(bars, prm.status);
        ok = false;
        break;
      }
      tc_fence_after();
      uint32_t v0[32], v1[32];
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(32 * quarter) << 16) + static_cast<uint32_t>(ab * 64);
      tmem_ld32(taddr, v0);
      tmem_ld32(taddr + 32, v1);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->acc_empty[ab]);
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        facc[j] += __uint_as_float(v0[j]);
        facc[32 + j] += __uint_as_float(v1[j]);
      }
      if (++in_fold == kFold) fold();
    }
    if (in_fold > 0 || first_fold) fold();
    if (lane < 16 && row < prm.p) {
      for (int j = row; j < prm.p; ++j)
        prm.partials[(size_t)gram::canon_index(row, j, prm.p) * gridDim.x + blockIdx.x] = dsum[j * 64 + row];
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
  gram::finish_gram(prm.partials, prm.counter, prm.K, prm.p, &bars->abort);
}

}  // namespace gramtc

// ---- host side
bool gram_tc_eligible(const void* G, int dtype, int p, long long n) {
  return dtype == 1 && p > 16 && p <= 64 && n % 8 == 0 && (reinterpret_cast<uintptr_t>(G) % 16) == 0 &&
         n < (1LL << 31) && encode_tiled() != nullptr;
}

cudaError_t launch_gram_tc(const void* G, int p, long long n, double* partials, unsigned int* counter, double* K,
                           int* status, cudaStream_t st) {
  EncodeTiledFn enc = encode_tiled();
  if (!enc) return cudaErrorNotSupported;
  CUtensorMap tmap;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(n), static_cast<cuuint64_t>(p)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(n) * 2};
  const cuuint32_t box[2] = {gramtc::kBoxCols, gramtc::kBoxRows};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(G), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  gramtc::Params prm{};
  prm.p = p;
  prm.G = static_cast<const uint4*>(G);
  prm.n = n;
  const long long stage_cols = gramtc::kBoxesPerStage * gramtc::kBoxCols;
  prm.num_tiles = (n + stage_cols - 1) / stage_cols;
  prm.partials = partials;
  prm.counter = counter;
  prm.K = K;
  prm.status = status;
  const int sms = sm_count();
  const int grid = static_cast<int>(prm.num_tiles < sms ? prm.num_tiles : sms);
  cudaError_t e = cudaMemsetAsync(counter, 0, sizeof(unsigned int), st);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gramtc::gram_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           static_cast<int>(gramtc::kSmemBytes));
  if (e != cudaSuccess) return e;
  gramtc::gram_tc_kernel<<<grid, gramtc::kThreads, gramtc::kSmemBytes, st>>>(tmap, prm);
  return cudaGetLastError();
}

}  // namespace fa
