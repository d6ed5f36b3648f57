// fa_gram_static: the Gram pass for callers that cannot allocate device memory.
//
// fa_gram needs a caller-provided workspace for the per-block partial sums.  Some callers have
// no way to obtain one: code running inside a communication or RPC callback, a plugin that is
// handed only its input and output buffers, a process whose memory pool is owned and fully
// committed by another runtime, or any place where a cudaMalloc would synchronise the device.
// For them the partial sums live in a fixed array inside this library's device image.  The
// array exists once per GPU that loads the library and stays until the process exits.
#include <stdint.h>

#include <atomic>

#include "../../include/fa.h"
#include "fa_kernels.h"

namespace {

// 160 block slots of at most 32*33/2 partial inner products each (675,840 bytes) + a 256-byte counter.
constexpr size_t kScratchDoubles = (size_t)FA_STATIC_MAX_BLOCKS * (FA_STATIC_MAX_P * (FA_STATIC_MAX_P + 1) / 2);
static __device__ __align__(256) double g_gram_scratch[kScratchDoubles + 32];

// Device address of the array, looked up once per device.  In host code `g_gram_scratch` is only a
// handle for the runtime; the kernels need the address that cudaGetSymbolAddress returns.
double* scratch_address(int* rc) {
  static std::atomic<double*> cached[64];              // per device; concurrent first calls look up the same address
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *rc = FA_ERR_CUDA; return nullptr; }
  double* addr = cached[dev].load(std::memory_order_acquire);
  if (!addr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_gram_scratch) != cudaSuccess || !ptr) { *rc = FA_ERR_CUDA; return nullptr; }
    addr = static_cast<double*>(ptr);
    cached[dev].store(addr, std::memory_order_release);
  }
  *rc = FA_OK;
  return addr;
}

}  // namespace

extern "C" int fa_gram_static(const void* G, int dtype, int p, long long n, double* K, void* stream) {
  if (!G || !K || p < 1 || n < 1 || (dtype != FA_F32 && dtype != FA_BF16)) return FA_ERR_ARG;
  if (p > FA_STATIC_MAX_P) return FA_ERR_STATIC_LIMIT;
  if ((reinterpret_cast<uintptr_t>(G) % (dtype == FA_F32 ? 4 : 2)) != 0 || (reinterpret_cast<uintptr_t>(K) % 8) != 0)
    return FA_ERR_ALIGN;
  if (fa::gram_num_blocks(p, n, dtype) > FA_STATIC_MAX_BLOCKS) return FA_ERR_STATIC_LIMIT;
  int rc = FA_OK;
  double* scratch = scratch_address(&rc);
  if (!scratch) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The counter (first 256 bytes) is cleared by a memset node on the stream before the kernel;
  // every block overwrites all of its partial sums and only those are read back, so nothing else
  // left in the array by an earlier call needs clearing.
  unsigned int* counter = reinterpret_cast<unsigned int*>(scratch);
  if (fa::launch_gram(G, dtype, p, n, scratch + 32, counter, K, nullptr, st) != cudaSuccess) return FA_ERR_CUDA;
  return FA_OK;
}
