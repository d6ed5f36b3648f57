// Shared between the Gram kernels that are fed by TMA tensor loads: the tensor maps of the row classes
// and how a staged tile is laid out (see fa_gram_tm.cu for the scheme).
#pragma once
#include "fa_tensor_map.cuh"

namespace fa {
namespace gramtm {

constexpr int kTileCols = 256;               // box width in elements
constexpr int kMaxClasses = 4;
constexpr int kFlushCols = 64;               // fp32 running sums cover at most this many columns
constexpr int kTriWarps = 12;                // p <= 16: 12 warps, 168 registers each
constexpr int kMaxDepth = 4;                 // stages per warp
constexpr size_t kStageBudget = 184 * 1024;  // bytes of shared memory for all stages

struct Maps { CUtensorMap map[kMaxClasses]; };

struct Layout {
  int depth;                   // stages per warp
  int q;                       // row classes
  int step;                    // columns a tile advances by
  int rows[kMaxClasses];       // rows in class c
  int rowbase[kMaxClasses];    // staged row index of the first row of class c
  int shift[kMaxClasses];      // elements between the map's row start and the row's own start
};

// Host: tensor maps and layout for a p x n matrix at G (16-byte aligned); false when the shape needs
// more than kMaxClasses row classes or the driver's encoder is not available.
bool build(const void* G, int dtype, int p, long long n, Maps& maps, Layout& lay);
bool available(const void* G, int dtype, long long n);

}  // namespace gramtm
}  // namespace fa
