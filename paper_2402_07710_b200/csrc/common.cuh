// Internal definitions shared by the CUDA translation units of spconv_b200.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <functional>
#include <vector>

#include "spconv_b200.h"

namespace spconv {

constexpr int kTileRows = 128;        // output rows per tensor-core tile (= UMMA M)
constexpr int kMaxCoord = 65534;      // each of b,x,y,z fits 16 bits; 0xFFFF is reserved for the empty key
constexpr uint64_t kEmptyKey = ~0ull;
constexpr int kMaskWordsMax = 4;      // tile offset masks cover kvol <= 128

// Device status word bits (OR-ed by kernels, read by the host).
enum : uint32_t {
  kDevCoordRange = 1u,
  kDevDuplicate = 2u,
  kDevTableFull = 4u,
  kDevPipeTimeout = 8u,
};

struct KmapDeviceArrays {
  int32_t* out_coords = nullptr;   // [n_out][4]
  int32_t* nbr = nullptr;          // [kvol][n_out]
  int32_t* pair_in = nullptr;      // [P]
  int32_t* pair_out = nullptr;     // [P]
  int32_t* tile_rows = nullptr;    // [n_tiles][128]
  int32_t* tile_nbr = nullptr;     // [n_tiles][kvol][128]   input rows of block (tile, k), present rows first (compacted), then -1
  uint8_t* tile_crow = nullptr;    // [n_tiles][kvol][128]   tile row (0..127) that each compacted entry feeds
  uint32_t* tile_mask = nullptr;   // [n_tiles][mask_words]  bit k set <=> block (tile, k) has a non-empty row
  int32_t* sorted_tiles = nullptr; // [n_tiles][1 + mask_words]  schedule: tiles in descending order of their number of
                                   // non-empty blocks, each record = tile index, then the tile's offset mask words
  uint32_t* tile_absent = nullptr; // [n_tiles][kvol][4]  bit r of the 128-bit word set <=> row r of block (tile, k) has no input
  uint32_t* status = nullptr;      // [1] device status word for forward kernels
};

}  // namespace spconv

struct spconv_kmap {
  int kernel = 0, stride = 0, dilation = 0, submanifold = 0, inverse = 0, kvol = 0;
  int device = 0;
  cudaStream_t stream = nullptr;      // stream the map was built on; its memory is released in this stream's order
  int mask_words = 1;
  int32_t n_tiles = 0;
  int64_t n_in = 0, n_out = 0, total_pairs = 0, tile_blocks = 0;
  spconv::KmapDeviceArrays d;
  std::vector<int64_t> offset_start;  // host [kvol+1]
};

namespace spconv {

// kmap.cu
// before_wait (optional, submanifold maps only): called once every kernel of the build has been enqueued and before
// the host waits for the device's report, with the handle's sizes and device pointers set (pair count and block
// count are not known yet); what it enqueues on the stream runs behind the build without a host round trip between.
// fine_coords (optional): builds the map of the inverse convolution instead: `coords` are then the coarse positions
// (rows of the input features), fine_coords [n_fine][4] the output rows, and submanifold must be 0.
int build_kmap_impl(const int32_t* coords, int64_t n, int stride, int dilation, int kernel, int submanifold,
                    cudaStream_t stream, spconv_kmap** out, const std::function<int(spconv_kmap*)>* before_wait = nullptr,
                    const int32_t* fine_coords = nullptr, int64_t n_fine = 0, const int* dense_grid = nullptr, int rows_as_given = 0);
// dense_grid (optional, host int[4] = B, X, Y, Z): the location table is a dense array over that grid instead of the
// hash table (submanifold maps with kernel size 1 or 3 only; the caller checks the shape and its size).
void destroy_kmap_impl(spconv_kmap* km);
void set_kmap_test_table_slots(long long slots);          // test hook, see spconv_test_hook

int voxelize_impl(const float* points, int64_t n, int point_stride, int n_feat, int batch_index, const float* origin,
                  const float* voxel_size, const int32_t* grid_shape, int32_t* coords_out, float* feats_out, int32_t* counts_out,
                  int64_t capacity, int64_t* n_voxels_host, cudaStream_t stream);

// forward_simt.cu
int forward_simt(const void* feats, const void* w, const spconv_kmap* km, void* out, int cin, int cout,
                 spconv_dtype_t dtype, cudaStream_t stream);

// forward_tc.cu
bool forward_tc_supported(int cin, int cout, spconv_dtype_t dtype);
void set_forward_tc_timeline(unsigned long long* buf);
void set_forward_tc_test_wait_limit_us(long long us);     // test hook, see spconv_test_hook
// strict_order: the kernel map may still be under construction by work that precedes the launch in the stream
// (the launch comes from build_kmap_impl's before_wait), so the kernel must not read it ahead of that work.
// one_offset_per_step: never take several offsets of a tile in one pipeline step (SPCONV_ALGO_TCGEN05_SINGLE).
int forward_tc(const void* feats, const void* w, const spconv_kmap* km, void* out, int cin, int cout,
               spconv_dtype_t dtype, cudaStream_t stream, bool strict_order = false, bool one_offset_per_step = false);

inline int dtype_size(spconv_dtype_t t) { return t == SPCONV_F32 ? 4 : 2; }

#define SPCONV_CUDA_TRY(expr)                          \
  do {                                                 \
    cudaError_t _e = (expr);                           \
    if (_e != cudaSuccess) {                           \
      (void)cudaGetLastError();                        \
      return _e == cudaErrorMemoryAllocation ? SPCONV_ERR_ALLOC : SPCONV_ERR_CUDA; \
    }                                                  \
  } while (0)

}  // namespace spconv
