// Kernel-map construction: location table (GPU hash table), offset table, per-offset pairs,
// output coordinates of strided convolution, and the tile plan of the tensor-core forward.
//
// Paper correspondence: "Create Location Table" (Sec. III-C.1) -> k_insert; "Create Offset Table"
// (Sec. III-C.2) -> k_subm_probe; the strided "lookup" / "unique points" kernels and the atomic
// counter of Sec. III-D -> k_strided_candidates / k_owner_* (ownership by atomicMin instead of an
// atomic counter, so the output numbering is the same on every run).
#include <cooperative_groups.h>
#include <cub/device/device_radix_sort.cuh>

#include <algorithm>
#include <atomic>
#include <chrono>
#include <functional>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include <cstdio>
#include <cstdlib>

#include "common.cuh"

namespace spconv {
namespace {

// Programmatic dependent launch.  A kernel started through launch_chained() may be scheduled while the kernel
// before it in the stream is still draining (its blocks then sit at chain_begin() until that kernel is complete
// and its memory visible), which hides the launch latency between the small kernels of a build.  chain_begin()
// is the first statement of every kernel that takes part; in a kernel launched the ordinary way it does nothing.
__device__ __forceinline__ void chain_begin() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
#ifdef SPCONV_KMAP_TIMELINE
// Development builds: globaltimer stamps of block 0 / thread 0 at the start (after the dependency wait) and the end of
// the build's kernels, slot 2 * id and 2 * id + 1.
__device__ unsigned long long g_kmap_timeline[32];
__device__ __forceinline__ void tl_stamp(int slot) {
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); g_kmap_timeline[slot] = t; }
}
#define SPCONV_TL(slot) tl_stamp(slot)
#define SPCONV_TL_RAW(slot, t) g_kmap_timeline[slot] = (t)
#else
#define SPCONV_TL(slot)
#define SPCONV_TL_RAW(slot, t)
#endif
// The fills a build starts with (location table and filter to all ones, totals to zero, the strided path's second
// table and owner words), as one kernel in the chain instead of separate memset nodes, which programmatic dependent
// launch cannot chain: between two builds of a sequence the launch latencies of those nodes were dead time.
struct FillRegions {
  uint4* ptr[4];
  unsigned long long count16[4];   // 16-byte words
  uint32_t value[4];
};
__global__ void __launch_bounds__(256) k_fill_regions(const __grid_constant__ FillRegions regions);

template <class... Params, class... Args>
cudaError_t launch_chained(void (*kernel)(Params...), dim3 grid, dim3 block, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t config = {};
  config.gridDim = grid;
  config.blockDim = block;
  config.dynamicSmemBytes = 0;
  config.stream = stream;
  cudaLaunchAttribute attribute[1];
  attribute[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attribute[0].val.programmaticStreamSerializationAllowed = 1;
  config.attrs = attribute;
  config.numAttrs = 1;
  return cudaLaunchKernelEx(&config, kernel, Params(args)...);
}

constexpr int kBlock = 256;

__device__ __forceinline__ uint64_t pack_key(int b, int x, int y, int z) {
  return (uint64_t(uint32_t(b)) << 48) | (uint64_t(uint32_t(x)) << 32) | (uint64_t(uint32_t(y)) << 16) |
         uint64_t(uint32_t(z));
}
__device__ __forceinline__ bool in_range(int v) { return uint32_t(v) <= uint32_t(kMaxCoord); }

// Offset k of a K^3 kernel as its three indices (k = (a*K + b)*K + c), from a table the host fills and passes as a
// kernel parameter: the runtime divisions this replaces were half of the probe kernels' instructions.
struct OffsetIndex {
  unsigned char v[128][4];
  int n;   // entries filled (kvol), or 0 when kvol > 128: then the kernels divide
};
__device__ __forceinline__ void offset_index(const OffsetIndex& t, int k, int K, int& a, int& b, int& c) {
  if (t.n != 0) {
    const uint32_t w = reinterpret_cast<const uint32_t*>(&t.v[0][0])[k];
    a = int(w & 255u); b = int((w >> 8) & 255u); c = int((w >> 16) & 255u);
  } else {
    a = k / (K * K); b = (k / K) % K; c = k % K;
  }
}
OffsetIndex make_offset_index(int K) {
  OffsetIndex t = {};
  const int kvol = K * K * K;
  if (kvol > 128) return t;
  for (int k = 0; k < kvol; ++k) {
    t.v[k][0] = (unsigned char)(k / (K * K)); t.v[k][1] = (unsigned char)((k / K) % K); t.v[k][2] = (unsigned char)(k % K);
  }
  t.n = kvol;
  return t;
}

// 32-bit mix of the two key halves (two independent multiplies, then one round of xor-shift-multiply): a short
// dependency chain, where a 64-bit finaliser's two dependent wide multiplies were most of a lookup's instructions.
__device__ __forceinline__ uint32_t hash_key(uint64_t k) {
  uint32_t h = (uint32_t(k) * 0x9E3779B1u) ^ (uint32_t(k >> 32) * 0x85EBCA77u);
  h ^= h >> 15; h *= 0x2C1B3C6Du; h ^= h >> 12;
  return h;
}

// Open addressing, linear probing.  Returns the slot that holds `key` (inserting it if absent) or -1
// if the bounded probe sequence found neither the key nor a free slot.  *was_present tells which.
// A slot is STRIDE 64-bit words wide and starts with its key.
template <int STRIDE>
__device__ __forceinline__ int table_insert(uint64_t* keys, uint32_t capmask, uint64_t key, bool* was_present) {
  uint32_t slot = hash_key(key) & capmask;
  for (uint32_t probe = 0; probe <= capmask; ++probe) {
    unsigned long long old = atomicCAS(reinterpret_cast<unsigned long long*>(keys + size_t(slot) * STRIDE),
                                       (unsigned long long)kEmptyKey, (unsigned long long)key);
    if (old == kEmptyKey) { *was_present = false; return int(slot); }
    if (old == key) { *was_present = true; return int(slot); }
    slot = (slot + 1) & capmask;
  }
  return -1;
}

// The location table keeps key and row index side by side in 16-byte slots (key | row | unused), so that a lookup
// that hits costs one memory request: the row arrives with the key it is compared against.
struct __align__(16) LocSlot { uint64_t key; int32_t row; int32_t unused; };
__device__ __forceinline__ LocSlot load_slot(const LocSlot* __restrict__ table, uint32_t slot) {
  const ulonglong2 raw = __ldg(reinterpret_cast<const ulonglong2*>(table) + slot);
  LocSlot s;
  s.key = raw.x; s.row = int32_t(uint32_t(raw.y)); s.unused = 0;
  return s;
}
__device__ __forceinline__ int table_find(const LocSlot* __restrict__ table, uint32_t capmask, uint64_t key) {
  uint32_t slot = hash_key(key) & capmask;
  for (uint32_t probe = 0; probe <= capmask; ++probe) {
    const LocSlot s = load_slot(table, slot);
    if (s.key == key) return s.row;
    if (s.key == kEmptyKey) return -1;
    slot = (slot + 1) & capmask;
  }
  return -1;
}

// Occupancy filter in front of the location table: one bit per cell of a 256 x 256 x 64 window onto which all
// positions are folded (x also shifted by the batch index), CLEAR where some inserted position folds to the cell
// (so that the byte pattern that empties the table's keys, 0xFF, also empties the filter).  A set bit proves that
// the table does not hold the position: five of six neighbour lookups of a surface-like input end there, with one
// read that neighbouring threads share (z runs along the bits of a word, y along the words of a line), instead of
// a read of a hashed, unshared table slot.  A clear bit proves nothing; the table decides.
constexpr uint32_t kOccWords = 131072;   // 4 Mi bits
__device__ __forceinline__ uint32_t occ_word(int b, int x, int y, int z) {
  return ((uint32_t(x + 37 * b) & 255u) << 9) | ((uint32_t(y) & 255u) << 1) | ((uint32_t(z) >> 5) & 1u);
}

// ---------------------------------------------------------------------------------------------
// Location table: coordinate -> input row.  One int4 load per voxel.
__global__ void k_insert(const int4* __restrict__ coords, int n, LocSlot* table, uint32_t capmask,
                         uint32_t* status, int4* __restrict__ coords_copy, uint32_t* __restrict__ occ = nullptr) {
  chain_begin();
  SPCONV_TL(0);
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int4 c = coords[i];
  if (coords_copy != nullptr) coords_copy[i] = c;   // submanifold: the output coordinates are the input's
  if (!(in_range(c.x) && in_range(c.y) && in_range(c.z) && in_range(c.w))) { atomicOr(status, kDevCoordRange); return; }
  bool present;
  const int slot = table_insert<2>(reinterpret_cast<uint64_t*>(table), capmask, pack_key(c.x, c.y, c.z, c.w), &present);
  if (slot < 0) { atomicOr(status, kDevTableFull); return; }
  if (present) { atomicOr(status, kDevDuplicate); return; }
  table[slot].row = i;
  if (occ != nullptr) atomicAnd(occ + occ_word(c.x, c.y, c.z, c.w), ~(1u << (c.w & 31)));
  SPCONV_TL(1);
}

// Offset table for submanifold convolution, offset-major: nbr[k][j] = input row at c_j + d*(kvec - r), or -1.
// grid = (ceil(n/256), kvol).  Also counts the hits of each block for the pair compaction.
__global__ void k_subm_probe(const int4* __restrict__ coords, int n, int K, int dil, const LocSlot* __restrict__ table,
                             uint32_t capmask, int32_t* __restrict__ nbr,
                             int32_t* __restrict__ blockcnt, unsigned* __restrict__ offset_cnt, const __grid_constant__ OffsetIndex index) {
  chain_begin();
  const int k = blockIdx.y;
  const int j = blockIdx.x * kBlock + threadIdx.x;
  const int r = (K - 1) / 2;
  int ia, ib, ic;
  offset_index(index, k, K, ia, ib, ic);
  const int dx = dil * (ia - r), dy = dil * (ib - r), dz = dil * (ic - r);
  int v = -1;
  if (j < n) {
    const int4 c = coords[j];
    const int x = c.y + dx, y = c.z + dy, z = c.w + dz;
    if ((dx | dy | dz) == 0) v = j;
    else if (in_range(x) && in_range(y) && in_range(z)) v = table_find(table, capmask, pack_key(c.x, x, y, z));
    nbr[size_t(k) * n + j] = v;
  }
  const int cnt = __syncthreads_count(v >= 0);
  if (threadIdx.x == 0) {
    blockcnt[size_t(k) * gridDim.x + blockIdx.x] = cnt;
    if (offset_cnt != nullptr && cnt != 0) atomicAdd(&offset_cnt[k], unsigned(cnt));   // per-offset totals (order-independent sums)
  }
}


// ---------------------------------------------------------------------------------------------
// Location table as a dense array over a stated grid (Sec. III-C.1: "a three-dimensional array as location
// table", the alternative the paper prefers where the domain is confined): cell (b, x, y, z) of a B x X x Y x Z
// grid holds the input row at that position or -1, at index ((b*X + x)*Y + y)*Z + z (z fastest, as the rows of a
// sorted input and the kernel offsets run).  A lookup is one read at a computed address, without hashing or
// probing; neighbouring positions are neighbouring words.
struct GridDims { int b, x, y, z; };
__device__ __forceinline__ bool in_grid(const GridDims& g, int b, int x, int y, int z) {
  return uint32_t(b) < uint32_t(g.b) && uint32_t(x) < uint32_t(g.x) && uint32_t(y) < uint32_t(g.y) && uint32_t(z) < uint32_t(g.z);
}
__device__ __forceinline__ size_t grid_cell(const GridDims& g, int b, int x, int y, int z) {
  return ((size_t(b) * g.x + x) * g.y + y) * g.z + z;
}
// One thread per input row, like the paper's createLCTKernel, with the batch index in the cell address and the
// two checks the printed kernel lacks: positions outside the grid and duplicates are reported.
__global__ void k_insert_dense(const int4* __restrict__ coords, int n, int32_t* __restrict__ cells, const __grid_constant__ GridDims grid,
                               uint32_t* status) {
  chain_begin();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int4 c = coords[i];
  if (!in_grid(grid, c.x, c.y, c.z, c.w)) { atomicOr(status, kDevCoordRange); return; }
  if (atomicCAS(cells + grid_cell(grid, c.x, c.y, c.z, c.w), -1, i) != -1) atomicOr(status, kDevDuplicate);
}

// ---------------------------------------------------------------------------------------------
// Offset table, every offset of one output row per thread (kernel volumes up to 32).
//   MODE 0, submanifold (Sec. III-C.2): row j looks at p_j + d*(kvec - r); the centre offset is j itself.
//   MODE 1, inverse convolution (Sec. III-E): the table was built over the coarse positions; fine position p_j is
//           related to coarse cell (p_j + pad - d*kvec) / s through offset kvec where that is a whole cell >= 0.
// The occupancy filter is consulted for every offset first (see occ_word); the table lookups of the offsets it
// does not rule out follow four at a time.  The table is written in two layouts: offset-major nbr[k][j] (the caller's
// view, the pair emission and the CUDA-core forward read it along j) and row-major rows of 32 entries
// nbr_rows[j][k] (the paper's OFT layout; the tile plan reads whole rows of permuted j).  row_mask[j] has bit k
// set where the row has an input through offset k.  Per block and offset the number of hits goes to blockcnt
// (the pair emission's bases), per offset the total to offset_cnt.
// DENSE: the location table is the dense array of k_insert_dense (`table` then points at its cells and `grid`
// gives its shape): every offset's cell is read directly, all reads in flight together, and there is no filter.
template <int K, int MODE, bool DENSE = false>
__global__ void __launch_bounds__(kBlock)
k_probe_rows(const int4* __restrict__ qcoords, int nq, int dil, int stride, const LocSlot* __restrict__ table,
             uint32_t capmask, const uint32_t* __restrict__ occ, int32_t* __restrict__ nbr,
             int32_t* __restrict__ nbr_rows, uint32_t* __restrict__ row_mask, int32_t* __restrict__ blockcnt,
             unsigned* __restrict__ offset_cnt, int4* __restrict__ coords_copy, uint32_t* __restrict__ status,
             const __grid_constant__ GridDims grid) {
  chain_begin();
  SPCONV_TL(2);
  constexpr int KV = K * K * K;
  static_assert(KV <= 32, "kernel volume");
  constexpr int r = (K - 1) / 2;
  __shared__ int s_v[KV][kBlock];   // the row's entries, written at run-time offsets, read back by the same thread
  __shared__ unsigned s_cnt[32];
  if (threadIdx.x < 32) s_cnt[threadIdx.x] = 0u;
  __syncthreads();
  const int tid = threadIdx.x, lane = tid & 31;
  const int j = blockIdx.x * kBlock + tid;
  const bool live = j < nq;
  int4 c = make_int4(0, 0, 0, 0);
  if (live) {
    c = qcoords[j];
    if (coords_copy != nullptr) coords_copy[j] = c;
  }
  bool usable = live;
  if (MODE == 1 && live && !(in_range(c.x) && in_range(c.y) && in_range(c.z) && in_range(c.w))) {
    atomicOr(status, kDevCoordRange);
    usable = false;
  }
  const int pad = dil * r;
  const bool pow2 = (stride & (stride - 1)) == 0;
  const int shift = __ffs(stride) - 1;
  // Position offset k of this row looks at; false if there is none (off the grid, out of range, the row itself).
  auto target = [&](int k, int& x, int& y, int& z) -> bool {
    const int a = k / (K * K), b = (k / K) % K, cc = k % K;
    if (MODE == 0) {
      x = c.y + dil * (a - r); y = c.z + dil * (b - r); z = c.w + dil * (cc - r);
      return usable && !(a == r && b == r && cc == r) && in_range(x) && in_range(y) && in_range(z);
    }
    const int nx = c.y + pad - dil * a, ny = c.z + pad - dil * b, nz = c.w + pad - dil * cc;
    const bool on_grid = pow2 ? (((nx | ny | nz) & (stride - 1)) == 0) : (nx % stride == 0 && ny % stride == 0 && nz % stride == 0);
    x = pow2 ? nx >> shift : nx / stride; y = pow2 ? ny >> shift : ny / stride; z = pow2 ? nz >> shift : nz / stride;
    return usable && nx >= 0 && ny >= 0 && nz >= 0 && on_grid && in_range(x) && in_range(y) && in_range(z);
  };
  // 1. candidates: offsets whose position the occupancy filter does not rule out (all reads in flight together)
  uint32_t cand = 0u;
  if constexpr (DENSE) {
    const int32_t* cells = reinterpret_cast<const int32_t*>(table);
    int got[KV];
#pragma unroll
    for (int k = 0; k < KV; ++k) {
      int x, y, z;
      const bool valid = target(k, x, y, z) && in_grid(grid, c.x, x, y, z);
      got[k] = valid ? __ldg(cells + grid_cell(grid, c.x, x, y, z)) : -1;
    }
#pragma unroll
    for (int k = 0; k < KV; ++k) s_v[k][tid] = (MODE == 0 && k == (r * K + r) * K + r && live) ? j : got[k];
  } else {
    // The filter keeps the 64 z-positions of a line (b, x, y) in two neighbouring words, so one 8-byte load serves the
    // K offsets of a line: K x K loads per row instead of K^3.
    uint2 line[K * K];
#pragma unroll
    for (int l = 0; l < K * K; ++l) {
      int x, y, z;
      // (a line is read if any of its K offsets has a position at all; x and y are the same for all of them)
      bool any = false;
#pragma unroll
      for (int cc = 0; cc < K; ++cc) { int x2, y2, z2; if (target(l * K + cc, x2, y2, z2)) { any = true; x = x2; y = y2; z = z2; } }
      line[l] = make_uint2(0xFFFFFFFFu, 0xFFFFFFFFu);
      if (any) line[l] = occ != nullptr ? __ldg(reinterpret_cast<const uint2*>(occ + (occ_word(c.x, x, y, z) & ~1u))) : make_uint2(0u, 0u);
    }
#pragma unroll
    for (int k = 0; k < KV; ++k) {
      int x, y, z;
      const bool valid = target(k, x, y, z);
      const uint32_t w = (z & 32) ? line[k / K].y : line[k / K].x;
      const uint32_t out = valid ? ((w >> (z & 31)) & 1u) : 1u;   // 1: ruled out
      cand |= (out ^ 1u) << k;
      s_v[k][tid] = (MODE == 0 && k == (r * K + r) * K + r && live) ? j : -1;
    }
  }
  // 2. the candidates' table lookups, four at a time
  while (cand != 0u) {
    constexpr int B = 4;
    int kk[B];
    uint64_t key[B];
    LocSlot got[B];
    uint32_t slot[B];
#pragma unroll
    for (int u = 0; u < B; ++u) {
      kk[u] = -1;
      key[u] = kEmptyKey; got[u].key = kEmptyKey; got[u].row = -1; slot[u] = 0u;
      if (cand != 0u) {
        kk[u] = __ffs(int(cand)) - 1;
        cand &= cand - 1u;
        int x, y, z;
        target(kk[u], x, y, z);
        key[u] = pack_key(c.x, x, y, z);
        slot[u] = hash_key(key[u]) & capmask;
        got[u] = load_slot(table, slot[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < B; ++u) {
      if (kk[u] < 0) continue;
      LocSlot g = got[u];
      for (uint32_t probe = 0; probe <= capmask; ++probe) {
        if (g.key == key[u]) { s_v[kk[u]][tid] = g.row; break; }
        if (g.key == kEmptyKey) break;
        slot[u] = (slot[u] + 1) & capmask;
        g = load_slot(table, slot[u]);
      }
    }
  }
  // 3. the row's entries leave in both layouts, with the row's offset set and the block's hit counts
  uint32_t mask = 0u;
  int v[KV];
#pragma unroll
  for (int k = 0; k < KV; ++k) {
    v[k] = s_v[k][tid];
    const bool present = v[k] >= 0;
    mask |= present ? (1u << k) : 0u;
    if (live) nbr[size_t(k) * nq + j] = v[k];
    const unsigned ballot = __ballot_sync(0xffffffffu, present);
    if (lane == 0 && ballot != 0u) atomicAdd(&s_cnt[k], unsigned(__popc(ballot)));
  }
  if (live) row_mask[j] = mask;
  // Row-major copy: the warp writes its 32 rows together, eight lanes per row (16 bytes each), so that a store
  // instruction covers four whole rows instead of touching 32 (the entries come back from shared memory).
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int q = lane & 7, rt = (tid & ~31) + 4 * i + (lane >> 3);
    const int jr = blockIdx.x * kBlock + rt;
    if (jr < nq && 4 * q < KV) {
      int4 t;
      t.x = s_v[4 * q][rt];
      t.y = 4 * q + 1 < KV ? s_v[4 * q + 1 < KV ? 4 * q + 1 : 0][rt] : -1;
      t.z = 4 * q + 2 < KV ? s_v[4 * q + 2 < KV ? 4 * q + 2 : 0][rt] : -1;
      t.w = 4 * q + 3 < KV ? s_v[4 * q + 3 < KV ? 4 * q + 3 : 0][rt] : -1;
      reinterpret_cast<int4*>(nbr_rows + size_t(jr) * 32)[q] = t;
    }
  }
  __syncthreads();
  if (threadIdx.x < KV) {
    const unsigned cnt = s_cnt[threadIdx.x];
    blockcnt[size_t(threadIdx.x) * gridDim.x + blockIdx.x] = int32_t(cnt);
    if (offset_cnt != nullptr && cnt != 0u) atomicAdd(&offset_cnt[threadIdx.x], cnt);
  }
  SPCONV_TL(3);
}

// Inverse convolution, any kernel volume: one offset per thread, grid = (ceil(nq/256), kvol); same outputs as
// k_subm_probe (offset-major table and per-block hit counts).
__global__ void k_inverse_probe(const int4* __restrict__ qcoords, int nq, int K, int stride, int dil, const LocSlot* __restrict__ table,
                                uint32_t capmask, int32_t* __restrict__ nbr,
                                int32_t* __restrict__ blockcnt, unsigned* __restrict__ offset_cnt, uint32_t* __restrict__ status,
                                const __grid_constant__ OffsetIndex index) {
  chain_begin();
  const int k = blockIdx.y;
  const int j = blockIdx.x * kBlock + threadIdx.x;
  int ia, ib, ic;
  offset_index(index, k, K, ia, ib, ic);
  const int pad = dil * ((K - 1) / 2);
  int v = -1;
  if (j < nq) {
    const int4 c = qcoords[j];
    if (!(in_range(c.x) && in_range(c.y) && in_range(c.z) && in_range(c.w))) {
      if (k == 0) atomicOr(status, kDevCoordRange);
    } else {
      const int nx = c.y + pad - dil * ia, ny = c.z + pad - dil * ib, nz = c.w + pad - dil * ic;
      if (nx >= 0 && ny >= 0 && nz >= 0 && nx % stride == 0 && ny % stride == 0 && nz % stride == 0) {
        const int x = nx / stride, y = ny / stride, z = nz / stride;
        if (in_range(x) && in_range(y) && in_range(z)) v = table_find(table, capmask, pack_key(c.x, x, y, z));
      }
    }
    nbr[size_t(k) * nq + j] = v;
  }
  const int cnt = __syncthreads_count(v >= 0);
  if (threadIdx.x == 0) {
    blockcnt[size_t(k) * gridDim.x + blockIdx.x] = cnt;
    if (offset_cnt != nullptr && cnt != 0) atomicAdd(&offset_cnt[k], unsigned(cnt));
  }
}

// Rank of every offset by descending count (ties: lower offset first): the bit position of the offset in
// the tile plan's row keys, most frequent offset -> bit 0, rarest -> most significant bit.
__device__ __forceinline__ int offset_rank(int k, int kvol, const long long* counts_or_null, const int64_t* offset_start_or_null,
                                           const unsigned* cnt32_or_null) {
  auto count_of = [&](int j) -> long long {
    if (cnt32_or_null != nullptr) return (long long)cnt32_or_null[j];
    if (offset_start_or_null != nullptr) return (long long)(offset_start_or_null[j + 1] - offset_start_or_null[j]);
    return counts_or_null[j];
  };
  const long long mine = count_of(k);
  int rank = 0;
  for (int j = 0; j < kvol; ++j) {
    const long long other = count_of(j);
    rank += (other > mine || (other == mine && j < k)) ? 1 : 0;
  }
  return rank;
}

// Exclusive scan of M block counts by one thread block of THREADS threads; also publishes
// offset_start[k] = excl[k*nblk], the grand total, and (when asked) the offsets' bit positions.
template <int THREADS>
__device__ void scan_counts_block(const int32_t* __restrict__ cnt, int64_t M, int64_t* __restrict__ excl, int nblk, int kvol,
                                  int64_t* __restrict__ offset_start, int64_t* __restrict__ total_out, int8_t* __restrict__ bitpos) {
  __shared__ int64_t s[THREADS];
  const int tid = threadIdx.x;
  const int64_t chunk = (M + THREADS - 1) / THREADS;
  const int64_t beg = min(int64_t(tid) * chunk, M), end = min(beg + chunk, M);
  // The first kKeep counts of a thread's chunk are read together and kept (a LiDAR-sized map has 9 per thread: one round
  // trip to memory instead of one per count, in each of the two passes).
  constexpr int kKeep = 16;
  int32_t keep[kKeep];
#pragma unroll
  for (int i = 0; i < kKeep; ++i) keep[i] = beg + i < end ? cnt[beg + i] : 0;
  int64_t sum = 0;
#pragma unroll
  for (int i = 0; i < kKeep; ++i) sum += keep[i];
  for (int64_t i = beg + kKeep; i < end; ++i) sum += cnt[i];
  s[tid] = sum;
  __syncthreads();
  for (int off = 1; off < THREADS; off <<= 1) {
    const int64_t t = tid >= off ? s[tid - off] : 0;
    __syncthreads();
    s[tid] += t;
    __syncthreads();
  }
  int64_t run = s[tid] - sum;
#pragma unroll
  for (int i = 0; i < kKeep; ++i) if (beg + i < end) { excl[beg + i] = run; run += keep[i]; }
  for (int64_t i = beg + kKeep; i < end; ++i) { excl[i] = run; run += cnt[i]; }
  __syncthreads();
  if (offset_start != nullptr) {
    for (int k = tid; k < kvol; k += THREADS) offset_start[k] = excl[int64_t(k) * nblk];
    if (tid == 0) offset_start[kvol] = s[THREADS - 1];
  }
  if (tid == 0 && total_out != nullptr) *total_out = s[THREADS - 1];
  if (bitpos != nullptr && offset_start != nullptr && kvol <= 32) {
    __syncthreads();
    if (tid < kvol) bitpos[tid] = int8_t(offset_rank(tid, kvol, nullptr, offset_start, nullptr));
  }
}

__global__ void __launch_bounds__(1024) k_scan_counts(const int32_t* __restrict__ cnt, int64_t M, int64_t* __restrict__ excl, int nblk,
                              int kvol, int64_t* __restrict__ offset_start, int64_t* __restrict__ total_out,
                              int8_t* __restrict__ bitpos) {
  chain_begin();
  SPCONV_TL(10);
  scan_counts_block<1024>(cnt, M, excl, nblk, kvol, offset_start, total_out, bitpos);
}

// Position of a flagged thread among the flagged threads of its block (warp ballot + popc, then the
// warp totals through shared memory).
__device__ __forceinline__ int block_rank(bool flag) {
  __shared__ int wsum[kBlock / 32];
  const unsigned ballot = __ballot_sync(0xffffffffu, flag);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) wsum[warp] = __popc(ballot);
  __syncthreads();
  int base = 0;
  for (int w = 0; w < warp; ++w) base += wsum[w];
  return base + __popc(ballot & ((1u << lane) - 1u));
}

// Per-offset (input, output) pairs from the offset table: stream compaction of nbr[k][:].
// The first list position of block (x, k) is either read from a scan of all blocks' hit counts (excl) or, with
// excl == nullptr, summed by the block itself from the probe kernel's counts: the totals of the offsets before k
// (offset_cnt) plus the hits of the blocks before x within offset k (blockcnt[k][0 .. x)).
__global__ void k_subm_emit(const int32_t* __restrict__ nbr, int n, const int64_t* __restrict__ excl,
                            const int32_t* __restrict__ blockcnt, const unsigned* __restrict__ offset_cnt,
                            int32_t* __restrict__ pair_in, int32_t* __restrict__ pair_out, int64_t capacity) {
  chain_begin();
  SPCONV_TL(8);
  __shared__ long long base_s;
  const int k = blockIdx.y;
  const int j = blockIdx.x * kBlock + threadIdx.x;
  const int v = j < n ? nbr[size_t(k) * n + j] : -1;
  if (excl == nullptr) {
    long long part = 0;
    for (int b = threadIdx.x; b < int(blockIdx.x); b += kBlock) part += blockcnt[size_t(k) * gridDim.x + b];
    if (int(threadIdx.x) < k) part += (long long)offset_cnt[threadIdx.x];
    if (threadIdx.x == 0) base_s = 0;
    __syncthreads();
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) part += __shfl_down_sync(0xffffffffu, part, off);
    if ((threadIdx.x & 31) == 0 && part != 0) atomicAdd(reinterpret_cast<unsigned long long*>(&base_s), (unsigned long long)part);
    __syncthreads();
  }
  const int rank = block_rank(v >= 0);
  if (v >= 0) {
    const int64_t p = (excl != nullptr ? excl[size_t(k) * gridDim.x + blockIdx.x] : int64_t(base_s)) + rank;
    if (p < capacity) {   // the lists may have been sized from an estimate (the host then repeats the emission)
      pair_in[p] = v;
      pair_out[p] = j;
    }
  }
  SPCONV_TL(9);
}

// ---------------------------------------------------------------------------------------------
// Strided / regular convolution.  Candidate (k, i): input i feeds output cell (p_i + pad - d*kvec)/s
// through offset k when every component is >= 0 and divisible by s (for K == s, pad == 0 this is
// o = floor(p/s), kvec = p mod s: Eq. 1-5).  Candidate id cid = k*n + i.
__global__ void k_strided_candidates(const int4* __restrict__ coords, int n, int K, int s, int dil, int pad,
                                     uint64_t* keys2, int32_t* owner_cid, uint32_t capmask2,
                                     int32_t* __restrict__ cand_slot, int32_t* __restrict__ blockcnt, uint32_t* status,
                                     const __grid_constant__ OffsetIndex index) {
  chain_begin();
  const int k = blockIdx.y;
  const int i = blockIdx.x * kBlock + threadIdx.x;
  int slot = -1;
  int ia, ib, ic;
  offset_index(index, k, K, ia, ib, ic);
  const bool pow2 = (s & (s - 1)) == 0;   // strides are 2 in practice: a mask and a shift instead of six divisions
  const int shift = __ffs(s) - 1;
  if (i < n) {
    const int4 c = coords[i];
    const int nx = c.y + pad - dil * ia, ny = c.z + pad - dil * ib, nz = c.w + pad - dil * ic;
    const bool on_grid = pow2 ? (((nx | ny | nz) & (s - 1)) == 0) : (nx % s == 0 && ny % s == 0 && nz % s == 0);
    if (nx >= 0 && ny >= 0 && nz >= 0 && on_grid) {
      const int ox = pow2 ? nx >> shift : nx / s, oy = pow2 ? ny >> shift : ny / s, oz = pow2 ? nz >> shift : nz / s;
      if (in_range(ox) && in_range(oy) && in_range(oz) && in_range(c.x)) {
        bool present;
        slot = table_insert<1>(keys2, capmask2, pack_key(c.x, ox, oy, oz), &present);
        if (slot < 0) atomicOr(status, kDevTableFull);
        else atomicMin(owner_cid + slot, k * n + i);   // the smallest candidate id owns the cell
      } else {
        atomicOr(status, kDevCoordRange);
      }
    }
    cand_slot[size_t(k) * n + i] = slot;
  }
  const int cnt = __syncthreads_count(slot >= 0);
  if (threadIdx.x == 0) blockcnt[size_t(k) * gridDim.x + blockIdx.x] = cnt;
}

__global__ void k_owner_count(const int32_t* __restrict__ cand_slot, const int32_t* __restrict__ owner_cid, int n,
                              int32_t* __restrict__ blockcnt) {
  chain_begin();
  const int k = blockIdx.y;
  const int i = blockIdx.x * kBlock + threadIdx.x;
  bool owner = false;
  if (i < n) {
    const int slot = cand_slot[size_t(k) * n + i];
    owner = slot >= 0 && owner_cid[slot] == k * n + i;
  }
  const int cnt = __syncthreads_count(owner);
  if (threadIdx.x == 0) blockcnt[size_t(k) * gridDim.x + blockIdx.x] = cnt;
}

// Number the output cells in ascending order of their owning candidate id and write their coordinates.
__global__ void k_owner_assign(const int32_t* __restrict__ cand_slot, const int32_t* __restrict__ owner_cid,
                               const uint64_t* __restrict__ keys2, int n, const int64_t* __restrict__ excl,
                               int32_t* __restrict__ slot_out, int4* __restrict__ out_coords) {
  chain_begin();
  const int k = blockIdx.y;
  const int i = blockIdx.x * kBlock + threadIdx.x;
  int slot = -1;
  bool owner = false;
  if (i < n) {
    slot = cand_slot[size_t(k) * n + i];
    owner = slot >= 0 && owner_cid[slot] == k * n + i;
  }
  const int rank = block_rank(owner);
  if (owner) {
    const int64_t o = excl[size_t(k) * gridDim.x + blockIdx.x] + rank;
    slot_out[slot] = int32_t(o);
    const uint64_t key = keys2[slot];
    out_coords[o] = make_int4(int(key >> 48), int((key >> 32) & 0xFFFF), int((key >> 16) & 0xFFFF), int(key & 0xFFFF));
  }
}

// Offset table and pair lists of the strided map (second stage of the paper's two-stage table).
__global__ void k_strided_emit(const int32_t* __restrict__ cand_slot, const int32_t* __restrict__ slot_out, int n,
                               int64_t n_out, const int64_t* __restrict__ excl, int32_t* __restrict__ nbr,
                               int32_t* __restrict__ pair_in, int32_t* __restrict__ pair_out, int32_t* __restrict__ nbr_rows) {
  chain_begin();
  const int k = blockIdx.y;
  const int i = blockIdx.x * kBlock + threadIdx.x;
  const int slot = i < n ? cand_slot[size_t(k) * n + i] : -1;
  const int rank = block_rank(slot >= 0);
  if (slot >= 0) {
    const int o = slot_out[slot];
    nbr[size_t(k) * n_out + o] = i;
    if (nbr_rows != nullptr) nbr_rows[size_t(o) * 32 + k] = i;   // the row-major copy the tile plan reads
    const int64_t p = excl[size_t(k) * gridDim.x + blockIdx.x] + rank;
    pair_in[p] = i;
    pair_out[p] = o;
  }
}

// ---------------------------------------------------------------------------------------------
// Tile plan.  Output rows are grouped into 128-row tiles for the tensor-core kernel.  Rows with the
// same set of non-empty offsets are placed together (sort by the offset bit mask, rarest offset as the
// most significant bit, walked in reflected-Gray order) so that a (tile, offset) block is either mostly
// full or absent and the kernel skips the absent ones.
// Row keys of the tile plan; also marks the unused rows of the last tile (tile_rows beyond n_out) with -1.
__global__ void k_row_keys(const int32_t* __restrict__ nbr, int64_t n_out, int64_t n_padded, int kvol,
                           const int8_t* __restrict__ bitpos, const unsigned* __restrict__ offset_cnt, uint32_t* __restrict__ keys,
                           int32_t* __restrict__ rows, int32_t* __restrict__ tile_rows) {
  __shared__ int8_t pos[32];
  if (threadIdx.x < 32)
    pos[threadIdx.x] = int(threadIdx.x) >= kvol ? int8_t(0) : (offset_cnt != nullptr ? int8_t(offset_rank(int(threadIdx.x), kvol, nullptr, nullptr, offset_cnt)) : bitpos[threadIdx.x]);
  __syncthreads();
  const int64_t o = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (o >= n_out) {
    if (o < n_padded) tile_rows[o] = -1;
    return;
  }
  uint32_t m = 0;
  for (int k = 0; k < kvol; ++k)
    if (nbr[size_t(k) * n_out + o] >= 0) m |= 1u << pos[k];
  // Gray -> binary: consecutive keys differ in one offset where possible.
  m ^= m >> 1; m ^= m >> 2; m ^= m >> 4; m ^= m >> 8; m ^= m >> 16;
  keys[o] = m;
  rows[o] = int32_t(o);
}

// Row keys and their stable LSD radix sort in one cooperative launch, for inputs small enough that every
// block is resident at once (the library sort's multi-kernel pipeline costs several times more than the
// work itself at 10^5 rows).  Block b owns the kSortTile consecutive items b * kSortTile ..; an item is (key, row).
// Per 8-bit pass: every warp ranks its items by digit with match_any (items of a warp are consecutive,
// rounds of 32 in order, so the ranks are stable), the block publishes its digit counts, the grid
// synchronises, every block derives its own global digit offsets from all blocks' counts, scatters, and the
// grid synchronises again before the next pass reads.  The last pass writes the rows to tile_rows; the
// unused rows of the last tile are set to -1.
// Every block sums all blocks' digit counts itself, so the traffic grows with the square of the block count:
// small inputs take 4 items per thread (more blocks, shorter passes), larger ones 8.
constexpr int kSortThreads = 256, kSortItemsSmall = 4, kSortItemsLarge = 8, kSortSmallMaxBlocks = 384;

template <int kSortItems>
__global__ void __launch_bounds__(kSortThreads)
k_sort_rows_coop(const int32_t* __restrict__ nbr, const int32_t* __restrict__ nbr_rows, const uint32_t* __restrict__ row_mask,
                 int64_t n_out, int64_t n_padded, int kvol, const int8_t* __restrict__ bitpos,
                 const unsigned* __restrict__ offset_cnt, int begin_bit, uint32_t* __restrict__ keys_a, int32_t* __restrict__ rows_a,
                 uint32_t* __restrict__ keys_b, int32_t* __restrict__ rows_b, uint32_t* __restrict__ block_hist /* [gridDim.x][256] */,
                 int32_t* __restrict__ tile_rows, const int32_t* __restrict__ scan_cnt, int64_t scan_m, int64_t* __restrict__ scan_excl,
                 int scan_nblk, int64_t* __restrict__ scan_offset_start, int64_t* __restrict__ scan_total) {
  chain_begin();
  SPCONV_TL(4);
  namespace cg = cooperative_groups;
  cg::grid_group grid = cg::this_grid();
  constexpr int kSortTile = kSortThreads * kSortItems;
  __shared__ int8_t pos[32];
  __shared__ uint32_t warp_hist[kSortThreads / 32][256];
  __shared__ uint32_t goff[256], before_s[256], total_s[256];
  __shared__ uint32_t wtot[kSortThreads / 32];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t lt = (1u << lane) - 1u;
  // Bit positions either ready-made (bitpos) or from the per-offset totals.
  if (tid < 32) pos[tid] = tid >= kvol ? int8_t(0) : (offset_cnt != nullptr ? int8_t(offset_rank(tid, kvol, nullptr, nullptr, offset_cnt)) : bitpos[tid]);
  __syncthreads();
  // With scan_cnt set the grid has one block more than the items need; that block scans the pair counts of the
  // probe kernel while the others form their keys (it holds no items, and joins every grid synchronisation).
  if (scan_cnt != nullptr && blockIdx.x == gridDim.x - 1)
    scan_counts_block<kSortThreads>(scan_cnt, scan_m, scan_excl, scan_nblk, kvol, scan_offset_start, scan_total, nullptr);
  // item r of this thread: index blockIdx.x * kSortTile + warp * (32 * kSortItems) + r * 32 + lane
  const int64_t base = int64_t(blockIdx.x) * kSortTile + warp * (32 * kSortItems) + lane;
  uint32_t key[kSortItems];
  int32_t row[kSortItems];
#pragma unroll
  for (int r = 0; r < kSortItems; ++r) {
    const int64_t o = base + r * 32;
    uint32_t m = 0;
    if (o < n_out) {
      // The row's offset set: ready-made (row_mask), from its row of the row-major table, or from the offset-major one.
      uint32_t raw = 0u;
      if (row_mask != nullptr) {
        raw = row_mask[o];
      } else if (nbr_rows != nullptr) {
        const int4* rp = reinterpret_cast<const int4*>(nbr_rows + size_t(o) * 32);
        for (int q = 0; 4 * q < kvol; ++q) {
          const int4 t = __ldcg(rp + q);
          raw |= (t.x >= 0 ? 1u : 0u) << (4 * q) | (t.y >= 0 ? 2u : 0u) << (4 * q) | (t.z >= 0 ? 4u : 0u) << (4 * q) | (t.w >= 0 ? 8u : 0u) << (4 * q);
        }
        raw &= kvol >= 32 ? 0xFFFFFFFFu : ((1u << kvol) - 1u);
      } else {
        for (int k = 0; k < kvol; ++k)
          if (nbr[size_t(k) * n_out + o] >= 0) raw |= 1u << k;
      }
      for (int k = 0; k < kvol; ++k) m |= ((raw >> k) & 1u) << pos[k];
      // Gray -> binary: consecutive keys differ in one offset where possible.
      m ^= m >> 1; m ^= m >> 2; m ^= m >> 4; m ^= m >> 8; m ^= m >> 16;
    } else if (o < n_padded) {
      tile_rows[o] = -1;
    }
    key[r] = m;
    row[r] = o < n_out ? int32_t(o) : -1;
  }
  const int n_bits = kvol - begin_bit;
  const int passes = (n_bits + 7) / 8;
  for (int p = 0; p < passes; ++p) {
    const int shift = begin_bit + 8 * p;
    const uint32_t dmask = (n_bits - 8 * p >= 8) ? 0xFFu : ((1u << (n_bits - 8 * p)) - 1u);
    for (int i = tid; i < (kSortThreads / 32) * 256; i += kSortThreads) (&warp_hist[0][0])[i] = 0u;
    __syncthreads();
    uint32_t local[kSortItems];   // rank of the item among its warp's items with the same digit
#pragma unroll
    for (int r = 0; r < kSortItems; ++r) {
      const bool valid = row[r] >= 0;
      const uint32_t dg = (key[r] >> shift) & dmask;
      const uint32_t peers = __match_any_sync(0xffffffffu, valid ? dg : (0x100u + uint32_t(lane)));
      uint32_t prior = 0;
      if (valid) prior = warp_hist[warp][dg];
      __syncwarp();
      if (valid && (peers & lt) == 0u) warp_hist[warp][dg] = prior + __popc(peers);
      __syncwarp();
      local[r] = prior + __popc(peers & lt);
    }
    __syncthreads();
    {  // digit tid: counts of the block's warps -> exclusive over warps; publish the block's count
      uint32_t run = 0;
#pragma unroll
      for (int w = 0; w < kSortThreads / 32; ++w) { const uint32_t c = warp_hist[w][tid]; warp_hist[w][tid] = run; run += c; }
      block_hist[size_t(blockIdx.x) * 256 + tid] = run;
    }
    grid.sync();
    {  // per digit: items of earlier blocks with this digit, and of all blocks.  Warp w sums the blocks b = w (mod 8);
       // a lane takes eight consecutive digits of a block's counts as two vector loads, and the loads of several
       // blocks are in flight together.
      before_s[tid] = 0u; total_s[tid] = 0u;
      __syncthreads();
      uint32_t bef[8], tot[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) { bef[j] = 0u; tot[j] = 0u; }
      // (small grids: one round trip for up to 96 blocks; the instantiation for large grids keeps fewer loads in
      // flight so that more of its blocks fit an SM, which is what bounds the rows a cooperative launch can take)
      constexpr int kBatch = kSortItems <= kSortItemsSmall ? 12 : 4;
      for (unsigned b0 = warp; b0 < gridDim.x; b0 += kBatch * (kSortThreads / 32)) {
        uint4 c[kBatch][2];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {   // (volatile: the loads are issued back to back, ahead of the sums)
          const unsigned b = b0 + u * (kSortThreads / 32);
          const uint4* src = reinterpret_cast<const uint4*>(block_hist + size_t(b < gridDim.x ? b : b0) * 256 + lane * 8);
          asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(c[u][0].x), "=r"(c[u][0].y), "=r"(c[u][0].z), "=r"(c[u][0].w) : "l"(src));
          asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(c[u][1].x), "=r"(c[u][1].y), "=r"(c[u][1].z), "=r"(c[u][1].w) : "l"(src + 1));
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const unsigned b = b0 + u * (kSortThreads / 32);
          if (b >= gridDim.x) continue;
          const bool earlier = b < blockIdx.x;
          const uint32_t vals8[8] = {c[u][0].x, c[u][0].y, c[u][0].z, c[u][0].w, c[u][1].x, c[u][1].y, c[u][1].z, c[u][1].w};
#pragma unroll
          for (int j = 0; j < 8; ++j) { tot[j] += vals8[j]; if (earlier) bef[j] += vals8[j]; }
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) { atomicAdd(&before_s[lane * 8 + j], bef[j]); atomicAdd(&total_s[lane * 8 + j], tot[j]); }
      __syncthreads();
      const uint32_t before = before_s[tid], total = total_s[tid];
      // digit tid: exclusive prefix of the totals over all smaller digits
      uint32_t incl = total;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, incl, off); if (lane >= off) incl += t; }
      if (lane == 31) wtot[warp] = incl;
      __syncthreads();
      uint32_t wbase = 0;
      for (int w = 0; w < warp; ++w) wbase += wtot[w];
      goff[tid] = wbase + incl - total + before;
    }
    __syncthreads();
    const bool last = p == passes - 1;
    uint32_t* kout = (p & 1) ? keys_a : keys_b;
    int32_t* rout = last ? tile_rows : ((p & 1) ? rows_a : rows_b);
#pragma unroll
    for (int r = 0; r < kSortItems; ++r) {
      if (row[r] < 0) continue;
      const uint32_t dg = (key[r] >> shift) & dmask;
      const uint32_t at = goff[dg] + warp_hist[warp][dg] + local[r];
      if (!last) kout[at] = key[r];
      rout[at] = row[r];
    }
    if (last) { SPCONV_TL(5); break; }
    grid.sync();
#pragma unroll
    for (int r = 0; r < kSortItems; ++r) {
      const int64_t o = base + r * 32;
      key[r] = o < n_out ? kout[o] : 0u;
      row[r] = o < n_out ? rout[o] : -1;
    }
    __syncthreads();   // warp_hist and goff are rewritten by the next pass
  }
}



__global__ void k_iota_rows(int32_t* rows, int64_t n_out, int64_t n_padded) {
  const int64_t o = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (o < n_padded) rows[o] = o < n_out ? int32_t(o) : -1;
}

// One block: copies the totals block into the host's pinned buffer and raises the flag behind it (the same
// report the tile plan's last block makes), for the point of a strided build where the host has to learn the
// number of output rows before it can size the map.
__global__ void k_report_totals(const int64_t* __restrict__ totals, int totals_words, int64_t* __restrict__ host_totals) {
  chain_begin();
  for (int i = threadIdx.x; i < totals_words; i += blockDim.x) host_totals[i] = __ldcg(totals + i);
  __threadfence_system();
  __syncthreads();
  if (threadIdx.x == 0) {
    *reinterpret_cast<volatile int64_t*>(host_totals + totals_words) = 1;
    __threadfence_system();
  }
}

// One block per tile: the tile's slice of the offset table, block by block.  For block (tile, k) the input rows
// that exist are listed first (tile_nbr, compacted, with the tile row each one feeds in tile_crow), so that the
// forward kernel copies only rows that exist; tile_absent marks the tile rows without an input (their
// accumulator lanes are left untouched by the MMA), tile_mask the offsets that have any row at all.
__device__ void schedule_tiles_block(const uint32_t* __restrict__ tile_mask, int n_tiles, int mask_words, int kvol,
                                     int32_t* __restrict__ sorted_tiles, uint32_t* __restrict__ status_words);

// The same schedule (tiles in descending order of their block count) when every tile has already taken its place
// among the tiles of its count (tile_within, from an atomic counter per count: class_cnt, at most 31 blocks per tile):
// the last block only turns the 32 counts into list positions and writes each record where it belongs.  Tiles of equal
// count come in the order their blocks finished; the forward's result does not depend on the schedule.
__device__ __forceinline__ void schedule_from_ranks(const uint32_t* __restrict__ tile_mask, const int32_t* __restrict__ tile_within,
                                                    const unsigned* __restrict__ class_cnt, int n_tiles,
                                                    int32_t* __restrict__ sorted_tiles, uint32_t* __restrict__ status_words) {
  __shared__ int s_base[32];
  const int tid = int(threadIdx.x), T = int(blockDim.x);
  if (tid < 16) status_words[tid] = 0u;   // the forward kernels' status record starts clean
  constexpr int kKeep = 8;
  uint32_t m[kKeep];
  int32_t w[kKeep];
#pragma unroll
  for (int i = 0; i < kKeep; ++i) {   // all reads in flight together, beside the counts'
    const int t = tid + i * T;
    m[i] = t < n_tiles ? __ldcg(tile_mask + t) : 0u;
    w[i] = t < n_tiles ? __ldcg(tile_within + t) : 0;
  }
  if (tid < 32) {
    const int c = int(__ldcg(class_cnt + tid));
    int incl = c;   // sum of the counts of this class and all heavier ones
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) { const int u = __shfl_down_sync(0xffffffffu, incl, off); if (tid + off < 32) incl += u; }
    s_base[tid] = incl - c;
  }
  __syncthreads();
  auto place = [&](int t, uint32_t mask, int32_t within) {
    int32_t* rec = sorted_tiles + size_t(s_base[__popc(mask)] + within) * 2;
    rec[0] = t;
    rec[1] = int32_t(mask);
  };
#pragma unroll
  for (int i = 0; i < kKeep; ++i) if (tid + i * T < n_tiles) place(tid + i * T, m[i], w[i]);
  for (int t = tid + kKeep * T; t < n_tiles; t += T) place(t, __ldcg(tile_mask + t), __ldcg(tile_within + t));
}

// SMALL (kvol <= 32): the thread's 27-odd table entries are fetched up front, so the block pays one memory
// latency instead of one per offset.
template <bool SMALL>
__global__ void k_tile_plan(const int32_t* __restrict__ tile_rows, const int32_t* __restrict__ nbr, int64_t n_out,
                            int kvol, int mask_words, int32_t* __restrict__ tile_nbr, uint8_t* __restrict__ tile_crow,
                            uint32_t* __restrict__ tile_mask, uint32_t* __restrict__ tile_absent,
                            unsigned long long* __restrict__ block_counter, unsigned* __restrict__ tiles_done,
                            int32_t* __restrict__ sorted_tiles, uint32_t* __restrict__ status_words,
                            const int64_t* __restrict__ totals, int totals_words, int64_t* __restrict__ host_totals) {
  chain_begin();
  __shared__ int wcnt[2][kTileRows / 32];
  __shared__ bool last_block;
  const int t = blockIdx.x, r = threadIdx.x, warp = r >> 5, lane = r & 31;
  const int row = tile_rows[size_t(t) * kTileRows + r];
  int pre[SMALL ? 32 : 1];
  if (SMALL) {
#pragma unroll
    for (int k = 0; k < 32; ++k) pre[SMALL ? k : 0] = (row >= 0 && k < kvol) ? nbr[size_t(k) * n_out + row] : -1;
  }
  uint32_t word = 0;
  int nblocks = 0;
  auto one_offset = [&](int k, int v) {
    const unsigned present = __ballot_sync(0xffffffffu, v >= 0);
    if (lane == 0) {
      tile_absent[(size_t(t) * kvol + k) * 4 + warp] = ~present;     // rows of this warp's 32 without an input
      wcnt[k & 1][warp] = __popc(present);
    }
    const int any = __syncthreads_or(v >= 0);
    int base = 0, total = 0;
#pragma unroll
    for (int w = 0; w < kTileRows / 32; ++w) { const int c = wcnt[k & 1][w]; if (w < warp) base += c; total += c; }
    const size_t blk = (size_t(t) * kvol + k) * kTileRows;
    if (v >= 0) {
      const int rank = base + __popc(present & ((1u << lane) - 1u));
      tile_nbr[blk + rank] = v;
      tile_crow[blk + rank] = uint8_t(r);
    }
    if (r >= total) { tile_nbr[blk + r] = -1; tile_crow[blk + r] = 0; }
    if (any) { word |= 1u << (k & 31); ++nblocks; }
    if ((k & 31) == 31 || k == kvol - 1) {
      if (r == 0) tile_mask[size_t(t) * mask_words + (k >> 5)] = word;
      word = 0;
    }
  };
  if (SMALL) {
    // All offsets at once: one ballot per offset, the warps' counts exchanged through shared memory with a single
    // block barrier, then every thread places its own entries.
    __shared__ uint8_t cnt_all[32][kTileRows / 32];
    uint32_t present[32];
#pragma unroll
    for (int k = 0; k < 32; ++k) {
      present[k] = __ballot_sync(0xffffffffu, pre[SMALL ? k : 0] >= 0);
      if (lane == k) cnt_all[k][warp] = uint8_t(__popc(present[k]));   // lane k publishes offset k's count of this warp
    }
    __syncthreads();
    const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
    for (int k = 0; k < 32; ++k) {
      if (k >= kvol) break;
      int base = 0, total = 0;
#pragma unroll
      for (int w = 0; w < kTileRows / 32; ++w) { const int c = cnt_all[k][w]; if (w < warp) base += c; total += c; }
      const int v = pre[SMALL ? k : 0];
      const size_t blk = (size_t(t) * kvol + k) * kTileRows;
      if (lane == 0) tile_absent[(size_t(t) * kvol + k) * 4 + warp] = ~present[k];   // rows of this warp's 32 without an input
      if (v >= 0) {
        const int rank = base + __popc(present[k] & lt);
        tile_nbr[blk + rank] = v;
        tile_crow[blk + rank] = uint8_t(r);
      }
      if (r >= total) { tile_nbr[blk + r] = -1; tile_crow[blk + r] = 0; }
      if (total > 0) { word |= 1u << (k & 31); ++nblocks; }
    }
    if (r == 0) tile_mask[size_t(t) * mask_words] = word;
  } else {
    for (int k = 0; k < kvol; ++k) one_offset(k, row >= 0 ? nbr[size_t(k) * n_out + row] : -1);
  }
  if (r == 0) atomicAdd(block_counter, (unsigned long long)nblocks);
  // The block that finishes last orders the tiles for the forward's schedule (all masks are written by then).
  __threadfence();
  __syncthreads();
  if (r == 0) last_block = atomicAdd(tiles_done, 1u) == gridDim.x - 1;
  __syncthreads();
  if (last_block) {
    __threadfence();
    schedule_tiles_block(tile_mask, int(gridDim.x), mask_words, kvol, sorted_tiles, status_words);
    // Everything the host waits for (error word, pair count, offset starts, block count) is final by now: the
    // last block writes it straight into the host's pinned buffer and raises the flag behind it, which spares
    // the build a copy and a stream synchronisation.
    if (host_totals != nullptr) {
      for (int i = threadIdx.x; i < totals_words; i += blockDim.x) host_totals[i] = __ldcg(totals + i);
      __threadfence_system();
      __syncthreads();
      if (threadIdx.x == 0) {
        *reinterpret_cast<volatile int64_t*>(host_totals + totals_words) = 1;
        __threadfence_system();
      }
    }
  }
}


// The same plan from the row-major table (kernel volumes up to 32): thread (warp w, lane k) takes offset k of the
// tile rows 32w .. 32w + 31.  A row of the table is one 128-byte line, so the 32 loads of a thread are 32
// coalesced warp loads, all in flight together, where the offset-major table costs a 32-byte sector per entry.
// The compacted lists are put together in shared memory and leave as whole lines.
constexpr int kPlanNbrPitch = kTileRows + 4;    // ints per offset in shared memory (16-byte aligned rows, banks skewed by 4)
constexpr int kPlanCrowPitch = kTileRows + 16;  // bytes per offset
__global__ void __launch_bounds__(kTileRows)
k_tile_plan_rows(const int32_t* __restrict__ tile_rows, const int32_t* __restrict__ nbr_rows, int kvol,
                 int32_t* __restrict__ tile_nbr, uint8_t* __restrict__ tile_crow, uint32_t* __restrict__ tile_mask,
                 uint32_t* __restrict__ tile_absent, unsigned long long* __restrict__ block_counter,
                 unsigned* __restrict__ tiles_done, int32_t* __restrict__ sorted_tiles, uint32_t* __restrict__ status_words,
                 const int64_t* __restrict__ totals, int totals_words, int64_t* __restrict__ host_totals, int report_from_counts,
                 unsigned* __restrict__ class_cnt, int32_t* __restrict__ tile_within) {
  chain_begin();
  SPCONV_TL(6);
  __shared__ __align__(16) int32_t s_nbr[32][kPlanNbrPitch];
  __shared__ __align__(16) uint8_t s_crow[32][kPlanCrowPitch];
  __shared__ int s_cnt[32][kTileRows / 32];
  __shared__ bool last_block;
  const int t = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int my_row = tile_rows[size_t(t) * kTileRows + tid];
  int v[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    const int row = __shfl_sync(0xffffffffu, my_row, i);
    v[i] = (row >= 0 && lane < kvol) ? __ldcg(nbr_rows + size_t(row) * 32 + lane) : -1;
  }
  uint32_t pm = 0u;
#pragma unroll
  for (int i = 0; i < 32; ++i) pm |= (v[i] >= 0 ? 1u : 0u) << i;
  s_cnt[lane][warp] = __popc(pm);
  if (lane < kvol) tile_absent[(size_t(t) * kvol + lane) * 4 + warp] = ~pm;   // rows of this warp's 32 without an input
  __syncthreads();
  int base = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kTileRows / 32; ++w) { const int c = s_cnt[lane][w]; if (w < warp) base += c; total += c; }
  {  // this thread's entries of offset `lane`, in row order, behind those of the warps before it
    int at = base;
#pragma unroll
    for (int i = 0; i < 32; ++i)
      if ((pm >> i) & 1u) { s_nbr[lane][at] = v[i]; s_crow[lane][at] = uint8_t(32 * warp + i); ++at; }
  }
  // entries past an offset's count: no row
  for (int k = 0; k < kvol; ++k) {
    int tk = 0;
#pragma unroll
    for (int w = 0; w < kTileRows / 32; ++w) tk += s_cnt[k][w];
    if (tid >= tk) { s_nbr[k][tid] = -1; s_crow[k][tid] = 0; }
  }
  const unsigned word = __ballot_sync(0xffffffffu, lane < kvol && total > 0);
  __syncthreads();
  {
    int4* dst = reinterpret_cast<int4*>(tile_nbr + size_t(t) * kvol * kTileRows);
    for (int i = tid; i < kvol * (kTileRows / 4); i += kTileRows) {
      const int k = i / (kTileRows / 4), q = i % (kTileRows / 4);
      dst[i] = *reinterpret_cast<const int4*>(&s_nbr[k][4 * q]);
    }
    int4* dstc = reinterpret_cast<int4*>(tile_crow + size_t(t) * kvol * kTileRows);
    for (int i = tid; i < kvol * (kTileRows / 16); i += kTileRows) {
      const int k = i / (kTileRows / 16), q = i % (kTileRows / 16);
      dstc[i] = *reinterpret_cast<const int4*>(&s_crow[k][16 * q]);
    }
  }
  if (tid == 0) {
    tile_mask[t] = word;
    atomicAdd(block_counter, (unsigned long long)__popc(word));
    // the tile's place among the tiles with the same number of blocks: all the last block needs to order the tiles
    if (class_cnt != nullptr) tile_within[t] = int32_t(atomicAdd(&class_cnt[__popc(word)], 1u));
  }
  // The block that finishes last orders the tiles for the forward's schedule and reports to the host (see k_tile_plan).
  __threadfence();
  __syncthreads();
  if (tid == 0) last_block = atomicAdd(tiles_done, 1u) == gridDim.x - 1;
  __syncthreads();
  if (last_block) {
    __threadfence();
    if (class_cnt != nullptr) schedule_from_ranks(tile_mask, tile_within, class_cnt, int(gridDim.x), sorted_tiles, status_words);
    else schedule_tiles_block(tile_mask, int(gridDim.x), 1, kvol, sorted_tiles, status_words);
    if (host_totals != nullptr) {
#ifdef SPCONV_KMAP_TIMELINE
      if (threadIdx.x == 0) { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); SPCONV_TL_RAW(7, t); }
#endif
      if (report_from_counts) {
        // Pair count and offset starts straight from the probe's per-offset totals (the words behind the totals block;
        // kvol <= 32): lane k reads offset k's total, a warp scan gives the starts, and every word of the report is
        // written once, all reads and all writes in flight together (one thread walking the offsets paid a round trip
        // to L2 per offset: 9 us).
        if (threadIdx.x < 32) {
          const int k = int(threadIdx.x);
          const unsigned* cnt = reinterpret_cast<const unsigned*>(totals + totals_words);
          const int64_t mine = k < kvol ? int64_t(__ldcg(cnt + k)) : 0;
          const int64_t head = k < 8 ? __ldcg(totals + k) : 0;
          int64_t incl = mine;
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) { const int64_t u = __shfl_up_sync(0xffffffffu, incl, off); if (k >= off) incl += u; }
          const int64_t total = __shfl_sync(0xffffffffu, incl, 31);
          if (k < 8) host_totals[k] = k == 1 ? total : head;
          if (k < kvol) host_totals[8 + k] = incl - mine;
          if (k == 0) host_totals[8 + kvol] = total;
        }
      } else {
        for (int i = threadIdx.x; i < totals_words; i += blockDim.x) host_totals[i] = __ldcg(totals + i);
      }
      __threadfence_system();
      __syncthreads();
      // (no fence behind the flag: nothing follows it, and a fence here only kept the kernel, and with it the forward
      // that waits for this kernel, 1.8 us longer)
      if (threadIdx.x == 0) *reinterpret_cast<volatile int64_t*>(host_totals + totals_words) = 1;
    }
  }
}

// Schedule of the tensor-core forward: tiles in descending order of their block count, tiles of equal count in
// ascending tile order (a stable counting sort by one thread block), so that dealing them out serpentine over the
// CTAs gives every CTA nearly the same number of blocks.  Used where the tiles have not taken their places within
// their count class while the plan's blocks ran (see schedule_from_ranks); the forward's result does not depend on the
// schedule.  Thread i owns the contiguous chunk of tiles [i * chunk, (i + 1) * chunk).  Kernel volumes beyond 31 offsets
// (more count classes than the per-thread counters hold) fall back to an unordered placement within a class.
__device__ void schedule_tiles_block(const uint32_t* __restrict__ tile_mask, int n_tiles, int mask_words, int kvol,
                                     int32_t* __restrict__ sorted_tiles, uint32_t* __restrict__ status_words) {
  if (threadIdx.x < 16) status_words[threadIdx.x] = 0u;   // the forward kernels' status record starts clean
  if (mask_words == 1 && kvol <= 31 && blockDim.x <= 128 && n_tiles <= 60000) {
    constexpr int kClasses = 32, kMaxThreads = 128, kKeep = 8;
    __shared__ uint16_t cnt[kClasses][kMaxThreads];   // tiles of class c in thread i's chunk, then their exclusive prefix over threads
    __shared__ int class_base[kClasses];
    const int T = int(blockDim.x), tid = int(threadIdx.x), lane = tid & 31, warp = tid >> 5;
    const int chunk = (n_tiles + T - 1) / T;
    const int beg = min(tid * chunk, n_tiles), end = min(beg + chunk, n_tiles);
    for (int c = 0; c < kClasses; ++c) cnt[c][tid] = 0;
    uint32_t mine[kKeep];
#pragma unroll
    for (int i = 0; i < kKeep; ++i) mine[i] = beg + i < end ? __ldcg(tile_mask + beg + i) : 0u;   // all reads in flight together
#pragma unroll
    for (int i = 0; i < kKeep; ++i) if (beg + i < end) cnt[__popc(mine[i])][tid] += 1;
    for (int t = beg + kKeep; t < end; ++t) cnt[__popc(__ldcg(tile_mask + t))][tid] += 1;
    __syncthreads();
    // per class: exclusive prefix over the threads (warp w takes the classes w, w + nwarps, ...) and the class total
    const int nwarps = (T + 31) / 32;
    for (int c = warp; c < kClasses; c += nwarps) {
      int run = 0;
      for (int i0 = 0; i0 < T; i0 += 32) {
        const int i = i0 + lane;
        const int v = i < T ? int(cnt[c][i]) : 0;
        int incl = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) { const int u = __shfl_up_sync(0xffffffffu, incl, off); if (lane >= off) incl += u; }
        if (i < T) cnt[c][i] = uint16_t(run + incl - v);
        run += __shfl_sync(0xffffffffu, incl, 31);
      }
      if (lane == 0) class_base[c] = run;   // the total for now
    }
    __syncthreads();
    if (tid == 0) {   // classes in descending order of their count value
      int run = 0;
      for (int c = kClasses - 1; c >= 0; --c) { const int total = class_base[c]; class_base[c] = run; run += total; }
    }
    __syncthreads();
    int placed[kClasses];
#pragma unroll
    for (int c = 0; c < kClasses; ++c) placed[c] = 0;
    auto place = [&](int t, uint32_t m) {
      const int c = __popc(m);
      int mine_before = 0;
#pragma unroll
      for (int q = 0; q < kClasses; ++q) if (q == c) { mine_before = placed[q]; placed[q] += 1; }
      int32_t* rec = sorted_tiles + size_t(class_base[c] + int(cnt[c][tid]) + mine_before) * 2;
      rec[0] = t;
      rec[1] = int32_t(m);
    };
#pragma unroll
    for (int i = 0; i < kKeep; ++i) if (beg + i < end) place(beg + i, mine[i]);
    for (int t = beg + kKeep; t < end; ++t) place(t, __ldcg(tile_mask + t));
    return;
  }
  __shared__ int hist[kMaskWordsMax * 32 + 2];
  __shared__ int base[kMaskWordsMax * 32 + 2];
  for (int i = threadIdx.x; i <= kvol; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  for (int t = threadIdx.x; t < n_tiles; t += blockDim.x) {
    int c = 0;
    for (int w = 0; w < mask_words; ++w) c += __popc(__ldcg(tile_mask + size_t(t) * mask_words + w));
    atomicAdd(&hist[c], 1);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    for (int c = kvol; c >= 0; --c) { base[c] = run; run += hist[c]; }
  }
  __syncthreads();
  // A schedule record is the tile followed by its offset mask, so that the forward kernel gets both with one
  // round trip to memory.
  for (int t = threadIdx.x; t < n_tiles; t += blockDim.x) {
    int c = 0;
    uint32_t words[kMaskWordsMax];
    for (int w = 0; w < mask_words; ++w) { words[w] = __ldcg(tile_mask + size_t(t) * mask_words + w); c += __popc(words[w]); }
    int32_t* rec = sorted_tiles + size_t(atomicAdd(&base[c], 1)) * (1 + mask_words);
    rec[0] = t;
    for (int w = 0; w < mask_words; ++w) rec[1 + w] = int32_t(words[w]);
  }
}

// ---------------------------------------------------------------------------------------------
struct Arena {
  char* base = nullptr;
  size_t size = 0, used = 0;
  template <class T> T* take(size_t count) {
    used = (used + 255) & ~size_t(255);
    T* p = reinterpret_cast<T*>(base + used);
    used += count * sizeof(T);
    return p;
  }
};
inline size_t pad256(size_t bytes) { return (bytes + 255) & ~size_t(255); }

// A second stream and two events per host thread and device, created on first use and kept (never destroyed:
// at thread or process exit the CUDA context may already be gone).
struct SideStream { cudaStream_t s = nullptr; cudaEvent_t fork = nullptr, join = nullptr; };
SideStream* side_stream_for(int device) {
  thread_local SideStream sets[64];
  if (device < 0 || device >= 64) return nullptr;
  SideStream& side = sets[device];
  if (side.s == nullptr) {
    cudaStream_t s = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    if (cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) != cudaSuccess || cudaEventCreateWithFlags(&a, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&b, cudaEventDisableTiming) != cudaSuccess) {
      (void)cudaGetLastError();
      return nullptr;   // the build then emits on the caller's stream
    }
    side.s = s; side.fork = a; side.join = b;
  }
  return &side;
}

__global__ void __launch_bounds__(256) k_fill_regions(const __grid_constant__ FillRegions regions) {
  chain_begin();
  const size_t stride = size_t(gridDim.x) * blockDim.x, first = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const uint4 v = make_uint4(regions.value[r], regions.value[r], regions.value[r], regions.value[r]);
    for (size_t i = first; i < regions.count16[r]; i += stride) regions.ptr[r][i] = v;
  }
}

uint32_t pow2_at_least(uint64_t v) {
  uint64_t c = 64;
  while (c < v) c <<= 1;
  return uint32_t(c);
}

struct Scratch {
  void* ptr = nullptr;
  cudaStream_t stream = nullptr;
  ~Scratch() { if (ptr) cudaFreeAsync(ptr, stream); }
};

// Small pinned buffers for the size read-back, recycled between builds (allocating pinned memory costs
// far more than a whole build).
struct PinnedPool {
  std::mutex mu;
  std::vector<std::pair<int64_t*, size_t>> free_list;
  int64_t* get(size_t count) {
    {
      std::lock_guard<std::mutex> lock(mu);
      for (size_t i = 0; i < free_list.size(); ++i)
        if (free_list[i].second >= count) {
          int64_t* p = free_list[i].first;
          free_list.erase(free_list.begin() + i);
          return p;
        }
    }
    int64_t* p = nullptr;
    if (cudaMallocHost(&p, std::max<size_t>(count, 160) * sizeof(int64_t)) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    return p;
  }
  void put(int64_t* p, size_t count) {
    std::lock_guard<std::mutex> lock(mu);
    free_list.emplace_back(p, std::max<size_t>(count, 160));
  }
};
PinnedPool g_pinned;
struct PinnedHost {
  int64_t* p = nullptr;
  size_t count = 0;
  cudaStream_t writer = nullptr;
  bool write_pending = false;   // a kernel on `writer` may still store into the buffer
  ~PinnedHost() {
    if (!p) return;
    if (write_pending) { (void)cudaStreamSynchronize(writer); (void)cudaGetLastError(); }
    g_pinned.put(p, count);
  }
};

// Keep freed stream-ordered allocations cached in the device's default memory pool instead of returning
// them to the driver at every synchronisation (a build allocates and frees scratch on each call).
void keep_pool_cached(int device) {
  static std::mutex mu;
  static bool done[64] = {false};
  std::lock_guard<std::mutex> lock(mu);
  if (device < 0 || device >= 64 || done[device]) return;
  cudaMemPool_t pool;
  if (cudaDeviceGetDefaultMemPool(&pool, device) == cudaSuccess) {
    uint64_t threshold = ~uint64_t(0);
    cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &threshold);
  }
  (void)cudaGetLastError();
  done[device] = true;
}

int device_status_to_error(uint32_t st) {
  if (st & kDevCoordRange) return SPCONV_ERR_COORD_RANGE;
  if (st & kDevDuplicate) return SPCONV_ERR_DUPLICATE_COORD;
  if (st & kDevTableFull) return SPCONV_ERR_TABLE_FULL;
  return SPCONV_OK;
}

// Number of blocks of the cooperative sort kernel that fit the device at once, for the instantiation with few items
// per thread (large = false) and the one with many (0 if cooperative launches are not supported).  An environment
// switch forces the library sort for testing.
int coop_sort_capacity(int device, bool large) {
  static int cap[64][2];
  static bool known[64] = {false};
  static std::mutex mu;
  if (device < 0 || device >= 64) return 0;
  std::lock_guard<std::mutex> lock(mu);
  if (!known[device]) {
    int coop = 0, sms = 0, per_small = 0, per_large = 0;
    const char* off = std::getenv("SPCONV_KMAP_LIBRARY_SORT");
    if (!(off != nullptr && off[0] == '1') &&
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, device) == cudaSuccess && coop != 0 &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) == cudaSuccess &&
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_small, k_sort_rows_coop<kSortItemsSmall>, kSortThreads, 0) == cudaSuccess &&
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_large, k_sort_rows_coop<kSortItemsLarge>, kSortThreads, 0) == cudaSuccess) {
      cap[device][0] = sms * per_small;
      cap[device][1] = sms * per_large;
    } else {
      cap[device][0] = cap[device][1] = 0;
    }
    (void)cudaGetLastError();
    known[device] = true;
  }
  return cap[device][large ? 1 : 0];
}


// Largest number of offsets along one axis through which a single input position can reach an output cell.
int max_candidates_per_axis(int K, int s, int d) {
  int best = 0;
  for (int res = 0; res < s; ++res) {
    int c = 0;
    for (int k = 0; k < K; ++k) if (((res - d * k) % s + s) % s == 0) ++c;
    best = std::max(best, c);
  }
  return best;
}

std::atomic<long long> g_test_table_slots{0};

}  // namespace

void set_kmap_test_table_slots(long long slots) { g_test_table_slots.store(slots > 0 ? slots : 0, std::memory_order_relaxed); }

void destroy_kmap_impl(spconv_kmap* km) {
  if (!km) return;
  // Two stream-ordered device allocations hold every array of the handle (see build_kmap_impl); they go
  // back to the pool in the order of the stream the map was built on.
  if (km->d.out_coords) cudaFreeAsync(km->d.out_coords, km->stream);
  if (km->d.pair_in) cudaFreeAsync(km->d.pair_in, km->stream);
  (void)cudaGetLastError();
  delete km;
}

#ifdef SPCONV_KMAP_TIMING
// Development builds: CUDA events after each stage of the build, printed when the build returns.
struct StageTimer {
  cudaStream_t stream; cudaEvent_t ev[32]; const char* name[32]; int n = 0;
  explicit StageTimer(cudaStream_t s) : stream(s) {}
  void mark(const char* what) { if (n < 32) { cudaEventCreate(&ev[n]); cudaEventRecord(ev[n], stream); name[n] = what; ++n; } }
  ~StageTimer() {
    cudaStreamSynchronize(stream);
    for (int i = 1; i < n; ++i) { float ms = 0; cudaEventElapsedTime(&ms, ev[i - 1], ev[i]); std::fprintf(stderr, "  kmap stage %-14s %7.1f us\n", name[i], ms * 1e3f); }
    for (int i = 0; i < n; ++i) cudaEventDestroy(ev[i]);
  }
};
#define SPCONV_STAGE(t, what) (t).mark(what)
#else
struct StageTimer { explicit StageTimer(cudaStream_t) {} };
#define SPCONV_STAGE(t, what)
#endif
#ifdef SPCONV_KMAP_TIMELINE
struct TimelineDump {
  cudaStream_t stream;
  std::chrono::steady_clock::time_point h0 = std::chrono::steady_clock::now();
  double hs[16]; const char* hn[16]; int nh = 0;
  void host(const char* what) { if (nh < 16) { hs[nh] = std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - h0).count(); hn[nh++] = what; } }
  ~TimelineDump() {
    for (int i = 0; i < nh; ++i) std::fprintf(stderr, "  host %-16s %8.2f us\n", hn[i], hs[i]);
    cudaDeviceSynchronize();
    unsigned long long t[32];
    if (cudaMemcpyFromSymbol(t, g_kmap_timeline, sizeof(t)) != cudaSuccess) return;
    const char* names[] = {"insert start", "insert end(b0)", "probe start", "probe end(b0)", "sort start", "sort end(b0)", "plan start", "plan report", "emit start", "emit end(b0)", "scan start"};
    for (int i = 0; i < 11; ++i) std::fprintf(stderr, "  tl %-16s %8.2f us\n", names[i], (double(t[i]) - double(t[0])) * 1e-3);
  }
};
#endif

int build_kmap_impl(const int32_t* coords, int64_t n, int stride, int dilation, int kernel, int submanifold,
                    cudaStream_t stream, spconv_kmap** out, const std::function<int(spconv_kmap*)>* before_wait,
                    const int32_t* fine_coords, int64_t n_fine, const int* dense_grid, int rows_as_given) {
  [[maybe_unused]] StageTimer stages(stream);
#ifdef SPCONV_KMAP_TIMELINE
  TimelineDump timeline_dump{stream};
#define SPCONV_HOST_TL(what) timeline_dump.host(what)
#else
#define SPCONV_HOST_TL(what)
#endif
  SPCONV_STAGE(stages, "start");
  const int K = kernel, s = stride, d = dilation;
  const int kvol = K * K * K;
  spconv_kmap* km = new (std::nothrow) spconv_kmap;
  if (!km) return SPCONV_ERR_ALLOC;
  struct Guard { spconv_kmap* km; ~Guard() { if (km) destroy_kmap_impl(km); } } guard{km};
  km->kernel = K; km->stride = s; km->dilation = d; km->submanifold = submanifold; km->kvol = kvol;
  // Inverse convolution (fine_coords given): the location table is built over `coords` (the coarse positions, the
  // rows of the input features) and probed from the fine positions, which are the output rows.  Like a submanifold
  // map its output rows are known up front, so both take the same path below with nq query rows.
  const bool inverse = fine_coords != nullptr;
  const bool known_outputs = submanifold || inverse;
  const int64_t nq = inverse ? n_fine : n;
  km->inverse = inverse ? 1 : 0;
  km->n_in = n;
  km->stream = stream;
  km->mask_words = (kvol + 31) / 32;
  km->offset_start.assign(size_t(kvol) + 1, 0);
  SPCONV_CUDA_TRY(cudaGetDevice(&km->device));
  if (nq == 0 || (n == 0 && !inverse)) {  // empty map: no device memory at all
    *out = km; guard.km = nullptr;
    return SPCONV_OK;
  }

  const int nblk = int((nq + kBlock - 1) / kBlock);
  const int64_t M = int64_t(nblk) * kvol;
  // Load factor of the location table: at most 1/4.  Probe sequences are walked by whole warps (a warp takes as
  // many rounds as its unluckiest lane), so short sequences matter more than the table's size.
  // Test hook (spconv_test_hook, SPCONV_HOOK_TABLE_SLOTS): a positive value forces the table to pow2(value) slots
  // whatever the input, so that a test can make the bounded probe sequence run out (SPCONV_ERR_TABLE_FULL).
  const long long forced_slots = g_test_table_slots.load(std::memory_order_relaxed);
  const uint32_t cap1 = forced_slots > 0 ? pow2_at_least(uint64_t(forced_slots)) : pow2_at_least(uint64_t(4) * std::max<int64_t>(n, 1));
  const dim3 grid_kn(nblk, kvol);
  const int4* coords4 = reinterpret_cast<const int4*>(coords);
  const int4* qcoords4 = inverse ? reinterpret_cast<const int4*>(fine_coords) : coords4;
  const int nblk_in = int((n + kBlock - 1) / kBlock);   // blocks over the rows that go into the location table
  // Kernel volumes up to 32 keep a second, row-major copy of the offset table (rows of 32 entries) for the tile plan.
  const bool rows_table = kvol <= 32;

  keep_pool_cached(km->device);
  PinnedHost host;
  host.count = 8 + size_t(kvol) + 1 + 1;   // totals, offset starts, ready flag
  host.p = g_pinned.get(host.count);
  if (!host.p) return SPCONV_ERR_ALLOC;
  int64_t* h_totals = host.p;            // [0] n_out, [1] P, [2] status word, [3] tile blocks
  int64_t* h_offset_start = host.p + 8;  // [kvol+1]

  // ----- scratch arena (freed stream-ordered when this function leaves)
  uint32_t cap2 = 0;
  int64_t n_out_max = n;
  if (!known_outputs) {
    const int cpa = max_candidates_per_axis(K, s, d);
    n_out_max = std::min<int64_t>(n * int64_t(cpa) * cpa * cpa, int64_t(2000000000));
    cap2 = pow2_at_least(uint64_t(2) * n_out_max);
  }
  // The tile plan sorts rows by their offset set when it fits one 32-bit key, unless the caller asked for tiles of
  // consecutive rows (SPCONV_ROWS_AS_GIVEN: no sort, more (tile, offset) blocks).
  const bool plan_sorted = kvol <= 32 && !rows_as_given;
  // The radix sort takes 8 bits per pass; the three passes over the 24 most significant key bits (the rarest
  // offsets) already bring the block count within a few per cent of the full sort's.
  const int sort_begin_bit = kvol > 24 ? kvol - 24 : 0;
  auto sort_bytes_for = [&](int64_t items, size_t* cub_bytes) {
    *cub_bytes = 0;
    if (!plan_sorted) return size_t(0);
    cub::DeviceRadixSort::SortPairs(nullptr, *cub_bytes, static_cast<uint32_t*>(nullptr), static_cast<uint32_t*>(nullptr),
                                    static_cast<int32_t*>(nullptr), static_cast<int32_t*>(nullptr), int(items), sort_begin_bit, kvol, stream);
    return pad256(*cub_bytes) + pad256(size_t(items) * 4) * 4 + pad256((size_t(items) / (kSortThreads * kSortItemsSmall) + 8) * 1024) +
           pad256((size_t(items) / kTileRows + 2) * 4) + 1024;
  };
  size_t cub_bytes = 0;
  size_t scratch_bytes = pad256(std::max(size_t(cap1) * sizeof(LocSlot), dense_grid != nullptr ? size_t(dense_grid[0]) * dense_grid[1] * dense_grid[2] * dense_grid[3] * 4 : size_t(0))) +
                         pad256(size_t(kOccWords) * 4) + pad256(size_t(M) * 4) * 2 +
                         pad256(size_t(M) * 8) * 2 + pad256((size_t(kvol) + 1 + 8 + 16) * 8) + pad256(32) + 4096;
  if (known_outputs) scratch_bytes += sort_bytes_for(nq, &cub_bytes);   // n_out is known: the sort's buffers ride along
  if (known_outputs && rows_table) scratch_bytes += pad256(size_t(nq) * 128) + pad256(size_t(nq) * 4);
  if (!known_outputs)
    scratch_bytes += pad256(size_t(cap2) * 8) + pad256(size_t(cap2) * 4) * 2 + pad256(size_t(kvol) * n * 4);
  Scratch scratch;
  scratch.stream = stream;
  SPCONV_CUDA_TRY(cudaMallocAsync(&scratch.ptr, scratch_bytes, stream));
  Arena sa{static_cast<char*>(scratch.ptr), scratch_bytes, 0};
  // Location table: the hash table with its occupancy filter right behind it (one fill empties both), or, where the
  // caller stated a grid, the dense array of that grid's cells (every byte 0xFF = -1: no row).
  GridDims grid_dims{0, 0, 0, 0};
  if (dense_grid != nullptr) grid_dims = GridDims{dense_grid[0], dense_grid[1], dense_grid[2], dense_grid[3]};
  const size_t dense_cells = dense_grid != nullptr ? size_t(dense_grid[0]) * dense_grid[1] * dense_grid[2] * dense_grid[3] : 0;
  LocSlot* table1 = dense_grid != nullptr ? reinterpret_cast<LocSlot*>(sa.take<int32_t>(dense_cells)) : sa.take<LocSlot>(cap1);
  uint32_t* occ = (known_outputs && rows_table && dense_grid == nullptr) ? sa.take<uint32_t>(kOccWords) : nullptr;
  const size_t table_fill_bytes = dense_grid != nullptr ? dense_cells * 4
                                  : occ != nullptr ? size_t(reinterpret_cast<char*>(occ + kOccWords) - reinterpret_cast<char*>(table1))
                                                   : size_t(cap1) * sizeof(LocSlot);
  int32_t* cnt_a = sa.take<int32_t>(M);
  int32_t* cnt_b = sa.take<int32_t>(M);
  int64_t* excl_a = sa.take<int64_t>(M);
  int64_t* excl_b = sa.take<int64_t>(M);
  // One zero-initialised block read back in one copy: totals [8] | offset_start [kvol + 1] | per-offset counts [32 x u32]
  const size_t totals_words = 8 + size_t(kvol) + 1;
  int64_t* d_totals = sa.take<int64_t>(totals_words + 32);   // ... | per-offset counts [32 x u32] | tiles per block count [32 x u32]
  int64_t* d_offset_start = d_totals + 8;
  // (32 counters: only maps with kvol <= 32 get per-offset totals, which is also where the tile plan sorts by them)
  unsigned* d_offset_cnt = kvol <= 32 ? reinterpret_cast<unsigned*>(d_totals + totals_words) : nullptr;
  unsigned* d_class_cnt = kvol <= 31 ? reinterpret_cast<unsigned*>(d_totals + totals_words + 16) : nullptr;
  int8_t* d_bitpos = sa.take<int8_t>(32);
  uint32_t* d_status = reinterpret_cast<uint32_t*>(d_totals + 2);
  unsigned long long* d_tile_blocks = reinterpret_cast<unsigned long long*>(d_totals + 3);
  unsigned* d_tiles_done = reinterpret_cast<unsigned*>(d_totals + 4);
  uint64_t* keys2 = nullptr; int32_t* owner_cid = nullptr; int32_t* slot_out = nullptr; int32_t* cand_slot = nullptr;
  int32_t* nbr_rows = nullptr;     // [n_out][32] row-major offset table (scratch)
  uint32_t* row_mask = nullptr;    // [n_out] offset set of every row, when the probe kernel forms it
  if (known_outputs && rows_table) {
    nbr_rows = sa.take<int32_t>(size_t(nq) * 32);
    row_mask = sa.take<uint32_t>(size_t(nq));
  }
  if (!known_outputs) {
    keys2 = sa.take<uint64_t>(cap2);
    owner_cid = sa.take<int32_t>(cap2);
    slot_out = sa.take<int32_t>(cap2);
    cand_slot = sa.take<int32_t>(size_t(kvol) * n);
  }

  // Persistent allocation 1: every array of the handle except the pair lists, for n_out output rows.
  auto allocate_map_arrays = [&](int64_t no) -> int {
    km->n_out = no;
    km->n_tiles = int32_t((no + kTileRows - 1) / kTileRows);
    const size_t bytes = pad256(size_t(no) * 16) + pad256(size_t(kvol) * no * 4) + pad256(size_t(km->n_tiles) * kTileRows * 4) +
                         pad256(size_t(km->n_tiles) * kvol * kTileRows * 4) + pad256(size_t(km->n_tiles) * km->mask_words * 4) +
                         pad256(size_t(km->n_tiles) * 4 * (1 + km->mask_words)) + pad256(size_t(km->n_tiles) * kvol * 16) +
                         pad256(size_t(km->n_tiles) * kvol * kTileRows) + pad256(64) + 2048;
    int32_t* base = nullptr;
    SPCONV_CUDA_TRY(cudaMallocAsync(reinterpret_cast<void**>(&base), bytes, stream));
    km->d.out_coords = base;  // owner pointer of allocation 1 (the first array starts at its base)
    Arena pa{reinterpret_cast<char*>(base), bytes, 0};
    km->d.out_coords = pa.take<int32_t>(size_t(no) * 4);
    km->d.nbr = pa.take<int32_t>(size_t(kvol) * no);
    km->d.tile_rows = pa.take<int32_t>(size_t(km->n_tiles) * kTileRows);
    km->d.tile_nbr = pa.take<int32_t>(size_t(km->n_tiles) * kvol * kTileRows);
    km->d.tile_mask = pa.take<uint32_t>(size_t(km->n_tiles) * km->mask_words);
    km->d.sorted_tiles = pa.take<int32_t>(size_t(km->n_tiles) * (1 + km->mask_words));
    km->d.tile_absent = pa.take<uint32_t>(size_t(km->n_tiles) * kvol * 4);
    km->d.tile_crow = pa.take<uint8_t>(size_t(km->n_tiles) * kvol * kTileRows);
    km->d.status = pa.take<uint32_t>(16);
    return SPCONV_OK;
  };
  // Tile plan of the tensor-core forward: rows sorted by offset set, cut into tiles, scheduled.  Needs
  // nbr, the per-offset counts' bit order (d_bitpos, written by k_scan_counts) and sort buffers.
  int64_t* flag_target = nullptr;   // pinned host buffer the tile plan's last block reports into (submanifold path)
  std::function<int()> after_sort;   // (submanifold path) enqueues the pair emission beside the tile plan
  // Maps whose outputs are known up front and whose kernel volume fits the 32 per-offset counters need no scan of the
  // probe's per-block counts: the report to the host and the bit order of the sort come from the per-offset totals,
  // and the emission's blocks sum their own list positions.
  const bool counts_based = known_outputs && d_offset_cnt != nullptr;
  const int32_t* plan_rows = nullptr;      // row-major offset table the sort and the tile plan read, when there is one
  const uint32_t* plan_row_mask = nullptr; // offset sets of the rows, when the probe kernel has formed them
  auto enqueue_tile_plan = [&](Arena& ta, size_t cub_tmp_bytes, bool scan_pending) -> int {
    const int64_t no = km->n_out, padded = int64_t(km->n_tiles) * kTileRows;
    const int rb = int((padded + kBlock - 1) / kBlock);
    if (plan_sorted) {
      uint32_t* rkeys = ta.take<uint32_t>(no);
      uint32_t* rkeys_sorted = ta.take<uint32_t>(no);
      int32_t* rrows = ta.take<int32_t>(no);
      int32_t* rrows_b = ta.take<int32_t>(no);
      // few items per thread while all such blocks (and the scan's block) are resident at once, else many
      const int small_blocks = int((padded + kSortThreads * kSortItemsSmall - 1) / (kSortThreads * kSortItemsSmall));
      const bool small_sort = small_blocks <= kSortSmallMaxBlocks && small_blocks + 1 <= coop_sort_capacity(km->device, false);
      const int sort_tile = kSortThreads * (small_sort ? kSortItemsSmall : kSortItemsLarge);
      const int sort_blocks = int((padded + sort_tile - 1) / sort_tile);
      uint32_t* block_hist = ta.take<uint32_t>(size_t(sort_blocks + 1) * 256);
      void* cub_tmp = ta.take<char>(cub_tmp_bytes);
      size_t tmp_bytes = cub_tmp_bytes;
      const unsigned* order_cnt = (scan_pending || counts_based) ? d_offset_cnt : nullptr;   // the probe's per-offset totals order the key bits
      if (sort_blocks + 1 <= coop_sort_capacity(km->device, !small_sort)) {
        // every block resident at once: keys and all sort passes in one cooperative launch
        const int32_t* nbr_arg = km->d.nbr;
        const int32_t* rows_arg = plan_rows;
        const uint32_t* mask_arg = plan_row_mask;
        int64_t no_arg = no, padded_arg = padded;
        int kvol_arg = kvol, begin_arg = sort_begin_bit;
        const int8_t* bitpos_arg = d_bitpos;
        const unsigned* cnt_arg = order_cnt;
        int32_t* tile_rows_arg = km->d.tile_rows;
        const int32_t* scan_cnt_arg = scan_pending ? cnt_a : nullptr;
        int64_t scan_m_arg = M;
        int64_t* scan_excl_arg = excl_a;
        int scan_nblk_arg = nblk;
        int64_t* scan_os_arg = d_offset_start;
        int64_t* scan_total_arg = d_totals + 1;
        void* args[] = {&nbr_arg, &rows_arg, &mask_arg, &no_arg, &padded_arg, &kvol_arg, &bitpos_arg, &cnt_arg, &begin_arg, &rkeys, &rrows, &rkeys_sorted,
                        &rrows_b, &block_hist, &tile_rows_arg, &scan_cnt_arg, &scan_m_arg, &scan_excl_arg, &scan_nblk_arg, &scan_os_arg,
                        &scan_total_arg};
        // (with the scan on board the grid has one block more; the capacity test above leaves room for it)
        void* kernel = small_sort ? reinterpret_cast<void*>(k_sort_rows_coop<kSortItemsSmall>) : reinterpret_cast<void*>(k_sort_rows_coop<kSortItemsLarge>);
        SPCONV_CUDA_TRY(cudaLaunchCooperativeKernel(kernel, dim3(sort_blocks + (scan_pending ? 1 : 0)), dim3(kSortThreads), args, 0, stream));
      } else {
        if (scan_pending) k_scan_counts<<<1, 1024, 0, stream>>>(cnt_a, M, excl_a, nblk, kvol, d_offset_start, d_totals + 1, d_bitpos);
        k_row_keys<<<rb, kBlock, 0, stream>>>(km->d.nbr, no, padded, kvol, d_bitpos, order_cnt, rkeys, rrows, km->d.tile_rows);
        SPCONV_CUDA_TRY(cub::DeviceRadixSort::SortPairs(cub_tmp, tmp_bytes, rkeys, rkeys_sorted, rrows, km->d.tile_rows, int(no),
                                                        sort_begin_bit, kvol, stream));
      }
    } else {
      if (scan_pending) k_scan_counts<<<1, 1024, 0, stream>>>(cnt_a, M, excl_a, nblk, kvol, d_offset_start, d_totals + 1, d_bitpos);
      k_iota_rows<<<rb, kBlock, 0, stream>>>(km->d.tile_rows, no, padded);
    }
    SPCONV_STAGE(stages, "sort");
    if (after_sort) { const int e = after_sort(); if (e != SPCONV_OK) return e; }
    if (plan_rows != nullptr) {
      int32_t* tile_within = (plan_sorted && d_class_cnt != nullptr) ? ta.take<int32_t>(size_t(km->n_tiles)) : nullptr;
      SPCONV_CUDA_TRY(launch_chained(k_tile_plan_rows, dim3(km->n_tiles), dim3(kTileRows), stream, static_cast<const int32_t*>(km->d.tile_rows),
                                     plan_rows, kvol, km->d.tile_nbr, km->d.tile_crow, km->d.tile_mask, km->d.tile_absent, d_tile_blocks,
                                     d_tiles_done, km->d.sorted_tiles, km->d.status, static_cast<const int64_t*>(d_totals),
                                     int(totals_words), flag_target, counts_based ? 1 : 0,
                                     tile_within != nullptr ? d_class_cnt : static_cast<unsigned*>(nullptr), tile_within));
    }
    else if (kvol <= 32)
      SPCONV_CUDA_TRY(launch_chained(k_tile_plan<true>, dim3(km->n_tiles), dim3(kTileRows), stream, km->d.tile_rows, km->d.nbr, no, kvol,
                                     km->mask_words, km->d.tile_nbr, km->d.tile_crow, km->d.tile_mask, km->d.tile_absent, d_tile_blocks,
                                     d_tiles_done, km->d.sorted_tiles, km->d.status, static_cast<const int64_t*>(d_totals),
                                     int(totals_words), flag_target));
    else
      k_tile_plan<false><<<km->n_tiles, kTileRows, 0, stream>>>(km->d.tile_rows, km->d.nbr, no, kvol, km->mask_words, km->d.tile_nbr,
                                                                km->d.tile_crow, km->d.tile_mask, km->d.tile_absent, d_tile_blocks, d_tiles_done,
                                                                km->d.sorted_tiles, km->d.status, static_cast<const int64_t*>(d_totals),
                                                                int(totals_words), flag_target);
    SPCONV_STAGE(stages, "tile_plan");
    return SPCONV_OK;
  };
  auto allocate_pairs = [&](int64_t capacity) -> int {
    const size_t half = pad256(size_t(std::max<int64_t>(capacity, 1)) * 4);
    int32_t* pairs = nullptr;
    SPCONV_CUDA_TRY(cudaMallocAsync(reinterpret_cast<void**>(&pairs), half * 2 + 512, stream));
    km->d.pair_in = pairs;  // owner pointer of allocation 2
    km->d.pair_out = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(pairs) + half);
    return SPCONV_OK;
  };

  // Wait for a report from the device: the totals block in the pinned buffer with the flag raised behind it.
  // The stream is queried now and then so that a failed launch ends the wait, and after a generous time the
  // ordinary synchronisation takes over.
  volatile int64_t* ready = h_totals + totals_words;
  const OffsetIndex offset_table = make_offset_index(K);
  auto expect_report = [&]() {
    *ready = 0;
    host.writer = stream;
    host.write_pending = true;
  };
  auto wait_for_report = [&]() -> int {
    const auto t0 = std::chrono::steady_clock::now();
    bool arrived = false;
    for (uint64_t spin = 0;; ++spin) {
      if (*ready == 1) { arrived = true; break; }
      if ((spin & 0x3FFu) == 0x3FFu) {
        const cudaError_t q = cudaStreamQuery(stream);
        if (q != cudaErrorNotReady) break;   // finished (the flag is there by now) or failed
        if (std::chrono::steady_clock::now() - t0 > std::chrono::milliseconds(20)) break;
      }
    }
    if (!arrived) {
      SPCONV_CUDA_TRY(cudaStreamSynchronize(stream));
      host.write_pending = false;
      if (*ready != 1) return SPCONV_ERR_CUDA;
    }
    host.write_pending = false;
    SPCONV_CUDA_TRY(cudaGetLastError());
    const int e = device_status_to_error(uint32_t(h_totals[2]));
    if (e != SPCONV_OK) return e;
    km->total_pairs = h_totals[1];
    for (int k = 0; k <= kvol; ++k) km->offset_start[k] = h_offset_start[k];
    return SPCONV_OK;
  };

  {  // (every region starts on a 256-byte boundary of the arena and is followed by padding up to the next one, so
     // rounding a size up to 16 bytes stays inside its own padding)
    FillRegions fr = {};
    fr.ptr[0] = reinterpret_cast<uint4*>(d_totals); fr.count16[0] = ((totals_words + 32) * sizeof(int64_t) + 15) / 16; fr.value[0] = 0u;
    fr.ptr[1] = reinterpret_cast<uint4*>(table1); fr.count16[1] = (table_fill_bytes + 15) / 16; fr.value[1] = 0xFFFFFFFFu;
    if (!known_outputs) {
      fr.ptr[2] = reinterpret_cast<uint4*>(keys2); fr.count16[2] = size_t(cap2) * 8 / 16; fr.value[2] = 0xFFFFFFFFu;
      fr.ptr[3] = reinterpret_cast<uint4*>(owner_cid); fr.count16[3] = size_t(cap2) * 4 / 16; fr.value[3] = 0x7F7F7F7Fu;
    }
    const size_t words = fr.count16[0] + fr.count16[1] + fr.count16[2] + fr.count16[3];
    const unsigned blocks = unsigned(std::min<size_t>((words + 255) / 256, 148 * 8));
    SPCONV_CUDA_TRY(launch_chained(k_fill_regions, dim3(blocks), dim3(256), stream, fr));
  }

  if (known_outputs) {
    // Every size is known up front (submanifold: n_out = n; inverse: the fine positions), so the whole map including
    // the tile plan is enqueued before the host waits once, for the error word and the pair count.
    // (the insert is enqueued before the handle's arrays are allocated where it does not write into them: the device
    // starts a build when its first kernels arrive, and every host call in front of them is time it stands idle)
    if (!rows_table) { const int e = allocate_map_arrays(nq); if (e != SPCONV_OK) return e; }
    SPCONV_STAGE(stages, "alloc+memset");
    SPCONV_HOST_TL("allocs+memsets");
    int4* out_coords4 = reinterpret_cast<int4*>(km->d.out_coords);   // (null until the arrays exist)
    if (n > 0 && dense_grid != nullptr)
      SPCONV_CUDA_TRY(launch_chained(k_insert_dense, dim3(nblk_in), dim3(kBlock), stream, coords4, int(n), reinterpret_cast<int32_t*>(table1),
                                     grid_dims, d_status));
    else if (n > 0)
      SPCONV_CUDA_TRY(launch_chained(k_insert, dim3(nblk_in), dim3(kBlock), stream, coords4, int(n), table1, cap1 - 1, d_status,
                                     (submanifold && !rows_table) ? out_coords4 : static_cast<int4*>(nullptr), occ));
    SPCONV_STAGE(stages, "insert");
    if (rows_table) {
      { const int e = allocate_map_arrays(nq); if (e != SPCONV_OK) return e; }
      out_coords4 = reinterpret_cast<int4*>(km->d.out_coords);
      // every offset of a row in one thread; also copies the rows' coordinates into the handle
      auto probe_rows = [&](auto kernel) {
        return launch_chained(kernel, dim3(nblk), dim3(kBlock), stream, qcoords4, int(nq), d, s, static_cast<const LocSlot*>(table1),
                              cap1 - 1, static_cast<const uint32_t*>(occ), km->d.nbr, nbr_rows, row_mask,
                              cnt_a, d_offset_cnt, out_coords4, d_status, grid_dims);
      };
      cudaError_t le = cudaErrorInvalidValue;
      if (dense_grid != nullptr) le = K == 1 ? probe_rows(k_probe_rows<1, 0, true>) : probe_rows(k_probe_rows<3, 0, true>);
      else if (!inverse) le = K == 1 ? probe_rows(k_probe_rows<1, 0>) : probe_rows(k_probe_rows<3, 0>);
      else le = K == 1 ? probe_rows(k_probe_rows<1, 1>) : K == 2 ? probe_rows(k_probe_rows<2, 1>) : probe_rows(k_probe_rows<3, 1>);
      SPCONV_CUDA_TRY(le);
      plan_rows = nbr_rows;
      plan_row_mask = row_mask;
    } else if (inverse) {
      SPCONV_CUDA_TRY(cudaMemcpyAsync(km->d.out_coords, fine_coords, size_t(nq) * 16, cudaMemcpyDeviceToDevice, stream));
      SPCONV_CUDA_TRY(launch_chained(k_inverse_probe, grid_kn, dim3(kBlock), stream, qcoords4, int(nq), K, s, d, static_cast<const LocSlot*>(table1),
                                     cap1 - 1, km->d.nbr, cnt_a, d_offset_cnt, d_status, offset_table));
    } else {
      SPCONV_CUDA_TRY(launch_chained(k_subm_probe, grid_kn, dim3(kBlock), stream, coords4, int(n), K, d, static_cast<const LocSlot*>(table1), cap1 - 1, km->d.nbr,
                                     cnt_a, d_offset_cnt, offset_table));
    }
    SPCONV_STAGE(stages, "probe");
    SPCONV_HOST_TL("insert+probe");
    // Pair lists: their exact size is only known on the device.  They are sized for 16 pairs per row (the
    // workloads have 4-13); a denser input gets exact lists and a second emission after the wait.  Nothing on the
    // way to the forward reads them, so their emission runs on a second stream beside the tile plan; the caller's
    // stream joins that stream again behind whatever the caller's hook enqueues (the forward of spconv_layer), or
    // at once.
    const int64_t pair_capacity = std::min<int64_t>(int64_t(kvol) * nq, 16 * nq);
    { const int e = allocate_pairs(pair_capacity); if (e != SPCONV_OK) return e; }
    const bool hooked = before_wait != nullptr && *before_wait;
    SideStream* side = side_stream_for(km->device);
    struct Rejoin {   // whatever happens after the fork, the caller's stream (which later frees the arrays) waits for the side stream
      cudaStream_t stream; SideStream* side; bool forked = false;
      ~Rejoin() { if (forked) { (void)cudaEventRecord(side->join, side->s); (void)cudaStreamWaitEvent(stream, side->join, 0); } }
    } rejoin{stream, side};
    // The emission needs the offset table and the probe's hit counts, not the sort or the tile plan, so it is
    // forked off behind the probe.  (Its blocks find their list positions themselves where per-offset totals
    // exist; otherwise they need the scan of the per-block counts, which rides in the sort's launch, and the fork
    // comes behind the sort.)
    const int64_t* emit_excl = counts_based ? nullptr : excl_a;
    auto fork_emit = [&]() -> int {
      if (side == nullptr) return SPCONV_OK;
      SPCONV_CUDA_TRY(cudaEventRecord(side->fork, stream));
      SPCONV_CUDA_TRY(cudaStreamWaitEvent(side->s, side->fork, 0));
      rejoin.forked = true;
      k_subm_emit<<<grid_kn, kBlock, 0, side->s>>>(km->d.nbr, int(nq), emit_excl, cnt_a, d_offset_cnt, km->d.pair_in, km->d.pair_out, pair_capacity);
      SPCONV_CUDA_TRY(cudaEventRecord(side->join, side->s));
      return SPCONV_OK;
    };
    if (counts_based) { const int e = fork_emit(); if (e != SPCONV_OK) return e; }
    else after_sort = fork_emit;
    SPCONV_HOST_TL("pairs+fork+emit");
    expect_report();
    flag_target = h_totals;
    { const int e = enqueue_tile_plan(sa, cub_bytes, !counts_based); if (e != SPCONV_OK) return e; }
    SPCONV_HOST_TL("sort+plan");
    flag_target = nullptr;
    after_sort = nullptr;
    if (side == nullptr)
      SPCONV_CUDA_TRY(launch_chained(k_subm_emit, grid_kn, dim3(kBlock), stream, static_cast<const int32_t*>(km->d.nbr), int(nq), emit_excl,
                                     static_cast<const int32_t*>(cnt_a), static_cast<const unsigned*>(d_offset_cnt), km->d.pair_in, km->d.pair_out,
                                     pair_capacity));
    SPCONV_STAGE(stages, "schedule");
    if (hooked) { const int e = (*before_wait)(km); if (e != SPCONV_OK) return e; }
    if (side != nullptr) {
      SPCONV_CUDA_TRY(cudaStreamWaitEvent(stream, side->join, 0));
      rejoin.forked = false;
    }
    SPCONV_HOST_TL("before wait");
    { const int e = wait_for_report(); if (e != SPCONV_OK) return e; }
    SPCONV_HOST_TL("after wait");
    SPCONV_STAGE(stages, "readback+sync");
    km->tile_blocks = h_totals[3];
    if (km->total_pairs > pair_capacity) {
      SPCONV_CUDA_TRY(cudaFreeAsync(km->d.pair_in, stream));
      km->d.pair_in = nullptr;
      { const int e = allocate_pairs(km->total_pairs); if (e != SPCONV_OK) return e; }
      SPCONV_CUDA_TRY(launch_chained(k_subm_emit, grid_kn, dim3(kBlock), stream, static_cast<const int32_t*>(km->d.nbr), int(nq), emit_excl,
                                     static_cast<const int32_t*>(cnt_a), static_cast<const unsigned*>(d_offset_cnt), km->d.pair_in, km->d.pair_out,
                                     km->total_pairs));
    }
    SPCONV_STAGE(stages, "alloc+emit");
    SPCONV_CUDA_TRY(cudaGetLastError());
  } else {
    // The number of output rows is only known on the device: one wait for the sizes, a second one at the end
    // for the tile plan's block count.
    const int pad = d * ((K - 1) / 2);
    SPCONV_CUDA_TRY(launch_chained(k_insert, dim3(nblk), dim3(kBlock), stream, coords4, int(n), table1, cap1 - 1, d_status,
                                   static_cast<int4*>(nullptr), static_cast<uint32_t*>(nullptr)));
    SPCONV_CUDA_TRY(launch_chained(k_strided_candidates, grid_kn, dim3(kBlock), stream, coords4, int(n), K, s, d, pad, keys2, owner_cid,
                                   cap2 - 1, cand_slot, cnt_a, d_status, offset_table));
    SPCONV_CUDA_TRY(launch_chained(k_scan_counts, dim3(1), dim3(1024), stream, static_cast<const int32_t*>(cnt_a), M, excl_a, nblk, kvol,
                                   d_offset_start, d_totals + 1, d_bitpos));
    SPCONV_CUDA_TRY(launch_chained(k_owner_count, grid_kn, dim3(kBlock), stream, static_cast<const int32_t*>(cand_slot),
                                   static_cast<const int32_t*>(owner_cid), int(n), cnt_b));
    SPCONV_CUDA_TRY(launch_chained(k_scan_counts, dim3(1), dim3(1024), stream, static_cast<const int32_t*>(cnt_b), M, excl_b, nblk, kvol,
                                   static_cast<int64_t*>(nullptr), d_totals + 0, static_cast<int8_t*>(nullptr)));
    expect_report();
    SPCONV_CUDA_TRY(launch_chained(k_report_totals, dim3(1), dim3(64), stream, static_cast<const int64_t*>(d_totals), int(totals_words),
                                   h_totals));
    { const int e = wait_for_report(); if (e != SPCONV_OK) return e; }
    { const int e = allocate_map_arrays(h_totals[0]); if (e != SPCONV_OK) return e; }
    const int64_t no = km->n_out;
    { const int e = allocate_pairs(km->total_pairs); if (e != SPCONV_OK) return e; }
    Scratch sort_scratch;
    sort_scratch.stream = stream;
    size_t cub2 = 0;
    const size_t bytes = sort_bytes_for(no, &cub2) + (rows_table ? pad256(size_t(no) * 128) : 0) + 512;
    SPCONV_CUDA_TRY(cudaMallocAsync(&sort_scratch.ptr, bytes, stream));
    Arena ta{static_cast<char*>(sort_scratch.ptr), bytes, 0};
    if (rows_table) {
      nbr_rows = ta.take<int32_t>(size_t(no) * 32);
      plan_rows = nbr_rows;
    }
    {  // both layouts of the offset table start as "no input row" (-1); one kernel in the chain, as at the start of a build
      FillRegions fr = {};
      fr.ptr[0] = reinterpret_cast<uint4*>(km->d.nbr); fr.count16[0] = (size_t(kvol) * no * 4 + 15) / 16; fr.value[0] = 0xFFFFFFFFu;
      if (nbr_rows != nullptr) { fr.ptr[1] = reinterpret_cast<uint4*>(nbr_rows); fr.count16[1] = size_t(no) * 128 / 16; fr.value[1] = 0xFFFFFFFFu; }
      const size_t words = fr.count16[0] + fr.count16[1];
      SPCONV_CUDA_TRY(launch_chained(k_fill_regions, dim3(unsigned(std::min<size_t>((words + 255) / 256, 148 * 8))), dim3(256), stream, fr));
    }
    SPCONV_CUDA_TRY(launch_chained(k_owner_assign, grid_kn, dim3(kBlock), stream, static_cast<const int32_t*>(cand_slot),
                                   static_cast<const int32_t*>(owner_cid), static_cast<const uint64_t*>(keys2), int(n),
                                   static_cast<const int64_t*>(excl_b), slot_out, reinterpret_cast<int4*>(km->d.out_coords)));
    SPCONV_CUDA_TRY(launch_chained(k_strided_emit, grid_kn, dim3(kBlock), stream, static_cast<const int32_t*>(cand_slot),
                                   static_cast<const int32_t*>(slot_out), int(n), km->n_out, static_cast<const int64_t*>(excl_a),
                                   km->d.nbr, km->d.pair_in, km->d.pair_out, nbr_rows));
    expect_report();
    flag_target = h_totals;
    { const int e = enqueue_tile_plan(ta, cub2, false); if (e != SPCONV_OK) return e; }
    flag_target = nullptr;
    { const int e = wait_for_report(); if (e != SPCONV_OK) return e; }
    km->tile_blocks = h_totals[3];
  }
  *out = km;
  guard.km = nullptr;
  return SPCONV_OK;
}

}  // namespace spconv


// =============================================================================================
// Voxelisation of raw points (see spconv_voxelize in the header): the step the paper assumes upstream of its
// operators (Sec. II-A).  Built from the parts of the strided map: every point's cell is inserted into a hash table
// of cells, the point with the lowest index owns the cell (atomicMin), cells are numbered in owner order -- the
// order of their first point, the same on every run -- and then every point adds its features to its cell's row.
namespace spconv {
namespace {

struct VoxGrid { float ox, oy, oz, vx, vy, vz; int gx, gy, gz, batch; };

// One thread per point: the cell in float32 exactly as floor((p - origin) / voxel_size), points outside the grid dropped.
__global__ void k_vox_cells(const float* __restrict__ points, int n, int stride_floats, const __grid_constant__ VoxGrid g,
                            uint64_t* keys, int32_t* owner, uint32_t capmask, int32_t* __restrict__ point_slot, uint32_t* status) {
  chain_begin();
  const int i = blockIdx.x * kBlock + threadIdx.x;
  if (i >= n) return;
  const float* p = points + size_t(i) * stride_floats;
  const float fx = floorf(__fdiv_rn(__fsub_rn(p[0], g.ox), g.vx)), fy = floorf(__fdiv_rn(__fsub_rn(p[1], g.oy), g.vy)),
              fz = floorf(__fdiv_rn(__fsub_rn(p[2], g.oz), g.vz));
  int slot = -1;
  if (fx >= 0.f && fx < float(g.gx) && fy >= 0.f && fy < float(g.gy) && fz >= 0.f && fz < float(g.gz)) {
    bool present;
    slot = table_insert<1>(keys, capmask, pack_key(g.batch, int(fx), int(fy), int(fz)), &present);
    if (slot < 0) atomicOr(status, kDevTableFull);
    else atomicMin(owner + slot, i);
  }
  point_slot[i] = slot;
}

// One thread per (point, feature): the point's features are added to its voxel's row; thread 0 of a point counts it.
__global__ void k_vox_accumulate(const float* __restrict__ points, int n, int stride_floats, int n_feat, const int32_t* __restrict__ point_slot,
                                 const int32_t* __restrict__ slot_voxel, float* __restrict__ feats, int32_t* __restrict__ counts) {
  chain_begin();
  const int64_t e = int64_t(blockIdx.x) * kBlock + threadIdx.x;
  const int cols = n_feat > 0 ? n_feat : 1;
  const int64_t i = e / cols;
  const int f = int(e - i * cols);
  if (i >= n) return;
  const int slot = point_slot[i];
  if (slot < 0) return;
  const int v = slot_voxel[slot];
  if (n_feat > 0) atomicAdd(feats + size_t(v) * n_feat + f, points[size_t(i) * stride_floats + 3 + f]);
  if (f == 0) atomicAdd(counts + v, 1);
}

__global__ void k_vox_normalize(float* __restrict__ feats, const int32_t* __restrict__ counts, int64_t m, int n_feat) {
  chain_begin();
  const int64_t e = int64_t(blockIdx.x) * kBlock + threadIdx.x;
  if (e >= m * n_feat) return;
  feats[e] = __fdiv_rn(feats[e], float(counts[e / n_feat]));
}

}  // namespace

int voxelize_impl(const float* points, int64_t n, int point_stride, int n_feat, int batch_index, const float* origin,
                  const float* voxel_size, const int32_t* grid_shape, int32_t* coords_out, float* feats_out, int32_t* counts_out,
                  int64_t capacity, int64_t* n_voxels_host, cudaStream_t stream) {
  *n_voxels_host = 0;
  if (n == 0) return SPCONV_OK;
  int device = 0;
  SPCONV_CUDA_TRY(cudaGetDevice(&device));
  keep_pool_cached(device);
  const int nblk = int((n + kBlock - 1) / kBlock);
  const uint32_t cap = pow2_at_least(uint64_t(2) * n);
  const size_t totals_words = 8;
  PinnedHost host;
  host.count = totals_words + 2;
  host.p = g_pinned.get(host.count);
  if (!host.p) return SPCONV_ERR_ALLOC;
  const size_t bytes = pad256(size_t(cap) * 8) + pad256(size_t(cap) * 4) * 2 + pad256(size_t(n) * 4) + pad256(size_t(nblk) * 4) +
                       pad256(size_t(nblk) * 8) + pad256(totals_words * 8) + pad256(size_t(capacity > 0 ? capacity : 1) * 4) + 4096;
  Scratch scratch;
  scratch.stream = stream;
  SPCONV_CUDA_TRY(cudaMallocAsync(&scratch.ptr, bytes, stream));
  Arena sa{static_cast<char*>(scratch.ptr), bytes, 0};
  uint64_t* keys = sa.take<uint64_t>(cap);
  int32_t* owner = sa.take<int32_t>(cap);
  int32_t* slot_voxel = sa.take<int32_t>(cap);
  int32_t* point_slot = sa.take<int32_t>(n);
  int32_t* cnt = sa.take<int32_t>(nblk);
  int64_t* excl = sa.take<int64_t>(nblk);
  int64_t* d_totals = sa.take<int64_t>(totals_words);
  int32_t* own_counts = counts_out != nullptr ? counts_out : sa.take<int32_t>(size_t(capacity > 0 ? capacity : 1));
  uint32_t* d_status = reinterpret_cast<uint32_t*>(d_totals + 2);
  SPCONV_CUDA_TRY(cudaMemsetAsync(d_totals, 0, totals_words * 8, stream));
  SPCONV_CUDA_TRY(cudaMemsetAsync(keys, 0xFF, size_t(cap) * 8, stream));
  SPCONV_CUDA_TRY(cudaMemsetAsync(owner, 0x7F, size_t(cap) * 4, stream));
  const VoxGrid g{origin[0], origin[1], origin[2], voxel_size[0], voxel_size[1], voxel_size[2], grid_shape[0], grid_shape[1], grid_shape[2], batch_index};
  SPCONV_CUDA_TRY(launch_chained(k_vox_cells, dim3(nblk), dim3(kBlock), stream, points, int(n), point_stride, g, keys, owner, cap - 1, point_slot, d_status));
  // owners = first points of their cells: counted per block, scanned, numbered (the strided map's kernels with one offset)
  SPCONV_CUDA_TRY(launch_chained(k_owner_count, dim3(nblk, 1), dim3(kBlock), stream, static_cast<const int32_t*>(point_slot),
                                 static_cast<const int32_t*>(owner), int(n), cnt));
  SPCONV_CUDA_TRY(launch_chained(k_scan_counts, dim3(1), dim3(1024), stream, static_cast<const int32_t*>(cnt), int64_t(nblk), excl, nblk, 1,
                                 static_cast<int64_t*>(nullptr), d_totals + 0, static_cast<int8_t*>(nullptr)));
  volatile int64_t* ready = host.p + totals_words;
  *ready = 0;
  host.writer = stream;
  host.write_pending = true;
  SPCONV_CUDA_TRY(launch_chained(k_report_totals, dim3(1), dim3(64), stream, static_cast<const int64_t*>(d_totals), int(totals_words), host.p));
  SPCONV_CUDA_TRY(cudaStreamSynchronize(stream));   // one wait: the caller needs the number of voxels
  host.write_pending = false;
  if (*ready != 1) return SPCONV_ERR_CUDA;
  if (uint32_t(host.p[2]) & kDevTableFull) return SPCONV_ERR_TABLE_FULL;
  const int64_t m = host.p[0];
  *n_voxels_host = m;
  if (m > capacity) return SPCONV_ERR_TOO_LARGE;
  if (m == 0) return SPCONV_OK;
  SPCONV_CUDA_TRY(launch_chained(k_owner_assign, dim3(nblk, 1), dim3(kBlock), stream, static_cast<const int32_t*>(point_slot),
                                 static_cast<const int32_t*>(owner), static_cast<const uint64_t*>(keys), int(n),
                                 static_cast<const int64_t*>(excl), slot_voxel, reinterpret_cast<int4*>(coords_out)));
  if (n_feat > 0) SPCONV_CUDA_TRY(cudaMemsetAsync(feats_out, 0, size_t(m) * n_feat * 4, stream));
  SPCONV_CUDA_TRY(cudaMemsetAsync(own_counts, 0, size_t(m) * 4, stream));
  const int cols = n_feat > 0 ? n_feat : 1;
  const int64_t acc_threads = n * cols;
  SPCONV_CUDA_TRY(launch_chained(k_vox_accumulate, dim3(unsigned((acc_threads + kBlock - 1) / kBlock)), dim3(kBlock), stream, points, int(n),
                                 point_stride, n_feat, static_cast<const int32_t*>(point_slot), static_cast<const int32_t*>(slot_voxel), feats_out,
                                 own_counts));
  if (n_feat > 0)
    SPCONV_CUDA_TRY(launch_chained(k_vox_normalize, dim3(unsigned((m * n_feat + kBlock - 1) / kBlock)), dim3(kBlock), stream, feats_out,
                                   static_cast<const int32_t*>(own_counts), m, n_feat));
  SPCONV_CUDA_TRY(cudaGetLastError());
  return SPCONV_OK;
}

}  // namespace spconv

// =============================================================================================
// Offset table without any allocation (see spconv_subm_offset_table_noalloc in the header).
//
// The hash table lives in this fixed array, which every GPU that loads the library keeps until the
// process exits.  Layout: kNoAllocSlots location-table slots of 16 bytes (key | row | unused) | one 256-byte block
// whose first word is the status word.
namespace spconv {
namespace {

constexpr uint32_t kNoAllocSlots = 2u * SPCONV_NOALLOC_MAX_VOXELS;   // power of two: at most half full
static_assert((kNoAllocSlots & (kNoAllocSlots - 1)) == 0, "slot count must be a power of two");
constexpr size_t kNoAllocBytes = size_t(kNoAllocSlots) * sizeof(LocSlot) + 256;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

// In host code the name g_noalloc_scratch is only a handle for the runtime, not an address a kernel
// could use; the device address is looked up once per device and cached here.
std::mutex g_noalloc_mu;
unsigned char* g_noalloc_ptr[64] = {nullptr};

// Same probing as k_subm_probe, without the per-block hit counts (they would need more scratch).
__global__ void k_subm_probe_only(const int4* __restrict__ coords, int n, int K, int dil, const LocSlot* __restrict__ table,
                                  uint32_t capmask, int32_t* __restrict__ nbr,
                                  const __grid_constant__ OffsetIndex index) {
  const int k = blockIdx.y;
  const int j = blockIdx.x * kBlock + threadIdx.x;
  if (j >= n) return;
  const int r = (K - 1) / 2;
  int ia, ib, ic;
  offset_index(index, k, K, ia, ib, ic);
  const int dx = dil * (ia - r), dy = dil * (ib - r), dz = dil * (ic - r);
  const int4 c = coords[j];
  const int x = c.y + dx, y = c.z + dy, z = c.w + dz;
  int v = -1;
  if ((dx | dy | dz) == 0) v = j;
  else if (in_range(x) && in_range(y) && in_range(z)) v = table_find(table, capmask, pack_key(c.x, x, y, z));
  nbr[size_t(k) * n + j] = v;
}

}  // namespace
}  // namespace spconv

extern "C" int spconv_subm_offset_table_noalloc(const int32_t* coords, int64_t n, int kernel_size, int dilation,
                                                int32_t* nbr_out, void* cuda_stream) {
  using namespace spconv;
  if (n < 0 || kernel_size < 1 || kernel_size > 16 || kernel_size % 2 == 0 || dilation < 1 || dilation > 4096)
    return SPCONV_ERR_INVALID_ARG;
  if (n > int64_t(SPCONV_NOALLOC_MAX_VOXELS)) return SPCONV_ERR_TOO_LARGE;
  if (n == 0) return SPCONV_OK;
  if (coords == nullptr || nbr_out == nullptr || (reinterpret_cast<uintptr_t>(coords) & 15u)) return SPCONV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

  // Set-up, once per device, with that device current: ask the runtime for the array's device address.
  int dev = -1;
  SPCONV_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SPCONV_ERR_INVALID_ARG;
  unsigned char* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_noalloc_mu);
    if (g_noalloc_ptr[dev] == nullptr) {
      void* p = nullptr;
      SPCONV_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
      g_noalloc_ptr[dev] = static_cast<unsigned char*>(p);
    }
    base = g_noalloc_ptr[dev];
  }
  LocSlot* table = reinterpret_cast<LocSlot*>(base);
  uint32_t* status = reinterpret_cast<uint32_t*>(base + size_t(kNoAllocSlots) * sizeof(LocSlot));

  // The array keeps whatever the previous call left: empty the slots this call will probe and the status word.
  const int K = kernel_size, kvol = K * K * K;
  const uint32_t cap = pow2_at_least(uint64_t(2) * n);
  const int nblk = int((n + kBlock - 1) / kBlock);
  SPCONV_CUDA_TRY(cudaMemsetAsync(table, 0xFF, size_t(cap) * sizeof(LocSlot), stream));
  SPCONV_CUDA_TRY(cudaMemsetAsync(status, 0, 256, stream));
  const int4* coords4 = reinterpret_cast<const int4*>(coords);
  k_insert<<<nblk, kBlock, 0, stream>>>(coords4, int(n), table, cap - 1, status, nullptr);
  k_subm_probe_only<<<dim3(nblk, kvol), kBlock, 0, stream>>>(coords4, int(n), K, dilation, table, cap - 1, nbr_out, make_offset_index(K));
  SPCONV_CUDA_TRY(cudaGetLastError());
  uint32_t st = 0;
  SPCONV_CUDA_TRY(cudaMemcpyAsync(&st, status, sizeof(st), cudaMemcpyDeviceToHost, stream));
  SPCONV_CUDA_TRY(cudaStreamSynchronize(stream));
  return device_status_to_error(st);
}

