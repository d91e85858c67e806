// C ABI of spconv_b200: argument checking and dispatch.  Every step of the path runs in the kernels of
// kmap.cu / forward_simt.cu / forward_tc.cu.
#include <cstring>

#include <initializer_list>
#include <mutex>

#include "common.cuh"

using namespace spconv;

extern "C" {

const char* spconv_strerror(int status) {
  switch (status) {
    case SPCONV_OK: return "ok";
    case SPCONV_ERR_INVALID_ARG: return "invalid argument";
    case SPCONV_ERR_COORD_RANGE: return "coordinate outside [0, 65534]";
    case SPCONV_ERR_DUPLICATE_COORD: return "duplicate input coordinate";
    case SPCONV_ERR_TABLE_FULL: return "hash table full";
    case SPCONV_ERR_ALLOC: return "allocation failed";
    case SPCONV_ERR_CUDA: return "CUDA runtime error";
    case SPCONV_ERR_PIPE_TIMEOUT: return "bounded wait inside a kernel ran out";
    case SPCONV_ERR_SHAPE_MISMATCH: return "arguments do not match the kernel map";
    case SPCONV_ERR_TOO_LARGE: return "size beyond the documented maximum";
  }
  return "unknown status";
}

namespace {
// spconv_build_kmap with build_kmap_impl's before_wait hook (used by spconv_layer).
int spconv_build_kmap_hooked(const int32_t* coords, int64_t n, int stride, int dilation, int kernel_size, int submanifold,
                             void* cuda_stream, spconv_kmap_t** kmap_out, const std::function<int(spconv_kmap*)>* before_wait,
                             int rows_as_given = 0) {
  if (kmap_out == nullptr) return SPCONV_ERR_INVALID_ARG;
  *kmap_out = nullptr;
  if (n < 0 || stride < 1 || dilation < 1 || kernel_size < 1) return SPCONV_ERR_INVALID_ARG;
  if (kernel_size > 16 || stride > 4096 || dilation > 4096) return SPCONV_ERR_INVALID_ARG;
  if (n > 0 && coords == nullptr) return SPCONV_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(coords) & 15u) return SPCONV_ERR_INVALID_ARG;
  submanifold = submanifold ? 1 : 0;
  if (submanifold && (stride != 1 || kernel_size % 2 == 0)) return SPCONV_ERR_INVALID_ARG;
  const int64_t kvol = int64_t(kernel_size) * kernel_size * kernel_size;
  if (n * kvol > int64_t(2000000000)) return SPCONV_ERR_TOO_LARGE;
  return build_kmap_impl(coords, n, stride, dilation, kernel_size, submanifold, static_cast<cudaStream_t>(cuda_stream), kmap_out, before_wait,
                         nullptr, 0, nullptr, rows_as_given);
}
}  // namespace

int spconv_build_kmap(const int32_t* coords, int64_t n, int stride, int dilation, int kernel_size, int submanifold,
                      void* cuda_stream, spconv_kmap_t** kmap_out) {
  return spconv_build_kmap_hooked(coords, n, stride, dilation, kernel_size, submanifold, cuda_stream, kmap_out, nullptr);
}

int spconv_build_kmap_ordered(const int32_t* coords, int64_t n, int stride, int dilation, int kernel_size, int submanifold,
                              int row_order, void* cuda_stream, spconv_kmap_t** kmap_out) {
  if (row_order != SPCONV_ROWS_BY_OFFSET_SET && row_order != SPCONV_ROWS_AS_GIVEN) {
    if (kmap_out != nullptr) *kmap_out = nullptr;
    return SPCONV_ERR_INVALID_ARG;
  }
  return spconv_build_kmap_hooked(coords, n, stride, dilation, kernel_size, submanifold, cuda_stream, kmap_out, nullptr,
                                  row_order == SPCONV_ROWS_AS_GIVEN ? 1 : 0);
}

int spconv_build_inverse_kmap(const int32_t* fine_coords, int64_t n_fine, const int32_t* coarse_coords, int64_t n_coarse,
                              int stride, int dilation, int kernel_size, void* cuda_stream, spconv_kmap_t** kmap_out) {
  if (kmap_out == nullptr) return SPCONV_ERR_INVALID_ARG;
  *kmap_out = nullptr;
  if (n_fine < 0 || n_coarse < 0 || stride < 1 || dilation < 1 || kernel_size < 1) return SPCONV_ERR_INVALID_ARG;
  if (kernel_size > 16 || stride > 4096 || dilation > 4096) return SPCONV_ERR_INVALID_ARG;
  if ((n_fine > 0 && fine_coords == nullptr) || (n_coarse > 0 && coarse_coords == nullptr)) return SPCONV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(fine_coords) & 15u) || (reinterpret_cast<uintptr_t>(coarse_coords) & 15u)) return SPCONV_ERR_INVALID_ARG;
  const int64_t kvol = int64_t(kernel_size) * kernel_size * kernel_size;
  if (n_fine * kvol > int64_t(2000000000) || n_coarse > int64_t(2000000000)) return SPCONV_ERR_TOO_LARGE;
  // a never-null query pointer selects the inverse path even when there are no fine rows
  static const int32_t none[4] = {0, 0, 0, 0};
  return build_kmap_impl(coarse_coords, n_coarse, stride, dilation, kernel_size, 0, static_cast<cudaStream_t>(cuda_stream), kmap_out,
                         nullptr, fine_coords != nullptr ? fine_coords : none, n_fine);
}

int spconv_build_kmap_dense(const int32_t* coords, int64_t n, const int32_t* grid_shape, int dilation, int kernel_size,
                            void* cuda_stream, spconv_kmap_t** kmap_out) {
  if (kmap_out == nullptr) return SPCONV_ERR_INVALID_ARG;
  *kmap_out = nullptr;
  if (n < 0 || dilation < 1 || dilation > 4096 || grid_shape == nullptr) return SPCONV_ERR_INVALID_ARG;
  if (kernel_size != 1 && kernel_size != 3) return SPCONV_ERR_INVALID_ARG;
  if (n > 0 && coords == nullptr) return SPCONV_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(coords) & 15u) return SPCONV_ERR_INVALID_ARG;
  int grid[4];
  int64_t cells = 1;
  for (int a = 0; a < 4; ++a) {
    if (grid_shape[a] < 1 || grid_shape[a] > 65535) return SPCONV_ERR_INVALID_ARG;
    grid[a] = grid_shape[a];
    cells *= grid_shape[a];
    if (cells > int64_t(SPCONV_DENSE_MAX_CELLS)) return SPCONV_ERR_TOO_LARGE;
  }
  if (n * int64_t(kernel_size) * kernel_size * kernel_size > int64_t(2000000000)) return SPCONV_ERR_TOO_LARGE;
  return build_kmap_impl(coords, n, 1, dilation, kernel_size, 1, static_cast<cudaStream_t>(cuda_stream), kmap_out, nullptr, nullptr, 0, grid);
}

int spconv_kmap_info(const spconv_kmap_t* km, spconv_kmap_info_t* info) {
  if (km == nullptr || info == nullptr) return SPCONV_ERR_INVALID_ARG;
  std::memset(info, 0, sizeof(*info));
  info->kernel_size = km->kernel; info->stride = km->stride; info->dilation = km->dilation;
  info->submanifold = km->submanifold; info->kvol = km->kvol; info->n_tiles = km->n_tiles;
  info->n_in = km->n_in; info->n_out = km->n_out; info->total_pairs = km->total_pairs;
  info->out_coords = km->d.out_coords; info->nbr = km->d.nbr;
  info->pair_in = km->d.pair_in; info->pair_out = km->d.pair_out;
  info->offset_start = km->offset_start.data();
  info->tile_rows = km->d.tile_rows; info->tile_blocks = km->tile_blocks;
  info->inverse = km->inverse;
  return SPCONV_OK;
}

void spconv_kmap_destroy(spconv_kmap_t* km) { destroy_kmap_impl(km); }

namespace {
// Argument checks and kernel choice of every forward entry point.  strict_order: see forward_tc().
int forward_checked(const void* feats, const void* weights, const spconv_kmap_t* km, void* out, int cin, int cout,
                    spconv_dtype_t dtype, spconv_algo_t algo, void* cuda_stream, bool strict_order) {
  if (km == nullptr) return SPCONV_ERR_INVALID_ARG;
  if (dtype != SPCONV_F32 && dtype != SPCONV_F16 && dtype != SPCONV_BF16) return SPCONV_ERR_INVALID_ARG;
  if (cin < 1 || cout < 1 || cin > 4096 || cout > 4096) return SPCONV_ERR_INVALID_ARG;
  const int esz = dtype_size(dtype);
  if ((cin * esz) % 16 != 0 || (cout * esz) % 16 != 0) return SPCONV_ERR_INVALID_ARG;
  if (weights == nullptr || (reinterpret_cast<uintptr_t>(weights) & 15u)) return SPCONV_ERR_INVALID_ARG;
  if (km->n_in > 0 && (feats == nullptr || (reinterpret_cast<uintptr_t>(feats) & 15u))) return SPCONV_ERR_INVALID_ARG;
  if (km->n_out > 0 && (out == nullptr || (reinterpret_cast<uintptr_t>(out) & 15u))) return SPCONV_ERR_INVALID_ARG;
  int dev = -1;
  SPCONV_CUDA_TRY(cudaGetDevice(&dev));
  if (dev != km->device) return SPCONV_ERR_SHAPE_MISMATCH;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  switch (algo) {
    case SPCONV_ALGO_AUTO:
      if (forward_tc_supported(cin, cout, dtype) && km->kvol <= 32)
        return forward_tc(feats, weights, km, out, cin, cout, dtype, stream, strict_order);
      return forward_simt(feats, weights, km, out, cin, cout, dtype, stream);
    case SPCONV_ALGO_SIMT:
      return forward_simt(feats, weights, km, out, cin, cout, dtype, stream);
    case SPCONV_ALGO_TCGEN05:
      return forward_tc(feats, weights, km, out, cin, cout, dtype, stream, strict_order);
    case SPCONV_ALGO_TCGEN05_SINGLE:
      return forward_tc(feats, weights, km, out, cin, cout, dtype, stream, strict_order, true);
  }
  return SPCONV_ERR_INVALID_ARG;
}
}  // namespace

int spconv_forward_algo(const void* feats, const void* weights, const spconv_kmap_t* km, void* out, int cin, int cout,
                        spconv_dtype_t dtype, spconv_algo_t algo, void* cuda_stream) {
  return forward_checked(feats, weights, km, out, cin, cout, dtype, algo, cuda_stream, false);
}

int spconv_layer(const int32_t* coords, int64_t n, const void* feats, const void* weights, int stride, int dilation,
                 int kernel_size, int submanifold, int cin, int cout, spconv_dtype_t dtype, void* out, int64_t out_capacity,
                 void* cuda_stream, spconv_kmap_t** kmap_out) {
  if (kmap_out == nullptr) return SPCONV_ERR_INVALID_ARG;
  *kmap_out = nullptr;
  if (out_capacity < 0 || (submanifold && out_capacity < n)) return SPCONV_ERR_INVALID_ARG;
  spconv_kmap_t* km = nullptr;
  if (submanifold) {
    // n_out = n is known up front: the forward is enqueued right behind the build's kernels, before the host waits
    // for the build's report, so that no host round trip separates the two on the device.
    int forward_status = SPCONV_OK;
    bool forward_enqueued = false;
    const std::function<int(spconv_kmap*)> enqueue_forward = [&](spconv_kmap* building) -> int {
      forward_status = forward_checked(feats, weights, building, out, cin, cout, dtype, SPCONV_ALGO_AUTO, cuda_stream, true);
      forward_enqueued = true;
      return forward_status;
    };
    const int e = spconv_build_kmap_hooked(coords, n, stride, dilation, kernel_size, submanifold, cuda_stream, &km, &enqueue_forward);
    if (e != SPCONV_OK) return e;
    if (!forward_enqueued) {   // (an empty map never reaches the hook)
      const int f = forward_checked(feats, weights, km, out, cin, cout, dtype, SPCONV_ALGO_AUTO, cuda_stream, false);
      if (f != SPCONV_OK) { spconv_kmap_destroy(km); return f; }
    }
  } else {
    const int e = spconv_build_kmap(coords, n, stride, dilation, kernel_size, submanifold, cuda_stream, &km);
    if (e != SPCONV_OK) return e;
    if (km->n_out > out_capacity) { spconv_kmap_destroy(km); return SPCONV_ERR_TOO_LARGE; }
    const int f = forward_checked(feats, weights, km, out, cin, cout, dtype, SPCONV_ALGO_AUTO, cuda_stream, false);
    if (f != SPCONV_OK) { spconv_kmap_destroy(km); return f; }
  }
  *kmap_out = km;
  return SPCONV_OK;
}

int spconv_forward(const void* feats, const void* weights, const spconv_kmap_t* km, void* out, int cin, int cout,
                   spconv_dtype_t dtype, void* cuda_stream) {
  return spconv_forward_algo(feats, weights, km, out, cin, cout, dtype, SPCONV_ALGO_AUTO, cuda_stream);
}

int spconv_last_device_status(const spconv_kmap_t* km, void* cuda_stream) {
  if (km == nullptr) return SPCONV_ERR_INVALID_ARG;
  if (km->d.status == nullptr) return SPCONV_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint32_t st = 0;
  SPCONV_CUDA_TRY(cudaMemcpyAsync(&st, km->d.status, sizeof(st), cudaMemcpyDeviceToHost, stream));
  SPCONV_CUDA_TRY(cudaMemsetAsync(km->d.status, 0, sizeof(st), stream));
  SPCONV_CUDA_TRY(cudaStreamSynchronize(stream));
  return (st & kDevPipeTimeout) ? SPCONV_ERR_PIPE_TIMEOUT : SPCONV_OK;
}

int spconv_layer_host(const int32_t* coords_host, int64_t n, const void* feats_host, const void* weights_host, int stride,
                      int dilation, int kernel_size, int submanifold, int cin, int cout, spconv_dtype_t dtype, void* out_host,
                      int32_t* out_coords_host, int64_t out_capacity, int64_t* n_out_host, void* cuda_stream) {
  if (n_out_host == nullptr || n < 0 || kernel_size < 1 || kernel_size > 16 || cin < 1 || cout < 1) return SPCONV_ERR_INVALID_ARG;
  if (dtype != SPCONV_F32 && dtype != SPCONV_F16 && dtype != SPCONV_BF16) return SPCONV_ERR_INVALID_ARG;
  if (n > 0 && (coords_host == nullptr || feats_host == nullptr)) return SPCONV_ERR_INVALID_ARG;
  if (weights_host == nullptr) return SPCONV_ERR_INVALID_ARG;
  *n_out_host = 0;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t esz = size_t(dtype_size(dtype));
  const size_t kvol = size_t(kernel_size) * kernel_size * kernel_size;
  const size_t b_coords = size_t(n) * 16, b_feats = size_t(n) * cin * esz, b_w = kvol * cin * cout * esz;
  auto up = [](size_t b) { return (b + 255) & ~size_t(255); };
  struct Dev { void* p = nullptr; cudaStream_t s; ~Dev() { if (p) cudaFreeAsync(p, s); } };
  Dev in; in.s = stream;
  SPCONV_CUDA_TRY(cudaMallocAsync(&in.p, up(b_coords) + up(b_feats) + up(b_w) + 256, stream));
  char* base = static_cast<char*>(in.p);
  int32_t* d_coords = reinterpret_cast<int32_t*>(base);
  void* d_feats = base + up(b_coords);
  void* d_w = base + up(b_coords) + up(b_feats);
  // The features and weights travel on a second stream while the first builds the kernel map from the
  // coordinates (the build needs nothing else), and the output coordinates travel back while the forward runs.
  // (The second stream and its events are created once per device and kept; calls on one device take turns.)
  struct SideSet { cudaStream_t s = nullptr; cudaEvent_t start = nullptr, inputs = nullptr, map_ready = nullptr, coords_back = nullptr; };
  static SideSet side_sets[64];
  static std::mutex side_mutex[64];
  int device = 0;
  SPCONV_CUDA_TRY(cudaGetDevice(&device));
  if (device < 0 || device >= 64) return SPCONV_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> side_lock(side_mutex[device]);
  SideSet& side = side_sets[device];
  if (side.s == nullptr) {
    SPCONV_CUDA_TRY(cudaStreamCreateWithFlags(&side.s, cudaStreamNonBlocking));
    for (cudaEvent_t* e : {&side.start, &side.inputs, &side.map_ready, &side.coords_back})
      SPCONV_CUDA_TRY(cudaEventCreateWithFlags(e, cudaEventDisableTiming));
  }
  // nothing of this call may still use the buffers released on the way out
  struct SideIdle { cudaStream_t s; ~SideIdle() { cudaStreamSynchronize(s); (void)cudaGetLastError(); } } side_idle{side.s};
  SPCONV_CUDA_TRY(cudaEventRecord(side.start, stream));          // the allocation above is stream-ordered
  SPCONV_CUDA_TRY(cudaStreamWaitEvent(side.s, side.start, 0));
  if (n > 0) {
    SPCONV_CUDA_TRY(cudaMemcpyAsync(d_coords, coords_host, b_coords, cudaMemcpyHostToDevice, stream));
    SPCONV_CUDA_TRY(cudaMemcpyAsync(d_feats, feats_host, b_feats, cudaMemcpyHostToDevice, side.s));
  }
  SPCONV_CUDA_TRY(cudaMemcpyAsync(d_w, weights_host, b_w, cudaMemcpyHostToDevice, side.s));
  SPCONV_CUDA_TRY(cudaEventRecord(side.inputs, side.s));
  spconv_kmap_t* km = nullptr;
  int st = spconv_build_kmap(d_coords, n, stride, dilation, kernel_size, submanifold, stream, &km);
  if (st != SPCONV_OK) return st;
  struct KmGuard { spconv_kmap_t* km; ~KmGuard() { spconv_kmap_destroy(km); } } kg{km};
  // (destroyed first: the second stream may still be reading the map's output coordinates on an error path)
  struct SideDone { cudaStream_t s; ~SideDone() { cudaStreamSynchronize(s); (void)cudaGetLastError(); } } side_done{side.s};
  *n_out_host = km->n_out;
  if (km->n_out > out_capacity) return SPCONV_ERR_TOO_LARGE;
  if (km->n_out == 0) return SPCONV_OK;
  if (out_host == nullptr) return SPCONV_ERR_INVALID_ARG;
  Dev outb; outb.s = stream;
  const size_t b_out = size_t(km->n_out) * cout * esz;
  SPCONV_CUDA_TRY(cudaMallocAsync(&outb.p, up(b_out), stream));
  if (out_coords_host != nullptr) {
    SPCONV_CUDA_TRY(cudaEventRecord(side.map_ready, stream));
    SPCONV_CUDA_TRY(cudaStreamWaitEvent(side.s, side.map_ready, 0));
    SPCONV_CUDA_TRY(cudaMemcpyAsync(out_coords_host, km->d.out_coords, size_t(km->n_out) * 16, cudaMemcpyDeviceToHost, side.s));
  }
  SPCONV_CUDA_TRY(cudaEventRecord(side.coords_back, side.s));
  SPCONV_CUDA_TRY(cudaStreamWaitEvent(stream, side.inputs, 0));
  st = spconv_forward(d_feats, d_w, km, outb.p, cin, cout, dtype, stream);
  if (st != SPCONV_OK) return st;
  SPCONV_CUDA_TRY(cudaMemcpyAsync(out_host, outb.p, b_out, cudaMemcpyDeviceToHost, stream));
  SPCONV_CUDA_TRY(cudaStreamWaitEvent(stream, side.coords_back, 0));   // the caller's stream ends after everything of this call
  return spconv_last_device_status(km, stream);
}

int spconv_voxelize(const float* points, int64_t n, int point_stride, int n_feat, int batch_index, const float* origin,
                    const float* voxel_size, const int32_t* grid_shape, int32_t* coords_out, float* feats_out, int32_t* counts_out,
                    int64_t capacity, int64_t* n_voxels_host, void* cuda_stream) {
  if (n_voxels_host == nullptr) return SPCONV_ERR_INVALID_ARG;
  *n_voxels_host = 0;
  if (n < 0 || n > int64_t(1000000000) || n_feat < 0 || point_stride < 3 + n_feat || point_stride > 1024 || capacity < 0) return SPCONV_ERR_INVALID_ARG;
  if (origin == nullptr || voxel_size == nullptr || grid_shape == nullptr) return SPCONV_ERR_INVALID_ARG;
  if (batch_index < 0 || batch_index > kMaxCoord) return SPCONV_ERR_INVALID_ARG;
  for (int a = 0; a < 3; ++a)
    if (!(voxel_size[a] > 0.f) || grid_shape[a] < 1 || grid_shape[a] > kMaxCoord + 1) return SPCONV_ERR_INVALID_ARG;
  if (n > 0 && (points == nullptr || coords_out == nullptr || (n_feat > 0 && feats_out == nullptr))) return SPCONV_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(coords_out) & 15u) return SPCONV_ERR_INVALID_ARG;
  return voxelize_impl(points, n, point_stride, n_feat, batch_index, origin, voxel_size, grid_shape, coords_out, feats_out, counts_out,
                       capacity, n_voxels_host, static_cast<cudaStream_t>(cuda_stream));
}

int spconv_kmap_status_words(const spconv_kmap_t* km, uint32_t* out16) {
  if (km == nullptr || out16 == nullptr) return SPCONV_ERR_INVALID_ARG;
  if (km->d.status == nullptr) { std::memset(out16, 0, 64); return SPCONV_OK; }
  return cudaMemcpy(out16, km->d.status, 64, cudaMemcpyDeviceToHost) == cudaSuccess ? SPCONV_OK : SPCONV_ERR_CUDA;
}

int spconv_test_hook(int which, long long value) {
  switch (which) {
    case SPCONV_HOOK_TABLE_SLOTS: set_kmap_test_table_slots(value); return SPCONV_OK;
    case SPCONV_HOOK_PIPE_WAIT_LIMIT_US: set_forward_tc_test_wait_limit_us(value); return SPCONV_OK;
  }
  return SPCONV_ERR_INVALID_ARG;
}

#ifdef SPCONV_TC_PROFILE
// Development builds only: per-CTA timeline buffer of the tensor-core forward (see forward_tc.cu).
void spconv_internal_set_timeline(void* device_buffer) { set_forward_tc_timeline(static_cast<unsigned long long*>(device_buffer)); }
#endif

}  // extern "C"
