/*
 * spconv_b200 -- sparse 3-D convolution over voxelised point clouds for NVIDIA B200 (sm_100a).
 *
 * C ABI of the library.  Two stages, as in the paper's workflow "create location table,
 * create offset table, compute result" (Sec. III-C):
 *
 *   1. spconv_build_kmap   location table (GPU hash table, Sec. III-C.1) + offset table and
 *                          per-offset (input, output) pairs (Sec. III-C.2); for strided
 *                          convolution also the output coordinates (Eq. 1-5, Sec. III-D).
 *   2. spconv_forward      out[o] = sum_k W_k^T in[nbr(o,k)]  (Algorithm 2, Sec. III-C.3).
 *
 * A kernel map depends only on the coordinates and (kernel, stride, dilation), never on the
 * features, channel counts or dtype: one handle serves any number of spconv_forward calls,
 * so layers that share coordinates share the map.
 *
 * Conventions
 *   - Every function returns an spconv_status_t (0 = success) unless stated otherwise.
 *     Nothing throws, aborts or traps; device-side problems are reported through a status
 *     word that the host reads.
 *   - Pointers are DEVICE pointers unless the parameter comment says "host".
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - The caller owns coords / feats / weights / out and must keep them alive until the
 *     stream has executed the call.  The library owns everything inside a kernel-map handle
 *     until spconv_kmap_destroy.
 *   - Coordinates are int32 rows (b, x, y, z) with 0 <= b,x,y,z <= 65534, all rows distinct.
 *   - Kernel offset numbering: k = kx*K^2 + ky*K + kz, kx,ky,kz in [0,K)  (Eq. 5).
 *   - Orientation is correlation: offset k of output cell q reads the input at position
 *     q*stride + dilation*(kx,ky,kz) - pad, pad = dilation*floor((K-1)/2).  (The offset-table
 *     figure of Sec. III-C.2 lists the (-1,-1) neighbour first and the (+1,+1) neighbour last.)
 *     With K == stride == 2 this is exactly Eq. 1-5: o = floor(p/s), k from p mod s.
 *   - Feature rows are row-major [n][C]; weights are row-major [K^3][Cin][Cout]; accumulation
 *     is fp32; the result is rounded once (nearest-even) to the feature dtype and OVERWRITES out
 *     (Algorithm 2 stores the sum; no bias, no activation).
 */
#ifndef SPCONV_B200_H_
#define SPCONV_B200_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct spconv_kmap spconv_kmap_t; /* opaque */

typedef enum {
  SPCONV_F32 = 0,
  SPCONV_F16 = 1,
  SPCONV_BF16 = 2
} spconv_dtype_t;

typedef enum {
  SPCONV_OK = 0,
  SPCONV_ERR_INVALID_ARG = 1,     /* null pointer, bad kernel/stride/dilation, unsupported channel count */
  SPCONV_ERR_COORD_RANGE = 2,     /* a coordinate component outside [0, 65534] */
  SPCONV_ERR_DUPLICATE_COORD = 3, /* two input rows with the same (b,x,y,z) */
  SPCONV_ERR_TABLE_FULL = 4,      /* hash probing exhausted the table (internal bound hit) */
  SPCONV_ERR_ALLOC = 5,           /* device or host allocation failed */
  SPCONV_ERR_CUDA = 6,            /* a CUDA runtime call failed */
  SPCONV_ERR_PIPE_TIMEOUT = 7,    /* a bounded wait inside a kernel ran out; out is undefined */
  SPCONV_ERR_SHAPE_MISMATCH = 8,  /* arguments inconsistent with the kernel map */
  SPCONV_ERR_TOO_LARGE = 9        /* size beyond a documented maximum */
} spconv_status_t;

/* Which forward kernel to run.  AUTO picks TCGEN05 when dtype is f16/bf16 and both channel
 * counts are in {16, 32, 64, 128}; everything else runs on the CUDA-core kernel. */
typedef enum {
  SPCONV_ALGO_AUTO = 0,
  SPCONV_ALGO_SIMT = 1,    /* fp32 FMA on CUDA cores (any dtype; the only exact-fp32 path) */
  SPCONV_ALGO_TCGEN05 = 2, /* implicit GEMM on 5th-gen tensor cores, fp32 accumulators in TMEM; a pipeline step takes as
                              many offsets of a tile as the shape allows (four for 16/32 channels in, two for 64 -> <=64) */
  SPCONV_ALGO_TCGEN05_SINGLE = 3 /* the same kernel with one offset per step (fixed grouping of one): for comparison */
} spconv_algo_t;

typedef struct {
  int32_t kernel_size, stride, dilation, submanifold;
  int32_t kvol;          /* K^3 */
  int32_t n_tiles;       /* 128-row output tiles of the tensor-core plan */
  int64_t n_in, n_out;
  int64_t total_pairs;   /* P = sum over offsets of the pair-list lengths */
  const int32_t* out_coords;   /* device [n_out][4]; submanifold: a copy of the input coords */
  const int32_t* nbr;          /* device [kvol][n_out]: input row feeding output row o via offset k, or -1.
                                  (The paper's offset table transposed so that consecutive threads touch
                                  consecutive ints.) */
  const int32_t* pair_in;      /* device [P]  input rows,  offset k occupying [offset_start[k], offset_start[k+1]) */
  const int32_t* pair_out;     /* device [P]  output rows, same positions */
  const int64_t* offset_start; /* HOST [kvol+1], owned by the handle */
  const int32_t* tile_rows;    /* device [n_tiles][128]: output row processed at each tile slot, -1 = padding */
  int64_t tile_blocks;         /* number of non-empty (tile, offset) blocks in the tensor-core plan */
  int32_t inverse;             /* 1 for a map from spconv_build_inverse_kmap */
  int32_t reserved;
} spconv_kmap_info_t;

/*
 * Build the kernel map of one layer.  [Sec. III-C.1-2; Sec. III-D; Eq. 1-5]
 *
 *   coords        device int32 [n][4] rows (b,x,y,z); 16-byte aligned; distinct; read only.
 *   n             number of input voxels, 0 <= n, n * K^3 <= 2,000,000,000.
 *   stride, dilation, kernel_size   >= 1 each.
 *   submanifold   1: outputs = inputs (same row numbering); requires stride == 1 and odd kernel_size.
 *                 0: regular convolution; output cells are all cells touched by at least one input,
 *                    unbounded above, o >= 0; their order is deterministic (run to run) but unspecified.
 *   cuda_stream   the work is enqueued here.  The call waits on the host until the device has reported the
 *                 sizes (n_out, P) and the error word, so it returns with the handle's sizes valid and every
 *                 error already detected.  For a submanifold map the last kernel, which writes the pair
 *                 lists, may still be running on cuda_stream at that moment: work enqueued on cuda_stream
 *                 afterwards is ordered behind it as usual; a consumer on another stream must first
 *                 synchronise with cuda_stream (an event), as for any stream-ordered producer.
 *   kmap_out      host; receives the handle on success, NULL on failure.
 *
 * Scratch memory (hash tables, counters) and the map's own arrays are taken from the device's default
 * stream-ordered pool (cudaMallocAsync); scratch is released before the call returns.  The first build
 * on a device raises that pool's release threshold so that later builds reuse the cached memory.
 * Errors: INVALID_ARG, TOO_LARGE, COORD_RANGE, DUPLICATE_COORD, TABLE_FULL, ALLOC, CUDA.
 */
int spconv_build_kmap(const int32_t* coords, int64_t n, int stride, int dilation, int kernel_size,
                      int submanifold, void* cuda_stream, spconv_kmap_t** kmap_out);

/*
 * spconv_build_kmap with the order of the tensor-core forward's row tiles chosen by the caller.  [Related work of
 * Sec. II-C: how (input, output) pairs are grouped into matrix products decides the padding they carry]
 *   SPCONV_ROWS_BY_OFFSET_SET  (what spconv_build_kmap does) rows sorted by the set of offsets through which they have
 *                              an input, so that a 128-row tile needs few offsets and its (tile, offset) blocks are
 *                              well filled; costs a sort per build.
 *   SPCONV_ROWS_AS_GIVEN       tile t holds output rows 128 t .. 128 t + 127: no sort (a shorter build), more and
 *                              emptier blocks (a slower forward), input rows of a tile close together when the caller's
 *                              row order is spatially coherent (e.g. Morton-sorted coordinates).
 * The kernel map itself (offset table, pairs, output coordinates) is the same for both; only the tile plan differs,
 * and with it the speed, never the result, of the tensor-core forward.
 */
typedef enum { SPCONV_ROWS_BY_OFFSET_SET = 0, SPCONV_ROWS_AS_GIVEN = 1 } spconv_row_order_t;
int spconv_build_kmap_ordered(const int32_t* coords, int64_t n, int stride, int dilation, int kernel_size, int submanifold,
                              int row_order, void* cuda_stream, spconv_kmap_t** kmap_out);

/*
 * Build the kernel map of an inverse (transposed) convolution, the up-sampling counterpart of a strided layer.
 * [Sec. III-E: location table over the index set after the convolution ("indices2"), then for every position of
 * the index set before it ("indices1") the related location in indices2 and its offset in the kernel]
 *
 *   fine_coords    device int32 [n_fine][4] rows (b,x,y,z): the positions BEFORE the strided convolution.  They are
 *                  the output rows of the inverse layer, numbered as given.  16-byte aligned, distinct (not
 *                  checked), read only.
 *   coarse_coords  device int32 [n_coarse][4]: the positions AFTER it (for instance the out_coords of the strided
 *                  layer's map, as a device pointer, no copy needed).  Row i is row i of the inverse layer's input
 *                  features.  16-byte aligned, distinct (checked), read only.
 *   stride, dilation, kernel_size   those of the strided convolution being inverted.
 * Fine position p is related to coarse cell q through offset kvec iff p = q*stride + dilation*kvec - pad,
 * pad = dilation*floor((K-1)/2): exactly the pairs of the strided convolution with the two roles swapped.  With
 * kernel_size == stride every fine position has one related cell (o = floor(p/s), offset p mod s, Eq. 1-5) and its
 * output row is the single product the paper describes; otherwise the related products are summed.  A fine
 * position none of whose related cells is in coarse_coords gets an all-zero output row.
 * The handle has n_in = n_coarse, n_out = n_fine, out_coords = a copy of fine_coords, and is used with
 * spconv_forward like any other: feats [n_coarse][cin], weights [K^3][cin][cout] (for the adjoint of a strided
 * layer pass that layer's W_k transposed), out [n_fine][cout].
 * Host wait, scratch memory, stream semantics and errors as for spconv_build_kmap.
 */
int spconv_build_inverse_kmap(const int32_t* fine_coords, int64_t n_fine, const int32_t* coarse_coords, int64_t n_coarse,
                              int stride, int dilation, int kernel_size, void* cuda_stream, spconv_kmap_t** kmap_out);

/*
 * Submanifold kernel map with the location table as a DENSE ARRAY over a stated grid instead of the hash table.
 * [Sec. III-C.1: "we can also use a three-dimensional array as location table", the variant the paper prefers
 * where the domain is confined; the printed createLCTKernel stores the row index at the cell's linear index, Eq. 6]
 *
 *   coords, n, dilation, cuda_stream, kmap_out   as for spconv_build_kmap with stride 1, submanifold 1.
 *   grid_shape    HOST int32[4] = (B, X, Y, Z): every input row must satisfy 0 <= b < B, 0 <= x < X, 0 <= y < Y,
 *                 0 <= z < Z (else SPCONV_ERR_COORD_RANGE); B*X*Y*Z <= SPCONV_DENSE_MAX_CELLS (else
 *                 SPCONV_ERR_TOO_LARGE): one int32 per cell is filled and probed per build (16 MiB at the limit).
 *   kernel_size   1 or 3.
 * The cell of (b, x, y, z) is ((b*X + x)*Y + y)*Z + z (the batch index is part of the address; Eq. 6 has none).
 * The resulting handle is indistinguishable from spconv_build_kmap's: same row numbering, offset table, pair
 * lists and tile plan, bit for bit.  Duplicates are detected as there.  Which of the two builds faster depends on
 * the grid's volume against the number of rows: the array costs its fill, the hash table its probing.
 * Errors: INVALID_ARG, TOO_LARGE, COORD_RANGE, DUPLICATE_COORD, ALLOC, CUDA.
 */
#define SPCONV_DENSE_MAX_CELLS 4194304
int spconv_build_kmap_dense(const int32_t* coords, int64_t n, const int32_t* grid_shape /* host [4] */, int dilation,
                            int kernel_size, void* cuda_stream, spconv_kmap_t** kmap_out);

/* Describe a kernel map.  `info` is host memory; the pointers inside stay valid until destroy. */
int spconv_kmap_info(const spconv_kmap_t* kmap, spconv_kmap_info_t* info);

/* Release a kernel map and all device memory it owns.  NULL is allowed.  The memory returns to the
 * stream-ordered pool in the order of the stream given to spconv_build_kmap (no device-wide
 * synchronisation): forwards that use the map on OTHER streams must have completed before this call,
 * and that stream must still exist. */
void spconv_kmap_destroy(spconv_kmap_t* kmap);

/*
 * Sparse convolution forward.  [Algorithm 2; Sec. III-C.3]
 *
 *   feats    device [n_in][cin]   of `dtype`, 16-byte aligned, read only.
 *   weights  device [K^3][cin][cout] of `dtype`, 16-byte aligned, read only.
 *   kmap     from spconv_build_kmap on the same device; not modified (safe to share between
 *            concurrent forwards on different streams).
 *   out      device [n_out][cout] of `dtype`, 16-byte aligned; every element is overwritten.
 *   cin,cout cin*sizeof(dtype) and cout*sizeof(dtype) must be multiples of 16 bytes.
 *
 * Asynchronous: the kernels are enqueued on cuda_stream and the call returns.  No allocation,
 * no synchronisation.  Each output row is produced by exactly one thread block from its list of
 * contributing rows, offsets in ascending order: no floating-point atomics, bit-reproducible.
 * Errors: INVALID_ARG, SHAPE_MISMATCH, CUDA.  A PIPE_TIMEOUT raised inside the tensor-core
 * kernel is reported by spconv_last_device_status.
 */
int spconv_forward(const void* feats, const void* weights, const spconv_kmap_t* kmap, void* out,
                   int cin, int cout, spconv_dtype_t dtype, void* cuda_stream);

/* Same, with the kernel chosen explicitly (tests and measurements).  TCGEN05 with an unsupported
 * dtype / channel count returns INVALID_ARG. */
int spconv_forward_algo(const void* feats, const void* weights, const spconv_kmap_t* kmap, void* out,
                        int cin, int cout, spconv_dtype_t dtype, spconv_algo_t algo, void* cuda_stream);

/* Synchronise `cuda_stream`, then return and clear the status word device kernels of this kernel
 * map wrote (SPCONV_OK or SPCONV_ERR_PIPE_TIMEOUT). */
int spconv_last_device_status(const spconv_kmap_t* kmap, void* cuda_stream);

/*
 * Whole layer on DEVICE buffers: build the kernel map and run the forward with one call.  [Sec. III-C: the two
 * stages of a layer, kernel map then convolution, back to back]
 *
 *   coords, n, stride, dilation, kernel_size, submanifold, cuda_stream   as for spconv_build_kmap
 *   feats, weights, cin, cout, dtype                                     as for spconv_forward
 *   out            device [out_capacity][cout]; rows [0, n_out) are written.
 *   out_capacity   rows `out` has room for.  Submanifold: must be >= n (else INVALID_ARG, nothing is enqueued).
 *                  Otherwise n_out is only known after the build: if it exceeds out_capacity the call returns
 *                  SPCONV_ERR_TOO_LARGE and builds no handle.
 *   kmap_out       host; receives the layer's kernel map (to be destroyed by the caller; it serves further
 *                  forwards over the same coordinates), NULL on failure.
 * For a submanifold layer the forward is enqueued behind the build's kernels BEFORE the host waits for the
 * build's report, so the device runs build and forward without a host round trip between them, and the pair lists,
 * which the forward does not read, are written on a second, library-owned stream (created once per host thread
 * and device, never destroyed) beside the tile plan; cuda_stream is made to wait for that stream behind the
 * forward, so everything the call enqueued is ordered before whatever the caller enqueues on cuda_stream next.
 * The results are those of spconv_build_kmap followed by spconv_forward.  Like spconv_build_kmap the call returns once the
 * sizes and the error word are known; the forward may still be running on cuda_stream then.  On an error
 * reported by the build, `out` may have been written with meaningless rows.
 * Errors: those of spconv_build_kmap and spconv_forward.
 */
int spconv_layer(const int32_t* coords, int64_t n, const void* feats, const void* weights, int stride, int dilation,
                 int kernel_size, int submanifold, int cin, int cout, spconv_dtype_t dtype, void* out,
                 int64_t out_capacity, void* cuda_stream, spconv_kmap_t** kmap_out);

/*
 * Whole layer from HOST buffers: copy coords / feats / weights to the device, build the kernel map,
 * run the forward, copy the result (and the output coordinates) back.  [Sec. III-A: the operator's
 * I/O is plain int and float arrays]
 *
 *   coords_host [n][4] int32, feats_host [n][cin], weights_host [K^3][cin][cout]   (host, read only)
 *   out_host         host; capacity out_capacity rows of cout elements
 *   out_coords_host  host or NULL; capacity out_capacity rows of 4 int32
 *   n_out_host       host; receives n_out.  If n_out > out_capacity nothing is copied back and the
 *                    call returns SPCONV_ERR_TOO_LARGE (n_out_host still set, so the caller can retry).
 * Synchronous with respect to cuda_stream.  Allocates and frees its device buffers itself.  Features and
 * weights are uploaded on a second, library-owned stream while the kernel map is built, and the output
 * coordinates come back while the forward runs (with pageable host buffers the copies simply serialise);
 * that stream and its events are created once per device, and concurrent calls on one device take turns.
 */
int spconv_layer_host(const int32_t* coords_host, int64_t n, const void* feats_host, const void* weights_host,
                      int stride, int dilation, int kernel_size, int submanifold,
                      int cin, int cout, spconv_dtype_t dtype,
                      void* out_host, int32_t* out_coords_host, int64_t out_capacity, int64_t* n_out_host,
                      void* cuda_stream);

/*
 * Submanifold offset table with NO allocation of any kind.  (The paper has no counterpart: its kernels
 * receive a location table that the caller has allocated.)
 *
 * Some callers may not allocate device memory at the point where they need the table: code that runs
 * inside another framework's execution step with all device memory already handed to that framework's
 * own allocator (an inference-engine plug-in's enqueue call is the typical case), or a control loop with
 * a memory budget fixed at start-up, where a cudaMalloc could fail, would stall the device, or is simply
 * forbidden.  spconv_build_kmap sizes and allocates its hash table per call; this entry point instead
 * probes a hash table kept in a fixed array inside the library (about 4 MiB, held by every GPU that loads
 * the library until the process exits) and writes straight into the caller's buffer.  It calls no
 * cudaMalloc / cudaFree, no stream-ordered allocator and no allocating library routine.  (The array is part
 * of the library's device code: the driver reserves it when it loads that code on a GPU, which with lazy
 * module loading can be as late as the first call that launches a kernel of the library there.)
 *
 *   coords      device int32 [n][4] rows (b,x,y,z), 16-byte aligned, distinct, read only.
 *   n           0 <= n <= SPCONV_NOALLOC_MAX_VOXELS; larger inputs return SPCONV_ERR_TOO_LARGE
 *               ("size beyond the documented maximum") and touch nothing.
 *   kernel_size odd, >= 1;  dilation >= 1  (stride is 1: outputs = inputs).
 *   nbr_out     device int32 [kernel_size^3][n], caller-owned; receives the same table as the `nbr`
 *               array of spconv_build_kmap(coords, n, 1, dilation, kernel_size, 1).
 *
 * The first call on a device looks up the device address of the fixed array (a one-time set-up done with
 * that device current); make that first call before starting any stream capture.  The call enqueues
 * its work on cuda_stream and synchronises that stream before returning, because it reports
 * COORD_RANGE / DUPLICATE_COORD.  All calls on one GPU share the one array, which keeps the previous call's
 * contents: each call first empties the slots and the status word it will use, and two calls that overlap
 * on the same GPU (from different streams or threads) race on it and must be serialised by the caller.
 * Errors: INVALID_ARG, TOO_LARGE, COORD_RANGE, DUPLICATE_COORD, TABLE_FULL, CUDA.
 */
#define SPCONV_NOALLOC_MAX_VOXELS 131072
int spconv_subm_offset_table_noalloc(const int32_t* coords, int64_t n, int kernel_size, int dilation,
                                     int32_t* nbr_out, void* cuda_stream);

/*
 * Voxelise raw points into the sparse tensor the operators take.  [Sec. II-A: the point cloud is "partitioned into
 * voxel grids" and becomes an index list (m, x, y, z) plus a feature array; the paper assumes this step upstream]
 *
 *   points        device float32 [n][point_stride]: columns 0-2 are x, y, z (any unit), columns 3 .. 3 + n_feat - 1 the
 *                 point's features; further columns are ignored.  Read only.
 *   n_feat        >= 0 feature columns;  batch_index  0 .. 65534, written into column 0 of every output coordinate.
 *   origin, voxel_size, grid_shape   HOST float[3], float[3] (> 0), int32[3] (1 .. 65535): the cell of a point is
 *                 floor((p - origin) / voxel_size) per axis, evaluated in float32 exactly in that order; points whose
 *                 cell is outside [0, grid_shape) are dropped.
 *   coords_out    device int32 [capacity][4], 16-byte aligned: one row (batch_index, x, y, z) per occupied cell, in
 *                 the order of the cells' first points (lowest point index first): the same on every run.
 *   feats_out     device float32 [capacity][n_feat]: mean of the features of the cell's points (fp32 sums through
 *                 atomic adds: the last bits may differ from run to run).  May be NULL when n_feat == 0.
 *   counts_out    device int32 [capacity] or NULL: points per cell.
 *   n_voxels_host HOST; receives the number of occupied cells.  If it exceeds `capacity` nothing is written to the
 *                 outputs and the call returns SPCONV_ERR_TOO_LARGE (n_voxels_host still set, so the caller can retry).
 * The call synchronises cuda_stream once (the caller has to learn the row count); the accumulation that follows is
 * asynchronous.  coords_out can be passed to spconv_build_kmap as it is (rows are distinct and in range).
 * Scratch memory comes from the device's stream-ordered pool.  Errors: INVALID_ARG, TOO_LARGE, TABLE_FULL, ALLOC, CUDA.
 */
int spconv_voxelize(const float* points, int64_t n, int point_stride, int n_feat, int batch_index, const float* origin /* host [3] */,
                    const float* voxel_size /* host [3] */, const int32_t* grid_shape /* host [3] */, int32_t* coords_out,
                    float* feats_out, int32_t* counts_out, int64_t capacity, int64_t* n_voxels_host /* host */, void* cuda_stream);

/*
 * Diagnostics: copy the 16 status words that device kernels of this kernel map write to host memory `out16`
 * (synchronous copy).  Word 0: status bits (8 = a bounded wait of the tensor-core forward ran out); word 1: code of
 * the first wait that gave up (role << 24 | step, top bit set); word 2: its CTA + 1.  Cleared by the next build of a
 * tile plan and, word 0 only, by spconv_last_device_status.
 */
int spconv_kmap_status_words(const spconv_kmap_t* kmap, uint32_t* out16 /* host */);

/*
 * Test hooks.  Not for production use: they exist so that tests can reach the failure paths that no valid input
 * reaches, without faulting or hanging the device.  Process-wide, take effect for calls made afterwards; value 0
 * restores the normal behaviour.
 *   SPCONV_HOOK_TABLE_SLOTS         force the location table to pow2(value) slots, whatever the input: with fewer
 *                                   slots than rows the bounded probe sequence runs out and the build returns
 *                                   SPCONV_ERR_TABLE_FULL.
 *   SPCONV_HOOK_PIPE_WAIT_LIMIT_US  shorten the time bound of every wait inside the tensor-core forward to `value`
 *                                   microseconds and withhold the weights of the first step of CTA 0, so that one
 *                                   wait runs out: the kernel gives up by itself and the status word reports
 *                                   SPCONV_ERR_PIPE_TIMEOUT.
 * Two more switches are environment variables read once per process: SPCONV_TC_MAX_CTAS=<n> caps the grid of the
 * tensor-core forward (small inputs then exercise many tiles per CTA and several rounds), and
 * SPCONV_KMAP_LIBRARY_SORT=1 sorts the tile plan's rows with the CUDA library's radix sort instead of the fused
 * cooperative launch (the path very large maps take).
 */
typedef enum { SPCONV_HOOK_TABLE_SLOTS = 1, SPCONV_HOOK_PIPE_WAIT_LIMIT_US = 2 } spconv_test_hook_t;
int spconv_test_hook(int which, long long value);

/* Static, never-NULL description of a status code. */
const char* spconv_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* SPCONV_B200_H_ */
