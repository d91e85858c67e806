// CUDA-core forward: output-stationary evaluation of Algorithm 2 with true fp32 FMAs.
//
// The production path for fp32 features (a single-pass tensor-core product would round the operands
// to 10 mantissa bits) and the fallback for channel counts the tensor-core kernel does not take.
// Like the paper's computeConv kernel (Sec. III-C.3) it stages the weights of the current offset in
// shared memory, but a block covers all output channels of its rows, so a gathered row is read once per
// offset instead of once per output channel.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <mutex>

#include "common.cuh"

namespace spconv {
namespace {

constexpr int kRows = 32;      // output rows per block
constexpr int kThreads = 256;  // 8 threads per row
constexpr int kCinChunk = 64;
constexpr int kCoutChunk = 128;

template <class T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <class T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <class T>
__global__ void __launch_bounds__(kThreads)
k_forward_simt(const T* __restrict__ feats, const T* __restrict__ w, const int32_t* __restrict__ nbr, int64_t n_out,
               int kvol, int cin, int cout, T* __restrict__ out) {
  __shared__ float xs[kRows][kCinChunk + 1];
  __shared__ float ws[kCinChunk][kCoutChunk];
  __shared__ int sidx[kRows][33];     // offset-table entries of the block's rows for 32 offsets at a time
  __shared__ unsigned active_offsets; // offsets of the current 32 that any row of the block has
  const int tid = threadIdx.x, row = tid >> 3, l8 = tid & 7;
  const int64_t grow = int64_t(blockIdx.x) * kRows + row;

  for (int co0 = 0; co0 < cout; co0 += kCoutChunk) {
    const int cw = min(kCoutChunk, cout - co0);
    float acc[kCoutChunk / 8];
#pragma unroll
    for (int m = 0; m < kCoutChunk / 8; ++m) acc[m] = 0.f;
    for (int k0 = 0; k0 < kvol; k0 += 32) {
      // One memory round trip fetches the table entries of 32 offsets (the eight threads of a row take four
      // each); offsets no row of the block has are then skipped without touching memory or a barrier.
      if (tid == 0) active_offsets = 0u;
      __syncthreads();
      unsigned mine = 0u;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int kk = l8 + 8 * j, k = k0 + kk;
        const int idx = (k < kvol && grow < n_out) ? nbr[size_t(k) * n_out + grow] : -1;
        sidx[row][kk] = idx;
        if (idx >= 0) mine |= 1u << kk;
      }
      if (mine) atomicOr(&active_offsets, mine);
      __syncthreads();
      unsigned todo = active_offsets;
      while (todo) {
        const int kk = __ffs(todo) - 1, k = k0 + kk;
        todo &= todo - 1u;
        for (int ci0 = 0; ci0 < cin; ci0 += kCinChunk) {
          const int cc = min(kCinChunk, cin - ci0);
          if (ci0) __syncthreads();
          for (int e = tid; e < cc * cw; e += kThreads) {
            const int c = e / cw, o = e - c * cw;
            ws[c][o] = to_f32<T>(w[(size_t(k) * cin + ci0 + c) * cout + co0 + o]);
          }
          for (int e = tid; e < kRows * cc; e += kThreads) {
            const int r = e / cc, c = e - r * cc;
            const int ir = sidx[r][kk];
            xs[r][c] = ir >= 0 ? to_f32<T>(feats[size_t(ir) * cin + ci0 + c]) : 0.f;
          }
          __syncthreads();
          for (int c = 0; c < cc; ++c) {
            const float xv = xs[row][c];
#pragma unroll
            for (int m = 0; m < kCoutChunk / 8; ++m) {
              const int o = l8 + 8 * m;
              if (o < cw) acc[m] = fmaf(xv, ws[c][o], acc[m]);
            }
          }
        }
        __syncthreads();  // xs / ws are rewritten by the next offset
      }
      __syncthreads();    // sidx and active_offsets are rewritten by the next 32 offsets
    }
    if (grow < n_out) {
#pragma unroll
      for (int m = 0; m < kCoutChunk / 8; ++m) {
        const int o = l8 + 8 * m;
        if (o < cw) out[size_t(grow) * cout + co0 + o] = from_f32<T>(acc[m]);
      }
    }
    __syncthreads();
  }
}


// fp32 fast path: all weights in shared memory, four output channels per thread, rows straight from global memory.
// The weights of every offset are staged once per block as they lie in memory ([K^3][Cin][Cout]); cout / 4
// neighbouring threads share an output row and each keeps four of its channels in registers; a thread fetches the
// row's offset-table entries 32 at a time (one round trip), then walks the offsets in ascending order and, where
// the row has an input, reads that input row with 16-byte loads (the threads of a row read the same addresses: one
// request) and multiplies it with 16-byte reads of the offset's weights.  Rows are independent, so apart from the
// one barrier behind the staging nothing waits for anything but its own loads; the result leaves as one 16-byte
// store per thread.  Taken when the weights fit (kvol * cin * cout * 4 bytes within the SM's shared memory).
constexpr int kRowsThreads = 256;
__global__ void __launch_bounds__(kRowsThreads)
k_forward_rows_f32(const float* __restrict__ feats, const float* __restrict__ w, const int32_t* __restrict__ nbr, int64_t n_out,
                   int kvol, int cin, int cout, float* __restrict__ out) {
  extern __shared__ __align__(16) float wsm[];   // [kvol][cin][cout]
  const int tid = threadIdx.x;
  const int tpr = cout >> 2;                       // threads per row
  const int rows_per_block = kRowsThreads / tpr;
  const int r = tid / tpr, t = tid - r * tpr;
  const int64_t row = int64_t(blockIdx.x) * rows_per_block + r;
  const bool live = r < rows_per_block && row < n_out;
  {
    const float4* src = reinterpret_cast<const float4*>(w);
    float4* dst = reinterpret_cast<float4*>(wsm);
    const int total4 = (kvol * cin * cout) >> 2;
    for (int i = tid; i < total4; i += kRowsThreads) dst[i] = __ldg(src + i);
  }
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  const int cin4 = cin >> 2;
  for (int k0 = 0; k0 < kvol; k0 += 32) {
    int idx[32];
#pragma unroll
    for (int u = 0; u < 32; ++u) idx[u] = (live && k0 + u < kvol) ? __ldg(nbr + size_t(k0 + u) * n_out + row) : -1;
    if (k0 == 0) __syncthreads();   // the weights are staged (the first entries were requested before the wait)
#pragma unroll
    for (int u = 0; u < 32; ++u) {
      if (idx[u] < 0) continue;
      const float4* xr = reinterpret_cast<const float4*>(feats + size_t(idx[u]) * cin);
      const float* wk = wsm + size_t(k0 + u) * cin * cout + 4 * t;
      for (int c4 = 0; c4 < cin4; ++c4) {
        const float4 xv = __ldg(xr + c4);
        const float4 w0 = *reinterpret_cast<const float4*>(wk + size_t(4 * c4 + 0) * cout);
        const float4 w1 = *reinterpret_cast<const float4*>(wk + size_t(4 * c4 + 1) * cout);
        const float4 w2 = *reinterpret_cast<const float4*>(wk + size_t(4 * c4 + 2) * cout);
        const float4 w3 = *reinterpret_cast<const float4*>(wk + size_t(4 * c4 + 3) * cout);
        acc.x = fmaf(xv.x, w0.x, acc.x); acc.y = fmaf(xv.x, w0.y, acc.y); acc.z = fmaf(xv.x, w0.z, acc.z); acc.w = fmaf(xv.x, w0.w, acc.w);
        acc.x = fmaf(xv.y, w1.x, acc.x); acc.y = fmaf(xv.y, w1.y, acc.y); acc.z = fmaf(xv.y, w1.z, acc.z); acc.w = fmaf(xv.y, w1.w, acc.w);
        acc.x = fmaf(xv.z, w2.x, acc.x); acc.y = fmaf(xv.z, w2.y, acc.y); acc.z = fmaf(xv.z, w2.z, acc.z); acc.w = fmaf(xv.z, w2.w, acc.w);
        acc.x = fmaf(xv.w, w3.x, acc.x); acc.y = fmaf(xv.w, w3.y, acc.y); acc.z = fmaf(xv.w, w3.z, acc.z); acc.w = fmaf(xv.w, w3.w, acc.w);
      }
    }
  }
  if (live) *reinterpret_cast<float4*>(out + size_t(row) * cout + 4 * t) = acc;
}

}  // namespace

int forward_simt(const void* feats, const void* w, const spconv_kmap* km, void* out, int cin, int cout,
                 spconv_dtype_t dtype, cudaStream_t stream) {
  if (km->n_out == 0) return SPCONV_OK;
  // fp32 with weights that fit shared memory: the all-weights-resident kernel
  const size_t w_bytes = size_t(km->kvol) * cin * cout * 4;
  if (dtype == SPCONV_F32 && cin % 4 == 0 && cout % 4 == 0 && cout >= 4 && cout <= 4 * kRowsThreads && w_bytes <= size_t(200) * 1024) {
    static std::mutex mu;
    static size_t smem_set[64] = {0};   // largest dynamic shared memory size enabled so far, per device
    const int dev = km->device;
    if (dev < 0 || dev >= 64) return SPCONV_ERR_INVALID_ARG;
    if (w_bytes > 48 * 1024) {
      std::lock_guard<std::mutex> lock(mu);
      if (smem_set[dev] < w_bytes) {
        SPCONV_CUDA_TRY(cudaFuncSetAttribute(k_forward_rows_f32, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        smem_set[dev] = size_t(200) * 1024;
      }
    }
    const int rows_per_block = kRowsThreads / (cout / 4);
    const unsigned row_blocks = unsigned((km->n_out + rows_per_block - 1) / rows_per_block);
    k_forward_rows_f32<<<row_blocks, kRowsThreads, w_bytes, stream>>>(static_cast<const float*>(feats), static_cast<const float*>(w), km->d.nbr,
                                                                      km->n_out, km->kvol, cin, cout, static_cast<float*>(out));
    SPCONV_CUDA_TRY(cudaGetLastError());
    return SPCONV_OK;
  }
  const unsigned blocks = unsigned((km->n_out + kRows - 1) / kRows);
  switch (dtype) {
    case SPCONV_F32:
      k_forward_simt<float><<<blocks, kThreads, 0, stream>>>(static_cast<const float*>(feats), static_cast<const float*>(w),
                                                            km->d.nbr, km->n_out, km->kvol, cin, cout, static_cast<float*>(out));
      break;
    case SPCONV_F16:
      k_forward_simt<__half><<<blocks, kThreads, 0, stream>>>(static_cast<const __half*>(feats), static_cast<const __half*>(w),
                                                             km->d.nbr, km->n_out, km->kvol, cin, cout, static_cast<__half*>(out));
      break;
    case SPCONV_BF16:
      k_forward_simt<__nv_bfloat16><<<blocks, kThreads, 0, stream>>>(
          static_cast<const __nv_bfloat16*>(feats), static_cast<const __nv_bfloat16*>(w), km->d.nbr, km->n_out, km->kvol, cin,
          cout, static_cast<__nv_bfloat16*>(out));
      break;
    default:
      return SPCONV_ERR_INVALID_ARG;
  }
  SPCONV_CUDA_TRY(cudaGetLastError());
  return SPCONV_OK;
}

}  // namespace spconv
