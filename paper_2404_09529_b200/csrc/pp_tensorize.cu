// TENSORIZE (Algorithm 1 (TENSORIZE)) on the device, for the host-buffer entry point: rows of a
// token-major tensor [T, H, D] (prompts back to back in original order) are scattered into the packed
// [R, M, H, D] layout, or gathered back from it. A row is H * D contiguous elements on both sides, so
// this is a row permutation by 16-byte copies; it lets the host side move each tensor with one large
// copy instead of one copy per prompt.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "pp_internal.h"

namespace pp {
namespace {

constexpr int kTzThreads = 256;
constexpr int kTzTokens = 8;    // tokens per block

// map: int64 tok_prefix[n_prompts + 1] (first token of each prompt), then int64 first_row[n_prompts]
// (flat packed row of each prompt's first token).
template <bool kToPacked>
__global__ void __launch_bounds__(kTzThreads)
tensorize_kernel(uint4* __restrict__ packed, uint4* __restrict__ tokens, const int64_t* __restrict__ map,
                 int32_t n_prompts, int64_t total_tokens, int32_t vec_per_row) {
  __shared__ int64_t s_row[kTzTokens];
  const int64_t tok0 = (int64_t)blockIdx.x * kTzTokens;
  if (threadIdx.x < kTzTokens) {
    const int64_t tok = tok0 + threadIdx.x;
    int64_t row = -1;
    if (tok < total_tokens) {
      int32_t lo = 0, hi = n_prompts - 1;           // last prompt whose first token is <= tok
      while (lo < hi) {
        const int32_t mid = (lo + hi + 1) >> 1;
        if (map[mid] <= tok) lo = mid; else hi = mid - 1;
      }
      row = map[n_prompts + 1 + lo] + (tok - map[lo]);
    }
    s_row[threadIdx.x] = row;
  }
  __syncthreads();
  const int units = kTzTokens * vec_per_row;
  for (int u0 = threadIdx.x; u0 < units; u0 += 4 * kTzThreads) {
    uint4 val[4];
    int64_t dst[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int u = u0 + i * kTzThreads;
      dst[i] = -1;
      if (u < units) {
        const int t = u / vec_per_row, w = u - t * vec_per_row;
        const int64_t row = s_row[t];
        if (row >= 0) {
          const int64_t p = row * vec_per_row + w, q = (tok0 + t) * vec_per_row + w;
          val[i] = kToPacked ? tokens[q] : packed[p];
          dst[i] = kToPacked ? p : q;
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (dst[i] >= 0) (kToPacked ? packed : tokens)[dst[i]] = val[i];
  }
}

// Zeroes the padding rows [bin_used[b], capacity) of every bin of up to three packed tensors (the
// attention kernels want finite values there); grid = (bins, row chunks).
struct PadTensors {
  uint4* base[3];
  int32_t vec_per_row[3];
};
__global__ void __launch_bounds__(kTzThreads)
zero_pad_rows_kernel(PadTensors t, const int64_t* __restrict__ bin_used, int32_t capacity) {
  const int32_t b = blockIdx.x;
  const int64_t used = bin_used[b];
  const int64_t pad_rows = capacity - used;
  for (int i = 0; i < 3; ++i) {
    if (!t.base[i]) continue;
    const int64_t n = pad_rows * t.vec_per_row[i];
    uint4* dst = t.base[i] + ((int64_t)b * capacity + used) * t.vec_per_row[i];
    for (int64_t u = (int64_t)blockIdx.y * kTzThreads + threadIdx.x; u < n; u += (int64_t)gridDim.y * kTzThreads)
      dst[u] = make_uint4(0u, 0u, 0u, 0u);
  }
}

}  // namespace

int launch_zero_pad_rows(void* q, void* k, void* v, int32_t q_row_bytes, int32_t kv_row_bytes,
                         const int64_t* d_bin_used, int32_t n_bins, int32_t capacity, void* stream) {
  PadTensors t;
  t.base[0] = static_cast<uint4*>(q); t.base[1] = static_cast<uint4*>(k); t.base[2] = static_cast<uint4*>(v);
  t.vec_per_row[0] = q_row_bytes / 16; t.vec_per_row[1] = t.vec_per_row[2] = kv_row_bytes / 16;
  zero_pad_rows_kernel<<<dim3((unsigned)n_bins, 8), kTzThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      t, d_bin_used, capacity);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? PP_OK : note_cuda_error((int)e, "padding-row kernel launch");
}

int launch_tensorize(bool to_packed, void* packed, void* tokens, const int64_t* d_map, int32_t n_prompts,
                     int64_t total_tokens, int32_t row_bytes, void* stream) {
  if (total_tokens <= 0) return PP_OK;
  const unsigned grid = (unsigned)((total_tokens + kTzTokens - 1) / kTzTokens);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (to_packed)
    tensorize_kernel<true><<<grid, kTzThreads, 0, s>>>(static_cast<uint4*>(packed), static_cast<uint4*>(tokens),
                                                       d_map, n_prompts, total_tokens, row_bytes / 16);
  else
    tensorize_kernel<false><<<grid, kTzThreads, 0, s>>>(static_cast<uint4*>(packed), static_cast<uint4*>(tokens),
                                                        d_map, n_prompts, total_tokens, row_bytes / 16);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? PP_OK : note_cuda_error((int)e, "tensorize kernel launch");
}

}  // namespace pp
