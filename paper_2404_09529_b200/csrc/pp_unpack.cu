// UNPACK (Algorithm 1 (UNPACK), Section 4.3): scatter every prompt's rotated keys and its values
// from the packed [R, M, Hkv, D] tensors into that prompt's own [Hkv, cap, D] cache, in
// original prompt order. Pure 16-byte copies; HBM-bound.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "pp_internal.h"

namespace pp {

// Table layout in int32 units: [0]=k, [1..3] reserved, then token_prefix[k+1], bin_of[k],
// off_of[k], cache_cap[k] (each block padded to a multiple of 4 ints), then cache_off int64[k].
__host__ __device__ static inline int64_t up4(int64_t x) { return (x + 3) & ~int64_t(3); }
size_t unpack_table_bytes(int32_t k) {
  if (k < 1) return 0;
  const int64_t ints = 4 + up4(k + 1) + 3 * up4(k);
  return (size_t)(ints * 4 + (int64_t)k * 8);
}

namespace {

constexpr int kUnpackThreads = 256;
constexpr int kUnpackTokens = 8;    // tokens per block

struct TokenRef {
  int64_t src_row;      // flat packed row (bin * M + off + p)
  int64_t dst_base;     // cache_off[i] + p * D   (element offset of head 0's row p)
  int64_t head_stride;  // cache_cap[i] * D
};

template <int D>
__global__ void __launch_bounds__(kUnpackThreads)
unpack_kernel(const uint4* __restrict__ k_rot, const uint4* __restrict__ v,
              __nv_bfloat16* __restrict__ k_cache, __nv_bfloat16* __restrict__ v_cache,
              const int32_t* __restrict__ table, int32_t n_prompts, int64_t total_tokens,
              int32_t capacity, int32_t n_kv_heads) {
  constexpr int kVecPerHead = D / 8;
  __shared__ TokenRef s_tok[kUnpackTokens];
  const int64_t tok0 = (int64_t)blockIdx.x * kUnpackTokens;
  const int32_t* prefix = table + 4;
  const int32_t* bin_of = prefix + up4(n_prompts + 1);
  const int32_t* off_of = bin_of + up4(n_prompts);
  const int32_t* cap_of = off_of + up4(n_prompts);
  const int64_t* cache_off = reinterpret_cast<const int64_t*>(cap_of + up4(n_prompts));

  if (threadIdx.x < kUnpackTokens) {
    const int64_t tok = tok0 + threadIdx.x;
    TokenRef ref{-1, 0, 0};
    if (tok < total_tokens) {
      int32_t lo = 0, hi = n_prompts - 1;           // last prompt whose prefix is <= tok
      while (lo < hi) {
        const int32_t mid = (lo + hi + 1) >> 1;
        if ((int64_t)prefix[mid] <= tok) lo = mid; else hi = mid - 1;
      }
      const int32_t p = (int32_t)(tok - prefix[lo]);
      ref.src_row = (int64_t)bin_of[lo] * capacity + off_of[lo] + p;
      ref.dst_base = cache_off[lo] + (int64_t)p * D;
      ref.head_stride = (int64_t)cap_of[lo] * D;
    }
    s_tok[threadIdx.x] = ref;
  }
  __syncthreads();

  const int vec_per_row = n_kv_heads * kVecPerHead;       // 16-byte vectors per packed row
  const int units = kUnpackTokens * 2 * vec_per_row;
  for (int u = threadIdx.x; u < units; u += kUnpackThreads) {
    const int t = u / (2 * vec_per_row);
    int w = u - t * 2 * vec_per_row;
    const bool is_v = w >= vec_per_row;
    if (is_v) w -= vec_per_row;
    const TokenRef ref = s_tok[t];
    if (ref.src_row < 0) continue;
    const int head = w / kVecPerHead;
    const int c = w - head * kVecPerHead;
    const uint4 val = __ldg((is_v ? v : k_rot) + ref.src_row * vec_per_row + w);
    __nv_bfloat16* dst = (is_v ? v_cache : k_cache) + ref.dst_base + head * ref.head_stride + c * 8;
    *reinterpret_cast<uint4*>(dst) = val;
  }
}

}  // namespace

int launch_unpack(const pp_attn_params& p, const int32_t* d_table, int32_t k, int64_t total_tokens,
                  const void* k_rot, const void* v, void* k_cache, void* v_cache, void* stream) {
  const unsigned grid = (unsigned)((total_tokens + kUnpackTokens - 1) / kUnpackTokens);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (p.head_dim == 128) {
    unpack_kernel<128><<<grid, kUnpackThreads, 0, s>>>(
        (const uint4*)k_rot, (const uint4*)v, (__nv_bfloat16*)k_cache, (__nv_bfloat16*)v_cache,
        d_table, k, total_tokens, p.capacity, p.n_kv_heads);
  } else {
    unpack_kernel<64><<<grid, kUnpackThreads, 0, s>>>(
        (const uint4*)k_rot, (const uint4*)v, (__nv_bfloat16*)k_cache, (__nv_bfloat16*)v_cache,
        d_table, k, total_tokens, p.capacity, p.n_kv_heads);
  }
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? PP_OK : note_cuda_error((int)e, "unpack kernel launch");
}

}  // namespace pp
