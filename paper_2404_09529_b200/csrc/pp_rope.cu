// Restart rotary positional encoding over the packed batch (Section 3.2, Algorithm 1 line 7).
// Each row's position is its bin-local row index minus the start row of the prompt it belongs
// to; Q and K rows are rotated in place. HBM-bound: every element is read once and written once.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "pp_internal.h"

namespace pp {
namespace {

constexpr int kRopeThreads = 256;
constexpr int kRopeRows = 4;        // packed rows per block
constexpr int kMaxHalf = 64;        // head_dim / 2 at most

struct RopeFreq {
  double inv_freq[kMaxHalf];        // theta_j = base^(-2j/D), computed in double on the host
};

__device__ __forceinline__ float2 bf2_to_f2(uint32_t u) {
  __nv_bfloat162 h = *reinterpret_cast<__nv_bfloat162*>(&u);
  return __bfloat1622float2(h);
}
__device__ __forceinline__ uint32_t f2_to_bf2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Rotates the 8 (lower, upper) pairs held in two 16-byte vectors.
__device__ __forceinline__ void rotate8(uint4& lo, uint4& hi, const float* cs, const float* sn) {
  uint32_t* l = reinterpret_cast<uint32_t*>(&lo);
  uint32_t* h = reinterpret_cast<uint32_t*>(&hi);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 a = bf2_to_f2(l[i]);
    const float2 b = bf2_to_f2(h[i]);
    const float c0 = cs[2 * i], c1 = cs[2 * i + 1], s0 = sn[2 * i], s1 = sn[2 * i + 1];
    l[i] = f2_to_bf2(a.x * c0 - b.x * s0, a.y * c1 - b.y * s1);
    h[i] = f2_to_bf2(b.x * c0 + a.x * s0, b.y * c1 + a.y * s1);
  }
}

template <int D>
__global__ void __launch_bounds__(kRopeThreads)
rope_kernel(__nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ k,
            const int32_t* __restrict__ table, int32_t off_bin_seg_ptr, int32_t off_bin_used,
            int32_t off_seg_start, int32_t n_bins, int32_t capacity, int32_t n_q_heads,
            int32_t n_kv_heads, const __grid_constant__ RopeFreq freq) {
  constexpr int kHalf = D / 2;
  constexpr int kUnitsPerHead = kHalf / 8;          // 16-byte vector pairs per head
  __shared__ int32_t s_pos[kRopeRows];              // restart position, -1 for padding rows
  __shared__ float s_cos[kRopeRows][kHalf];
  __shared__ float s_sin[kRopeRows][kHalf];

  const int64_t row0 = (int64_t)blockIdx.x * kRopeRows;
  const int64_t n_rows = (int64_t)n_bins * capacity;
  const int tid = threadIdx.x;

  if (tid < kRopeRows) {
    const int64_t row = row0 + tid;
    int32_t pos = -1;
    if (row < n_rows) {
      const int32_t b = (int32_t)(row / capacity);
      const int32_t t = (int32_t)(row - (int64_t)b * capacity);
      if (t < table[off_bin_used + b]) {
        // last segment of bin b whose start row is <= t
        int32_t lo = table[off_bin_seg_ptr + b], hi = table[off_bin_seg_ptr + b + 1] - 1;
        while (lo < hi) {
          const int32_t mid = (lo + hi + 1) >> 1;
          if (table[off_seg_start + mid] <= t) lo = mid; else hi = mid - 1;
        }
        pos = t - table[off_seg_start + lo];
      }
    }
    s_pos[tid] = pos;
  }
  __syncthreads();

  if (tid < kRopeRows * kHalf) {
    const int r = tid / kHalf, j = tid % kHalf;
    const int32_t pos = s_pos[r];
    float sn = 0.f, cs = 1.f;
    if (pos > 0) {
      // angle in double, reduced to [-pi, pi] before the single-precision sincos, so that the
      // argument error stays ~1e-7 rad even at positions of several 10^4
      const double ang = (double)pos * freq.inv_freq[j];
      const double n = rint(ang * 0.15915494309189535);                 // 1 / (2 pi)
      double red = fma(-n, 6.283185307179586, ang);
      red = fma(-n, 2.4492935982947064e-16, red);                      // low part of 2 pi
      sincosf((float)red, &sn, &cs);
    }
    s_cos[r][j] = cs;
    s_sin[r][j] = sn;
  }
  __syncthreads();

  const int units_per_row = (n_q_heads + n_kv_heads) * kUnitsPerHead;
  for (int u = tid; u < kRopeRows * units_per_row; u += kRopeThreads) {
    const int r = u / units_per_row;
    const int w = u - r * units_per_row;
    if (s_pos[r] <= 0) continue;                    // padding row, or position 0 (identity)
    const int head = w / kUnitsPerHead;
    const int c = w - head * kUnitsPerHead;
    const int64_t row = row0 + r;
    __nv_bfloat16* base = head < n_q_heads
        ? q + (row * n_q_heads + head) * D
        : k + (row * n_kv_heads + (head - n_q_heads)) * D;
    uint4* p_lo = reinterpret_cast<uint4*>(base + c * 8);
    uint4* p_hi = reinterpret_cast<uint4*>(base + kHalf + c * 8);
    uint4 lo = *p_lo, hi = *p_hi;
    rotate8(lo, hi, &s_cos[r][c * 8], &s_sin[r][c * 8]);
    *p_lo = lo;
    *p_hi = hi;
  }
}

}  // namespace

int launch_rope(const pp_attn_params& p, const int32_t* d_table, const TableLayout& L, void* q,
                void* k, void* stream) {
  RopeFreq freq;
  const int half = p.head_dim / 2;
  for (int j = 0; j < kMaxHalf; ++j)
    freq.inv_freq[j] = j < half ? pow((double)p.rope_base, -2.0 * j / (double)p.head_dim) : 0.0;
  const int64_t n_rows = (int64_t)p.n_bins * p.capacity;
  const unsigned grid = (unsigned)((n_rows + kRopeRows - 1) / kRopeRows);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (p.head_dim == 128) {
    rope_kernel<128><<<grid, kRopeThreads, 0, s>>>(
        (__nv_bfloat16*)q, (__nv_bfloat16*)k, d_table, L.bin_seg_ptr, L.bin_used, L.seg_start,
        p.n_bins, p.capacity, p.n_q_heads, p.n_kv_heads, freq);
  } else {
    rope_kernel<64><<<grid, kRopeThreads, 0, s>>>(
        (__nv_bfloat16*)q, (__nv_bfloat16*)k, d_table, L.bin_seg_ptr, L.bin_used, L.seg_start,
        p.n_bins, p.capacity, p.n_q_heads, p.n_kv_heads, freq);
  }
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? PP_OK : note_cuda_error((int)e, "rope kernel launch");
}

}  // namespace pp
