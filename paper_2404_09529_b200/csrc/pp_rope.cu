// Restart rotary positional encoding over the packed batch (Section 3.2, Algorithm 1 (RESTART-PE)).
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
    // written with explicit fma/mul so that every kernel that rotates gives the same bits
    l[i] = f2_to_bf2(__fmaf_rn(a.x, c0, -__fmul_rn(b.x, s0)), __fmaf_rn(a.y, c1, -__fmul_rn(b.y, s1)));
    h[i] = f2_to_bf2(__fmaf_rn(b.x, c0, __fmul_rn(a.x, s0)), __fmaf_rn(b.y, c1, __fmul_rn(a.y, s1)));
  }
}

template <int D>
__global__ void __launch_bounds__(kRopeThreads)
rope_kernel(const __nv_bfloat16* q, __nv_bfloat16* q_out, __nv_bfloat16* __restrict__ k,
            const int32_t* __restrict__ table, int32_t off_bin_seg_ptr, int32_t off_bin_used,
            int32_t off_seg_start, int32_t n_bins, int32_t capacity, int32_t n_q_heads,
            int32_t n_kv_heads, const __grid_constant__ RopeFreq freq) {
  constexpr int kHalf = D / 2;
  constexpr int kUnitsPerHead = kHalf / 8;          // 16-byte vector pairs per head
  __shared__ int32_t s_pos[kRopeRows];              // restart position, -1 for padding rows
  __shared__ float s_cos[kRopeRows][kHalf];
  __shared__ float s_sin[kRopeRows][kHalf];

  pdl_launch_dependents();      // the attention kernel may set up while this one runs
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
    const bool in_place = (q_out == q);
    // padding rows are skipped; position 0 is the identity (copied only when Q goes elsewhere)
    if (s_pos[r] < 0 || (s_pos[r] == 0 && (in_place || w >= n_q_heads * kUnitsPerHead))) continue;
    const int head = w / kUnitsPerHead;
    const int c = w - head * kUnitsPerHead;
    const int64_t row = row0 + r;
    const bool is_q = head < n_q_heads;
    const int64_t off = is_q ? (row * n_q_heads + head) * D : (row * n_kv_heads + (head - n_q_heads)) * D;
    const __nv_bfloat16* src = is_q ? q + off : k + off;
    __nv_bfloat16* dst = is_q ? q_out + off : k + off;
    uint4 lo = *reinterpret_cast<const uint4*>(src + c * 8);
    uint4 hi = *reinterpret_cast<const uint4*>(src + kHalf + c * 8);
    if (s_pos[r] > 0) rotate8(lo, hi, &s_cos[r][c * 8], &s_sin[r][c * 8]);
    *reinterpret_cast<uint4*>(dst + c * 8) = lo;
    *reinterpret_cast<uint4*>(dst + kHalf + c * 8) = hi;
  }
}

// cos/sin of position * theta_j for every position of a bin, laid out [j / 2][pos][j % 2] as
// (cos, sin) pairs, so that threads working on consecutive rows (positions) read consecutive
// 16-byte pieces. Read by the fused kernels.
__global__ void __launch_bounds__(256)
rope_table_kernel(float2* __restrict__ table, int32_t capacity, int32_t half,
                  const __grid_constant__ RopeFreq freq) {
  pdl_launch_dependents();      // the fused K/V kernel may set up while this one runs
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)capacity * half) return;
  const int32_t pos = (int32_t)(idx / half), j = (int32_t)(idx - (int64_t)pos * half);
  float sn = 0.f, cs = 1.f;
  if (pos > 0) {      // same arithmetic as rope_kernel, so both give identical bits
    const double ang = (double)pos * freq.inv_freq[j];
    const double n = rint(ang * 0.15915494309189535);
    double red = fma(-n, 6.283185307179586, ang);
    red = fma(-n, 2.4492935982947064e-16, red);
    sincosf((float)red, &sn, &cs);
  }
  table[((size_t)(j >> 1) * capacity + pos) * 2 + (j & 1)] = make_float2(cs, sn);
}

// Fused K rotation + UNPACK (Algorithm 1 (RESTART-PE to UNPACK) in one pass over K and V): every real packed
// row of K is rotated (cos/sin from the table), written back to the packed tensor (the attention
// kernel reads it there) and into its prompt's K cache; the V row is copied into the V cache.
struct SegExt {                    // per-segment arrays appended to the prefill table
  int32_t off_true_len, off_cap, off_cache_off;   // int32 offsets into the table (cache_off: int64 data)
};

// Packed rows per block of the fused K/V kernel: 8 where a row of K is several KB (many KV heads), 32
// where it is at most 2 KB, so that a block always has tens of KB to move for its set-up cost.
constexpr int kRuRowsWide = 8, kRuRowsNarrow = 32;
constexpr int kRuNarrowRowElems = 1024;   // n_kv_heads * D up to which a row counts as narrow
constexpr int kRuV = 8;      // 16-byte V copies in flight per thread
constexpr int kRuK = 2;      // (lower, upper) K pairs in flight per thread
template <int D, int kRuRows>
__global__ void __launch_bounds__(kRopeThreads)
rope_unpack_kernel(__nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                   __nv_bfloat16* __restrict__ k_cache, __nv_bfloat16* __restrict__ v_cache,
                   const int32_t* __restrict__ table, int32_t off_bin_seg_ptr, int32_t off_bin_used,
                   int32_t off_seg_start, SegExt ext, const float2* __restrict__ rope_table,
                   int32_t n_bins, int32_t capacity, int32_t n_kv_heads) {
  constexpr int kHalf = D / 2;
  constexpr int kPairUnits = kHalf / 8;             // (lower, upper) 16-byte pairs per head
  constexpr int kVecs = D / 8;                      // 16-byte vectors per head
  __shared__ int32_t s_pos[kRuRows];              // restart position, -1 for padding rows
  __shared__ int64_t s_dst[kRuRows];              // cache element offset of (head 0, this position); -1: not cached
  __shared__ int64_t s_head_stride[kRuRows];      // cache_cap * D
  __shared__ float4 s_tab[kRuRows][D / 4];          // (cos, sin) of j = 2g, 2g + 1 at each row's position

  pdl_launch_dependents();      // the attention kernel may set up while this one runs
  const int64_t row0 = (int64_t)blockIdx.x * kRuRows;
  const int64_t n_rows = (int64_t)n_bins * capacity;
  const int tid = threadIdx.x;
  if (tid < kRuRows) {
    const int64_t row = row0 + tid;
    int32_t pos = -1;
    int64_t dst = -1, stride = 0;
    if (row < n_rows) {
      const int32_t b = (int32_t)(row / capacity);
      const int32_t t = (int32_t)(row - (int64_t)b * capacity);
      if (t < table[off_bin_used + b]) {
        int32_t lo = table[off_bin_seg_ptr + b], hi = table[off_bin_seg_ptr + b + 1] - 1;
        while (lo < hi) {
          const int32_t mid = (lo + hi + 1) >> 1;
          if (table[off_seg_start + mid] <= t) lo = mid; else hi = mid - 1;
        }
        pos = t - table[off_seg_start + lo];
        if (pos < table[ext.off_true_len + lo]) {   // rows past the prompt's true length are not cached
          const int64_t* coff = reinterpret_cast<const int64_t*>(table + ext.off_cache_off);
          stride = (int64_t)table[ext.off_cap + lo] * D;
          dst = coff[lo] + (int64_t)pos * D;
        }
      }
    }
    s_pos[tid] = pos;
    s_dst[tid] = dst;
    s_head_stride[tid] = stride;
  }
  __syncthreads();
  pdl_wait();                   // the rotation table is written by the kernel before this one
  // each row's D/2 (cos, sin) pairs once, for all heads: D/4 16-byte loads per row, one per thread
  for (int u = tid; u < kRuRows * (D / 4); u += kRopeThreads) {
    const int r = u / (D / 4), g = u - r * (D / 4);
    const int32_t pos = s_pos[r];
    if (pos > 0) s_tab[r][g] = __ldg(reinterpret_cast<const float4*>(rope_table) + (size_t)g * (size_t)capacity + pos);
  }

  // V rows first: plain 16-byte copies, four in flight per thread
  const int units_v = n_kv_heads * kVecs;
  for (int u0 = tid; u0 < kRuRows * units_v; u0 += kRuV * kRopeThreads) {
    uint4 val[kRuV];
    int64_t dsts[kRuV];
#pragma unroll
    for (int i = 0; i < kRuV; ++i) {
      const int u = u0 + i * kRopeThreads;
      dsts[i] = -1;
      if (u < kRuRows * units_v) {
        const int r = u / units_v, w = u - r * units_v;
        if (s_dst[r] >= 0) {
          const int head = w / kVecs, c = w - head * kVecs;
          val[i] = __ldg(reinterpret_cast<const uint4*>(v + ((row0 + r) * n_kv_heads + head) * D + c * 8));
          dsts[i] = s_dst[r] + head * s_head_stride[r] + c * 8;
        }
      }
    }
#pragma unroll
    for (int i = 0; i < kRuV; ++i)
      if (dsts[i] >= 0) *reinterpret_cast<uint4*>(v_cache + dsts[i]) = val[i];
  }
  __syncthreads();
  // K rows: rotate, write back to the packed tensor and into the cache; two pairs in flight
  const int units_k = n_kv_heads * kPairUnits;
  for (int u0 = tid; u0 < kRuRows * units_k; u0 += kRuK * kRopeThreads) {
    uint4 lo[kRuK], hi[kRuK];
    int rr[kRuK], hh[kRuK], cc[kRuK];
#pragma unroll
    for (int i = 0; i < kRuK; ++i) {
      const int u = u0 + i * kRopeThreads;
      rr[i] = -1;
      if (u < kRuRows * units_k) {
        const int r = u / units_k, w = u - r * units_k;
        if (s_pos[r] >= 0) {
          rr[i] = r; hh[i] = w / kPairUnits; cc[i] = w - hh[i] * kPairUnits;
          const __nv_bfloat16* base = k + ((row0 + r) * n_kv_heads + hh[i]) * D;
          lo[i] = *reinterpret_cast<const uint4*>(base + cc[i] * 8);
          hi[i] = *reinterpret_cast<const uint4*>(base + kHalf + cc[i] * 8);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < kRuK; ++i) {
      if (rr[i] < 0) continue;
      const int r = rr[i], head = hh[i], c = cc[i];
      const int32_t pos = s_pos[r];
      __nv_bfloat16* base = k + ((row0 + r) * n_kv_heads + head) * D;
      if (pos > 0) {
        float cs[8], sn[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 t4 = s_tab[r][c * 4 + q];
          cs[2 * q] = t4.x; sn[2 * q] = t4.y; cs[2 * q + 1] = t4.z; sn[2 * q + 1] = t4.w;
        }
        rotate8(lo[i], hi[i], cs, sn);
        *reinterpret_cast<uint4*>(base + c * 8) = lo[i];
        *reinterpret_cast<uint4*>(base + kHalf + c * 8) = hi[i];
      }
      if (s_dst[r] >= 0) {
        __nv_bfloat16* cd = k_cache + s_dst[r] + head * s_head_stride[r];
        *reinterpret_cast<uint4*>(cd + c * 8) = lo[i];
        *reinterpret_cast<uint4*>(cd + kHalf + c * 8) = hi[i];
      }
    }
  }
}

RopeFreq make_freq(const pp_attn_params& p) {
  RopeFreq freq;
  const int half = p.head_dim / 2;
  for (int j = 0; j < kMaxHalf; ++j)
    freq.inv_freq[j] = j < half ? pow((double)p.rope_base, -2.0 * j / (double)p.head_dim) : 0.0;
  return freq;
}

}  // namespace

int launch_rope_table(const pp_attn_params& p, void* table, void* stream) {
  const RopeFreq freq = make_freq(p);
  const int half = p.head_dim / 2;
  const int64_t n = (int64_t)p.capacity * half;
  rope_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<float2*>(table), p.capacity, half, freq);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? PP_OK : note_cuda_error((int)e, "rope table kernel launch");
}

int launch_rope_unpack(const pp_attn_params& p, const int32_t* d_table, const TableLayout& L,
                       int32_t off_true_len, int32_t off_cap, int32_t off_cache_off, const void* rope_table,
                       void* k, const void* v, void* k_cache, void* v_cache, void* stream) {
  const int64_t n_rows = (int64_t)p.n_bins * p.capacity;
  const bool narrow = p.n_kv_heads * p.head_dim <= kRuNarrowRowElems;
  const int rows = narrow ? kRuRowsNarrow : kRuRowsWide;
  const unsigned grid = (unsigned)((n_rows + rows - 1) / rows);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const SegExt ext{off_true_len, off_cap, off_cache_off};
  cudaError_t launch_err = cudaSuccess;
#define PP_RU_LAUNCH(DD, RR)                                                                                      \
  launch_err = launch_dependent(rope_unpack_kernel<DD, RR>, dim3(grid), dim3(kRopeThreads), 0, s,                 \
      (__nv_bfloat16*)k, (const __nv_bfloat16*)v, (__nv_bfloat16*)k_cache, (__nv_bfloat16*)v_cache, d_table,      \
      L.bin_seg_ptr, L.bin_used, L.seg_start, ext, (const float2*)rope_table, p.n_bins, p.capacity, p.n_kv_heads)
  if (p.head_dim == 128) {
    if (narrow) PP_RU_LAUNCH(128, kRuRowsNarrow); else PP_RU_LAUNCH(128, kRuRowsWide);
  } else {
    if (narrow) PP_RU_LAUNCH(64, kRuRowsNarrow); else PP_RU_LAUNCH(64, kRuRowsWide);
  }
#undef PP_RU_LAUNCH
  const cudaError_t e = launch_err != cudaSuccess ? launch_err : cudaGetLastError();
  return e == cudaSuccess ? PP_OK : note_cuda_error((int)e, "rope+unpack kernel launch");
}

int launch_rope(const pp_attn_params& p, const int32_t* d_table, const TableLayout& L, const void* q,
                void* q_out, void* k, void* stream) {
  const RopeFreq freq = make_freq(p);
  const int64_t n_rows = (int64_t)p.n_bins * p.capacity;
  const unsigned grid = (unsigned)((n_rows + kRopeRows - 1) / kRopeRows);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (p.head_dim == 128) {
    rope_kernel<128><<<grid, kRopeThreads, 0, s>>>(
        (const __nv_bfloat16*)q, (__nv_bfloat16*)q_out, (__nv_bfloat16*)k, d_table, L.bin_seg_ptr, L.bin_used, L.seg_start,
        p.n_bins, p.capacity, p.n_q_heads, p.n_kv_heads, freq);
  } else {
    rope_kernel<64><<<grid, kRopeThreads, 0, s>>>(
        (const __nv_bfloat16*)q, (__nv_bfloat16*)q_out, (__nv_bfloat16*)k, d_table, L.bin_seg_ptr, L.bin_used, L.seg_start,
        p.n_bins, p.capacity, p.n_q_heads, p.n_kv_heads, freq);
  }
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? PP_OK : note_cuda_error((int)e, "rope kernel launch");
}

}  // namespace pp
