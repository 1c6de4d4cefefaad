// One generation step over the per-prompt caches that UNPACK produced (Section 7 of the prepacking
// paper, "prepacking for generation"): the caches are never padded, so the step reads exactly the
// keys and values every prompt has. Three kernels:
//   decode_append_kernel     rotates the new token's q and k by its position (= tokens cached so far),
//                            appends k' and v to the prompt's caches, leaves q' in the workspace
//   decode_partial_kernel    one CTA per (chunk of 256 or 64 cached keys, KV head): scores, online softmax
//                            and P V for the query heads of that KV head, partial (m, l, o) out
//   decode_combine_kernel    merges a prompt's chunks into o
// HBM-bound: K and V of every cached token are read once.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>

#include "pp_internal.h"

namespace pp {
namespace {

constexpr int kDecodeThreads = 128;     // 4 warps per CTA
constexpr int kMaxGroup = 8;            // query heads per KV head supported by the partial kernel

struct DecodeFreq {
  double inv_freq[64];                  // theta_j = base^(-2j/D), computed in double on the host
};

// Offsets (int32 units) inside the uploaded table: chunks[n_chunks][3] = (prompt, first key, keys),
// chunk_ptr[k + 1], lengths[k], cache_cap[k], cache_off int64[k].
struct DecodeTable {
  int32_t chunks, chunk_ptr, lengths, cache_cap, cache_off;
};

template <int D>
__global__ void __launch_bounds__(kDecodeThreads)
decode_append_kernel(const __nv_bfloat16* __restrict__ q_new, const __nv_bfloat16* __restrict__ k_new,
                     const __nv_bfloat16* __restrict__ v_new, __nv_bfloat16* __restrict__ q_rot,
                     __nv_bfloat16* __restrict__ k_cache, __nv_bfloat16* __restrict__ v_cache,
                     const int32_t* __restrict__ table, DecodeTable T, int32_t n_q_heads, int32_t n_kv_heads,
                     const __grid_constant__ DecodeFreq freq) {
  constexpr int kHalf = D / 2;
  __shared__ float s_cos[kHalf], s_sin[kHalf];
  pdl_launch_dependents();      // the partial kernel may set up while this one runs
  const int i = blockIdx.x;
  const int32_t pos = table[T.lengths + i];                      // position of the new token
  const int64_t cap = table[T.cache_cap + i];
  const int64_t base = reinterpret_cast<const int64_t*>(table + T.cache_off)[i];
  if (threadIdx.x < kHalf) {
    float sn = 0.f, cs = 1.f;
    if (pos > 0) {      // same reduction as the prefill kernels
      const double ang = (double)pos * freq.inv_freq[threadIdx.x];
      const double n = rint(ang * 0.15915494309189535);
      double red = fma(-n, 6.283185307179586, ang);
      red = fma(-n, 2.4492935982947064e-16, red);
      sincosf((float)red, &sn, &cs);
    }
    s_cos[threadIdx.x] = cs;
    s_sin[threadIdx.x] = sn;
  }
  __syncthreads();
  // Units of eight (j, j + D/2) pairs: (head, group of eight j) of q, then of k. 16-byte accesses, and
  // the loads of up to four units are issued before the first store (the compiler cannot prove
  // that the destinations do not alias the sources, so it would serialise them otherwise).
  constexpr int kGroups = kHalf / 8;
  const int n_units = (n_q_heads + n_kv_heads) * kGroups;
  for (int u0 = threadIdx.x; u0 < n_units; u0 += 4 * kDecodeThreads) {
    uint4 lo[4], hi[4];
    __nv_bfloat16* dst[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const int u = u0 + x * kDecodeThreads;
      dst[x] = nullptr;
      if (u < n_units) {
        const int head = u / kGroups, g = u - head * kGroups;
        const bool is_k = head >= n_q_heads;
        const __nv_bfloat16* src = is_k ? k_new + ((int64_t)i * n_kv_heads + (head - n_q_heads)) * D
                                        : q_new + ((int64_t)i * n_q_heads + head) * D;
        dst[x] = (is_k ? k_cache + base + ((int64_t)(head - n_q_heads) * cap + pos) * D
                       : q_rot + ((int64_t)i * n_q_heads + head) * D) + 8 * g;
        lo[x] = __ldg(reinterpret_cast<const uint4*>(src + 8 * g));
        hi[x] = __ldg(reinterpret_cast<const uint4*>(src + 8 * g + kHalf));
      }
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      if (!dst[x]) continue;
      const int j0 = (int)((u0 + x * kDecodeThreads) % kGroups) * 8;
      uint32_t* l32 = reinterpret_cast<uint32_t*>(&lo[x]);
      uint32_t* h32 = reinterpret_cast<uint32_t*>(&hi[x]);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&l32[e]));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&h32[e]));
        const float c0 = s_cos[j0 + 2 * e], s0 = s_sin[j0 + 2 * e], c1 = s_cos[j0 + 2 * e + 1], s1 = s_sin[j0 + 2 * e + 1];
        const __nv_bfloat162 lo2 = __floats2bfloat162_rn(__fmaf_rn(a.x, c0, -__fmul_rn(b.x, s0)),
                                                         __fmaf_rn(a.y, c1, -__fmul_rn(b.y, s1)));
        const __nv_bfloat162 hi2 = __floats2bfloat162_rn(__fmaf_rn(b.x, c0, __fmul_rn(a.x, s0)),
                                                         __fmaf_rn(b.y, c1, __fmul_rn(a.y, s1)));
        l32[e] = *reinterpret_cast<const uint32_t*>(&lo2);
        h32[e] = *reinterpret_cast<const uint32_t*>(&hi2);
      }
      *reinterpret_cast<uint4*>(dst[x]) = lo[x];
      *reinterpret_cast<uint4*>(dst[x] + kHalf) = hi[x];
    }
  }
  // v is copied as it is
  for (int u = threadIdx.x; u < n_kv_heads * (D / 8); u += kDecodeThreads) {
    const int head = u / (D / 8), g = u - head * (D / 8);
    *reinterpret_cast<uint4*>(v_cache + base + ((int64_t)head * cap + pos) * D + 8 * g) =
        __ldg(reinterpret_cast<const uint4*>(v_new + ((int64_t)i * n_kv_heads + head) * D + 8 * g));
  }
}

// partial results: [chunk][query head][D + 2] floats = (m, l, o[D]), m in scaled log2 units.
// G: compile-time bound on the query heads per KV head (1, 2, 4 or 8), so that a small group does
// not pay registers for a large one.
template <int D, int G>
__global__ void __launch_bounds__(kDecodeThreads)
decode_partial_kernel(const __nv_bfloat16* __restrict__ q_rot, const __nv_bfloat16* __restrict__ k_cache,
                      const __nv_bfloat16* __restrict__ v_cache, float* __restrict__ partial,
                      const int32_t* __restrict__ table, DecodeTable T, int32_t n_q_heads, int32_t n_kv_heads,
                      int32_t group, float scale_log2) {
  constexpr int E = D / 32;                       // elements of a row per lane
  __shared__ float s_m[4][G], s_l[4][G], s_o[4][G][D];
  const int chunk = blockIdx.x, kvh = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = table[T.chunks + 3 * chunk], key0 = table[T.chunks + 3 * chunk + 1], n_keys = table[T.chunks + 3 * chunk + 2];
  const int64_t cap = table[T.cache_cap + i];
  const int64_t base = reinterpret_cast<const int64_t*>(table + T.cache_off)[i] + (int64_t)kvh * cap * D;
  pdl_launch_dependents();      // the combine kernel may set up while this one runs
  pdl_wait();                   // rotated queries and the appended K / V rows come from the append kernel
  float q[G][E], acc[G][E], m[G], l[G];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    m[h] = -INFINITY;
    l[h] = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) {
      acc[h][e] = 0.f;
      q[h][e] = (h < group) ? __bfloat162float(q_rot[((int64_t)i * n_q_heads + kvh * group + h) * D + lane * E + e]) : 0.f;
    }
  }
  // one 4- or 8-byte load per lane and row; four keys per iteration keep eight loads in flight
  auto load_row = [&](const __nv_bfloat16* p, float (&out)[E]) {
    if constexpr (E == 4) {
      const uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
      const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.x));
      const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.y));
      out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
    } else {
      const uint32_t u = __ldg(reinterpret_cast<const uint32_t*>(p));
      const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u));
      out[0] = a.x; out[1] = a.y;
    }
  };
  auto one_key = [&](const float (&kk)[E], const float (&vv)[E]) {
#pragma unroll
    for (int h = 0; h < G; ++h) {
      if (h >= group) break;
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) s = fmaf(q[h][e], kk[e], s);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      s *= scale_log2;
      const float m_new = fmaxf(m[h], s);
      const float alpha = exp2f(m[h] - m_new), p = exp2f(s - m_new);      // exp2f(-inf) = 0 on the first key
      l[h] = l[h] * alpha + p;
#pragma unroll
      for (int e = 0; e < E; ++e) acc[h][e] = acc[h][e] * alpha + p * vv[e];
      m[h] = m_new;
    }
  };
  const __nv_bfloat16* kbase = k_cache + base + (int64_t)key0 * D + lane * E;
  const __nv_bfloat16* vbase = v_cache + base + (int64_t)key0 * D + lane * E;
  int t = warp;
  for (; t + 12 < n_keys; t += 16) {
    float kx[4][E], vx[4][E];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      load_row(kbase + (int64_t)(t + 4 * u) * D, kx[u]);
      load_row(vbase + (int64_t)(t + 4 * u) * D, vx[u]);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) one_key(kx[u], vx[u]);
  }
  for (; t < n_keys; t += 4) {
    float k0[E], v0[E];
    load_row(kbase + (int64_t)t * D, k0);
    load_row(vbase + (int64_t)t * D, v0);
    one_key(k0, v0);
  }
  // merge the four warps
#pragma unroll
  for (int h = 0; h < G; ++h) {
    if (h >= group) break;
    if (lane == 0) { s_m[warp][h] = m[h]; s_l[warp][h] = l[h]; }
#pragma unroll
    for (int e = 0; e < E; ++e) s_o[warp][h][lane * E + e] = acc[h][e];
  }
  __syncthreads();
  for (int u = threadIdx.x; u < group * D; u += kDecodeThreads) {
    const int h = u / D, d = u - h * D;
    float mm = -INFINITY;
    for (int w = 0; w < 4; ++w) mm = fmaxf(mm, s_m[w][h]);
    float ll = 0.f, oo = 0.f;
    for (int w = 0; w < 4; ++w) {
      const float f = (s_m[w][h] == -INFINITY) ? 0.f : exp2f(s_m[w][h] - mm);
      ll += s_l[w][h] * f;
      oo += s_o[w][h][d] * f;
    }
    float* out = partial + ((int64_t)chunk * n_q_heads + kvh * group + h) * (D + 2);
    if (d == 0) { out[0] = mm; out[1] = ll; }
    out[2 + d] = oo;
  }
}

template <int D>
__global__ void __launch_bounds__(D)
decode_combine_kernel(const float* __restrict__ partial, __nv_bfloat16* __restrict__ o,
                      const int32_t* __restrict__ table, DecodeTable T, int32_t n_q_heads) {
  const int i = blockIdx.x, head = blockIdx.y, d = threadIdx.x;
  const int c0 = table[T.chunk_ptr + i], c1 = table[T.chunk_ptr + i + 1];
  pdl_wait();                   // the partial results come from the kernel before this one
  float mm = -INFINITY;
  for (int c = c0; c < c1; ++c) mm = fmaxf(mm, partial[((int64_t)c * n_q_heads + head) * (D + 2)]);
  float ll = 0.f, oo = 0.f;
  for (int c = c0; c < c1; ++c) {
    const float* p = partial + ((int64_t)c * n_q_heads + head) * (D + 2);
    const float f = exp2f(p[0] - mm);
    ll += p[1] * f;
    oo += p[2 + d] * f;
  }
  o[((int64_t)i * n_q_heads + head) * D + d] = __float2bfloat16_rn(oo / ll);
}

// Keys per chunk: 256 when that already gives every SM several CTAs, else 64, so that a small batch
// (a few prompts, one of them long) is spread over more CTAs and each warp's chain of dependent row
// loads is a quarter as long.
constexpr int kChunkKeysLarge = 256, kChunkKeysSmall = 64;
constexpr int64_t kChunkCtasWanted = 148 * 8;

int64_t count_chunks(const int32_t* lengths, int32_t k, int chunk_keys) {
  int64_t n = 0;
  for (int32_t i = 0; i < k; ++i) n += ((int64_t)lengths[i] + 1 + chunk_keys - 1) / chunk_keys;
  return n;
}
size_t up4(size_t x) { return (x + 3) & ~size_t(3); }

struct DecodeLayout {
  DecodeTable T;
  size_t table_ints, q_rot_bytes_off, partial_bytes_off, total_bytes;
  int64_t n_chunks;
  int chunk_keys;
};
DecodeLayout decode_layout(const pp_attn_params& p, const int32_t* lengths, int32_t k) {
  DecodeLayout L;
  L.chunk_keys = kChunkKeysLarge;
  L.n_chunks = count_chunks(lengths, k, L.chunk_keys);
  if (L.n_chunks * p.n_kv_heads < kChunkCtasWanted) {
    L.chunk_keys = kChunkKeysSmall;
    L.n_chunks = count_chunks(lengths, k, L.chunk_keys);
  }
  size_t off = 0;
  L.T.chunks = (int32_t)off; off += up4(3 * (size_t)L.n_chunks);
  L.T.chunk_ptr = (int32_t)off; off += up4((size_t)k + 1);
  L.T.lengths = (int32_t)off; off += up4((size_t)k);
  L.T.cache_cap = (int32_t)off; off += up4((size_t)k);
  L.T.cache_off = (int32_t)off; off += 2 * (size_t)k;
  L.table_ints = off;
  L.q_rot_bytes_off = (off * 4 + 255) & ~size_t(255);
  L.partial_bytes_off = (L.q_rot_bytes_off + (size_t)k * p.n_q_heads * p.head_dim * 2 + 255) & ~size_t(255);
  L.total_bytes = L.partial_bytes_off + (size_t)L.n_chunks * p.n_q_heads * (p.head_dim + 2) * sizeof(float);
  return L;
}

int check_decode_params(const pp_attn_params* p) {
  if (!p) return PP_ERR_INVALID_ARG;
  if (p->n_q_heads < 1 || p->n_kv_heads < 1) return PP_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return PP_ERR_UNSUPPORTED;
  if (p->n_q_heads % p->n_kv_heads != 0 || p->n_q_heads / p->n_kv_heads > kMaxGroup) return PP_ERR_UNSUPPORTED;
  if (p->n_kv_heads > 65535 || p->n_q_heads > 65535) return PP_ERR_UNSUPPORTED;
  if (!(p->rope_base > 0.f) || p->softmax_scale < 0.f) return PP_ERR_INVALID_ARG;
  return PP_OK;
}

}  // namespace
}  // namespace pp

extern "C" size_t pp_decode_workspace_bytes(const pp_attn_params* params, const int32_t* lengths, int32_t k) {
  if (pp::check_decode_params(params) != PP_OK || !lengths || k < 1) return 0;
  for (int32_t i = 0; i < k; ++i)
    if (lengths[i] < 1) return 0;
  return pp::decode_layout(*params, lengths, k).total_bytes;
}

extern "C" int pp_decode_step(const pp_attn_params* params, const int32_t* lengths, int32_t k,
                              const void* q_new, const void* k_new, const void* v_new, void* o,
                              void* k_cache, void* v_cache, const int64_t* cache_off, const int32_t* cache_cap,
                              void* workspace, void* host_workspace, size_t workspace_bytes, void* stream) {
  int st = pp::check_decode_params(params);
  if (st != PP_OK) return st;
  if (!lengths || k < 1 || !q_new || !k_new || !v_new || !o || !k_cache || !v_cache || !cache_off || !cache_cap ||
      !workspace || !host_workspace)
    return PP_ERR_INVALID_ARG;
  auto al = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
  if (!al(q_new) || !al(k_new) || !al(v_new) || !al(o) || !al(k_cache) || !al(v_cache) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return PP_ERR_ALIGNMENT;
  for (int32_t i = 0; i < k; ++i) {
    if (lengths[i] < 1 || cache_cap[i] <= lengths[i]) return PP_ERR_LENGTH;     // room for one more token
    if (cache_off[i] < 0) return PP_ERR_INVALID_ARG;
    if (cache_off[i] % 8 != 0) return PP_ERR_ALIGNMENT;
  }
  const pp::DecodeLayout L = pp::decode_layout(*params, lengths, k);
  if (L.n_chunks > INT32_MAX / 4) return PP_ERR_UNSUPPORTED;
  if (workspace_bytes < L.total_bytes) return PP_ERR_BUFFER_TOO_SMALL;
  int32_t* h = static_cast<int32_t*>(host_workspace);
  int64_t* h_off = reinterpret_cast<int64_t*>(h + L.T.cache_off);
  int32_t c = 0;
  for (int32_t i = 0; i < k; ++i) {
    h[L.T.chunk_ptr + i] = c;
    const int32_t n = lengths[i] + 1;                     // the new token is attended too
    for (int32_t key0 = 0; key0 < n; key0 += L.chunk_keys, ++c) {
      h[L.T.chunks + 3 * c] = i;
      h[L.T.chunks + 3 * c + 1] = key0;
      h[L.T.chunks + 3 * c + 2] = n - key0 < L.chunk_keys ? n - key0 : L.chunk_keys;
    }
    h[L.T.lengths + i] = lengths[i];
    h[L.T.cache_cap + i] = cache_cap[i];
    h_off[i] = cache_off[i];
  }
  h[L.T.chunk_ptr + k] = c;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(workspace, host_workspace, L.table_ints * sizeof(int32_t), cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return pp::note_cuda_error((int)e, "decode table upload");
  const int32_t* d_table = static_cast<const int32_t*>(workspace);
  __nv_bfloat16* q_rot = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + L.q_rot_bytes_off);
  float* partial = reinterpret_cast<float*>(static_cast<char*>(workspace) + L.partial_bytes_off);
  pp::DecodeFreq freq;
  const int half = params->head_dim / 2;
  for (int j = 0; j < 64; ++j)
    freq.inv_freq[j] = j < half ? pow((double)params->rope_base, -2.0 * j / (double)params->head_dim) : 0.0;
  const float scale = params->softmax_scale > 0.f ? params->softmax_scale : 1.0f / sqrtf((float)params->head_dim);
  const float scale_log2 = scale * 1.4426950408889634f;
  const int group = params->n_q_heads / params->n_kv_heads;
  const dim3 grid_p((unsigned)L.n_chunks, (unsigned)params->n_kv_heads), grid_c((unsigned)k, (unsigned)params->n_q_heads);
  cudaError_t le = cudaSuccess;
#define PP_DECODE_PARTIAL(DD, GG)                                                                                \
  le = pp::launch_dependent(pp::decode_partial_kernel<DD, GG>, grid_p, dim3(pp::kDecodeThreads), 0, s,           \
      (const __nv_bfloat16*)q_rot, (const __nv_bfloat16*)k_cache, (const __nv_bfloat16*)v_cache, partial, d_table, L.T, \
      params->n_q_heads, params->n_kv_heads, group, scale_log2)
#define PP_DECODE_LAUNCH(DD)                                                                                     \
  pp::decode_append_kernel<DD><<<k, pp::kDecodeThreads, 0, s>>>(                                                 \
      (const __nv_bfloat16*)q_new, (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new, q_rot,              \
      (__nv_bfloat16*)k_cache, (__nv_bfloat16*)v_cache, d_table, L.T, params->n_q_heads, params->n_kv_heads, freq); \
  if (group == 1) PP_DECODE_PARTIAL(DD, 1); else if (group == 2) PP_DECODE_PARTIAL(DD, 2);                       \
  else if (group <= 4) PP_DECODE_PARTIAL(DD, 4); else PP_DECODE_PARTIAL(DD, 8);                                  \
  if (le == cudaSuccess)                                                                                         \
    le = pp::launch_dependent(pp::decode_combine_kernel<DD>, grid_c, dim3(DD), 0, s, (const float*)partial,      \
                              (__nv_bfloat16*)o, d_table, L.T, params->n_q_heads)
  if (params->head_dim == 128) { PP_DECODE_LAUNCH(128); } else { PP_DECODE_LAUNCH(64); }
#undef PP_DECODE_LAUNCH
#undef PP_DECODE_PARTIAL
  e = le != cudaSuccess ? le : cudaGetLastError();
  return e == cudaSuccess ? PP_OK : pp::note_cuda_error((int)e, "decode kernel launch");
}
