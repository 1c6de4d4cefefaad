// C-ABI entry points that touch the device: argument validation, table upload, kernel launches.
// Algorithm 1 lines 5-8 of the prepacking paper; see include/pp.h for the contracts.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "pp_internal.h"

namespace pp {

static thread_local char g_cuda_error[256] = "";

int note_cuda_error(int cuda_error, const char* what) {
  const char* txt = cuda_error >= 0 ? cudaGetErrorString((cudaError_t)cuda_error) : "n/a";
  std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s (%d)", what, txt, cuda_error);
  return PP_ERR_CUDA;
}

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_params(const pp_attn_params* p) {
  if (!p) return PP_ERR_INVALID_ARG;
  if (p->n_q_heads < 1 || p->n_kv_heads < 1 || p->capacity < 1 || p->n_bins < 1) return PP_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return PP_ERR_UNSUPPORTED;
  if (p->n_q_heads % p->n_kv_heads != 0) return PP_ERR_UNSUPPORTED;
  if (p->n_kv_heads > 65535) return PP_ERR_UNSUPPORTED;
  if (!(p->rope_base > 0.f) || p->softmax_scale < 0.f) return PP_ERR_INVALID_ARG;
  return PP_OK;
}

// The kernels are built for sm_100a only.
int check_device() {
  static thread_local int cached_dev = -1;
  static thread_local int cached_status = PP_OK;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return note_cuda_error((int)e, "cudaGetDevice");
  if (dev == cached_dev) return cached_status;
  int major = 0;
  e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (e != cudaSuccess) return note_cuda_error((int)e, "cudaDeviceGetAttribute");
  cached_dev = dev;
  cached_status = (major == 10) ? PP_OK : PP_ERR_UNSUPPORTED;
  return cached_status;
}

}  // namespace
}  // namespace pp

extern "C" const char* pp_last_cuda_error(void) { return pp::g_cuda_error; }

extern "C" size_t pp_prefill_workspace_bytes(const pp_attn_params* params, int32_t k) {
  if (pp::check_params(params) != PP_OK || k < 1) return 0;
  return sizeof(int32_t) * pp::prefill_table_ints(params->n_bins, params->capacity, k);
}

extern "C" int pp_prefill_attention(const pp_attn_params* params, const int32_t* bin_seg_ptr,
                                    const int32_t* seg_start, const int32_t* seg_len, int32_t k,
                                    void* q, void* k_, const void* v, void* o, void* workspace,
                                    void* host_workspace, size_t workspace_bytes,
                                    int32_t* device_status, void* stream) {
  int st = pp::check_params(params);
  if (st != PP_OK) return st;
  const int flags = params->flags;
  const bool do_rope = !(flags & PP_FLAG_SKIP_ROPE);
  const bool do_attn = !(flags & PP_FLAG_ROPE_ONLY);
  if (!q || !k_ || !workspace || !host_workspace) return PP_ERR_INVALID_ARG;
  if (do_attn && (!v || !o)) return PP_ERR_INVALID_ARG;
  st = pp::validate_packing(params->n_bins, params->capacity, bin_seg_ptr, seg_start, seg_len, k);
  if (st != PP_OK) return st;
  if (!pp::aligned16(q) || !pp::aligned16(k_) || !pp::aligned16(workspace) ||
      (do_attn && (!pp::aligned16(v) || !pp::aligned16(o))))
    return PP_ERR_ALIGNMENT;
  const size_t need = pp_prefill_workspace_bytes(params, k);
  if (workspace_bytes < need) return PP_ERR_BUFFER_TOO_SMALL;
  if ((st = pp::check_device()) != PP_OK) return st;

  pp::TableLayout L;
  st = pp::build_prefill_tables(params->n_bins, params->capacity, bin_seg_ptr, seg_start, seg_len, k,
                                params->n_q_heads / params->n_kv_heads,
                                static_cast<int32_t*>(host_workspace), workspace_bytes / sizeof(int32_t), &L);
  if (st != PP_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(workspace, host_workspace, sizeof(int32_t) * (size_t)L.total_ints,
                                  cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return pp::note_cuda_error((int)e, "table upload");
  int32_t* d_table = static_cast<int32_t*>(workspace);
  if (do_rope) {
    st = pp::launch_rope(*params, d_table, L, q, q, k_, stream);
    if (st != PP_OK) return st;
  }
  if (do_attn) {
    st = pp::launch_attention(*params, d_table, L, q, k_, v, o, nullptr, device_status, stream);
    if (st != PP_OK) return st;
  }
  return PP_OK;
}

// ------------------------------------------------------------------------------------------
// Fused path: rotation of K + UNPACK in one pass, Q rotated inside the attention kernel
// ------------------------------------------------------------------------------------------
namespace pp {
namespace {
struct FusedLayout {
  size_t table_ints;      // prefill table (segment table + work list)
  size_t off_true_len, off_cap, off_cache_off;   // int32 offsets of the per-segment arrays
  size_t upload_ints;     // ints copied from the host staging buffer
  size_t off_rope_bytes;  // byte offset of the cos/sin table (device only)
  size_t total_bytes;
};
FusedLayout fused_layout(const pp_attn_params& p, int32_t k) {
  auto up4 = [](size_t x) { return (x + 3) & ~size_t(3); };
  FusedLayout f;
  f.table_ints = prefill_table_ints(p.n_bins, p.capacity, k);
  f.off_true_len = up4(f.table_ints);
  f.off_cap = f.off_true_len + up4((size_t)k);
  f.off_cache_off = f.off_cap + up4((size_t)k);          // multiple of 4 ints: 16-byte aligned int64 data
  f.upload_ints = f.off_cache_off + 2 * (size_t)k;
  f.off_rope_bytes = (f.upload_ints * sizeof(int32_t) + 255) & ~size_t(255);
  f.total_bytes = f.off_rope_bytes + (size_t)p.capacity * (p.head_dim / 2) * sizeof(float) * 2;
  return f;
}
}  // namespace
}  // namespace pp

extern "C" size_t pp_prefill_fused_workspace_bytes(const pp_attn_params* params, int32_t k) {
  if (pp::check_params(params) != PP_OK || k < 1) return 0;
  return pp::fused_layout(*params, k).total_bytes;
}

extern "C" int pp_prefill_fused(const pp_attn_params* params, const int32_t* bin_seg_ptr,
                                const int32_t* seg_start, const int32_t* seg_len, const int32_t* seg_prompt,
                                int32_t k, const int32_t* lengths, const void* q, void* k_,
                                const void* v, void* o, void* k_cache, void* v_cache, const int64_t* cache_off, const int32_t* cache_cap,
                                void* workspace, void* host_workspace, size_t workspace_bytes,
                                int32_t* device_status, void* stream) {
  int st = pp::check_params(params);
  if (st != PP_OK) return st;
  if (!q || !k_ || !v || !o || !k_cache || !v_cache || !cache_off || !cache_cap || !seg_prompt || !lengths ||
      !workspace || !host_workspace)
    return PP_ERR_INVALID_ARG;
  st = pp::validate_packing(params->n_bins, params->capacity, bin_seg_ptr, seg_start, seg_len, k);
  if (st != PP_OK) return st;
  if (!pp::aligned16(q) || !pp::aligned16(k_) || !pp::aligned16(v) || !pp::aligned16(o) ||
      !pp::aligned16(k_cache) || !pp::aligned16(v_cache) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return PP_ERR_ALIGNMENT;
  const pp::FusedLayout f = pp::fused_layout(*params, k);
  if (workspace_bytes < f.total_bytes) return PP_ERR_BUFFER_TOO_SMALL;
  int32_t* h = static_cast<int32_t*>(host_workspace);
  int64_t* h_coff = reinterpret_cast<int64_t*>(h + f.off_cache_off);
  for (int32_t s = 0; s < k; ++s) {
    const int32_t i = seg_prompt[s];
    if (i < 0 || i >= k) return PP_ERR_INVALID_ARG;
    if (lengths[i] < 1 || lengths[i] > seg_len[s] || cache_cap[i] < lengths[i]) return PP_ERR_LENGTH;
    if (cache_off[i] < 0) return PP_ERR_INVALID_ARG;
    if (cache_off[i] % 8 != 0) return PP_ERR_ALIGNMENT;
    h[f.off_true_len + s] = lengths[i];
    h[f.off_cap + s] = cache_cap[i];
    h_coff[s] = cache_off[i];
  }
  if ((st = pp::check_device()) != PP_OK) return st;
  pp::TableLayout L;
  st = pp::build_prefill_tables(params->n_bins, params->capacity, bin_seg_ptr, seg_start, seg_len, k,
                                params->n_q_heads / params->n_kv_heads, h, f.table_ints, &L);
  if (st != PP_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(workspace, host_workspace, sizeof(int32_t) * f.upload_ints,
                                  cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return pp::note_cuda_error((int)e, "table upload");
  int32_t* d_table = static_cast<int32_t*>(workspace);
  void* rope_table = static_cast<char*>(workspace) + f.off_rope_bytes;
  if ((st = pp::launch_rope_table(*params, rope_table, stream)) != PP_OK) return st;
  if (!(params->flags & PP_FLAG_SKIP_ROPE)) {       // flag: k_ is rotated and the caches are filled already
    st = pp::launch_rope_unpack(*params, d_table, L, (int32_t)f.off_true_len, (int32_t)f.off_cap,
                                (int32_t)f.off_cache_off, rope_table, k_, v, k_cache, v_cache, stream);
    if (st != PP_OK) return st;
  }
  if (params->flags & PP_FLAG_ROPE_ONLY) return PP_OK;
  // the attention kernel rotates every Q tile in shared memory, so Q is read from HBM once
  return pp::launch_attention(*params, d_table, L, q, k_, v, o, rope_table, device_status, stream);
}

extern "C" int pp_selftest_bounded_wait(int32_t* device_status, uint32_t limit_ms, void* stream) {
  if (!device_status || limit_ms == 0 || limit_ms > 1000) return PP_ERR_INVALID_ARG;
  int st = pp::check_device();
  if (st != PP_OK) return st;
  return pp::launch_bounded_wait_selftest(device_status, (uint64_t)limit_ms * 1000000ull, stream);
}

extern "C" size_t pp_unpack_workspace_bytes(int32_t k) { return pp::unpack_table_bytes(k); }

extern "C" int pp_unpack_kv(const pp_attn_params* params, const int32_t* bin_of, const int32_t* off_of,
                            const int32_t* lengths, int32_t k, const void* k_rot, const void* v,
                            void* k_cache, void* v_cache, const int64_t* cache_off,
                            const int32_t* cache_cap, void* workspace, void* host_workspace,
                            size_t workspace_bytes, void* stream) {
  int st = pp::check_params(params);
  if (st != PP_OK) return st;
  if (!bin_of || !off_of || !lengths || k < 1 || !k_rot || !v || !k_cache || !v_cache || !cache_off ||
      !cache_cap || !workspace || !host_workspace)
    return PP_ERR_INVALID_ARG;
  if (!pp::aligned16(k_rot) || !pp::aligned16(v) || !pp::aligned16(k_cache) || !pp::aligned16(v_cache) ||
      !pp::aligned16(workspace))
    return PP_ERR_ALIGNMENT;
  if (workspace_bytes < pp::unpack_table_bytes(k)) return PP_ERR_BUFFER_TOO_SMALL;
  int64_t total = 0;
  for (int32_t i = 0; i < k; ++i) {
    if (lengths[i] < 1 || cache_cap[i] < lengths[i]) return PP_ERR_LENGTH;
    if (bin_of[i] < 0 || bin_of[i] >= params->n_bins || off_of[i] < 0 ||
        (int64_t)off_of[i] + lengths[i] > params->capacity)
      return PP_ERR_INVALID_ARG;
    if (cache_off[i] < 0) return PP_ERR_INVALID_ARG;
    if (cache_off[i] % 8 != 0) return PP_ERR_ALIGNMENT;
    total += lengths[i];
    if (total > INT32_MAX) return PP_ERR_UNSUPPORTED;
  }
  if ((st = pp::check_device()) != PP_OK) return st;

  auto up4 = [](int64_t x) { return (x + 3) & ~int64_t(3); };
  int32_t* t = static_cast<int32_t*>(host_workspace);
  std::memset(t, 0, 16);
  t[0] = k;
  int32_t* prefix = t + 4;
  int32_t* h_bin = prefix + up4(k + 1);
  int32_t* h_off = h_bin + up4(k);
  int32_t* h_cap = h_off + up4(k);
  int64_t* h_coff = reinterpret_cast<int64_t*>(h_cap + up4(k));
  prefix[0] = 0;
  for (int32_t i = 0; i < k; ++i) {
    prefix[i + 1] = prefix[i] + lengths[i];
    h_bin[i] = bin_of[i];
    h_off[i] = off_of[i];
    h_cap[i] = cache_cap[i];
    h_coff[i] = cache_off[i];
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(workspace, host_workspace, pp::unpack_table_bytes(k),
                                  cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return pp::note_cuda_error((int)e, "unpack table upload");
  return pp::launch_unpack(*params, static_cast<const int32_t*>(workspace), k, total, k_rot, v, k_cache,
                           v_cache, stream);
}

// ------------------------------------------------------------------------------------------
// Whole path from host buffers
// ------------------------------------------------------------------------------------------
namespace pp {
namespace {

size_t up256(size_t x) { return (x + 255) & ~size_t(255); }

constexpr int kHostGroups = 4;     // groups of bins pp_prefill_host pipelines over its own streams

struct ArenaPlan {
  size_t q, k, v, o, kc, vc, ws_attn, ws_attn_stride, ws_unpack, ws_unpack_stride, status, total;
};

ArenaPlan plan_arena(const pp_attn_params& p, int32_t n_bins, int32_t capacity, int64_t total_tokens, int32_t k) {
  ArenaPlan a{};
  const size_t rows = (size_t)n_bins * capacity;
  const size_t qb = rows * p.n_q_heads * p.head_dim * 2, kb = rows * p.n_kv_heads * p.head_dim * 2;
  const size_t cb = (size_t)total_tokens * p.n_kv_heads * p.head_dim * 2;
  size_t off = 0;
  a.q = off; off += up256(qb);
  a.k = off; off += up256(kb);
  a.v = off; off += up256(kb);
  a.o = off; off += up256(qb);
  a.kc = off; off += up256(cb);
  a.vc = off; off += up256(cb);
  // one table workspace per group (each sized for the whole batch: they are small)
  a.ws_attn_stride = up256(sizeof(int32_t) * prefill_table_ints(n_bins, capacity, k));
  a.ws_attn = off; off += kHostGroups * a.ws_attn_stride;
  a.ws_unpack_stride = up256(unpack_table_bytes(k));
  a.ws_unpack = off; off += kHostGroups * a.ws_unpack_stride;
  a.status = off; off += 256;
  a.total = off;
  return a;
}

// Streams and events pp_prefill_host pipelines over, created on first use per device.
struct HostPipe {
  cudaStream_t stream[kHostGroups] = {};
  cudaEvent_t done[kHostGroups] = {};
  cudaEvent_t start = nullptr;
  int device = -1;
};
int host_pipe(HostPipe** out) {
  static thread_local HostPipe pipe;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return note_cuda_error((int)e, "cudaGetDevice");
  if (pipe.device != dev) {
    for (int g = 0; g < kHostGroups; ++g) {
      if ((e = cudaStreamCreateWithFlags(&pipe.stream[g], cudaStreamNonBlocking)) != cudaSuccess)
        return note_cuda_error((int)e, "cudaStreamCreate");
      if ((e = cudaEventCreateWithFlags(&pipe.done[g], cudaEventDisableTiming)) != cudaSuccess)
        return note_cuda_error((int)e, "cudaEventCreate");
    }
    if ((e = cudaEventCreateWithFlags(&pipe.start, cudaEventDisableTiming)) != cudaSuccess)
      return note_cuda_error((int)e, "cudaEventCreate");
    pipe.device = dev;
  }
  *out = &pipe;
  return PP_OK;
}

}  // namespace
}  // namespace pp

extern "C" size_t pp_prefill_host_arena_bytes(const pp_attn_params* params, const int32_t* lengths, int32_t k) {
  if (!params || !lengths || k < 1) return 0;
  if (params->head_dim != 64 && params->head_dim != 128) return 0;
  int32_t r = 0, cap = 0;
  if (pp_pack(lengths, k, 0, &r, &cap, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr) != PP_OK) return 0;
  int64_t total = 0;
  for (int32_t i = 0; i < k; ++i) total += lengths[i];
  return pp::plan_arena(*params, r, cap, total, k).total;
}

extern "C" int pp_prefill_host(pp_attn_params* params, const int32_t* lengths, int32_t k,
                               const void* q_host, const void* k_host, const void* v_host, void* o_host,
                               void* k_cache_host, void* v_cache_host, void* arena, size_t arena_bytes,
                               void* stream) {
  if (!params || !lengths || k < 1 || !q_host || !k_host || !v_host || !o_host || !k_cache_host ||
      !v_cache_host || !arena)
    return PP_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(arena) & 255u) return PP_ERR_ALIGNMENT;
  try {
    std::vector<int32_t> bin_seg_ptr(k + 1), seg_prompt(k), seg_start(k), seg_len(k), bin_of(k), off_of(k);
    int32_t r = 0, cap = 0;
    int st = pp_pack(lengths, k, 0, &r, &cap, bin_seg_ptr.data(), seg_prompt.data(), seg_start.data(),
                     seg_len.data(), bin_of.data(), off_of.data());
    if (st != PP_OK) return st;
    params->capacity = cap;
    params->n_bins = r;
    params->flags = 0;
    if ((st = pp::check_params(params)) != PP_OK) return st;
    int64_t total = 0;
    std::vector<int64_t> tok_off(k), cache_off(k);
    for (int32_t i = 0; i < k; ++i) {
      tok_off[i] = total;
      cache_off[i] = total * params->n_kv_heads * params->head_dim;
      total += lengths[i];
    }
    const pp::ArenaPlan a = pp::plan_arena(*params, r, cap, total, k);
    if (arena_bytes < a.total) return PP_ERR_BUFFER_TOO_SMALL;
    char* base = static_cast<char*>(arena);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t q_row = (size_t)params->n_q_heads * params->head_dim * 2;
    const size_t kv_row = (size_t)params->n_kv_heads * params->head_dim * 2;
    cudaError_t e;
#define PP_TRY(call, what) do { e = (call); if (e != cudaSuccess) return pp::note_cuda_error((int)e, what); } while (0)
    // The bins are cut into up to kHostGroups groups, each with its own stream: uploads of one group
    // overlap the kernels of another and the downloads of a third (PCIe is full duplex), instead of
    // all uploads, then all kernels, then all downloads.
    pp::HostPipe* pipe = nullptr;
    if ((st = pp::host_pipe(&pipe)) != PP_OK) return st;
    // Only worth it when the per-prompt copies are large: with many small prompts the copies are
    // latency-bound and one stream with two large cache downloads is faster.
    const size_t mean_prompt_bytes = (size_t)(total / k) * (q_row + 2 * kv_row);
    const int n_groups = mean_prompt_bytes >= (size_t(1) << 20) ? std::min<int>(pp::kHostGroups, r) : 1;
    PP_TRY(cudaMemsetAsync(base + a.status, 0, 4, s), "memset status");
    PP_TRY(cudaEventRecord(pipe->start, s), "event record");
    // host staging for the tables of every group (pageable: the copies stage them before returning)
    std::vector<std::vector<int32_t>> h_ws_attn(n_groups);
    std::vector<std::vector<int64_t>> h_ws_unpack(n_groups);
    std::vector<int32_t> g_ptr, g_bin_of, g_off_of, g_len, g_ids;
    std::vector<int64_t> g_cache_off;
    for (int g = 0; g < n_groups; ++g) {
      const int32_t b0 = (int32_t)((int64_t)r * g / n_groups), b1 = (int32_t)((int64_t)r * (g + 1) / n_groups);
      const int32_t s0 = bin_seg_ptr[b0], s1 = bin_seg_ptr[b1], kg = s1 - s0;
      cudaStream_t sg = pipe->stream[g];
      PP_TRY(cudaStreamWaitEvent(sg, pipe->start, 0), "stream wait");
      // TENSORIZE: zero the group's packed rows (padding rows must be finite), then one copy per prompt
      const size_t rows0 = (size_t)b0 * cap, nrows = (size_t)(b1 - b0) * cap;
      PP_TRY(cudaMemsetAsync(base + a.q + rows0 * q_row, 0, nrows * q_row, sg), "memset packed q");
      PP_TRY(cudaMemsetAsync(base + a.k + rows0 * kv_row, 0, nrows * kv_row, sg), "memset packed k");
      PP_TRY(cudaMemsetAsync(base + a.v + rows0 * kv_row, 0, nrows * kv_row, sg), "memset packed v");
      g_ptr.assign(bin_seg_ptr.begin() + b0, bin_seg_ptr.begin() + b1 + 1);
      for (int32_t& x : g_ptr) x -= s0;
      g_ids.assign(seg_prompt.begin() + s0, seg_prompt.begin() + s1);       // the group's prompts
      g_bin_of.resize(kg); g_off_of.resize(kg); g_len.resize(kg); g_cache_off.resize(kg);
      for (int32_t j = 0; j < kg; ++j) {
        const int32_t i = g_ids[j];
        g_bin_of[j] = bin_of[i] - b0;
        g_off_of[j] = off_of[i];
        g_len[j] = lengths[i];
        g_cache_off[j] = cache_off[i];
        const size_t row = (size_t)bin_of[i] * cap + off_of[i];
        PP_TRY(cudaMemcpyAsync(base + a.q + row * q_row, (const char*)q_host + tok_off[i] * q_row,
                               lengths[i] * q_row, cudaMemcpyHostToDevice, sg), "H2D q");
        PP_TRY(cudaMemcpyAsync(base + a.k + row * kv_row, (const char*)k_host + tok_off[i] * kv_row,
                               lengths[i] * kv_row, cudaMemcpyHostToDevice, sg), "H2D k");
        PP_TRY(cudaMemcpyAsync(base + a.v + row * kv_row, (const char*)v_host + tok_off[i] * kv_row,
                               lengths[i] * kv_row, cudaMemcpyHostToDevice, sg), "H2D v");
      }
      pp_attn_params gp = *params;
      gp.n_bins = b1 - b0;
      h_ws_attn[g].resize(pp::prefill_table_ints(gp.n_bins, cap, kg));
      h_ws_unpack[g].resize((pp::unpack_table_bytes(kg) + 7) / 8);
      st = pp_prefill_attention(&gp, g_ptr.data(), seg_start.data() + s0, seg_len.data() + s0, kg,
                                base + a.q + rows0 * q_row, base + a.k + rows0 * kv_row, base + a.v + rows0 * kv_row,
                                base + a.o + rows0 * q_row, base + a.ws_attn + g * a.ws_attn_stride,
                                h_ws_attn[g].data(), h_ws_attn[g].size() * sizeof(int32_t),
                                reinterpret_cast<int32_t*>(base + a.status), sg);
      if (st != PP_OK) return st;
      st = pp_unpack_kv(&gp, g_bin_of.data(), g_off_of.data(), g_len.data(), kg, base + a.k + rows0 * kv_row,
                        base + a.v + rows0 * kv_row, base + a.kc, base + a.vc, g_cache_off.data(), g_len.data(),
                        base + a.ws_unpack + g * a.ws_unpack_stride, h_ws_unpack[g].data(),
                        h_ws_unpack[g].size() * 8, sg);
      if (st != PP_OK) return st;
      // UNPACK to the host, prompt by prompt (caches and O are in original order there); a single
      // group takes the caches in two large copies instead
      if (n_groups == 1) {
        const size_t cache_bytes = (size_t)total * kv_row;
        PP_TRY(cudaMemcpyAsync(k_cache_host, base + a.kc, cache_bytes, cudaMemcpyDeviceToHost, sg), "D2H k cache");
        PP_TRY(cudaMemcpyAsync(v_cache_host, base + a.vc, cache_bytes, cudaMemcpyDeviceToHost, sg), "D2H v cache");
      }
      for (int32_t j = 0; j < kg; ++j) {
        const int32_t i = g_ids[j];
        const size_t row = (size_t)bin_of[i] * cap + off_of[i];
        const size_t cbytes = (size_t)lengths[i] * kv_row;
        if (n_groups > 1) {
          PP_TRY(cudaMemcpyAsync((char*)k_cache_host + cache_off[i] * 2, base + a.kc + cache_off[i] * 2, cbytes,
                                 cudaMemcpyDeviceToHost, sg), "D2H k cache");
          PP_TRY(cudaMemcpyAsync((char*)v_cache_host + cache_off[i] * 2, base + a.vc + cache_off[i] * 2, cbytes,
                                 cudaMemcpyDeviceToHost, sg), "D2H v cache");
        }
        PP_TRY(cudaMemcpyAsync((char*)o_host + tok_off[i] * q_row, base + a.o + row * q_row, lengths[i] * q_row,
                               cudaMemcpyDeviceToHost, sg), "D2H o");
      }
      PP_TRY(cudaEventRecord(pipe->done[g], sg), "event record");
      PP_TRY(cudaStreamWaitEvent(s, pipe->done[g], 0), "stream wait");
    }
    int32_t status = 0;
    PP_TRY(cudaMemcpyAsync(&status, base + a.status, 4, cudaMemcpyDeviceToHost, s), "D2H status");
    PP_TRY(cudaStreamSynchronize(s), "stream synchronize");
#undef PP_TRY
    return status == 0 ? PP_OK : PP_ERR_DEVICE_TIMEOUT;
  } catch (const std::bad_alloc&) {
    return PP_ERR_NO_MEMORY;
  }
}
