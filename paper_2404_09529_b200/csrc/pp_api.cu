// C-ABI entry points that touch the device: argument validation, table upload, kernel launches.
// Algorithm 1 (TENSORIZE to UNPACK) of the prepacking paper; see include/pp.h for the contracts.
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

// What an entry point does with its tables. pp_prefill_host splits a call in two so that the small
// table uploads go in front of its large data uploads: a table upload that is queued behind another
// stream's bulk copy would hold its kernels back for milliseconds. Never reachable through
// pp_attn_params.flags: the public entry points reject every bit they do not document.
enum class TableStep { kUploadAndLaunch, kUploadOnly, kLaunchOnly };
constexpr int kPublicFlags = PP_FLAG_SKIP_ROPE | PP_FLAG_ROPE_ONLY | PP_FLAG_KEEP_ROPE_TABLE;

int check_params(const pp_attn_params* p) {
  if (!p) return PP_ERR_INVALID_ARG;
  if (p->n_q_heads < 1 || p->n_kv_heads < 1 || p->capacity < 1 || p->n_bins < 1) return PP_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return PP_ERR_UNSUPPORTED;
  if (p->n_q_heads % p->n_kv_heads != 0) return PP_ERR_UNSUPPORTED;
  if (p->n_kv_heads > 65535) return PP_ERR_UNSUPPORTED;
  if (!(p->rope_base > 0.f) || p->softmax_scale < 0.f) return PP_ERR_INVALID_ARG;
  if (p->flags & ~kPublicFlags) return PP_ERR_INVALID_ARG;
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
  return sizeof(int32_t) * pp::prefill_table_ints(params->n_bins, params->capacity, k,
                                                  params->n_q_heads / params->n_kv_heads);
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
  f.table_ints = prefill_table_ints(p.n_bins, p.capacity, k, p.n_q_heads / p.n_kv_heads);
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

extern "C" size_t pp_prefill_fused_host_bytes(const pp_attn_params* params, int32_t k) {
  if (pp::check_params(params) != PP_OK || k < 1) return 0;
  return sizeof(int32_t) * pp::fused_layout(*params, k).upload_ints;
}

namespace pp {
namespace {
// The kernels of the fused path on tables that are (or will be, in stream order) in `workspace`.
int launch_fused_kernels(const pp_attn_params& p, const TableLayout& L, const FusedLayout& f, const void* q,
                         void* k_, const void* v, void* o, void* k_cache, void* v_cache, void* workspace,
                         int32_t* device_status, void* stream) {
  int st;
  int32_t* d_table = static_cast<int32_t*>(workspace);
  void* rope_table = static_cast<char*>(workspace) + f.off_rope_bytes;
  if (!(p.flags & PP_FLAG_KEEP_ROPE_TABLE)) {
    if ((st = launch_rope_table(p, rope_table, stream)) != PP_OK) return st;
  }
  if (!(p.flags & PP_FLAG_SKIP_ROPE)) {       // flag: k_ is rotated and the caches are filled already
    st = launch_rope_unpack(p, d_table, L, (int32_t)f.off_true_len, (int32_t)f.off_cap,
                            (int32_t)f.off_cache_off, rope_table, k_, v, k_cache, v_cache, stream);
    if (st != PP_OK) return st;
  }
  if (p.flags & PP_FLAG_ROPE_ONLY) return PP_OK;
  // the attention kernel rotates every Q tile in shared memory, so Q is read from HBM once
  return launch_attention(p, d_table, L, q, k_, v, o, rope_table, device_status, stream);
}

// pp_prefill_fused, optionally cut in two: kUploadOnly validates, builds and uploads the tables,
// launches nothing and hands the table layout back through `layout`; kLaunchOnly takes that layout,
// touches neither the host staging buffer (its upload may still be in flight) nor the arguments
// already checked, and launches the kernels on the tables in `workspace`.
int prefill_fused_impl(const pp_attn_params* params, const int32_t* bin_seg_ptr, const int32_t* seg_start,
                       const int32_t* seg_len, const int32_t* seg_prompt, int32_t k, const int32_t* lengths,
                       const void* q, void* k_, const void* v, void* o, void* k_cache, void* v_cache,
                       const int64_t* cache_off, const int32_t* cache_cap, void* workspace,
                       void* host_workspace, size_t workspace_bytes, int32_t* device_status, void* stream,
                       TableStep step, TableLayout* layout) {
  int st = check_params(params);
  if (st != PP_OK) return st;
  if (step == TableStep::kLaunchOnly) {
    const FusedLayout f = fused_layout(*params, k);
    return launch_fused_kernels(*params, *layout, f, q, k_, v, o, k_cache, v_cache, workspace, device_status, stream);
  }
  if (!q || !k_ || !v || !o || !k_cache || !v_cache || !cache_off || !cache_cap || !seg_prompt || !lengths ||
      !workspace || !host_workspace)
    return PP_ERR_INVALID_ARG;
  st = validate_packing(params->n_bins, params->capacity, bin_seg_ptr, seg_start, seg_len, k);
  if (st != PP_OK) return st;
  if (!aligned16(q) || !aligned16(k_) || !aligned16(v) || !aligned16(o) ||
      !aligned16(k_cache) || !aligned16(v_cache) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return PP_ERR_ALIGNMENT;
  const FusedLayout f = fused_layout(*params, k);
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
  if ((st = check_device()) != PP_OK) return st;
  TableLayout L;
  st = build_prefill_tables(params->n_bins, params->capacity, bin_seg_ptr, seg_start, seg_len, k,
                            params->n_q_heads / params->n_kv_heads, h, f.table_ints, &L);
  if (st != PP_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(workspace, host_workspace, sizeof(int32_t) * f.upload_ints,
                                  cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return note_cuda_error((int)e, "table upload");
  if (layout) *layout = L;
  if (step == TableStep::kUploadOnly) return PP_OK;
  return launch_fused_kernels(*params, L, f, q, k_, v, o, k_cache, v_cache, workspace, device_status, stream);
}
}  // namespace
}  // namespace pp

extern "C" int pp_prefill_fused(const pp_attn_params* params, const int32_t* bin_seg_ptr,
                                const int32_t* seg_start, const int32_t* seg_len, const int32_t* seg_prompt,
                                int32_t k, const int32_t* lengths, const void* q, void* k_,
                                const void* v, void* o, void* k_cache, void* v_cache, const int64_t* cache_off, const int32_t* cache_cap,
                                void* workspace, void* host_workspace, size_t workspace_bytes,
                                int32_t* device_status, void* stream) {
  return pp::prefill_fused_impl(params, bin_seg_ptr, seg_start, seg_len, seg_prompt, k, lengths, q, k_, v, o,
                                k_cache, v_cache, cache_off, cache_cap, workspace, host_workspace, workspace_bytes,
                                device_status, stream, pp::TableStep::kUploadAndLaunch, nullptr);
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

constexpr int kHostGroupsMax = 16;     // groups of prompts pp_prefill_host can pipeline over its own streams
constexpr int kHostGroupsDefault = 8;
thread_local int g_host_groups = 0;    // pp_prefill_host_groups(); 0 = choose by batch size

// How pp_prefill_host cuts a batch: contiguous ranges of prompts (original order) with about equal
// token counts, each packed on its own with the batch-wide capacity, so that every tensor of a
// group is one contiguous range on the host.
struct HostGroup {
  int32_t i0 = 0, i1 = 0;          // prompts [i0, i1)
  int64_t t0 = 0, t1 = 0;          // tokens [t0, t1)
  int32_t bin0 = 0, n_bins = 0;    // bins [bin0, bin0 + n_bins) of the packed buffers
  std::vector<int32_t> bin_seg_ptr, seg_prompt, seg_start, seg_len, bin_of, off_of;
};
struct HostPlan {
  int32_t capacity = 0, n_bins = 0;
  int64_t total_tokens = 0;
  std::vector<HostGroup> groups;
  // arena offsets (bytes)
  size_t q = 0, k = 0, v = 0, o = 0, q_tok = 0, k_tok = 0, v_tok = 0, o_tok = 0, kc = 0, vc = 0;
  size_t ws = 0, ws_stride = 0, map = 0, map_stride = 0;
  size_t status = 0, total = 0;
};

int plan_host(const pp_attn_params& p, const int32_t* lengths, int32_t k, HostPlan* out) {
  HostPlan& h = *out;
  int32_t m = 0;
  for (int32_t i = 0; i < k; ++i) {
    if (lengths[i] < 1) return PP_ERR_LENGTH;
    m = std::max(m, lengths[i]);
    h.total_tokens += lengths[i];
  }
  h.capacity = m;
  const size_t q_row = (size_t)p.n_q_heads * p.head_dim * 2, kv_row = (size_t)p.n_kv_heads * p.head_dim * 2;
  // pipelining pays once the transfers are tens of megabytes; small batches stay in one group
  const size_t batch_bytes = (size_t)h.total_tokens * (q_row + 2 * kv_row);
  int n_groups = batch_bytes >= (size_t(32) << 20) ? kHostGroupsDefault : 1;
  if (g_host_groups > 0) n_groups = g_host_groups;
  n_groups = std::min<int>(n_groups, k);
  h.groups.resize(n_groups);
  int32_t i = 0;
  int64_t t = 0;
  for (int g = 0; g < n_groups; ++g) {
    HostGroup& G = h.groups[g];
    G.i0 = i;
    G.t0 = t;
    const int64_t target = h.total_tokens * (g + 1) / n_groups;
    // at least one prompt per group, and leave at least one for each group after this one
    while (i < k - (n_groups - 1 - g) && (i == G.i0 || t + lengths[i] <= target || g == n_groups - 1)) t += lengths[i++];
    G.i1 = i;
    G.t1 = t;
    const int32_t kg = G.i1 - G.i0;
    G.bin_seg_ptr.resize(kg + 1); G.seg_prompt.resize(kg); G.seg_start.resize(kg); G.seg_len.resize(kg);
    G.bin_of.resize(kg); G.off_of.resize(kg);
    int32_t r = 0, cap = 0;
    const int st = pp_pack(lengths + G.i0, kg, m, &r, &cap, G.bin_seg_ptr.data(), G.seg_prompt.data(),
                           G.seg_start.data(), G.seg_len.data(), G.bin_of.data(), G.off_of.data());
    if (st != PP_OK) return st;
    G.bin0 = h.n_bins;
    G.n_bins = r;
    h.n_bins += r;
  }
  const size_t rows = (size_t)h.n_bins * m;
  const size_t T = (size_t)h.total_tokens;
  size_t off = 0;
  h.q = off; off += up256(rows * q_row);
  h.k = off; off += up256(rows * kv_row);
  h.v = off; off += up256(rows * kv_row);
  h.o = off; off += up256(rows * q_row);
  h.q_tok = off; off += up256(T * q_row);
  h.k_tok = off; off += up256(T * kv_row);
  h.v_tok = off; off += up256(T * kv_row);
  h.o_tok = off; off += up256(T * q_row);
  h.kc = off; off += up256(T * kv_row);
  h.vc = off; off += up256(T * kv_row);
  // per-group workspace of the fused call, each sized for the whole batch (they are small)
  pp_attn_params whole = p;
  whole.capacity = m;
  whole.n_bins = h.n_bins;
  h.ws_stride = up256(fused_layout(whole, k).total_bytes);
  h.ws = off; off += n_groups * h.ws_stride;
  h.map_stride = up256(sizeof(int64_t) * (2 * (size_t)k + 1 + (size_t)h.n_bins));
  h.map = off; off += n_groups * h.map_stride;
  h.status = off; off += 256;
  h.total = off;
  return PP_OK;
}

// Streams and events pp_prefill_host pipelines over, created on first use per device.
struct HostPipe {
  cudaStream_t stream[kHostGroupsMax] = {};
  cudaEvent_t done[kHostGroupsMax] = {};
  cudaEvent_t start = nullptr;
  void* staging[kHostGroupsMax] = {};        // pinned host staging for each group's tables
  size_t staging_bytes[kHostGroupsMax] = {};
  int device = -1;
};
// Pinned staging of at least `bytes` for group g (kept and grown across calls; every call ends with a
// synchronize, so a buffer is never reused while a copy still reads it).
int host_staging(HostPipe* pipe, int g, size_t bytes, void** out) {
  if (pipe->staging_bytes[g] < bytes) {
    if (pipe->staging[g]) cudaFreeHost(pipe->staging[g]);
    pipe->staging[g] = nullptr;
    pipe->staging_bytes[g] = 0;
    const size_t want = (bytes + (size_t(1) << 16)) & ~((size_t(1) << 16) - 1);
    const cudaError_t e = cudaHostAlloc(&pipe->staging[g], want, cudaHostAllocDefault);
    if (e != cudaSuccess) return note_cuda_error((int)e, "cudaHostAlloc");
    pipe->staging_bytes[g] = want;
  }
  *out = pipe->staging[g];
  return PP_OK;
}
int host_pipe(HostPipe** out) {
  static thread_local HostPipe pipe;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return note_cuda_error((int)e, "cudaGetDevice");
  if (pipe.device != dev) {
    // first use on this device (or a call that failed half-way): drop whatever an earlier device or
    // attempt left behind. Handles are destroyed with the device they were made on current.
    if (pipe.device >= 0 && cudaSetDevice(pipe.device) != cudaSuccess) (void)cudaGetLastError();
    for (int g = 0; g < kHostGroupsMax; ++g) {
      if (pipe.stream[g]) { cudaStreamDestroy(pipe.stream[g]); pipe.stream[g] = nullptr; }
      if (pipe.done[g]) { cudaEventDestroy(pipe.done[g]); pipe.done[g] = nullptr; }
    }
    if (pipe.start) { cudaEventDestroy(pipe.start); pipe.start = nullptr; }
    if (pipe.device >= 0 && (e = cudaSetDevice(dev)) != cudaSuccess) return note_cuda_error((int)e, "cudaSetDevice");
    pipe.device = -1;
    for (int g = 0; g < kHostGroupsMax; ++g) {
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

extern "C" int32_t pp_prefill_host_groups(int32_t n_groups) {
  const int32_t before = pp::g_host_groups;
  if (n_groups >= 0 && n_groups <= pp::kHostGroupsMax) pp::g_host_groups = n_groups;
  return before;
}

extern "C" size_t pp_prefill_host_arena_bytes(const pp_attn_params* params, const int32_t* lengths, int32_t k) {
  if (!params || !lengths || k < 1) return 0;
  if (params->head_dim != 64 && params->head_dim != 128) return 0;
  if (params->n_q_heads < 1 || params->n_kv_heads < 1) return 0;
  try {
    pp::HostPlan h;
    if (pp::plan_host(*params, lengths, k, &h) != PP_OK) return 0;
    return h.total;
  } catch (const std::bad_alloc&) {
    return 0;
  }
}

extern "C" int pp_prefill_host(pp_attn_params* params, const int32_t* lengths, int32_t k,
                               const void* q_host, const void* k_host, const void* v_host, void* o_host,
                               void* k_cache_host, void* v_cache_host, void* arena, size_t arena_bytes,
                               void* stream) {
  if (!params || !lengths || k < 1 || !q_host || !k_host || !v_host || !o_host || !k_cache_host ||
      !v_cache_host || !arena)
    return PP_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(arena) & 255u) return PP_ERR_ALIGNMENT;
  if (params->head_dim != 64 && params->head_dim != 128) return PP_ERR_UNSUPPORTED;
  if (params->n_q_heads < 1 || params->n_kv_heads < 1) return PP_ERR_INVALID_ARG;
  try {
    pp::HostPlan h;
    int st = pp::plan_host(*params, lengths, k, &h);
    if (st != PP_OK) return st;
    params->capacity = h.capacity;
    params->n_bins = h.n_bins;
    params->flags = 0;
    if ((st = pp::check_params(params)) != PP_OK) return st;
    if (arena_bytes < h.total) return PP_ERR_BUFFER_TOO_SMALL;
    char* base = static_cast<char*>(arena);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int32_t cap = h.capacity;
    const size_t q_row = (size_t)params->n_q_heads * params->head_dim * 2;
    const size_t kv_row = (size_t)params->n_kv_heads * params->head_dim * 2;
    cudaError_t e;
    // Every group runs on its own stream: one upload per tensor, TENSORIZE on the device, the two
    // kernels of the fused path (which write the caches in token order), O gathered back to token
    // order, one download per tensor. The uploads of one group overlap the kernels of another and
    // the downloads of a third (PCIe is full duplex).
    pp::HostPipe* pipe = nullptr;
    if ((st = pp::host_pipe(&pipe)) != PP_OK) return st;
    // On an error in the middle of the pipeline, work already queued on the internal streams still
    // reads and writes the caller's buffers: wait for it before handing the error back.
    auto bail = [&](int code) {
      for (int g = 0; g < pp::kHostGroupsMax; ++g) (void)cudaStreamSynchronize(pipe->stream[g]);
      (void)cudaStreamSynchronize(s);
      return code;
    };
#define PP_TRY(call, what) do { e = (call); if (e != cudaSuccess) return bail(pp::note_cuda_error((int)e, what)); } while (0)
    const int n_groups = (int)h.groups.size();
    PP_TRY(cudaMemsetAsync(base + h.status, 0, 4, s), "memset status");
    PP_TRY(cudaEventRecord(pipe->start, s), "event record");
    std::vector<int64_t> g_cache_off;
    int32_t* d_status = reinterpret_cast<int32_t*>(base + h.status);
    for (int g = 0; g < n_groups; ++g) {
      const pp::HostGroup& G = h.groups[g];
      const int32_t kg = G.i1 - G.i0;
      const size_t tok0 = (size_t)G.t0, ntok = (size_t)(G.t1 - G.t0);
      const size_t rows0 = (size_t)G.bin0 * cap;
      cudaStream_t sg = pipe->stream[g];
      PP_TRY(cudaStreamWaitEvent(sg, pipe->start, 0), "stream wait");
      // The small uploads first (token -> packed row map, rows used per bin, and the group's tables,
      // from pinned staging): queued behind another group's bulk copies they would hold this group's
      // kernels back for milliseconds.
      pp_attn_params gp = *params;
      gp.n_bins = G.n_bins;
      const size_t map_ints64 = 2 * (size_t)kg + 1 + (size_t)G.n_bins;
      const size_t map_bytes = pp::up256(sizeof(int64_t) * map_ints64);
      const size_t tab_bytes = pp::up256(pp::fused_layout(gp, kg).total_bytes);
      void* stage = nullptr;
      if ((st = pp::host_staging(pipe, g, map_bytes + tab_bytes, &stage)) != PP_OK) return bail(st);
      int64_t* map = static_cast<int64_t*>(stage);
      int64_t* used = map + 2 * (size_t)kg + 1;
      g_cache_off.resize(kg);
      int64_t t = 0;
      for (int32_t j = 0; j < kg; ++j) {
        map[j] = t;
        map[kg + 1 + j] = (int64_t)G.bin_of[j] * cap + G.off_of[j];
        g_cache_off[j] = (int64_t)(tok0 + (size_t)t) * params->n_kv_heads * params->head_dim;
        t += lengths[G.i0 + j];
      }
      map[kg] = t;
      for (int32_t b = 0; b < G.n_bins; ++b) {
        const int32_t last = G.bin_seg_ptr[b + 1] - 1;
        used[b] = (int64_t)G.seg_start[last] + G.seg_len[last];
      }
      int64_t* d_map = reinterpret_cast<int64_t*>(base + h.map + g * h.map_stride);
      PP_TRY(cudaMemcpyAsync(d_map, map, sizeof(int64_t) * map_ints64, cudaMemcpyHostToDevice, sg), "H2D map");
      char* gq = base + h.q + rows0 * q_row;
      char* gk = base + h.k + rows0 * kv_row;
      char* gv = base + h.v + rows0 * kv_row;
      char* go = base + h.o + rows0 * q_row;
      char* gws = base + h.ws + g * h.ws_stride;
      void* gstage = static_cast<char*>(stage) + map_bytes;
      pp::TableLayout g_layout;
      st = pp::prefill_fused_impl(&gp, G.bin_seg_ptr.data(), G.seg_start.data(), G.seg_len.data(), G.seg_prompt.data(),
                                  kg, lengths + G.i0, gq, gk, gv, go, base + h.kc, base + h.vc, g_cache_off.data(),
                                  lengths + G.i0, gws, gstage, tab_bytes, d_status, sg, pp::TableStep::kUploadOnly, &g_layout);
      if (st != PP_OK) return bail(st);
      PP_TRY(cudaMemcpyAsync(base + h.q_tok + tok0 * q_row, (const char*)q_host + tok0 * q_row, ntok * q_row,
                             cudaMemcpyHostToDevice, sg), "H2D q");
      PP_TRY(cudaMemcpyAsync(base + h.k_tok + tok0 * kv_row, (const char*)k_host + tok0 * kv_row, ntok * kv_row,
                             cudaMemcpyHostToDevice, sg), "H2D k");
      PP_TRY(cudaMemcpyAsync(base + h.v_tok + tok0 * kv_row, (const char*)v_host + tok0 * kv_row, ntok * kv_row,
                             cudaMemcpyHostToDevice, sg), "H2D v");
      // TENSORIZE: padding rows of the packed tensors zeroed (they must be finite), real rows scattered
      if ((st = pp::launch_zero_pad_rows(gq, gk, gv, (int32_t)q_row, (int32_t)kv_row, d_map + 2 * (size_t)kg + 1,
                                         G.n_bins, cap, sg)) != PP_OK) return bail(st);
      if ((st = pp::launch_tensorize(true, gq, base + h.q_tok + tok0 * q_row, d_map, kg, (int64_t)ntok, (int32_t)q_row, sg)) != PP_OK) return bail(st);
      if ((st = pp::launch_tensorize(true, gk, base + h.k_tok + tok0 * kv_row, d_map, kg, (int64_t)ntok, (int32_t)kv_row, sg)) != PP_OK) return bail(st);
      if ((st = pp::launch_tensorize(true, gv, base + h.v_tok + tok0 * kv_row, d_map, kg, (int64_t)ntok, (int32_t)kv_row, sg)) != PP_OK) return bail(st);
      st = pp::prefill_fused_impl(&gp, G.bin_seg_ptr.data(), G.seg_start.data(), G.seg_len.data(), G.seg_prompt.data(),
                                  kg, lengths + G.i0, gq, gk, gv, go, base + h.kc, base + h.vc, g_cache_off.data(),
                                  lengths + G.i0, gws, gstage, tab_bytes, d_status, sg, pp::TableStep::kLaunchOnly, &g_layout);
      if (st != PP_OK) return bail(st);
      // the caches are final once the first kernel of the fused path has run; O follows the attention
      if ((st = pp::launch_tensorize(false, go, base + h.o_tok + tok0 * q_row, d_map, kg, (int64_t)ntok, (int32_t)q_row, sg)) != PP_OK) return bail(st);
      PP_TRY(cudaMemcpyAsync((char*)k_cache_host + tok0 * kv_row, base + h.kc + tok0 * kv_row, ntok * kv_row,
                             cudaMemcpyDeviceToHost, sg), "D2H k cache");
      PP_TRY(cudaMemcpyAsync((char*)v_cache_host + tok0 * kv_row, base + h.vc + tok0 * kv_row, ntok * kv_row,
                             cudaMemcpyDeviceToHost, sg), "D2H v cache");
      PP_TRY(cudaMemcpyAsync((char*)o_host + tok0 * q_row, base + h.o_tok + tok0 * q_row, ntok * q_row,
                             cudaMemcpyDeviceToHost, sg), "D2H o");
      PP_TRY(cudaEventRecord(pipe->done[g], sg), "event record");
      PP_TRY(cudaStreamWaitEvent(s, pipe->done[g], 0), "stream wait");
    }
    int32_t status = 0;
    PP_TRY(cudaMemcpyAsync(&status, base + h.status, 4, cudaMemcpyDeviceToHost, s), "D2H status");
    PP_TRY(cudaStreamSynchronize(s), "stream synchronize");
#undef PP_TRY
    return status == 0 ? PP_OK : PP_ERR_DEVICE_TIMEOUT;
  } catch (const std::bad_alloc&) {
    return PP_ERR_NO_MEMORY;
  }
}
