// pp_unpack_kv_static: the UNPACK scatter for callers that cannot allocate device memory.
//
// Some callers run where cudaMalloc is off limits: inside a serving loop whose memory pool was
// sized and frozen at start-up, in a plug-in that is handed tensors but no allocator, or in code
// that must not touch the allocator because another component owns all of the device's memory.
// pp_unpack_kv needs a small device table (token prefix, bin/offset/capacity per prompt, cache
// offsets) and asks the caller for a workspace to hold it. This variant keeps that table in a
// fixed array that lives inside the library image instead, so the caller passes only inputs and
// outputs. The price is a hard limit on the number of prompts per call and one shared table per
// GPU. The paper has no counterpart for this entry point; it is a packaging convenience.
#include <cuda_runtime.h>

#include <mutex>

#include "pp_internal.h"

namespace {

constexpr int32_t kStaticMaxPrompts = 4096;
// unpack_table_bytes(4096) = (4 + 4100 + 3 * 4096) * 4 + 4096 * 8 = 98336, rounded up to 256
constexpr size_t kStaticTableBytes = 98560;
constexpr int kMaxDevices = 64;

// The scratch itself: part of the library image, present on every GPU that loads the library
// until the process exits. In host code this name is only a handle for cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_unpack_table[kStaticTableBytes];

// Host-side staging for the table; cudaMemcpyAsync from ordinary host memory stages the bytes
// before it returns, so the buffer is free again when the call returns.
alignas(64) unsigned char g_unpack_table_host[kStaticTableBytes];

std::mutex g_mutex;
void* g_device_table[kMaxDevices] = {};

}  // namespace

extern "C" int32_t pp_unpack_static_max_prompts(void) { return kStaticMaxPrompts; }

extern "C" int pp_unpack_kv_static(const pp_attn_params* params, const int32_t* bin_of,
                                   const int32_t* off_of, const int32_t* lengths, int32_t k,
                                   const void* k_rot, const void* v, void* k_cache, void* v_cache,
                                   const int64_t* cache_off, const int32_t* cache_cap, void* stream) {
  if (k < 1) return PP_ERR_INVALID_ARG;
  if (k > kStaticMaxPrompts || pp::unpack_table_bytes(k) > kStaticTableBytes) return PP_ERR_TOO_LARGE;
  std::lock_guard<std::mutex> lock(g_mutex);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return pp::note_cuda_error((int)e, "cudaGetDevice");
  if (dev < 0 || dev >= kMaxDevices) return PP_ERR_UNSUPPORTED;
  if (g_device_table[dev] == nullptr) {
    // once per device, with that device current: turn the symbol into a device address
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_unpack_table);
    if (e != cudaSuccess || ptr == nullptr) return pp::note_cuda_error((int)e, "cudaGetSymbolAddress");
    g_device_table[dev] = ptr;
  }
  // Same validation, table build, upload and kernel as pp_unpack_kv; only the table's home differs.
  // The table is rewritten in full for the k prompts of this call, so nothing left over from an
  // earlier call is read.
  return pp_unpack_kv(params, bin_of, off_of, lengths, k, k_rot, v, k_cache, v_cache, cache_off, cache_cap,
                      g_device_table[dev], g_unpack_table_host, kStaticTableBytes, stream);
}
