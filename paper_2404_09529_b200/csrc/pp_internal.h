// Internal declarations shared by the translation units of the prepack-b200 library.
#ifndef PREPACK_B200_PP_INTERNAL_H_
#define PREPACK_B200_PP_INTERNAL_H_

#include <cstddef>
#include <cstdint>

#include "../../include/pp.h"

namespace pp {

constexpr int kTileM = 128;      // query rows per work item (tcgen05 MMA M)
constexpr int kTileN = 128;      // key rows per inner step (tcgen05 MMA N of Q.K^T), shared-stream mode
constexpr int kTileNShort = 64;  // the same in independent-slot mode (short work items)
constexpr int kHeaderInts = 16;  // table header, see build_prefill_tables
constexpr int kHeaderCounter = 10;   // header word the persistent CTAs draw work indices from
constexpr int kItemInts = 16;
constexpr int kMaxFold = 8;      // most query heads of one KV head folded into the rows of a query tile

// One entry of the attention work list: two query-tile slots sharing one key/value tile stream.
struct WorkItem {
  int32_t bin;
  int32_t kv_row0;      // first key row of the stream (multiple of the mode's key tile)
  int32_t n_kv_tiles;   // key tiles in the stream
  int32_t q_row0[2];    // first query row of each slot; -1 = slot unused
  int32_t jb1;          // slot 1 takes part in key tiles [jb1, n_kv_tiles)
  int32_t je0;          // slot 0 takes part in key tiles [0, je0)
  int32_t cost;         // (slot, key tile) steps, for longest-first ordering
  int32_t bin_used;     // occupied rows of the bin
  int32_t seg_end;      // one past the bin's last segment index
  int32_t key_lo[2];    // start row of the prompt that holds the slot's first query row
  int32_t seg_first[2]; // segment index of that prompt
  int32_t single_seg;   // bit t set: all real rows of slot t belong to that one prompt
  int32_t reserved;
};

// Offsets (in int32 units) of the blocks inside the prefill table that is built on the host and
// copied to the device workspace.
struct TableLayout {
  int32_t bin_seg_ptr = 0;  // [R+1]
  int32_t bin_used = 0;     // [R]   occupied rows per bin
  int32_t seg_start = 0;    // [k]   bin-local first row of each segment
  int32_t items = 0;        // [n_items] WorkItem, longest first
  int32_t n_items = 0;
  int32_t total_ints = 0;
  bool independent_slots = false;   // items are single tiles, drawn by each slot on its own
  bool pair_rows = false;           // shared-stream mode: the two slots are consecutive row tiles of one head
  int32_t fold = 1;                 // independent mode: query heads folded into a query tile (128 / fold bin rows each)
};

int validate_packing(int32_t n_bins, int32_t capacity, const int32_t* bin_seg_ptr,
                     const int32_t* seg_start, const int32_t* seg_len, int32_t k);
size_t prefill_table_ints(int32_t n_bins, int32_t capacity, int32_t k, int32_t group);
int32_t max_fold(int32_t group);   // largest power of two <= kMaxFold that divides the GQA group
int build_prefill_tables(int32_t n_bins, int32_t capacity, const int32_t* bin_seg_ptr,
                         const int32_t* seg_start, const int32_t* seg_len, int32_t k, int32_t group,
                         int32_t* out, size_t out_ints, TableLayout* layout);

// Records a failed CUDA call for pp_last_cuda_error(); returns PP_ERR_CUDA.
int note_cuda_error(int cuda_error, const char* what);

// Kernel launchers (device pointers, stream = cudaStream_t as void*). Return a PP_* status.
// Rotates the n_q_heads heads of q into q_out (may be the same buffer) and the n_kv_heads heads of k
// in place; pass n_q_heads or n_kv_heads = 0 in `p` to rotate only the other tensor.
int launch_rope(const pp_attn_params& p, const int32_t* d_table, const TableLayout& L,
                const void* q, void* q_out, void* k, void* stream);
// rope_table: device [D/4][capacity][2] (cos, sin) pairs, or null. When given, q holds the raw
// queries and the kernel rotates each Q tile in shared memory before use.
int launch_attention(const pp_attn_params& p, int32_t* d_table, const TableLayout& L,
                     const void* q, const void* k, const void* v, void* o, const void* rope_table,
                     int32_t* device_status, void* stream);
// Fused K rotation + UNPACK; the three offsets locate per-segment arrays inside the table
// (true length, cache capacity: int32; cache element offset: int64).
int launch_rope_unpack(const pp_attn_params& p, const int32_t* d_table, const TableLayout& L,
                       int32_t off_true_len, int32_t off_cap, int32_t off_cache_off, const void* rope_table,
                       void* k, const void* v, void* k_cache, void* v_cache, void* stream);
// Fills rope_table for positions 0 .. capacity-1.
int launch_rope_table(const pp_attn_params& p, void* table, void* stream);
int launch_unpack(const pp_attn_params& p, const int32_t* d_table, int32_t k, int64_t total_tokens,
                  const void* k_rot, const void* v, void* k_cache, void* v_cache, void* stream);

// Row scatter (to_packed) / gather between a token-major tensor [T, row_bytes] and the packed layout.
// d_map: device int64 tok_prefix[n_prompts + 1] followed by first_row[n_prompts].
int launch_tensorize(bool to_packed, void* packed, void* tokens, const int64_t* d_map, int32_t n_prompts,
                     int64_t total_tokens, int32_t row_bytes, void* stream);

// Zeroes rows [bin_used[b], capacity) of every bin of the packed q / k / v (null pointers are skipped).
int launch_zero_pad_rows(void* q, void* k, void* v, int32_t q_row_bytes, int32_t kv_row_bytes,
                         const int64_t* d_bin_used, int32_t n_bins, int32_t capacity, void* stream);

int launch_bounded_wait_selftest(int32_t* device_status, uint64_t limit_ns, void* stream);

// Unpack table (int32 units): header 4 ints, then token_prefix[k+1], bin_of[k], off_of[k],
// cache_cap[k], cache_off as int64[k] (8-byte aligned).
size_t unpack_table_bytes(int32_t k);

#ifdef __CUDACC__
// Programmatic dependent launch. A kernel of the path that is launched with launch_dependent() may
// start while the kernel before it in the stream is still finishing: its blocks are scheduled once
// every block of that kernel has called pdl_launch_dependents() (or exited), run their set-up, and
// block in pdl_wait() until that kernel has completed and its writes are visible. Work queued
// before that kernel has completed by then in any case. Launched the ordinary way, both calls
// do nothing.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif  // __CUDACC__

}  // namespace pp

#endif  // PREPACK_B200_PP_INTERNAL_H_
