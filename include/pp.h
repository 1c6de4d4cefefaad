/*
 * prepack-b200: C ABI of the prepacked-prefill attention hot path for NVIDIA B200 (sm_100a).
 *
 * The library follows the steps of Algorithm 1 ("Prepacking") of arXiv 2404.09529:
 *   BINPACK            -> pp_pack                 (host)
 *   TENSORIZE          -> layout contract below   (no call)
 *   INDEPENDENT-MASK   -> applied inside pp_prefill_attention, never materialised
 *   RESTART-PE         -> applied inside pp_prefill_attention (rotary), also
 *                         available as explicit ids from pp_fill_position_ids
 *   forward + UNPACK   -> pp_prefill_attention (the attention of one layer) and
 *                         pp_unpack_kv
 *
 * Conventions
 *   - Every function returns an int status (PP_OK = 0, errors < 0). Nothing aborts or throws.
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA global memory of the
 *     current device. The library never allocates device memory; callers own every buffer.
 *   - Streams are passed as void* (a cudaStream_t); NULL is the default stream. Device work is
 *     enqueued on that stream and the call returns without synchronising unless stated.
 *   - Tensors are bf16. Packed tensors are dense [R, M, H, D] (bins, rows per bin = capacity,
 *     heads, head_dim), row t of bin b being the token at bin-local offset t (TENSORIZE,
 *     Section 3.1: bins are tail-padded to the bin size). Rows at or after the bin's used
 *     length are padding: they must hold finite values (zeros are fine) and their outputs are
 *     unspecified.
 *   - Packing arrays are int32, "segments" are prompts in bin-major placement order.
 */
#ifndef PREPACK_B200_PP_H_
#define PREPACK_B200_PP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  PP_OK = 0,
  PP_ERR_INVALID_ARG = -1,      /* null pointer, k < 1, inconsistent packing arrays            */
  PP_ERR_LENGTH = -2,           /* a prompt length < 1 or > capacity                          */
  PP_ERR_BUFFER_TOO_SMALL = -3, /* workspace / arena smaller than the *_bytes query            */
  PP_ERR_UNSUPPORTED = -4,      /* head_dim not in {64,128}, Hq % Hkv != 0, device not sm_100  */
  PP_ERR_ALIGNMENT = -5,        /* a device tensor pointer is not 16-byte aligned              */
  PP_ERR_CUDA = -6,             /* a CUDA runtime/driver call failed (see pp_last_cuda_error)  */
  PP_ERR_DEVICE_TIMEOUT = -7,   /* a bounded device-side wait gave up (device status word)     */
  PP_ERR_NO_MEMORY = -8,        /* host allocation failed                                      */
  PP_ERR_TOO_LARGE = -9         /* more prompts than the built-in scratch of a *_static call   */
};

/* Flags for pp_attn_params.flags. Every other bit must be zero: the entry points that read the
 * field answer PP_ERR_INVALID_ARG to a bit they do not know. */
enum {
  PP_FLAG_SKIP_ROPE = 1,  /* q and k already carry the rotary encoding: run attention only     */
  PP_FLAG_ROPE_ONLY = 2,  /* apply the restart rotary encoding to q and k, skip attention      */
  PP_FLAG_KEEP_ROPE_TABLE = 4  /* pp_prefill_fused only: the workspace was last used by a
                             pp_prefill_fused call with the same capacity, head_dim and rope_base
                             and nothing else has written to it since, so its cos/sin table is
                             still valid and is not rebuilt                                      */
};

typedef struct pp_attn_params {
  int32_t n_q_heads;     /* Hq                                                                 */
  int32_t n_kv_heads;    /* Hkv, divides Hq; query head h reads KV head h / (Hq / Hkv)          */
  int32_t head_dim;      /* D: 64 or 128                                                       */
  float rope_base;       /* rotary base; theta_j = base^(-2j/D), pairs (j, j + D/2)             */
  float softmax_scale;   /* 0 selects 1/sqrt(D) (Section 2.1)                                  */
  int32_t capacity;      /* M: rows per bin (Algorithm 1 (bin size): the longest prompt)           */
  int32_t n_bins;        /* R                                                                  */
  int32_t flags;         /* PP_FLAG_* or 0                                                     */
} pp_attn_params;

/* Library version (major * 10000 + minor * 100 + patch). */
int pp_version(void);
/* Static, never-NULL description of a status code. */
const char* pp_strerror(int status);
/* Text of the last CUDA error seen by the calling thread inside the library ("" if none). */
const char* pp_last_cuda_error(void);

/*
 * BINPACK -- Section 3.1 and Algorithm 1 (bin size, BINPACK). Host only, deterministic.
 * First-fit-decreasing of k prompt lengths into bins of `capacity` rows (0 selects the longest
 * prompt, the paper's choice). Items are taken by length descending, equal lengths by original
 * index ascending; each goes to the lowest-numbered bin with room, else opens a new bin; bins
 * are numbered in creation order and keep their items in placement order.
 * Outputs (caller-allocated host arrays; any may be NULL to skip it except n_bins):
 *   n_bins       [1]    r
 *   capacity_out [1]    the capacity used
 *   bin_seg_ptr  [k+1]  CSR over segments; entries 0..r are written
 *   seg_prompt   [k]    original prompt index of each segment
 *   seg_start    [k]    bin-local start row of each segment (the paper's idx)
 *   seg_len      [k]    length of each segment
 *   bin_of,off_of[k]    inverse map, original prompt order: prompt i lives in bin bin_of[i] at
 *                       rows off_of[i] .. off_of[i]+lengths[i]-1
 * Errors: PP_ERR_INVALID_ARG (NULL lengths/n_bins, k < 1), PP_ERR_LENGTH, PP_ERR_NO_MEMORY.
 */
int pp_pack(const int32_t* lengths, int32_t k, int32_t capacity,
            int32_t* n_bins, int32_t* capacity_out,
            int32_t* bin_seg_ptr, int32_t* seg_prompt, int32_t* seg_start, int32_t* seg_len,
            int32_t* bin_of, int32_t* off_of);

/*
 * RESTART-PE as explicit ids -- Section 3.2, Algorithm 1 (RESTART-PE). Host only.
 * position_ids [n_bins*capacity]: 0,1,2,... restarting at every segment start; padding rows 0.
 * segment_ids  [n_bins*capacity]: index into the seg_* arrays; padding rows -1. Either output
 * may be NULL. Errors: PP_ERR_INVALID_ARG on NULL inputs or segments that do not tile a bin
 * contiguously from row 0 within `capacity`.
 */
int pp_fill_position_ids(int32_t n_bins, int32_t capacity, const int32_t* bin_seg_ptr,
                         const int32_t* seg_start, const int32_t* seg_len,
                         int32_t* position_ids, int32_t* segment_ids);

/*
 * How the attention kernel will walk a packed batch -- the INDEPENDENT-MASK step of Algorithm 1 and
 * Section 3.2 turned into a tile work list: a query tile visits only the key tiles between the start
 * of the first prompt it touches and its own last row. Host only, launches nothing; for tests, cost
 * models and schedulers. info (int32[8], caller-allocated) receives
 *   [0] mode: 0 = shared-stream (the two query tiles of a CTA share one stream of 128-row key
 *       tiles; long prompts), 1 = independent (every query tile walks its own 64-row key tiles)
 *   [1] pairing of the two query tiles of a work item: 0 = two query heads of one KV head over the
 *       same rows, 1 = two consecutive row tiles of one head, 2 = none (independent mode)
 *   [2] work-list entries (per KV head and head pair / head)
 *   [3] (query tile, key tile) steps summed over the entries
 *   [4] key rows per tile (128 or 64)
 *   [5] entries whose second query tile is unused (the unpaired last row tile of a bin)
 *   [6] entries whose second query tile joins the key stream after its first tile
 *   [7] query heads folded into the rows of one query tile (1 = none)
 * Errors: PP_ERR_INVALID_ARG, PP_ERR_LENGTH, PP_ERR_UNSUPPORTED, PP_ERR_NO_MEMORY.
 */
int pp_prefill_schedule_info(const pp_attn_params* params, const int32_t* bin_seg_ptr,
                             const int32_t* seg_start, const int32_t* seg_len, int32_t k,
                             int32_t* info);

/*
 * Bytes of workspace pp_prefill_attention needs, for a batch of k prompts packed as `params`
 * says (same size for the device workspace and for the host staging buffer). 0 on bad input.
 */
size_t pp_prefill_workspace_bytes(const pp_attn_params* params, int32_t k);

/*
 * Prefill attention over the packed batch -- Algorithm 1 (INDEPENDENT-MASK to UNPACK) for one attention layer:
 * restart rotary encoding of q and k (Section 3.2), then per bin and query head
 *   o_i = sum_j softmax_j(q'_i . k'_j * scale) v_j   over keys j of the SAME prompt with j <= i
 * (independent mask M' of Section 3.2: a lower-triangular block per prompt span, zero elsewhere).
 *
 *   params                         shapes, see pp_attn_params
 *   bin_seg_ptr, seg_start, seg_len, k
 *                                  host packing arrays from pp_pack (k = number of segments)
 *   q   device [R, M, Hq,  D] bf16 in/out: overwritten with the rotated queries
 *   k_  device [R, M, Hkv, D] bf16 in/out: overwritten with the rotated keys (this is the
 *                                  packed K cache that pp_unpack_kv reads)
 *   v   device [R, M, Hkv, D] bf16 read only
 *   o   device [R, M, Hq,  D] bf16 out; padding rows unspecified
 *   workspace       device, >= pp_prefill_workspace_bytes, 16-byte aligned; holds the segment
 *                   table and the tile work list for the duration of the enqueued work
 *   host_workspace  host, same size (pinned memory keeps the call asynchronous); the library
 *                   builds the tables here and copies them with one async H2D on `stream`; it
 *                   must stay untouched until that copy has run
 *   device_status   device int32 or NULL; set non-zero by the kernel if a bounded wait inside
 *                   it gave up (then outputs are invalid). The caller zeroes and reads it. Every
 *                   wait in the kernel is limited to 2 s; the environment variables
 *                   PP_WAIT_LIMIT_MS / PP_WAIT_LIMIT_US, read at each call, override the limit.
 * The kernels of one call may be launched as programmatic dependents of one another (set-up of a
 * kernel overlapping the end of the kernel before it); nothing of that is visible to the caller:
 * stream order holds for everything the caller enqueues before and after the call.
 * Arithmetic: rotation in fp32 with one rounding to bf16; scores and outputs accumulated in
 * fp32 on the tensor cores, probabilities rounded to bf16 before the P.V product.
 * Errors (all detected before anything is enqueued): PP_ERR_INVALID_ARG, PP_ERR_LENGTH,
 * PP_ERR_UNSUPPORTED, PP_ERR_ALIGNMENT, PP_ERR_BUFFER_TOO_SMALL; PP_ERR_CUDA from launches.
 */
int pp_prefill_attention(const pp_attn_params* params,
                         const int32_t* bin_seg_ptr, const int32_t* seg_start,
                         const int32_t* seg_len, int32_t k,
                         void* q, void* k_, const void* v, void* o,
                         void* workspace, void* host_workspace, size_t workspace_bytes,
                         int32_t* device_status, void* stream);

/*
 * The same result as pp_prefill_attention followed by pp_unpack_kv (Algorithm 1 (INDEPENDENT-MASK to UNPACK) for one
 * attention layer), with fewer passes over HBM: one kernel rotates K, writes it back to the packed
 * tensor and into the per-prompt K caches and copies V into the V caches; the attention kernel
 * rotates each Q tile on the fly, so q is read only.
 *   bin_seg_ptr, seg_start, seg_len, seg_prompt, k   host packing arrays from pp_pack
 *   lengths      host [k], original prompt order: rows of each prompt to cache (<= its segment)
 *   q            device [R, M, Hq, D] bf16, raw queries, read only
 *   k_           device [R, M, Hkv, D] bf16 in/out: overwritten with the rotated keys
 *   v, o         as in pp_prefill_attention
 *   k_cache, v_cache, cache_off, cache_cap   as in pp_unpack_kv (original prompt order)
 *   workspace    device, >= pp_prefill_fused_workspace_bytes, 256-byte aligned (tables and a
 *                cos/sin table of capacity * D/2 pairs); host_workspace: host staging of at least
 *                pp_prefill_fused_host_bytes (the tables, which are what is uploaded; the cos/sin
 *                table is built on the device), pinned memory keeps the call asynchronous
 * params->flags: PP_FLAG_ROPE_ONLY runs only the rotation / unpack kernels, PP_FLAG_SKIP_ROPE only the
 * attention kernel (k_ holds rotated keys already). Outputs are bit-identical to the two-call path.
 * Errors as the two calls it replaces.
 */
size_t pp_prefill_fused_workspace_bytes(const pp_attn_params* params, int32_t k);
size_t pp_prefill_fused_host_bytes(const pp_attn_params* params, int32_t k);
int pp_prefill_fused(const pp_attn_params* params,
                     const int32_t* bin_seg_ptr, const int32_t* seg_start, const int32_t* seg_len,
                     const int32_t* seg_prompt, int32_t k, const int32_t* lengths,
                     const void* q, void* k_, const void* v, void* o,
                     void* k_cache, void* v_cache, const int64_t* cache_off, const int32_t* cache_cap,
                     void* workspace, void* host_workspace, size_t workspace_bytes,
                     int32_t* device_status, void* stream);

/*
 * Self-test of the kernels' bounded waits (every mbarrier wait inside pp_prefill_attention gives up
 * after a time limit instead of spinning forever). Enqueues a one-block kernel in which a thread
 * waits on a barrier that nothing signals; after limit_ms (1..1000) the wait gives up and writes
 * the non-zero code 77 to *device_status (device int32, zeroed by the caller), and the kernel
 * returns normally. No counterpart in the paper. Errors: PP_ERR_INVALID_ARG, PP_ERR_UNSUPPORTED,
 * PP_ERR_CUDA.
 */
int pp_selftest_bounded_wait(int32_t* device_status, uint32_t limit_ms, void* stream);

/* Bytes of workspace pp_unpack_kv needs for k prompts (device and host staging alike). */
size_t pp_unpack_workspace_bytes(int32_t k);

/*
 * UNPACK -- Algorithm 1 (UNPACK), Section 4.3: copy each prompt's rotated keys and its values out
 * of the packed tensors into that prompt's own cache, in original prompt order.
 *   cache[i][h][p][:] = packed[bin_of[i], off_of[i] + p, h, :]   for p < lengths[i]
 *   bin_of, off_of, lengths  host [k], original prompt order (lengths may be shorter than the
 *                            packed segment, e.g. in padded mode; only that many rows are copied)
 *   k_rot, v       device [R, M, Hkv, D] bf16 (k_rot = the k_ tensor after pp_prefill_attention)
 *   k_cache, v_cache device bf16 pools; prompt i's block starts at element cache_off[i] and is
 *                  laid out [Hkv, cache_cap[i], D]; rows >= lengths[i] are left untouched
 *   cache_off      host int64 [k], multiples of 8 elements; cache_cap host int32 [k] >= lengths
 *   workspace / host_workspace  >= pp_unpack_workspace_bytes(k), as for pp_prefill_attention
 * Pure copy, bit exact. Errors: PP_ERR_INVALID_ARG, PP_ERR_LENGTH, PP_ERR_ALIGNMENT,
 * PP_ERR_BUFFER_TOO_SMALL, PP_ERR_UNSUPPORTED, PP_ERR_CUDA.
 */
int pp_unpack_kv(const pp_attn_params* params,
                 const int32_t* bin_of, const int32_t* off_of, const int32_t* lengths, int32_t k,
                 const void* k_rot, const void* v, void* k_cache, void* v_cache,
                 const int64_t* cache_off, const int32_t* cache_cap,
                 void* workspace, void* host_workspace, size_t workspace_bytes, void* stream);

/*
 * pp_unpack_kv without a caller workspace (the paper has no counterpart; this is for users of the
 * library who may not allocate device memory: a serving process whose pool was carved up at
 * start-up, a plug-in that receives tensors but no allocator, code running while another
 * component owns the allocator). Arguments and result are those of pp_unpack_kv minus the two
 * workspaces: the per-prompt table lives in a fixed device array inside the library image (about
 * 96 KiB on every GPU that loads the library, held until the process exits), so
 *   - k may not exceed pp_unpack_static_max_prompts() (4096); more gives PP_ERR_TOO_LARGE and
 *     nothing is enqueued;
 *   - the call allocates nothing, on the host or on the device;
 *   - the first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture;
 *   - all calls on one GPU share the one table: two calls whose device work can overlap (different
 *     streams, or different host threads without ordering between their streams) race on it.
 *     Calls on the same stream are safe, and the table is rewritten in full on every call.
 */
int32_t pp_unpack_static_max_prompts(void);
int pp_unpack_kv_static(const pp_attn_params* params,
                        const int32_t* bin_of, const int32_t* off_of, const int32_t* lengths, int32_t k,
                        const void* k_rot, const void* v, void* k_cache, void* v_cache,
                        const int64_t* cache_off, const int32_t* cache_cap, void* stream);

/*
 * One generation step over the per-prompt caches -- Section 7 (prepacking for generation). For
 * every prompt i the new token sits at position lengths[i] (the number of tokens its caches hold):
 * its query and key are rotated by that position, the rotated key and the value are appended to
 * the caches at row lengths[i], and the query attends to rows 0 .. lengths[i]. The caches are the
 * unpadded per-prompt blocks that pp_unpack_kv / pp_prefill_fused fill, so the step reads exactly
 * the keys and values each prompt has, whatever the other prompts' lengths are.
 *   params       n_q_heads, n_kv_heads (at most 8 query heads per KV head), head_dim, rope_base,
 *                softmax_scale are read; capacity, n_bins and flags are ignored
 *   lengths      host [k]: tokens already in each prompt's caches (>= 1)
 *   q_new        device [k, Hq, D] bf16, k_new / v_new device [k, Hkv, D] bf16: the new tokens' raw
 *                projections, read only
 *   o            device [k, Hq, D] bf16 out
 *   k_cache, v_cache, cache_off, cache_cap   as in pp_unpack_kv; cache_cap[i] > lengths[i]
 *   workspace    device, >= pp_decode_workspace_bytes(params, lengths, k), 256-byte aligned;
 *                host_workspace: host staging of the same size or at least the table part (pinned
 *                memory keeps the call asynchronous)
 * Asynchronous on `stream`. Errors: PP_ERR_INVALID_ARG, PP_ERR_LENGTH (no room for one more token),
 * PP_ERR_UNSUPPORTED (head_dim, group size), PP_ERR_ALIGNMENT, PP_ERR_BUFFER_TOO_SMALL, PP_ERR_CUDA.
 */
size_t pp_decode_workspace_bytes(const pp_attn_params* params, const int32_t* lengths, int32_t k);
int pp_decode_step(const pp_attn_params* params, const int32_t* lengths, int32_t k,
                   const void* q_new, const void* k_new, const void* v_new, void* o,
                   void* k_cache, void* v_cache, const int64_t* cache_off, const int32_t* cache_cap,
                   void* workspace, void* host_workspace, size_t workspace_bytes, void* stream);

/*
 * Whole path from host memory (Algorithm 1 (bin size to UNPACK) for one attention layer), for callers whose
 * tensors live on the host. Every tensor goes up in large contiguous copies, is laid out as the
 * packed batch by device kernels (TENSORIZE, padding rows zeroed), the kernels of pp_prefill_fused
 * run there and write the caches in token order, O is gathered back into token order and the
 * outputs are copied back; `stream` is synchronised before the call returns.
 *   params                   n_q_heads, n_kv_heads, head_dim, rope_base, softmax_scale are
 *                            read; capacity and n_bins are filled in from the packing
 *   q_host                   host bf16 [T, Hq, D], tokens of prompt 0, then prompt 1, ...
 *   k_host, v_host           host bf16 [T, Hkv, D], same order (T = sum of lengths)
 *   o_host                   host out bf16 [T, Hq, D], same order
 *   k_cache_host, v_cache_host host out bf16; prompt i at element Hkv*D*(sum of earlier
 *                            lengths), laid out [Hkv, lengths[i], D]
 *   arena, arena_bytes       device scratch >= pp_prefill_host_arena_bytes(params, lengths, k),
 *                            256-byte aligned
 * Pinned host buffers give full copy bandwidth; pageable ones work too. A batch of 32 MB or more
 * is cut into up to eight groups of consecutive prompts with about equal token counts. Each
 * group is packed on its own (pp_pack with the batch-wide capacity = longest prompt; n_bins is the
 * sum over the groups) and runs on a stream the library creates once per device and thread, so
 * the uploads of one group overlap the kernels of another and the downloads of a third. Smaller
 * batches are one group, packed exactly as pp_pack packs the whole batch. The caches do not depend
 * on the grouping; O depends on it only through the position of tile boundaries (summation
 * order). Work already queued on `stream` is waited for first.
 * pp_prefill_host_groups(n) fixes the number of groups for later calls of the calling thread
 * (1 .. 16; 1 gives exactly the packing of pp_pack over the whole batch and with it O bit-identical
 * to the device entry points; 0 restores the choice by batch size) and returns the previous setting;
 * an n outside 0 .. 16 changes nothing.
 * Errors: as pp_prefill_fused, plus PP_ERR_DEVICE_TIMEOUT.
 */
int32_t pp_prefill_host_groups(int32_t n_groups);
size_t pp_prefill_host_arena_bytes(const pp_attn_params* params, const int32_t* lengths, int32_t k);
int pp_prefill_host(pp_attn_params* params, const int32_t* lengths, int32_t k,
                    const void* q_host, const void* k_host, const void* v_host,
                    void* o_host, void* k_cache_host, void* v_cache_host,
                    void* arena, size_t arena_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PREPACK_B200_PP_H_ */
