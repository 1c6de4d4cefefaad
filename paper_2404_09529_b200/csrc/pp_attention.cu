// Packed-varlen prefill attention for sm_100a (Sections 2.1 and 3.2 of the prepacking paper):
//   o_i = sum_j softmax_j(q'_i . k'_j * scale) v_j   over keys j of the same prompt with j <= i.
// The independent mask M' (a lower-triangular block per prompt span) is never built: every query
// row carries the key range [start row of its prompt, its own row], and the host work list
// restricts each query tile to the key tiles that can intersect such a range.
//
// Persistent kernel, one CTA per SM, 640 threads, two 128-row query-tile slots per CTA. CTAs draw
// work from a global counter (items are listed KV-head-major, longest first). Two modes, chosen on
// the host from the mean number of key tiles per query tile:
//
// Shared-stream mode (long items). A work item has two slots that share one stream of 128-row
// key/value tiles: two query heads of one KV head over the same rows (even GQA group), or two
// consecutive row tiles of one head.
//   warp 0       draws and decodes items, TMA-loads the K / V tile rings
//   warp 1       issues tcgen05.mma: S_t = Q_t K^T into TMEM, O_t += P_t V with P_t read from TMEM;
//                the two slots alternate so that one slot's MMAs run while the other's softmax works
//   warps 2-3    TMA-load Q of slot 0 / slot 1
//   warps 4-11   softmax and epilogue of slot 0: two threads per query row (TMEM lane = row), one per
//                64-key half of a tile; the row maximum is exchanged through shared memory
//   warps 12-19  the same for slot 1
// Independent mode (short items). Every slot draws its own items (one query tile each) and walks
// their 64-row key tiles on its own; S_t has two 64-column buffers so that the scores of tile k+1
// and the product P(k) V(k) are computed while the softmax threads work on tile k.
// With several query heads per KV head (GQA) the heads are folded into the rows of a query tile:
// 128 / f bin rows x f heads (tile row m = bin row m / f, head m % f; f = 2, 4 or 8 dividing the
// group), loaded and stored as one TMA box over (row, head). One stream of key tiles then serves
// the f heads, a short prompt fills a tile with heads instead of empty rows, and an item's key
// tiles start at the first row of the first prompt it touches rather than at a tile boundary.
//   warps 0-1    issue the tcgen05.mma of slot 0 / slot 1
//   warps 2-3    draw items and TMA-load Q, K, V of slot 0 / slot 1 (two K and two V stages each)
//   warps 4-7    softmax threads of slot 0, one per query row; they never leave the tile loop
//   warps 8-11   helper threads of slot 0, one per row: rotate the next item's Q in shared memory
//                (fused path) and run the previous item's epilogue
//   warps 12-19  the same for slot 1
// Softmax: tcgen05.ld the thread's scores, mask to the row's key range, lazy running maximum (O is
// rescaled only when the maximum grows by more than 2^8), exp2, P written as bf16 over the S
// columns. Epilogue: O / l goes through a swizzled staging buffer and a TMA store.
// TMEM: S0 | S1 | O0 | O1 = 512 columns. Every wait is an mbarrier wait with a time limit, also the
// rendezvous between warps (no named barriers), so a failed wait ends the kernel with a status code.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdlib>
#include <type_traits>

#include "pp_device_once.h"
#include "pp_internal.h"

namespace pp {
namespace {

constexpr int BM = kTileM;
constexpr int kAttnThreads = 640;
constexpr int kSoftmaxThreads = 256;       // per slot: two threads per query row
constexpr uint32_t kTmemCols = 512;
constexpr int kRegsSoftmax = 104;          // setmaxnreg budgets: 640 threads start with 96 registers each;
constexpr int kRegsSoftmaxIndep = 120;     // independent mode: 256 softmax threads at 120, 256 helper threads at 88
constexpr int kRegsHelper = 88;
constexpr int kRegsOther = 64;              // warps 0-3 give back 32 each, the 512 softmax threads take 8 each
constexpr uint32_t kRing = 3;               // decoded work items in flight between the fetching thread and its readers
constexpr int kRingInts = 20;              // ints per ring entry

// BN: key rows per tile. 128 in shared-stream mode; 64 in independent mode, where every slot owns
// two K and two V stages and two S buffers (see the kernel).
template <int D, int BN> struct AttnCfg {
  static constexpr int kKStages = (D == 128 && BN == 128) ? 2 : 4;
  static constexpr int kVStages = (D == 128 && BN == 128) ? 2 : 4;
  static constexpr int kChunks = D / 64;                     // 128-byte swizzle spans per row
  static constexpr int kQBytes = BM * D * 2;                 // per slot
  static constexpr int kKVBytes = BN * D * 2;
  // barriers + work ring (1024) and the row-maximum exchange buffer [slot][half][row] (2048), placed
  // in front of the 1024-byte-aligned tiles; at D = 128 the total is exactly the 227 KB limit
  static constexpr int kMiscBytes = 3072;
  static constexpr int kStageOBytes = BM * 128;              // per slot: one 64-column box of O
  static constexpr int kTileBytes = 2 * kQBytes + (kKStages + kVStages) * kKVBytes + 2 * kStageOBytes;
  static constexpr int kSmemBytes = kMiscBytes + kTileBytes;
  static constexpr uint32_t kTmemS = 0;                      // S_t at 128 * t
  static constexpr uint32_t kTmemO = 256;                    // O_t at 256 + D * t
};

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

// Every wait in the kernel goes through here: it gives up after `limit_ns`, records why in the
// device status word and raises the CTA-wide abort flag so that all roles leave their loops.
struct WaitCtx {
  volatile int* abort_flag;     // shared
  int32_t* status;              // global, may be null
  unsigned long long limit_ns;
};
__device__ __forceinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const WaitCtx& w, int code) {
  // The clock is read only every 32 failed polls (each poll may park the thread in hardware for a
  // while), so a short wait costs nothing but the polls; the limit counts from the first reading.
  unsigned long long t0 = 0;
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 31u) == 0) {
      if (*w.abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > w.limit_ns) {
        *w.abort_flag = 1;
        if (w.status) atomicCAS(w.status, 0, code);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& w, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, w, code);
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1,
                                             int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
      ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { __syncwarp(); asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { __syncwarp(); asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors (tcgen05), 128-byte swizzle, rows of 128 bytes, 8-row groups
// 1024 bytes apart. Low word: start address >> 4 and (MN-major operands only) the distance between
// 64-element spans of the MN dimension >> 4. High word: constant (8-row group stride, descriptor
// version, swizzle mode). Stepping along a tile only ever adds a small constant to the low word.
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
  return ((saddr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16);
}
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n.reg .b64 da, db;\nsetp.ne.b32 p, %4, 0;\n"
      "mov.b64 da, {%1, %5};\nmov.b64 db, {%2, %5};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n.reg .b64 db;\nsetp.ne.b32 p, %4, 0;\n"
      "mov.b64 db, {%2, %5};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi) : "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  __syncwarp();
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  __syncwarp();
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  __syncwarp();
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(taddr) : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float y;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
  return y;
}
// Packed pairs of fp32 (sm_100 f32x2 arithmetic): halves the FMA-pipe instruction count of the
// softmax inner loop.
__device__ __forceinline__ uint64_t pack_f2(uint32_t lo, uint32_t hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}
__device__ __forceinline__ void unpack_f2(uint64_t x, float& lo, float& hi) {
  uint32_t a, b;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(x));
  lo = __uint_as_float(a);
  hi = __uint_as_float(b);
}
__device__ __forceinline__ uint64_t fma_f2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add_f2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);     // .x (low 16 bits) = lo
  return *reinterpret_cast<uint32_t*>(&h);
}

// Bits [c_lo, c_hi] of a 64-bit word set (none if the interval is empty); c_hi <= 63, c_lo >= 0.
__device__ __forceinline__ uint64_t visible_mask64(int c_lo, int c_hi) {
  if (c_hi < c_lo) return 0ull;
  return (~0ull << c_lo) & (~0ull >> (63 - c_hi));
}

// Instruction descriptor: fp32 accumulate, bf16 A and B, A K-major, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(uint32_t n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((n >> 3) << 17) |
         ((128u >> 4) << 24);
}

struct AttnArgs {
  const int32_t* table;
  int32_t* counter;              // global work counter (a header word of the table)
  int32_t off_bin_seg_ptr, off_bin_used, off_seg_start, off_items;
  int32_t n_items;               // geometry entries in the work list
  int32_t subs;                  // work indices per (KV head, geometry entry)
  int32_t pair_heads;            // 1: slots are two query heads; 0: two row tiles of one head
  int32_t group;                 // query heads per KV head
  int32_t fold;                  // independent mode: query heads folded into a query tile (tile row m is
  int32_t fold_shift;            //   bin row q_row0 + (m >> fold_shift) of head head[0] + (m & (fold - 1)))
  int32_t n_q_heads;
  int32_t capacity;              // rows per bin
  int32_t total_work;            // n_kv_heads * n_items * subs
  float scale_log2;              // softmax scale * log2(e)
  __nv_bfloat16* o;
  const float2* rope_table;      // [D/4][capacity][2] (cos, sin) pairs, or null: Q arrives already rotated
  int32_t* status;
  unsigned long long wait_limit_ns;
};

// What one work index means for a CTA.
struct Work {
  int bin, kv_row0, n, q_row0[2], jb[2], je[2], head[2], kv_head;
  int bin_used, seg_end, key_lo[2], seg_first[2], single_seg;
};

__device__ __forceinline__ void decode_work(const AttnArgs& a, int w, Work& wk) {
  const int sub = w % a.subs;
  const int rest = w / a.subs;
  const int gi = rest % a.n_items;
  wk.kv_head = rest / a.n_items;
  const int4* p = reinterpret_cast<const int4*>(a.table + a.off_items + kItemInts * gi);
  const int4 x = __ldg(p), y = __ldg(p + 1);
  wk.bin = x.x; wk.kv_row0 = x.y; wk.n = x.z; wk.q_row0[0] = x.w; wk.q_row0[1] = y.x;
  wk.jb[0] = 0; wk.je[0] = y.z;
  wk.jb[1] = y.y; wk.je[1] = (y.x >= 0) ? x.z : y.y;       // unused slot: empty range
  wk.bin_used = 0;
  if (a.pair_heads) {
    wk.head[0] = wk.kv_head * a.group + 2 * sub;
    wk.head[1] = wk.head[0] + 1;
  } else {
    wk.head[0] = wk.head[1] = wk.kv_head * a.group + sub * a.fold;
  }
}

// Second half of a work-list entry: what the softmax threads need to place their rows.
__device__ __forceinline__ void decode_rows(const AttnArgs& a, int w, Work& wk) {
  const int gi = (w / a.subs) % a.n_items;
  const int4* p = reinterpret_cast<const int4*>(a.table + a.off_items + kItemInts * gi);
  const int4 x = __ldg(p + 2), y = __ldg(p + 3);
  wk.bin_used = x.x; wk.seg_end = x.y; wk.key_lo[0] = x.z; wk.key_lo[1] = x.w;
  wk.seg_first[0] = y.x; wk.seg_first[1] = y.y; wk.single_seg = y.z;
}

// The fetching thread decodes an item once and publishes it in shared memory; every other role
// reads it from there instead of going back to global memory.
__device__ __forceinline__ void ring_write(volatile int* e, int w, const Work& wk) {
  e[0] = w; e[1] = wk.bin; e[2] = wk.kv_row0; e[3] = wk.n;
  e[4] = wk.q_row0[0]; e[5] = wk.q_row0[1]; e[6] = wk.jb[1]; e[7] = wk.je[0];
  e[8] = wk.je[1]; e[9] = wk.head[0]; e[10] = wk.head[1]; e[11] = wk.kv_head;
  e[12] = wk.bin_used; e[13] = wk.seg_end; e[14] = wk.key_lo[0]; e[15] = wk.key_lo[1];
  e[16] = wk.seg_first[0]; e[17] = wk.seg_first[1]; e[18] = wk.single_seg;
}

enum WaitCode { kWaitItemFull = 1, kWaitItemEmpty, kWaitQFull, kWaitQEmpty, kWaitKFull, kWaitKEmpty,
                kWaitVFull, kWaitVEmpty, kWaitS, kWaitP, kWaitOFull, kWaitOEmpty, kWaitPair, kWaitRowSum };

// Start row of the prompt that holds bin-local row `i_row`, among the prompts seg_begin .. seg_end-1
// of a bin whose start rows (ascending) are in `starts`; `lo` if none of them starts at or before the
// row. All 32 lanes call it with the same range and with row_max = the largest row of the warp: the
// starts are loaded 32 at a time, one per lane, and handed round with shuffles, so the walk costs one
// memory round trip per 32 prompts.
__device__ __forceinline__ int seg_start_at(const int32_t* starts, int seg_begin, int seg_end, int i_row, int row_max,
                                            int lo, int lane) {
  for (int base = seg_begin; base < seg_end; base += 32) {
    const int cnt = min(32, seg_end - base);
    const int mine = (lane < cnt) ? __ldg(starts + base + lane) : 0x7fffffff;
    for (int sg = 0; sg < cnt; ++sg) {
      const int st = __shfl_sync(0xffffffffu, mine, sg);
      if (st > row_max) return lo;                     // warp-uniform: no later prompt starts in these rows
      if (st <= i_row) lo = st;
    }
  }
  return lo;
}

// kIndep = false: the two slots of a CTA work on one item and share its K/V stream (long
//   sequences, GQA head pairs). kIndep = true: every slot draws its own single-tile items and loads
//   its own K/V tiles (64 rows each), so neither slot ever waits for the other (short prompts, where
//   pairing two row tiles of different length would leave one slot idle for a tile per item).
template <int D, bool kIndep>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o,
                 const AttnArgs args) {
  constexpr int BN = kIndep ? kTileNShort : kTileN;
  using Cfg = AttnCfg<D, BN>;
  constexpr int NK = Cfg::kKStages, NV = Cfg::kVStages, kChunks = Cfg::kChunks;

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t s_misc = smem_u32(smem_raw);
  uint8_t* misc = smem_raw;
  const uint32_t s_q = (s_misc + 3072u + 1023u) & ~1023u;       // [2] slots; tiles need 1024-byte alignment
  const uint32_t s_k = s_q + 2 * Cfg::kQBytes;                  // [NK]
  const uint32_t s_v = s_k + NK * Cfg::kKVBytes;                // [NV]
  const uint32_t s_stage_o = s_v + NV * Cfg::kKVBytes;          // [2] slots, epilogue staging
  {
    uint32_t dyn_bytes;
    asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_bytes));
    if (s_stage_o + 2 * Cfg::kStageOBytes > s_misc + dyn_bytes) {   // base less aligned than expected
      if (threadIdx.x == 0 && args.status) atomicCAS(args.status, 0, 100);
      return;
    }
  }
  // mbarriers, 8 bytes each
  const uint32_t bar_item_full = s_misc + 0;     // [2 rings][kRing]
  const uint32_t bar_item_empty = s_misc + 64;   // [2 rings][kRing]
  const uint32_t bar_q_full = s_misc + 128;      // [2]
  const uint32_t bar_q_empty = s_misc + 144;     // [2]
  const uint32_t bar_s_full = s_misc + 160;      // [2 slots][2 S buffers]; shared mode uses [t][0]
  const uint32_t bar_p_full = s_misc + 192;      // [2 slots][2 S buffers]
  const uint32_t bar_o_full = s_misc + 224;      // [2]
  const uint32_t bar_o_empty = s_misc + 240;     // [2]
  const uint32_t bar_k_full = s_misc + 256;      // [4]; independent mode: [2 slots][2 stages]
  const uint32_t bar_k_empty = s_misc + 288;     // [4]
  const uint32_t bar_v_full = s_misc + 320;      // [4]
  const uint32_t bar_v_empty = s_misc + 352;     // [4]
  const uint32_t bar_q_rot = s_misc + 384;       // [2] Q_t has been rotated in place (fused path)
  const uint32_t bar_pair0 = s_misc + 896;       // [2 slots][4 quadrants] rendezvous of the two warps that share rows
  const uint32_t bar_l_ready = s_misc + 976;     // [2][2] independent mode: the slot's row sums of item i are in shared memory ([slot][i & 1])
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(misc + 400);
  volatile int* s_abort = reinterpret_cast<volatile int*>(misc + 404);
  volatile int* s_ring = reinterpret_cast<volatile int*>(misc + 416);   // [2 rings][kRing][kRingInts]
  volatile float* s_xchg = reinterpret_cast<volatile float*>(misc + 1024);   // [2 slots][2 halves][128 rows]
  static_assert(416 + 2 * kRing * kRingInts * 4 <= 896, "ring does not fit");
  static_assert(NK <= 4 && NV <= 4, "barrier slots");

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const WaitCtx wctx{s_abort, args.status, args.wait_limit_ns};

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2 * (int)kRing; ++i) {
      mbar_init(bar_item_full + 8 * i, 1);
      // readers of a ring entry: the MMA thread and the softmax threads of the slot(s) it feeds;
      // in shared mode also the two Q loaders
      mbar_init(bar_item_empty + 8 * i, kIndep ? 1 + kSoftmaxThreads : 1 + 2 + 2 * kSoftmaxThreads);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_q_full + 8 * i, 1);
      mbar_init(bar_q_empty + 8 * i, 1);
      mbar_init(bar_q_rot + 8 * i, kIndep ? kSoftmaxThreads / 2 : kSoftmaxThreads);
      for (int b = 0; b < 2; ++b) {
        mbar_init(bar_s_full + 8 * (2 * i + b), 1);
        mbar_init(bar_p_full + 8 * (2 * i + b), kIndep ? kSoftmaxThreads / 2 : kSoftmaxThreads);
      }
      mbar_init(bar_o_full + 8 * i, 1);
      mbar_init(bar_o_empty + 8 * i, kIndep ? kSoftmaxThreads / 2 : kSoftmaxThreads);
      mbar_init(bar_l_ready + 16 * i, kSoftmaxThreads / 2);
      mbar_init(bar_l_ready + 16 * i + 8, kSoftmaxThreads / 2);
      for (int qd = 0; qd < 4; ++qd) mbar_init(bar_pair0 + 8 * (4 * i + qd), 64);
    }
    for (int s = 0; s < NK; ++s) { mbar_init(bar_k_full + 8 * s, 1); mbar_init(bar_k_empty + 8 * s, 1); }
    for (int s = 0; s < NV; ++s) { mbar_init(bar_v_full + 8 * s, 1); mbar_init(bar_v_empty + 8 * s, 1); }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(s_tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem_base;
  // Everything above is set-up that touches no tensor: with a programmatic dependent launch it runs
  // while the kernel before this one (rotation / cache scatter) is still finishing.
  pdl_wait();

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
    if constexpr (kIndep) {
      if (warp >= 2 && lane == 0) {
        // -------------------------------------------------------------- producer of slot t:
        // draws the slot's own items, loads Q and the item's K / V tiles (one stage each)
        const int t = warp - 2;
        const uint32_t ring_bar = 8 * (uint32_t)t * kRing;
        volatile int* ring_base = s_ring + t * (int)kRing * kRingInts;
        uint32_t it_n = 0, kc = 0;
        Work wk;
        while (true) {
          int w = atomicAdd(args.counter, 1);
          if (w >= args.total_work) w = -1;
          if (w >= 0) {
            decode_work(args, w, wk);
            decode_rows(args, w, wk);
          }
          const uint32_t ring = it_n % kRing;
          if (!mbar_wait(bar_item_empty + ring_bar + 8 * ring, ((it_n / kRing) & 1u) ^ 1u, wctx, kWaitItemEmpty)) break;
          if (w >= 0) ring_write(ring_base + ring * kRingInts, w, wk);
          else ring_base[ring * kRingInts] = -1;
          mbar_arrive(bar_item_full + ring_bar + 8 * ring);
          if (w < 0) break;
          // the slot's last Q.K^T of the previous item must have finished reading the Q buffer
          if (!mbar_wait(bar_q_empty + 8 * t, (it_n & 1u) ^ 1u, wctx, kWaitQEmpty)) break;
          mbar_expect_tx(bar_q_full + 8 * t, Cfg::kQBytes);
          for (int c = 0; c < kChunks; ++c)
            tma_load_4d(s_q + t * Cfg::kQBytes + c * (BM * 128), &map_q, bar_q_full + 8 * t,
                        c * 64, wk.head[0], wk.q_row0[0], wk.bin);
          bool ok = true;
          for (int j = 0; ok && j < wk.n; ++j, ++kc) {
            const int kv0 = wk.kv_row0 + j * BN;
            const uint32_t st = 2u * (uint32_t)t + (kc & 1u);          // the slot's stage for this tile
            const uint32_t free_parity = ((kc >> 1) & 1u) ^ 1u;
            ok = mbar_wait(bar_k_empty + 8 * st, free_parity, wctx, kWaitKEmpty);
            if (!ok) break;
            mbar_expect_tx(bar_k_full + 8 * st, Cfg::kKVBytes);
            for (int c = 0; c < kChunks; ++c)
              tma_load_4d(s_k + st * Cfg::kKVBytes + c * (BN * 128), &map_k, bar_k_full + 8 * st,
                          c * 64, wk.kv_head, kv0, wk.bin);
            ok = mbar_wait(bar_v_empty + 8 * st, free_parity, wctx, kWaitVEmpty);
            if (!ok) break;
            mbar_expect_tx(bar_v_full + 8 * st, Cfg::kKVBytes);
            for (int c = 0; c < kChunks; ++c)
              tma_load_4d(s_v + st * Cfg::kKVBytes + c * (BN * 128), &map_v, bar_v_full + 8 * st,
                          c * 64, wk.kv_head, kv0, wk.bin);
          }
          if (!ok) break;
          ++it_n;
        }
      } else if (warp < 2 && lane == 0) {
        // -------------------------------------------------------------- MMA issuer of slot t
        // One issuing thread per slot (warps 0 and 1 sit on different schedulers), plain blocking
        // waits. S_t has two 64-column buffers, tile k of the slot's stream uses buffer k & 1, and
        // P(k) is written over S(k). The issue order  S(k+1), then P(k) V(k)  lets the tensor pipe
        // compute the next scores while the softmax threads work on tile k, and P(k) V(k) while they
        // work on tile k+1; the pipe runs one thread's MMAs in order, so S(k+2) cannot overwrite
        // P(k) before P(k) V(k) has read it.
        const int t = warp;
        constexpr uint32_t idesc_qk = instr_desc(BN, false);
        constexpr uint32_t idesc_pv = instr_desc(D, true);
        const uint32_t a_lo = desc_lo(s_q, 0) + (uint32_t)t * (Cfg::kQBytes >> 4);
        const uint32_t k_lo = desc_lo(s_k, 0) + 2u * (uint32_t)t * (Cfg::kKVBytes >> 4);
        const uint32_t v_lo = desc_lo(s_v, BN * 128) + 2u * (uint32_t)t * (Cfg::kKVBytes >> 4);
        const uint32_t tm_s = tmem_base + Cfg::kTmemS + 128u * (uint32_t)t;
        const uint32_t tm_o = tmem_base + Cfg::kTmemO + (uint32_t)D * (uint32_t)t;
        const uint32_t bar_q_ready = (args.rope_table ? bar_q_rot : bar_q_full) + 8 * t;
        const uint32_t b_item_full = bar_item_full + 8 * (uint32_t)t * kRing;
        const uint32_t b_item_empty = bar_item_empty + 8 * (uint32_t)t * kRing;
        const uint32_t b_k_full = bar_k_full + 16 * t, b_k_empty = bar_k_empty + 16 * t;   // [stage]
        const uint32_t b_v_full = bar_v_full + 16 * t, b_v_empty = bar_v_empty + 16 * t;
        const uint32_t b_s_full = bar_s_full + 16 * t, b_p_full = bar_p_full + 16 * t;     // [buffer]
        const uint32_t b_o_full = bar_o_full + 8 * t, b_o_empty = bar_o_empty + 8 * t;
        const uint32_t b_q_empty = bar_q_empty + 8 * t;
        uint32_t it_n = 0, kc = 0;       // items and key tiles consumed
        bool ok = true;
        // S(kq) = Q_t K(kq)^T into buffer kq & 1
        auto issue_qk = [&](const uint32_t kq, const bool last_of_item) -> bool {
          const uint32_t b = kq & 1u;
          if (!mbar_wait(b_k_full + 8 * b, (kq >> 1) & 1u, wctx, kWaitKFull)) return false;
          tc_fence_after();
          const uint32_t d = tm_s + 64u * b;
          const uint32_t kb = k_lo + b * (Cfg::kKVBytes >> 4);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            constexpr uint32_t kChunkQ = (BM * 128) >> 4, kChunkK = (BN * 128) >> 4;
            mma_ss(d, a_lo + (uint32_t)(kk >> 2) * kChunkQ + (uint32_t)(kk & 3) * 2,
                   kb + (uint32_t)(kk >> 2) * kChunkK + (uint32_t)(kk & 3) * 2, idesc_qk, kk > 0 ? 1u : 0u);
          }
          tc_commit(b_k_empty + 8 * b);
          tc_commit(b_s_full + 8 * b);
          if (last_of_item) tc_commit(b_q_empty);     // last read of Q_t in this item
          return true;
        };
        // The slot's tiles form one stream across items: while the softmax threads work on tile k,
        // the scores of the stream's next tile are computed, also when that tile opens the slot's
        // next item (its Q was loaded as soon as this item's last scores had been issued).
        int w = -1, n = 0, j = 0;
        {
          if (!mbar_wait(b_item_full, 0u, wctx, kWaitItemFull)) ok = false;
          if (ok) {
            const volatile int* e = s_ring + (t * (int)kRing) * kRingInts;
            w = e[0]; n = e[3];
            mbar_arrive(b_item_empty);
          }
        }
        if (ok && w >= 0) ok = mbar_wait(bar_q_ready, 0u, wctx, kWaitQFull) && issue_qk(kc, n == 1);
        while (ok && w >= 0) {
          const bool last_tile = (j + 1 == n);
          int w_next = w, n_next = n;
          bool have = true, last_flag = (j + 2 == n);
          // With one tile per item the next item's scores would be issued before the previous item's
          // epilogue has read O_t; the softmax threads must not get that far ahead of it.
          if (j == 0 && last_tile && !(ok = mbar_wait(b_o_empty, (it_n & 1u) ^ 1u, wctx, kWaitOEmpty))) break;
          if (last_tile) {
            const uint32_t item = it_n + 1u, ring = item % kRing;
            if (!(ok = mbar_wait(b_item_full + 8 * ring, (item / kRing) & 1u, wctx, kWaitItemFull))) break;
            const volatile int* e = s_ring + (t * (int)kRing + (int)ring) * kRingInts;
            w_next = e[0]; n_next = e[3];
            mbar_arrive(b_item_empty + 8 * ring);
            have = w_next >= 0;
            last_flag = n_next == 1;
            if (have && !(ok = mbar_wait(bar_q_ready, item & 1u, wctx, kWaitQFull))) break;
          }
          if (have && !(ok = issue_qk(kc + 1, last_flag))) break;
          // the previous item's epilogue must have read O_t before it is overwritten
          if (j == 0 && !last_tile && !(ok = mbar_wait(b_o_empty, (it_n & 1u) ^ 1u, wctx, kWaitOEmpty))) break;
          const uint32_t b = kc & 1u, parity = (kc >> 1) & 1u;
          if (!(ok = mbar_wait(b_p_full + 8 * b, parity, wctx, kWaitP))) break;
          if (!(ok = mbar_wait(b_v_full + 8 * b, parity, wctx, kWaitVFull))) break;
          tc_fence_after();            // O_t (+)= P(k) V(k)
          const uint32_t a = tm_s + 64u * b;
          const uint32_t vb = v_lo + b * (Cfg::kKVBytes >> 4);
          mma_ts(tm_o, a, vb, idesc_pv, j == 0 ? 0u : 1u);
#pragma unroll
          for (int kk = 1; kk < BN / 16; ++kk)
            mma_ts(tm_o, a + kk * 8, vb + (uint32_t)kk * ((16 * 128) >> 4), idesc_pv, 1u);
          tc_commit(b_v_empty + 8 * b);
          ++kc;
          if (last_tile) {
            tc_commit(b_o_full);
            ++it_n;
            w = w_next; n = n_next; j = 0;
          } else {
            ++j;
          }
        }
      }
    } else {
    if (warp == 0 && lane == 0) {
      // ---------------------------------------------------------------- work fetch + K/V producer
      uint32_t it_n = 0, kc = 0;
      Work wk;
      while (true) {
        int w = atomicAdd(args.counter, 1);
        if (w >= args.total_work) w = -1;
        if (w >= 0) {
          decode_work(args, w, wk);
          decode_rows(args, w, wk);
        }
        const uint32_t ring = it_n % kRing;
        if (!mbar_wait(bar_item_empty + 8 * ring, ((it_n / kRing) & 1u) ^ 1u, wctx, kWaitItemEmpty)) break;
        if (w >= 0) ring_write(s_ring + ring * kRingInts, w, wk);
        else s_ring[ring * kRingInts] = -1;
        mbar_arrive(bar_item_full + 8 * ring);
        if (w < 0) break;
        bool ok = true;
        for (int j = 0; ok && j < wk.n; ++j, ++kc) {
          const int kv0 = wk.kv_row0 + j * BN;
          uint32_t s = kc % NK;
          ok = mbar_wait(bar_k_empty + 8 * s, ((kc / NK) & 1u) ^ 1u, wctx, kWaitKEmpty);
          if (!ok) break;
          mbar_expect_tx(bar_k_full + 8 * s, Cfg::kKVBytes);
          for (int c = 0; c < kChunks; ++c)
            tma_load_4d(s_k + s * Cfg::kKVBytes + c * (BN * 128), &map_k, bar_k_full + 8 * s,
                        c * 64, wk.kv_head, kv0, wk.bin);
          s = kc % NV;
          ok = mbar_wait(bar_v_empty + 8 * s, ((kc / NV) & 1u) ^ 1u, wctx, kWaitVEmpty);
          if (!ok) break;
          mbar_expect_tx(bar_v_full + 8 * s, Cfg::kKVBytes);
          for (int c = 0; c < kChunks; ++c)
            tma_load_4d(s_v + s * Cfg::kKVBytes + c * (BN * 128), &map_v, bar_v_full + 8 * s,
                        c * 64, wk.kv_head, kv0, wk.bin);
        }
        if (!ok) break;
        ++it_n;
      }
    } else if (warp >= 2 && lane == 0) {
      // ---------------------------------------------------------------- Q loader of slot t
      const int t = warp - 2;
      uint32_t it_n = 0;
      while (true) {
        const uint32_t ring = it_n % kRing;
        if (!mbar_wait(bar_item_full + 8 * ring, (it_n / kRing) & 1u, wctx, kWaitItemFull)) break;
        const volatile int* e = s_ring + ring * kRingInts;
        const int w = e[0], bin = e[1];
        const int q_row0 = e[4 + t], head = e[9 + t];
        const bool used = t ? (e[6] < e[8]) : (e[7] > 0);
        mbar_arrive(bar_item_empty + 8 * ring);
        if (w < 0) break;
        // the slot's last Q.K^T of the previous item must have finished reading the buffer
        if (!mbar_wait(bar_q_empty + 8 * t, (it_n & 1u) ^ 1u, wctx, kWaitQEmpty)) break;
        if (used) {
          mbar_expect_tx(bar_q_full + 8 * t, Cfg::kQBytes);
          for (int c = 0; c < kChunks; ++c)
            tma_load_4d(s_q + t * Cfg::kQBytes + c * (BM * 128), &map_q, bar_q_full + 8 * t,
                        c * 64, head, q_row0, bin);
        } else {
          mbar_arrive(bar_q_full + 8 * t);
        }
        ++it_n;
      }
    } else if (warp == 1 && lane == 0) {
      // ---------------------------------------------------------------- MMA issuer
      // Kept lean on purpose: one thread feeds the tensor pipe, so every scalar instruction
      // between two tcgen05.mma counts. Descriptor low words are precomputed; inside a group of
      // MMAs only compile-time constants are added.
      constexpr uint32_t idesc_qk = instr_desc(BN, false);
      constexpr uint32_t idesc_pv = instr_desc(D, true);
      const uint32_t q_lo0 = desc_lo(s_q, 0), k_lo0 = desc_lo(s_k, 0), v_lo0 = desc_lo(s_v, BN * 128);
      uint32_t it_n = 0, kc0 = 0, vc0 = 0, tc0 = 0, tc1 = 0;
      int n = 0, je0 = 0, jb1 = 0, je1 = 0;
      bool ok = true;
      // S_t = Q_t K_j^T; the K stage is released after the last slot that reads it
      auto issue_qk = [&](const int t, const int j) -> bool {
        const uint32_t kc = kc0 + (uint32_t)j, s = kc % NK;
        if (!mbar_wait(bar_k_full + 8 * s, (kc / NK) & 1u, wctx, kWaitKFull)) return false;
        tc_fence_after();
        const uint32_t d = tmem_base + Cfg::kTmemS + 128u * t;
        const uint32_t a_lo = q_lo0 + (uint32_t)t * (Cfg::kQBytes >> 4);
        const uint32_t b_lo = k_lo0 + s * (Cfg::kKVBytes >> 4);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          constexpr uint32_t kChunkQ = (BM * 128) >> 4, kChunkK = (BN * 128) >> 4;
          mma_ss(d, a_lo + (uint32_t)(kk >> 2) * kChunkQ + (uint32_t)(kk & 3) * 2,
                 b_lo + (uint32_t)(kk >> 2) * kChunkK + (uint32_t)(kk & 3) * 2, idesc_qk, kk > 0 ? 1u : 0u);
        }
        if (t == 1 || !(j >= jb1 && j < je1)) tc_commit(bar_k_empty + 8 * s);
        tc_commit(bar_s_full + 16 * t);
        // the slot's last scores of this item: its Q buffer is free for the next item's Q from here on
        if (j + 1 == (t ? je1 : je0)) tc_commit(bar_q_empty + 8 * t);
        return true;
      };
      // O_t (+)= P_t V_j, then either the next S_t or the end-of-item signals of slot t
      auto slot_step = [&](const int t, const int j, const int jb, const int je, uint32_t& tcount) -> bool {
        if (j >= jb && j < je) {
          const bool first = (j == jb);
          // the previous item's epilogue must have read O_t before it is overwritten
          if (first && !mbar_wait(bar_o_empty + 8 * t, (it_n & 1u) ^ 1u, wctx, kWaitOEmpty)) return false;
          if (!mbar_wait(bar_p_full + 16 * t, tcount & 1u, wctx, kWaitP)) return false;
          const uint32_t vc = vc0 + (uint32_t)j, s = vc % NV;
          if (!mbar_wait(bar_v_full + 8 * s, (vc / NV) & 1u, wctx, kWaitVFull)) return false;
          tc_fence_after();
          const uint32_t a = tmem_base + Cfg::kTmemS + 128u * t;
          const uint32_t d = tmem_base + Cfg::kTmemO + (uint32_t)D * t;
          const uint32_t b_lo = v_lo0 + s * (Cfg::kKVBytes >> 4);
          mma_ts(d, a, b_lo, idesc_pv, first ? 0u : 1u);
#pragma unroll
          for (int kk = 1; kk < BN / 16; ++kk)
            mma_ts(d, a + kk * 8, b_lo + (uint32_t)kk * ((16 * 128) >> 4), idesc_pv, 1u);
          ++tcount;
          if (t == 1 || !(j >= jb1 && j < je1)) tc_commit(bar_v_empty + 8 * s);
          if (j + 1 < je) return issue_qk(t, j + 1);
          tc_commit(bar_o_full + 8 * t);       // slot t is done with this item
          return true;
        }
        if (j + 1 == jb && jb < je) return issue_qk(t, j + 1);   // slot t joins the key loop at the next tile
        return true;
      };
      while (ok) {
        const uint32_t ring = it_n % kRing;
        if (!mbar_wait(bar_item_full + 8 * ring, (it_n / kRing) & 1u, wctx, kWaitItemFull)) break;
        const volatile int* e = s_ring + ring * kRingInts;
        const int w = e[0];
        n = e[3]; jb1 = e[6]; je0 = e[7]; je1 = e[8];
        mbar_arrive(bar_item_empty + 8 * ring);
        if (w < 0) break;
        const uint32_t bar_q_ready = args.rope_table ? bar_q_rot : bar_q_full;
        ok = mbar_wait(bar_q_ready + 0, it_n & 1u, wctx, kWaitQFull) &&
             mbar_wait(bar_q_ready + 8, it_n & 1u, wctx, kWaitQFull);
        if (!ok) break;
        if (je0 > 0) ok = issue_qk(0, 0);
        if (ok && jb1 == 0 && je1 > 0) ok = issue_qk(1, 0);
        for (int j = 0; ok && j < n; ++j) {
          ok = slot_step(0, j, 0, je0, tc0);
          if (ok) ok = slot_step(1, j, jb1, je1, tc1);
        }
        if (!ok) break;
        // Unused slot: keep its per-item barriers in step. o_full must not complete two phases
        // before every softmax thread has seen the first, so wait until all of them are past the
        // previous item's o_full (they signal that on o_empty).
        if (je0 <= 0) {
          if (!(ok = mbar_wait(bar_o_empty + 0, (it_n & 1u) ^ 1u, wctx, kWaitOEmpty))) break;
          mbar_arrive(bar_q_empty + 0);
          mbar_arrive(bar_o_full + 0);
        }
        if (jb1 >= je1) {
          if (!(ok = mbar_wait(bar_o_empty + 8, (it_n & 1u) ^ 1u, wctx, kWaitOEmpty))) break;
          mbar_arrive(bar_q_empty + 8);
          mbar_arrive(bar_o_full + 8);
        }
        kc0 += (uint32_t)n;
        vc0 += (uint32_t)n;
        ++it_n;
      }
    }
    }   // shared-stream roles
  } else {
    // ------------------------------------------------------------------ softmax + epilogue
    const int t = (warp - 4) >> 3;                   // slot
    const int h = ((warp - 4) >> 2) & 1;             // shared mode: which 64 keys of a 128-key tile this thread owns
    const int quad = warp & 3;                       // TMEM lane quadrant this warp may access
    const int row = quad * 32 + lane;                // query row inside the tile
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const uint32_t tmem_s = tmem_base + Cfg::kTmemS + 128u * t + lane_base;
    const uint32_t tmem_o = tmem_base + Cfg::kTmemO + (uint32_t)D * t + lane_base;

    if constexpr (kIndep) {
      // ---------------------------------------------------------------- independent mode
      // Per slot: warps with h == 0 are the softmax threads, one per query row (all 64 scores of a
      // tile), and never leave the tile loop; warps with h == 1 are helper threads, one per row, which
      // rotate the next item's Q in shared memory (fused path) and run the epilogue of the previous
      // item, both off the softmax threads' critical path.
      const float c_scale = args.scale_log2;
      const int32_t* tb = args.table;
      const int fs = args.fold_shift;                  // tile row m holds bin row q_row0 + (m >> fs)
      const uint32_t ring0 = (uint32_t)t * kRing;
      // row sums travel from the softmax thread to the helper of the same row, double-buffered by item
      volatile float* x_l = s_xchg + t * 128 + row;            // + 256 * (item & 1)
      bool ok = true;
      // key range [key_lo, key_hi] of this thread's row from a ring entry (empty for padding rows)
      // (all lanes of the warp call it together: the prompts' start rows are loaded once per warp)
      auto row_range = [&](const volatile int* e, int& key_lo, int& key_hi) {
        const int i_row = e[4] + (row >> fs);
        int lo = e[14];
        if (!(e[18] & 1))
          lo = seg_start_at(tb + args.off_seg_start, e[16] + 1, e[13], i_row, e[4] + ((quad * 32 + 31) >> fs), lo, lane);
        const bool real = i_row < e[12];
        key_lo = real ? lo : 1;
        key_hi = real ? i_row : 0;
      };
      if (h == 0) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmaxIndep));
        uint32_t it_n = 0, tcount = 0;
        while (true) {
          const uint32_t ring = ring0 + it_n % kRing;
          ok = __all_sync(0xffffffffu, mbar_wait(bar_item_full + 8 * ring, (it_n / kRing) & 1u, wctx, kWaitItemFull));
          if (!ok) break;
          const volatile int* e = s_ring + ring * kRingInts;
          const int w = e[0], item_kv_row0 = e[2], n_tiles = e[3];
          int key_lo, key_hi;
          if (w >= 0) row_range(e, key_lo, key_hi);
          mbar_arrive(bar_item_empty + 8 * ring);
          if (w < 0) break;
          float m_run = -INFINITY;      // running maximum of the row, in scaled log2 units
          float l_run = 0.f;            // running sum of exp2(s * c - m_run)
          for (int j = 0; j < n_tiles; ++j) {
            constexpr int EPT = BN;                              // scores per thread and tile
            constexpr int NCH = EPT / 32;                        // 32-column TMEM round trips
            const int kv0 = item_kv_row0 + j * BN;
            const int c_lo = max(key_lo - kv0, 0);
            const int c_hi = min(key_hi - kv0, EPT - 1);         // visible columns [c_lo, c_hi]
            // one warp reduction for all the per-warp flags of the tile: which 32-column chunks
            // somebody can see, and whether any row's interval ends or begins inside the tile
            static_assert(NCH == 2, "flag bits below are laid out for two chunks");
            const uint64_t vis = visible_mask64(c_lo, c_hi);     // bit i: column i is visible to this row
            const uint32_t vis_lo = (uint32_t)vis, vis_hi = (uint32_t)(vis >> 32);
            const uint32_t lane_flags = (uint32_t)(vis_lo != 0u) | ((uint32_t)(vis_hi != 0u) << 1) |
                                        ((uint32_t)(~vis != 0ull) << 2);
            const uint32_t warp_flags = __reduce_or_sync(0xffffffffu, lane_flags);
            const bool need[NCH] = {(warp_flags & 1u) != 0, (warp_flags & 2u) != 0};
            const bool cut = (warp_flags & 4u) != 0;
            const uint32_t sbuf = tcount & 1u;                   // tile k of the stream lives in S buffer k & 1
            const uint32_t tmem_sb = tmem_s + 64u * sbuf;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_s_full + 8 * (2 * t + sbuf), (tcount >> 1) & 1u, wctx, kWaitS));
            if (!ok) break;
            tc_fence_after();
            uint32_t v[EPT];
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
              if (need[ch]) {
                tmem_ld32(tmem_sb + 32 * ch, *reinterpret_cast<uint32_t(*)[32]>(&v[32 * ch]));
              } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[32 * ch + i] = 0xff800000u;        // -inf
              }
            }
            tc_wait_ld();
            // masked tiles (the causal diagonal, the first tile of a prompt): one select per score,
            // steered by the bits of the row's visibility mask
            if (cut) {
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] = (vis_lo & (1u << i)) ? v[i] : 0xff800000u;
#pragma unroll
              for (int i = 0; i < 32; ++i) v[32 + i] = (vis_hi & (1u << i)) ? v[32 + i] : 0xff800000u;
            }
            float mx;
            {
              float m0 = fmax3(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]));
              float m1 = fmax3(__uint_as_float(v[3]), __uint_as_float(v[4]), __uint_as_float(v[5]));
              float m2 = fmax3(__uint_as_float(v[6]), __uint_as_float(v[7]), __uint_as_float(v[8]));
              float m3 = fmax3(__uint_as_float(v[9]), __uint_as_float(v[10]), __uint_as_float(v[11]));
#pragma unroll
              for (int i = 12; i + 7 < EPT; i += 8) {
                m0 = fmax3(m0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
                m1 = fmax3(m1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
                m2 = fmax3(m2, __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
                m3 = fmax3(m3, __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
              }
              m0 = fmax3(m0, __uint_as_float(v[EPT - 4]), __uint_as_float(v[EPT - 3]));
              m1 = fmax3(m1, __uint_as_float(v[EPT - 2]), __uint_as_float(v[EPT - 1]));
              mx = fmaxf(fmax3(m0, m1, m2), m3);
            }
            // lazy running-maximum update: keep the stale maximum while the new one is < 2^8 above it
            const float m_tile = mx * c_scale;
            float m_new = m_run;
            if (m_tile > m_run + 8.f) m_new = m_tile;
            const bool rescale = (m_new != m_run) && (m_run != -INFINITY);
            const float alpha = rescale ? fast_exp2(m_run - m_new) : 1.f;
            if (j > 0 && __any_sync(0xffffffffu, rescale)) {
              // S(k) is computed ahead of P(k-1) V(k-1), so O_t is stable only once that product has
              // been committed: the release of the V stage it read is the same event
              const uint32_t kp = tcount - 1u;
              ok = __all_sync(0xffffffffu, mbar_wait(bar_v_empty + 8 * (2 * t + (kp & 1u)), (kp >> 1) & 1u, wctx, kWaitVEmpty));
              if (!ok) break;
              tc_fence_after();
#pragma unroll 1
              for (int ch = 0; ch < D / 16; ++ch) {          // rare path: keep it small
                uint32_t ov[16];
                tmem_ld16(tmem_o + ch * 16, ov);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
                tmem_st16(tmem_o + ch * 16, ov);
              }
            }
            l_run *= alpha;
            m_run = m_new;
            const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;
            // p = exp2(s * c - m), row sum, P (bf16) written over the first half of the S buffer
            const uint64_t c2 = pack_f2(__float_as_uint(c_scale), __float_as_uint(c_scale));
            const uint64_t negm2 = pack_f2(__float_as_uint(neg_m), __float_as_uint(neg_m));
            uint64_t sum_a = 0ull, sum_b = 0ull;
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
              uint32_t pk[16];
              if (need[ch]) {
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                  float p0, p1, p2, p3;
                  unpack_f2(fma_f2(pack_f2(v[ch * 32 + i], v[ch * 32 + i + 1]), c2, negm2), p0, p1);
                  unpack_f2(fma_f2(pack_f2(v[ch * 32 + i + 2], v[ch * 32 + i + 3]), c2, negm2), p2, p3);
                  p0 = fast_exp2(p0); p1 = fast_exp2(p1); p2 = fast_exp2(p2); p3 = fast_exp2(p3);
                  sum_a = add_f2(sum_a, pack_f2(__float_as_uint(p0), __float_as_uint(p1)));
                  sum_b = add_f2(sum_b, pack_f2(__float_as_uint(p2), __float_as_uint(p3)));
                  pk[i >> 1] = pack_bf16(p0, p1);
                  pk[(i >> 1) + 1] = pack_bf16(p2, p3);
                }
              } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) pk[i] = 0u;
              }
              // S(k) was read completely above, so P(k) may overwrite its first columns
              tmem_st16(tmem_sb + ch * 16, pk);
            }
            float sum0, sum1, sum2, sum3;
            unpack_f2(sum_a, sum0, sum1);
            unpack_f2(sum_b, sum2, sum3);
            l_run += (sum0 + sum2) + (sum1 + sum3);
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bar_p_full + 8 * (2 * t + sbuf));
            ++tcount;
          }
          if (!ok) break;
          // The row sum goes to the helper thread of this row (arrive has release semantics). The
          // softmax threads can finish item i+1 before the helpers have picked up item i, but not
          // item i+2 (its scores are issued after the epilogue of item i has read O_t), so the
          // hand-over is double-buffered by item parity, barrier included.
          x_l[256 * (it_n & 1u)] = l_run;
          mbar_arrive(bar_l_ready + 16 * t + 8 * (it_n & 1u));
          ++it_n;
        }
      } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsHelper));
        uint32_t it_n = 0;
        int p_q_row0 = 0, p_head = 0, p_bin = 0;         // coordinates of the previous item (its epilogue is due)
        while (true) {
          const uint32_t ring = ring0 + it_n % kRing;
          ok = __all_sync(0xffffffffu, mbar_wait(bar_item_full + 8 * ring, (it_n / kRing) & 1u, wctx, kWaitItemFull));
          if (!ok) break;
          const volatile int* e = s_ring + ring * kRingInts;
          const int w = e[0], c_bin = e[1], c_q_row0 = e[4], c_head = e[9];
          int key_lo = 1, key_hi = 0;
          if (w >= 0 && args.rope_table) row_range(e, key_lo, key_hi);
          mbar_arrive(bar_item_empty + 8 * ring);
          if (w >= 0 && args.rope_table) {
            // rotate row `row` of this item's Q in shared memory by the angles of its position, with
            // the same fp32 arithmetic and rounding as the stand-alone kernel, then report Q_t ready
            ok = __all_sync(0xffffffffu, mbar_wait(bar_q_full + 8 * t, it_n & 1u, wctx, kWaitQFull));
            if (!ok) break;
            const int pos = key_hi - key_lo;             // < 0 for padding rows
            if (pos > 0) {
              constexpr int kUnits = D / 16;             // 16-byte (lower, upper) unit pairs per row
              const uint32_t q_row = s_q + (uint32_t)t * Cfg::kQBytes + (uint32_t)row * 128;
              // table[g][pos] = (cos, sin) of j = 2g and 2g + 1: consecutive rows read consecutive 16 bytes
              const float4* tab = reinterpret_cast<const float4*>(args.rope_table) + pos;
#pragma unroll 1
              for (int u0 = 0; u0 < kUnits; u0 += 2) {
                float4 cs[2][4];                         // table loads of two units first: one L2 round trip
#pragma unroll
                for (int uu = 0; uu < 2; ++uu)
#pragma unroll
                  for (int i = 0; i < 4; ++i)
                    cs[uu][i] = __ldg(tab + (size_t)((u0 + uu) * 4 + i) * (size_t)args.capacity);
#pragma unroll
                for (int uu = 0; uu < 2; ++uu) {
                  const int u = u0 + uu;                 // pairs (8u .. 8u+7, + D/2)
                  const uint32_t a_lo = q_row + ((((uint32_t)u) ^ ((uint32_t)row & 7u)) << 4);
                  const uint32_t a_hi = (D == 128)
                      ? q_row + (BM * 128) + ((((uint32_t)u) ^ ((uint32_t)row & 7u)) << 4)
                      : q_row + ((((uint32_t)(u + kUnits)) ^ ((uint32_t)row & 7u)) << 4);
                  uint32_t lo[4], hi[4];
                  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(lo[0]), "=r"(lo[1]), "=r"(lo[2]), "=r"(lo[3]) : "r"(a_lo));
                  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(hi[0]), "=r"(hi[1]), "=r"(hi[2]), "=r"(hi[3]) : "r"(a_hi));
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    const float4 c = cs[uu][i];          // (cos, sin) of two consecutive j
                    const __nv_bfloat162 l2 = *reinterpret_cast<__nv_bfloat162*>(&lo[i]);
                    const __nv_bfloat162 h2 = *reinterpret_cast<__nv_bfloat162*>(&hi[i]);
                    const float2 a = __bfloat1622float2(l2), b = __bfloat1622float2(h2);
                    lo[i] = pack_bf16(__fmaf_rn(a.x, c.x, -__fmul_rn(b.x, c.y)), __fmaf_rn(a.y, c.z, -__fmul_rn(b.y, c.w)));
                    hi[i] = pack_bf16(__fmaf_rn(b.x, c.x, __fmul_rn(a.x, c.y)), __fmaf_rn(b.y, c.z, __fmul_rn(a.y, c.w)));
                  }
                  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_lo), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]) : "memory");
                  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_hi), "r"(hi[0]), "r"(hi[1]), "r"(hi[2]), "r"(hi[3]) : "memory");
                }
              }
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // visible to the tensor core
            }
            mbar_arrive(bar_q_rot + 8 * t);
          }
          if (it_n > 0) {
            // epilogue of the previous item: O_t / l -> bf16 -> shared memory (128-byte swizzle) -> TMA store
            const uint32_t pi = it_n - 1u;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_o_full + 8 * t, pi & 1u, wctx, kWaitOFull));
            if (!ok) break;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_l_ready + 16 * t + 8 * (pi & 1u), (pi >> 1) & 1u, wctx, kWaitRowSum));
            if (!ok) break;
            tc_fence_after();
            const float l_row = x_l[256 * (pi & 1u)];
            const float inv_l = l_row > 0.f ? 1.f / l_row : 0.f;
            // Each warp stages and stores its own 32 rows (a 32-row TMA box), so the epilogue needs
            // no rendezvous between warps: lane 0 issues the warp's stores and is the one to wait
            // until the previous store has read the staging rows.
            const uint32_t stage = s_stage_o + (uint32_t)t * Cfg::kStageOBytes + (uint32_t)quad * (32 * 128);
            const uint32_t stage_row = stage + (uint32_t)lane * 128;
            const int p_row0 = p_q_row0 + ((32 * quad) >> fs);   // the warp's 32 tile rows: 32 >> fs bin rows x fold heads
#pragma unroll 1
            for (int hh = 0; hh < D / 64; ++hh) {          // 64 columns (one TMA box) at a time
              if (lane == 0) tma_store_wait_read();
              __syncwarp();
              uint32_t ov[64];
              tmem_ld32(tmem_o + hh * 64, *reinterpret_cast<uint32_t(*)[32]>(&ov[0]));
              tmem_ld32(tmem_o + hh * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&ov[32]));
              tc_wait_ld();
              if (hh == D / 64 - 1) {
                tc_fence_before();
                mbar_arrive(bar_o_empty + 8 * t);        // O_t may be overwritten by the next item now
              }
#pragma unroll
              for (int c16 = 0; c16 < 8; ++c16) {
                const uint32_t addr = stage_row + (((uint32_t)c16 ^ ((uint32_t)lane & 7u)) << 4);
                const uint32_t w0 = pack_bf16(__uint_as_float(ov[c16 * 8 + 0]) * inv_l, __uint_as_float(ov[c16 * 8 + 1]) * inv_l);
                const uint32_t w1 = pack_bf16(__uint_as_float(ov[c16 * 8 + 2]) * inv_l, __uint_as_float(ov[c16 * 8 + 3]) * inv_l);
                const uint32_t w2 = pack_bf16(__uint_as_float(ov[c16 * 8 + 4]) * inv_l, __uint_as_float(ov[c16 * 8 + 5]) * inv_l);
                const uint32_t w3 = pack_bf16(__uint_as_float(ov[c16 * 8 + 6]) * inv_l, __uint_as_float(ov[c16 * 8 + 7]) * inv_l);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
              }
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
              __syncwarp();
              if (lane == 0 && p_row0 < args.capacity) {
                tma_store_4d(&map_o, stage, hh * 64, p_head, p_row0, p_bin);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
              }
            }
            if (!ok) break;
          }
          if (w < 0) break;
          p_q_row0 = c_q_row0; p_head = c_head; p_bin = c_bin;
          ++it_n;
        }
        if (lane == 0) tma_store_wait_read();    // staging must outlive the last store's read
      }
    } else {
    // ---------------------------------------------------------------- shared-stream mode
    // All softmax warps run the same code (slot and half at run time): the unrolled row loops are
    // large and several copies of them would not stay resident in the instruction caches.
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    volatile float* x_mine = s_xchg + (t * 2 + h) * 128 + row;
    volatile float* x_other = s_xchg + (t * 2 + (h ^ 1)) * 128 + row;
    // Rendezvous points are mbarriers (arrive, then a bounded wait) rather than named barriers, so
    // that a warp whose partner gave up on a wait cannot be left waiting for it.
    const uint32_t bar_pair = bar_pair0 + 8 * (uint32_t)(t * 4 + quad);
    uint32_t pair_ph = 0;
    auto rendezvous = [&](const uint32_t bar, uint32_t& ph, const int code) -> bool {
      mbar_arrive(bar);
      const bool r = __all_sync(0xffffffffu, mbar_wait(bar, ph, wctx, code));
      ph ^= 1u;
      return r;
    };
    const float c_scale = args.scale_log2;
    const int32_t* tb = args.table;
    uint32_t it_n = 0, tcount = 0;
    bool ok = true;
    // Rotates this thread's part of row `row` of Q_t in shared memory by the angles of position
    // `pos` (<= 0: nothing to do), with the same fp32 arithmetic and rounding as the stand-alone
    // kernel, then reports the slot's Q as ready. Waits for the TMA load of Q first.
    auto rotate_q = [&](const int pos, const uint32_t parity) -> bool {
      if (!__all_sync(0xffffffffu, mbar_wait(bar_q_full + 8 * t, parity, wctx, kWaitQFull))) return false;
      if (pos > 0) {
        constexpr int kUnits = D / 16;                 // 16-byte units per half of a row
        const uint32_t q_row = s_q + (uint32_t)t * Cfg::kQBytes + (uint32_t)row * 128;
        // table[g][pos] = (cos, sin) of j = 2g and 2g + 1: consecutive rows read consecutive 16 bytes
        const float4* tab = reinterpret_cast<const float4*>(args.rope_table) + pos;
        float4 cs[kUnits / 2][4];                      // all table loads first: one L2 round trip
#pragma unroll
        for (int uu = 0; uu < kUnits / 2; ++uu)
#pragma unroll
          for (int i = 0; i < 4; ++i)
            cs[uu][i] = __ldg(tab + (size_t)((h * (kUnits / 2) + uu) * 4 + i) * (size_t)args.capacity);
#pragma unroll
        for (int uu = 0; uu < kUnits / 2; ++uu) {
          const int u = h * (kUnits / 2) + uu;         // pairs (8u .. 8u+7, + D/2)
          const uint32_t a_lo = q_row + ((((uint32_t)u) ^ ((uint32_t)row & 7u)) << 4);
          const uint32_t a_hi = (D == 128)
              ? q_row + (BM * 128) + ((((uint32_t)u) ^ ((uint32_t)row & 7u)) << 4)
              : q_row + ((((uint32_t)(u + kUnits)) ^ ((uint32_t)row & 7u)) << 4);
          uint32_t lo[4], hi[4];
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(lo[0]), "=r"(lo[1]), "=r"(lo[2]), "=r"(lo[3]) : "r"(a_lo));
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(hi[0]), "=r"(hi[1]), "=r"(hi[2]), "=r"(hi[3]) : "r"(a_hi));
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float4 c = cs[uu][i];                // (cos, sin) of two consecutive j
            const __nv_bfloat162 l2 = *reinterpret_cast<__nv_bfloat162*>(&lo[i]);
            const __nv_bfloat162 h2 = *reinterpret_cast<__nv_bfloat162*>(&hi[i]);
            const float2 a = __bfloat1622float2(l2), b = __bfloat1622float2(h2);
            lo[i] = pack_bf16(__fmaf_rn(a.x, c.x, -__fmul_rn(b.x, c.y)), __fmaf_rn(a.y, c.z, -__fmul_rn(b.y, c.w)));
            hi[i] = pack_bf16(__fmaf_rn(b.x, c.x, __fmul_rn(a.x, c.y)), __fmaf_rn(b.y, c.z, __fmul_rn(a.y, c.w)));
          }
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_lo), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]) : "memory");
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_hi), "r"(hi[0]), "r"(hi[1]), "r"(hi[2]), "r"(hi[3]) : "memory");
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // visible to the tensor core
      }
      mbar_arrive(bar_q_rot + 8 * t);
      return true;
    };
    while (true) {
      // in independent mode slot t has its own ring, and an item describes one tile (its slot-0 fields)
      const uint32_t ring = it_n % kRing;
      const int f = t;                                 // which slot fields of the entry to read
      ok = __all_sync(0xffffffffu, mbar_wait(bar_item_full + 8 * ring, (it_n / kRing) & 1u, wctx, kWaitItemFull));
      if (!ok) break;
      const volatile int* e = s_ring + ring * kRingInts;
      const int w = e[0];
      const int item_bin = e[1], item_kv_row0 = e[2];
      const int jb_t = f ? e[6] : 0, je_t = f ? e[8] : e[7];
      const int q_row0_t = e[4 + f], head_t = e[9 + f];
      const int bin_used = e[12], seg_end = e[13], key_lo_t = e[14 + f], seg_first_t = e[16 + f];
      const int single_seg = e[18] >> f;
      mbar_arrive(bar_item_empty + 8 * ring);
      if (w < 0) break;
      const bool used = jb_t < je_t;
      const int i_row = q_row0_t + row;                // bin-local query row
      int key_lo = 1, key_hi = 0;                      // visible keys [key_lo, key_hi]; empty for padding
      if (used) {                                      // warp-uniform
        int lo = key_lo_t;
        if (!(single_seg & 1))                         // several prompts in this tile: find this row's
          lo = seg_start_at(tb + args.off_seg_start, seg_first_t + 1, seg_end, i_row, i_row - lane + 31, lo, lane);
        if (i_row < bin_used) { key_lo = lo; key_hi = i_row; }
      }
      // Fused path: Q arrives raw and is rotated in shared memory.
      if (args.rope_table) {
        ok = rotate_q(used ? key_hi - key_lo : -1, it_n & 1u);
        if (!ok) break;
      }
      float m_run = -INFINITY;      // running maximum of the whole row, in scaled log2 units
      float l_run = 0.f;            // this thread's share of the running sum of exp2(s * c - m_run)

      for (int j = jb_t; j < je_t; ++j) {
        constexpr int EPT = BN / 2;                          // scores per thread and tile
        constexpr int NCH = EPT / 32;                        // 32-column TMEM round trips
        const int kv0 = item_kv_row0 + j * BN + EPT * h;     // first key of this thread's half
        const int c_lo = max(key_lo - kv0, 0);
        const int c_hi = min(key_hi - kv0, EPT - 1);         // visible columns [c_lo, c_hi] of the half
        // one warp reduction for all the per-warp flags of the tile: which 32-column chunks somebody
        // can see, and whether any row's interval ends or begins inside this half of the tile
        static_assert(NCH == 2, "flag bits below are laid out for two chunks");
        const uint64_t vis = visible_mask64(c_lo, c_hi);     // bit i: column i is visible to this row
        const uint32_t vis_lo = (uint32_t)vis, vis_hi = (uint32_t)(vis >> 32);
        const uint32_t lane_flags = (uint32_t)(vis_lo != 0u) | ((uint32_t)(vis_hi != 0u) << 1) |
                            ((uint32_t)(~vis != 0ull) << 2);
        const uint32_t warp_flags = __reduce_or_sync(0xffffffffu, lane_flags);
        const bool need[NCH] = {(warp_flags & 1u) != 0, (warp_flags & 2u) != 0};
        const bool cut = (warp_flags & 4u) != 0;
        const uint32_t sbuf = 0u;
        const uint32_t tparity = tcount & 1u;
        const uint32_t tmem_sb = tmem_s;
        ok = __all_sync(0xffffffffu, mbar_wait(bar_s_full + 8 * (2 * t + sbuf), tparity, wctx, kWaitS));
        if (!ok) break;                                      // warp-uniform
        tc_fence_after();

        // this thread's scores
        uint32_t v[EPT];
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
          if (need[ch]) {
            tmem_ld32(tmem_sb + EPT * h + 32 * ch, *reinterpret_cast<uint32_t(*)[32]>(&v[32 * ch]));
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[32 * ch + i] = 0xff800000u;        // -inf
          }
        }
        tc_wait_ld();
        // masked tiles (the causal diagonal, the first tile of a prompt): one select per score,
        // steered by the bits of the row's visibility mask
        if (cut) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = (vis_lo & (1u << i)) ? v[i] : 0xff800000u;
#pragma unroll
          for (int i = 0; i < 32; ++i) v[32 + i] = (vis_hi & (1u << i)) ? v[32 + i] : 0xff800000u;
        }
        float mx;
        {
          float m0 = fmax3(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]));
          float m1 = fmax3(__uint_as_float(v[3]), __uint_as_float(v[4]), __uint_as_float(v[5]));
          float m2 = fmax3(__uint_as_float(v[6]), __uint_as_float(v[7]), __uint_as_float(v[8]));
          float m3 = fmax3(__uint_as_float(v[9]), __uint_as_float(v[10]), __uint_as_float(v[11]));
#pragma unroll
          for (int i = 12; i + 7 < EPT; i += 8) {
            m0 = fmax3(m0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
            m1 = fmax3(m1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
            m2 = fmax3(m2, __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
            m3 = fmax3(m3, __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
          }
          // 12 + 8 * n = EPT - 4; the last four
          m0 = fmax3(m0, __uint_as_float(v[EPT - 4]), __uint_as_float(v[EPT - 3]));
          m1 = fmax3(m1, __uint_as_float(v[EPT - 2]), __uint_as_float(v[EPT - 1]));
          mx = fmaxf(fmax3(m0, m1, m2), m3);
        }
        // Row maximum over both halves. The barrier also orders the two halves' S reads before
        // either writes P over the S columns.
        *x_mine = mx;
        if (!(ok = rendezvous(bar_pair, pair_ph, kWaitPair))) break;
        mx = fmaxf(mx, *x_other);
        // lazy running-maximum update: keep the stale maximum while the new one is < 2^8 above it
        const float m_tile = mx * c_scale;
        float m_new = m_run;
        if (m_tile > m_run + 8.f) m_new = m_tile;
        const bool rescale = (m_new != m_run) && (m_run != -INFINITY);
        const float alpha = rescale ? fast_exp2(m_run - m_new) : 1.f;
        if (j > jb_t && __any_sync(0xffffffffu, rescale)) {
          // (S_t ready implies that the previous P_t V product has finished.) Each half rescales its
          // own D/2 columns of the row.
#pragma unroll 1
          for (int ch = 0; ch < D / 32; ++ch) {          // rare path: keep it small
            uint32_t ov[16];
            tmem_ld16(tmem_o + (D / 2) * h + ch * 16, ov);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
            tmem_st16(tmem_o + (D / 2) * h + ch * 16, ov);
          }
        }
        l_run *= alpha;
        m_run = m_new;
        const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;

        // p = exp2(s * c - m), row sum, P (bf16) written over the S columns
        const uint64_t c2 = pack_f2(__float_as_uint(c_scale), __float_as_uint(c_scale));
        const uint64_t negm2 = pack_f2(__float_as_uint(neg_m), __float_as_uint(neg_m));
        uint64_t sum_a = 0ull, sum_b = 0ull;                 // two packed accumulators
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
          uint32_t pk[16];
          if (need[ch]) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              float p0, p1, p2, p3;
              unpack_f2(fma_f2(pack_f2(v[ch * 32 + i], v[ch * 32 + i + 1]), c2, negm2), p0, p1);
              unpack_f2(fma_f2(pack_f2(v[ch * 32 + i + 2], v[ch * 32 + i + 3]), c2, negm2), p2, p3);
              p0 = fast_exp2(p0); p1 = fast_exp2(p1); p2 = fast_exp2(p2); p3 = fast_exp2(p3);
              sum_a = add_f2(sum_a, pack_f2(__float_as_uint(p0), __float_as_uint(p1)));
              sum_b = add_f2(sum_b, pack_f2(__float_as_uint(p2), __float_as_uint(p3)));
              pk[i >> 1] = pack_bf16(p0, p1);
              pk[(i >> 1) + 1] = pack_bf16(p2, p3);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = 0u;
          }
          tmem_st16(tmem_sb + (EPT / 2) * h + ch * 16, pk);
        }
        float sum0, sum1, sum2, sum3;
        unpack_f2(sum_a, sum0, sum1);
        unpack_f2(sum_b, sum2, sum3);
        l_run += (sum0 + sum2) + (sum1 + sum3);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p_full + 8 * (2 * t + sbuf));
        ++tcount;
      }
      if (!ok) break;

      // epilogue: O_t / l -> bf16 -> shared memory (128-byte swizzle) -> TMA store
      ok = __all_sync(0xffffffffu, mbar_wait(bar_o_full + 8 * t, it_n & 1u, wctx, kWaitOFull));
      if (!ok) break;
      if (used) {
        // the half-1 threads hand their share of the row sum to the half-0 threads, which run the
        // epilogue; the second barrier keeps the exchange slot from being reused too early
        if (h == 1) *x_mine = l_run;
        if (!(ok = rendezvous(bar_pair, pair_ph, kWaitPair))) break;
        const float l_row = (h == 0) ? l_run + *x_other : 0.f;
        if (!(ok = rendezvous(bar_pair, pair_ph, kWaitPair))) break;
        if (h == 1) mbar_arrive(bar_o_empty + 8 * t);      // this thread is past o_full and never reads O_t
        if (h == 0) {
          tc_fence_after();
          const float inv_l = l_row > 0.f ? 1.f / l_row : 0.f;
          // each warp stages and stores its own 32 rows (a 32-row TMA box): no rendezvous between
          // warps; lane 0 issues the warp's stores and waits for the previous one to have read the rows
          const uint32_t stage = s_stage_o + (uint32_t)t * Cfg::kStageOBytes + (uint32_t)quad * (32 * 128);
          const uint32_t stage_row = stage + (uint32_t)lane * 128;
          const int row0_w = q_row0_t + 32 * quad;
#pragma unroll 1
          for (int hh = 0; hh < D / 64; ++hh) {          // 64 columns (one TMA box) at a time
            if (lane == 0) tma_store_wait_read();
            __syncwarp();
            uint32_t ov[64];
            tmem_ld32(tmem_o + hh * 64, *reinterpret_cast<uint32_t(*)[32]>(&ov[0]));
            tmem_ld32(tmem_o + hh * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&ov[32]));
            tc_wait_ld();
            if (hh == D / 64 - 1) {
              tc_fence_before();
              mbar_arrive(bar_o_empty + 8 * t);        // O_t may be overwritten by the next item now
            }
#pragma unroll
            for (int c16 = 0; c16 < 8; ++c16) {
              const uint32_t addr = stage_row + (((uint32_t)c16 ^ ((uint32_t)lane & 7u)) << 4);
              const uint32_t w0 = pack_bf16(__uint_as_float(ov[c16 * 8 + 0]) * inv_l, __uint_as_float(ov[c16 * 8 + 1]) * inv_l);
              const uint32_t w1 = pack_bf16(__uint_as_float(ov[c16 * 8 + 2]) * inv_l, __uint_as_float(ov[c16 * 8 + 3]) * inv_l);
              const uint32_t w2 = pack_bf16(__uint_as_float(ov[c16 * 8 + 4]) * inv_l, __uint_as_float(ov[c16 * 8 + 5]) * inv_l);
              const uint32_t w3 = pack_bf16(__uint_as_float(ov[c16 * 8 + 6]) * inv_l, __uint_as_float(ov[c16 * 8 + 7]) * inv_l);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0 && row0_w < args.capacity) {
              tma_store_4d(&map_o, stage, hh * 64, head_t, row0_w, item_bin);
              asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
          }
        }
      } else {
        mbar_arrive(bar_o_empty + 8 * t);
      }
      if (!ok) break;
      ++it_n;
    }
    if (h == 0 && lane == 0) tma_store_wait_read();    // staging must outlive the last store's read
    }   // shared-stream mode
  }

  tc_fence_before();
  __syncthreads();
  if (*s_abort) {
    // A wait gave up: TMA loads and MMAs of this CTA may still be in flight. Give them time to land
    // (they take microseconds) before shared memory and TMEM are handed back.
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 100000ull) {}
    __syncthreads();
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// Self-test of the bounded-wait mechanism: one thread waits on an mbarrier that nothing ever
// arrives on. The wait must give up after `limit_ns`, write its code to the status word and let
// the kernel return normally.
__global__ void bounded_wait_selftest_kernel(int32_t* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const WaitCtx wctx{&abort_flag, status, limit_ns};
  if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, wctx, 77);
  __syncthreads();
}

// ------------------------------------------------------------------------------------------
// Host side: tensor maps and launch
// ------------------------------------------------------------------------------------------
using EncodeFn = PFN_cuTensorMapEncodeTiled_v12000;

EncodeFn get_encode_fn() {
  static EncodeFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeFn>(p);
  }();
  return fn;
}

// 4-D map over a dense [R, M, H, D] bf16 tensor; box = 64 elements x `heads` heads x `rows` rows x 1 bin
// (in shared memory: row-major over (row, head), 128 bytes each).
int make_map(CUtensorMap* map, const void* ptr, int64_t R, int64_t M, int64_t H, int64_t D, int rows, int heads = 1) {
  EncodeFn enc = get_encode_fn();
  if (!enc) return note_cuda_error(-1, "cuTensorMapEncodeTiled entry point not found");
  cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)M, (cuuint64_t)R};
  cuuint64_t strides[3] = {(cuuint64_t)(D * 2), (cuuint64_t)(H * D * 2), (cuuint64_t)(M * H * D * 2)};
  cuuint32_t box[4] = {64u, (cuuint32_t)heads, (cuuint32_t)rows, 1u};
  cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides,
                         box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? PP_OK : note_cuda_error((int)r, "cuTensorMapEncodeTiled");
}

unsigned long long wait_limit_ns() {
  // Debug overrides of the device-side wait limit, in milliseconds or microseconds.
  if (const char* e = std::getenv("PP_WAIT_LIMIT_MS")) {
    const long ms = std::atol(e);
    if (ms > 0) return (unsigned long long)ms * 1000000ull;
  }
  if (const char* e = std::getenv("PP_WAIT_LIMIT_US")) {
    const long us = std::atol(e);
    if (us > 0) return (unsigned long long)us * 1000ull;
  }
  return 2000000000ull;   // 2 s
}

int sm_count() {
  static thread_local int cached_dev = -1, cached = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (dev != cached_dev) {
    if (cudaDeviceGetAttribute(&cached, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    cached_dev = dev;
  }
  return cached;
}

template <int D, bool kIndep>
int launch_attention_t(const pp_attn_params& p, int32_t* d_table, const TableLayout& L, const void* q,
                       const void* k, const void* v, void* o, const void* rope_table, int32_t* device_status,
                       cudaStream_t stream) {
  constexpr int BN = kIndep ? kTileNShort : kTileN;
  using Cfg = AttnCfg<D, BN>;
  CUtensorMap mq, mk, mv, mo;
  int st;
  const int fold = kIndep ? L.fold : 1;
  int fold_shift = 0;
  while ((1 << fold_shift) < fold) ++fold_shift;
  if ((st = make_map(&mq, q, p.n_bins, p.capacity, p.n_q_heads, D, BM / fold, fold)) != PP_OK) return st;
  if ((st = make_map(&mk, k, p.n_bins, p.capacity, p.n_kv_heads, D, BN)) != PP_OK) return st;
  if ((st = make_map(&mv, v, p.n_bins, p.capacity, p.n_kv_heads, D, BN)) != PP_OK) return st;
  if ((st = make_map(&mo, o, p.n_bins, p.capacity, p.n_q_heads, D, 32 / fold, fold)) != PP_OK) return st;   // one warp's rows per store
  // the shared-memory opt-in of a kernel is a per-device attribute
  static DeviceOnce configured;     // per template instance
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return note_cuda_error(-1, "cudaGetDevice");
  if (!configured.done(dev)) {
    cudaError_t e = cudaFuncSetAttribute(attention_kernel<D, kIndep>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         Cfg::kSmemBytes);
    if (e != cudaSuccess) return note_cuda_error((int)e, "cudaFuncSetAttribute(smem)");
    configured.mark(dev);
  }
  const int sms = sm_count();
  if (sms <= 0) return note_cuda_error(-1, "multiprocessor count");
  AttnArgs a;
  a.table = d_table;
  a.counter = d_table + kHeaderCounter;
  a.off_bin_seg_ptr = L.bin_seg_ptr;
  a.off_bin_used = L.bin_used;
  a.off_seg_start = L.seg_start;
  a.off_items = L.items;
  a.n_items = L.n_items;
  a.group = p.n_q_heads / p.n_kv_heads;
  a.pair_heads = (!kIndep && a.group % 2 == 0) ? 1 : 0;
  a.fold = fold;
  a.fold_shift = fold_shift;
  a.subs = a.pair_heads ? a.group / 2 : a.group / fold;
  a.n_q_heads = p.n_q_heads;
  a.capacity = p.capacity;
  const int64_t total = (int64_t)p.n_kv_heads * L.n_items * a.subs;
  if (total > INT32_MAX) return PP_ERR_UNSUPPORTED;
  a.total_work = (int32_t)total;
  const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / sqrtf((float)D);
  a.scale_log2 = scale * 1.4426950408889634f;
  a.o = static_cast<__nv_bfloat16*>(o);
  a.rope_table = static_cast<const float2*>(rope_table);
  a.status = device_status;
  a.wait_limit_ns = wait_limit_ns();
  const unsigned grid = (unsigned)(total < sms ? total : sms);
  const cudaError_t launch_err = launch_dependent(attention_kernel<D, kIndep>, dim3(grid), dim3(kAttnThreads),
                                                  (size_t)Cfg::kSmemBytes, stream, mq, mk, mv, mo, a);
  const cudaError_t e = launch_err != cudaSuccess ? launch_err : cudaGetLastError();
  return e == cudaSuccess ? PP_OK : note_cuda_error((int)e, "attention kernel launch");
}

}  // namespace

int launch_bounded_wait_selftest(int32_t* device_status, uint64_t limit_ns, void* stream) {
  bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(device_status, limit_ns);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? PP_OK : note_cuda_error((int)e, "self-test kernel launch");
}

int launch_attention(const pp_attn_params& p, int32_t* d_table, const TableLayout& L, const void* q,
                     const void* k, const void* v, void* o, const void* rope_table, int32_t* device_status,
                     void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (L.independent_slots) {
    if (p.head_dim == 128) return launch_attention_t<128, true>(p, d_table, L, q, k, v, o, rope_table, device_status, s);
    return launch_attention_t<64, true>(p, d_table, L, q, k, v, o, rope_table, device_status, s);
  }
  if (p.head_dim == 128) return launch_attention_t<128, false>(p, d_table, L, q, k, v, o, rope_table, device_status, s);
  return launch_attention_t<64, false>(p, d_table, L, q, k, v, o, rope_table, device_status, s);
}

}  // namespace pp
