// Packed-varlen prefill attention for sm_100a (Sections 2.1 and 3.2 of the prepacking paper):
//   o_i = sum_j softmax_j(q'_i . k'_j * scale) v_j   over keys j of the same prompt with j <= i.
// The independent mask M' (a lower-triangular block per prompt span) is never built: every query
// row carries the key range [start row of its prompt, its own row], and the host work list
// restricts each 128-row query tile to the key tiles that can intersect such a range.
//
// One CTA = one (query tile, query head). Warp roles:
//   warp 0      TMA producer (Q once, then the K and V tiles of the key loop), TMEM allocator
//   warp 1      tcgen05.mma issuer: S = Q K^T into TMEM, then O += P V with P read from TMEM
//   warps 2-5   online softmax, one query row per thread (TMEM lane = row): tcgen05.ld S,
//               mask, exp2, tcgen05.st P (bf16, over the S columns), rescale O when the running
//               maximum moved, and the epilogue (O / l -> bf16 -> shared -> TMA store)
// Two CTAs share an SM (256 TMEM columns each), so one CTA's MMAs overlap the other's softmax.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdlib>

#include "pp_internal.h"

namespace pp {
namespace {

constexpr int BM = kTileM;
constexpr int BN = kTileN;
constexpr int kAttnThreads = 192;
constexpr int kSoftmaxThreads = 128;
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kTmemColS = 0;      // S (fp32, BN columns); P (bf16 pairs, BN/2 columns) aliases it
constexpr uint32_t kTmemColO = 128;    // O (fp32, D columns)

template <int D> struct AttnCfg {
  static constexpr int kStages = (D == 128) ? 1 : 2;
  static constexpr int kChunks = D / 64;                     // 128-byte swizzle spans per row
  static constexpr int kQBytes = BM * D * 2;
  static constexpr int kKVBytes = BN * D * 2;
  static constexpr int kBarBytes = 256;
  static constexpr int kSmemBytes = 1024 /*alignment slack*/ + kQBytes + 2 * kStages * kKVBytes + kBarBytes;
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
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const WaitCtx& w, int code) {
  const unsigned long long t0 = global_ns();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 31u) == 0) {
      if (*w.abort_flag) return false;
      if (global_ns() - t0 > w.limit_ns) {
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
__device__ __forceinline__ void tma_store_commit_and_wait() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { __syncwarp(); asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { __syncwarp(); asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
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
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  __syncwarp();
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
        "r"(taddr) : "memory");
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
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);     // .x (low 16 bits) = lo
  return *reinterpret_cast<uint32_t*>(&h);
}

// Shared-memory matrix descriptors (tcgen05), 128-byte swizzle, rows of 128 bytes, 8-row groups
// 1024 bytes apart. `lbo_bytes` is the distance between 64-element spans of the MN dimension
// (only read for MN-major operands).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
         ((uint64_t)(1024u >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 A and B, A K-major, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(uint32_t n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((n >> 3) << 17) |
         ((128u >> 4) << 24);
}

struct AttnArgs {
  const int32_t* table;
  int32_t off_bin_seg_ptr, off_bin_used, off_seg_start, off_items;
  int32_t group;                 // query heads per KV head
  float scale_log2;              // softmax scale * log2(e)
  int32_t* status;
  unsigned long long wait_limit_ns;
};

enum WaitCode { kWaitQ = 1, kWaitKFull, kWaitVFull, kWaitKEmpty, kWaitVEmpty, kWaitS, kWaitP, kWaitO };

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 2)
attention_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o,
                 const AttnArgs args) {
  using Cfg = AttnCfg<D>;
  constexpr int kStages = Cfg::kStages;
  constexpr int kChunks = Cfg::kChunks;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t s_q = smem_base;
  const uint32_t s_k = s_q + Cfg::kQBytes;
  const uint32_t s_v = s_k + kStages * Cfg::kKVBytes;
  const uint32_t s_bar = s_v + kStages * Cfg::kKVBytes;
  uint8_t* bar_generic = smem_raw + (s_bar - smem_u32(smem_raw));
  // barrier slots (8 bytes each)
  const uint32_t bar_q = s_bar + 0;
  const uint32_t bar_s = s_bar + 8;
  const uint32_t bar_p = s_bar + 16;
  const uint32_t bar_o = s_bar + 24;
  const uint32_t bar_kfull = s_bar + 32;                  // [kStages]
  const uint32_t bar_kempty = bar_kfull + 8 * kStages;
  const uint32_t bar_vfull = bar_kempty + 8 * kStages;
  const uint32_t bar_vempty = bar_vfull + 8 * kStages;
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(bar_generic + 128);
  volatile int* s_abort = reinterpret_cast<volatile int*>(bar_generic + 132);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // work item
  const int item_idx = blockIdx.x / args.group;
  const int q_head = blockIdx.y * args.group + (blockIdx.x - item_idx * args.group);
  const int kv_head = blockIdx.y;
  const int4 item = *reinterpret_cast<const int4*>(args.table + args.off_items + 4 * item_idx);
  const int bin = item.x, q_row0 = item.y, kv_row0 = item.z, n_tiles = item.w;

  const WaitCtx wctx{s_abort, args.status, args.wait_limit_ns};

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_p, kSoftmaxThreads);
    mbar_init(bar_o, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_kfull + 8 * s, 1);
      mbar_init(bar_kempty + 8 * s, 1);
      mbar_init(bar_vfull + 8 * s, 1);
      mbar_init(bar_vempty + 8 * s, 1);
    }
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
  const uint32_t tmem_s = tmem_base + kTmemColS;
  const uint32_t tmem_o = tmem_base + kTmemColO;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(bar_q, Cfg::kQBytes);
      for (int c = 0; c < kChunks; ++c)
        tma_load_4d(s_q + c * (BM * 128), &map_q, bar_q, c * 64, q_head, q_row0, bin);
      for (int j = 0; j < n_tiles; ++j) {
        const int s = j % kStages;
        const uint32_t use = (uint32_t)(j / kStages);
        const int kv0 = kv_row0 + j * BN;
        if (!mbar_wait(bar_kempty + 8 * s, (use & 1u) ^ 1u, wctx, kWaitKEmpty)) break;
        mbar_expect_tx(bar_kfull + 8 * s, Cfg::kKVBytes);
        for (int c = 0; c < kChunks; ++c)
          tma_load_4d(s_k + s * Cfg::kKVBytes + c * (BN * 128), &map_k, bar_kfull + 8 * s,
                      c * 64, kv_head, kv0, bin);
        if (!mbar_wait(bar_vempty + 8 * s, (use & 1u) ^ 1u, wctx, kWaitVEmpty)) break;
        mbar_expect_tx(bar_vfull + 8 * s, Cfg::kKVBytes);
        for (int c = 0; c < kChunks; ++c)
          tma_load_4d(s_v + s * Cfg::kKVBytes + c * (BN * 128), &map_v, bar_vfull + 8 * s,
                      c * 64, kv_head, kv0, bin);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(BN, false);
      constexpr uint32_t idesc_pv = instr_desc(D, true);
      bool ok = mbar_wait(bar_q, 0, wctx, kWaitQ);
      for (int j = 0; ok && j < n_tiles; ++j) {
        const int s = j % kStages;
        const uint32_t use = (uint32_t)(j / kStages);
        // S = Q K^T
        if (!mbar_wait(bar_kfull + 8 * s, use & 1u, wctx, kWaitKFull)) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t koff = (uint32_t)(kk >> 2) * (BM * 128) + (uint32_t)(kk & 3) * 32;
          mma_ss(tmem_s, smem_desc(s_q + koff, 0), smem_desc(s_k + s * Cfg::kKVBytes + koff, 0),
                 idesc_qk, kk > 0);
        }
        tc_commit(bar_kempty + 8 * s);       // K tile consumed
        tc_commit(bar_s);                    // S ready (also: every earlier MMA has finished)
        // O += P V
        if (!mbar_wait(bar_p, (uint32_t)j & 1u, wctx, kWaitP)) break;
        if (!mbar_wait(bar_vfull + 8 * s, use & 1u, wctx, kWaitVFull)) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < BN / 16; ++kk) {
          mma_ts(tmem_o, tmem_s + kk * 8,
                 smem_desc(s_v + s * Cfg::kKVBytes + kk * (16 * 128), BN * 128), idesc_pv,
                 (j > 0 || kk > 0) ? 1u : 0u);
        }
        tc_commit(bar_vempty + 8 * s);       // V tile consumed
        if (j == n_tiles - 1) tc_commit(bar_o);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue
    const int quad = warp & 3;                       // TMEM lane quadrant this warp may access
    const int row = quad * 32 + lane;                // query row inside the tile
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const int i_row = q_row0 + row;                  // bin-local query row
    int key_lo = 1, key_hi = 0;                      // visible keys [key_lo, key_hi]; empty for padding
    {
      const int32_t* tb = args.table;
      if (i_row < tb[args.off_bin_used + bin]) {
        int lo = tb[args.off_bin_seg_ptr + bin], hi = tb[args.off_bin_seg_ptr + bin + 1] - 1;
        while (lo < hi) {
          const int mid = (lo + hi + 1) >> 1;
          if (tb[args.off_seg_start + mid] <= i_row) lo = mid; else hi = mid - 1;
        }
        key_lo = tb[args.off_seg_start + lo];
        key_hi = i_row;
      }
    }
    const float c_scale = args.scale_log2;
    float m_run = -INFINITY;      // running maximum, in scaled log2 units
    float l_run = 0.f;            // running sum of exp2(s * c - m_run)
    bool ok = true;
    uint32_t v[32];

    for (int j = 0; j < n_tiles; ++j) {
      const int kv0 = kv_row0 + j * BN;
      const int c_lo = max(key_lo - kv0, 0);
      const int c_hi = min(key_hi - kv0, BN - 1);          // visible columns [c_lo, c_hi]
      const bool full = (c_lo == 0) && (c_hi == BN - 1);
      ok = __all_sync(0xffffffffu, mbar_wait(bar_s, (uint32_t)j & 1u, wctx, kWaitS));
      if (!ok) break;                                       // warp-uniform
      tc_fence_after();

      // which 32-column chunks does any row of this warp need?
      uint32_t need_mask = 0;
#pragma unroll
      for (int ch = 0; ch < BN / 32; ++ch) {
        const bool need = max(c_lo, ch * 32) <= min(c_hi, ch * 32 + 31);
        if (__any_sync(0xffffffffu, need)) need_mask |= 1u << ch;
      }

      // pass 1: row maximum over the visible columns
      float mx = -INFINITY;
#pragma unroll
      for (int ch = 0; ch < BN / 32; ++ch) {
        if (!(need_mask & (1u << ch))) continue;
        tmem_ld32(tmem_s + lane_base + ch * 32, v);
        tc_wait_ld();
        if (full) {
#pragma unroll
          for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(v[i]));
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int col = ch * 32 + i;
            if (col >= c_lo && col <= c_hi) mx = fmaxf(mx, __uint_as_float(v[i]));
          }
        }
      }
      // lazy running-maximum update: keep the stale maximum while the new one is < 2^8 above it
      const float m_tile = mx * c_scale;
      float m_new = m_run;
      if (m_tile > m_run + 8.f) m_new = m_tile;
      const bool rescale = (m_new != m_run) && (m_run != -INFINITY);
      const float alpha = rescale ? fast_exp2(m_run - m_new) : 1.f;
      if (j > 0 && __any_sync(0xffffffffu, rescale)) {
#pragma unroll
        for (int ch = 0; ch < D / 32; ++ch) {
          tmem_ld32(tmem_o + lane_base + ch * 32, v);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
          tmem_st32(tmem_o + lane_base + ch * 32, v);
        }
      }
      l_run *= alpha;
      m_run = m_new;

      // pass 2: p = exp2(s * c - m), row sum, P (bf16) over the S columns
      float sum = 0.f;
#pragma unroll
      for (int ch = 0; ch < BN / 32; ++ch) {
        uint32_t pk[16];
        if (need_mask & (1u << ch)) {
          tmem_ld32(tmem_s + lane_base + ch * 32, v);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const int col = ch * 32 + i;
            float p0 = fast_exp2(fmaf(__uint_as_float(v[i]), c_scale, -m_run));
            float p1 = fast_exp2(fmaf(__uint_as_float(v[i + 1]), c_scale, -m_run));
            if (!full) {
              if (!(col >= c_lo && col <= c_hi)) p0 = 0.f;
              if (!(col + 1 >= c_lo && col + 1 <= c_hi)) p1 = 0.f;
            }
            sum += p0 + p1;
            pk[i >> 1] = pack_bf16(p0, p1);
          }
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) pk[i] = 0u;
        }
        tmem_st16(tmem_s + lane_base + ch * 16, pk);
      }
      l_run += sum;
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar_p);
    }

    // epilogue: O / l -> bf16 -> shared (128-byte swizzle, the Q buffer is free by now) -> TMA
    ok = __all_sync(0xffffffffu, ok && mbar_wait(bar_o, 0, wctx, kWaitO));
    if (ok) {
      tc_fence_after();
      const float inv_l = l_run > 0.f ? 1.f / l_run : 0.f;
#pragma unroll
      for (int ch = 0; ch < D / 32; ++ch) {
        tmem_ld32(tmem_o + lane_base + ch * 32, v);
        tc_wait_ld();
        const uint32_t box = s_q + (uint32_t)(ch >> 1) * (BM * 128) + (uint32_t)row * 128;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          const uint32_t c16 = (uint32_t)((ch & 1) * 4 + q4);
          const uint32_t addr = box + ((c16 ^ ((uint32_t)row & 7u)) << 4);
          const uint32_t w0 = pack_bf16(__uint_as_float(v[q4 * 8 + 0]) * inv_l, __uint_as_float(v[q4 * 8 + 1]) * inv_l);
          const uint32_t w1 = pack_bf16(__uint_as_float(v[q4 * 8 + 2]) * inv_l, __uint_as_float(v[q4 * 8 + 3]) * inv_l);
          const uint32_t w2 = pack_bf16(__uint_as_float(v[q4 * 8 + 4]) * inv_l, __uint_as_float(v[q4 * 8 + 5]) * inv_l);
          const uint32_t w3 = pack_bf16(__uint_as_float(v[q4 * 8 + 6]) * inv_l, __uint_as_float(v[q4 * 8 + 7]) * inv_l);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // all four softmax warps meet here whether or not a wait gave up
    asm volatile("bar.sync 1, %0;" ::"n"(kSoftmaxThreads) : "memory");
    if (ok && !*s_abort && warp == 2 && lane == 0) {
      for (int c = 0; c < kChunks; ++c)
        tma_store_4d(&map_o, s_q + c * (BM * 128), c * 64, q_head, q_row0, bin);
      tma_store_commit_and_wait();
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
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

// 4-D map over a dense [R, M, H, D] bf16 tensor; box = 64 elements x 1 head x `rows` rows x 1 bin.
int make_map(CUtensorMap* map, const void* ptr, int64_t R, int64_t M, int64_t H, int64_t D, int rows) {
  EncodeFn enc = get_encode_fn();
  if (!enc) return note_cuda_error(-1, "cuTensorMapEncodeTiled entry point not found");
  cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)M, (cuuint64_t)R};
  cuuint64_t strides[3] = {(cuuint64_t)(D * 2), (cuuint64_t)(H * D * 2), (cuuint64_t)(M * H * D * 2)};
  cuuint32_t box[4] = {64u, 1u, (cuuint32_t)rows, 1u};
  cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides,
                         box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? PP_OK : note_cuda_error((int)r, "cuTensorMapEncodeTiled");
}

unsigned long long wait_limit_ns() {
  // Debug override of the device-side wait limit, in milliseconds.
  if (const char* e = std::getenv("PP_WAIT_LIMIT_MS")) {
    const long ms = std::atol(e);
    if (ms > 0) return (unsigned long long)ms * 1000000ull;
  }
  return 2000000000ull;   // 2 s
}

template <int D>
int launch_attention_t(const pp_attn_params& p, const int32_t* d_table, const TableLayout& L,
                       const void* q, const void* k, const void* v, void* o, int32_t* device_status,
                       cudaStream_t stream) {
  using Cfg = AttnCfg<D>;
  CUtensorMap mq, mk, mv, mo;
  int st;
  if ((st = make_map(&mq, q, p.n_bins, p.capacity, p.n_q_heads, D, BM)) != PP_OK) return st;
  if ((st = make_map(&mk, k, p.n_bins, p.capacity, p.n_kv_heads, D, BN)) != PP_OK) return st;
  if ((st = make_map(&mv, v, p.n_bins, p.capacity, p.n_kv_heads, D, BN)) != PP_OK) return st;
  if ((st = make_map(&mo, o, p.n_bins, p.capacity, p.n_q_heads, D, BM)) != PP_OK) return st;
  static bool configured = false;   // per process, per template instance
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(attention_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         Cfg::kSmemBytes);
    if (e != cudaSuccess) return note_cuda_error((int)e, "cudaFuncSetAttribute(smem)");
    cudaFuncSetAttribute(attention_kernel<D>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    configured = true;
  }
  AttnArgs a;
  a.table = d_table;
  a.off_bin_seg_ptr = L.bin_seg_ptr;
  a.off_bin_used = L.bin_used;
  a.off_seg_start = L.seg_start;
  a.off_items = L.items;
  a.group = p.n_q_heads / p.n_kv_heads;
  const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / sqrtf((float)D);
  a.scale_log2 = scale * 1.4426950408889634f;
  a.status = device_status;
  a.wait_limit_ns = wait_limit_ns();
  dim3 grid((unsigned)(L.n_items * a.group), (unsigned)p.n_kv_heads, 1);
  attention_kernel<D><<<grid, kAttnThreads, Cfg::kSmemBytes, stream>>>(mq, mk, mv, mo, a);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? PP_OK : note_cuda_error((int)e, "attention kernel launch");
}

}  // namespace

int launch_attention(const pp_attn_params& p, const int32_t* d_table, const TableLayout& L,
                     const void* q, const void* k, const void* v, void* o, int32_t* device_status,
                     void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (p.head_dim == 128) return launch_attention_t<128>(p, d_table, L, q, k, v, o, device_status, s);
  return launch_attention_t<64>(p, d_table, L, q, k, v, o, device_status, s);
}

}  // namespace pp
