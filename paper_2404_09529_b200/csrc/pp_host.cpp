// Host side of the prepack-b200 library: BINPACK (first-fit-decreasing), RESTART-PE ids,
// status strings, and the tile work list that the attention kernel walks.
// Algorithm 1 (bin size to RESTART-PE) and Sections 3.1-3.2 of the prepacking paper.
#include "pp_internal.h"

#include <algorithm>
#include <cstring>
#include <new>
#include <numeric>
#include <vector>

extern "C" int pp_version(void) { return 100; }

extern "C" const char* pp_strerror(int status) {
  switch (status) {
    case PP_OK: return "ok";
    case PP_ERR_INVALID_ARG: return "invalid argument";
    case PP_ERR_LENGTH: return "prompt length < 1 or > bin capacity";
    case PP_ERR_BUFFER_TOO_SMALL: return "workspace or arena too small";
    case PP_ERR_UNSUPPORTED: return "unsupported shape or device (needs head_dim 64/128, Hq % Hkv == 0, sm_100)";
    case PP_ERR_ALIGNMENT: return "device pointer or offset not 16-byte aligned";
    case PP_ERR_CUDA: return "CUDA call failed";
    case PP_ERR_DEVICE_TIMEOUT: return "bounded device-side wait gave up";
    case PP_ERR_NO_MEMORY: return "host allocation failed";
    case PP_ERR_TOO_LARGE: return "more prompts than the built-in scratch of the static entry point holds";
    default: return "unknown status";
  }
}

namespace {

// Tournament tree over bin slots holding each bin's free rows; answers "lowest-numbered bin
// with at least `need` free rows" in O(log k). Unopened slots hold 0 free rows.
class FirstFitTree {
 public:
  explicit FirstFitTree(int n) {
    size_ = 1;
    while (size_ < n) size_ <<= 1;
    free_.assign(2 * size_, 0);
  }
  // Lowest slot index with free >= need, or -1.
  int find(int need) const {
    if (free_[1] < need) return -1;
    int node = 1;
    while (node < size_) node = (free_[2 * node] >= need) ? 2 * node : 2 * node + 1;
    return node - size_;
  }
  void set(int slot, int value) {
    int node = slot + size_;
    free_[node] = value;
    for (node >>= 1; node >= 1; node >>= 1) free_[node] = std::max(free_[2 * node], free_[2 * node + 1]);
  }
  int get(int slot) const { return free_[slot + size_]; }

 private:
  int size_;
  std::vector<int> free_;
};

}  // namespace

extern "C" int pp_pack(const int32_t* lengths, int32_t k, int32_t capacity, int32_t* n_bins,
                       int32_t* capacity_out, int32_t* bin_seg_ptr, int32_t* seg_prompt,
                       int32_t* seg_start, int32_t* seg_len, int32_t* bin_of, int32_t* off_of) {
  if (lengths == nullptr || n_bins == nullptr || k < 1 || capacity < 0) return PP_ERR_INVALID_ARG;
  int32_t longest = 0;
  for (int32_t i = 0; i < k; ++i) {
    if (lengths[i] < 1) return PP_ERR_LENGTH;
    longest = std::max(longest, lengths[i]);
  }
  const int32_t cap = capacity == 0 ? longest : capacity;
  if (longest > cap) return PP_ERR_LENGTH;
  try {
    // items by length descending, equal lengths by original index ascending: a counting sort over
    // the lengths (they are at most `cap`), falling back to a comparison sort for few long prompts
    std::vector<int32_t> order(k);
    if ((int64_t)longest <= 8 * (int64_t)k + 1024) {
      std::vector<int32_t> first(longest + 2, 0);             // first[l] = items longer than l, so far: counts
      for (int32_t i = 0; i < k; ++i) ++first[lengths[i]];
      int32_t run = 0;
      for (int32_t l = longest; l >= 1; --l) { const int32_t c = first[l]; first[l] = run; run += c; }
      for (int32_t i = 0; i < k; ++i) order[first[lengths[i]]++] = i;
    } else {
      std::iota(order.begin(), order.end(), 0);
      std::stable_sort(order.begin(), order.end(),
                       [&](int32_t a, int32_t b) { return lengths[a] > lengths[b]; });
    }
    FirstFitTree tree(k);
    std::vector<int32_t> item_bin(k), item_off(k), bin_count;
    int32_t r = 0;
    for (int32_t idx = 0; idx < k; ++idx) {
      const int32_t i = order[idx];
      int b = tree.find(lengths[i]);
      if (b < 0) {            // open a new bin
        b = r++;
        tree.set(b, cap);
        bin_count.push_back(0);
      }
      const int32_t free_rows = tree.get(b);
      item_bin[i] = b;
      item_off[i] = cap - free_rows;
      tree.set(b, free_rows - lengths[i]);
      bin_count[b] += 1;
    }
    // CSR over segments, bin-major, placement order inside a bin (= the order items were taken)
    std::vector<int32_t> ptr(r + 1, 0);
    for (int32_t b = 0; b < r; ++b) ptr[b + 1] = ptr[b] + bin_count[b];
    std::vector<int32_t> cursor(ptr.begin(), ptr.end() - 1);
    for (int32_t idx = 0; idx < k; ++idx) {
      const int32_t i = order[idx];
      const int32_t s = cursor[item_bin[i]]++;
      if (seg_prompt) seg_prompt[s] = i;
      if (seg_start) seg_start[s] = item_off[i];
      if (seg_len) seg_len[s] = lengths[i];
    }
    if (bin_seg_ptr) std::copy(ptr.begin(), ptr.end(), bin_seg_ptr);
    if (bin_of) std::copy(item_bin.begin(), item_bin.end(), bin_of);
    if (off_of) std::copy(item_off.begin(), item_off.end(), off_of);
    *n_bins = r;
    if (capacity_out) *capacity_out = cap;
  } catch (const std::bad_alloc&) {
    return PP_ERR_NO_MEMORY;
  }
  return PP_OK;
}

namespace pp {

int validate_packing(int32_t n_bins, int32_t capacity, const int32_t* bin_seg_ptr,
                     const int32_t* seg_start, const int32_t* seg_len, int32_t k) {
  if (!bin_seg_ptr || !seg_start || !seg_len || n_bins < 1 || capacity < 1 || k < 1)
    return PP_ERR_INVALID_ARG;
  if (bin_seg_ptr[0] != 0 || bin_seg_ptr[n_bins] != k) return PP_ERR_INVALID_ARG;
  for (int32_t b = 0; b < n_bins; ++b) {
    if (bin_seg_ptr[b + 1] <= bin_seg_ptr[b]) return PP_ERR_INVALID_ARG;   // no empty bins
    int64_t off = 0;
    for (int32_t s = bin_seg_ptr[b]; s < bin_seg_ptr[b + 1]; ++s) {
      if (seg_len[s] < 1) return PP_ERR_LENGTH;
      if (seg_start[s] != off) return PP_ERR_INVALID_ARG;                  // contiguous from row 0
      off += seg_len[s];
      if (off > capacity) return PP_ERR_LENGTH;
    }
  }
  return PP_OK;
}

}  // namespace pp

extern "C" int pp_fill_position_ids(int32_t n_bins, int32_t capacity, const int32_t* bin_seg_ptr,
                                    const int32_t* seg_start, const int32_t* seg_len,
                                    int32_t* position_ids, int32_t* segment_ids) {
  if (!bin_seg_ptr || n_bins < 1) return PP_ERR_INVALID_ARG;
  const int32_t k = bin_seg_ptr[n_bins];
  const int st = pp::validate_packing(n_bins, capacity, bin_seg_ptr, seg_start, seg_len, k);
  if (st != PP_OK) return st;
  for (int32_t b = 0; b < n_bins; ++b) {
    int32_t* pos = position_ids ? position_ids + (size_t)b * capacity : nullptr;
    int32_t* sid = segment_ids ? segment_ids + (size_t)b * capacity : nullptr;
    int32_t row = 0;
    for (int32_t s = bin_seg_ptr[b]; s < bin_seg_ptr[b + 1]; ++s)
      for (int32_t p = 0; p < seg_len[s]; ++p, ++row) {
        if (pos) pos[row] = p;
        if (sid) sid[row] = s;
      }
    for (; row < capacity; ++row) {
      if (pos) pos[row] = 0;
      if (sid) sid[row] = -1;
    }
  }
  return PP_OK;
}

// ------------------------------------------------------------------------------------------
// Tile work list (Section 3.2: the independent mask is block lower-triangular per prompt span,
// so a query tile only ever needs the key rows from the start of the first prompt it touches
// up to its own last row).
//
// A work item feeds the two query-tile slots of one persistent CTA, which share one stream of
// key/value tiles. With an even number of query heads per KV head the two slots are two query
// heads over the same 128 rows (identical key ranges); otherwise they are two consecutive
// 128-row tiles of one head, slot 1 joining the key loop at tile jb1 and slot 0 leaving it after
// its diagonal tile je0 - 1.
// ------------------------------------------------------------------------------------------
namespace pp {

int32_t max_fold(int32_t group) {
  for (int32_t f = kMaxFold; f > 1; f >>= 1)
    if (group % f == 0) return f;
  return 1;
}

size_t prefill_table_ints(int32_t n_bins, int32_t capacity, int32_t k, int32_t group) {
  // sized for the shortest query tiles any mode can choose (head folding shortens them)
  const int32_t rq = kTileM / max_fold(group);
  const int64_t q_tiles = (int64_t)n_bins * ((capacity + rq - 1) / rq);
  // header + bin_seg_ptr + bin_used + seg_start + items (kItemInts ints each), each block 4-int aligned
  auto up4 = [](int64_t x) { return (x + 3) & ~int64_t(3); };
  return (size_t)(kHeaderInts + up4(n_bins + 1) + up4(n_bins) + up4(k) + kItemInts * q_tiles);
}

namespace {
// Mean key tiles per 128-row query tile of the packing: the measure of how long work items are.
double mean_key_tiles(int32_t n_bins, const int32_t* bin_seg_ptr, const int32_t* seg_start,
                      const int32_t* seg_len) {
  int64_t q_tiles = 0, kv_tiles = 0;
  for (int32_t b = 0; b < n_bins; ++b) {
    const int32_t s_lo = bin_seg_ptr[b], s_hi = bin_seg_ptr[b + 1];
    const int32_t used = seg_start[s_hi - 1] + seg_len[s_hi - 1];
    int32_t s = s_lo;
    for (int32_t q0 = 0; q0 < used; q0 += kTileM) {
      while (s + 1 < s_hi && seg_start[s + 1] <= q0) ++s;
      const int32_t kv_lo = (seg_start[s] / kTileN) * kTileN;
      kv_tiles += (std::min(q0 + kTileM, used) - kv_lo + kTileN - 1) / kTileN;
      ++q_tiles;
    }
  }
  return q_tiles ? (double)kv_tiles / (double)q_tiles : 0.0;
}
}  // namespace

int build_prefill_tables(int32_t n_bins, int32_t capacity, const int32_t* bin_seg_ptr,
                         const int32_t* seg_start, const int32_t* seg_len, int32_t k, int32_t group,
                         int32_t* out, size_t out_ints, TableLayout* layout) {
  // How the two query-tile slots of a CTA are fed:
  //  - even number of query heads per KV head: two heads over the same rows share a K/V stream;
  //  - otherwise, long items: two consecutive row tiles of one head share a K/V stream (halves the
  //    K/V traffic from L2, which long sequences need);
  //  - otherwise, short items: every slot draws its own single-tile items (a pair of row tiles
  //    of different length would leave one slot idle for a tile per item).
  const bool even_group = (group % 2) == 0;
  const bool independent = mean_key_tiles(n_bins, bin_seg_ptr, seg_start, seg_len) < 8.0;
  const bool pair_rows = !even_group && !independent;
  const int32_t tile_n = independent ? kTileNShort : kTileN;   // key rows per tile of the chosen mode
  //  - short items and several query heads per KV head: the heads are folded into the rows of a
  //    query tile (128 / fold rows x fold heads), so one stream of key tiles serves all of them and a
  //    short prompt fills a tile with heads instead of leaving most of its rows empty
  const int32_t fold = independent ? max_fold(group) : 1;
  const int32_t rq = kTileM / fold;                            // bin rows per query tile
  auto up4 = [](int64_t x) { return (x + 3) & ~int64_t(3); };
  TableLayout L;
  L.bin_seg_ptr = kHeaderInts;
  L.bin_used = L.bin_seg_ptr + (int32_t)up4(n_bins + 1);
  L.seg_start = L.bin_used + (int32_t)up4(n_bins);
  L.items = L.seg_start + (int32_t)up4(k);
  if (out_ints < prefill_table_ints(n_bins, capacity, k, group)) return PP_ERR_BUFFER_TOO_SMALL;
  std::memset(out, 0, sizeof(int32_t) * (size_t)L.items);
  std::memcpy(out + L.bin_seg_ptr, bin_seg_ptr, sizeof(int32_t) * (size_t)(n_bins + 1));
  std::memcpy(out + L.seg_start, seg_start, sizeof(int32_t) * (size_t)k);
  std::vector<WorkItem> items;
  try {
    items.reserve((size_t)n_bins * ((capacity + rq - 1) / rq));
    for (int32_t b = 0; b < n_bins; ++b) {
      const int32_t s_lo = bin_seg_ptr[b], s_hi = bin_seg_ptr[b + 1];
      const int32_t used = seg_start[s_hi - 1] + seg_len[s_hi - 1];
      out[L.bin_used + b] = used;
      int32_t s = s_lo, s_slot0 = s_lo;     // cursors over the bin's segments: query rows only move forward
      // first key row that query tile q0 can see: the start of the prompt that holds row q0, rounded
      // down to a key tile where two slots share the stream (their tiles must coincide)
      auto kv_lo_of = [&](int32_t q0) {
        while (s + 1 < s_hi && seg_start[s + 1] <= q0) ++s;       // segment holding row q0
        return independent ? seg_start[s] : (seg_start[s] / tile_n) * tile_n;
      };
      const int32_t step = pair_rows ? 2 * kTileM : rq;
      for (int32_t q0 = 0; q0 < used; q0 += step) {
        WorkItem it{};
        it.bin = b;
        it.kv_row0 = kv_lo_of(q0);
        it.q_row0[0] = q0;
        if (!pair_rows) {                       // two heads, same rows
          it.q_row0[1] = q0;
          it.n_kv_tiles = (std::min(q0 + rq, used) - it.kv_row0 + tile_n - 1) / tile_n;
          it.jb1 = 0;
          it.je0 = it.n_kv_tiles;
        } else if (q0 + kTileM < used) {        // two consecutive row tiles
          const int32_t q1 = q0 + kTileM;
          it.q_row0[1] = q1;
          it.jb1 = (kv_lo_of(q1) - it.kv_row0) / tile_n;
          it.je0 = (q1 - it.kv_row0) / tile_n;  // slot 0 ends with its diagonal tile
          it.n_kv_tiles = (std::min(q1 + kTileM, used) - it.kv_row0 + tile_n - 1) / tile_n;
        } else {                                // last, unpaired row tile of the bin
          it.q_row0[1] = -1;
          it.n_kv_tiles = (used - it.kv_row0 + tile_n - 1) / tile_n;
          it.jb1 = it.n_kv_tiles;
          it.je0 = it.n_kv_tiles;
        }
        it.cost = it.je0 + (it.q_row0[1] >= 0 ? it.n_kv_tiles - it.jb1 : 0);
        it.bin_used = used;
        it.seg_end = s_hi;
        for (int t = 0; t < 2; ++t) {
          const int32_t q = it.q_row0[t];
          if (q < 0) continue;
          // segment holding row q: slot 0's rows ascend from item to item, slot 1 starts from slot 0's
          int32_t sf = s_slot0;
          while (sf + 1 < s_hi && seg_start[sf + 1] <= q) ++sf;
          if (t == 0) s_slot0 = sf;
          it.seg_first[t] = sf;
          it.key_lo[t] = seg_start[sf];
          const int32_t last_row = std::min(q + rq, used) - 1;
          if (sf + 1 >= s_hi || seg_start[sf + 1] > last_row) it.single_seg |= 1 << t;
        }
        items.push_back(it);
      }
    }
    // Longest first: CTAs draw items in list order, which gives longest-processing-time-first
    // scheduling; ties keep bin/row order (a stable counting sort over the costs).
    {
      int32_t max_cost = 0;
      for (const WorkItem& it : items) max_cost = std::max(max_cost, it.cost);
      std::vector<int32_t> first(max_cost + 2, 0);
      for (const WorkItem& it : items) ++first[it.cost];
      int32_t run = 0;
      for (int32_t c = max_cost; c >= 0; --c) { const int32_t n = first[c]; first[c] = run; run += n; }
      std::vector<WorkItem> sorted(items.size());
      for (const WorkItem& it : items) sorted[first[it.cost]++] = it;
      items.swap(sorted);
    }
  } catch (const std::bad_alloc&) {
    return PP_ERR_NO_MEMORY;
  }
  static_assert(sizeof(WorkItem) == kItemInts * sizeof(int32_t), "work item layout");
  std::memcpy(out + L.items, items.data(), sizeof(WorkItem) * items.size());
  L.n_items = (int32_t)items.size();
  out[0] = 0x50504b32;  // "PPK2"
  out[1] = L.n_items;
  out[2] = n_bins;
  out[3] = capacity;
  out[4] = k;
  out[5] = L.bin_seg_ptr;
  out[6] = L.bin_used;
  out[7] = L.seg_start;
  out[8] = L.items;
  int64_t tiles = 0;
  for (const WorkItem& it : items) tiles += it.cost;
  out[9] = (int32_t)std::min<int64_t>(tiles, INT32_MAX);
  out[kHeaderCounter] = 0;   // work counter the CTAs draw from; reset by every upload
  L.total_ints = (int32_t)(L.items + kItemInts * (int64_t)items.size());
  L.independent_slots = independent;
  L.pair_rows = pair_rows;
  L.fold = fold;
  if (layout) *layout = L;
  return PP_OK;
}

}  // namespace pp

extern "C" int pp_prefill_schedule_info(const pp_attn_params* params, const int32_t* bin_seg_ptr,
                                        const int32_t* seg_start, const int32_t* seg_len, int32_t k,
                                        int32_t* info) {
  if (!params || !info) return PP_ERR_INVALID_ARG;
  if (params->n_q_heads < 1 || params->n_kv_heads < 1) return PP_ERR_INVALID_ARG;
  if (params->n_q_heads % params->n_kv_heads != 0) return PP_ERR_UNSUPPORTED;
  int st = pp::validate_packing(params->n_bins, params->capacity, bin_seg_ptr, seg_start, seg_len, k);
  if (st != PP_OK) return st;
  try {
    const int32_t group = params->n_q_heads / params->n_kv_heads;
    std::vector<int32_t> table(pp::prefill_table_ints(params->n_bins, params->capacity, k, group));
    pp::TableLayout L;
    st = pp::build_prefill_tables(params->n_bins, params->capacity, bin_seg_ptr, seg_start, seg_len, k,
                                  group, table.data(), table.size(), &L);
    if (st != PP_OK) return st;
    const pp::WorkItem* items = reinterpret_cast<const pp::WorkItem*>(table.data() + L.items);
    int64_t steps = 0;
    int32_t unpaired = 0, late = 0;
    for (int32_t i = 0; i < L.n_items; ++i) {
      steps += items[i].cost;
      if (items[i].q_row0[1] < 0) ++unpaired;
      else if (items[i].jb1 > 0) ++late;
    }
    info[0] = L.independent_slots ? 1 : 0;
    info[1] = L.independent_slots ? 2 : (L.pair_rows ? 1 : 0);
    info[2] = L.n_items;
    info[3] = (int32_t)std::min<int64_t>(steps, INT32_MAX);
    info[4] = L.independent_slots ? pp::kTileNShort : pp::kTileN;
    info[5] = unpaired;
    info[6] = late;
    info[7] = L.fold;
  } catch (const std::bad_alloc&) {
    return PP_ERR_NO_MEMORY;
  }
  return PP_OK;
}
