// Internal interface of the range-partitioned merge of the workers' row lists (the sparse part
// of the server aggregation for up to 32 workers).
//
// Every worker's list of row ids ascends, so the part of it that falls into a range of R
// consecutive row ids is one contiguous piece, found by binary search.  One CTA takes one range:
// a table of R words in shared memory holds, for each row id of the range, the set of workers
// whose list contains it (one bit per worker).  Non-zero words, in order, ARE the merged list of
// distinct ids; the set bits of a word, in order, are the contributions of that row in ascending
// worker order.  No sort and no waiting on other CTAs, and nothing depends on how the ids are
// distributed: a range never holds more than R * K entries.
#pragma once
#include "common.cuh"

namespace antdt {

constexpr int kRangeMaxWorkers = 32;        // one bit per worker in a 32-bit word
constexpr int kRangeLog2 = 12;              // 4096 row ids per range (measured best of 1024..8192)
constexpr int kRangeMaxLog2 = 13;           // 8192 for tables beyond 2^30 rows (bounds the scratch)
constexpr int64_t kRangeMaxRanges = (int64_t)1 << (31 - kRangeMaxLog2);  // n_rows < 2^31

// log2 of the range width.  The wide ranges also serve an input that is sparse in the table
// (fewer than 64 entries per narrow range on average): a range CTA's cost is mostly its fixed part
// then, so half as many CTAs finish sooner.
inline int range_log2(int64_t n_rows, int64_t in_cap) {
  if (n_rows > ((int64_t)kRangeMaxRanges << kRangeLog2)) return kRangeMaxLog2;
  const int64_t narrow = (n_rows + ((int64_t)1 << kRangeLog2) - 1) >> kRangeLog2;
  return in_cap < 64 * narrow ? kRangeMaxLog2 : kRangeLog2;
}

struct RangeLayout {
  size_t bnd;       // int32 [K][P+1]  first entry of worker w at or after row id b*R
  size_t distinct;  // int32 [P]       distinct row ids in range b
  size_t base;      // int64 [P+1]     distinct row ids before range b; [P] = total
  size_t bytes;
};
// Sized for the largest table (the workspace query does not know n_rows).
RangeLayout range_layout(int K);

// Sets the kernel attributes of this path on the current device (idempotent).
void range_prepare_device();

// Merge order of the workers' lists, ready for the tile reduction (tile_reduce.cuh):
//   wuo_in [K+1] raw offsets (clamped to in_cap into wuo_out), dropped_bits: bit w = ignore worker w
//   agg_ids [out_cap]   distinct row ids ascending;  n_agg = their number
//   n_entries [2]       {0, entries of the workers that count}
//   src [in_cap]        position (in the concatenated lists) of the entry at each merge slot;
//                       slots ordered by (row id, worker)
//   head_bits           bit i set iff slot i is the first contribution of its row (zeroed here)
//   tile_first          index into agg_ids of the row that slot t*tile belongs to
//                       (head_bits and tile_first may both be nullptr: a reader that goes by
//                       row_start needs neither)
//   row_start [out_cap] merge slot of the first contribution of each row of agg_ids, or nullptr
//   src_worker [in_cap] the worker of every merge slot (one byte), or nullptr
//   weights_host [K]    the workers' weights; the first kernel carries them to weights_dev [K]
//                       as a parameter (nullptr: the caller has put them there already)
void range_merge_order(const int32_t* uniq_ids, const int64_t* wuo_in, int64_t in_cap, int64_t n_rows,
                       int K, uint32_t dropped_bits, int32_t* agg_ids, int64_t* n_agg, int64_t out_cap,
                       int64_t* wuo_out, int64_t* n_entries, uint32_t* src, uint32_t* head_bits,
                       int32_t* tile_first, int tile, uint32_t* row_start, uint8_t* src_worker,
                       const float* weights_host,
                       float* weights_dev, char* ws, const RangeLayout& L, int32_t* status,
                       cudaStream_t s);

}  // namespace antdt
