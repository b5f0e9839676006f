// Internal interface of the segmented radix sort and the "unique runs" pass built on it.
//
// sort:  stable LSD radix sort of (key, value) pairs, independently inside each of S
//        contiguous segments of one array (segment = one worker's occurrences in the backward
//        pass; one segment holding everything in the aggregation).  Sorting inside the
//        segments keeps the keys 32-bit whatever the worker count and saves the passes the
//        worker bits would cost.
// runs:  from the sorted keys, the distinct keys of every segment with the start of each run,
//        the number of runs before each segment, a bit per element marking run heads and, per
//        fixed-size tile of elements, the index of the run its first element belongs to.
//
// All sizes that are only known on the device (the element count of the aggregation) are read
// there: grids are sized from host-side capacities and the kernels loop to the device count.
#pragma once
#include "common.cuh"

namespace antdt {

constexpr int kSortCtasPerSM = 3;                            // scatter CTAs resident per SM
constexpr int kSortChunksTarget = kNumSM * kSortCtasPerSM;  // work units of the sort: one CTA each
constexpr int kSortThreads = 256;
constexpr int kSortItems = 16;
constexpr int kSortTile = kSortThreads * kSortItems;  // 4096 pairs staged in shared memory
constexpr int kSortMaxBits = 9;                       // up to 512 bins per pass
constexpr int kSortMaxBins = 1 << kSortMaxBits;
constexpr int kMaxSegments = 1024;
constexpr int kSetupMaxWorkers = 255;  // worker offsets that fit one kernel-parameter blob (2 KB)

// Device-side description of the chunks (written by segsort_setup, read by every pass).
struct SortDesc {
  int64_t n;           // elements
  int64_t chunk_elems; // multiple of kSortTile
  int32_t n_chunks;
  int32_t n_segments;
  int32_t pad[2];
};

// Byte layout of the sort's scratch inside a caller workspace (all offsets 256-byte aligned).
struct SortLayout {
  size_t desc;         // SortDesc
  size_t seg_bounds;   // int64 [S+1]   sanitised segment bounds
  size_t seg_first;    // int32 [S+1]   first chunk of each segment
  size_t chunk_seg;    // int32 [C]
  size_t chunk_begin;  // int64 [C]
  size_t chunk_end;    // int64 [C]
  size_t hist;         // uint32 [C * 512]
  size_t bin_base;     // uint32 [S * 512]
  size_t chunk_runs;   // int64 [16 C + 1]  run counts per strip of a chunk (runs pass)
  size_t bytes;        // total
  int max_chunks;      // C
  int n_segments;      // S
};
SortLayout sort_layout(int n_segments);

inline int sort_passes(int key_bits) { return (key_bits + kSortMaxBits - 1) / kSortMaxBits; }
// Words of the head-bit mask of n elements; readers look one tile past the last element.
inline size_t head_bits_words(int64_t n) { return (size_t)(n / 32) + 4; }
inline int bits_for(int64_t n_values) {  // bits needed for values in [0, n_values)
  int b = 1;
  while (b < 31 && (1ll << b) < n_values) ++b;
  return b;
}

// Sets the kernel attributes the sort needs on the current device (idempotent, cheap).
void segsort_prepare_device();

// seg_bounds_dev: int64 [S+1] device, ascending, last = element count (<= n_cap).  Builds the
// chunk descriptors in `ws` (laid out by sort_layout).
void segsort_setup(const int64_t* seg_bounds_dev, int n_segments, int64_t n_cap, char* ws,
                   const SortLayout& L, cudaStream_t s);

// The backward's set-up in ONE launch when there are at most kSetupMaxWorkers workers: takes the
// host's worker_sample_offsets [K+1] as a kernel parameter, derives every worker's occurrence
// range from bag_offsets (these are the sort's segments), writes 1/b_w to worker_b [K], checks the
// ends of bag_offsets, and builds the chunk descriptors.  false: too many workers, nothing launched.
bool segsort_setup_workers(const int64_t* wso_host, int n_workers, int bags_per_sample,
                           const int64_t* bag_offsets, int64_t n_bags, int64_t nnz, float* worker_b,
                           char* ws, const SortLayout& L, int32_t* status, cudaStream_t s);

// Sorts by the low key_bits bits.  keys_in is read only; the sorted pairs land in
// keys_out/vals_out; keys_tmp/vals_tmp are scratch of the same size.  vals_in == nullptr means
// "value = element index".  check_rows > 0: keys >= check_rows raise ID_OUT_OF_RANGE.
// n_cap: the element count the set-up was given (a host-side bound on the chunks that exist).
// agg only selects the names under which the launches are accounted.
void segsort_run(const uint32_t* keys_in, const uint32_t* vals_in, uint32_t* keys_out,
                 uint32_t* vals_out, uint32_t* keys_tmp, uint32_t* vals_tmp, int key_bits,
                 int64_t check_rows, int64_t n_cap, char* ws, const SortLayout& L, int32_t* status,
                 cudaStream_t s, bool agg = false);

// Runs of equal keys inside the segments of a sorted array.
//   uniq_keys  [out_cap]    key of each run, in array order
//   run_start  [out_cap+1]  first element of each run; entry [n_runs] = n
//   seg_runs   [S+1]        runs before each segment; [S] = n_runs  (may be nullptr)
//   n_runs_out one int64    (may be nullptr)
//   head_bits  [head_bits_words(n_cap)] bit i set iff element i starts a run (zeroed here unless head_bits_zeroed)
//   tile_first [n_cap/tile+1] run index of element t*tile (may be nullptr); tile a power of 2
// More runs than out_cap -> CAPACITY in status, the excess is not written.
void segsort_runs(const uint32_t* sorted_keys, int64_t n_cap, int32_t* uniq_keys,
                  int64_t* run_start, int64_t* seg_runs, int64_t* n_runs_out, int64_t out_cap,
                  uint32_t* head_bits, int32_t* tile_first, int tile, char* ws,
                  const SortLayout& L, int32_t* status, cudaStream_t s, bool agg = false,
                  bool head_bits_zeroed = false);  // true: the caller cleared head_bits on this stream

}  // namespace antdt
