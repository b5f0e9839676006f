// Range-partitioned merge of the workers' row lists (see agg_range.cuh).
//
//   split    first entry of every worker's list at or after each range boundary (binary search)
//   count    per range: worker-set table in shared memory -> number of distinct row ids
//   scan     distinct ids before each range; total = n_agg; capacity check
//   emit     per range: the table again, prefix sums over it, then every entry's slot in the
//            (row id, worker) order -> the same arrays the sort-based path hands to the tile
//            reduction (positions in merge order, head bits, first run of each tile, agg_ids)
//
// A direct gather-and-sum per distinct id inside the range CTA was measured first: 2.5 ms on the
// 100M-row workload against 1.06 ms for the tile reduction on the merge order, whose walk keeps
// four row loads in flight per lane and has no per-row search.
#include "agg_range.cuh"
#include "segsort.cuh"

namespace antdt {
namespace {

constexpr int kRaThreads = 256;
constexpr int kRaWarps = kRaThreads / 32;
constexpr int kRaBatch = 4;  // entries a thread loads before it processes them

size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

// ---------------------------------------------------------------------------------------
struct WeightBlob { float w[kRangeMaxWorkers]; };  // the workers' weights, a kernel parameter

__global__ void __launch_bounds__(kRaThreads)
range_split_kernel(const int32_t* __restrict__ ids, const int64_t* __restrict__ wuo_in, int K,
                   int64_t in_cap, int r_log2, int64_t P, uint32_t dropped,
                   int64_t* __restrict__ wuo_out, int64_t* __restrict__ n_entries,
                   int32_t* __restrict__ bnd, const WeightBlob weights, float* __restrict__ weights_out,
                   int32_t* status) {
  __shared__ int64_t s_wuo[kRangeMaxWorkers + 1];
  if (blockIdx.x == 0 && weights_out && threadIdx.x < K) weights_out[threadIdx.x] = weights.w[threadIdx.x];
  if (threadIdx.x == 0) {  // ascending and inside [0, in_cap], whatever came in
    int64_t prev = 0, kept = 0;
    for (int i = 0; i <= K; ++i) {
      int64_t v = wuo_in[i];
      v = v < prev ? prev : v;
      v = v > in_cap ? in_cap : v;
      s_wuo[i] = v;
      if (i > 0 && !((dropped >> (i - 1)) & 1u)) kept += v - prev;
      prev = v;
      if (blockIdx.x == 0) wuo_out[i] = v;
    }
    if (blockIdx.x == 0) {
      n_entries[0] = 0;   // read as [begin, end) of the merged entries by the reduction
      n_entries[1] = kept;
      if (wuo_in[K] < 0 || wuo_in[K] > in_cap) set_status(status, ANTDT_ERR_CAPACITY);
    }
  }
  __syncthreads();
  const int64_t idx = (int64_t)blockIdx.x * kRaThreads + threadIdx.x;
  if (idx >= (int64_t)K * (P + 1)) return;
  const int w = (int)(idx / (P + 1));
  const int64_t b = idx % (P + 1);
  const uint64_t key = (uint64_t)b << r_log2;  // b == P: past the last row id
  int64_t lo = s_wuo[w], hi = s_wuo[w + 1];
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if ((uint64_t)(uint32_t)__ldg(ids + mid) < key) lo = mid + 1; else hi = mid;
  }
  bnd[(size_t)w * (P + 1) + b] = (int32_t)lo;
  if (b == P && lo < s_wuo[w + 1]) set_status(status, ANTDT_ERR_ID_OUT_OF_RANGE);  // ids past the table
}

// The pieces of range b: worker w's entries [s_beg[w], s_beg[w] + size) with s_off[w] entries of
// earlier workers before them (s_off[K] = entries in the range; a dropped worker's piece is
// empty).  Also the number of entries of all earlier ranges.  One barrier inside.
struct Pieces { int entries; int64_t before; };
__device__ __forceinline__ Pieces range_pieces(const int32_t* __restrict__ bnd,
                                               const int64_t* __restrict__ wuo, int K, int64_t P,
                                               int64_t b, uint32_t dropped, int32_t* s_beg,
                                               int32_t* s_off, int64_t* s_before) {
  if (threadIdx.x < 32) {
    const int w = threadIdx.x;
    int beg = 0, size = 0;
    int64_t before = 0;
    if (w < K && !((dropped >> w) & 1u)) {
      beg = __ldg(bnd + (size_t)w * (P + 1) + b);
      const int end = __ldg(bnd + (size_t)w * (P + 1) + b + 1);
      size = end > beg ? end - beg : 0;  // a list that does not ascend: treated as empty here
      before = (int64_t)beg - __ldg(wuo + w);
    }
    int incl = size;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (w >= o) incl += t;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
    s_beg[w] = beg;
    s_off[w] = incl - size;
    if (w == 31) s_off[32] = incl;
    if (w == 0) *s_before = before;
  }
  __syncthreads();
  Pieces p;
  p.entries = s_off[32];
  p.before = *s_before;
  return p;
}

// Entry e of the range (entries numbered worker by worker): its worker and its position in the
// concatenated lists.
__device__ __forceinline__ void entry_of(int e, const int32_t* s_beg, const int32_t* s_off, int& w,
                                         int& j) {
  int lo = 0, hi = 32;  // last w with s_off[w] <= e: the non-empty piece that holds e
#pragma unroll
  for (int step = 0; step < 5; ++step) {
    const int mid = (lo + hi) >> 1;
    if (s_off[mid] <= e) lo = mid; else hi = mid;
  }
  w = lo;
  j = s_beg[lo] + (e - s_off[lo]);
}

// One pass over the range's entries, a batch of loads in flight per thread.  f(w, j, id, kl)
// for the entries whose row id lies in the range and in the table; the others raise
// ID_OUT_OF_RANGE and are skipped.
template <typename F>
__device__ __forceinline__ void for_each_entry(const int32_t* __restrict__ ids, int entries, int R,
                                               uint32_t base_key, int64_t n_rows, const int32_t* s_beg,
                                               const int32_t* s_off, int32_t* status, F f) {
  for (int e0 = threadIdx.x; e0 < entries; e0 += kRaBatch * kRaThreads) {
    int w[kRaBatch], j[kRaBatch];
    uint32_t id[kRaBatch];
#pragma unroll
    for (int t = 0; t < kRaBatch; ++t) {
      const int e = e0 + t * kRaThreads;
      entry_of(e < entries ? e : e0, s_beg, s_off, w[t], j[t]);
      id[t] = (uint32_t)__ldg(ids + j[t]);
    }
#pragma unroll
    for (int t = 0; t < kRaBatch; ++t) {
      if (e0 + t * kRaThreads >= entries) break;
      const uint32_t kl = id[t] - base_key;
      if (kl < (uint32_t)R && (int64_t)id[t] < n_rows) f(w[t], j[t], id[t], kl);
      else set_status(status, ANTDT_ERR_ID_OUT_OF_RANGE);
    }
  }
}

// Exclusive prefix sums of two per-thread counts over the CTA's 256 threads; totals returned
// through the references.  s_tmp: 16 ints.  Two barriers.
__device__ __forceinline__ void block_scan2(int& a, int& b, int& tot_a, int& tot_b, int32_t* s_tmp) {
  const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
  int ia = a, ib = b;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int ta = __shfl_up_sync(0xffffffffu, ia, o), tb = __shfl_up_sync(0xffffffffu, ib, o);
    if (lane >= o) { ia += ta; ib += tb; }
  }
  if (lane == 31) { s_tmp[wp] = ia; s_tmp[kRaWarps + wp] = ib; }
  __syncthreads();
  int pa = 0, pb = 0;
  tot_a = 0; tot_b = 0;
#pragma unroll
  for (int i = 0; i < kRaWarps; ++i) {
    const int va = s_tmp[i], vb = s_tmp[kRaWarps + i];
    pa += i < wp ? va : 0; pb += i < wp ? vb : 0;
    tot_a += va; tot_b += vb;
  }
  a = pa + ia - a;
  b = pb + ib - b;
  __syncthreads();
}

// Distinct row ids of range b: one presence bit per row id of the range.
__global__ void __launch_bounds__(kRaThreads)
range_count_kernel(const int32_t* __restrict__ ids, const int32_t* __restrict__ bnd,
                   const int64_t* __restrict__ wuo, int K, int64_t P, int r_log2, int64_t n_rows,
                   uint32_t dropped, int32_t* __restrict__ distinct, int32_t* status) {
  __shared__ uint32_t pres[(1 << kRangeMaxLog2) / 32];
  __shared__ int64_t s_before;
  __shared__ int32_t s_beg[32], s_off[33], s_tmp[2 * kRaWarps];
  const int R = 1 << r_log2;
  const int64_t b = blockIdx.x;
  const Pieces pc = range_pieces(bnd, wuo, K, P, b, dropped, s_beg, s_off, &s_before);
  if (pc.entries == 0) {
    if (threadIdx.x == 0) distinct[b] = 0;
    return;
  }
  if (threadIdx.x < R / 32) pres[threadIdx.x] = 0u;
  __syncthreads();
  for_each_entry(ids, pc.entries, R, (uint32_t)(b << r_log2), n_rows, s_beg, s_off, status,
                 [&](int, int, uint32_t, uint32_t kl) { atomicOr(&pres[kl >> 5], 1u << (kl & 31)); });
  __syncthreads();
  int cnt = threadIdx.x < R / 32 ? __popc(pres[threadIdx.x]) : 0, zero = 0, tot, tz;
  block_scan2(cnt, zero, tot, tz, s_tmp);
  if (threadIdx.x == 0) distinct[b] = tot;
}

// Exclusive scan of distinct[P] -> base[P+1]; one CTA of 1024 threads, consecutive ranges per
// thread.
__global__ void __launch_bounds__(1024)
range_scan_kernel(const int32_t* __restrict__ distinct, int64_t P, int64_t* __restrict__ base,
                  int64_t* __restrict__ n_agg, int64_t out_cap, int32_t* status) {
  __shared__ int64_t warp_tot[32];
  const int tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;
  const int64_t per = (P + 1023) / 1024;
  const int64_t c0 = (int64_t)tid * per, c1 = min(P, c0 + per);
  int64_t mine = 0;
  for (int64_t c = c0; c < c1; ++c) mine += distinct[c];
  int64_t incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int64_t t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_tot[wp] = incl;
  __syncthreads();
  if (wp == 0) {
    const int64_t v = warp_tot[lane];
    int64_t wi = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int64_t t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    warp_tot[lane] = wi - v;
    if (lane == 31) {
      base[P] = wi;
      *n_agg = wi;
      if (wi > out_cap) set_status(status, ANTDT_ERR_CAPACITY);
    }
  }
  __syncthreads();
  int64_t run = incl - mine + warp_tot[wp];
  for (int64_t c = c0; c < c1; ++c) {
    base[c] = run;
    run += distinct[c];
  }
}

// Writes the merge order of range b: for every entry its slot in the (row id, worker) order,
//   src[slot] = position of the entry in the concatenated lists,
// a head bit where a row's contributions start, agg_ids, and the run index of every entry whose
// slot starts a reduction tile.  slot = entries of earlier ranges + contributions of smaller row
// ids of this range + earlier workers holding the same row id.
//
// Shared memory: mask[R] (worker set per row id), pres[R/32] (presence bits: the table is
// sparse, so everything after the fill walks presence words and present ids only), per presence
// word the present ids before it (wrank), per present id the contributions before it (first_c).
// The worker sets are as wide as the worker count needs (8, 16 or 32 bits, packed into words) and
// first_c is 16 bits wide when a range cannot hold more than 2^16 entries: a CTA's shared memory
// decides how many ranges an SM works on at once, and with few entries per range the kernel's
// time is the number of CTA waves times a CTA's chain of global round trips.
struct EmitShape {
  int mask_lg;  // worker sets per 32-bit word, log2: 0, 1 (up to 16 workers), 2 (up to 8)
  int fc16;     // first_c holds 16-bit values
};
__host__ __device__ inline EmitShape emit_shape(int r_log2, int K) {
  EmitShape e;
  e.mask_lg = K <= 8 ? 2 : (K <= 16 ? 1 : 0);
  e.fc16 = ((int64_t)K << r_log2) <= 65536 ? 1 : 0;
  return e;
}

__global__ void __launch_bounds__(kRaThreads)
range_emit_kernel(const int32_t* __restrict__ ids, const int32_t* __restrict__ bnd,
                  const int64_t* __restrict__ wuo, int K, int64_t P, int r_log2, int64_t n_rows,
                  uint32_t dropped, const int64_t* __restrict__ base, int32_t* __restrict__ agg_ids,
                  int64_t out_cap, uint32_t* __restrict__ src, uint32_t* head_bits,
                  int32_t* __restrict__ tile_first, int tile_shift, uint32_t* __restrict__ row_start,
                  uint8_t* __restrict__ src_worker, int32_t* status) {
  extern __shared__ __align__(16) unsigned char ra_smem[];
  const int R = 1 << r_log2;
  const int nW = R / 32;  // presence words: at most 256 = one per thread
  const EmitShape shp = emit_shape(r_log2, K);
  const int lg = shp.mask_lg, sub = (1 << lg) - 1, sub_sh = 5 - lg;
  const uint32_t set_bits = 0xffffffffu >> (32 - (32 >> lg));
  uint32_t* mask = reinterpret_cast<uint32_t*>(ra_smem);  // R >> lg words
  uint32_t* first_c = mask + (R >> lg);
  unsigned short* first_c16 = reinterpret_cast<unsigned short*>(first_c);
  int64_t* s_before = reinterpret_cast<int64_t*>(first_c + (shp.fc16 ? R / 2 : R));
  auto workers_of = [&](int kl) { return (mask[kl >> lg] >> ((kl & sub) << sub_sh)) & set_bits; };
  uint32_t* pres = reinterpret_cast<uint32_t*>(s_before + 1);  // [256]
  int32_t* wrank = reinterpret_cast<int32_t*>(pres + 256);     // [256]
  int32_t* s_beg = wrank + 256;  // [32]
  int32_t* s_off = s_beg + 32;   // [33]
  int32_t* s_tmp = s_off + 33;   // [16]
  uint32_t* hb = reinterpret_cast<uint32_t*>(s_tmp + 16);  // head bits of this range's slots
  const int64_t b = blockIdx.x;
  const int tid = threadIdx.x;
  const int64_t u0 = __ldg(base + b);  // requested now: every global round trip here is serial
  const Pieces pc = range_pieces(bnd, wuo, K, P, b, dropped, s_beg, s_off, s_before);
  if (pc.entries == 0) return;
  // A worker lists a row id at most once, so a range holds at most R*K entries and the arrays
  // below are sized for that.  More means a list that does not strictly ascend: flag it and
  // leave the range out (its slots keep the zeroed head bits; the reduction bounds every index).
  if (pc.entries > (K << r_log2)) {
    if (tid == 0) set_status(status, ANTDT_ERR_BAD_OFFSETS);
    return;
  }
  // hb word i is global head-bit word (before >> 5) + i, same bit positions
  const int hb_shift = (int)(pc.before & 31);
  const int n_hw = (hb_shift + pc.entries + 31) >> 5;
  if (head_bits)  // (a reader that goes by row_start needs neither the head bits nor tile_first)
    for (int i = tid; i < n_hw; i += kRaThreads) hb[i] = 0u;
  if (tid < nW) pres[tid] = 0u;
  {
    uint4* m4 = reinterpret_cast<uint4*>(mask);
    for (int i = tid; i < (R >> lg) / 4; i += kRaThreads) m4[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  __syncthreads();
  const uint32_t base_key = (uint32_t)(b << r_log2);
  for_each_entry(ids, pc.entries, R, base_key, n_rows, s_beg, s_off, status,
                 [&](int w, int, uint32_t, uint32_t kl) {
                   atomicOr(&mask[kl >> lg], (1u << w) << ((kl & sub) << sub_sh));
                   atomicOr(&pres[kl >> 5], 1u << (kl & 31));
                 });
  __syncthreads();

  // thread q owns presence word q: present ids and contributions in it, prefix sums over the words
  const uint32_t pw = tid < nW ? pres[tid] : 0u;
  int n_ids = __popc(pw), n_con = 0;
  for (uint32_t rest = pw; rest; rest &= rest - 1u) n_con += __popc(workers_of(tid * 32 + __ffs((int)rest) - 1));
  int tot_ids, tot_con;
  block_scan2(n_ids, n_con, tot_ids, tot_con, s_tmp);  // now exclusive prefixes
  if (tid < nW) {
    wrank[tid] = n_ids;
    int t = n_ids, first = n_con;
    for (uint32_t rest = pw; rest; rest &= rest - 1u) {
      if (shp.fc16) first_c16[t++] = (unsigned short)first;
      else first_c[t++] = (uint32_t)first;
      if (head_bits) atomicOr(&hb[(hb_shift + first) >> 5], 1u << ((hb_shift + first) & 31));
      first += __popc(workers_of(tid * 32 + __ffs((int)rest) - 1));
    }
  }
  __syncthreads();

  // whole words of the head-bit mask are stored, words shared with a neighbour range are merged
  for (int i = tid; head_bits && i < n_hw; i += kRaThreads) {
    const uint32_t word = hb[i];
    if (word == 0u) continue;
    const int64_t g = (pc.before >> 5) + i;
    if (g * 32 >= pc.before && g * 32 + 32 <= pc.before + pc.entries) head_bits[g] = word;
    else atomicOr(&head_bits[g], word);
  }
  const int64_t tile_mask = ((int64_t)1 << tile_shift) - 1;
  for_each_entry(ids, pc.entries, R, base_key, n_rows, s_beg, s_off, nullptr,
                 [&](int w, int j, uint32_t id, uint32_t kl) {
                   const int t = wrank[kl >> 5] + __popc(pres[kl >> 5] & ((1u << (kl & 31)) - 1u));
                   const int slot = __popc(workers_of((int)kl) & ((1u << w) - 1u));
                   const int64_t dest = pc.before + (int64_t)(shp.fc16 ? first_c16[t] : first_c[t]) + slot;
                   const int64_t u = u0 + t;
                   src[dest] = (uint32_t)j;
                   if (src_worker) src_worker[dest] = (uint8_t)w;  // saves the reader a search
                   if (slot == 0 && u < out_cap) {
                     agg_ids[u] = (int32_t)id;
                     if (row_start) row_start[u] = (uint32_t)dest;  // the row's first merge slot
                   }
                   if (tile_first && (dest & tile_mask) == 0) tile_first[dest >> tile_shift] = (int32_t)u;
                 });
}

size_t emit_smem(int r_log2, int K) {  // tables, small arrays, head bits of up to R*K slots
  const size_t R = (size_t)1 << r_log2;
  const EmitShape e = emit_shape(r_log2, K);
  return 4 * (R >> e.mask_lg) + (e.fc16 ? 2 : 4) * R + 8 + 4 * (256 + 256 + 32 + 33 + 16) +
         4 * (R * (size_t)K / 32 + 2) + 12;
}

}  // namespace

RangeLayout range_layout(int K) {
  RangeLayout L;
  size_t o = 0;
  const size_t P = (size_t)kRangeMaxRanges;
  L.bnd = o;      o = align_up(o + 4 * (size_t)K * (P + 1));
  L.distinct = o; o = align_up(o + 4 * P);
  L.base = o;     o = align_up(o + 8 * (P + 1));
  L.bytes = o;
  return L;
}

void range_prepare_device() {
  static bool attr_set[64] = {};
  int dev_id = 0;
  cudaGetDevice(&dev_id);
  bool& done = attr_set[dev_id & 63];
  if (done) return;
  cudaFuncSetAttribute(range_emit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       (int)emit_smem(kRangeMaxLog2, kRangeMaxWorkers));
  done = true;
}

void range_merge_order(const int32_t* uniq_ids, const int64_t* wuo_in, int64_t in_cap, int64_t n_rows,
                       int K, uint32_t dropped_bits, int32_t* agg_ids, int64_t* n_agg, int64_t out_cap,
                       int64_t* wuo_out, int64_t* n_entries, uint32_t* src, uint32_t* head_bits,
                       int32_t* tile_first, int tile, uint32_t* row_start, uint8_t* src_worker,
                       const float* weights_host,
                       float* weights_dev, char* ws, const RangeLayout& L, int32_t* status,
                       cudaStream_t s) {
  range_prepare_device();
  WeightBlob wb;
  for (int i = 0; i < kRangeMaxWorkers; ++i) wb.w[i] = (weights_host && i < K) ? weights_host[i] : 0.f;
  const int r_log2 = range_log2(n_rows, in_cap);
  const int64_t P = (n_rows + ((int64_t)1 << r_log2) - 1) >> r_log2;  // <= kRangeMaxRanges
  int32_t* bnd = (int32_t*)(ws + L.bnd);
  int32_t* distinct = (int32_t*)(ws + L.distinct);
  int64_t* base = (int64_t*)(ws + L.base);
  int tile_shift = 0;
  while ((1 << tile_shift) < tile) ++tile_shift;
  const int64_t n_search = (int64_t)K * (P + 1);
  ANTDT_LAUNCH("agg_range_split", range_split_kernel, (unsigned)((n_search + kRaThreads - 1) / kRaThreads),
               kRaThreads, 0, s, uniq_ids, wuo_in, K, in_cap, r_log2, P, dropped_bits, wuo_out, n_entries,
               bnd, wb, weights_host ? weights_dev : nullptr, status);
  ANTDT_LAUNCH("agg_range_count", range_count_kernel, (unsigned)P, kRaThreads, 0, s,
               uniq_ids, bnd, wuo_out, K, P, r_log2, n_rows, dropped_bits, distinct, status);
  ANTDT_LAUNCH("agg_range_scan", range_scan_kernel, 1, 1024, 0, s, distinct, P, base, n_agg, out_cap,
               status);
  if (head_bits) cudaMemsetAsync(head_bits, 0, head_bits_words(in_cap) * 4, s);
  // every tile's entry is written unless ids were skipped as invalid: start from a valid index
  if (tile_first) cudaMemsetAsync(tile_first, 0, 4 * ((size_t)((in_cap + tile - 1) >> tile_shift) + 1), s);
  ANTDT_LAUNCH("agg_range_emit", range_emit_kernel, (unsigned)P, kRaThreads, emit_smem(r_log2, K), s,
               uniq_ids, bnd, wuo_out, K, P, r_log2, n_rows, dropped_bits, base, agg_ids, out_cap, src,
               head_bits, tile_first, tile_shift, row_start, src_worker, status);
}

}  // namespace antdt
