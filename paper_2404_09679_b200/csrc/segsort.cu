// Segmented stable LSD radix sort of (key, value) pairs and the run-detection pass over the
// sorted keys.  Integer work only: results are bit-exact and independent of scheduling.
//
// Work decomposition: every segment is cut into chunks of chunk_elems consecutive elements
// (about kSortChunksTarget chunks in all, one CTA each, so a pass is a single wave on 148 SMs
// at 4 CTAs per SM).  One pass = histogram per chunk -> exclusive scan over (bin, chunk) inside
// each segment -> scatter.  The scatter ranks a 4096-pair tile with warp match/ballot
// (stable: tile order is warp-striped), reorders the tile in shared memory by bin and writes
// each bin's run with consecutive threads, so global stores are as coalesced as the digit
// distribution allows.
#include "segsort.cuh"

namespace antdt {
namespace {

size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

// ---------------------------------------------------------------------------------------
// block-wide exclusive scan of int64 over blockDim.x == 1024 threads, one value per thread
// ---------------------------------------------------------------------------------------
__device__ int64_t block_exclusive_scan_1024(int64_t v, int64_t* total, int64_t* warp_tot /*[32]*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int64_t incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int64_t t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int64_t w = warp_tot[lane];
    int64_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int64_t t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    warp_tot[lane] = wi - w;  // exclusive prefix of warp totals
    if (lane == 31) *total = wi;
  }
  __syncthreads();
  return incl - v + warp_tot[warp];
}

// ---------------------------------------------------------------------------------------
// setup: sanitise the segment bounds and cut the segments into chunks
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
segsort_setup_kernel(const int64_t* __restrict__ bounds_in, int S, int64_t n_cap, SortDesc* desc,
                     int64_t* seg_bounds, int32_t* seg_first, int32_t* chunk_seg,
                     int64_t* chunk_begin, int64_t* chunk_end, int max_chunks) {
  __shared__ int64_t sb[kMaxSegments + 1];
  __shared__ int32_t sf[kMaxSegments + 1];
  __shared__ int64_t s_chunk_elems;
  const int tid = threadIdx.x;
  if (tid == 0) {
    int64_t prev = 0;
    for (int s = 0; s <= S; ++s) {  // ascending and inside [0, n_cap], whatever came in
      int64_t v = bounds_in[s];
      v = v < prev ? prev : v;
      v = v > n_cap ? n_cap : v;
      sb[s] = v;
      prev = v;
    }
    const int64_t total = sb[S] - sb[0];
    int64_t ce = (total + kSortChunksTarget - 1) / kSortChunksTarget;
    ce = ((ce + kSortTile - 1) / kSortTile) * kSortTile;
    if (ce < kSortTile) ce = kSortTile;
    s_chunk_elems = ce;
    int32_t c = 0;
    for (int s = 0; s < S; ++s) {
      sf[s] = c;
      c += (int32_t)((sb[s + 1] - sb[s] + ce - 1) / ce);
    }
    sf[S] = c < max_chunks ? c : max_chunks;  // c <= target + S always; the clamp is a guard
    desc->n = sb[S];
    desc->chunk_elems = ce;
    desc->n_chunks = sf[S];
    desc->n_segments = S;
  }
  __syncthreads();
  const int64_t ce = s_chunk_elems;
  const int n_chunks = sf[S];
  for (int s = tid; s <= S; s += blockDim.x) {
    seg_bounds[s] = sb[s];
    seg_first[s] = sf[s];
  }
  for (int c = tid; c < n_chunks; c += blockDim.x) {
    int lo = 0, hi = S;  // last segment with sf[seg] <= c that is not empty of chunks
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (sf[mid] <= c) lo = mid; else hi = mid;
    }
    const int64_t b = sb[lo] + (int64_t)(c - sf[lo]) * ce;
    chunk_seg[c] = lo;
    chunk_begin[c] = b;
    chunk_end[c] = min(b + ce, sb[lo + 1]);
  }
}

// ---------------------------------------------------------------------------------------
// pass step 1: digit histogram of every chunk
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSortThreads)
radix_hist_kernel(const uint32_t* __restrict__ keys, int shift, uint32_t mask,
                  const SortDesc* __restrict__ desc, const int64_t* __restrict__ chunk_begin,
                  const int64_t* __restrict__ chunk_end, uint32_t* __restrict__ hist,
                  int64_t check_rows, int32_t* status) {
  const int c = blockIdx.x;
  if (c >= desc->n_chunks) return;
  __shared__ uint32_t sh[kSortMaxBins];
  const int tid = threadIdx.x, lane = tid & 31;
  for (int d = tid; d < kSortMaxBins; d += kSortThreads) sh[d] = 0;
  __syncthreads();
  const int64_t b = chunk_begin[c], e = chunk_end[c];
  bool bad = false;
  for (int64_t i0 = b; i0 < e; i0 += kSortThreads) {
    const int64_t i = i0 + tid;
    const bool valid = i < e;
    uint32_t d = kSortMaxBins;  // sentinel: matches only other idle lanes
    if (valid) {
      const uint32_t k = __ldg(keys + i);
      bad |= (check_rows > 0 && (int64_t)k >= check_rows);
      d = (k >> shift) & mask;
    }
    // one shared-memory add per distinct digit in the warp (hot rows would serialise otherwise)
    const unsigned m = __match_any_sync(0xffffffffu, d);
    if (valid && lane == __ffs(m) - 1) atomicAdd(&sh[d], (uint32_t)__popc(m));
  }
  if (bad) set_status(status, ANTDT_ERR_ID_OUT_OF_RANGE);
  __syncthreads();
  for (int d = tid; d < kSortMaxBins; d += kSortThreads) hist[(size_t)c * kSortMaxBins + d] = sh[d];
}

// ---------------------------------------------------------------------------------------
// pass step 2: per segment, exclusive scan over chunks inside each bin and over the bins
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSortMaxBins)
radix_scan_kernel(const SortDesc* __restrict__ desc, const int32_t* __restrict__ seg_first,
                  uint32_t* hist, uint32_t* __restrict__ bin_base) {
  const int s = blockIdx.x;
  if (s >= desc->n_segments) return;
  const int d = threadIdx.x;
  const int c0 = seg_first[s], c1 = seg_first[s + 1];
  uint32_t run = 0;
  constexpr int kBatch = 8;
  for (int c = c0; c < c1; c += kBatch) {
    uint32_t t[kBatch];
#pragma unroll
    for (int j = 0; j < kBatch; ++j)
      t[j] = (c + j < c1) ? hist[(size_t)(c + j) * kSortMaxBins + d] : 0u;
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
      if (c + j < c1) hist[(size_t)(c + j) * kSortMaxBins + d] = run;
      run += t[j];
    }
  }
  __shared__ uint32_t tmp[kSortMaxBins];
  tmp[d] = run;
  __syncthreads();
  for (int o = 1; o < kSortMaxBins; o <<= 1) {
    const uint32_t v = d >= o ? tmp[d - o] : 0u;
    __syncthreads();
    tmp[d] += v;
    __syncthreads();
  }
  bin_base[(size_t)s * kSortMaxBins + d] = tmp[d] - run;
}

// ---------------------------------------------------------------------------------------
// pass step 3: stable scatter
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSortThreads)
radix_scatter_kernel(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
                     uint32_t* __restrict__ keys_out, uint32_t* __restrict__ vals_out, int shift,
                     uint32_t mask, const SortDesc* __restrict__ desc,
                     const int32_t* __restrict__ chunk_seg, const int64_t* __restrict__ seg_bounds,
                     const int64_t* __restrict__ chunk_begin, const int64_t* __restrict__ chunk_end,
                     const uint32_t* __restrict__ hist, const uint32_t* __restrict__ bin_base) {
  const int c = blockIdx.x;
  if (c >= desc->n_chunks) return;
  constexpr int kWarps = kSortThreads / 32;
  __shared__ uint32_t gbase[kSortMaxBins];      // next global slot of every bin (this chunk)
  __shared__ uint32_t bin_start[kSortMaxBins];  // first slot of every bin inside the tile
  __shared__ uint32_t bin_cnt[kSortMaxBins];
  __shared__ unsigned short wh[kWarps][kSortMaxBins];
  __shared__ uint32_t skeys[kSortTile];
  __shared__ uint32_t svals[kSortTile];
  __shared__ uint32_t warp_tot[kWarps];

  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const unsigned lt = (1u << lane) - 1u;
  const int seg = chunk_seg[c];
  const uint32_t seg_begin = (uint32_t)seg_bounds[seg];
  for (int d = tid; d < kSortMaxBins; d += kSortThreads)
    gbase[d] = seg_begin + bin_base[(size_t)seg * kSortMaxBins + d] +
               hist[(size_t)c * kSortMaxBins + d];

  const int64_t cb = chunk_begin[c], ce = chunk_end[c];
  for (int64_t pos = cb; pos < ce; pos += kSortTile) {
    const int tile_n = (int)min((int64_t)kSortTile, ce - pos);
    uint32_t k[kSortItems], v[kSortItems];
    unsigned short rank[kSortItems];
    // warp-striped: warp w owns elements [w*512, w*512+512) of the tile, item i of lane l is
    // element w*512 + i*32 + l, so (item, lane) order is element order
    const int wbase = w * (32 * kSortItems) + lane;
#pragma unroll
    for (int i = 0; i < kSortItems; ++i) {
      const int j = wbase + i * 32;
      if (j < tile_n) {
        k[i] = __ldg(keys_in + pos + j);
        v[i] = vals_in ? __ldg(vals_in + pos + j) : (uint32_t)(pos + j);
      } else {
        k[i] = 0xffffffffu;
        v[i] = 0;
      }
    }
    uint32_t* whz = reinterpret_cast<uint32_t*>(&wh[0][0]);
    for (int d = tid; d < kWarps * kSortMaxBins / 2; d += kSortThreads) whz[d] = 0;
    __syncthreads();  // (A) also: the previous tile's write-out is over

#pragma unroll
    for (int i = 0; i < kSortItems; ++i) {
      const bool valid = wbase + i * 32 < tile_n;
      const uint32_t d = valid ? ((k[i] >> shift) & mask) : (uint32_t)kSortMaxBins;
      const unsigned m = __match_any_sync(0xffffffffu, d);
      const int leader = __ffs(m) - 1;
      uint32_t old = 0;
      if (valid && lane == leader) {
        old = wh[w][d];
        wh[w][d] = (unsigned short)(old + __popc(m));
      }
      old = __shfl_sync(0xffffffffu, old, leader);
      rank[i] = (unsigned short)(old + __popc(m & lt));
      __syncwarp();
    }
    __syncthreads();  // (B)

    // per bin: exclusive scan over the warps; bin totals
    for (int d = tid; d < kSortMaxBins; d += kSortThreads) {
      uint32_t s = 0;
#pragma unroll
      for (int ww = 0; ww < kWarps; ++ww) {
        const uint32_t t = wh[ww][d];
        wh[ww][d] = (unsigned short)s;
        s += t;
      }
      bin_cnt[d] = s;
    }
    __syncthreads();  // (C)

    {  // exclusive scan over the 512 bins: thread t owns bins 2t and 2t+1
      const uint32_t a = bin_cnt[2 * tid], b2 = bin_cnt[2 * tid + 1];
      uint32_t incl = a + b2;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      if (lane == 31) warp_tot[w] = incl;
      __syncthreads();
      uint32_t wp = 0;
#pragma unroll
      for (int ww = 0; ww < kWarps; ++ww) wp += (ww < w) ? warp_tot[ww] : 0u;
      const uint32_t excl = incl - (a + b2) + wp;
      bin_start[2 * tid] = excl;
      bin_start[2 * tid + 1] = excl + a;
    }
    __syncthreads();  // (D)

#pragma unroll
    for (int i = 0; i < kSortItems; ++i) {
      if (wbase + i * 32 < tile_n) {
        const uint32_t d = (k[i] >> shift) & mask;
        const uint32_t p = bin_start[d] + wh[w][d] + rank[i];
        skeys[p] = k[i];
        svals[p] = v[i];
      }
    }
    __syncthreads();  // (E)

    for (int j = tid; j < tile_n; j += kSortThreads) {
      const uint32_t kk = skeys[j];
      const uint32_t d = (kk >> shift) & mask;
      const uint32_t g = gbase[d] + ((uint32_t)j - bin_start[d]);
      keys_out[g] = kk;
      vals_out[g] = svals[j];
    }
    __syncthreads();  // (F)
    for (int d = tid; d < kSortMaxBins; d += kSortThreads) gbase[d] += bin_cnt[d];
  }
}

// ---------------------------------------------------------------------------------------
// runs of equal keys
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSortThreads)
runs_count_kernel(const uint32_t* __restrict__ keys, const SortDesc* __restrict__ desc,
                  const int32_t* __restrict__ chunk_seg, const int64_t* __restrict__ seg_bounds,
                  const int64_t* __restrict__ chunk_begin, const int64_t* __restrict__ chunk_end,
                  int64_t* __restrict__ chunk_runs) {
  const int c = blockIdx.x;
  if (c >= desc->n_chunks) return;
  const int tid = threadIdx.x;
  const int64_t b = chunk_begin[c], e = chunk_end[c];
  const int64_t seg_begin = seg_bounds[chunk_seg[c]];
  int cnt = 0;
  for (int64_t i = b + tid; i < e; i += kSortThreads)
    cnt += (i == seg_begin) || (__ldg(keys + i) != __ldg(keys + i - 1));
  __shared__ int wsum[kSortThreads / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) cnt += __shfl_down_sync(0xffffffffu, cnt, o);
  if ((tid & 31) == 0) wsum[tid >> 5] = cnt;
  __syncthreads();
  if (tid == 0) {
    int t = 0;
    for (int ww = 0; ww < kSortThreads / 32; ++ww) t += wsum[ww];
    chunk_runs[c] = t;
  }
}

__global__ void __launch_bounds__(1024)
runs_scan_kernel(const SortDesc* __restrict__ desc, const int32_t* __restrict__ seg_first,
                 int64_t* chunk_runs, int64_t* seg_runs, int64_t* n_runs_out, int64_t* run_start,
                 int64_t out_cap, int32_t* status) {
  __shared__ int64_t warp_tot[32];
  __shared__ int64_t total;
  const int n_chunks = desc->n_chunks;
  const int tid = threadIdx.x;
  const int per = (n_chunks + 1023) / 1024;  // consecutive chunks per thread
  const int c0 = tid * per, c1 = min(n_chunks, c0 + per);
  int64_t mine = 0;
  for (int c = c0; c < c1; ++c) mine += chunk_runs[c];
  int64_t excl = block_exclusive_scan_1024(mine, &total, warp_tot);
  for (int c = c0; c < c1; ++c) {
    const int64_t t = chunk_runs[c];
    chunk_runs[c] = excl;
    excl += t;
  }
  __syncthreads();
  if (tid == 0) {
    chunk_runs[n_chunks] = total;
    if (n_runs_out) *n_runs_out = total;
    run_start[total < out_cap ? total : out_cap] = desc->n;
    if (total > out_cap) set_status(status, ANTDT_ERR_CAPACITY);
  }
  __syncthreads();
  if (seg_runs)
    for (int s = tid; s <= desc->n_segments; s += blockDim.x) seg_runs[s] = chunk_runs[seg_first[s]];
}

__global__ void __launch_bounds__(kSortThreads)
runs_emit_kernel(const uint32_t* __restrict__ keys, const SortDesc* __restrict__ desc,
                 const int32_t* __restrict__ chunk_seg, const int64_t* __restrict__ seg_bounds,
                 const int64_t* __restrict__ chunk_begin, const int64_t* __restrict__ chunk_end,
                 const int64_t* __restrict__ chunk_runs, int32_t* __restrict__ uniq_keys,
                 int64_t* __restrict__ run_start, int64_t out_cap, uint32_t* head_bits,
                 int32_t* __restrict__ tile_first, int tile) {
  const int c = blockIdx.x;
  if (c >= desc->n_chunks) return;
  constexpr int kWarps = kSortThreads / 32;
  __shared__ int wtot[kWarps];
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int64_t b = chunk_begin[c], e = chunk_end[c];
  const int64_t seg_begin = seg_bounds[chunk_seg[c]];
  int64_t running = chunk_runs[c];  // runs that start before this chunk
  for (int64_t i0 = b; i0 < e; i0 += kSortThreads) {
    const int64_t i = i0 + tid;
    const bool valid = i < e;
    uint32_t key = 0;
    bool head = false;
    if (valid) {
      key = __ldg(keys + i);
      head = (i == seg_begin) || (key != __ldg(keys + i - 1));
    }
    const unsigned bal = __ballot_sync(0xffffffffu, head);
    if (lane == 0) wtot[w] = __popc(bal);
    __syncthreads();
    int before = 0, all = 0;
#pragma unroll
    for (int ww = 0; ww < kWarps; ++ww) {
      const int t = wtot[ww];
      before += ww < w ? t : 0;
      all += t;
    }
    const int64_t incl = running + before + __popc(bal & ((2u << lane) - 1u));
    if (head) {
      const int64_t r = incl - 1;
      if (r < out_cap) {
        uniq_keys[r] = (int32_t)key;
        run_start[r] = i;
      }
    }
    if (valid && tile_first && (i % tile) == 0) tile_first[i / tile] = (int32_t)(incl - 1);
    if (head_bits && lane == 0 && bal) {  // the warp's 32 flags straddle at most two words
      const int64_t first = i0 + w * 32;
      const int sh = (int)(first & 31);
      atomicOr(&head_bits[first >> 5], bal << sh);
      if (sh && (bal >> (32 - sh))) atomicOr(&head_bits[(first >> 5) + 1], bal >> (32 - sh));
    }
    running += all;
    __syncthreads();
  }
}

}  // namespace

// =========================================================================================
SortLayout sort_layout(int S) {
  SortLayout L;
  const size_t C = (size_t)kSortChunksTarget + (size_t)S;
  L.max_chunks = (int)C;
  size_t o = 0;
  L.desc = o;        o = align_up(o + sizeof(SortDesc));
  L.seg_bounds = o;  o = align_up(o + 8 * ((size_t)S + 1));
  L.seg_first = o;   o = align_up(o + 4 * ((size_t)S + 1));
  L.chunk_seg = o;   o = align_up(o + 4 * C);
  L.chunk_begin = o; o = align_up(o + 8 * C);
  L.chunk_end = o;   o = align_up(o + 8 * C);
  L.hist = o;        o = align_up(o + 4 * C * kSortMaxBins);
  L.bin_base = o;    o = align_up(o + 4 * (size_t)S * kSortMaxBins);
  L.chunk_runs = o;  o = align_up(o + 8 * (C + 1));
  L.bytes = o;
  return L;
}

void segsort_setup(const int64_t* seg_bounds_dev, int S, int64_t n_cap, char* ws,
                   const SortLayout& L, cudaStream_t s) {
  ANTDT_LAUNCH("segsort_setup", segsort_setup_kernel, 1, 1024, 0, s, seg_bounds_dev, S, n_cap,
               (SortDesc*)(ws + L.desc), (int64_t*)(ws + L.seg_bounds),
               (int32_t*)(ws + L.seg_first), (int32_t*)(ws + L.chunk_seg),
               (int64_t*)(ws + L.chunk_begin), (int64_t*)(ws + L.chunk_end), L.max_chunks);
}

void segsort_run(const uint32_t* keys_in, const uint32_t* vals_in, uint32_t* keys_out,
                 uint32_t* vals_out, uint32_t* keys_tmp, uint32_t* vals_tmp, int key_bits,
                 int64_t check_rows, char* ws, const SortLayout& L, int32_t* status,
                 cudaStream_t s) {
  const SortDesc* desc = (const SortDesc*)(ws + L.desc);
  const int64_t* seg_bounds = (const int64_t*)(ws + L.seg_bounds);
  const int32_t* seg_first = (const int32_t*)(ws + L.seg_first);
  const int32_t* chunk_seg = (const int32_t*)(ws + L.chunk_seg);
  const int64_t* chunk_begin = (const int64_t*)(ws + L.chunk_begin);
  const int64_t* chunk_end = (const int64_t*)(ws + L.chunk_end);
  uint32_t* hist = (uint32_t*)(ws + L.hist);
  uint32_t* bin_base = (uint32_t*)(ws + L.bin_base);
  const int P = sort_passes(key_bits);
  // spread the bits evenly over the passes
  int shift = 0;
  const uint32_t* kin = keys_in;
  const uint32_t* vin = vals_in;
  const int S = L.max_chunks - kSortChunksTarget;
  for (int p = 0; p < P; ++p) {
    const int bits = (key_bits - shift + (P - p) - 1) / (P - p);
    const uint32_t mask = (1u << bits) - 1u;
    // the last pass lands in the output buffers, the one before in the temporaries, ...
    const bool to_out = ((P - 1 - p) % 2) == 0;
    uint32_t* kout = to_out ? keys_out : keys_tmp;
    uint32_t* vout = to_out ? vals_out : vals_tmp;
    ANTDT_LAUNCH("radix_hist", radix_hist_kernel, L.max_chunks, kSortThreads, 0, s, kin, shift,
                 mask, desc, chunk_begin, chunk_end, hist, p == 0 ? check_rows : (int64_t)0, status);
    ANTDT_LAUNCH("radix_scan", radix_scan_kernel, S, kSortMaxBins, 0, s, desc, seg_first, hist,
                 bin_base);
    ANTDT_LAUNCH("radix_scatter", radix_scatter_kernel, L.max_chunks, kSortThreads, 0, s, kin, vin,
                 kout, vout, shift, mask, desc, chunk_seg, seg_bounds, chunk_begin, chunk_end, hist,
                 bin_base);
    kin = kout;
    vin = vout;
    shift += bits;
  }
}

void segsort_runs(const uint32_t* sorted_keys, int64_t n_cap, int32_t* uniq_keys,
                  int64_t* run_start, int64_t* seg_runs, int64_t* n_runs_out, int64_t out_cap,
                  uint32_t* head_bits, int32_t* tile_first, int tile, char* ws,
                  const SortLayout& L, int32_t* status, cudaStream_t s) {
  const SortDesc* desc = (const SortDesc*)(ws + L.desc);
  const int64_t* seg_bounds = (const int64_t*)(ws + L.seg_bounds);
  const int32_t* seg_first = (const int32_t*)(ws + L.seg_first);
  const int32_t* chunk_seg = (const int32_t*)(ws + L.chunk_seg);
  const int64_t* chunk_begin = (const int64_t*)(ws + L.chunk_begin);
  const int64_t* chunk_end = (const int64_t*)(ws + L.chunk_end);
  int64_t* chunk_runs = (int64_t*)(ws + L.chunk_runs);
  if (head_bits) cudaMemsetAsync(head_bits, 0, head_bits_words(n_cap) * 4, s);
  ANTDT_LAUNCH("runs_count", runs_count_kernel, L.max_chunks, kSortThreads, 0, s, sorted_keys,
               desc, chunk_seg, seg_bounds, chunk_begin, chunk_end, chunk_runs);
  ANTDT_LAUNCH("runs_scan", runs_scan_kernel, 1, 1024, 0, s, desc, seg_first, chunk_runs, seg_runs,
               n_runs_out, run_start, out_cap, status);
  ANTDT_LAUNCH("runs_emit", runs_emit_kernel, L.max_chunks, kSortThreads, 0, s, sorted_keys, desc,
               chunk_seg, seg_bounds, chunk_begin, chunk_end, chunk_runs, uniq_keys, run_start,
               out_cap, head_bits, tile_first, tile);
}

}  // namespace antdt
