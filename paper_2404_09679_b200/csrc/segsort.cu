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
// The body of the set-up, run by one CTA of 1024 threads.  bounds_in may be global or shared memory.
__device__ __forceinline__ void segsort_setup_body(const int64_t* bounds_in, int S, int64_t n_cap,
                                                   SortDesc* desc, int64_t* seg_bounds, int32_t* seg_first,
                                                   int32_t* chunk_seg, int64_t* chunk_begin,
                                                   int64_t* chunk_end, int max_chunks) {
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
    // every segment ends in a partial chunk: aim for (slots - S) chunks so that all of them
    // are resident at once (one wave at kSortCtasPerSM CTAs per SM)
    const int64_t target = max(kSortChunksTarget / 2, kSortChunksTarget - S);
    int64_t ce = (total + target - 1) / target;
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

__global__ void __launch_bounds__(1024)
segsort_setup_kernel(const int64_t* __restrict__ bounds_in, int S, int64_t n_cap, SortDesc* desc,
                     int64_t* seg_bounds, int32_t* seg_first, int32_t* chunk_seg,
                     int64_t* chunk_begin, int64_t* chunk_end, int max_chunks) {
  segsort_setup_body(bounds_in, S, n_cap, desc, seg_bounds, seg_first, chunk_seg, chunk_begin, chunk_end,
                     max_chunks);
}

// The backward's set-up in one launch: the workers' sample offsets arrive as a kernel parameter,
// their occurrence ranges are read off bag_offsets (the segments of the sort), 1/b_w is written,
// the offsets' ends are checked, and the chunks are cut as above.
struct WorkerBlob { int64_t wso[kSetupMaxWorkers + 1]; };
__global__ void __launch_bounds__(1024)
bwd_setup_kernel(const WorkerBlob blob, int K, int F, const int64_t* __restrict__ bag_offsets,
                 int64_t n_bags, int64_t nnz, float* __restrict__ worker_b, SortDesc* desc,
                 int64_t* seg_bounds, int32_t* seg_first, int32_t* chunk_seg, int64_t* chunk_begin,
                 int64_t* chunk_end, int max_chunks, int32_t* status) {
  __shared__ int64_t s_occ[kSetupMaxWorkers + 1];
  const int tid = threadIdx.x;
  if (tid == 0 && (bag_offsets[0] != 0 || bag_offsets[n_bags] != nnz))
    set_status(status, ANTDT_ERR_BAD_OFFSETS);
  for (int w = tid; w <= K; w += blockDim.x) {
    s_occ[w] = bag_offsets[blob.wso[w] * (int64_t)F];  // host checked: 0 <= bag <= n_bags
    if (w < K) worker_b[w] = 1.0f / (float)(blob.wso[w + 1] - blob.wso[w]);  // inf for an empty worker: unused
  }
  __syncthreads();
  segsort_setup_body(s_occ, K, nnz, desc, seg_bounds, seg_first, chunk_seg, chunk_begin, chunk_end,
                     max_chunks);
}

// ---------------------------------------------------------------------------------------
// pass step 1: digit histogram of every chunk
// Each thread takes 8 consecutive keys (two 16-byte loads where the run of 8 lies inside the
// chunk) and adds run lengths, not single keys, to the shared histogram: after the first pass
// equal keys sit together, so a hot row costs one shared-memory add per 8 keys instead of
// serialising a warp on one counter.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void hist_add8(uint32_t* sh, const uint32_t (&k)[8], int shift, uint32_t mask) {
  uint32_t cur = (k[0] >> shift) & mask, cnt = 1;
#pragma unroll
  for (int j = 1; j < 8; ++j) {
    const uint32_t d = (k[j] >> shift) & mask;
    if (d == cur) {
      ++cnt;
    } else {
      atomicAdd(&sh[cur], cnt);
      cur = d;
      cnt = 1;
    }
  }
  atomicAdd(&sh[cur], cnt);
}

constexpr int kHistThreads = 512;  // 3 CTAs per SM: all 48 warp slots hold loads in flight

__global__ void __launch_bounds__(kHistThreads, kSortCtasPerSM)
radix_hist_kernel(const uint32_t* __restrict__ keys, int shift, uint32_t mask,
                  const SortDesc* __restrict__ desc, const int64_t* __restrict__ chunk_begin,
                  const int64_t* __restrict__ chunk_end, uint32_t* __restrict__ hist,
                  int64_t check_rows, int32_t* status) {
  const int c = blockIdx.x;
  if (c >= desc->n_chunks) return;
  __shared__ uint32_t sh[kSortMaxBins];
  const int tid = threadIdx.x;
  for (int d = tid; d < kSortMaxBins; d += kHistThreads) sh[d] = 0;
  __syncthreads();
  const int64_t b = chunk_begin[c], e = chunk_end[c];
  const uint32_t limit = check_rows > 0 ? (uint32_t)check_rows : 0xffffffffu;
  uint32_t kmax = 0;
  // groups of 8 keys that start on a 16-byte boundary, whatever the array's own alignment
  const int64_t off = (int64_t)((reinterpret_cast<uintptr_t>(keys) >> 2) & 3);
  const int64_t ab = ((b + off) & ~(int64_t)7) - off;
  constexpr int64_t kStep = (int64_t)kHistThreads * 8;
  for (int64_t base = ab + (int64_t)tid * 8; base < e; base += 2 * kStep) {
    const int64_t base2 = base + kStep;
    const bool full1 = base >= b && base + 8 <= e;
    const bool full2 = base2 >= b && base2 + 8 <= e;
    uint4 x0, x1, y0, y1;
    if (full1) {
      x0 = __ldg(reinterpret_cast<const uint4*>(keys + base));
      x1 = __ldg(reinterpret_cast<const uint4*>(keys + base) + 1);
    }
    if (full2) {
      y0 = __ldg(reinterpret_cast<const uint4*>(keys + base2));
      y1 = __ldg(reinterpret_cast<const uint4*>(keys + base2) + 1);
    }
    if (full1) {
      const uint32_t k[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
      for (int j = 0; j < 8; ++j) kmax = max(kmax, k[j]);
      hist_add8(sh, k, shift, mask);
    } else {
      for (int64_t i = max(base, b); i < min(base + 8, e); ++i) {
        const uint32_t k = __ldg(keys + i);
        kmax = max(kmax, k);
        atomicAdd(&sh[(k >> shift) & mask], 1u);
      }
    }
    if (full2) {
      const uint32_t k[8] = {y0.x, y0.y, y0.z, y0.w, y1.x, y1.y, y1.z, y1.w};
#pragma unroll
      for (int j = 0; j < 8; ++j) kmax = max(kmax, k[j]);
      hist_add8(sh, k, shift, mask);
    } else {
      for (int64_t i = max(base2, b); i < min(base2 + 8, e); ++i) {
        const uint32_t k = __ldg(keys + i);
        kmax = max(kmax, k);
        atomicAdd(&sh[(k >> shift) & mask], 1u);
      }
    }
  }
  if (kmax >= limit && check_rows > 0) set_status(status, ANTDT_ERR_ID_OUT_OF_RANGE);
  __syncthreads();
  for (int d = tid; d < kSortMaxBins; d += kHistThreads) hist[(size_t)c * kSortMaxBins + d] = sh[d];
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
// 512 threads x 8 pairs per tile of 4096.  Phases per tile (a block barrier between each):
// load -> rank inside the warp (match.any + per-warp counters) -> exclusive scan of the
// counters over the warps and over the bins -> reorder the tile in shared memory -> write
// every bin's run to its global slot with consecutive threads.
// ---------------------------------------------------------------------------------------
constexpr int kFoldScanChunks = 128;  // up to this many chunks the scatter scans the counts itself
constexpr int kScatThreads = 512;
constexpr int kScatItems = kSortTile / kScatThreads;  // 8
constexpr int kScatWarps = kScatThreads / 32;         // 16
constexpr size_t kScatSmem = 3 * kSortMaxBins * 4 + kScatWarps * kSortMaxBins * 2 + 2 * kSortTile * 4 + 64;

__global__ void __launch_bounds__(kScatThreads, kSortCtasPerSM)
radix_scatter_kernel(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
                     uint32_t* __restrict__ keys_out, uint32_t* __restrict__ vals_out, int shift,
                     uint32_t mask, const SortDesc* __restrict__ desc,
                     const int32_t* __restrict__ chunk_seg, const int64_t* __restrict__ seg_bounds,
                     const int64_t* __restrict__ chunk_begin, const int64_t* __restrict__ chunk_end,
                     const uint32_t* __restrict__ hist, const uint32_t* __restrict__ bin_base,
                     const int32_t* __restrict__ seg_first) {
  const int c = blockIdx.x;
  if (c >= desc->n_chunks) return;
  extern __shared__ __align__(16) unsigned char scat_smem[];
  uint32_t* gbase = reinterpret_cast<uint32_t*>(scat_smem);  // next global slot of every bin
  uint32_t* bin_start = gbase + kSortMaxBins;                // first slot of every bin in the tile
  uint32_t* bin_cnt = bin_start + kSortMaxBins;              // gbase - bin_start of the current tile
  uint2* spairs = reinterpret_cast<uint2*>(bin_cnt + kSortMaxBins);  // (key, value), 8-byte aligned
  uint32_t* warp_tot = reinterpret_cast<uint32_t*>(spairs + kSortTile);  // [16]
  unsigned short* wh = reinterpret_cast<unsigned short*>(warp_tot + 16);  // [16][512]

  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const unsigned lt = (1u << lane) - 1u;
  const int seg = chunk_seg[c];
  const uint32_t seg_begin = (uint32_t)seg_bounds[seg];
  if (seg_first) {
    // few chunks (a small input): `hist` holds the raw counts and this CTA sums its segment's
    // chunks itself - bin totals, the part before its own chunk, the scan over the bins - which
    // costs a microsecond and saves the scan kernel between the histogram and this one
    const int c0 = seg_first[seg], c1 = seg_first[seg + 1];
    uint32_t pre = 0, tot = 0;
    for (int cc = c0; cc < c1; cc += 4) {
      uint32_t h[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) h[j] = cc + j < c1 ? hist[(size_t)(cc + j) * kSortMaxBins + tid] : 0u;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        pre += cc + j < c ? h[j] : 0u;
        tot += h[j];
      }
    }
    uint32_t incl = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[w] = incl;
    __syncthreads();
    uint32_t wp = 0;
#pragma unroll
    for (int ww = 0; ww < kScatWarps; ++ww) wp += (ww < w) ? warp_tot[ww] : 0u;
    gbase[tid] = seg_begin + (incl - tot + wp) + pre;
    // warp_tot is written again only after the tile loop's barriers (A) and (B)
  } else {
    gbase[tid] = seg_begin + bin_base[(size_t)seg * kSortMaxBins + tid] + hist[(size_t)c * kSortMaxBins + tid];
  }
  unsigned short* my_wh = wh + w * kSortMaxBins;

  const int64_t cb = chunk_begin[c], ce = chunk_end[c];
  for (int64_t pos = cb; pos < ce; pos += kSortTile) {
    const int tile_n = (int)min((int64_t)kSortTile, ce - pos);
    uint32_t k[kScatItems], v[kScatItems];
    unsigned short rank[kScatItems];
    // warp-striped: warp w owns elements [w*256, w*256+256) of the tile, item i of lane l is
    // element w*256 + i*32 + l, so (item, lane) order is element order
    const int wbase = w * (32 * kScatItems) + lane;
#pragma unroll
    for (int i = 0; i < kScatItems; ++i) {
      const int j = wbase + i * 32;
      const bool valid = j < tile_n;
      k[i] = valid ? __ldg(keys_in + pos + j) : 0xffffffffu;
      v[i] = valid ? (vals_in ? __ldg(vals_in + pos + j) : (uint32_t)(pos + j)) : 0u;
    }
    {
      uint32_t* whz = reinterpret_cast<uint32_t*>(wh);
#pragma unroll
      for (int d = 0; d < kScatWarps * kSortMaxBins / 2 / kScatThreads; ++d) whz[tid + d * kScatThreads] = 0;
    }
    __syncthreads();  // (A) also: the previous tile's write-out is over

    // peer masks of all items first (independent, their latencies overlap), counters after
    unsigned pm[kScatItems];
#pragma unroll
    for (int i = 0; i < kScatItems; ++i) {
      const bool valid = wbase + i * 32 < tile_n;
      const uint32_t d = valid ? ((k[i] >> shift) & mask) : (uint32_t)kSortMaxBins;
      pm[i] = __match_any_sync(0xffffffffu, d);
    }
#pragma unroll
    for (int i = 0; i < kScatItems; ++i) {
      const bool valid = wbase + i * 32 < tile_n;
      const uint32_t d = (k[i] >> shift) & mask;
      const unsigned m = pm[i];
      // every peer reads the counter (one broadcast), the first peer then bumps it
      const uint32_t old = valid ? my_wh[d] : 0u;
      __syncwarp();
      if (valid && (m & lt) == 0) my_wh[d] = (unsigned short)(old + __popc(m));
      __syncwarp();
      rank[i] = (unsigned short)(old + __popc(m & lt));
    }
    __syncthreads();  // (B)

    {  // per bin (one per thread): exclusive scan over the warps; bin totals
      uint32_t sum = 0;
#pragma unroll
      for (int ww = 0; ww < kScatWarps; ++ww) {
        const uint32_t t = wh[ww * kSortMaxBins + tid];
        wh[ww * kSortMaxBins + tid] = (unsigned short)sum;
        sum += t;
      }
      // exclusive scan over the 512 bins
      uint32_t incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      if (lane == 31) warp_tot[w] = incl;
      __syncthreads();  // (C)
      uint32_t wp = 0;
#pragma unroll
      for (int ww = 0; ww < kScatWarps; ++ww) wp += (ww < w) ? warp_tot[ww] : 0u;
      const uint32_t bs = incl - sum + wp;
      bin_start[tid] = bs;
      bin_cnt[tid] = gbase[tid] - bs;  // global slot of tile slot j in this bin = j + this
      gbase[tid] += sum;               // for the next tile (only this thread touches its bin)
    }
    __syncthreads();  // (D)

#pragma unroll
    for (int i = 0; i < kScatItems; ++i) {
      if (wbase + i * 32 < tile_n) {
        const uint32_t d = (k[i] >> shift) & mask;
        const uint32_t p = bin_start[d] + my_wh[d] + rank[i];
        spairs[p] = make_uint2(k[i], v[i]);
      }
    }
    __syncthreads();  // (E)

#pragma unroll
    for (int i = 0; i < kScatItems; ++i) {
      const int j = tid + i * kScatThreads;
      if (j < tile_n) {
        const uint2 kv = spairs[j];
        const uint32_t g = bin_cnt[(kv.x >> shift) & mask] + (uint32_t)j;
        keys_out[g] = kv.x;
        vals_out[g] = kv.y;
      }
    }
    // the next tile's barrier (A) orders these reads before the next (D) rewrites bin_cnt
  }
}

// ---------------------------------------------------------------------------------------
// runs of equal keys
// A chunk is cut into kRunStrips 128-aligned strips, one warp each.  count: heads per strip;
// scan: exclusive scan over all strips of all chunks; emit: every warp walks its strip once,
// knowing how many runs start before it.  A lane takes 4 consecutive keys (one 16-byte load), so
// a warp step covers 128 keys = four whole words of the head-bit mask; two steps are in flight.
// No block barrier inside the walks.
// ---------------------------------------------------------------------------------------
constexpr int kRunThreads = 512;
constexpr int kRunStrips = kRunThreads / 32;  // 16

struct Strip { int64_t s0, lo, hi; };  // 128-aligned start, clipped [lo, hi)

__device__ __forceinline__ Strip strip_of(int64_t b, int64_t e, int w) {
  const int64_t ab = b & ~(int64_t)127;
  const int64_t len = (((e - ab) + kRunStrips - 1) / kRunStrips + 127) & ~(int64_t)127;
  Strip st;
  st.s0 = ab + (int64_t)w * len;
  st.lo = max(st.s0, b);
  st.hi = min(e, st.s0 + len);
  return st;
}

// The 4 keys [i, i+4) of a lane (i is a multiple of 4; the key buffers are 16-byte aligned).
// Keys outside [lo, hi) are not loaded.
__device__ __forceinline__ void load4(const uint32_t* __restrict__ keys, int64_t i, const Strip& st,
                                      uint32_t (&k)[4]) {
  if (i >= st.lo && i + 4 <= st.hi) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(keys + i));
    k[0] = v.x; k[1] = v.y; k[2] = v.z; k[3] = v.w;
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j) k[j] = (i + j >= st.lo && i + j < st.hi) ? __ldg(keys + i + j) : 0u;
  }
}

// 4-bit mask: bit j set iff key i+j is inside the strip and starts a run.  prev_k3 is the last
// key of the lane to the left (meaningful when that key lies inside the strip).
__device__ __forceinline__ unsigned heads4(const uint32_t* __restrict__ keys, int64_t i, const Strip& st,
                                           int64_t seg_begin, const uint32_t (&k)[4], uint32_t prev_k3,
                                           int lane) {
  unsigned m = 0;
  uint32_t prev = prev_k3;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int64_t e = i + j;
    if (e >= st.lo && e < st.hi) {
      bool h;
      if (e == seg_begin) h = true;
      else {
        if (e == st.lo || (j == 0 && lane == 0)) prev = __ldg(keys + e - 1);
        h = k[j] != prev;
      }
      m |= h ? (1u << j) : 0u;
    }
    prev = k[j];
  }
  return m;
}

__global__ void __launch_bounds__(kRunThreads)
runs_count_kernel(const uint32_t* __restrict__ keys, const SortDesc* __restrict__ desc,
                  const int32_t* __restrict__ chunk_seg, const int64_t* __restrict__ seg_bounds,
                  const int64_t* __restrict__ chunk_begin, const int64_t* __restrict__ chunk_end,
                  int64_t* __restrict__ strip_runs) {
  const int c = blockIdx.x;
  if (c >= desc->n_chunks) return;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const Strip st = strip_of(chunk_begin[c], chunk_end[c], w);
  const int64_t seg_begin = seg_bounds[chunk_seg[c]];
  int cnt = 0;
  for (int64_t j0 = st.s0; j0 < st.hi; j0 += 256) {
    uint32_t ka[4], kb[4];
    const int64_t ia = j0 + lane * 4, ib = ia + 128;
    load4(keys, ia, st, ka);
    load4(keys, ib, st, kb);
    const uint32_t pa = __shfl_up_sync(0xffffffffu, ka[3], 1);
    const uint32_t pb = __shfl_up_sync(0xffffffffu, kb[3], 1);
    cnt += __popc(heads4(keys, ia, st, seg_begin, ka, pa, lane));
    cnt += __popc(heads4(keys, ib, st, seg_begin, kb, pb, lane));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) cnt += __shfl_down_sync(0xffffffffu, cnt, o);
  if (lane == 0) strip_runs[(size_t)c * kRunStrips + w] = cnt;
}

__global__ void __launch_bounds__(1024)
runs_scan_kernel(const SortDesc* __restrict__ desc, const int32_t* __restrict__ seg_first,
                 int64_t* strip_runs, int64_t* seg_runs, int64_t* n_runs_out, int64_t* run_start,
                 int64_t out_cap, int32_t* status) {
  __shared__ int64_t warp_tot[32];
  __shared__ int64_t total;
  const int n = desc->n_chunks * kRunStrips;
  const int tid = threadIdx.x;
  const int per = (n + 1023) / 1024;  // consecutive strips per thread
  const int c0 = tid * per, c1 = min(n, c0 + per);
  int64_t mine = 0;
  for (int c = c0; c < c1; ++c) mine += strip_runs[c];
  int64_t excl = block_exclusive_scan_1024(mine, &total, warp_tot);
  for (int c = c0; c < c1; ++c) {
    const int64_t t = strip_runs[c];
    strip_runs[c] = excl;
    excl += t;
  }
  __syncthreads();
  if (tid == 0) {
    strip_runs[n] = total;
    if (n_runs_out) *n_runs_out = total;
    run_start[total < out_cap ? total : out_cap] = desc->n;
    if (total > out_cap) set_status(status, ANTDT_ERR_CAPACITY);
  }
  __syncthreads();
  if (seg_runs)
    for (int s = tid; s <= desc->n_segments; s += blockDim.x)
      seg_runs[s] = strip_runs[(size_t)seg_first[s] * kRunStrips];
}

// One warp step of the emit walk: the 128 keys [i0, i0+128), 4 per lane.
__device__ __forceinline__ void emit_step(const uint32_t* __restrict__ keys, int64_t i0, const Strip& st,
                                          int64_t b, int64_t e, int64_t seg_begin, const uint32_t (&k)[4],
                                          int lane, int64_t& running, int32_t* __restrict__ uniq_keys,
                                          int64_t* __restrict__ run_start, int64_t out_cap,
                                          uint32_t* head_bits, int32_t* __restrict__ tile_first,
                                          int tile_shift) {
  const int64_t i = i0 + lane * 4;
  const uint32_t prev = __shfl_up_sync(0xffffffffu, k[3], 1);
  const unsigned m = heads4(keys, i, st, seg_begin, k, prev, lane);
  // heads in the lanes to the left: inclusive warp scan of the per-lane counts
  const int mine = __popc(m);
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  int64_t r = running + (incl - mine);  // runs that start before this lane's first key
  if (tile_first && i >= st.lo && i < st.hi && (i & (((int64_t)1 << tile_shift) - 1)) == 0)
    tile_first[i >> tile_shift] = (int32_t)(r + (m & 1u) - 1);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if ((m >> j) & 1u) {
      if (r < out_cap) {
        uniq_keys[r] = (int32_t)k[j];
        run_start[r] = i + j;
      }
      ++r;
    }
  }
  if (head_bits) {
    // 8 lanes make one 32-bit word of the mask; words inside the chunk are stored whole, the
    // chunk's first and last word (shared with a neighbour) are merged with an atomic OR
    unsigned word = m << ((lane & 7) * 4);
    word |= __shfl_xor_sync(0xffffffffu, word, 1);
    word |= __shfl_xor_sync(0xffffffffu, word, 2);
    word |= __shfl_xor_sync(0xffffffffu, word, 4);
    if ((lane & 7) == 0 && word) {
      const int64_t w0 = i0 + (lane >> 3) * 32;
      if (w0 >= b && w0 + 32 <= e) head_bits[w0 >> 5] = word;
      else atomicOr(&head_bits[w0 >> 5], word);
    }
  }
  running += __shfl_sync(0xffffffffu, incl, 31);
}

__global__ void __launch_bounds__(kRunThreads)
runs_emit_kernel(const uint32_t* __restrict__ keys, const SortDesc* __restrict__ desc,
                 const int32_t* __restrict__ chunk_seg, const int64_t* __restrict__ seg_bounds,
                 const int64_t* __restrict__ chunk_begin, const int64_t* __restrict__ chunk_end,
                 const int64_t* __restrict__ strip_runs, int32_t* __restrict__ uniq_keys,
                 int64_t* __restrict__ run_start, int64_t out_cap, uint32_t* head_bits,
                 int32_t* __restrict__ tile_first, int tile_shift) {
  const int c = blockIdx.x;
  if (c >= desc->n_chunks) return;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int64_t b = chunk_begin[c], e = chunk_end[c];
  const Strip st = strip_of(b, e, w);
  const int64_t seg_begin = seg_bounds[chunk_seg[c]];
  int64_t running = strip_runs[(size_t)c * kRunStrips + w];  // runs that start before this strip
  for (int64_t j0 = st.s0; j0 < st.hi; j0 += 256) {
    uint32_t ka[4], kb[4];
    load4(keys, j0 + lane * 4, st, ka);
    load4(keys, j0 + 128 + lane * 4, st, kb);
    emit_step(keys, j0, st, b, e, seg_begin, ka, lane, running, uniq_keys, run_start, out_cap,
              head_bits, tile_first, tile_shift);
    if (j0 + 128 < st.hi)
      emit_step(keys, j0 + 128, st, b, e, seg_begin, kb, lane, running, uniq_keys, run_start, out_cap,
                head_bits, tile_first, tile_shift);
  }
}

}  // namespace

// =========================================================================================
SortLayout sort_layout(int S) {
  SortLayout L;
  const size_t C = (size_t)kSortChunksTarget + (size_t)S;
  L.max_chunks = (int)C;
  L.n_segments = S;
  size_t o = 0;
  L.desc = o;        o = align_up(o + sizeof(SortDesc));
  L.seg_bounds = o;  o = align_up(o + 8 * ((size_t)S + 1));
  L.seg_first = o;   o = align_up(o + 4 * ((size_t)S + 1));
  L.chunk_seg = o;   o = align_up(o + 4 * C);
  L.chunk_begin = o; o = align_up(o + 8 * C);
  L.chunk_end = o;   o = align_up(o + 8 * C);
  L.hist = o;        o = align_up(o + 4 * C * kSortMaxBins);
  L.bin_base = o;    o = align_up(o + 4 * (size_t)S * kSortMaxBins);
  L.chunk_runs = o;  o = align_up(o + 8 * (C * 16 + 1));
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

bool segsort_setup_workers(const int64_t* wso_host, int K, int F, const int64_t* bag_offsets,
                           int64_t n_bags, int64_t nnz, float* worker_b, char* ws, const SortLayout& L,
                           int32_t* status, cudaStream_t s) {
  if (K > kSetupMaxWorkers) return false;
  WorkerBlob blob;
  for (int i = 0; i <= K; ++i) blob.wso[i] = wso_host[i];
  for (int i = K + 1; i <= kSetupMaxWorkers; ++i) blob.wso[i] = 0;
  ANTDT_LAUNCH("bwd_setup", bwd_setup_kernel, 1, 1024, 0, s, blob, K, F, bag_offsets, n_bags, nnz, worker_b,
               (SortDesc*)(ws + L.desc), (int64_t*)(ws + L.seg_bounds), (int32_t*)(ws + L.seg_first),
               (int32_t*)(ws + L.chunk_seg), (int64_t*)(ws + L.chunk_begin), (int64_t*)(ws + L.chunk_end),
               L.max_chunks, status);
  return true;
}

// Per device, once: opt in to the scatter's 55 KB of dynamic shared memory (3 CTAs per SM).
// Not a stream operation; callers that capture a stream call it before the capture starts.
void segsort_prepare_device() {
  static bool attr_set[64] = {};
  int dev_id = 0;
  cudaGetDevice(&dev_id);
  bool& done = attr_set[dev_id & 63];
  if (done) return;
  cudaFuncSetAttribute(radix_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       (int)kScatSmem);
  cudaFuncSetAttribute(radix_scatter_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                       cudaSharedmemCarveoutMaxShared);
  done = true;
}

// Chunks the set-up can have cut for n_cap elements: a chunk holds at least one tile, and every
// segment may end in a partial one.
static int chunk_bound(int64_t n_cap, const SortLayout& L) {
  const int64_t c = (n_cap > 0 ? n_cap : 0) / kSortTile + L.n_segments + 1;
  return (int)(c < L.max_chunks ? c : L.max_chunks);
}

void segsort_run(const uint32_t* keys_in, const uint32_t* vals_in, uint32_t* keys_out,
                 uint32_t* vals_out, uint32_t* keys_tmp, uint32_t* vals_tmp, int key_bits,
                 int64_t check_rows, int64_t n_cap, char* ws, const SortLayout& L, int32_t* status,
                 cudaStream_t s, bool agg) {
  const SortDesc* desc = (const SortDesc*)(ws + L.desc);
  const int64_t* seg_bounds = (const int64_t*)(ws + L.seg_bounds);
  const int32_t* seg_first = (const int32_t*)(ws + L.seg_first);
  const int32_t* chunk_seg = (const int32_t*)(ws + L.chunk_seg);
  const int64_t* chunk_begin = (const int64_t*)(ws + L.chunk_begin);
  const int64_t* chunk_end = (const int64_t*)(ws + L.chunk_end);
  uint32_t* hist = (uint32_t*)(ws + L.hist);
  uint32_t* bin_base = (uint32_t*)(ws + L.bin_base);
  const int P = sort_passes(key_bits);
  segsort_prepare_device();
  // spread the bits evenly over the passes
  int shift = 0;
  const uint32_t* kin = keys_in;
  const uint32_t* vin = vals_in;
  const int S = L.n_segments;
  for (int p = 0; p < P; ++p) {
    const int bits = (key_bits - shift + (P - p) - 1) / (P - p);
    const uint32_t mask = (1u << bits) - 1u;
    // the last pass lands in the output buffers, the one before in the temporaries, ...
    const bool to_out = ((P - 1 - p) % 2) == 0;
    uint32_t* kout = to_out ? keys_out : keys_tmp;
    uint32_t* vout = to_out ? vals_out : vals_tmp;
    ANTDT_LAUNCH(agg ? "agg_radix_hist" : "radix_hist", radix_hist_kernel, L.max_chunks, kHistThreads, 0, s, kin, shift,
                 mask, desc, chunk_begin, chunk_end, hist, p == 0 ? check_rows : (int64_t)0, status);
    // with few chunks every scatter CTA scans the counts it needs itself (one launch less)
    const bool fold_scan = chunk_bound(n_cap, L) <= kFoldScanChunks;
    if (!fold_scan)
      ANTDT_LAUNCH(agg ? "agg_radix_scan" : "radix_scan", radix_scan_kernel, S, kSortMaxBins, 0, s, desc, seg_first, hist,
                   bin_base);
    ANTDT_LAUNCH(agg ? "agg_radix_scatter" : "radix_scatter", radix_scatter_kernel, L.max_chunks, kScatThreads, kScatSmem, s, kin, vin,
                 kout, vout, shift, mask, desc, chunk_seg, seg_bounds, chunk_begin, chunk_end, hist,
                 bin_base, fold_scan ? seg_first : (const int32_t*)nullptr);
    kin = kout;
    vin = vout;
    shift += bits;
  }
}

void segsort_runs(const uint32_t* sorted_keys, int64_t n_cap, int32_t* uniq_keys,
                  int64_t* run_start, int64_t* seg_runs, int64_t* n_runs_out, int64_t out_cap,
                  uint32_t* head_bits, int32_t* tile_first, int tile, char* ws,
                  const SortLayout& L, int32_t* status, cudaStream_t s, bool agg, bool head_bits_zeroed) {
  const SortDesc* desc = (const SortDesc*)(ws + L.desc);
  const int64_t* seg_bounds = (const int64_t*)(ws + L.seg_bounds);
  const int32_t* seg_first = (const int32_t*)(ws + L.seg_first);
  const int32_t* chunk_seg = (const int32_t*)(ws + L.chunk_seg);
  const int64_t* chunk_begin = (const int64_t*)(ws + L.chunk_begin);
  const int64_t* chunk_end = (const int64_t*)(ws + L.chunk_end);
  int64_t* chunk_runs = (int64_t*)(ws + L.chunk_runs);
  if (head_bits && !head_bits_zeroed) cudaMemsetAsync(head_bits, 0, head_bits_words(n_cap) * 4, s);
  int tile_shift = 0;
  while ((1 << tile_shift) < tile) ++tile_shift;  // tile is a power of two
  ANTDT_LAUNCH(agg ? "agg_runs_count" : "runs_count", runs_count_kernel, L.max_chunks, kRunThreads, 0, s, sorted_keys,
               desc, chunk_seg, seg_bounds, chunk_begin, chunk_end, chunk_runs);
  ANTDT_LAUNCH(agg ? "agg_runs_scan" : "runs_scan", runs_scan_kernel, 1, 1024, 0, s, desc, seg_first, chunk_runs, seg_runs,
               n_runs_out, run_start, out_cap, status);
  ANTDT_LAUNCH(agg ? "agg_runs_emit" : "runs_emit", runs_emit_kernel, L.max_chunks, kRunThreads, 0, s, sorted_keys, desc,
               chunk_seg, seg_bounds, chunk_begin, chunk_end, chunk_runs, uniq_keys, run_start,
               out_cap, head_bits, tile_first, tile_shift);
}

}  // namespace antdt
