// Worker backward: per-worker dedup of row ids and segmented reduction of d_pooled rows to
// the worker's mean row gradients.
//
//   prep      occurrence range of every worker (from bag_offsets), 1/b_w scale, offset checks
//   expand    bag index of every occurrence (the sort's payload)
//   sort      stable radix sort by row id inside each worker's range     (segsort.cu)
//   runs      distinct rows, run starts, head bits, first run of each tile (segsort.cu)
//   reduce    tile-parallel segmented sum of gathered d_pooled rows        (bwd_walk.cuh)
//   fixup     rows whose occurrences leave a CTA's stretch of tiles: ordered sum of partials
//
// The reduction is balanced by occurrences, not by rows: a tile is 64 (small inputs: 16) consecutive
// sorted occurrences whatever rows they belong to, so a row that holds 20% of a field's
// occurrences costs its tiles no more than anyone else's.  Every sum has a fixed order (inside a
// tile by sorted position, across tiles by tile index), no floating-point atomics anywhere.
#include "segsort.cuh"
#include "bwd_walk.cuh"

namespace antdt {
namespace {

size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

struct BwdLayout {
  SortLayout sort;
  size_t sort_ws, wso, occ_bounds, worker_b, keys_a, keys_b, vals_t, head_bits, tile_first,
      head_part, tail_part, flags, tasks, bytes;
};

BwdLayout bwd_layout(int64_t nnz, int dim, int K, int tile_len) {
  BwdLayout L;
  L.sort = sort_layout(K);
  const size_t n = (size_t)(nnz > 0 ? nnz : 1);
  const size_t tile = (size_t)tile_len;
  const size_t n_tiles = (n + tile - 1) / tile;
  size_t o = 0;
  L.sort_ws = o;    o = align_up(o + L.sort.bytes);
  L.wso = o;        o = align_up(o + 8 * ((size_t)K + 1));
  L.occ_bounds = o; o = align_up(o + 8 * ((size_t)K + 1));
  L.worker_b = o;   o = align_up(o + 4 * (size_t)K);
  L.keys_a = o;     o = align_up(o + 4 * n);
  L.keys_b = o;     o = align_up(o + 4 * n);
  L.vals_t = o;     o = align_up(o + 4 * n);
  L.head_bits = o;  o = align_up(o + 4 * head_bits_words((int64_t)n));
  L.tile_first = o; o = align_up(o + 4 * (n_tiles + 1));
  const size_t n_str = walk_stretches((int64_t)n, tile_len, dim);
  L.head_part = o;  o = align_up(o + 4 * n_str * (size_t)dim);
  L.tail_part = o;  o = align_up(o + 4 * n_str * (size_t)dim);
  L.flags = o;      o = align_up(o + n_str);
  L.tasks = o;      o = align_up(o + 4 * (2 * n_str + 4));
  L.bytes = o;
  return L;
}

// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
bwd_prep_kernel(const int64_t* __restrict__ wso, int K, int F, const int64_t* __restrict__ bag_offsets,
                int64_t n_bags, int64_t nnz, int64_t* __restrict__ occ_bounds,
                float* __restrict__ worker_b, int32_t* status) {
  const int tid = threadIdx.x;
  if (tid == 0 && (bag_offsets[0] != 0 || bag_offsets[n_bags] != nnz))
    set_status(status, ANTDT_ERR_BAD_OFFSETS);
  for (int w = tid; w <= K; w += blockDim.x) {
    const int64_t bag = wso[w] * (int64_t)F;  // host checked: 0 <= bag <= n_bags
    occ_bounds[w] = bag_offsets[bag];          // the sort setup clamps and orders these
    if (w < K) worker_b[w] = 1.0f / (float)(wso[w + 1] - wso[w]);  // 1/b_w (inf for an empty worker: unused)
  }
}

// One warp expands 32 consecutive bags: lane l holds the end offset of bag b0+l, every
// occurrence of the warp's range finds its bag by a 5-step search over the lanes' values.
__global__ void __launch_bounds__(256)
expand_bags_kernel(const int64_t* __restrict__ bag_offsets, int64_t n_bags, int64_t nnz,
                   uint32_t* __restrict__ occ_bag, int32_t* status, uint32_t* __restrict__ zero_words,
                   int64_t n_zero_words, int32_t* __restrict__ zero_pair) {
  // scratch that later kernels of the call expect zeroed (the run heads' bit mask, the fix-up's
  // task counter): cleared here, on the way, instead of by two memsets in the chain of launches
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_zero_words;
       i += (int64_t)gridDim.x * blockDim.x)
    zero_words[i] = 0u;
  if (blockIdx.x == 0 && threadIdx.x < 2 && zero_pair) zero_pair[threadIdx.x] = 0;
  const int lane = threadIdx.x & 31;
  const int64_t b0 = ((int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 32;
  if (b0 >= n_bags) return;
  const int64_t b = min(b0 + lane, n_bags - 1);
  const int64_t lo = bag_offsets[b], hi = bag_offsets[b + 1];
  const bool bad = lo < 0 || hi < lo || hi > nnz;
  if (__any_sync(0xffffffffu, bad)) {  // skip the whole group; readers bound-check bag indices
    if (lane == 0) set_status(status, ANTDT_ERR_BAD_OFFSETS);
    return;
  }
  const int64_t first = __shfl_sync(0xffffffffu, lo, 0);
  const int64_t last = __shfl_sync(0xffffffffu, hi, 31);  // lanes past n_bags repeat the last bag
  const int64_t span = last - first;
  if (span >= (1ll << 31)) return;  // cannot happen: nnz < 2^31
  const int my_end = (int)(hi - first);  // ascending over the lanes
  for (int64_t base = 0; base < span; base += 32) {
    const int o = (int)base + lane;
    // first lane whose end is > o
    int l = 0;
#pragma unroll
    for (int step = 16; step > 0; step >>= 1) {
      const int e = __shfl_sync(0xffffffffu, my_end, l + step - 1);
      if (e <= o) l += step;
    }
    if (o < span) occ_bag[first + o] = (uint32_t)min(b0 + l, n_bags - 1);
  }
}

}  // namespace
}  // namespace antdt

extern "C" size_t antdt_embbag_bwd_dedup_workspace_bytes(int64_t nnz, int64_t n_bags, int32_t dim,
                                                         int32_t n_workers) {
  (void)n_bags;
  if (nnz < 0 || dim < 1 || n_workers < 1 || n_workers > antdt::kMaxSegments) return 0;
  return antdt::bwd_layout(nnz, dim, n_workers, antdt::red_tile_for(nnz)).bytes;
}

extern "C" size_t antdt_embbag_bwd_dedup_min_workspace_bytes(int64_t nnz, int64_t n_bags, int32_t dim,
                                                             int32_t n_workers) {
  (void)n_bags;
  if (nnz < 0 || dim < 1 || n_workers < 1 || n_workers > antdt::kMaxSegments) return 0;
  return antdt::bwd_layout(nnz, dim, n_workers, antdt::kRedTile).bytes;
}

namespace antdt {
// The entry point's body.  d_pooled is first read by the tile reduction; a caller that is still
// copying it in on another stream passes the event that marks its arrival (the sort and the
// run detection, which only need the ids, then overlap the copy).
int32_t bwd_dedup_impl(
    const int32_t* row_ids, int64_t nnz, const int64_t* bag_offsets, int64_t n_bags,
    int32_t bags_per_sample, const float* d_pooled, int32_t dim, int64_t n_rows, int32_t n_workers,
    const int64_t* worker_sample_offsets, int32_t* uniq_ids, int64_t* worker_uniq_offsets,
    int64_t* seg_offsets, int32_t* sorted_occ, float* uniq_grads, int64_t out_cap, void* ws,
    size_t ws_bytes, int32_t* dev_status, void* stream, const PooledArrival* arrival,
    cudaEvent_t ids_done) {
  const int K = n_workers;
  if (nnz < 0 || n_bags < 0 || nnz >= (1ll << 31) || n_bags >= (1ll << 31) || n_rows < 1 ||
      n_rows >= (1ll << 31) || dim < 4 || dim > 1024 || dim % 4 || K < 1 || K > kMaxSegments ||
      bags_per_sample < 1 || out_cap < 0)
    return ANTDT_ERR_INVALID_ARG;
  if (!bag_offsets || !worker_sample_offsets || !worker_uniq_offsets || !seg_offsets || !ws)
    return ANTDT_ERR_INVALID_ARG;
  if (nnz > 0 && (!row_ids || !d_pooled || !sorted_occ)) return ANTDT_ERR_INVALID_ARG;
  if (nnz > 0 && n_bags == 0) return ANTDT_ERR_INVALID_ARG;  // occurrences that belong to no bag
  if (out_cap > 0 && (!uniq_ids || !uniq_grads)) return ANTDT_ERR_INVALID_ARG;
  if (!aligned16(d_pooled) || !aligned16(uniq_grads) || !aligned16(ws)) return ANTDT_ERR_INVALID_ARG;
  if (worker_sample_offsets[0] != 0) return ANTDT_ERR_INVALID_ARG;
  for (int w = 0; w < K; ++w)
    if (worker_sample_offsets[w + 1] < worker_sample_offsets[w]) return ANTDT_ERR_INVALID_ARG;
  if (worker_sample_offsets[K] * (int64_t)bags_per_sample != n_bags) return ANTDT_ERR_INVALID_ARG;
  // short reduction tiles for a small input when the workspace has room for their partial sums,
  // the long tiles (the minimum workspace) otherwise
  int tile_len = red_tile_for(nnz);
  BwdLayout L = bwd_layout(nnz, dim, K, tile_len);
  if (ws_bytes < L.bytes && tile_len != kRedTile) {
    tile_len = kRedTile;
    L = bwd_layout(nnz, dim, K, tile_len);
  }
  if (ws_bytes < L.bytes) return ANTDT_ERR_WORKSPACE_TOO_SMALL;

  cudaStream_t s = (cudaStream_t)stream;
  char* w8 = static_cast<char*>(ws);
  int64_t* d_wso = (int64_t*)(w8 + L.wso);
  int64_t* d_occ_bounds = (int64_t*)(w8 + L.occ_bounds);
  float* d_worker_b = (float*)(w8 + L.worker_b);
  uint32_t* keys_a = (uint32_t*)(w8 + L.keys_a);
  uint32_t* keys_b = (uint32_t*)(w8 + L.keys_b);
  uint32_t* vals_t = (uint32_t*)(w8 + L.vals_t);
  char* sort_ws = w8 + L.sort_ws;

  // one launch for up to 255 workers; beyond that the offsets travel in pieces
  if (!segsort_setup_workers(worker_sample_offsets, K, (int)bags_per_sample, bag_offsets, n_bags, nnz,
                             d_worker_b, sort_ws, L.sort, dev_status, s)) {
    upload_small(worker_sample_offsets, 8 * ((size_t)K + 1), d_wso, s);
    ANTDT_LAUNCH("bwd_prep", bwd_prep_kernel, 1, 1024, 0, s, d_wso, K, (int)bags_per_sample,
                 bag_offsets, n_bags, nnz, d_occ_bounds, d_worker_b, dev_status);
    segsort_setup(d_occ_bounds, K, nnz, sort_ws, L.sort, s);
  }

  const int key_bits = bits_for(n_rows);
  const int P = sort_passes(key_bits);
  // payload ping-pong ends in sorted_occ: start in whichever buffer makes the last pass land there
  uint32_t* occ_out = reinterpret_cast<uint32_t*>(sorted_occ);
  uint32_t* expand_to = (P % 2 == 1) ? vals_t : occ_out;
  bool scratch_zeroed = false;
  if (n_bags > 0 && nnz > 0) {
    const unsigned grid = (unsigned)((n_bags + 32 * 8 - 1) / (32 * 8));
    ANTDT_LAUNCH("expand_bags", expand_bags_kernel, grid, 256, 0, s, bag_offsets, n_bags, nnz,
                 expand_to, dev_status, (uint32_t*)(w8 + L.head_bits), (int64_t)head_bits_words(nnz),
                 (int32_t*)(w8 + L.tasks));
    scratch_zeroed = true;
  }
  segsort_run(reinterpret_cast<const uint32_t*>(row_ids), expand_to, keys_a, occ_out, keys_b,
              vals_t, key_bits, n_rows, nnz, sort_ws, L.sort, dev_status, s);
  segsort_runs(keys_a, nnz, uniq_ids, seg_offsets, worker_uniq_offsets, nullptr, out_cap,
               (uint32_t*)(w8 + L.head_bits), (int32_t*)(w8 + L.tile_first), tile_len, sort_ws,
               L.sort, dev_status, s, false, scratch_zeroed);
  if (ids_done && cudaEventRecord(ids_done, s) != cudaSuccess) return ANTDT_ERR_CUDA;
  if (nnz > 0) {
    TileArgs t;
    t.payload = occ_out;
    t.head_bits = (const uint32_t*)(w8 + L.head_bits);
    t.tile_first = (const int32_t*)(w8 + L.tile_first);
    t.tile = tile_len;
    t.rows = d_pooled;
    t.dim = dim;
    t.n_host = nnz;
    t.n_dev = nullptr;
    t.payload_limit = n_bags;
    t.bounds = (const int64_t*)(sort_ws + L.sort.seg_bounds);  // sanitised worker ranges
    t.scales = d_worker_b;
    t.K = K;
    t.out_cap = out_cap;
    t.out = uniq_grads;
    WalkScratch tasks;
    tasks.head_part = (float*)(w8 + L.head_part);
    tasks.tail_part = (float*)(w8 + L.tail_part);
    tasks.flags = (uint8_t*)(w8 + L.flags);
    tasks.tasks = (int32_t*)(w8 + L.tasks);
    tasks.tasks_zeroed = scratch_zeroed;
    if (!arrival || arrival->n < 1) {
      launch_bwd_walk(t, tasks, "seg_reduce_tiles", "seg_reduce_fixup", s);
    } else {
      // d_pooled is arriving piece by piece: a tile is walked as soon as the piece that holds
      // its last entry is there (the sort and the run detection above needed the ids only)
      const int64_t n_tiles = (nnz + tile_len - 1) / tile_len;
      const int64_t tps = walk_tiles_per_stretch(dim);
      int64_t done = 0;  // tiles issued so far
      t.fixup = false;
      for (int c = 0; c < arrival->n; ++c) {
        if (cudaStreamWaitEvent(s, arrival->ready[c], 0) != cudaSuccess) return ANTDT_ERR_CUDA;
        int64_t upto = n_tiles;  // the last piece takes every remaining tile
        if (c + 1 < arrival->n) {
          const int64_t e = arrival->entry_end[c];
          upto = e <= 0 ? 0 : (e >= nnz ? n_tiles : e / tile_len);  // tiles that end before entry e
          if (upto < n_tiles) upto = upto / tps * tps;              // a launch walks whole stretches
        }
        if (upto <= done) continue;
        t.tile_begin = done;
        t.tile_end = upto;
        launch_bwd_walk(t, tasks, "seg_reduce_tiles", "seg_reduce_fixup", s);
        done = upto;
      }
      t.walk = false;
      t.fixup = true;
      launch_bwd_walk(t, tasks, "seg_reduce_tiles", "seg_reduce_fixup", s);
    }
  }
  return cuda_ok();
}
}  // namespace antdt

extern "C" int32_t antdt_embbag_bwd_dedup(
    const int32_t* row_ids, int64_t nnz, const int64_t* bag_offsets, int64_t n_bags,
    int32_t bags_per_sample, const float* d_pooled, int32_t dim, int64_t n_rows, int32_t n_workers,
    const int64_t* worker_sample_offsets, int32_t* uniq_ids, int64_t* worker_uniq_offsets,
    int64_t* seg_offsets, int32_t* sorted_occ, float* uniq_grads, int64_t out_cap, void* ws,
    size_t ws_bytes, int32_t* dev_status, void* stream) {
  return antdt::bwd_dedup_impl(row_ids, nnz, bag_offsets, n_bags, bags_per_sample, d_pooled, dim,
                               n_rows, n_workers, worker_sample_offsets, uniq_ids,
                               worker_uniq_offsets, seg_offsets, sorted_occ, uniq_grads, out_cap, ws,
                               ws_bytes, dev_status, stream, nullptr);
}
