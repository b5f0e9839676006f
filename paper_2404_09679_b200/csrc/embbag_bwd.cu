// Worker backward: per-worker dedup of row ids and segmented reduction of d_pooled rows to
// the worker's mean row gradients.
//
//   prep      occurrence range of every worker (from bag_offsets), 1/b_w scale, offset checks
//   expand    bag index of every occurrence (the sort's payload)
//   sort      stable radix sort by row id inside each worker's range     (segsort.cu)
//   runs      distinct rows, run starts, head bits, first run of each tile (segsort.cu)
//   reduce    tile-parallel segmented sum of gathered d_pooled rows
//   fixup     rows whose occurrences straddle tiles: ordered sum of the tiles' partials
//
// The reduction is balanced by occurrences, not by rows: a tile is kRedTile consecutive
// sorted occurrences whatever rows they belong to, so a row that holds 20% of a field's
// occurrences costs its tiles no more than anyone else's.  Every sum has a fixed order (inside a
// tile by sorted position, across tiles by tile index), no floating-point atomics anywhere.
#include "segsort.cuh"

namespace antdt {
namespace {

constexpr int kRedTile = 64;  // sorted occurrences per reduction tile (multiple of 32)
constexpr int kRedThreads = 256;
constexpr int kRedUnroll = 4;

size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

struct BwdLayout {
  SortLayout sort;
  size_t sort_ws, wso, occ_bounds, worker_b, keys_a, keys_b, vals_t, head_bits, tile_first,
      head_part, tail_part, bytes;
};

BwdLayout bwd_layout(int64_t nnz, int dim, int K) {
  BwdLayout L;
  L.sort = sort_layout(K);
  const size_t n = (size_t)(nnz > 0 ? nnz : 1);
  const size_t n_tiles = (n + kRedTile - 1) / kRedTile;
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
  L.head_part = o;  o = align_up(o + 4 * n_tiles * (size_t)dim);
  L.tail_part = o;  o = align_up(o + 4 * n_tiles * (size_t)dim);
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
                   uint32_t* __restrict__ occ_bag, int32_t* status) {
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

// ---------------------------------------------------------------------------------------
// Tile reduction.  A group of G lanes (one 16-byte vector of the row per lane and VPL step)
// walks kRedTile = 64 consecutive sorted occurrences, summing gathered d_pooled rows; a run that
// starts and ends inside the tile is written out (times 1/b_w), the pieces of runs that cross
// the tile's edges go to head_part / tail_part for the fix-up pass.
//
// The kernel is issue-bound once a worker's d_pooled slice sits in L2, so the walk is built to
// cost few instructions per occurrence: the tile's run ends are one 64-bit mask consumed with
// constant shifts, the bag indices of G occurrences live in one register per lane and are
// broadcast by shuffle, kRedUnroll row loads are in flight before the first add, and the
// worker (for the 1/b_w scale) is only re-resolved when the walk crosses a worker boundary.
// ---------------------------------------------------------------------------------------
template <int G, int VPL>
__global__ void __launch_bounds__(kRedThreads)
seg_reduce_tiles_kernel(const uint32_t* __restrict__ sorted_occ, const uint32_t* __restrict__ head_bits,
                        const int32_t* __restrict__ tile_first, const float* __restrict__ d_pooled,
                        int dim, int64_t n, int64_t n_bags, const int64_t* __restrict__ occ_bounds,
                        const float* __restrict__ worker_inv, int K, int64_t out_cap,
                        float* __restrict__ uniq_grads, float* __restrict__ head_part,
                        float* __restrict__ tail_part) {
  extern __shared__ int64_t s_bounds[];  // [K+1]
  for (int i = threadIdx.x; i <= K; i += blockDim.x) s_bounds[i] = occ_bounds[i];
  __syncthreads();
  const int lg = threadIdx.x & (G - 1);
  const int64_t tile = (int64_t)blockIdx.x * (kRedThreads / G) + threadIdx.x / G;
  const int64_t o_begin = tile * kRedTile;
  if (o_begin >= n) return;
  const int nv = (int)min((int64_t)kRedTile, n - o_begin);  // occurrences in this tile
  const unsigned gmask = group_mask<G>();
  const int nvec = dim / 4;
  constexpr int U = (G < kRedUnroll) ? G : kRedUnroll;

  // run heads of positions o_begin .. o_begin+64; occurrence r closes its run iff r+1 is a head
  const uint32_t* hw = head_bits + (o_begin >> 5);
  const uint32_t h0 = __ldg(hw), h1 = __ldg(hw + 1), h2 = __ldg(hw + 2);
  const uint64_t heads = (uint64_t)h0 | ((uint64_t)h1 << 32);
  uint64_t ends = (heads >> 1) | ((uint64_t)(h2 & 1u) << 63);
  const bool last_tile = o_begin + kRedTile >= n;
  if (last_tile) ends = (ends & ((1ull << (nv - 1)) - 1ull)) | (1ull << (nv - 1));  // array end closes
  const bool open_tail = !last_tile && !(h2 & 1u);  // the last run goes on in the next tile

  int64_t u = tile_first[tile];
  bool started = (h0 & 1u) != 0;
  int w = interval_of(s_bounds, K + 1, o_begin);
  if (w > K - 1) w = K - 1;
  // tile-relative position at which the next worker starts (beyond the tile: never reached)
  int next_w_rel = (int)min((int64_t)(kRedTile + 1), s_bounds[w + 1] - o_begin);
  float inv = worker_inv[w];

  float4 acc[VPL];
#pragma unroll
  for (int k = 0; k < VPL; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
  const uint32_t row_stride = (uint32_t)dim;

  for (int q = 0; q * G < nv; ++q) {
    int my_bag = -1;
    if (q * G + lg < nv) {
      const uint32_t bg = __ldg(sorted_occ + o_begin + q * G + lg);
      my_bag = ((int64_t)bg < n_bags) ? (int)bg : -1;  // -1: payload of a skipped (malformed) bag
    }
#pragma unroll
    for (int j0 = 0; j0 < G; j0 += U) {
      float4 v[U][VPL];
#pragma unroll
      for (int t = 0; t < U; ++t) {
        const int bag = __shfl_sync(gmask, my_bag, j0 + t, G);
        const float* rp = d_pooled + (size_t)((uint32_t)(bag < 0 ? 0 : bag)) * row_stride;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          const int vi = lg + k * G;
          v[t][k] = (bag >= 0 && vi < nvec) ? ldg_f4(rp + 4 * vi) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
#pragma unroll
      for (int t = 0; t < U; ++t) {
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          acc[k].x += v[t][k].x; acc[k].y += v[t][k].y;
          acc[k].z += v[t][k].z; acc[k].w += v[t][k].w;
        }
        if ((ends >> (j0 + t)) & 1ull) {  // this occurrence closes its run
          float* dst;
          float sc = 1.f;
          if (started) {
            const int rel = q * G + j0 + t;
            if (rel >= next_w_rel) {  // crossed into a later worker's range
              const int64_t o = o_begin + rel;
              while (w < K - 1 && o >= s_bounds[w + 1]) ++w;
              next_w_rel = (int)min((int64_t)(kRedTile + 1), s_bounds[w + 1] - o_begin);
              if (w == K - 1) next_w_rel = kRedTile + 1;
              inv = worker_inv[w];
            }
            sc = inv;
            dst = (u < out_cap) ? uniq_grads + (size_t)u * row_stride : nullptr;
          } else {
            dst = head_part + (size_t)tile * row_stride;
          }
          if (dst) {
#pragma unroll
            for (int k = 0; k < VPL; ++k) {
              const int vi = lg + k * G;
              if (vi < nvec)
                reinterpret_cast<float4*>(dst)[vi] =
                    make_float4(acc[k].x * sc, acc[k].y * sc, acc[k].z * sc, acc[k].w * sc);
            }
          }
          ++u;
          started = true;
#pragma unroll
          for (int k = 0; k < VPL; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
    }
    ends = (G >= 64) ? 0ull : (ends >> (G & 63));
  }
  if (open_tail) {
    float* dst = (started ? tail_part : head_part) + (size_t)tile * row_stride;
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
      const int vi = lg + k * G;
      if (vi < nvec) reinterpret_cast<float4*>(dst)[vi] = acc[k];
    }
  }
}

// Fix-up: the tile in which a straddling run STARTS owns it.  total = its tail piece, then
// the head pieces of the following tiles in order until the run ends.
template <int G, int VPL>
__global__ void __launch_bounds__(kRedThreads)
seg_reduce_fixup_kernel(const uint32_t* __restrict__ head_bits, const int32_t* __restrict__ tile_first,
                        int dim, int64_t n, const int64_t* __restrict__ occ_bounds,
                        const float* __restrict__ worker_inv, int K, int64_t out_cap,
                        float* __restrict__ uniq_grads, const float* __restrict__ head_part,
                        const float* __restrict__ tail_part) {
  const int lg = threadIdx.x & (G - 1);
  const int64_t tile = (int64_t)blockIdx.x * (kRedThreads / G) + threadIdx.x / G;
  const int64_t o_begin = tile * kRedTile;
  if (o_begin >= n) return;
  const int64_t o_end = o_begin + kRedTile;
  if (o_end >= n) return;  // the last tile's runs all end inside it
  const int nvec = dim / 4;
  uint32_t hb[kRedTile / 32 + 1];
#pragma unroll
  for (int i = 0; i <= kRedTile / 32; ++i) hb[i] = __ldg(head_bits + (o_begin >> 5) + i);
  if (hb[kRedTile / 32] & 1u) return;  // next tile starts a new run: nothing straddles
  int heads = 0;
#pragma unroll
  for (int i = 0; i < kRedTile / 32; ++i) heads += __popc(hb[i]);
  if (heads == 0) return;  // the straddling run started earlier: its start tile owns it
  const int64_t u = (int64_t)tile_first[tile] + heads - ((hb[0] & 1u) ? 1 : 0);
  if (u >= out_cap) return;

  float4 tot[VPL];
#pragma unroll
  for (int k = 0; k < VPL; ++k) {
    const int vi = lg + k * G;
    tot[k] = vi < nvec ? reinterpret_cast<const float4*>(tail_part + (size_t)tile * dim)[vi]
                       : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int64_t t2 = tile + 1;; ++t2) {
    const int64_t b2 = t2 * kRedTile;
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
      const int vi = lg + k * G;
      if (vi >= nvec) continue;
      const float4 p = reinterpret_cast<const float4*>(head_part + (size_t)t2 * dim)[vi];
      tot[k].x += p.x; tot[k].y += p.y; tot[k].z += p.z; tot[k].w += p.w;
    }
    if (b2 + kRedTile >= n) break;  // ran to the end of the array
    bool ends = false;              // a head inside t2, or at the start of the tile after it
#pragma unroll
    for (int i = 0; i < kRedTile / 32; ++i) ends |= __ldg(head_bits + (b2 >> 5) + i) != 0u;
    ends |= (__ldg(head_bits + (b2 >> 5) + kRedTile / 32) & 1u) != 0u;
    if (ends) break;
  }
  // worker of the run = worker of any of its occurrences
  int w = interval_of(occ_bounds, K + 1, o_end - 1);
  if (w > K - 1) w = K - 1;
  const float scale = worker_inv[w];
  float* dst = uniq_grads + (size_t)u * dim;
#pragma unroll
  for (int k = 0; k < VPL; ++k) {
    const int vi = lg + k * G;
    if (vi >= nvec) continue;
    float4 r = tot[k];
    r.x *= scale; r.y *= scale; r.z *= scale; r.w *= scale;
    reinterpret_cast<float4*>(dst)[vi] = r;
  }
}

template <int G, int VPL>
void launch_reduce(const BwdLayout& L, char* ws, const uint32_t* sorted_occ, const float* d_pooled,
                   int dim, int64_t nnz, int64_t n_bags, int K, int64_t out_cap, float* uniq_grads,
                   cudaStream_t s) {
  const int64_t n_tiles = (nnz + kRedTile - 1) / kRedTile;
  const int64_t tpb = kRedThreads / G;
  const unsigned grid = (unsigned)((n_tiles + tpb - 1) / tpb);
  const uint32_t* head_bits = (const uint32_t*)(ws + L.head_bits);
  const int32_t* tile_first = (const int32_t*)(ws + L.tile_first);
  const int64_t* occ_bounds = (const int64_t*)(ws + L.sort_ws + L.sort.seg_bounds);
  const float* worker_b = (const float*)(ws + L.worker_b);
  float* head_part = (float*)(ws + L.head_part);
  float* tail_part = (float*)(ws + L.tail_part);
  ANTDT_LAUNCH("seg_reduce_tiles", (seg_reduce_tiles_kernel<G, VPL>), grid, kRedThreads,
               8 * ((size_t)K + 1), s, sorted_occ, head_bits, tile_first, d_pooled, dim, nnz,
               n_bags, occ_bounds, worker_b, K, out_cap, uniq_grads, head_part, tail_part);
  ANTDT_LAUNCH("seg_reduce_fixup", (seg_reduce_fixup_kernel<G, VPL>), grid, kRedThreads, 0, s,
               head_bits, tile_first, dim, nnz, occ_bounds, worker_b, K, out_cap, uniq_grads,
               head_part, tail_part);
}

}  // namespace
}  // namespace antdt

extern "C" size_t antdt_embbag_bwd_dedup_workspace_bytes(int64_t nnz, int64_t n_bags, int32_t dim,
                                                         int32_t n_workers) {
  (void)n_bags;
  if (nnz < 0 || dim < 1 || n_workers < 1 || n_workers > antdt::kMaxSegments) return 0;
  return antdt::bwd_layout(nnz, dim, n_workers).bytes;
}

extern "C" int32_t antdt_embbag_bwd_dedup(
    const int32_t* row_ids, int64_t nnz, const int64_t* bag_offsets, int64_t n_bags,
    int32_t bags_per_sample, const float* d_pooled, int32_t dim, int64_t n_rows, int32_t n_workers,
    const int64_t* worker_sample_offsets, int32_t* uniq_ids, int64_t* worker_uniq_offsets,
    int64_t* seg_offsets, int32_t* sorted_occ, float* uniq_grads, int64_t out_cap, void* ws,
    size_t ws_bytes, int32_t* dev_status, void* stream) {
  using namespace antdt;
  const int K = n_workers;
  if (nnz < 0 || n_bags < 0 || nnz >= (1ll << 31) || n_bags >= (1ll << 31) || n_rows < 1 ||
      n_rows >= (1ll << 31) || dim < 4 || dim > 1024 || dim % 4 || K < 1 || K > kMaxSegments ||
      bags_per_sample < 1 || out_cap < 0)
    return ANTDT_ERR_INVALID_ARG;
  if (!bag_offsets || !worker_sample_offsets || !worker_uniq_offsets || !seg_offsets || !ws)
    return ANTDT_ERR_INVALID_ARG;
  if (nnz > 0 && (!row_ids || !d_pooled || !sorted_occ)) return ANTDT_ERR_INVALID_ARG;
  if (out_cap > 0 && (!uniq_ids || !uniq_grads)) return ANTDT_ERR_INVALID_ARG;
  if (!aligned16(d_pooled) || !aligned16(uniq_grads) || !aligned16(ws)) return ANTDT_ERR_INVALID_ARG;
  if (worker_sample_offsets[0] != 0) return ANTDT_ERR_INVALID_ARG;
  for (int w = 0; w < K; ++w)
    if (worker_sample_offsets[w + 1] < worker_sample_offsets[w]) return ANTDT_ERR_INVALID_ARG;
  if (worker_sample_offsets[K] * (int64_t)bags_per_sample != n_bags) return ANTDT_ERR_INVALID_ARG;
  const BwdLayout L = bwd_layout(nnz, dim, K);
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

  upload_small(worker_sample_offsets, 8 * ((size_t)K + 1), d_wso, s);
  ANTDT_LAUNCH("bwd_prep", bwd_prep_kernel, 1, 1024, 0, s, d_wso, K, (int)bags_per_sample,
               bag_offsets, n_bags, nnz, d_occ_bounds, d_worker_b, dev_status);
  segsort_setup(d_occ_bounds, K, nnz, sort_ws, L.sort, s);

  const int key_bits = bits_for(n_rows);
  const int P = sort_passes(key_bits);
  // payload ping-pong ends in sorted_occ: start in whichever buffer makes the last pass land there
  uint32_t* occ_out = reinterpret_cast<uint32_t*>(sorted_occ);
  uint32_t* expand_to = (P % 2 == 1) ? vals_t : occ_out;
  if (n_bags > 0 && nnz > 0) {
    const unsigned grid = (unsigned)((n_bags + 32 * 8 - 1) / (32 * 8));
    ANTDT_LAUNCH("expand_bags", expand_bags_kernel, grid, 256, 0, s, bag_offsets, n_bags, nnz,
                 expand_to, dev_status);
  }
  segsort_run(reinterpret_cast<const uint32_t*>(row_ids), expand_to, keys_a, occ_out, keys_b,
              vals_t, key_bits, n_rows, sort_ws, L.sort, dev_status, s);
  segsort_runs(keys_a, nnz, uniq_ids, seg_offsets, worker_uniq_offsets, nullptr, out_cap,
               (uint32_t*)(w8 + L.head_bits), (int32_t*)(w8 + L.tile_first), kRedTile, sort_ws,
               L.sort, dev_status, s);
  if (nnz > 0) {
    const int nvec = dim / 4;
#define RED_CASE(G, VPL)                                                                    \
  launch_reduce<G, VPL>(L, w8, occ_out, d_pooled, dim, nnz, n_bags, K, out_cap, uniq_grads, s);
    if (nvec <= 1) { RED_CASE(1, 1) }
    else if (nvec <= 2) { RED_CASE(2, 1) }
    else if (nvec <= 4) { RED_CASE(4, 1) }
    else if (nvec <= 8) { RED_CASE(8, 1) }
    else if (nvec <= 16) { RED_CASE(16, 1) }
    else if (nvec <= 32) { RED_CASE(32, 1) }
    else if (nvec <= 64) { RED_CASE(32, 2) }
    else if (nvec <= 128) { RED_CASE(32, 4) }
    else { RED_CASE(32, 8) }
#undef RED_CASE
  }
  return cuda_ok();
}
