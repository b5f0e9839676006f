// Tile-parallel segmented reduction of gathered rows for the server aggregation: the weighted sum
// of the workers' gradient rows per aggregated row.  (The worker backward has its own walk,
// bwd_walk.cuh, built on the same tiles.)
//
// The merge-order array of payloads (row indices into `rows`) is cut into tiles of 64 (16 for a
// small input) consecutive entries whatever runs they belong to, so the work is balanced by
// entries, not by runs.  A group of G lanes (one 16-byte vector of the row per lane and VPL step)
// walks one tile; a run that starts and ends inside the tile is written out, the pieces of runs
// that cross the tile's edges go to head_part / tail_part, and the fix-up pass lets the tile where
// such a run STARTS add its tail piece and the following head pieces in tile order.  Every sum has
// a fixed order (ascending worker inside a row): no floating-point atomics, bit-reproducible.
//
// The payloads of G entries live in one register per lane and are broadcast by shuffle,
// kRedUnroll row loads are in flight before the first add, slots without data are predicated off,
// and every entry carries its worker's weight (found by a search of the position in the workers'
// offsets, done once per lane and broadcast).
#pragma once
#include "common.cuh"

namespace antdt {

constexpr int kRedTile = 64;       // sorted entries per reduction tile of a large input
constexpr int kRedTileSmall = 16;  // ... of a small one: a tile is walked serially, so a small input
                                   // needs short tiles to fill the machine and to end soon
constexpr int64_t kRedSmallN = (int64_t)1 << 20;
// Tile length for an input of at most n entries (n: the host-side bound the launch is sized by).
inline int red_tile_for(int64_t n) { return n <= kRedSmallN ? kRedTileSmall : kRedTile; }
constexpr int kRedThreads = 256;
constexpr int kRedUnroll = 4;

struct TileArgs {
  const uint32_t* payload;    // [n] sorted payloads: row index into `rows`
  const uint32_t* head_bits;  // bit i set iff entry i starts a run
  const int32_t* tile_first;  // run index of entry t*tile
  int tile;                   // red_tile_for(n_host)
  const float* rows;          // gathered matrix [payload_limit, dim]
  int dim;
  int64_t n_host;             // entries (upper bound when n_dev is given)
  const int64_t* n_dev;       // device-side entry count or nullptr
  int64_t payload_limit;      // rows of the matrix (>= 1); a payload >= this reads the last row
  const int64_t* bounds;      // backward walk: entry range of every worker [K+1];
                              // aggregation: payload range of every worker [K+1]
  const float* scales;        // backward walk: 1/b_w [K]; aggregation: weight w_i [K]
  int K;
  int64_t out_cap;
  float* out;                 // [out_cap, dim]
  float* head_part;           // [n_tiles, dim]   (aggregation; the backward walk has its own scratch)
  float* tail_part;           // [n_tiles, dim]
  // Which part of the work a launch_tile_reduce call issues (defaults: everything).  A caller
  // whose `rows` arrive in pieces walks the tiles piece by piece and runs the fix-up last.
  int64_t tile_begin = 0;     // first tile of the walk
  int64_t tile_end = -1;      // one past its last tile; -1: to the end
  bool walk = true;           // issue the tile walk over [tile_begin, tile_end)
  bool fixup = true;          // issue the fix-up pass (over all tiles)
};

// The hot pointers are separate __restrict__ parameters (not read through the struct) so that
// the compiler may move row loads across the run-end stores.
template <int G, int VPL, int TILE>
__global__ void __launch_bounds__(kRedThreads, (VPL == 1 ? 6 : 1))
tile_reduce_kernel(const TileArgs a, const uint32_t* __restrict__ payload,
                   const uint32_t* __restrict__ head_bits, const int32_t* __restrict__ tile_first,
                   const float* __restrict__ rows, float* __restrict__ out,
                   float* __restrict__ head_part, float* __restrict__ tail_part) {
  extern __shared__ int64_t s_bounds[];  // payload range of every worker [K+1], then K weights
  float* s_w = reinterpret_cast<float*>(s_bounds + (a.K + 1));
  const int K = a.K;
  for (int i = threadIdx.x; i <= K; i += blockDim.x) s_bounds[i] = a.bounds[i];
  for (int i = threadIdx.x; i < K; i += blockDim.x) s_w[i] = a.scales[i];
  __syncthreads();
  const int64_t n = a.n_dev ? min(*a.n_dev, a.n_host) : a.n_host;
  const int lg = threadIdx.x & (G - 1);
  const int64_t tile = a.tile_begin + (int64_t)blockIdx.x * (kRedThreads / G) + threadIdx.x / G;
  const int64_t o_begin = tile * TILE;
  if (tile >= a.tile_end || o_begin >= n) return;
  const int nv = (int)min((int64_t)TILE, n - o_begin);  // entries in this tile
  const unsigned gmask = group_mask<G>();
  const int dim = a.dim;
  const int nvec = dim / 4;
  constexpr int U = (G < kRedUnroll) ? G : kRedUnroll;

  // run heads of positions o_begin .. o_begin+TILE; entry r closes its run iff r+1 is a head
  const uint32_t* hw = head_bits + (o_begin >> 5);
  const bool last_tile = o_begin + TILE >= n;
  uint64_t ends;
  bool open_tail, started;
  if (TILE == 64) {
    const uint32_t h0 = __ldg(hw), h1 = __ldg(hw + 1), h2 = __ldg(hw + 2);
    const uint64_t heads = (uint64_t)h0 | ((uint64_t)h1 << 32);
    ends = (heads >> 1) | ((uint64_t)(h2 & 1u) << 63);
    open_tail = !last_tile && !(h2 & 1u);  // the last run goes on in the next tile
    started = (h0 & 1u) != 0;
  } else {  // TILE < 32 and a power of two: the tile's bits and the next one lie in two words
    const uint64_t heads = ((uint64_t)__ldg(hw) | ((uint64_t)__ldg(hw + 1) << 32)) >> (o_begin & 31);
    ends = (heads >> 1) & ((1ull << (TILE & 63)) - 1ull);
    open_tail = !last_tile && !((heads >> (TILE & 63)) & 1ull);
    started = (heads & 1ull) != 0;
  }
  if (last_tile) ends = (ends & ((1ull << (nv - 1)) - 1ull)) | (1ull << (nv - 1));  // array end closes

  int64_t u = tile_first[tile];
  float4 acc[VPL];
#pragma unroll
  for (int k = 0; k < VPL; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
  const uint32_t row_stride = (uint32_t)dim;

  constexpr int GE = G < TILE ? G : TILE;  // entries a group step covers
  for (int q = 0; q * GE < nv; ++q) {
    // slots without data are marked -1 and their loads predicated off
    int my_row = -1;
    float my_wt = 0.f;
    if (lg < GE && q * GE + lg < nv) {
      const uint32_t p = __ldg(payload + o_begin + q * GE + lg);
      my_row = ((int64_t)p < a.payload_limit) ? (int)p : -1;
      if (my_row >= 0) {
        int wl = interval_of(s_bounds, K + 1, (int64_t)p);
        my_wt = s_w[wl > K - 1 ? K - 1 : wl];
      }
    }
#pragma unroll
    for (int j0 = 0; j0 < GE; j0 += U) {
      float4 v[U][VPL];
      float wt[U];
#pragma unroll
      for (int t = 0; t < U; ++t) {
        const int row = __shfl_sync(gmask, my_row, j0 + t, G);
        wt[t] = __shfl_sync(gmask, my_wt, j0 + t, G);
        const float* rp = rows + (size_t)((uint32_t)(row < 0 ? 0 : row)) * row_stride;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          const int vi = lg + k * G;
          v[t][k] = (row >= 0 && vi < nvec) ? ldg_f4(rp + 4 * vi) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
#pragma unroll
      for (int t = 0; t < U; ++t) {
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          acc[k].x = fmaf(wt[t], v[t][k].x, acc[k].x); acc[k].y = fmaf(wt[t], v[t][k].y, acc[k].y);
          acc[k].z = fmaf(wt[t], v[t][k].z, acc[k].z); acc[k].w = fmaf(wt[t], v[t][k].w, acc[k].w);
        }
        if ((ends >> (j0 + t)) & 1ull) {  // this entry closes its run
          float* dst;
          if (started) dst = (u < a.out_cap) ? out + (size_t)u * row_stride : nullptr;
          else dst = head_part + (size_t)tile * row_stride;
          if (dst) {
#pragma unroll
            for (int k = 0; k < VPL; ++k) {
              const int vi = lg + k * G;
              if (vi < nvec) reinterpret_cast<float4*>(dst)[vi] = acc[k];
            }
          }
          ++u;
          started = true;
#pragma unroll
          for (int k = 0; k < VPL; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
    }
    ends >>= GE;
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

// Head bits of the TILE entries from pos (a multiple of TILE), and the single bit at pos.
template <int TILE>
__device__ __forceinline__ uint64_t tile_heads(const uint32_t* __restrict__ hb, int64_t pos) {
  if (TILE == 64) {
    const uint32_t* w = hb + (pos >> 5);
    return (uint64_t)__ldg(w) | ((uint64_t)__ldg(w + 1) << 32);
  }
  return (uint64_t)(__ldg(hb + (pos >> 5)) >> (pos & 31)) & ((1ull << (TILE & 63)) - 1ull);  // inside one word
}
__device__ __forceinline__ bool head_at(const uint32_t* __restrict__ hb, int64_t pos) {
  return ((__ldg(hb + (pos >> 5)) >> (pos & 31)) & 1u) != 0u;
}

// Fix-up: the tile in which a straddling run STARTS owns it.  total = its tail piece, then
// the head pieces of the following tiles in order until the run ends.
template <int G, int VPL, int TILE>
__global__ void __launch_bounds__(kRedThreads)
tile_fixup_kernel(const TileArgs a) {
  const int64_t n = a.n_dev ? min(*a.n_dev, a.n_host) : a.n_host;
  const int lg = threadIdx.x & (G - 1);
  const int64_t tile = (int64_t)blockIdx.x * (kRedThreads / G) + threadIdx.x / G;
  const int64_t o_begin = tile * TILE;
  if (o_begin >= n) return;
  const int64_t o_end = o_begin + TILE;
  if (o_end >= n) return;  // the last tile's runs all end inside it
  const int dim = a.dim;
  const int nvec = dim / 4;
  // The pass is a chain of dependent loads for little data, so everything whose address only
  // depends on the tile index is requested up front: the head bits of this tile and the next
  // (a straddling run nearly always ends there), the run index, this tile's tail piece and the
  // next tile's head piece.  (The mask and the partial arrays reach one tile past the end.)
  const uint64_t cur = tile_heads<TILE>(a.head_bits, o_begin);
  const uint64_t nxt_heads = tile_heads<TILE>(a.head_bits, o_end);
  const bool after = head_at(a.head_bits, o_end + TILE);
  const int32_t first_run = __ldg(a.tile_first + tile);
  float4 tot[VPL], nxt[VPL];
#pragma unroll
  for (int k = 0; k < VPL; ++k) {
    const int vi = lg + k * G;
    const bool in = vi < nvec;
    tot[k] = in ? reinterpret_cast<const float4*>(a.tail_part + (size_t)tile * dim)[vi]
                : make_float4(0.f, 0.f, 0.f, 0.f);
    nxt[k] = in ? reinterpret_cast<const float4*>(a.head_part + (size_t)(tile + 1) * dim)[vi]
                : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  if (nxt_heads & 1ull) return;  // next tile starts a new run: nothing straddles
  const int heads = __popcll(cur);
  if (heads == 0) return;  // the straddling run started earlier: its start tile owns it
  const int64_t u = (int64_t)first_run + heads - ((cur & 1ull) ? 1 : 0);
  if (u >= a.out_cap) return;

#pragma unroll
  for (int k = 0; k < VPL; ++k) {
    tot[k].x += nxt[k].x; tot[k].y += nxt[k].y; tot[k].z += nxt[k].z; tot[k].w += nxt[k].w;
  }
  // does the run go on past tile+1?  (no head inside it nor at the start of the tile after it)
  bool open = o_end + TILE < n && nxt_heads == 0ull && !after;
  for (int64_t t2 = tile + 2; open; ++t2) {
    const int64_t b2 = t2 * TILE;
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
      const int vi = lg + k * G;
      if (vi >= nvec) continue;
      const float4 p = reinterpret_cast<const float4*>(a.head_part + (size_t)t2 * dim)[vi];
      tot[k].x += p.x; tot[k].y += p.y; tot[k].z += p.z; tot[k].w += p.w;
    }
    if (b2 + TILE >= n) break;  // ran to the end of the array
    // a head inside t2, or at the start of the tile after it, ends the run
    if (tile_heads<TILE>(a.head_bits, b2) != 0ull || head_at(a.head_bits, b2 + TILE)) break;
  }
  float* dst = a.out + (size_t)u * dim;
#pragma unroll
  for (int k = 0; k < VPL; ++k) {
    const int vi = lg + k * G;
    if (vi < nvec) reinterpret_cast<float4*>(dst)[vi] = tot[k];
  }
}

template <int G, int VPL, int TILE>
void launch_tile_reduce_t(const TileArgs& a_in, const char* name_tiles, const char* name_fixup,
                          cudaStream_t s) {
  const int64_t n_tiles = (a_in.n_host + TILE - 1) / TILE;
  const int64_t tpb = kRedThreads / G;
  TileArgs a = a_in;
  if (a.tile_begin < 0) a.tile_begin = 0;
  if (a.tile_end < 0 || a.tile_end > n_tiles) a.tile_end = n_tiles;
  const size_t smem = 8 * ((size_t)a.K + 1) + 4 * (size_t)a.K;
  if (a.walk && a.tile_end > a.tile_begin) {
    const unsigned grid = (unsigned)((a.tile_end - a.tile_begin + tpb - 1) / tpb);
    ANTDT_LAUNCH(name_tiles, (tile_reduce_kernel<G, VPL, TILE>), grid, kRedThreads, smem, s, a,
                 a.payload, a.head_bits, a.tile_first, a.rows, a.out, a.head_part, a.tail_part);
  }
  if (a.fixup && n_tiles > 0) {
    const unsigned grid = (unsigned)((n_tiles + tpb - 1) / tpb);
    ANTDT_LAUNCH(name_fixup, (tile_fixup_kernel<G, VPL, TILE>), grid, kRedThreads, 0, s, a);
  }
}

template <int G, int VPL>
void launch_tile_reduce_gv(const TileArgs& a, const char* name_tiles, const char* name_fixup,
                           cudaStream_t s) {
  if (a.tile == kRedTileSmall) launch_tile_reduce_t<G, VPL, kRedTileSmall>(a, name_tiles, name_fixup, s);
  else launch_tile_reduce_t<G, VPL, kRedTile>(a, name_tiles, name_fixup, s);
}

inline void launch_tile_reduce(const TileArgs& a, const char* name_tiles, const char* name_fixup,
                               cudaStream_t s) {
  const int nvec = a.dim / 4;
#define TILE_CASE(G, VPL) launch_tile_reduce_gv<G, VPL>(a, name_tiles, name_fixup, s)
  if (nvec <= 1) TILE_CASE(1, 1);
  else if (nvec <= 2) TILE_CASE(2, 1);
  else if (nvec <= 4) TILE_CASE(4, 1);
  else if (nvec <= 8) TILE_CASE(8, 1);
  else if (nvec <= 16) TILE_CASE(16, 1);
  else if (nvec <= 32) TILE_CASE(32, 1);
  else if (nvec <= 64) TILE_CASE(32, 2);
  else if (nvec <= 128) TILE_CASE(32, 4);
  else TILE_CASE(32, 8);
#undef TILE_CASE
}

}  // namespace antdt
