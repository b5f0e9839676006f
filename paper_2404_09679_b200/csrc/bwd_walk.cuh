// The worker backward's segmented sum: per (worker, row) run of the sorted occurrences, the sum
// of the d_pooled rows the run's occurrences point at, times 1/b_w.
//
// Work is cut by occurrences, not by runs: a tile is TILE (64; 16 for a small input) consecutive
// sorted occurrences whatever runs they belong to, walked by a group of G lanes that hold one
// 16-byte vector of the row each; the 256/G tiles of a CTA are consecutive and form a stretch.
//
//   walk      A run inside a tile is written out directly.  What a tile holds of a run that crosses
//             its edges stays on chip: the sum before the tile's first run end and the sum after
//             its last one go to shared memory, and after one barrier the tile in which such a run
//             STARTS adds the following tiles' pieces in tile order and writes the row.  Only a
//             run that leaves the stretch touches global partials: the stretch's leading piece
//             (head_part), its trailing piece (tail_part), one flag byte per stretch, and a task
//             (stretch, run index) appended to a list by the stretch in which the run starts.
//   fix-up    one lane group per task: tail piece of its stretch, then the leading pieces of the
//             following stretches until one holds a run end (flags of G stretches are looked at
//             together, the pieces of a span are requested together).
// Every sum has a fixed order (entry order inside a tile, tile order, stretch order): no
// floating-point atomics, bit-reproducible.  The task list is filled with an integer atomic; the
// order of the tasks does not matter, each writes its own row.
//
// The walk is built like a plain gather: eight payloads per lane with two 16-byte loads (the
// lanes of a group read the same addresses, one request), eight row loads in flight, then
// either eight unconditional adds (no run ends in any of the warp's tiles in this span: one
// warp vote, so the branch is uniform and costs no reconvergence) or eight predicated
// add / scale-store / reset steps without a branch.  A tile that is ragged, holds a worker
// boundary or might pass the output capacity takes a compact per-entry loop instead; a warp
// votes once at the start which of the two it runs.
#pragma once
#include "tile_reduce.cuh"

namespace antdt {

template <int VPL>
struct WalkChunk { static constexpr int value = VPL == 1 ? 8 : (VPL == 2 ? 4 : 2); };

// Flag byte of a tile (shared memory) and of a stretch (global): does a run that enters from the
// left end inside; does the first entry start a run.  kNoTile marks a lane group without a tile.
enum : uint8_t { kCloses = 1, kStartsRun = 2, kNoTile = 4 };

// Scratch of the walk beyond the sort's: per stretch a leading and a trailing partial row and a
// flag byte; the task list (word 0: count; task i at words 2+2i, 3+2i: stretch, run index).
struct WalkScratch {
  float* head_part;   // [n_stretches, dim]
  float* tail_part;   // [n_stretches, dim]
  uint8_t* flags;     // [n_stretches]
  int32_t* tasks;     // [2 n_stretches + 4]
  bool tasks_zeroed = false;  // the caller has cleared the list's counter on this stream already
};
inline int walk_tiles_per_stretch(int dim) {  // = lane groups per CTA, see launch_bwd_walk
  const int nvec = dim / 4;
  int g = 1;
  while (g < nvec && g < 32) g <<= 1;
  return kRedThreads / g;
}
inline size_t walk_stretches(int64_t n, int tile, int dim) {
  const int64_t n_tiles = (n + tile - 1) / tile;
  const int tps = walk_tiles_per_stretch(dim);
  return (size_t)((n_tiles + tps - 1) / tps) + 1;
}

// acc += the row `piece` (this lane's vectors of it)
template <int G, int VPL>
__device__ __forceinline__ void add_row(float4 (&acc)[VPL], const float* piece, int lg, int nvec) {
#pragma unroll
  for (int k = 0; k < VPL; ++k) {
    if (lg + k * G < nvec) {
      const float4 x = reinterpret_cast<const float4*>(piece)[lg + k * G];
      acc[k].x += x.x; acc[k].y += x.y; acc[k].z += x.z; acc[k].w += x.w;
    }
  }
}
// row = acc * s
template <int G, int VPL>
__device__ __forceinline__ void put_row(float* row, const float4 (&acc)[VPL], float s, int lg, int nvec) {
#pragma unroll
  for (int k = 0; k < VPL; ++k)
    if (lg + k * G < nvec)
      reinterpret_cast<float4*>(row)[lg + k * G] =
          make_float4(acc[k].x * s, acc[k].y * s, acc[k].z * s, acc[k].w * s);
}

template <int G, int VPL, int TILE>
__global__ void __launch_bounds__(kRedThreads, (VPL == 1 ? 4 : 1))
bwd_walk_kernel(const TileArgs a, const uint32_t* __restrict__ payload,
                const uint32_t* __restrict__ head_bits, const int32_t* __restrict__ tile_first,
                const float* __restrict__ rows, float* __restrict__ out, const WalkScratch ws,
                const int payload_vec) {
  constexpr int TPS = kRedThreads / G;  // tiles per stretch
  constexpr int CH = WalkChunk<VPL>::value;
  constexpr unsigned kFull = 0xffffffffu;
  extern __shared__ __align__(16) unsigned char walk_smem[];
  const int dim = a.dim;
  const int K = a.K;
  float* s_headp = reinterpret_cast<float*>(walk_smem);   // [TPS][dim] sum before the first run end
  float* s_carry = s_headp + (size_t)TPS * dim;           // [TPS][dim] sum after the last run end
  int64_t* s_bounds = reinterpret_cast<int64_t*>(s_carry + (size_t)TPS * dim);  // [K+1]
  uint8_t* s_flag = reinterpret_cast<uint8_t*>(s_bounds + (K + 1));             // [TPS]
  for (int i = threadIdx.x; i <= K; i += blockDim.x) s_bounds[i] = a.bounds[i];
  __syncthreads();
  const int64_t n = a.n_host;
  const int lg = threadIdx.x & (G - 1);
  const int grp = threadIdx.x / G;
  const int64_t tile0 = a.tile_begin + (int64_t)blockIdx.x * TPS;  // a multiple of TPS
  const int64_t stretch = tile0 / TPS;
  const int64_t tile = tile0 + grp;
  const int64_t o_begin = tile * TILE;
  const bool in_range = tile < a.tile_end && o_begin < n;
  const int nvec = dim / 4;
  const uint32_t row_stride = (uint32_t)dim;
  const uint32_t last_row = (uint32_t)(a.payload_limit - 1);
  float* my_headp = s_headp + (size_t)grp * dim;

  // run heads of positions o_begin .. o_begin+TILE; entry r closes its run iff r+1 is a head
  uint64_t ends = 0;
  bool open_tail = false, started = false, last_tile = false;
  int nv = 0, w = 0;
  int64_t u = 0;
  if (in_range) {
    nv = (int)min((int64_t)TILE, n - o_begin);
    const uint32_t* hw = head_bits + (o_begin >> 5);
    last_tile = o_begin + TILE >= n;
    if (TILE == 64) {
      const uint32_t h0 = __ldg(hw), h1 = __ldg(hw + 1), h2 = __ldg(hw + 2);
      const uint64_t heads = (uint64_t)h0 | ((uint64_t)h1 << 32);
      ends = (heads >> 1) | ((uint64_t)(h2 & 1u) << 63);
      open_tail = !last_tile && !(h2 & 1u);
      started = (h0 & 1u) != 0;
    } else {  // TILE < 32 and a power of two: the tile's bits and the next one lie in two words
      const uint64_t heads = ((uint64_t)__ldg(hw) | ((uint64_t)__ldg(hw + 1) << 32)) >> (o_begin & 31);
      ends = (heads >> 1) & ((1ull << (TILE & 63)) - 1ull);
      open_tail = !last_tile && !((heads >> (TILE & 63)) & 1ull);
      started = (heads & 1ull) != 0;
    }
    if (last_tile) ends = (ends & ((1ull << (nv - 1)) - 1ull)) | (1ull << (nv - 1));  // array end closes
    u = tile_first[tile];
    w = interval_of(s_bounds, K + 1, o_begin);
    if (w > K - 1) w = K - 1;
  }
  const bool closes = ends != 0ull;
  // the plain walk needs: a whole tile, one worker, every run index below the capacity
  const bool plain = in_range && !last_tile && (w == K - 1 || s_bounds[w + 1] >= o_begin + TILE) &&
                     u + (int64_t)__popcll(ends) < a.out_cap;

  int vi_c[VPL];
#pragma unroll
  for (int k = 0; k < VPL; ++k) vi_c[k] = min(lg + k * G, nvec - 1);  // idle lanes re-read the last vector
  float4 acc[VPL];
#pragma unroll
  for (int k = 0; k < VPL; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
  float inv = in_range ? a.scales[w] : 0.f;

  if (__all_sync(kFull, !in_range)) {
    // nothing to walk in this warp; it still joins the stretch's barrier below
  } else if (__all_sync(kFull, plain || !in_range)) {
    // ---- plain walk (groups without a tile run along with empty masks and store nothing; they
    // read the array's first tile, which exists because a whole tile lies before this warp's) ----
    float sc = started ? inv : 1.f;
    // where the run that is open now goes when it closes; where the one after it goes
    float* dst = started ? out + (size_t)u * row_stride : my_headp;
    float* nxt = out + (size_t)(u + 1) * row_stride;
    const uint32_t* pp = payload + (in_range ? o_begin : 0);
#pragma unroll 1
    for (int c = 0; c < TILE / CH; ++c) {
      uint32_t p[CH];
      if (CH >= 4 && payload_vec) {  // 16-byte aligned: the tile starts on a multiple of 16 entries
#pragma unroll
        for (int t = 0; t + 3 < CH; t += 4) {
          const uint4 q = __ldg(reinterpret_cast<const uint4*>(pp + c * CH + t));
          p[t] = q.x; p[t + 1] = q.y; p[t + 2] = q.z; p[t + 3] = q.w;
        }
      } else {
#pragma unroll
        for (int t = 0; t < CH; ++t) p[t] = __ldg(pp + c * CH + t);
      }
      float4 v[CH][VPL];
#pragma unroll
      for (int t = 0; t < CH; ++t) {
        const float* rp = rows + (size_t)min(p[t], last_row) * row_stride;
#pragma unroll
        for (int k = 0; k < VPL; ++k) v[t][k] = ldg_f4(rp + 4 * vi_c[k]);
      }
      const uint32_t e = in_range ? (uint32_t)(ends & ((1u << CH) - 1u)) : 0u;
      ends >>= CH;
      if (!__any_sync(kFull, e != 0u)) {
#pragma unroll
        for (int t = 0; t < CH; ++t) {
#pragma unroll
          for (int k = 0; k < VPL; ++k) {
            acc[k].x += v[t][k].x; acc[k].y += v[t][k].y;
            acc[k].z += v[t][k].z; acc[k].w += v[t][k].w;
          }
        }
        continue;
      }
#pragma unroll
      for (int t = 0; t < CH; ++t) {
        const bool close = (e >> t) & 1u;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          acc[k].x += v[t][k].x; acc[k].y += v[t][k].y;
          acc[k].z += v[t][k].z; acc[k].w += v[t][k].w;
          if (close && lg + k * G < nvec)
            reinterpret_cast<float4*>(dst)[lg + k * G] =
                make_float4(acc[k].x * sc, acc[k].y * sc, acc[k].z * sc, acc[k].w * sc);
          acc[k].x = close ? 0.f : acc[k].x; acc[k].y = close ? 0.f : acc[k].y;
          acc[k].z = close ? 0.f : acc[k].z; acc[k].w = close ? 0.f : acc[k].w;
        }
        dst = close ? nxt : dst;
        nxt = close ? nxt + row_stride : nxt;
        sc = close ? inv : sc;
        u += close ? 1 : 0;
      }
    }
  } else if (in_range) {
    // ---- per-entry walk of the few tiles that are ragged, span workers or may pass the capacity ----
    bool closed_any = false;
#pragma unroll 1
    for (int r = 0; r < nv; ++r) {
      const uint32_t p = min(__ldg(payload + o_begin + r), last_row);
      add_row<G, VPL>(acc, rows + (size_t)p * row_stride, lg, nvec);
      if (!((ends >> r) & 1ull)) continue;
      if (started || closed_any) {
        const int64_t o = o_begin + r;  // the run's worker is the worker of any of its entries
        while (w < K - 1 && o >= s_bounds[w + 1]) ++w;
        if (u < a.out_cap) put_row<G, VPL>(out + (size_t)u * row_stride, acc, a.scales[w], lg, nvec);
      } else {
        put_row<G, VPL>(my_headp, acc, 1.f, lg, nvec);
      }
#pragma unroll
      for (int k = 0; k < VPL; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      ++u;
      closed_any = true;
    }
    if (open_tail) {  // the worker of the run that stays open: that of the tile's last entry
      const int64_t o = o_begin + nv - 1;
      while (w < K - 1 && o >= s_bounds[w + 1]) ++w;
      inv = a.scales[w];
    }
  }

  // ---- the stretch: pieces of runs that cross tile edges meet in shared memory ----
  // A tile that a run enters from the left holds of it: the sum up to its first run end (headp)
  // if it has one - the run ends there - else all of itself (carry), and the run goes on.
  if (in_range && open_tail) put_row<G, VPL>(s_carry + (size_t)grp * dim, acc, 1.f, lg, nvec);
  if (lg == 0)
    s_flag[grp] = in_range ? (uint8_t)((closes ? kCloses : 0) | (started ? kStartsRun : 0)) : (uint8_t)kNoTile;
  __syncthreads();
  if (!in_range) return;
  if (grp == 0) {
    // the stretch's own record: its flag byte and, if a run enters it, that run's piece in it
    bool any_close = false;
    float4 tot[VPL];
#pragma unroll
    for (int k = 0; k < VPL; ++k) tot[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int g = 0; g < TPS; ++g) {
      const uint8_t f = s_flag[g];
      if (f & kNoTile) break;
      if (!started) add_row<G, VPL>(tot, ((f & kCloses) ? s_headp : s_carry) + (size_t)g * dim, lg, nvec);
      if (f & kCloses) { any_close = true; break; }
    }
    if (!started) put_row<G, VPL>(ws.head_part + (size_t)stretch * dim, tot, 1.f, lg, nvec);
    if (lg == 0) ws.flags[stretch] = (uint8_t)((any_close ? kCloses : 0) | (started ? kStartsRun : 0));
  }
  if (open_tail && (started || closes)) {
    // the run that is open at this tile's end started here: collect what follows
    bool done = false;
    for (int g = grp + 1; g < TPS && !done; ++g) {
      const uint8_t f = s_flag[g];
      if (f & kNoTile) break;
      add_row<G, VPL>(acc, ((f & kCloses) ? s_headp : s_carry) + (size_t)g * dim, lg, nvec);
      done = (f & kCloses) != 0;
    }
    if (done) {
      if (u < a.out_cap) put_row<G, VPL>(out + (size_t)u * row_stride, acc, inv, lg, nvec);
    } else {  // it leaves the stretch
      put_row<G, VPL>(ws.tail_part + (size_t)stretch * dim, acc, 1.f, lg, nvec);
      if (lg == 0 && u < a.out_cap) {
        const int slot = atomicAdd(ws.tasks, 1);
        ws.tasks[2 + 2 * (size_t)slot] = (int32_t)stretch;
        ws.tasks[3 + 2 * (size_t)slot] = (int32_t)u;
      }
    }
  }
}

// Fix-up: one lane group per task, see the head of this file.
template <int G, int VPL, int TILE>
__global__ void __launch_bounds__(kRedThreads)
bwd_fixup_kernel(const TileArgs a, const WalkScratch ws) {
  constexpr int TPS = kRedThreads / G;
  constexpr int64_t SPAN = (int64_t)TPS * TILE;  // entries of a stretch
  const int n_tasks = ws.tasks[0];
  const int64_t n = a.n_host;
  const int64_t last = (n - 1) / SPAN;  // the last stretch; n >= 1 here
  const int lg = threadIdx.x & (G - 1);
  const int glane0 = (threadIdx.x & 31) & ~(G - 1);  // first lane of this group in its warp
  const unsigned gmask = group_mask<G>();
  const int dim = a.dim;
  const int nvec = dim / 4;
  const int groups = gridDim.x * TPS;
  for (int t = blockIdx.x * TPS + threadIdx.x / G; t < n_tasks; t += groups) {
    const int64_t s0 = ws.tasks[2 + 2 * (size_t)t];
    const int64_t u = ws.tasks[3 + 2 * (size_t)t];
    float4 tot[VPL];
#pragma unroll
    for (int k = 0; k < VPL; ++k) tot[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    add_row<G, VPL>(tot, ws.tail_part + (size_t)s0 * dim, lg, nvec);
    int w = interval_of(a.bounds, a.K + 1, min(n, (s0 + 1) * SPAN) - 1);  // worker of the run's entries
    if (w > a.K - 1) w = a.K - 1;
    const float scale = a.scales[w];
    int64_t j = s0 + 1;  // next stretch whose leading piece may belong to the run
    for (;;) {
      // lane l: does the run stop in stretch j+l?  (a run end inside it; the last stretch has one)
      const int64_t mine = j + lg;
      const uint8_t f = mine <= last ? ws.flags[mine] : (uint8_t)(kCloses | kStartsRun);
      const unsigned stops = (__ballot_sync(gmask, (f & kCloses) != 0) >> glane0) &
                             ((G == 32) ? 0xffffffffu : ((1u << (G & 31)) - 1u));
      const int fs = stops ? __ffs((int)stops) - 1 : G;  // stretches j .. j+fs-1 lie inside the run
      const int f_end = __shfl_sync(gmask, (int)f, fs < G ? fs : 0, G);
      const int take = fs + ((fs < G && !(f_end & kStartsRun)) ? 1 : 0);  // pieces to add, in order
      for (int i0 = 0; i0 < take; i0 += 4) {
        float4 x[4][VPL];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int k = 0; k < VPL; ++k) {
            const int vi = lg + k * G;
            x[i][k] = (i0 + i < take && vi < nvec)
                          ? reinterpret_cast<const float4*>(ws.head_part + (size_t)(j + i0 + i) * dim)[vi]
                          : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int k = 0; k < VPL; ++k) {
            if (i0 + i < take) {
              tot[k].x += x[i][k].x; tot[k].y += x[i][k].y; tot[k].z += x[i][k].z; tot[k].w += x[i][k].w;
            }
          }
      }
      if (fs < G) break;
      j += G;
    }
    if (u < a.out_cap) put_row<G, VPL>(a.out + (size_t)u * dim, tot, scale, lg, nvec);
  }
}

template <int G, int VPL, int TILE>
void launch_bwd_walk_t(const TileArgs& a_in, const WalkScratch& ws, const char* name_tiles,
                       const char* name_fixup, cudaStream_t s) {
  constexpr int TPS = kRedThreads / G;
  const int64_t n_tiles = (a_in.n_host + TILE - 1) / TILE;
  TileArgs a = a_in;
  if (a.tile_begin < 0) a.tile_begin = 0;
  if (a.tile_end < 0 || a.tile_end > n_tiles) a.tile_end = n_tiles;
  a.tile_begin = a.tile_begin / TPS * TPS;  // a launch covers whole stretches (callers cut there)
  const size_t smem = 2 * (size_t)TPS * a.dim * 4 + 8 * ((size_t)a.K + 1) + TPS;
  if (smem > 48 * 1024) {  // rows of 1024 floats: more than the default dynamic shared memory
    static bool attr_set[64] = {};
    int dev_id = 0;
    cudaGetDevice(&dev_id);
    if (!attr_set[dev_id & 63]) {
      cudaFuncSetAttribute(bwd_walk_kernel<G, VPL, TILE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)(2 * (size_t)TPS * 1024 * 4 + 8 * ((size_t)kMaxSegments + 1) + TPS));
      attr_set[dev_id & 63] = true;
    }
  }
  if (a.walk && a.tile_end > a.tile_begin) {
    if (a.tile_begin == 0 && !ws.tasks_zeroed) cudaMemsetAsync(ws.tasks, 0, 8, s);  // a new list
    const unsigned grid = (unsigned)((a.tile_end - a.tile_begin + TPS - 1) / TPS);
    const int vec = aligned16(a.payload) ? 1 : 0;
    ANTDT_LAUNCH(name_tiles, (bwd_walk_kernel<G, VPL, TILE>), grid, kRedThreads, smem, s, a, a.payload,
                 a.head_bits, a.tile_first, a.rows, a.out, ws, vec);
  }
  if (a.fixup && n_tiles > TPS) {
    const int64_t want = ((n_tiles + TPS - 1) / TPS + TPS - 1) / TPS;
    const unsigned grid = (unsigned)(want < 8 * kNumSM ? want : 8 * kNumSM);
    ANTDT_LAUNCH(name_fixup, (bwd_fixup_kernel<G, VPL, TILE>), grid, kRedThreads, 0, s, a, ws);
  }
}

template <int G, int VPL>
void launch_bwd_walk_gv(const TileArgs& a, const WalkScratch& ws, const char* nt, const char* nf,
                        cudaStream_t s) {
  if (a.tile == kRedTileSmall) launch_bwd_walk_t<G, VPL, kRedTileSmall>(a, ws, nt, nf, s);
  else launch_bwd_walk_t<G, VPL, kRedTile>(a, ws, nt, nf, s);
}

// The lane-group width chosen here is what walk_tiles_per_stretch assumes.
inline void launch_bwd_walk(const TileArgs& a, const WalkScratch& ws, const char* nt, const char* nf,
                            cudaStream_t s) {
  const int nvec = a.dim / 4;
#define WALK_CASE(G, VPL) launch_bwd_walk_gv<G, VPL>(a, ws, nt, nf, s)
  if (nvec <= 1) WALK_CASE(1, 1);
  else if (nvec <= 2) WALK_CASE(2, 1);
  else if (nvec <= 4) WALK_CASE(4, 1);
  else if (nvec <= 8) WALK_CASE(8, 1);
  else if (nvec <= 16) WALK_CASE(16, 1);
  else if (nvec <= 32) WALK_CASE(32, 1);
  else if (nvec <= 64) WALK_CASE(32, 2);
  else if (nvec <= 128) WALK_CASE(32, 4);
  else WALK_CASE(32, 8);
#undef WALK_CASE
}

}  // namespace antdt
