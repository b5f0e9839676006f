// Server aggregation: batch-size weighted sum of the workers' mean gradients.
//
// Sparse part, up to 32 workers: the range-partitioned merge of agg_range.cu (no sort).
// Sparse part, more workers: the workers' row lists (each ascending) are merged by one stable radix sort of
// (row id, position in the concatenated list); equal rows then sit together in ascending
// worker order, and the tile-parallel segmented reduction (tile_reduce.cuh) forms each row's
// weighted sum of its <= K contributions in that fixed order.  Because the sorted positions of
// one worker ascend with the row id, the gather of the workers' gradient rows is K
// forward-moving streams, not a random walk.
// Dense part: a K-way streaming reduction, one 16-byte vector per thread and worker.
#include "agg_range.cuh"
#include "opt_math.cuh"
#include "segsort.cuh"
#include "tile_reduce.cuh"

namespace antdt {
namespace {

size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

struct AggLayout {
  SortLayout sort;
  RangeLayout range;
  size_t range_ws;
  size_t sort_ws, bounds, weights, wuo, cwuo, drop, keys_a, keys_b, src, vals_t, run_start, head_bits,
      tile_first, head_part, tail_part, row_start, src_worker, bytes;
};

AggLayout agg_layout(int64_t in_cap, int K, int dim) {
  AggLayout L;
  L.sort = sort_layout(1);
  const size_t n = (size_t)(in_cap > 0 ? in_cap : 1);
  size_t o = 0;
  L.sort_ws = o;   o = align_up(o + L.sort.bytes);
  L.bounds = o;    o = align_up(o + 16);
  L.weights = o;   o = align_up(o + 4 * (size_t)K);
  L.wuo = o;       o = align_up(o + 8 * ((size_t)K + 1));
  L.cwuo = o;      o = align_up(o + 8 * ((size_t)K + 1));
  L.drop = o;      o = align_up(o + 4 * (size_t)K);
  L.keys_a = o;    o = align_up(o + 4 * n);
  L.keys_b = o;    o = align_up(o + 4 * n);
  L.src = o;       o = align_up(o + 4 * n);
  L.vals_t = o;    o = align_up(o + 4 * n);
  L.run_start = o; o = align_up(o + 8 * (n + 1));
  const size_t tile = (size_t)red_tile_for((int64_t)n);
  const size_t n_tiles = (n + tile - 1) / tile;
  L.head_bits = o;  o = align_up(o + 4 * head_bits_words((int64_t)n));
  L.tile_first = o; o = align_up(o + 4 * (n_tiles + 1));
  L.head_part = o;  o = align_up(o + 4 * n_tiles * (size_t)dim);
  L.tail_part = o;  o = align_up(o + 4 * n_tiles * (size_t)dim);
  L.row_start = o;  o = align_up(o + 4 * (n + 1));
  L.src_worker = o; o = align_up(o + n + 1);
  L.range_ws = o;
  if (K <= kRangeMaxWorkers) {  // scratch of the range-partitioned merge (up to 32 workers)
    L.range = range_layout(K);
    o = align_up(o + L.range.bytes);
  }
  L.bytes = o;
  return L;
}

// bounds of the single sort segment = [0, total rows of all workers], clamped to the capacity
__global__ void agg_prep_kernel(const int64_t* __restrict__ wuo_in, int K, int64_t in_cap,
                                int64_t* __restrict__ bounds, int64_t* __restrict__ wuo,
                                int32_t* status) {
  const int tid = threadIdx.x;
  for (int i = tid; i <= K; i += blockDim.x) {
    int64_t v = wuo_in[i];
    if (v < 0) v = 0;
    if (v > in_cap) v = in_cap;
    wuo[i] = v;
  }
  if (tid == 0) {
    int64_t n = wuo_in[K];
    if (n < 0 || n > in_cap) {
      set_status(status, ANTDT_ERR_CAPACITY);
      n = n < 0 ? 0 : in_cap;
    }
    bounds[0] = 0;
    bounds[1] = n;
  }
}

// Backup-workers variant: only the surviving workers' lists are merged.  prep computes where
// each survivor's list starts in the compacted concatenation, compact copies (row id, original
// position) of the survivors' entries there; the original position stays the payload, so the
// reduction finds rows and weights exactly as in the plain variant.
__global__ void agg_prep_backup_kernel(const int64_t* __restrict__ wuo_in, const uint32_t* __restrict__ drop,
                                       int K, int64_t in_cap, int64_t* __restrict__ bounds,
                                       int64_t* __restrict__ wuo, int64_t* __restrict__ cwuo,
                                       int32_t* status) {
  if (threadIdx.x != 0) return;
  int64_t prev = 0, acc = 0;
  for (int i = 0; i <= K; ++i) {  // K <= 1024: a serial pass is enough
    int64_t v = wuo_in[i];
    v = v < prev ? prev : v;
    v = v > in_cap ? in_cap : v;
    wuo[i] = v;
    if (i > 0) {
      cwuo[i - 1] = acc;
      if (!drop[i - 1]) acc += v - prev;
    }
    prev = v;
  }
  cwuo[K] = acc;
  if (wuo_in[K] < 0 || wuo_in[K] > in_cap) set_status(status, ANTDT_ERR_CAPACITY);
  bounds[0] = 0;
  bounds[1] = acc;
}

__global__ void __launch_bounds__(256)
agg_compact_kernel(const int32_t* __restrict__ uniq_ids, const int64_t* __restrict__ wuo,
                   const int64_t* __restrict__ cwuo, const uint32_t* __restrict__ drop, int K,
                   uint32_t* __restrict__ keys_c, uint32_t* __restrict__ vals_c) {
  extern __shared__ int64_t s_cw[];  // wuo [K+1], cwuo [K+1], then K drop flags
  int64_t* s_wuo = s_cw;
  int64_t* s_cwuo = s_cw + (K + 1);
  uint32_t* s_drop = reinterpret_cast<uint32_t*>(s_cw + 2 * (K + 1));
  for (int i = threadIdx.x; i <= K; i += blockDim.x) { s_wuo[i] = wuo[i]; s_cwuo[i] = cwuo[i]; }
  for (int i = threadIdx.x; i < K; i += blockDim.x) s_drop[i] = drop[i];
  __syncthreads();
  const int64_t n = s_wuo[K];
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < n; p += step) {
    int w = interval_of(s_wuo, K + 1, p);
    if (w > K - 1) w = K - 1;
    if (s_drop[w]) continue;
    const int64_t dst = s_cwuo[w] + (p - s_wuo[w]);
    keys_c[dst] = (uint32_t)uniq_ids[p];
    vals_c[dst] = (uint32_t)p;
  }
}

// dense_out[e] = sum_i w_i * g_i[e], ascending i, one float4 per thread; a worker of weight 0
// (empty or dropped) is not read at all
__global__ void __launch_bounds__(256)
dense_wsum_kernel(const float* __restrict__ grads, int64_t n4, int64_t stride,
                  const float* __restrict__ weights, int K, float* __restrict__ out) {
  extern __shared__ float s_wd[];
  for (int i = threadIdx.x; i < K; i += blockDim.x) s_wd[i] = weights[i];
  __syncthreads();
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n4; e += step) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const float* p = grads + 4 * e;
    int i = 0;
    for (; i + 4 <= K; i += 4) {
      float4 v[4];
#pragma unroll
      for (int t = 0; t < 4; ++t)
        v[t] = s_wd[i + t] != 0.f ? ldg_f4(p + (size_t)(i + t) * stride) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float w = s_wd[i + t];
        acc.x = fmaf(w, v[t].x, acc.x); acc.y = fmaf(w, v[t].y, acc.y);
        acc.z = fmaf(w, v[t].z, acc.z); acc.w = fmaf(w, v[t].w, acc.w);
      }
    }
    for (; i < K; ++i) {
      const float w = s_wd[i];
      if (w == 0.f) continue;
      const float4 v = ldg_f4(p + (size_t)i * stride);
      acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y);
      acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
    }
    reinterpret_cast<float4*>(out)[e] = acc;
  }
}

// Aggregation and update in one pass (up to 32 workers): a group of G lanes owns one aggregated
// row.  Its contributions are the merge slots [row_start[u], row_start[u+1]) in ascending worker
// order; the table and state vectors of the row are requested before the gather, the weighted sum
// is formed in that fixed order and goes straight into the Adagrad / Adam arithmetic, so the
// aggregated gradient is never written to or read back from memory (agg_out, if given, receives
// it all the same).  No partial sums, no second pass: a row has at most K contributions.
struct FusedUpdate {
  void* table; int dtype; int opt; OptParams p; float* state0; float* state1; float* agg_out;
};

// Rows a lane group has in flight, CTAs per SM and the grid.  The kernel is a chain of dependent
// loads per row (slots -> positions -> gradient rows), so warps in flight count for more than
// loads in flight per warp, and the grid decides how close in time neighbouring rows are worked
// on.  Measured on B200 (100M x 64 bf16 table, Adagrad, 16 workers, 16.7 M contributions to 9.2 M
// rows; the two separate kernels take 2.73 ms): 1 row, 8 CTAs/SM, grid of 16 resident waves,
// parameters and state prefetched towards L2 before the sum and loaded after it 2.33 ms (loaded
// after it without the prefetch 2.42, loaded before it 2.58); 32 waves 2.58;
// 8 waves 2.62; 4 waves 2.74; 2 waves 2.88; 1 wave 2.95; one row per lane group and no stride
// 3.30; 6 CTAs/SM 3.05; 2 rows in flight 3.5-4.1; 4 rows 5.0.  Adam (fp32 rows, 16 and 32
// workers): 2.91 / 1.96 ms against 3.22 / 2.20 for the two kernels; at 6 CTAs/SM 3.26 / 2.30.
__device__ __forceinline__ void prefetch_l2(const void* p) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}
constexpr int kFusedRows = 1;
constexpr int kFusedWaves = 16;
constexpr int kFusedCtas = 8;
template <int G, int VPL, bool ADAM, bool BF16>
__global__ void __launch_bounds__(256, (VPL == 1 ? kFusedCtas : 1))
agg_update_kernel(const uint32_t* __restrict__ row_start, const uint32_t* __restrict__ src,
                  const int32_t* __restrict__ agg_ids, const int64_t* __restrict__ n_agg_dev,
                  int64_t out_cap, const int64_t* __restrict__ n_entries,
                  const float* __restrict__ grads, int64_t in_cap,
                  const uint8_t* __restrict__ src_worker, const float* __restrict__ weights, int K,
                  void* table, int64_t n_rows, int dim, OptParams p, float* state0, float* state1,
                  float* __restrict__ agg_out) {
  extern __shared__ float s_w[];  // the K weights
  for (int i = threadIdx.x; i < K; i += blockDim.x) s_w[i] = weights[i];
  __syncthreads();
  constexpr int R = VPL == 1 ? kFusedRows : 1;  // rows a lane group has in flight
  const int lg = threadIdx.x & (G - 1);
  const int nvec = dim / 4;
  // 32-bit row numbers and slots (fewer than 2^31 of each): the kernel is bound by its instruction
  // stream and by the registers that live across the chain of loads
  const uint32_t n = (uint32_t)min(*n_agg_dev, out_cap);
  const uint32_t total = (uint32_t)min(n_entries[1], in_cap);
  const uint32_t stride = gridDim.x * (256 / G);
  for (uint32_t u0 = blockIdx.x * (256 / G) + threadIdx.x / G; u0 < n; u0 += R * stride) {
    uint32_t s0[R], s1[R];
    int32_t row[R];
    bool ok[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const uint32_t u = u0 + r * stride;
      ok[r] = u < n;
      s0[r] = ok[r] ? __ldg(row_start + u) : 0u;
      s1[r] = ok[r] ? (u + 1 < n ? __ldg(row_start + u + 1) : total) : 0u;
      row[r] = ok[r] ? __ldg(agg_ids + u) : -1;
    }
    uint32_t longest = 0;
#pragma unroll
    for (int r = 0; r < R; ++r) {
      ok[r] = ok[r] && (uint32_t)row[r] < (uint32_t)n_rows && s0[r] <= total;  // else flagged by the merge
      if (s1[r] > total) s1[r] = total;
      if (s1[r] > s0[r] + (uint32_t)K) s1[r] = s0[r] + (uint32_t)K;  // a row has at most K contributions
      if (!ok[r]) s1[r] = s0[r];
      longest = max(longest, s1[r] - s0[r]);
    }
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int vi = lg + j * G;
      if (vi >= nvec) continue;
      size_t at[R];
      float4 w[R], a0[R], a1[R], g[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        at[r] = (size_t)(ok[r] ? row[r] : 0) * dim + 4 * (size_t)vi;
        g[r] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ok[r]) {  // towards L2 now (costs no register), into registers after the sum
          prefetch_l2(static_cast<const char*>(table) + at[r] * (BF16 ? 2 : 4));
          prefetch_l2(state0 + at[r]);
          if (ADAM) prefetch_l2(state1 + at[r]);
        }
      }
      for (uint32_t e = 0; e < longest; e += 2) {
        float4 v[R][2];
        float wt[R][2];
#pragma unroll
        for (int r = 0; r < R; ++r) {
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            wt[r][t] = 0.f;
            v[r][t] = make_float4(0.f, 0.f, 0.f, 0.f);
            const uint32_t o = s0[r] + e + t;
            if (o < s1[r]) {
              const uint32_t pos = __ldg(src + o);
              if ((int64_t)pos < in_cap) {
                const int wl = (int)__ldg(src_worker + o);  // written beside src[o] by the merge
                wt[r][t] = s_w[wl > K - 1 ? K - 1 : wl];
                v[r][t] = ldg_f4(grads + (size_t)pos * dim + 4 * vi);
              }
            }
          }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            g[r].x = fmaf(wt[r][t], v[r][t].x, g[r].x); g[r].y = fmaf(wt[r][t], v[r][t].y, g[r].y);
            g[r].z = fmaf(wt[r][t], v[r][t].z, g[r].z); g[r].w = fmaf(wt[r][t], v[r][t].w, g[r].w);
          }
        }
      }
      // the row's parameters and state are requested only now: asking for them before the sum
      // (to overlap their latency with it) costs registers that the 64 warps per SM do not have
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (ok[r]) {
          w[r] = load_row4(table, BF16, at[r]);
          a0[r] = *reinterpret_cast<const float4*>(state0 + at[r]);
          if (ADAM) a1[r] = *reinterpret_cast<const float4*>(state1 + at[r]);
        }
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (!ok[r]) continue;
        if (agg_out) reinterpret_cast<float4*>(agg_out + (size_t)(u0 + r * stride) * dim)[vi] = g[r];
        if (ADAM) {
          w[r].x = adam1(a0[r].x, a1[r].x, g[r].x, w[r].x, p); w[r].y = adam1(a0[r].y, a1[r].y, g[r].y, w[r].y, p);
          w[r].z = adam1(a0[r].z, a1[r].z, g[r].z, w[r].z, p); w[r].w = adam1(a0[r].w, a1[r].w, g[r].w, w[r].w, p);
          *reinterpret_cast<float4*>(state1 + at[r]) = a1[r];
        } else {
          w[r].x = adagrad1(a0[r].x, g[r].x, w[r].x, p); w[r].y = adagrad1(a0[r].y, g[r].y, w[r].y, p);
          w[r].z = adagrad1(a0[r].z, g[r].z, w[r].z, p); w[r].w = adagrad1(a0[r].w, g[r].w, w[r].w, p);
        }
        *reinterpret_cast<float4*>(state0 + at[r]) = a0[r];
        store_row4(table, BF16, at[r], w[r]);
      }
    }
  }
}

template <int G, int VPL>
void launch_agg_update(const FusedUpdate& fu, const uint32_t* row_start, const uint32_t* src,
                       const antdt_sparse_part* sp, int64_t out_cap, const int64_t* n_entries,
                       const uint8_t* src_worker, const float* weights, int K, cudaStream_t s) {
  const int64_t gpb = 256 / G;
  const int64_t want = (out_cap + gpb - 1) / gpb;
  const size_t smem = 4 * (size_t)K;
  const bool adam = fu.opt == ANTDT_OPT_ADAM, bf16 = fu.dtype == ANTDT_BF16;
  const int64_t cap = (int64_t)kNumSM * kFusedCtas * kFusedWaves;
  const unsigned grid = (unsigned)(want > cap ? cap : (want < 1 ? 1 : want));
#define FU_GO(A, B)                                                                              \
  ANTDT_LAUNCH("agg_update", (agg_update_kernel<G, VPL, A, B>), grid, 256, smem, s, row_start, src, \
               sp->agg_ids, sp->n_agg, out_cap, n_entries, sp->uniq_grads, sp->in_cap, src_worker, weights, K, \
               fu.table, sp->n_rows, sp->dim, fu.p, fu.state0, fu.state1, fu.agg_out)
  if (adam) { if (bf16) FU_GO(true, true); else FU_GO(true, false); }
  else      { if (bf16) FU_GO(false, true); else FU_GO(false, false); }
#undef FU_GO
}

}  // namespace
}  // namespace antdt

extern "C" size_t antdt_weighted_aggregate_workspace_bytes(int64_t in_cap, int32_t dim,
                                                           int32_t n_workers) {
  if (in_cap < 0 || dim < 0 || dim > 1024 || n_workers < 1 || n_workers > antdt::kMaxSegments)
    return 0;
  return antdt::agg_layout(in_cap, n_workers, dim).bytes;
}

namespace antdt {
namespace {
// More than 32 workers: merge order by one stable radix sort of (row id, position).
void sort_merge_order(const antdt_sparse_part* sp, const uint8_t* dropped, bool any_dropped, int K,
                      int64_t in_cap, int64_t agg_cap, char* w8, const AggLayout& L,
                      int32_t* dev_status, cudaStream_t s) {
    char* sort_ws = w8 + L.sort_ws;
    int64_t* bounds = (int64_t*)(w8 + L.bounds);
    uint32_t* keys_a = (uint32_t*)(w8 + L.keys_a);
    const uint32_t* sort_keys = reinterpret_cast<const uint32_t*>(sp->uniq_ids);
    const uint32_t* sort_vals = nullptr;  // payload = position in the concatenated lists
    const int key_bits = bits_for(sp->n_rows);
    if (!any_dropped) {
      ANTDT_LAUNCH("agg_prep", agg_prep_kernel, 1, 256, 0, s, sp->worker_uniq_offsets, K, in_cap,
                   bounds, (int64_t*)(w8 + L.wuo), dev_status);
    } else {
      uint32_t hd[kMaxSegments];
      for (int i = 0; i < K; ++i) hd[i] = dropped[i] ? 1u : 0u;
      uint32_t* d_drop = (uint32_t*)(w8 + L.drop);
      int64_t* cwuo = (int64_t*)(w8 + L.cwuo);
      upload_small(hd, 4 * (size_t)K, d_drop, s);
      ANTDT_LAUNCH("agg_prep", agg_prep_backup_kernel, 1, 32, 0, s, sp->worker_uniq_offsets, d_drop,
                   K, in_cap, bounds, (int64_t*)(w8 + L.wuo), cwuo, dev_status);
      // the compacted input lives in the pair of sort buffers that the first pass does not
      // write: the temporaries when the pass count is odd, the outputs when it is even
      const bool odd = sort_passes(key_bits) % 2 == 1;
      uint32_t* keys_c = (uint32_t*)(w8 + (odd ? L.keys_b : L.keys_a));
      uint32_t* vals_c = (uint32_t*)(w8 + (odd ? L.vals_t : L.src));
      if (in_cap > 0) {
        int64_t want = (in_cap + 255) / 256;
        const int64_t gcap = (int64_t)kNumSM * 16;
        ANTDT_LAUNCH("agg_compact", agg_compact_kernel, (unsigned)(want > gcap ? gcap : want), 256,
                     16 * ((size_t)K + 1) + 4 * (size_t)K, s, sp->uniq_ids,
                     (const int64_t*)(w8 + L.wuo), cwuo, d_drop, K, keys_c, vals_c);
      }
      sort_keys = keys_c;
      sort_vals = vals_c;
    }
    segsort_setup(bounds, 1, in_cap, sort_ws, L.sort, s);
    segsort_run(sort_keys, sort_vals, keys_a, (uint32_t*)(w8 + L.src), (uint32_t*)(w8 + L.keys_b),
                (uint32_t*)(w8 + L.vals_t), key_bits, 0, in_cap, sort_ws, L.sort, dev_status, s, true);
    segsort_runs(keys_a, in_cap, sp->agg_ids, (int64_t*)(w8 + L.run_start), nullptr, sp->n_agg,
                 agg_cap, (uint32_t*)(w8 + L.head_bits),
                 (int32_t*)(w8 + L.tile_first), red_tile_for(in_cap > 0 ? in_cap : 1), sort_ws, L.sort, dev_status, s, true);
}

int32_t aggregate_impl(const antdt_sparse_part* sp, const antdt_dense_part* dp,
                       const int64_t* batch_sizes, const uint8_t* dropped, int32_t n_workers,
                       void* ws, size_t ws_bytes, int32_t* dev_status, void* stream,
                       const FusedUpdate* fu = nullptr, const OrderFork* fork = nullptr) {
  const int K = n_workers;
  if (K < 1 || K > kMaxSegments || !batch_sizes || !ws || !aligned16(ws)) return ANTDT_ERR_INVALID_ARG;
  double tot = 0.0;
  bool any_dropped = false;
  for (int i = 0; i < K; ++i) {
    if (batch_sizes[i] < 0) return ANTDT_ERR_INVALID_ARG;
    const bool d = dropped && dropped[i];
    any_dropped |= d;
    if (!d) tot += (double)batch_sizes[i];
  }
  if (!(tot > 0.0)) return ANTDT_ERR_INVALID_ARG;
  const int64_t in_cap = sp ? sp->in_cap : 0;
  if (sp) {
    if (sp->dim < 4 || sp->dim > 1024 || sp->dim % 4 || sp->n_rows < 1 || sp->n_rows >= (1ll << 31) ||
        sp->in_cap < 0 || sp->in_cap >= (1ll << 31) || sp->out_cap < 0 || !sp->worker_uniq_offsets ||
        !sp->n_agg)
      return ANTDT_ERR_INVALID_ARG;
    if (sp->in_cap > 0 && (!sp->uniq_ids || !sp->uniq_grads)) return ANTDT_ERR_INVALID_ARG;
    const bool fused = fu && K <= kRangeMaxWorkers;  // then agg_grads is optional
    if (sp->out_cap > 0 && (!sp->agg_ids || (!sp->agg_grads && !fused))) return ANTDT_ERR_INVALID_ARG;
    if (!aligned16(sp->uniq_grads) || !aligned16(sp->agg_grads)) return ANTDT_ERR_INVALID_ARG;
  }
  if (dp) {
    if (dp->n < 0 || dp->n % 4 || dp->stride < dp->n || dp->stride % 4) return ANTDT_ERR_INVALID_ARG;
    if (dp->n > 0 && (!dp->grads || !dp->out || !aligned16(dp->grads) || !aligned16(dp->out)))
      return ANTDT_ERR_INVALID_ARG;
  }
  const AggLayout L = agg_layout(in_cap, K, sp ? sp->dim : 0);
  if (ws_bytes < L.bytes) return ANTDT_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t s = (cudaStream_t)stream;
  char* w8 = static_cast<char*>(ws);

  // w_i = b_i / sum_j b_j, formed in double, used in fp32
  float hw[kMaxSegments];
  for (int i = 0; i < K; ++i)
    hw[i] = (dropped && dropped[i]) ? 0.f : (float)((double)batch_sizes[i] / tot);
  // the range merge (up to 32 workers, sparse part present) carries the weights itself
  const bool by_ranges = sp && K <= kRangeMaxWorkers && in_cap > 0;
  if (!by_ranges) upload_small(hw, 4 * (size_t)K, w8 + L.weights, s);

  if (sp) {
    int64_t* bounds = (int64_t*)(w8 + L.bounds);
    const int64_t agg_cap = sp->out_cap < in_cap ? sp->out_cap : in_cap;
    if (K <= kRangeMaxWorkers && in_cap > 0) {
      // up to 32 workers: the merge order comes from the range-partitioned pass, no sort
      uint32_t dropped_bits = 0;
      for (int i = 0; i < K; ++i)
        if (dropped && dropped[i]) dropped_bits |= 1u << i;
      // the order needs the id lists only: on a forked step it runs beside the backward's sums
      cudaStream_t so = fork ? fork->side : s;
      if (fork && cudaStreamWaitEvent(so, fork->ids_ready, 0) != cudaSuccess) return ANTDT_ERR_CUDA;
      range_merge_order(sp->uniq_ids, sp->worker_uniq_offsets, in_cap, sp->n_rows, K, dropped_bits,
                        sp->agg_ids, sp->n_agg, agg_cap, (int64_t*)(w8 + L.wuo), bounds,
                        (uint32_t*)(w8 + L.src), fu ? nullptr : (uint32_t*)(w8 + L.head_bits),
                        fu ? nullptr : (int32_t*)(w8 + L.tile_first), red_tile_for(in_cap),
                        fu ? (uint32_t*)(w8 + L.row_start) : nullptr,
                        fu ? (uint8_t*)(w8 + L.src_worker) : nullptr, hw, (float*)(w8 + L.weights),
                        w8 + L.range_ws, L.range, dev_status, so);
      if (fork && (cudaEventRecord(fork->order_done, so) != cudaSuccess ||
                   cudaStreamWaitEvent(s, fork->order_done, 0) != cudaSuccess))
        return ANTDT_ERR_CUDA;
    } else {
      sort_merge_order(sp, dropped, any_dropped, K, in_cap, agg_cap, w8, L, dev_status, s);
    }
    if (fu && K <= kRangeMaxWorkers && in_cap > 0) {
      // one pass: every aggregated row is summed and applied by the lane group that owns it
      FusedUpdate f = *fu;
      f.agg_out = sp->agg_grads;
      const uint32_t* rs = (const uint32_t*)(w8 + L.row_start);
      const uint32_t* src = (const uint32_t*)(w8 + L.src);
      const uint8_t* sw = (const uint8_t*)(w8 + L.src_worker);
      const float* wts = (const float*)(w8 + L.weights);
      const int nvec = sp->dim / 4;
#define FU_CASE(G, VPL) launch_agg_update<G, VPL>(f, rs, src, sp, agg_cap, bounds, sw, wts, K, s)
      if (nvec <= 1) FU_CASE(1, 1);
      else if (nvec <= 2) FU_CASE(2, 1);
      else if (nvec <= 4) FU_CASE(4, 1);
      else if (nvec <= 8) FU_CASE(8, 1);
      else if (nvec <= 16) FU_CASE(16, 1);
      else if (nvec <= 32) FU_CASE(32, 1);
      else if (nvec <= 64) FU_CASE(32, 2);
      else if (nvec <= 128) FU_CASE(32, 4);
      else FU_CASE(32, 8);
#undef FU_CASE
    } else if (in_cap > 0) {
      TileArgs t;
      t.payload = (const uint32_t*)(w8 + L.src);
      t.head_bits = (const uint32_t*)(w8 + L.head_bits);
      t.tile_first = (const int32_t*)(w8 + L.tile_first);
      t.tile = red_tile_for(in_cap);
      t.rows = sp->uniq_grads;
      t.dim = sp->dim;
      t.n_host = in_cap;
      t.n_dev = bounds + 1;  // the clamped total of the workers' lists
      t.payload_limit = in_cap;
      t.bounds = (const int64_t*)(w8 + L.wuo);
      t.scales = (const float*)(w8 + L.weights);
      t.K = K;
      t.out_cap = sp->out_cap < in_cap ? sp->out_cap : in_cap;
      t.out = sp->agg_grads;
      t.head_part = (float*)(w8 + L.head_part);
      t.tail_part = (float*)(w8 + L.tail_part);
      launch_tile_reduce(t, "agg_reduce", "agg_fixup", s);
    }
  }
  if (dp && dp->n > 0) {
    const int64_t n4 = dp->n / 4;
    int64_t want = (n4 + 255) / 256;
    const int64_t cap = (int64_t)kNumSM * 16;
    const unsigned grid = (unsigned)(want > cap ? cap : want);
    ANTDT_LAUNCH("dense_wsum", dense_wsum_kernel, grid, 256, 4 * (size_t)K, s, dp->grads, n4,
                 dp->stride, (const float*)(w8 + L.weights), K, dp->out);
  }
  return cuda_ok();
}
}  // namespace

int32_t weighted_aggregate_forked(const antdt_sparse_part* sp, const antdt_dense_part* dp,
                                  const int64_t* batch_sizes, int32_t n_workers, void* ws,
                                  size_t ws_bytes, int32_t* dev_status, void* stream,
                                  const OrderFork* fork) {
  return aggregate_impl(sp, dp, batch_sizes, nullptr, n_workers, ws, ws_bytes, dev_status, stream,
                        nullptr, fork);
}
}  // namespace antdt

extern "C" int32_t antdt_weighted_aggregate(const antdt_sparse_part* sp, const antdt_dense_part* dp,
                                            const int64_t* batch_sizes, int32_t n_workers, void* ws,
                                            size_t ws_bytes, int32_t* dev_status, void* stream) {
  return antdt::aggregate_impl(sp, dp, batch_sizes, nullptr, n_workers, ws, ws_bytes, dev_status,
                               stream);
}

extern "C" int32_t antdt_weighted_aggregate_backup(const antdt_sparse_part* sp,
                                                   const antdt_dense_part* dp,
                                                   const int64_t* batch_sizes, const uint8_t* dropped,
                                                   int32_t n_workers, void* ws, size_t ws_bytes,
                                                   int32_t* dev_status, void* stream) {
  if (!dropped) return ANTDT_ERR_INVALID_ARG;
  return antdt::aggregate_impl(sp, dp, batch_sizes, dropped, n_workers, ws, ws_bytes, dev_status,
                               stream);
}

// Aggregation followed by the sparse update in one call; with up to 32 workers in one pass over
// the aggregated rows (agg_update_kernel), otherwise the two steps one after the other.
namespace antdt {
int32_t aggregate_update_forked(const antdt_sparse_part* sp, const antdt_dense_part* dp,
                                const int64_t* batch_sizes, int32_t n_workers, void* table,
                                int32_t dtype, int32_t opt, float lr, float eps, float beta1,
                                float beta2, int64_t step, float* state0, float* state1, void* ws,
                                size_t ws_bytes, int32_t* dev_status, void* stream,
                                const OrderFork* fork) {
  if (!sp || !table || !state0 || step < 1) return ANTDT_ERR_INVALID_ARG;
  if (dtype != ANTDT_F32 && dtype != ANTDT_BF16) return ANTDT_ERR_INVALID_ARG;
  if (sp->dim % (dtype == ANTDT_BF16 ? 8 : 4)) return ANTDT_ERR_INVALID_ARG;
  if (opt != ANTDT_OPT_ADAGRAD && opt != ANTDT_OPT_ADAM) return ANTDT_ERR_INVALID_ARG;
  if (opt == ANTDT_OPT_ADAM && !state1) return ANTDT_ERR_INVALID_ARG;
  if (!aligned16(table) || !aligned16(state0) || !aligned16(state1)) return ANTDT_ERR_INVALID_ARG;
  if (n_workers > kRangeMaxWorkers) {  // the sort-based merge: two steps, agg_grads is needed
    if (sp->out_cap > 0 && !sp->agg_grads) return ANTDT_ERR_INVALID_ARG;
    const int32_t rc = aggregate_impl(sp, dp, batch_sizes, nullptr, n_workers, ws, ws_bytes,
                                      dev_status, stream);
    if (rc != ANTDT_OK) return rc;
    const int64_t cap = sp->out_cap < sp->in_cap ? sp->out_cap : sp->in_cap;
    return antdt_sparse_opt_update(table, dtype, sp->n_rows, sp->dim, sp->agg_ids, sp->agg_grads,
                                   sp->n_agg, cap, opt, lr, eps, beta1, beta2, step, state0, state1,
                                   dev_status, stream);
  }
  FusedUpdate fu;
  fu.table = table; fu.dtype = dtype; fu.opt = opt; fu.state0 = state0; fu.state1 = state1;
  fu.agg_out = nullptr;
  fu.p = make_opt_params(lr, eps, beta1, beta2, step);
  return aggregate_impl(sp, dp, batch_sizes, nullptr, n_workers, ws, ws_bytes, dev_status, stream, &fu,
                        fork);
}
}  // namespace antdt

extern "C" int32_t antdt_aggregate_update(const antdt_sparse_part* sp, const antdt_dense_part* dp,
                                          const int64_t* batch_sizes, int32_t n_workers, void* table,
                                          int32_t dtype, int32_t opt, float lr, float eps, float beta1,
                                          float beta2, int64_t step, float* state0, float* state1,
                                          void* ws, size_t ws_bytes, int32_t* dev_status, void* stream) {
  return antdt::aggregate_update_forked(sp, dp, batch_sizes, n_workers, table, dtype, opt, lr, eps, beta1,
                                        beta2, step, state0, state1, ws, ws_bytes, dev_status, stream,
                                        nullptr);
}
