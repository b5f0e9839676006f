// Shared device/host helpers of the CUDA translation units: launch bookkeeping, the status
// word, 128-bit row access, group (sub-warp) shuffles.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "antdt.h"

namespace antdt {

// ---- launch bookkeeping (runtime.cu) --------------------------------------------------
int prof_begin(const char* name, cudaStream_t s);
void prof_end(int token, cudaStream_t s);
// While on, this thread's launches are counted but not bracketed by events (a stream that is
// being captured cannot time its nodes).
void prof_untimed(bool on);
// Adds n to the launch counter: kernels that ran as nodes of a replayed graph.
void count_launches(int64_t n);

// Launch `kernel` and account for it (launch counter; CUDA-event bracket when profiling is on).
#define ANTDT_LAUNCH(name, kernel, grid, block, smem, stream, ...)        \
  do {                                                                    \
    int _tok = antdt::prof_begin(name, stream);                           \
    kernel<<<(grid), (block), (smem), (stream)>>>(__VA_ARGS__);           \
    antdt::prof_end(_tok, stream);                                        \
  } while (0)

static inline int32_t cuda_ok() {
  return cudaGetLastError() == cudaSuccess ? ANTDT_OK : ANTDT_ERR_CUDA;
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Copies a small host array (worker tables: a few KB at most) to device memory through kernel
// parameters, 2 KB per launch, so the call neither blocks on the stream nor needs page-locked
// memory.  bytes % 4 == 0.  Defined in runtime.cu.
void upload_small(const void* host, size_t bytes, void* dev, cudaStream_t s);

// A d_pooled matrix that is still being copied in when the backward is issued, in n pieces:
// piece c holds the rows that the occurrences before entry_end[c] (ascending, host array) refer
// to - in a step these are the workers' sample ranges - and is complete once ready[c] has
// happened.  Later events imply the earlier ones (one copy stream).
struct PooledArrival {
  int n;
  const int64_t* entry_end;
  const cudaEvent_t* ready;
};

int32_t bwd_dedup_impl(const int32_t* row_ids, int64_t nnz, const int64_t* bag_offsets,
                       int64_t n_bags, int32_t bags_per_sample, const float* d_pooled, int32_t dim,
                       int64_t n_rows, int32_t n_workers, const int64_t* worker_sample_offsets,
                       int32_t* uniq_ids, int64_t* worker_uniq_offsets, int64_t* seg_offsets,
                       int32_t* sorted_occ, float* uniq_grads, int64_t out_cap, void* ws,
                       size_t ws_bytes, int32_t* dev_status, void* stream,
                       const PooledArrival* arrival,
                       cudaEvent_t ids_done = nullptr);  // embbag_bwd.cu; ids_done: recorded once the
                                                         // distinct ids and their offsets are written

// A second stream for the aggregation's merge order, which needs the workers' id lists but not
// their gradients: the order kernels wait for ids_ready on `side`, and the caller's stream waits
// for them (order_done) before it sums.  Used where the two chains are short enough to overlap.
struct OrderFork {
  cudaStream_t side;
  cudaEvent_t ids_ready, order_done;
};
int32_t weighted_aggregate_forked(const antdt_sparse_part* sp, const antdt_dense_part* dp,
                                  const int64_t* batch_sizes, int32_t n_workers, void* ws,
                                  size_t ws_bytes, int32_t* dev_status, void* stream,
                                  const OrderFork* fork);  // aggregate.cu
int32_t aggregate_update_forked(const antdt_sparse_part* sp, const antdt_dense_part* dp,
                                const int64_t* batch_sizes, int32_t n_workers, void* table,
                                int32_t dtype, int32_t opt, float lr, float eps, float beta1,
                                float beta2, int64_t step, float* state0, float* state1, void* ws,
                                size_t ws_bytes, int32_t* dev_status, void* stream,
                                const OrderFork* fork);  // aggregate.cu

int32_t fwd_impl(const void* table, int32_t dtype, int64_t n_rows, int32_t dim, const int32_t* row_ids,
                 int64_t nnz, const int64_t* bag_offsets, int64_t n_bags, float* pooled,
                 int32_t* dev_status, void* stream, int32_t bags_per_sample);  // embbag_fwd.cu

constexpr int kNumSM = 148;  // B200: 2 dies x 74 SMs; grids are sized in multiples of this

// ---- device helpers -------------------------------------------------------------------
// First error wins; a NULL status word means "skip silently".
__device__ __forceinline__ void set_status(int32_t* st, int32_t code) {
  if (st) atomicCAS(st, 0, code);
}

// Mask of the G-lane group this lane belongs to (G a power of two <= 32).
template <int G>
__device__ __forceinline__ unsigned group_mask() {
  if (G == 32) return 0xffffffffu;
  unsigned lane = threadIdx.x & 31u;
  return ((1u << G) - 1u) << (lane & ~(unsigned)(G - 1));
}

__device__ __forceinline__ float4 ldg_f4(const float* p) {
  return __ldg(reinterpret_cast<const float4*>(p));
}

// Packed pairs of fp32 in one 64-bit register: sm_100 adds / multiplies two lanes per
// instruction (each lane rounded exactly like the scalar operation).
__device__ __forceinline__ uint64_t f32x2_pack(uint32_t lo_bits, uint32_t hi_bits) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo_bits), "r"(hi_bits));
  return r;
}
__device__ __forceinline__ uint64_t f32x2_add(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t f32x2_mul(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ ulonglong2 ldg_u64x2(const void* p) {
  return __ldg(reinterpret_cast<const ulonglong2*>(p));
}

// 8 bf16 (one 16-byte vector) widened to fp32; widening is exact.
__device__ __forceinline__ void bf16x8_to_f32(const uint4& v, float* f) {
  f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
  f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
  f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
  f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
}

// Two fp32 -> packed bf16x2, round to nearest even (lo in the low half).
__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// upper_bound(a[0..n), x) - 1 for ascending a with a[0] <= x: the interval that holds x.
__device__ __forceinline__ int interval_of(const int64_t* a, int n, int64_t x) {
  int lo = 0, hi = n;  // invariant: a[lo] <= x, (hi == n or a[hi] > x)
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (a[mid] <= x) lo = mid; else hi = mid;
  }
  return lo;
}

}  // namespace antdt
