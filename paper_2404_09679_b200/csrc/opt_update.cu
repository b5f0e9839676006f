// Server update: sparse Adagrad / Adam on the aggregated rows only.
//
// One group of G lanes per row, four consecutive elements per lane: fp32 rows and the fp32
// state and gradient rows move as 16-byte vectors; bf16 table rows as 8-byte vectors (four
// bf16), widened to fp32, updated and stored back round-to-nearest-even.  The ids ascend, so
// the row accesses sweep the table forward.  Division and square root are the IEEE-rounded
// ones (no fast-math).
#include "opt_math.cuh"

namespace antdt {
namespace {

constexpr int kOptThreads = 256;

// Rows a lane group has in flight.  Measured on B200: Adam (four 16-byte streams per row) gains
// from two rows a stride apart; Adagrad is faster with one row and the higher occupancy.
constexpr int kOptRowsAdam = 2;

template <int G, int VPL, bool ADAM, bool BF16>
__global__ void __launch_bounds__(kOptThreads)
sparse_opt_kernel(void* table, int64_t n_rows, int dim, const int32_t* __restrict__ ids,
                  const float* __restrict__ grads, const int64_t* __restrict__ n_ids_dev,
                  int64_t max_ids, OptParams p, float* state0, float* state1, int32_t* status) {
  const int lg = threadIdx.x & (G - 1);
  const int nvec = dim / 4;
  const int64_t n = min(*n_ids_dev, max_ids);
  const int64_t stride = (int64_t)gridDim.x * (kOptThreads / G);
  constexpr int R = (ADAM && VPL == 1) ? kOptRowsAdam : 1;
  for (int64_t k0 = (int64_t)blockIdx.x * (kOptThreads / G) + threadIdx.x / G; k0 < n; k0 += R * stride) {
    int64_t row[R];
    bool ok[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int64_t k = k0 + r * stride;
      row[r] = k < n ? (int64_t)__ldg(ids + k) : -1;
      ok[r] = row[r] >= 0 && row[r] < n_rows;
      if (k < n && !ok[r] && lg == 0) set_status(status, ANTDT_ERR_ID_OUT_OF_RANGE);
    }
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int vi = lg + j * G;
      if (vi >= nvec) continue;
      float4 g[R], w[R], s0[R], s1[R];
      size_t at[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (!ok[r]) continue;
        at[r] = (size_t)row[r] * dim + 4 * (size_t)vi;
        g[r] = ldg_f4(grads + (size_t)(k0 + r * stride) * dim + 4 * vi);
        w[r] = load_row4(table, BF16, at[r]);
        s0[r] = *reinterpret_cast<const float4*>(state0 + at[r]);
        if (ADAM) s1[r] = *reinterpret_cast<const float4*>(state1 + at[r]);
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (!ok[r]) continue;
        if (ADAM) {
          w[r].x = adam1(s0[r].x, s1[r].x, g[r].x, w[r].x, p); w[r].y = adam1(s0[r].y, s1[r].y, g[r].y, w[r].y, p);
          w[r].z = adam1(s0[r].z, s1[r].z, g[r].z, w[r].z, p); w[r].w = adam1(s0[r].w, s1[r].w, g[r].w, w[r].w, p);
          *reinterpret_cast<float4*>(state1 + at[r]) = s1[r];
        } else {
          w[r].x = adagrad1(s0[r].x, g[r].x, w[r].x, p); w[r].y = adagrad1(s0[r].y, g[r].y, w[r].y, p);
          w[r].z = adagrad1(s0[r].z, g[r].z, w[r].z, p); w[r].w = adagrad1(s0[r].w, g[r].w, w[r].w, p);
        }
        *reinterpret_cast<float4*>(state0 + at[r]) = s0[r];
        store_row4(table, BF16, at[r], w[r]);
      }
    }
  }
}

// Row-wise Adagrad: one accumulator per row, fed with the mean square of the row's gradient.
// The group's lanes sum their own squares, a butterfly over the group makes the row's total (the
// same value in every lane), lane 0 stores the accumulator.
template <int G, int VPL, bool BF16>
__global__ void __launch_bounds__(kOptThreads)
rowwise_adagrad_kernel(void* table, int64_t n_rows, int dim, const int32_t* __restrict__ ids,
                       const float* __restrict__ grads, const int64_t* __restrict__ n_ids_dev,
                       int64_t max_ids, OptParams p, float* state0, int32_t* status) {
  const int lg = threadIdx.x & (G - 1);
  const int nvec = dim / 4;
  const unsigned gmask = group_mask<G>();
  const int64_t n = min(*n_ids_dev, max_ids);
  const int64_t stride = (int64_t)gridDim.x * (kOptThreads / G);
  const float dimf = (float)dim;
  for (int64_t k = (int64_t)blockIdx.x * (kOptThreads / G) + threadIdx.x / G; k < n; k += stride) {
    const int64_t row = __ldg(ids + k);
    if (row < 0 || row >= n_rows) {  // the whole group takes this branch together
      if (lg == 0) set_status(status, ANTDT_ERR_ID_OUT_OF_RANGE);
      continue;
    }
    float4 g[VPL], w[VPL];
    const float acc0 = state0[row];
    float sq = 0.f;
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int vi = lg + j * G;
      if (vi < nvec) {
        g[j] = ldg_f4(grads + (size_t)k * dim + 4 * vi);
        w[j] = load_row4(table, BF16, (size_t)row * dim + 4 * (size_t)vi);
        sq = fmaf(g[j].x, g[j].x, sq); sq = fmaf(g[j].y, g[j].y, sq);
        sq = fmaf(g[j].z, g[j].z, sq); sq = fmaf(g[j].w, g[j].w, sq);
      }
    }
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) sq += __shfl_xor_sync(gmask, sq, o, G);
    const float acc = acc0 + sq / dimf;
    const float den = sqrtf(acc) + p.eps;
    if (lg == 0) state0[row] = acc;
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int vi = lg + j * G;
      if (vi < nvec) {
        w[j].x -= p.lr * g[j].x / den; w[j].y -= p.lr * g[j].y / den;
        w[j].z -= p.lr * g[j].z / den; w[j].w -= p.lr * g[j].w / den;
        store_row4(table, BF16, (size_t)row * dim + 4 * (size_t)vi, w[j]);
      }
    }
  }
}

// Dense parameters: the same element-wise rules, four elements per thread, streaming.
template <bool ADAM>
__global__ void __launch_bounds__(kOptThreads)
dense_opt_kernel(float* __restrict__ params, const float* __restrict__ grad, int64_t n4, OptParams p,
                 float* __restrict__ state0, float* __restrict__ state1) {
  const int64_t stride = (int64_t)gridDim.x * kOptThreads;
  for (int64_t e = (int64_t)blockIdx.x * kOptThreads + threadIdx.x; e < n4; e += stride) {
    const float4 g = ldg_f4(grad + 4 * e);
    float4 w = reinterpret_cast<const float4*>(params)[e];
    float4 s0 = reinterpret_cast<const float4*>(state0)[e];
    if (ADAM) {
      float4 s1 = reinterpret_cast<const float4*>(state1)[e];
      w.x = adam1(s0.x, s1.x, g.x, w.x, p); w.y = adam1(s0.y, s1.y, g.y, w.y, p);
      w.z = adam1(s0.z, s1.z, g.z, w.z, p); w.w = adam1(s0.w, s1.w, g.w, w.w, p);
      reinterpret_cast<float4*>(state1)[e] = s1;
    } else {
      w.x = adagrad1(s0.x, g.x, w.x, p); w.y = adagrad1(s0.y, g.y, w.y, p);
      w.z = adagrad1(s0.z, g.z, w.z, p); w.w = adagrad1(s0.w, g.w, w.w, p);
    }
    reinterpret_cast<float4*>(state0)[e] = s0;
    reinterpret_cast<float4*>(params)[e] = w;
  }
}

template <int G, int VPL>
void launch_rowwise(bool bf16, void* table, int64_t n_rows, int dim, const int32_t* ids,
                    const float* grads, const int64_t* n_ids_dev, int64_t max_ids, const OptParams& p,
                    float* state0, int32_t* status, cudaStream_t s) {
  const int64_t gpb = kOptThreads / G;
  const int64_t want = (max_ids + gpb - 1) / gpb;
  const int64_t cap = (int64_t)kNumSM * 16;
  const unsigned grid = (unsigned)(want > cap ? cap : want);
  if (bf16)
    ANTDT_LAUNCH("sparse_rowwise_adagrad", (rowwise_adagrad_kernel<G, VPL, true>), grid, kOptThreads,
                 0, s, table, n_rows, dim, ids, grads, n_ids_dev, max_ids, p, state0, status);
  else
    ANTDT_LAUNCH("sparse_rowwise_adagrad", (rowwise_adagrad_kernel<G, VPL, false>), grid, kOptThreads,
                 0, s, table, n_rows, dim, ids, grads, n_ids_dev, max_ids, p, state0, status);
}

template <int G, int VPL>
void launch_opt(bool adam, bool bf16, void* table, int64_t n_rows, int dim, const int32_t* ids,
                const float* grads, const int64_t* n_ids_dev, int64_t max_ids, const OptParams& p,
                float* state0, float* state1, int32_t* status, cudaStream_t s) {
  const int64_t gpb = kOptThreads / G;
  const int64_t want = (max_ids + gpb - 1) / gpb;
  const int64_t cap = (int64_t)kNumSM * 16;
  const unsigned grid = (unsigned)(want > cap ? cap : want);
#define OPT_GO(A, B)                                                                            \
  ANTDT_LAUNCH(A ? "sparse_adam" : "sparse_adagrad", (sparse_opt_kernel<G, VPL, A, B>), grid,   \
               kOptThreads, 0, s, table, n_rows, dim, ids, grads, n_ids_dev, max_ids, p, state0, \
               state1, status)
  if (adam) { if (bf16) OPT_GO(true, true); else OPT_GO(true, false); }
  else      { if (bf16) OPT_GO(false, true); else OPT_GO(false, false); }
#undef OPT_GO
}

}  // namespace
}  // namespace antdt

extern "C" int32_t antdt_sparse_opt_update(void* table, int32_t dtype, int64_t n_rows, int32_t dim,
                                           const int32_t* ids, const float* grads,
                                           const int64_t* n_ids_dev, int64_t max_ids, int32_t opt,
                                           float lr, float eps, float beta1, float beta2,
                                           int64_t step, float* state0, float* state1,
                                           int32_t* dev_status, void* stream) {
  using namespace antdt;
  if (n_rows < 1 || n_rows >= (1ll << 31) || dim < 4 || dim > 1024 || max_ids < 0 || step < 1)
    return ANTDT_ERR_INVALID_ARG;
  if (dtype != ANTDT_F32 && dtype != ANTDT_BF16) return ANTDT_ERR_INVALID_ARG;
  if (dim % (dtype == ANTDT_BF16 ? 8 : 4)) return ANTDT_ERR_INVALID_ARG;
  if (opt != ANTDT_OPT_ADAGRAD && opt != ANTDT_OPT_ADAM && opt != ANTDT_OPT_ROWWISE_ADAGRAD)
    return ANTDT_ERR_INVALID_ARG;
  if (max_ids == 0) return ANTDT_OK;
  if (!table || !ids || !grads || !n_ids_dev || !state0 || (opt == ANTDT_OPT_ADAM && !state1))
    return ANTDT_ERR_INVALID_ARG;
  if (!aligned16(table) || !aligned16(grads) || !aligned16(state1)) return ANTDT_ERR_INVALID_ARG;
  if (opt == ANTDT_OPT_ROWWISE_ADAGRAD ? (reinterpret_cast<uintptr_t>(state0) & 3u) != 0 : !aligned16(state0))
    return ANTDT_ERR_INVALID_ARG;
  const OptParams p = make_opt_params(lr, eps, beta1, beta2, step);
  const bool adam = opt == ANTDT_OPT_ADAM, bf16 = dtype == ANTDT_BF16;
  cudaStream_t s = (cudaStream_t)stream;
  const int nvec = dim / 4;
  if (opt == ANTDT_OPT_ROWWISE_ADAGRAD) {
#define ROW_CASE(G, VPL) \
  launch_rowwise<G, VPL>(bf16, table, n_rows, dim, ids, grads, n_ids_dev, max_ids, p, state0, dev_status, s);
    if (nvec <= 1) { ROW_CASE(1, 1) }
    else if (nvec <= 2) { ROW_CASE(2, 1) }
    else if (nvec <= 4) { ROW_CASE(4, 1) }
    else if (nvec <= 8) { ROW_CASE(8, 1) }
    else if (nvec <= 16) { ROW_CASE(16, 1) }
    else if (nvec <= 32) { ROW_CASE(32, 1) }
    else if (nvec <= 64) { ROW_CASE(32, 2) }
    else if (nvec <= 128) { ROW_CASE(32, 4) }
    else { ROW_CASE(32, 8) }
#undef ROW_CASE
    return cuda_ok();
  }
#define OPT_CASE(G, VPL)                                                                       \
  launch_opt<G, VPL>(adam, bf16, table, n_rows, dim, ids, grads, n_ids_dev, max_ids, p, state0, \
                     state1, dev_status, s);
  if (nvec <= 1) { OPT_CASE(1, 1) }
  else if (nvec <= 2) { OPT_CASE(2, 1) }
  else if (nvec <= 4) { OPT_CASE(4, 1) }
  else if (nvec <= 8) { OPT_CASE(8, 1) }
  else if (nvec <= 16) { OPT_CASE(16, 1) }
  else if (nvec <= 32) { OPT_CASE(32, 1) }
  else if (nvec <= 64) { OPT_CASE(32, 2) }
  else if (nvec <= 128) { OPT_CASE(32, 4) }
  else { OPT_CASE(32, 8) }
#undef OPT_CASE
  return cuda_ok();
}

extern "C" int32_t antdt_dense_opt_update(float* params, const float* grad, int64_t n, int32_t opt,
                                          float lr, float eps, float beta1, float beta2,
                                          int64_t step, float* state0, float* state1, void* stream) {
  using namespace antdt;
  if (n < 0 || n % 4 || step < 1) return ANTDT_ERR_INVALID_ARG;
  if (opt != ANTDT_OPT_ADAGRAD && opt != ANTDT_OPT_ADAM) return ANTDT_ERR_INVALID_ARG;
  if (n == 0) return ANTDT_OK;
  if (!params || !grad || !state0 || (opt == ANTDT_OPT_ADAM && !state1)) return ANTDT_ERR_INVALID_ARG;
  if (!aligned16(params) || !aligned16(grad) || !aligned16(state0) || !aligned16(state1))
    return ANTDT_ERR_INVALID_ARG;
  const OptParams p = make_opt_params(lr, eps, beta1, beta2, step);
  const int64_t n4 = n / 4;
  const int64_t want = (n4 + kOptThreads - 1) / kOptThreads;
  const int64_t cap = (int64_t)kNumSM * 16;
  const unsigned grid = (unsigned)(want > cap ? cap : want);
  cudaStream_t s = (cudaStream_t)stream;
  if (opt == ANTDT_OPT_ADAM)
    ANTDT_LAUNCH("dense_adam", dense_opt_kernel<true>, grid, kOptThreads, 0, s, params, grad, n4, p,
                 state0, state1);
  else
    ANTDT_LAUNCH("dense_adagrad", dense_opt_kernel<false>, grid, kOptThreads, 0, s, params, grad, n4,
                 p, state0, state1);
  return cuda_ok();
}
