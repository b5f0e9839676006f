// Server update: sparse Adagrad / Adam on the aggregated rows only.
//
// One group of G lanes per row, four consecutive elements per lane: fp32 rows and the fp32
// state and gradient rows move as 16-byte vectors; bf16 table rows as 8-byte vectors (four
// bf16), widened to fp32, updated and stored back round-to-nearest-even.  The ids ascend, so
// the row accesses sweep the table forward.  Division and square root are the IEEE-rounded
// ones (no fast-math).
#include "common.cuh"

namespace antdt {
namespace {

constexpr int kOptThreads = 256;

struct OptParams {
  float lr, eps, beta1, beta2;
  float omb1, omb2;  // 1 - beta
  float bc1, bc2;    // 1 - beta^t
};

__device__ __forceinline__ float4 load_row4(const void* table, bool bf16, size_t elem) {
  if (bf16) {
    const uint2 v = *reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(table) + elem);
    return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u),
                       __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
  }
  return *reinterpret_cast<const float4*>(static_cast<const float*>(table) + elem);
}

__device__ __forceinline__ void store_row4(void* table, bool bf16, size_t elem, float4 w) {
  if (bf16) {
    uint2 v;
    v.x = pack_bf16x2_rn(w.x, w.y);
    v.y = pack_bf16x2_rn(w.z, w.w);
    *reinterpret_cast<uint2*>(static_cast<uint16_t*>(table) + elem) = v;
  } else {
    *reinterpret_cast<float4*>(static_cast<float*>(table) + elem) = w;
  }
}

__device__ __forceinline__ float adagrad1(float& acc, float g, float w, const OptParams& p) {
  acc = fmaf(g, g, acc);
  return w - p.lr * g / (sqrtf(acc) + p.eps);
}

__device__ __forceinline__ float adam1(float& m, float& v, float g, float w, const OptParams& p) {
  m = fmaf(p.beta1, m, p.omb1 * g);
  v = fmaf(p.beta2, v, p.omb2 * g * g);
  return w - p.lr * (m / p.bc1) / (sqrtf(v / p.bc2) + p.eps);
}

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
  if (opt != ANTDT_OPT_ADAGRAD && opt != ANTDT_OPT_ADAM) return ANTDT_ERR_INVALID_ARG;
  if (max_ids == 0) return ANTDT_OK;
  if (!table || !ids || !grads || !n_ids_dev || !state0 || (opt == ANTDT_OPT_ADAM && !state1))
    return ANTDT_ERR_INVALID_ARG;
  if (!aligned16(table) || !aligned16(grads) || !aligned16(state0) || !aligned16(state1))
    return ANTDT_ERR_INVALID_ARG;
  OptParams p;
  p.lr = lr; p.eps = eps; p.beta1 = beta1; p.beta2 = beta2;
  p.omb1 = (float)(1.0 - (double)beta1);
  p.omb2 = (float)(1.0 - (double)beta2);
  p.bc1 = (float)(1.0 - pow((double)beta1, (double)step));
  p.bc2 = (float)(1.0 - pow((double)beta2, (double)step));
  const bool adam = opt == ANTDT_OPT_ADAM, bf16 = dtype == ANTDT_BF16;
  cudaStream_t s = (cudaStream_t)stream;
  const int nvec = dim / 4;
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
