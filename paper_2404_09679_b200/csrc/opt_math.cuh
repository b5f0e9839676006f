// Element-wise arithmetic of the server update (Adagrad, Adam) and the 4-element row accessors,
// shared by the update kernels and the fused aggregate-and-update kernel.  fp32 throughout; the
// division and the square root are the IEEE-rounded ones (no fast-math).
#pragma once
#include <math.h>

#include "common.cuh"

namespace antdt {

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

inline OptParams make_opt_params(float lr, float eps, float beta1, float beta2, int64_t step) {
  OptParams p;
  p.lr = lr; p.eps = eps; p.beta1 = beta1; p.beta2 = beta2;
  p.omb1 = (float)(1.0 - (double)beta1);
  p.omb2 = (float)(1.0 - (double)beta2);
  p.bc1 = (float)(1.0 - pow((double)beta1, (double)step));
  p.bc2 = (float)(1.0 - pow((double)beta2, (double)step));
  return p;
}

}  // namespace antdt
