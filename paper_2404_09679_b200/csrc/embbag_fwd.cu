// Worker forward: embedding-bag gather with sum pooling.
//
// One group of G lanes owns one bag; a row is read as G (x VPL) 16-byte vectors, so a warp
// issues fully coalesced 128-bit loads over 32/G rows at once.  The bag's id list is staged
// through the group's registers G ids at a time (one coalesced load, then shuffles), and U row
// loads are put in flight before any is consumed.  The path is a random gather bound by HBM
// (hot rows by L2); there is no contraction here and so no tensor-core work.
#include "common.cuh"

namespace antdt {
namespace {

constexpr int kFwdThreads = 128;
constexpr int kFwdUnroll = 4;

template <int G, int VPL, bool BF16, bool BY_FIELD>
__global__ void __launch_bounds__(kFwdThreads, (VPL == 1 ? 12 : 1))
embbag_fwd_kernel(const void* __restrict__ table, int64_t n_rows, int dim,
                  const int32_t* __restrict__ row_ids, int64_t nnz,
                  const int64_t* __restrict__ bag_offsets, int64_t n_bags,
                  float* __restrict__ pooled, int32_t* status, int fields, int64_t sample_blocks) {
  constexpr int EPV = BF16 ? 8 : 4;   // elements per 16-byte vector
  constexpr int PAIRS = EPV / 2;      // packed fp32 pairs per vector
  constexpr int U = (G < kFwdUnroll) ? G : kFwdUnroll;
  const int lg = threadIdx.x & (G - 1);
  // Bags are sample-major (bag = sample * fields + field).  When the caller knows `fields`, a CTA
  // takes the bags of ONE field of consecutive samples and consecutive CTAs stay on that field,
  // so that what is resident on an SM (and in L2) at one time draws from one field's hot rows.
  int64_t bag;
  if (BY_FIELD) {
    const int64_t f = blockIdx.x / sample_blocks, sb = blockIdx.x % sample_blocks;
    bag = (sb * (kFwdThreads / G) + (threadIdx.x / G)) * fields + f;
  } else {
    bag = (int64_t)blockIdx.x * (kFwdThreads / G) + (threadIdx.x / G);
  }
  if (bag >= n_bags) return;
  const unsigned gmask = group_mask<G>();
  const int nvec = dim / EPV;

  int64_t begin = bag_offsets[bag], end = bag_offsets[bag + 1];
  if (begin < 0 || end < begin || end > nnz) {  // never dereference through bad offsets
    if (lg == 0) set_status(status, ANTDT_ERR_BAD_OFFSETS);
    end = begin = 0;
  }
  const int len = (int)(end - begin);
  const int32_t* ids = row_ids + begin;
  const uint32_t limit = (uint32_t)n_rows;

  uint64_t acc[VPL][PAIRS];  // fp32 sums as packed pairs
#pragma unroll
  for (int k = 0; k < VPL; ++k)
#pragma unroll
    for (int e = 0; e < PAIRS; ++e) acc[k][e] = 0ull;

  const char* tbl = static_cast<const char*>(table);
  const uint32_t row_bytes = (uint32_t)dim * (BF16 ? 2u : 4u);

  for (int base = 0; base < len; base += G) {
    // G ids of the bag in one coalesced load; -1 marks "no row" (past the end, or out of range)
    int my_id = -1;
    if (base + lg < len) {
      my_id = __ldg(ids + base + lg);
      if ((uint32_t)my_id >= limit) {
        set_status(status, ANTDT_ERR_ID_OUT_OF_RANGE);
        my_id = -1;  // skipped: contributes nothing
      }
    }
#pragma unroll
    for (int j0 = 0; j0 < G; j0 += U) {
      if (base + j0 >= len) break;
      uint4 v[U][VPL];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int id = __shfl_sync(gmask, my_id, j0 + u, G);
        const uint4* rp = reinterpret_cast<const uint4*>(tbl + (size_t)(uint32_t)(id < 0 ? 0 : id) * row_bytes);
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          const int vi = lg + k * G;
          v[u][k] = (id >= 0 && vi < nvec) ? __ldg(rp + vi) : make_uint4(0u, 0u, 0u, 0u);
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          if (BF16) {  // bf16 -> fp32 is a 16-bit shift; a zero vector adds +0.0
            acc[k][0] = f32x2_add(acc[k][0], f32x2_pack(v[u][k].x << 16, v[u][k].x & 0xffff0000u));
            acc[k][1] = f32x2_add(acc[k][1], f32x2_pack(v[u][k].y << 16, v[u][k].y & 0xffff0000u));
            acc[k][2] = f32x2_add(acc[k][2], f32x2_pack(v[u][k].z << 16, v[u][k].z & 0xffff0000u));
            acc[k][3] = f32x2_add(acc[k][3], f32x2_pack(v[u][k].w << 16, v[u][k].w & 0xffff0000u));
          } else {
            acc[k][0] = f32x2_add(acc[k][0], f32x2_pack(v[u][k].x, v[u][k].y));
            acc[k][1] = f32x2_add(acc[k][1], f32x2_pack(v[u][k].z, v[u][k].w));
          }
        }
      }
    }
  }

  float* out = pooled + bag * (int64_t)dim;
#pragma unroll
  for (int k = 0; k < VPL; ++k) {
    const int vi = lg + k * G;
    if (vi >= nvec) continue;
    ulonglong2* o = reinterpret_cast<ulonglong2*>(out + (size_t)vi * EPV);
    o[0] = make_ulonglong2(acc[k][0], acc[k][1]);
    if (BF16) o[1] = make_ulonglong2(acc[k][2], acc[k][3]);
  }
}

template <int G, int VPL, bool BF16>
void launch_fwd(const void* table, int64_t n_rows, int dim, const int32_t* row_ids, int64_t nnz,
                const int64_t* bag_offsets, int64_t n_bags, float* pooled, int32_t* status,
                cudaStream_t s, int fields) {
  const int64_t gpb = kFwdThreads / G;
  int64_t grid = (n_bags + gpb - 1) / gpb, sample_blocks = 0;
  if (fields > 0 && n_bags % fields == 0) {
    sample_blocks = (n_bags / fields + gpb - 1) / gpb;
    grid = sample_blocks * fields;
  } else {
    fields = 0;
  }
  if (fields > 0)
    ANTDT_LAUNCH("embbag_fwd", (embbag_fwd_kernel<G, VPL, BF16, true>), (unsigned)grid, kFwdThreads, 0, s,
                 table, n_rows, dim, row_ids, nnz, bag_offsets, n_bags, pooled, status, fields, sample_blocks);
  else
    ANTDT_LAUNCH("embbag_fwd", (embbag_fwd_kernel<G, VPL, BF16, false>), (unsigned)grid, kFwdThreads, 0, s,
                 table, n_rows, dim, row_ids, nnz, bag_offsets, n_bags, pooled, status, fields, sample_blocks);
}

template <bool BF16>
int32_t dispatch_fwd(int nvec, const void* table, int64_t n_rows, int dim, const int32_t* row_ids,
                     int64_t nnz, const int64_t* bag_offsets, int64_t n_bags, float* pooled,
                     int32_t* status, cudaStream_t s, int fields) {
#define FWD_CASE(G, VPL)                                                                      \
  launch_fwd<G, VPL, BF16>(table, n_rows, dim, row_ids, nnz, bag_offsets, n_bags, pooled,     \
                           status, s, fields);                                                \
  return ANTDT_OK;
  if (nvec <= 1) { FWD_CASE(1, 1) }
  if (nvec <= 2) { FWD_CASE(2, 1) }
  if (nvec <= 4) { FWD_CASE(4, 1) }
  if (nvec <= 8) { FWD_CASE(8, 1) }
  if (nvec <= 16) { FWD_CASE(16, 1) }
  if (nvec <= 32) { FWD_CASE(32, 1) }
  if (nvec <= 64) { FWD_CASE(32, 2) }
  if (nvec <= 128) { FWD_CASE(32, 4) }
  if (nvec <= 256) { FWD_CASE(32, 8) }
#undef FWD_CASE
  return ANTDT_ERR_INVALID_ARG;
}

}  // namespace
}  // namespace antdt

namespace antdt {
// The entry point's body; bags_per_sample > 0 (the step knows it) selects the field-major order.
int32_t fwd_impl(const void* table, int32_t dtype, int64_t n_rows, int32_t dim, const int32_t* row_ids,
                 int64_t nnz, const int64_t* bag_offsets, int64_t n_bags, float* pooled,
                 int32_t* dev_status, void* stream, int32_t bags_per_sample) {
  if (n_bags < 0 || nnz < 0 || n_rows < 1 || n_rows >= (1ll << 31) || nnz >= (1ll << 31) ||
      n_bags >= (1ll << 31) || dim < 1 || dim > 1024)
    return ANTDT_ERR_INVALID_ARG;
  if (dtype != ANTDT_F32 && dtype != ANTDT_BF16) return ANTDT_ERR_INVALID_ARG;
  if (dim % (dtype == ANTDT_BF16 ? 8 : 4)) return ANTDT_ERR_INVALID_ARG;
  if (n_bags == 0) return ANTDT_OK;
  if (!table || !bag_offsets || !pooled || (nnz > 0 && !row_ids)) return ANTDT_ERR_INVALID_ARG;
  if (!aligned16(table) || !aligned16(pooled)) return ANTDT_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  // Field-major order pays when a bag's id list fills a 32-byte sector (eight ids or more on
  // average): measured -12% on 100 fields x 10 ids x 256-byte rows, -2% on 40 x 20 x 128-byte rows,
  // but +8% on 30 fields x 4.5 ids, where the scattered id reads cost more than the rows gain.
  const int fields = (bags_per_sample > 1 && nnz >= 8 * n_bags) ? bags_per_sample : 0;
  int32_t rc;
  if (dtype == ANTDT_BF16)
    rc = dispatch_fwd<true>(dim / 8, table, n_rows, dim, row_ids, nnz, bag_offsets, n_bags, pooled,
                            dev_status, s, fields);
  else
    rc = dispatch_fwd<false>(dim / 4, table, n_rows, dim, row_ids, nnz, bag_offsets, n_bags,
                             pooled, dev_status, s, fields);
  if (rc != ANTDT_OK) return rc;
  return cuda_ok();
}
}  // namespace antdt

extern "C" int32_t antdt_embbag_fwd(const void* table, int32_t dtype, int64_t n_rows, int32_t dim,
                                    const int32_t* row_ids, int64_t nnz,
                                    const int64_t* bag_offsets, int64_t n_bags, float* pooled,
                                    int32_t* dev_status, void* stream) {
  return antdt::fwd_impl(table, dtype, n_rows, dim, row_ids, nnz, bag_offsets, n_bags, pooled,
                         dev_status, stream, 0);
}
