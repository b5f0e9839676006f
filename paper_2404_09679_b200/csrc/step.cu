// One whole BSP step from host buffers: stage in, run the four device calls, stage out.
#include "common.cuh"

extern "C" int32_t antdt_bsp_step_host(const antdt_step_desc* d, void* stream) {
  if (!d) return ANTDT_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t D = (size_t)d->dim;
  if (d->nnz < 0 || d->n_bags < 0 || d->dim < 1 || !d->h_bag_offsets || !d->d_bag_offsets ||
      !d->d_status || !d->h_status || !d->d_n_agg || !d->h_n_agg)
    return ANTDT_ERR_INVALID_ARG;
  if (d->nnz > 0 && (!d->h_row_ids || !d->d_row_ids || !d->h_d_pooled || !d->d_d_pooled))
    return ANTDT_ERR_INVALID_ARG;
  const bool dense = d->h_dense_grads && d->dense_n > 0;
  if (dense && (!d->d_dense_grads || !d->d_dense_out || !d->h_dense_out)) return ANTDT_ERR_INVALID_ARG;

#define CK(x) do { if ((x) != cudaSuccess) return ANTDT_ERR_CUDA; } while (0)
  CK(cudaMemsetAsync(d->d_status, 0, 4, s));
  CK(cudaMemcpyAsync(d->d_bag_offsets, d->h_bag_offsets, 8 * ((size_t)d->n_bags + 1),
                     cudaMemcpyHostToDevice, s));
  if (d->nnz > 0)
    CK(cudaMemcpyAsync(d->d_row_ids, d->h_row_ids, 4 * (size_t)d->nnz, cudaMemcpyHostToDevice, s));
  int32_t rc = antdt_embbag_fwd(d->table, d->dtype, d->n_rows, d->dim, d->d_row_ids, d->nnz,
                                d->d_bag_offsets, d->n_bags, d->d_pooled_out, d->d_status, stream);
  if (rc != ANTDT_OK) return rc;
  if (d->h_pooled && d->n_bags > 0)
    CK(cudaMemcpyAsync(d->h_pooled, d->d_pooled_out, 4 * (size_t)d->n_bags * D,
                       cudaMemcpyDeviceToHost, s));
  if (d->n_bags > 0)
    CK(cudaMemcpyAsync(d->d_d_pooled, d->h_d_pooled, 4 * (size_t)d->n_bags * D,
                       cudaMemcpyHostToDevice, s));
  rc = antdt_embbag_bwd_dedup(d->d_row_ids, d->nnz, d->d_bag_offsets, d->n_bags, d->bags_per_sample,
                              d->d_d_pooled, d->dim, d->n_rows, d->n_workers,
                              d->worker_sample_offsets, d->d_uniq_ids, d->d_worker_uniq_offsets,
                              d->d_seg_offsets, d->d_sorted_occ, d->d_uniq_grads, d->uniq_cap, d->ws,
                              d->ws_bytes, d->d_status, stream);
  if (rc != ANTDT_OK) return rc;
  if (dense)
    CK(cudaMemcpyAsync(d->d_dense_grads, d->h_dense_grads,
                       4 * (size_t)d->n_workers * (size_t)d->dense_n, cudaMemcpyHostToDevice, s));
  antdt_sparse_part sp;
  sp.dim = d->dim; sp.n_rows = d->n_rows; sp.uniq_ids = d->d_uniq_ids;
  sp.worker_uniq_offsets = d->d_worker_uniq_offsets; sp.uniq_grads = d->d_uniq_grads;
  sp.in_cap = d->uniq_cap; sp.agg_ids = d->d_agg_ids; sp.agg_grads = d->d_agg_grads;
  sp.n_agg = d->d_n_agg; sp.out_cap = d->agg_cap;
  antdt_dense_part dp;
  dp.grads = d->d_dense_grads; dp.n = d->dense_n; dp.stride = d->dense_n; dp.out = d->d_dense_out;
  rc = antdt_weighted_aggregate(&sp, dense ? &dp : nullptr, d->batch_sizes, d->n_workers, d->ws,
                                d->ws_bytes, d->d_status, stream);
  if (rc != ANTDT_OK) return rc;
  rc = antdt_sparse_opt_update(d->table, d->dtype, d->n_rows, d->dim, d->d_agg_ids, d->d_agg_grads,
                               d->d_n_agg, d->agg_cap, d->opt, d->lr, d->eps, d->beta1, d->beta2,
                               d->step, d->state0, d->state1, d->d_status, stream);
  if (rc != ANTDT_OK) return rc;
  if (dense)
    CK(cudaMemcpyAsync(d->h_dense_out, d->d_dense_out, 4 * (size_t)d->dense_n,
                       cudaMemcpyDeviceToHost, s));
  CK(cudaMemcpyAsync(d->h_n_agg, d->d_n_agg, 8, cudaMemcpyDeviceToHost, s));
  CK(cudaMemcpyAsync(d->h_status, d->d_status, 4, cudaMemcpyDeviceToHost, s));
#undef CK
  return ANTDT_OK;
}
