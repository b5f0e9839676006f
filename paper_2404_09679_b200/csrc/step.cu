// One whole BSP step from host buffers: stage in, run the four device calls, stage out.
#include <mutex>

#include "common.cuh"

namespace {
// Side streams and events of the host-buffer step, created on first use for each device.
struct StepStreams {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start, ids, dy, dense, fwd, done, outdone;
};
StepStreams g_ss[64];
std::mutex g_ss_mu;

StepStreams* step_streams() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lk(g_ss_mu);
  StepStreams& ss = g_ss[dev];
  if (!ss.ready) {
    if (cudaStreamCreateWithFlags(&ss.in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&ss.out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    cudaEvent_t* ev[] = {&ss.start, &ss.ids, &ss.dy, &ss.dense, &ss.fwd, &ss.done, &ss.outdone};
    for (cudaEvent_t* e : ev)
      if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    ss.ready = true;
  }
  return &ss;
}
}  // namespace

// The copies run on two side streams so that the host-to-device copy of d_pooled overlaps the
// forward kernel and the device-to-host copy of the pooled output overlaps the backward; the
// caller's stream waits for all of it at the end, so synchronising `stream` is enough.
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
  StepStreams* ss = step_streams();
  if (!ss) return ANTDT_ERR_CUDA;

#define CK(x) do { if ((x) != cudaSuccess) return ANTDT_ERR_CUDA; } while (0)
  // inputs: everything earlier on the caller's stream first (the staging buffers are reused)
  CK(cudaEventRecord(ss->start, s));
  CK(cudaStreamWaitEvent(ss->in, ss->start, 0));
  CK(cudaStreamWaitEvent(ss->out, ss->start, 0));
  CK(cudaMemcpyAsync(d->d_bag_offsets, d->h_bag_offsets, 8 * ((size_t)d->n_bags + 1),
                     cudaMemcpyHostToDevice, ss->in));
  if (d->nnz > 0)
    CK(cudaMemcpyAsync(d->d_row_ids, d->h_row_ids, 4 * (size_t)d->nnz, cudaMemcpyHostToDevice,
                       ss->in));
  CK(cudaEventRecord(ss->ids, ss->in));
  if (d->n_bags > 0)
    CK(cudaMemcpyAsync(d->d_d_pooled, d->h_d_pooled, 4 * (size_t)d->n_bags * D,
                       cudaMemcpyHostToDevice, ss->in));
  CK(cudaEventRecord(ss->dy, ss->in));
  if (dense)
    CK(cudaMemcpyAsync(d->d_dense_grads, d->h_dense_grads,
                       4 * (size_t)d->n_workers * (size_t)d->dense_n, cudaMemcpyHostToDevice,
                       ss->in));
  CK(cudaEventRecord(ss->dense, ss->in));

  // compute on the caller's stream
  CK(cudaMemsetAsync(d->d_status, 0, 4, s));
  CK(cudaStreamWaitEvent(s, ss->ids, 0));
  int32_t rc = antdt_embbag_fwd(d->table, d->dtype, d->n_rows, d->dim, d->d_row_ids, d->nnz,
                                d->d_bag_offsets, d->n_bags, d->d_pooled_out, d->d_status, stream);
  if (rc != ANTDT_OK) return rc;
  CK(cudaEventRecord(ss->fwd, s));
  CK(cudaStreamWaitEvent(ss->out, ss->fwd, 0));
  if (d->h_pooled && d->n_bags > 0)
    CK(cudaMemcpyAsync(d->h_pooled, d->d_pooled_out, 4 * (size_t)d->n_bags * D,
                       cudaMemcpyDeviceToHost, ss->out));
  rc = antdt::bwd_dedup_impl(d->d_row_ids, d->nnz, d->d_bag_offsets, d->n_bags, d->bags_per_sample,
                              d->d_d_pooled, d->dim, d->n_rows, d->n_workers,
                              d->worker_sample_offsets, d->d_uniq_ids, d->d_worker_uniq_offsets,
                              d->d_seg_offsets, d->d_sorted_occ, d->d_uniq_grads, d->uniq_cap, d->ws,
                              d->ws_bytes, d->d_status, stream, ss->dy);
  if (rc != ANTDT_OK) return rc;
  CK(cudaStreamWaitEvent(s, ss->dense, 0));
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
  CK(cudaEventRecord(ss->done, s));

  // results
  CK(cudaStreamWaitEvent(ss->out, ss->done, 0));
  if (dense)
    CK(cudaMemcpyAsync(d->h_dense_out, d->d_dense_out, 4 * (size_t)d->dense_n,
                       cudaMemcpyDeviceToHost, ss->out));
  CK(cudaMemcpyAsync(d->h_n_agg, d->d_n_agg, 8, cudaMemcpyDeviceToHost, ss->out));
  CK(cudaMemcpyAsync(d->h_status, d->d_status, 4, cudaMemcpyDeviceToHost, ss->out));
  CK(cudaEventRecord(ss->outdone, ss->out));
  CK(cudaStreamWaitEvent(s, ss->outdone, 0));
#undef CK
  return ANTDT_OK;
}

// The same four calls for a batch that is already resident in device memory: nothing is copied,
// no side stream is used, the status word is left as the caller set it.
extern "C" int32_t antdt_bsp_step_device(const antdt_step_desc* d, void* stream) {
  if (!d || d->nnz < 0 || d->n_bags < 0 || d->dim < 1 || !d->d_bag_offsets || !d->d_n_agg)
    return ANTDT_ERR_INVALID_ARG;
  const bool dense = d->d_dense_grads && d->dense_n > 0;
  if (dense && !d->d_dense_out) return ANTDT_ERR_INVALID_ARG;
  int32_t rc = antdt_embbag_fwd(d->table, d->dtype, d->n_rows, d->dim, d->d_row_ids, d->nnz,
                                d->d_bag_offsets, d->n_bags, d->d_pooled_out, d->d_status, stream);
  if (rc != ANTDT_OK) return rc;
  rc = antdt_embbag_bwd_dedup(d->d_row_ids, d->nnz, d->d_bag_offsets, d->n_bags, d->bags_per_sample,
                              d->d_d_pooled, d->dim, d->n_rows, d->n_workers,
                              d->worker_sample_offsets, d->d_uniq_ids, d->d_worker_uniq_offsets,
                              d->d_seg_offsets, d->d_sorted_occ, d->d_uniq_grads, d->uniq_cap, d->ws,
                              d->ws_bytes, d->d_status, stream);
  if (rc != ANTDT_OK) return rc;
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
  return antdt_sparse_opt_update(d->table, d->dtype, d->n_rows, d->dim, d->d_agg_ids, d->d_agg_grads,
                                 d->d_n_agg, d->agg_cap, d->opt, d->lr, d->eps, d->beta1, d->beta2,
                                 d->step, d->state0, d->state1, d->d_status, stream);
}
