// One whole BSP step from host buffers: stage in, run the four device calls, stage out.
#include <string.h>

#include <mutex>
#include <vector>

#include "agg_range.cuh"
#include "common.cuh"
#include "segsort.cuh"

namespace antdt {
// The server half of a step: aggregate, then update; in one pass when the descriptor asks for it.
static int32_t server_step(const antdt_step_desc* d, antdt_sparse_part* sp, const antdt_dense_part* dp,
                           void* stream, const OrderFork* fork = nullptr, size_t ws_skip = 0) {
  if (d->fuse_update && (d->opt == ANTDT_OPT_ADAGRAD || d->opt == ANTDT_OPT_ADAM)) {
    if (d->n_workers <= kRangeMaxWorkers) sp->agg_grads = nullptr;  // not materialised
    return aggregate_update_forked(sp, dp, d->batch_sizes, d->n_workers, d->table, d->dtype, d->opt,
                                   d->lr, d->eps, d->beta1, d->beta2, d->step, d->state0, d->state1,
                                   static_cast<char*>(d->ws) + ws_skip, d->ws_bytes - ws_skip,
                                   d->d_status, stream, fork);
  }
  // a forked step keeps the aggregation's scratch behind the backward's (both are live at once)
  int32_t rc = weighted_aggregate_forked(sp, dp, d->batch_sizes, d->n_workers,
                                         static_cast<char*>(d->ws) + ws_skip, d->ws_bytes - ws_skip,
                                         d->d_status, stream, fork);
  if (rc != ANTDT_OK) return rc;
  return antdt_sparse_opt_update(d->table, d->dtype, d->n_rows, d->dim, d->d_agg_ids, d->d_agg_grads,
                                 d->d_n_agg, d->agg_cap, d->opt, d->lr, d->eps, d->beta1, d->beta2,
                                 d->step, d->state0, d->state1, d->d_status, stream);
}
}  // namespace antdt

namespace {
// Side streams and events of the host-buffer step, created on first use for each device.
constexpr int kMaxPieces = 16;  // the d_pooled copy is cut into at most this many pieces
struct StepStreams {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaStream_t side_fwd = nullptr, side_order = nullptr;  // branches of a forked device step
  cudaEvent_t start, ids, dense, fwd, done, outdone;
  cudaEvent_t fork, fwd_done, ids_done, order_done;
  cudaEvent_t piece[kMaxPieces];
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
    if (cudaStreamCreateWithFlags(&ss.side_fwd, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&ss.side_order, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    cudaEvent_t* ev[] = {&ss.start, &ss.ids, &ss.dense, &ss.fwd, &ss.done, &ss.outdone,
                         &ss.fork, &ss.fwd_done, &ss.ids_done, &ss.order_done};
    for (cudaEvent_t* e : ev)
      if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    for (cudaEvent_t& e : ss.piece)
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
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
  // inputs: everything earlier on the caller's stream first (the staging buffers are reused),
  // unless the caller vouches that this descriptor's set is idle: then the copies start at once
  // and run under whatever the stream is still computing (the previous step)
  if (!d->staging_idle) {
    CK(cudaEventRecord(ss->start, s));
    CK(cudaStreamWaitEvent(ss->in, ss->start, 0));
    CK(cudaStreamWaitEvent(ss->out, ss->start, 0));
  }
  CK(cudaMemcpyAsync(d->d_bag_offsets, d->h_bag_offsets, 8 * ((size_t)d->n_bags + 1),
                     cudaMemcpyHostToDevice, ss->in));
  if (d->nnz > 0)
    CK(cudaMemcpyAsync(d->d_row_ids, d->h_row_ids, 4 * (size_t)d->nnz, cudaMemcpyHostToDevice,
                       ss->in));
  CK(cudaEventRecord(ss->ids, ss->in));
  // d_pooled is the largest input and the backward's reduction is the first to read it: it is
  // copied in pieces of whole workers, each with its own event, so that the reduction of a
  // worker's occurrences starts when that worker's rows are there (only the last piece's
  // reduction is left once the copy ends).  Small inputs travel as one piece.
  int n_pieces = 0;
  int64_t piece_entry_end[kMaxPieces];
  if (d->n_bags > 0) {
    const int K = d->n_workers;
    const int64_t F = d->bags_per_sample;
    const size_t row_bytes = 4 * D;
    const bool cut = K > 1 && F > 0 && d->worker_sample_offsets &&
                     (size_t)d->n_bags * row_bytes >= ((size_t)8 << 20);
    const int want = cut ? (K < kMaxPieces ? K : kMaxPieces) : 1;
    int64_t bag0 = 0;
    int w0 = 0;
    for (int c = 0; c < want; ++c) {
      // workers [w0, w1): an equal share of the workers per piece, the last piece takes the rest
      const int w1 = c + 1 == want ? K : (int)(((int64_t)(c + 1) * K) / want);
      int64_t bag1 = c + 1 == want ? d->n_bags : d->worker_sample_offsets[w1] * F;
      if (bag1 < bag0) bag1 = bag0;
      if (bag1 > d->n_bags) bag1 = d->n_bags;
      if (bag1 > bag0)
        CK(cudaMemcpyAsync(d->d_d_pooled + (size_t)bag0 * D, d->h_d_pooled + (size_t)bag0 * D,
                           (size_t)(bag1 - bag0) * row_bytes, cudaMemcpyHostToDevice, ss->in));
      CK(cudaEventRecord(ss->piece[c], ss->in));
      int64_t e = d->h_bag_offsets[bag1];  // occurrences before the piece's end (host copy)
      if (e < 0) e = 0;
      if (e > d->nnz) e = d->nnz;
      piece_entry_end[c] = e;
      bag0 = bag1;
      w0 = w1;
    }
    (void)w0;
    n_pieces = want;
  }
  if (dense)
    CK(cudaMemcpyAsync(d->d_dense_grads, d->h_dense_grads,
                       4 * (size_t)d->n_workers * (size_t)d->dense_n, cudaMemcpyHostToDevice,
                       ss->in));
  CK(cudaEventRecord(ss->dense, ss->in));

  // compute on the caller's stream
  CK(cudaMemsetAsync(d->d_status, 0, 4, s));
  CK(cudaStreamWaitEvent(s, ss->ids, 0));
  int32_t rc = antdt::fwd_impl(d->table, d->dtype, d->n_rows, d->dim, d->d_row_ids, d->nnz,
                               d->d_bag_offsets, d->n_bags, d->d_pooled_out, d->d_status, stream,
                               d->bags_per_sample);
  if (rc != ANTDT_OK) return rc;
  CK(cudaEventRecord(ss->fwd, s));
  CK(cudaStreamWaitEvent(ss->out, ss->fwd, 0));
  if (d->h_pooled && d->n_bags > 0)
    CK(cudaMemcpyAsync(d->h_pooled, d->d_pooled_out, 4 * (size_t)d->n_bags * D,
                       cudaMemcpyDeviceToHost, ss->out));
  antdt::PooledArrival arrival{n_pieces, piece_entry_end, ss->piece};
  rc = antdt::bwd_dedup_impl(d->d_row_ids, d->nnz, d->d_bag_offsets, d->n_bags, d->bags_per_sample,
                              d->d_d_pooled, d->dim, d->n_rows, d->n_workers,
                              d->worker_sample_offsets, d->d_uniq_ids, d->d_worker_uniq_offsets,
                              d->d_seg_offsets, d->d_sorted_occ, d->d_uniq_grads, d->uniq_cap, d->ws,
                              d->ws_bytes, d->d_status, stream, n_pieces > 0 ? &arrival : nullptr);
  if (rc != ANTDT_OK) return rc;
  CK(cudaStreamWaitEvent(s, ss->dense, 0));
  antdt_sparse_part sp;
  sp.dim = d->dim; sp.n_rows = d->n_rows; sp.uniq_ids = d->d_uniq_ids;
  sp.worker_uniq_offsets = d->d_worker_uniq_offsets; sp.uniq_grads = d->d_uniq_grads;
  sp.in_cap = d->uniq_cap; sp.agg_ids = d->d_agg_ids; sp.agg_grads = d->d_agg_grads;
  sp.n_agg = d->d_n_agg; sp.out_cap = d->agg_cap;
  antdt_dense_part dp;
  dp.grads = d->d_dense_grads; dp.n = d->dense_n; dp.stride = d->dense_n; dp.out = d->d_dense_out;
  rc = antdt::server_step(d, &sp, dense ? &dp : nullptr, stream);
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
// the status word is left as the caller set it.
//
// forked: the step as three chains instead of one.  The forward needs nothing from the backward,
// and the aggregation's merge order needs the workers' id lists but not their gradients, so both
// run on side streams beside the backward (fork and join by events; in a capture they become
// parallel branches of the graph).  It pays on small batches, where no kernel fills the device
// and the step time is the length of the dependency chain; it needs the aggregation's scratch
// behind the backward's instead of on top of it.
namespace {
constexpr int64_t kForkMaxNnz = (int64_t)1 << 22;

size_t fork_ws_skip(const antdt_step_desc* d) {  // 0: no room (or no reason) to fork
  if (d->nnz < 1 || d->nnz > kForkMaxNnz || d->n_workers > antdt::kRangeMaxWorkers ||
      d->uniq_cap < 1)
    return 0;
  const size_t b = antdt_embbag_bwd_dedup_workspace_bytes(d->nnz, d->n_bags, d->dim, d->n_workers);
  const size_t a = antdt_weighted_aggregate_workspace_bytes(d->uniq_cap, d->dim, d->n_workers);
  const size_t skip = (b + 255) / 256 * 256;
  if (b == 0 || a == 0 || d->ws_bytes < skip + a) return 0;
  return skip;
}

int32_t device_step(const antdt_step_desc* d, void* stream, bool forked) {
  if (!d || d->nnz < 0 || d->n_bags < 0 || d->dim < 1 || !d->d_bag_offsets || !d->d_n_agg)
    return ANTDT_ERR_INVALID_ARG;
  const bool dense = d->d_dense_grads && d->dense_n > 0;
  if (dense && !d->d_dense_out) return ANTDT_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  StepStreams* ss = nullptr;
  size_t ws_skip = 0;
  if (forked && (ws_skip = fork_ws_skip(d)) > 0) ss = step_streams();
  if (!ss) ws_skip = 0;
#define CK(x) do { if ((x) != cudaSuccess) return ANTDT_ERR_CUDA; } while (0)
  void* fwd_stream = stream;
  if (ss) {
    CK(cudaEventRecord(ss->fork, s));
    CK(cudaStreamWaitEvent(ss->side_fwd, ss->fork, 0));
    fwd_stream = ss->side_fwd;
  }
  int32_t rc = antdt::fwd_impl(d->table, d->dtype, d->n_rows, d->dim, d->d_row_ids, d->nnz,
                               d->d_bag_offsets, d->n_bags, d->d_pooled_out, d->d_status, fwd_stream,
                               d->bags_per_sample);
  if (ss) CK(cudaEventRecord(ss->fwd_done, ss->side_fwd));  // joined below even after an error
  if (rc == ANTDT_OK)
    rc = antdt::bwd_dedup_impl(d->d_row_ids, d->nnz, d->d_bag_offsets, d->n_bags, d->bags_per_sample,
                               d->d_d_pooled, d->dim, d->n_rows, d->n_workers,
                               d->worker_sample_offsets, d->d_uniq_ids, d->d_worker_uniq_offsets,
                               d->d_seg_offsets, d->d_sorted_occ, d->d_uniq_grads, d->uniq_cap, d->ws,
                               d->ws_bytes, d->d_status, stream, nullptr, ss ? ss->ids_done : nullptr);
  // the update writes the table the forward reads
  if (ss) CK(cudaStreamWaitEvent(s, ss->fwd_done, 0));
  if (rc != ANTDT_OK) return rc;
  antdt_sparse_part sp;
  sp.dim = d->dim; sp.n_rows = d->n_rows; sp.uniq_ids = d->d_uniq_ids;
  sp.worker_uniq_offsets = d->d_worker_uniq_offsets; sp.uniq_grads = d->d_uniq_grads;
  sp.in_cap = d->uniq_cap; sp.agg_ids = d->d_agg_ids; sp.agg_grads = d->d_agg_grads;
  sp.n_agg = d->d_n_agg; sp.out_cap = d->agg_cap;
  antdt_dense_part dp;
  dp.grads = d->d_dense_grads; dp.n = d->dense_n; dp.stride = d->dense_n; dp.out = d->d_dense_out;
  antdt::OrderFork fork;
  if (ss) fork = antdt::OrderFork{ss->side_order, ss->ids_done, ss->order_done};
  return antdt::server_step(d, &sp, dense ? &dp : nullptr, stream, ss ? &fork : nullptr, ws_skip);
#undef CK
}
}  // namespace

extern "C" int32_t antdt_bsp_step_device(const antdt_step_desc* d, void* stream) {
  return device_step(d, stream, false);
}

extern "C" size_t antdt_bsp_step_workspace_bytes(int64_t nnz, int64_t n_bags, int32_t dim,
                                                 int32_t n_workers, int64_t uniq_cap) {
  const size_t b = antdt_embbag_bwd_dedup_workspace_bytes(nnz, n_bags, dim, n_workers);
  const size_t a = antdt_weighted_aggregate_workspace_bytes(uniq_cap, dim, n_workers);
  if (b == 0 || a == 0) return 0;
  if (nnz <= kForkMaxNnz && n_workers <= antdt::kRangeMaxWorkers) return (b + 255) / 256 * 256 + a;
  return b > a ? b : a;
}

// ---------------------------------------------------------------------------------------
// The device-resident step replayed as a CUDA graph.
// A step is 30-40 short launches; on small batches the launches, not the kernels, are the step
// time.  The four calls are captured once per distinct descriptor and replayed with a single
// graph launch.  Everything a captured launch depends on is in the key: every scalar and device
// pointer of the descriptor and the CONTENTS of the two host arrays (they reach the device as
// kernel parameters).  What the pointers point at may change freely between replays.
// ---------------------------------------------------------------------------------------
namespace {
constexpr size_t kGraphSlots = 8;  // executable graphs kept per device

struct GraphEntry {
  std::vector<uint64_t> key;
  cudaGraphExec_t exec = nullptr;
  int64_t n_kernels = 0;
  uint64_t tick = 0;
};
struct GraphCache {
  std::vector<GraphEntry> entries;
  uint64_t tick = 0;
};
GraphCache g_gc[64];
std::mutex g_gc_mu;

uint64_t bits_of(const void* p) { return (uint64_t)reinterpret_cast<uintptr_t>(p); }
uint64_t bits_of(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }

std::vector<uint64_t> graph_key(const antdt_step_desc* d) {
  std::vector<uint64_t> k;
  const int K = d->n_workers;
  k.reserve(48 + 2 * (size_t)K);
  const uint64_t head[] = {
      bits_of(d->table), (uint64_t)d->dtype, (uint64_t)d->n_rows, (uint64_t)d->dim,
      bits_of(d->state0), bits_of(d->state1), (uint64_t)d->opt, bits_of(d->lr), bits_of(d->eps),
      bits_of(d->beta1), bits_of(d->beta2),
      (uint64_t)(d->step >= 1),  // the Adagrad variants do not use the step number
      (uint64_t)d->nnz, (uint64_t)d->n_bags, (uint64_t)d->bags_per_sample, (uint64_t)d->dense_n,
      (uint64_t)K, bits_of(d->d_row_ids), bits_of(d->d_bag_offsets), bits_of(d->d_pooled_out),
      bits_of(d->d_d_pooled), bits_of(d->d_dense_grads), bits_of(d->d_dense_out),
      bits_of(d->d_uniq_ids), bits_of(d->d_worker_uniq_offsets), bits_of(d->d_seg_offsets),
      bits_of(d->d_sorted_occ), bits_of(d->d_uniq_grads), (uint64_t)d->uniq_cap,
      bits_of(d->d_agg_ids), bits_of(d->d_agg_grads), bits_of(d->d_n_agg), (uint64_t)d->agg_cap,
      bits_of(d->ws), (uint64_t)d->ws_bytes, bits_of(d->d_status), (uint64_t)(d->fuse_update != 0)};
  k.assign(head, head + sizeof(head) / sizeof(head[0]));
  for (int i = 0; i <= K; ++i) k.push_back((uint64_t)d->worker_sample_offsets[i]);
  for (int i = 0; i < K; ++i) k.push_back((uint64_t)d->batch_sizes[i]);
  return k;
}
}  // namespace

extern "C" int32_t antdt_bsp_step_graph(const antdt_step_desc* d, void* stream) {
  if (!d || d->n_workers < 1 || d->n_workers > antdt::kMaxSegments || !d->worker_sample_offsets ||
      !d->batch_sizes)
    return ANTDT_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &cs) != cudaSuccess) {
    cudaGetLastError();
    return ANTDT_ERR_CUDA;
  }
  // inside somebody else's capture the launches simply join that graph
  if (cs != cudaStreamCaptureStatusNone) return antdt_bsp_step_device(d, stream);
  // Adam's bias corrections depend on the step number and travel as kernel parameters, so no two
  // steps share a graph: a capture per step would cost more than the launches it replaces
  if (d->opt == ANTDT_OPT_ADAM) return antdt_bsp_step_device(d, stream);
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ANTDT_ERR_CUDA;
  const std::vector<uint64_t> key = graph_key(d);

  std::lock_guard<std::mutex> lk(g_gc_mu);
  GraphCache& gc = g_gc[dev];
  ++gc.tick;
  for (GraphEntry& e : gc.entries) {
    if (e.key == key) {
      e.tick = gc.tick;
      if (cudaGraphLaunch(e.exec, s) != cudaSuccess) return ANTDT_ERR_CUDA;
      antdt::count_launches(e.n_kernels);
      return ANTDT_OK;
    }
  }

  // miss: capture the four calls
  antdt::segsort_prepare_device();
  antdt::range_prepare_device();
  if (cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();  // e.g. the legacy default stream cannot be captured: plain launches
    return antdt_bsp_step_device(d, stream);
  }
  const int64_t before = antdt_launch_count();
  antdt::prof_untimed(true);
  const int32_t rc = device_step(d, stream, true);  // forked where the descriptor allows it
  antdt::prof_untimed(false);
  const int64_t n_kernels = antdt_launch_count() - before;
  antdt::count_launches(-n_kernels);  // captured, not run
  cudaGraph_t g = nullptr;
  const cudaError_t ce = cudaStreamEndCapture(s, &g);
  if (rc != ANTDT_OK || ce != cudaSuccess || !g) {
    if (g) cudaGraphDestroy(g);
    cudaGetLastError();
    return rc != ANTDT_OK ? rc : ANTDT_ERR_CUDA;
  }

  GraphEntry* slot = nullptr;
  if (gc.entries.size() < kGraphSlots) {
    gc.entries.emplace_back();
    slot = &gc.entries.back();
  } else {  // least recently used; its executable is updated in place when the shape matches
    slot = &gc.entries[0];
    for (GraphEntry& e : gc.entries)
      if (e.tick < slot->tick) slot = &e;
  }
  if (slot->exec) {
    cudaGraphExecUpdateResultInfo info;
    if (cudaGraphExecUpdate(slot->exec, g, &info) != cudaSuccess) {
      cudaGetLastError();
      cudaGraphExecDestroy(slot->exec);
      slot->exec = nullptr;
    }
  }
  if (!slot->exec && cudaGraphInstantiate(&slot->exec, g, 0) != cudaSuccess) {
    cudaGetLastError();
    cudaGraphDestroy(g);
    slot->exec = nullptr;
    slot->key.clear();
    slot->tick = 0;
    return ANTDT_ERR_CUDA;
  }
  cudaGraphDestroy(g);
  slot->key = key;
  slot->n_kernels = n_kernels;
  slot->tick = gc.tick;
  if (cudaGraphLaunch(slot->exec, s) != cudaSuccess) return ANTDT_ERR_CUDA;
  antdt::count_launches(n_kernels);
  return ANTDT_OK;
}

extern "C" int32_t antdt_bsp_step_graph_reset(void) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ANTDT_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_gc_mu);
  for (GraphEntry& e : g_gc[dev].entries)
    if (e.exec) cudaGraphExecDestroy(e.exec);
  g_gc[dev].entries.clear();
  return ANTDT_OK;
}
