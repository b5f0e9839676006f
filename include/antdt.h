/*
 * antdt.h -- C-ABI boundary of the BSP sparse-ranking hot path.
 *
 * One synchronous (BSP) iteration of data-parallel training, as the paper's problem
 * formulation states it (Section II): every worker i of n computes a local gradient on its
 * local batch B_i, the servers aggregate the local gradients of all workers and update the
 * parameters, and the global batch B = sum_i B_i is fixed (Eq. 1).  Here the n workers are
 * simulated on one GPU, the model is the sparse-feature (embedding-bag) part of a ranking
 * model, and the calls below are the steps of that iteration:
 *
 *   antdt_shard_plan         host   Stateful Dynamic Data Sharding (Section V-C) + the
 *                                   ADJUST_BS batch sizes (Section VI-A, Eq. 2-3)
 *   antdt_embbag_fwd         device worker forward: gather + sum pooling
 *   antdt_embbag_bwd_dedup   device worker backward: per-worker dedup of row ids and
 *                                   segmented reduction to mean row gradients
 *   antdt_weighted_aggregate device server: batch-size weighted aggregation (sparse + dense)
 *   antdt_sparse_opt_update  device server: sparse Adagrad / Adam row update
 *
 * Conventions
 *   - Every call returns an int32 status (ANTDT_OK = 0).  Nothing aborts, throws or traps.
 *   - The caller owns every buffer.  Device calls allocate no device memory; scratch is a
 *     caller-provided workspace whose size comes from the matching *_workspace_bytes call.
 *   - "device" pointers are CUDA global memory of the current device; "host" pointers are
 *     ordinary host memory.  `stream` is a cudaStream_t passed as void* (NULL = legacy default
 *     stream).  Device calls are asynchronous on that stream.
 *   - Argument errors that the host can see are returned before anything is launched.
 *     Errors only the device can see (row id outside [0, n_rows), offsets that do not ascend,
 *     output capacity exceeded) are written to the caller's int32 `dev_status` word (first
 *     error wins, the word must be zeroed by the caller before a chain of calls); the
 *     offending element is skipped, never dereferenced.  antdt_read_status fetches it.
 *   - Counts produced on the device stay on the device as int64 so that the chain of calls
 *     needs no host synchronisation.
 *   - Layout: all matrices are row-major and dense ([rows, dim], stride dim).  Bags are a CSR
 *     list: bag b holds row_ids[bag_offsets[b] .. bag_offsets[b+1]).  Bags are ordered
 *     sample-major (sample s, field f -> bag s*bags_per_sample + f) and the samples of worker 0
 *     come first, then worker 1, ... (worker w owns samples
 *     [worker_sample_offsets[w], worker_sample_offsets[w+1])).
 *   - Limits: dim % 4 == 0 (fp32 rows) or dim % 8 == 0 (bf16 rows), dim <= 1024, all row
 *     buffers 16-byte aligned, n_rows < 2^31, nnz < 2^31, n_bags < 2^31, n_workers <= 1024.
 */
#ifndef ANTDT_H
#define ANTDT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ------------------------------------------------------------------- */
enum {
  ANTDT_OK = 0,
  ANTDT_ERR_INVALID_ARG = 1,         /* a host-visible argument is malformed              */
  ANTDT_ERR_ID_OUT_OF_RANGE = 2,     /* device saw a row id outside [0, n_rows)           */
  ANTDT_ERR_WORKSPACE_TOO_SMALL = 3, /* ws_bytes below the *_workspace_bytes figure       */
  ANTDT_ERR_CAPACITY = 4,            /* an output buffer's capacity would be exceeded     */
  ANTDT_ERR_CUDA = 5,                /* a CUDA runtime call or launch failed              */
  ANTDT_ERR_TIMEOUT = 6,             /* a bounded device-side wait ran out                */
  ANTDT_ERR_EXHAUSTED = 7,           /* the shard queue is empty: the epoch is over       */
  ANTDT_ERR_STATE = 8,               /* call not valid in the handle's current state      */
  ANTDT_ERR_BAD_OFFSETS = 9,         /* device saw bag offsets (or sorted id lists) that
                                        do not ascend / fit                               */
  ANTDT_ERR_INFEASIBLE = 10          /* a planning problem has no feasible point          */
};

enum { ANTDT_F32 = 0, ANTDT_BF16 = 1 };                  /* table row element type        */
enum { ANTDT_RULE_PROPORTIONAL = 0, ANTDT_RULE_MINMAX = 1 };
enum { ANTDT_OPT_ADAGRAD = 0, ANTDT_OPT_ADAM = 1, ANTDT_OPT_ROWWISE_ADAGRAD = 2 };
enum { ANTDT_SHARD_TODO = 0, ANTDT_SHARD_DOING = 1, ANTDT_SHARD_DONE = 2 };

/* ===================================================================================== */
/* Host planner: Stateful Dynamic Data Sharding + batch-size adjustment                  */
/* ===================================================================================== */

/* A contiguous run of dataset sample indices [start, start+len).  Section V-C.1: a shard
 * (and so every piece of one) is just two integers, start offset and length. */
typedef struct { int64_t start, len; } antdt_range;

typedef struct antdt_dds antdt_dds; /* opaque; host memory owned by the library */

/* Section V-C.1.  Splits n_samples samples into ceil(n_samples / (global_batch *
 * batches_per_shard)) shards of global_batch*batches_per_shard consecutive samples (the last
 * one shorter), all in state TODO, and queues them in index order; shuffle_seed != 0 permutes
 * the queue with a seeded Fisher-Yates (the Shard Shuffler's permutation of whole shards).
 * *out receives the handle; release it with antdt_dds_destroy.
 * INVALID_ARG: NULL out, n_samples < 1, global_batch < 1, batches_per_shard < 1,
 * n_workers outside [1, 1024]. */
int32_t antdt_dds_create(antdt_dds** out, int64_t n_samples, int64_t global_batch,
                         int32_t batches_per_shard, int32_t n_workers, uint64_t shuffle_seed);
void antdt_dds_destroy(antdt_dds* dds);

/* Batch sizes alone (stateless).  Section VI-A: first iteration B_i = B/n (speeds == NULL,
 * remainder to the lowest worker indices); afterwards ADJUST_BS solves Eq. 3,
 *     min z  s.t.  z >= B_i / v_i,  sum_i B_i = B,
 * with v_i the worker throughputs.  rule PROPORTIONAL: B_i = B*v_i/sum(v) rounded by largest
 * remainder (ties to the lower index), workers whose share is below min_batch pinned to
 * min_batch and the rest re-shared.  rule MINMAX: the exact integer optimum of Eq. 3 with
 * B_i >= min_batch, built one sample at a time (each unit goes to the worker with the
 * smallest (B_i+1)/v_i, ties to the lower index).
 * speeds: host [n_workers] or NULL; batch_sizes: host out [n_workers], sums to global_batch.
 * INVALID_ARG: a speed that is not finite and > 0, min_batch < 0,
 * min_batch*n_workers > global_batch, unknown rule. */
int32_t antdt_batch_sizes(const double* speeds, int32_t n_workers, int64_t global_batch,
                          int32_t rule, int64_t min_batch, int64_t* batch_sizes);

/* One BSP step of the data service (Sections V-C.1 to V-C.3).  Computes this step's batch
 * sizes as antdt_batch_sizes does, then serves each worker, in ascending worker index, its
 * batch_sizes[i] samples from the shard it currently holds; a worker whose shard runs out
 * fetches the TODO shard at the head of the queue (it becomes DOING and cannot go to anyone
 * else) and goes on, so a worker's step is a short list of ranges.  A shard whose last sample
 * was served is DONE when the call returns (the step's gradients count as pushed) unless
 * antdt_dds_requeue_worker reports, before the next antdt_shard_plan, that the worker's push
 * failed.  When the queue is empty a worker's step is short: counts[i] < batch_sizes[i].
 *   batch_sizes   host out [K]   planned sizes, sum = global_batch
 *   range_offsets host out [K+1] CSR offsets into ranges
 *   ranges        host out [ranges_cap]
 *   counts        host out [K]   samples actually served (= batch_sizes off the epoch tail)
 * Returns EXHAUSTED (and all counts 0) when nothing is left to serve, CAPACITY (state
 * unchanged) when ranges_cap is too small, INVALID_ARG as antdt_batch_sizes. */
int32_t antdt_shard_plan(antdt_dds* dds, const double* speeds, int32_t rule, int64_t min_batch,
                         int64_t* batch_sizes, int64_t* range_offsets, antdt_range* ranges,
                         int64_t ranges_cap, int64_t* counts);

/* Section V-C.3, last paragraph: the shards of a lost worker (BACKUP_WORKERS drop,
 * KILL_RESTART) go back to TODO at the END of the queue and will be served again in full
 * (at-least-once): first every shard whose last sample the latest antdt_shard_plan call served
 * to this worker (a shard is DONE only once its gradients are pushed, and this worker's were
 * not), in the order it finished them, then the shard it is DOING.  Call it between the plan
 * call whose gradients were lost and the next one; later, only the DOING shard is returned.
 * No-op if the worker holds and finished nothing. */
int32_t antdt_dds_requeue_worker(antdt_dds* dds, int32_t worker);

/* Shard bookkeeping used by the integrity checks (Section VII-D: #DONE = ceil(N/(B*M))). */
int64_t antdt_dds_num_shards(const antdt_dds* dds);
int32_t antdt_dds_counts(const antdt_dds* dds, int64_t* todo, int64_t* doing, int64_t* done);
/* state: ANTDT_SHARD_*; owner: worker holding it or -1; r: the shard's (start, len). */
int32_t antdt_dds_shard_info(const antdt_dds* dds, int64_t shard, int32_t* state,
                             int32_t* owner, antdt_range* r);
/* Serialise / restore the whole service state (the "data reading state" a checkpoint holds,
 * Section VII-D.3).  save with buf == NULL only reports the size in *used.  load creates a
 * new handle.  CAPACITY if cap is too small, INVALID_ARG on a malformed image. */
int32_t antdt_dds_save(const antdt_dds* dds, void* buf, size_t cap, size_t* used);
int32_t antdt_dds_load(antdt_dds** out, const void* buf, size_t len);

/* ---- controller front end (AntDT-ND, worker side) ------------------------------------ */
enum { ANTDT_ACTION_NONE = 0, ANTDT_ACTION_ADJUST_BS = 1, ANTDT_ACTION_KILL_RESTART = 2 };
typedef struct antdt_ctl antdt_ctl; /* opaque; host memory owned by the library */

/* Section VI-A steps 2-5.  Keeps, per worker, the last window_trans and window_per reports
 * (L^trans, L^per counted in reports), lambda = the slowness ratio (> 1; the paper uses 1.5).
 * antdt_ctl_report: one (batch size, batch processing time in seconds) report of a worker.
 * antdt_ctl_decide (every worker must have reported once, else STATE):
 *   speeds[i]     v_i = mean over worker i's short window of batch_size / BPT of each report
 *                 (the reading taken of the paper's throughput formula)
 *   transient[i]  1 iff mean BPT over the short window >= lambda * (mean of those over workers)
 *   persistent[i] the same over the long window
 *   action        KILL_RESTART if any persistent straggler (the caller decides whether the
 *                 cluster is busy), else ADJUST_BS if any transient one (feed `speeds` to
 *                 antdt_shard_plan), else NONE.
 * All arrays host [n_workers]. */
int32_t antdt_ctl_create(antdt_ctl** out, int32_t n_workers, int32_t window_trans,
                         int32_t window_per, double lambda);
void antdt_ctl_destroy(antdt_ctl* ctl);
int32_t antdt_ctl_report(antdt_ctl* ctl, int32_t worker, int64_t batch_size, double bpt_seconds);
int32_t antdt_ctl_decide(const antdt_ctl* ctl, double* speeds, int32_t* transient,
                         int32_t* persistent, int32_t* action);

/* AntDT-DD, Section VI-B, Eq. 4 (its constraint read with the sum over the k device types):
 *     min max_i C_i * B_i / v_i
 *     s.t. sum_i n_i * C_i * B_i = B,  Bmin_i <= B_i <= Bmax_i,  Cmin <= C_i <= Cmax,
 * all integers: device type i (n_i devices, throughput v_i) runs C_i accumulated micro-batches
 * of B_i samples before the synchronisation.  Exact, by enumeration with pruning (k <= 8; meant
 * for the handful of device types of a heterogeneous cluster); among equal optima the
 * lexicographically smallest (C_1..C_k, B_1..B_k) is returned.  Each device of type i then
 * enters the step with local batch C_i*B_i (accumulating C_i mean gradients of B_i samples is
 * the mean over C_i*B_i samples, so the device path needs nothing else).
 * Host arrays of n_types entries; z_out (may be NULL) receives the optimum.
 * INFEASIBLE when no assignment meets the equality. */
int32_t antdt_dd_solve(int32_t n_types, const int32_t* n_devices, const double* speeds,
                       int64_t global_batch, const int64_t* batch_min, const int64_t* batch_max,
                       int32_t accum_min, int32_t accum_max, int64_t* batch_out, int32_t* accum_out,
                       double* z_out);

/* ===================================================================================== */
/* Device path                                                                           */
/* ===================================================================================== */

/* Worker forward (Section II: the forward part of T_i^w on the local batch B_i), for the
 * sparse part of the model: pooled[b, :] = sum over j in bag b of table[row_ids[j], :].
 * An id repeated inside a bag counts each time; an empty bag gives zeros.  fp32 accumulation
 * in bag order.
 *   table       device [n_rows, dim]  fp32 or bf16 (dtype), read only
 *   row_ids     device [nnz]          int32 row index into table
 *   bag_offsets device [n_bags+1]     int64, ascending, bag_offsets[0] = 0, last = nnz
 *   pooled      device out [n_bags, dim] fp32
 *   dev_status  device int32 word (may be NULL: errors are then only skipped) */
int32_t antdt_embbag_fwd(const void* table, int32_t dtype, int64_t n_rows, int32_t dim,
                         const int32_t* row_ids, int64_t nnz, const int64_t* bag_offsets,
                         int64_t n_bags, float* pooled, int32_t* dev_status, void* stream);

/* Worker backward (Section II: the backpropagation part of T_i^w; each worker produces the
 * gradient of ITS local batch, which it then pushes).  For every worker w separately:
 * the distinct rows its samples touch, ascending (uniq_ids), and for each of them the mean
 * gradient over the worker's b_w = worker_sample_offsets[w+1]-worker_sample_offsets[w] samples,
 *     uniq_grads[u, :] = (1/b_w) * sum over occurrences o of that row in worker w of
 *                         d_pooled[bag(o), :],
 * by a stable radix sort of the occurrences by row id and a segmented sum in sorted order --
 * no floating-point atomics, the result is bit-reproducible from call to call.
 *   d_pooled             device [n_bags, dim] fp32, gradient w.r.t. pooled (per-sample loss)
 *   worker_sample_offsets host  [K+1] int64 ascending, [0] = 0, [K]*bags_per_sample = n_bags
 *   uniq_ids             device out [out_cap] int32, grouped by worker, ascending inside one
 *   worker_uniq_offsets  device out [K+1] int64; worker w's rows are
 *                        [worker_uniq_offsets[w], worker_uniq_offsets[w+1]); [K] = total
 *   seg_offsets          device out [out_cap+1] int64; the occurrences of unique row u are
 *                        sorted positions [seg_offsets[u], seg_offsets[u+1])
 *   sorted_occ           device out [nnz] int32; bag index of each occurrence in sorted order
 *                        (worker, row id, then original position: all three unique)
 *   uniq_grads           device out [out_cap, dim] fp32
 *   out_cap              capacity in rows; nnz always suffices; CAPACITY -> dev_status
 *   ws, ws_bytes         device scratch.  antdt_embbag_bwd_dedup_workspace_bytes(...) is the size
 *                        to allocate; antdt_embbag_bwd_dedup_min_workspace_bytes(...) is the least
 *                        the call accepts (WORKSPACE_TOO_SMALL below it).  The two differ for up to
 *                        2^20 occurrences only: with the larger one the reduction walks 16-entry
 *                        tiles, which keeps a small input spread over the whole GPU; with less it
 *                        walks the 64-entry tiles of large inputs.  Results are the same up to the
 *                        order of the floating-point sums (both orders are fixed). */
size_t antdt_embbag_bwd_dedup_workspace_bytes(int64_t nnz, int64_t n_bags, int32_t dim,
                                              int32_t n_workers);
size_t antdt_embbag_bwd_dedup_min_workspace_bytes(int64_t nnz, int64_t n_bags, int32_t dim,
                                                  int32_t n_workers);
int32_t antdt_embbag_bwd_dedup(const int32_t* row_ids, int64_t nnz, const int64_t* bag_offsets,
                               int64_t n_bags, int32_t bags_per_sample, const float* d_pooled,
                               int32_t dim, int64_t n_rows, int32_t n_workers,
                               const int64_t* worker_sample_offsets, int32_t* uniq_ids,
                               int64_t* worker_uniq_offsets, int64_t* seg_offsets,
                               int32_t* sorted_occ, float* uniq_grads, int64_t out_cap,
                               void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/* The same backward + dedup step for callers that cannot allocate device memory.  (The paper
 * has no counterpart: this is a packaging variant of antdt_embbag_bwd_dedup, not a step of the
 * method.)  Some hosts of this library may not call cudaMalloc at the point where they run a
 * step: code running inside an allocator-free real-time or serving loop, a plug-in that must live
 * within a memory budget fixed at load time, a process whose device memory is entirely owned by
 * another framework's pool.  For them the scratch is a fixed array of
 * ANTDT_STATIC_SCRATCH_BYTES that lives inside the library's device image: every GPU that loads
 * the library holds it from load to exit, whether or not this call is ever used.
 *   - Arguments and results are those of antdt_embbag_bwd_dedup without ws / ws_bytes; inputs and
 *     outputs are still the caller's buffers.
 *   - Limit: antdt_embbag_bwd_dedup_min_workspace_bytes(nnz, n_bags, dim, n_workers) must not exceed
 *     ANTDT_STATIC_SCRATCH_BYTES (24 MiB: roughly 1.1 million occurrences at dim 64, 1.7 million at
 *     dim 16, with up to 64 workers).  Beyond it the call returns ANTDT_ERR_CAPACITY and launches
 *     nothing.
 *   - The call itself makes no cudaMalloc / cudaFree and no allocating library call.  The first
 *     call on each device looks up the array's device address (cudaGetSymbolAddress, with that
 *     device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array and find in it whatever the previous call left;
 *     the call clears the parts that must start at zero itself.  Two calls that overlap on the
 *     GPU (different streams, or the same stream from two threads without ordering) race on it:
 *     serialise them. */
#define ANTDT_STATIC_SCRATCH_BYTES (24u << 20)
int32_t antdt_embbag_bwd_dedup_static(const int32_t* row_ids, int64_t nnz,
                                      const int64_t* bag_offsets, int64_t n_bags,
                                      int32_t bags_per_sample, const float* d_pooled, int32_t dim,
                                      int64_t n_rows, int32_t n_workers,
                                      const int64_t* worker_sample_offsets, int32_t* uniq_ids,
                                      int64_t* worker_uniq_offsets, int64_t* seg_offsets,
                                      int32_t* sorted_occ, float* uniq_grads, int64_t out_cap,
                                      int32_t* dev_status, void* stream);

/* Server aggregation (Section II: the servers combine the local gradients of all workers into
 * one; the global batch is fixed, Eq. 1's last constraint).  Workers push MEAN gradients
 * over unequal local batches, so the aggregate that equals the mean over the global batch is
 *     G = sum_i (b_i / sum_j b_j) * G_i.
 * Sparse part: agg_ids = ascending union of the workers' row lists, a worker that does not
 * hold a row contributes nothing; summed in ascending worker order.  Dense part: the same
 * weights over K dense vectors.  Either part may be NULL.  Every worker's list must ascend
 * strictly (what antdt_embbag_bwd_dedup writes does); a list of up to 32 workers that repeats
 * ids so often that a stretch of 4096 consecutive row ids (8192 for tables beyond 2^30 rows or
 * inputs that hit the table sparsely) holds more entries than K times its width raises
 * BAD_OFFSETS in dev_status and that stretch is left out of the result.
 *   batch_sizes host [K] int64: the b_i actually served this step (counts), sum > 0. */
typedef struct {
  int32_t dim;
  int64_t n_rows;                     /* table rows: ids are < n_rows                      */
  const int32_t* uniq_ids;            /* device [in_cap]      \                            */
  const int64_t* worker_uniq_offsets; /* device [K+1]          > antdt_embbag_bwd_dedup's  */
  const float* uniq_grads;            /* device [in_cap, dim] /  outputs                   */
  int64_t in_cap;                     /* upper bound of worker_uniq_offsets[K]             */
  int32_t* agg_ids;                   /* device out [out_cap]                              */
  float* agg_grads;                   /* device out [out_cap, dim]                         */
  int64_t* n_agg;                     /* device out, one int64                             */
  int64_t out_cap;                    /* rows; in_cap always suffices                      */
} antdt_sparse_part;

typedef struct {
  const float* grads; /* device [K, stride], worker i's vector at grads + i*stride        */
  int64_t n;          /* elements per vector, n % 4 == 0                                  */
  int64_t stride;     /* >= n, stride % 4 == 0                                            */
  float* out;         /* device out [n]                                                   */
} antdt_dense_part;

size_t antdt_weighted_aggregate_workspace_bytes(int64_t in_cap, int32_t dim, int32_t n_workers);
int32_t antdt_weighted_aggregate(const antdt_sparse_part* sp, const antdt_dense_part* dp,
                                 const int64_t* batch_sizes, int32_t n_workers, void* ws,
                                 size_t ws_bytes, int32_t* dev_status, void* stream);

/* Backup-workers variant of the aggregation (the replication-based baseline the paper compares
 * with, Section VII-A.3: the gradients of the b slowest workers are disregarded in an iteration
 * and their samples go back to the shard service, antdt_dds_requeue_worker).  dropped: host
 * [K], non-zero = this worker's lists and dense vector are ignored altogether: rows that only
 * dropped workers touched are not in agg_ids, and the weights are b_i / sum over the SURVIVING
 * workers' b_j, so the result is the mean gradient over the samples that count.  Everything
 * else as antdt_weighted_aggregate (same workspace size). */
int32_t antdt_weighted_aggregate_backup(const antdt_sparse_part* sp, const antdt_dense_part* dp,
                                        const int64_t* batch_sizes, const uint8_t* dropped,
                                        int32_t n_workers, void* ws, size_t ws_bytes,
                                        int32_t* dev_status, void* stream);

/* Server update (Section II: the servers then apply the gradient to the parameters), on the rows in ids only;
 * every other row of table and state is left bit-identical.
 *   Adagrad: state0 += g*g;  w -= lr * g / (sqrt(state0) + eps)
 *   Adam:    state0 = b1*state0 + (1-b1)*g;  state1 = b2*state1 + (1-b2)*g*g;
 *            w -= lr * (state0/(1-b1^step)) / (sqrt(state1/(1-b2^step)) + eps)
 *   Row-wise Adagrad (one accumulator per ROW, for tables whose optimizer state must stay a
 *            1/dim fraction of the table):  state0[row] += (1/dim) sum_c g_c*g_c;
 *            w_c -= lr * g_c / (sqrt(state0[row]) + eps);  state0 is device [n_rows] fp32.
 * step is the global 1-based iteration.  Arithmetic is fp32; bf16 rows are widened, updated
 * and stored back round-to-nearest-even.  ids must be distinct (aggregate's output is).
 *   table  device [n_rows, dim] dtype, in/out      state0/state1 device [n_rows, dim] fp32
 *   ids    device [*n_ids_dev] int32               grads  device [*n_ids_dev, dim] fp32
 *   n_ids_dev device int64 (count stays on device); max_ids: host upper bound for it */
int32_t antdt_sparse_opt_update(void* table, int32_t dtype, int64_t n_rows, int32_t dim,
                                const int32_t* ids, const float* grads,
                                const int64_t* n_ids_dev, int64_t max_ids, int32_t opt, float lr,
                                float eps, float beta1, float beta2, int64_t step, float* state0,
                                float* state1, int32_t* dev_status, void* stream);

/* Aggregation and sparse update in one call (Section II: the servers aggregate the local
 * gradients and update the parameters - one step of theirs): the result in table / state0 /
 * state1 is that of antdt_weighted_aggregate followed by antdt_sparse_opt_update with the same
 * arguments (opt: ANTDT_OPT_ADAGRAD or ANTDT_OPT_ADAM), up to the rounding order of the weighted
 * sums (ascending worker, one fused multiply-add per contribution).  With up to 32 workers it is
 * ONE pass over the aggregated rows: each row's contributions are summed by the lane group that
 * then applies them, so the aggregated gradients are neither written nor read back;
 * sp->agg_grads may then be NULL (not materialised) - if given it is filled as usual.  agg_ids,
 * n_agg and the dense part are produced as by antdt_weighted_aggregate.  With more than 32
 * workers the two steps run one after the other and sp->agg_grads is required.
 * Workspace: antdt_weighted_aggregate_workspace_bytes.  Errors as the two calls'. */
int32_t antdt_aggregate_update(const antdt_sparse_part* sp, const antdt_dense_part* dp,
                               const int64_t* batch_sizes, int32_t n_workers, void* table,
                               int32_t dtype, int32_t opt, float lr, float eps, float beta1,
                               float beta2, int64_t step, float* state0, float* state1, void* ws,
                               size_t ws_bytes, int32_t* dev_status, void* stream);

/* Server update of the DENSE parameters (Section II: after aggregating, the servers update
 * the parameters): the element-wise Adagrad / Adam formulas above on a dense fp32 vector, with
 * the gradient antdt_weighted_aggregate's dense part produced.  Every element is touched.
 *   params, state0, state1 (Adam only): device [n] fp32, in/out      grad: device [n] fp32
 *   n % 4 == 0, all pointers 16-byte aligned; opt is ANTDT_OPT_ADAGRAD or ANTDT_OPT_ADAM.
 * Asynchronous on stream; returns ANTDT_OK, ANTDT_ERR_INVALID_ARG or ANTDT_ERR_CUDA. */
int32_t antdt_dense_opt_update(float* params, const float* grad, int64_t n, int32_t opt, float lr,
                               float eps, float beta1, float beta2, int64_t step, float* state0,
                               float* state1, void* stream);

/* One whole step from HOST buffers: copies the step's inputs to the caller's device staging
 * buffers, runs fwd, bwd_dedup, aggregate and update in order on `stream`, and copies the
 * results (pooled, dense_out, n_agg, status) back.  The copies run on two internal side
 * streams (created on the first call on a device) so that they overlap the kernels; `stream`
 * waits for all of them before the call's work on it ends, so synchronising `stream` (or an
 * event recorded on it after the call) is enough.  Host buffers should be page-locked for the
 * copies to overlap.  Every pointer of the descriptor is described beside its field.
 *
 * Two steps in flight.  By default the input copies wait for everything issued earlier on
 * `stream`, because the staging buffers may still be in use by it.  A caller that keeps TWO
 * sets of the buffers the copies touch - d_row_ids, d_bag_offsets, d_d_pooled, d_dense_grads,
 * d_pooled_out, d_dense_out, d_n_agg, d_status and the h_* outputs - and alternates them sets
 * staging_idle = 1: the copies of step s+1 then start at once and run under the kernels of step
 * s (the kernels themselves stay in order on `stream`; table, state, workspace and the other
 * intermediates are shared).  The caller records an event on `stream` after each call and waits
 * for that event before it reads the step's h_* results or reuses its set. */
typedef struct {
  /* model state, device resident */
  void* table; int32_t dtype; int64_t n_rows; int32_t dim;
  float* state0; float* state1;
  int32_t opt; float lr, eps, beta1, beta2; int64_t step;
  /* this step's batch: host inputs */
  const int32_t* h_row_ids; int64_t nnz;
  const int64_t* h_bag_offsets; int64_t n_bags; int32_t bags_per_sample;
  const float* h_d_pooled;              /* host [n_bags, dim]                              */
  const float* h_dense_grads;           /* host [K, dense_n] or NULL                       */
  int64_t dense_n;
  int32_t n_workers;
  const int64_t* worker_sample_offsets; /* host [K+1]                                      */
  const int64_t* batch_sizes;           /* host [K]                                        */
  /* device staging, caller allocated */
  int32_t* d_row_ids; int64_t* d_bag_offsets; float* d_pooled_out; float* d_d_pooled;
  float* d_dense_grads; float* d_dense_out;
  int32_t* d_uniq_ids; int64_t* d_worker_uniq_offsets; int64_t* d_seg_offsets;
  int32_t* d_sorted_occ; float* d_uniq_grads; int64_t uniq_cap;
  int32_t* d_agg_ids; float* d_agg_grads; int64_t* d_n_agg; int64_t agg_cap;
  void* ws; size_t ws_bytes;            /* >= max of the two workspace figures             */
  int32_t* d_status;
  /* host outputs */
  float* h_pooled;                      /* host [n_bags, dim]                              */
  float* h_dense_out;                   /* host [dense_n] or NULL                          */
  int64_t* h_n_agg; int32_t* h_status;  /* one element each                                */
  int32_t staging_idle;                 /* antdt_bsp_step_host only, see above; 0 = wait     */
  int32_t fuse_update;                  /* 1: aggregate and update through                   */
                                        /* antdt_aggregate_update, d_agg_grads not written   */
} antdt_step_desc;
int32_t antdt_bsp_step_host(const antdt_step_desc* d, void* stream);
/* The same step for a batch that already sits in device memory: the d_row_ids, d_bag_offsets,
 * d_d_pooled and d_dense_grads fields of the descriptor are the inputs, every h_* field is
 * ignored, nothing is copied, and the status word is neither cleared nor read back.  One host
 * call instead of four: for small batches the per-call host cost is the step time. */
int32_t antdt_bsp_step_device(const antdt_step_desc* d, void* stream);
/* The same device-resident step (Section II's iteration: local gradients, aggregation, update),
 * replayed as ONE CUDA graph launch.  A step is 30-40 short kernels; on small batches their
 * launches, not their run time, are the step time.  The first call with a given descriptor
 * captures antdt_bsp_step_device on `stream` (thread-local capture mode), instantiates the graph
 * and launches it; later calls whose descriptor is equal launch the kept executable graph.
 *   - "Equal" covers every scalar and device pointer the device step reads, and the CONTENTS of
 *     worker_sample_offsets[K+1] and batch_sizes[K] (they travel as kernel parameters); the
 *     value of `step` is not part of it.  What the device pointers point at may differ from
 *     call to call.
 *   - opt == ANTDT_OPT_ADAM is issued as the plain launches of antdt_bsp_step_device: its bias
 *     corrections change with every step and are kernel parameters, so no graph could be
 *     replayed and a capture per step costs more than it saves.
 *   - Up to 8 executable graphs are kept per device, least recently used replaced; a replaced
 *     one is updated in place when the new capture has the same shape, else re-instantiated.  A
 *     descriptor that changes every step therefore still runs as a graph, at the host cost of one
 *     capture and update per step.
 *   - Argument errors are those of the four calls, found while capturing; nothing runs then.
 *   - If `stream` is already being captured by the caller, the four calls are issued into that
 *     capture instead; a stream that cannot be captured (the legacy default stream) gets the
 *     plain launches of antdt_bsp_step_device.
 *   - Ownership: the graphs reference the caller's buffers; keep the buffers alive while graphs
 *     that name them may be replayed, or drop the graphs with antdt_bsp_step_graph_reset.  The
 *     executables are driver objects, the only thing this library ever creates on a device.
 *   - Per-kernel event timing (antdt_profile_enable) does not see kernels inside a graph;
 *     antdt_launch_count counts a replay's kernel nodes.
 *   - Small batches (at most 2^22 occurrences, at most 32 workers) are captured
 *     as three branches when the workspace has room: the forward beside the backward, and the
 *     aggregation's merge order (which needs the workers' id lists, not their gradients) beside
 *     the backward's sums.  No kernel fills the device there, so the step time is the length of
 *     the dependency chain.  The results are those of the one-chain step.  Room means ws_bytes
 *     >= antdt_bsp_step_workspace_bytes(...): the aggregation's scratch then sits behind the
 *     backward's instead of on top of it.  The branches use two library-owned side streams.
 * Returns ANTDT_OK, an argument error, or ANTDT_ERR_CUDA. */
int32_t antdt_bsp_step_graph(const antdt_step_desc* d, void* stream);
/* Workspace of a step: the larger of the backward's and the aggregation's figures; their sum
 * (the backward's rounded up to 256 bytes) for a batch small enough for the three-branch graph.
 * 0 for arguments either figure rejects. */
size_t antdt_bsp_step_workspace_bytes(int64_t nnz, int64_t n_bags, int32_t dim, int32_t n_workers,
                                      int64_t uniq_cap);
/* Destroys the executable graphs kept for the current device. */
int32_t antdt_bsp_step_graph_reset(void);

/* ---- helpers ------------------------------------------------------------------------ */
/* Synchronises `stream`, copies the status word to the host and returns it (or
 * ANTDT_ERR_CUDA).  dev_status: device int32. */
int32_t antdt_read_status(const int32_t* dev_status, void* stream);
/* Number of kernels this library has launched since it was loaded. */
int64_t antdt_launch_count(void);
/* Per-kernel device timing: when enabled, every launch is bracketed by CUDA events on its
 * stream.  antdt_profile_get synchronises the recorded events and reports, for kernel slot
 * idx in [0, antdt_profile_kernels()), its name, launches and summed milliseconds since
 * antdt_profile_enable(1). */
int32_t antdt_profile_enable(int32_t on);
int32_t antdt_profile_kernels(void);
int32_t antdt_profile_get(int32_t idx, char* name, size_t name_cap, int64_t* launches,
                          double* total_ms);
/* Measurement aid (the paper has no counterpart): the plainest gather there is, for finding the
 * rate at which this GPU's SMs can pull scattered rows out of L2, the ceiling that the
 * gathering kernels of the step meet once the rows they repeat are cache resident.  Output
 * row o = sum of the per_out rows rows[idx[o*per_out + j]] (an index outside [0, n_rows) reads
 * row 0).  rows device [n_rows, dim] fp32, dim one of 16 / 32 / 64 / 128, 16-byte aligned;
 * idx device [n_out*per_out] int32; out device [n_out, dim].  Time it with events on `stream`
 * on a matrix of a few tens of MB with uniformly random idx. */
int32_t antdt_probe_gather(const float* rows, int64_t n_rows, int32_t dim, const int32_t* idx,
                           int64_t n_out, int32_t per_out, float* out, void* stream);
const char* antdt_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ANTDT_H */
