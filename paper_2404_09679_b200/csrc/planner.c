/*
 * Host planner: Stateful Dynamic Data Sharding (Section V-C) and the ADJUST_BS batch sizes
 * (Section VI-A, Eq. 2-3).  Plain C, no device code; produces per-worker sample ranges only.
 *
 * Data layout: shards live in three parallel arrays; the TODO queue is a growing array of
 * shard indices with a head cursor (a requeued shard is appended, so the array holds at most
 * n_shards + #requeues entries); every worker has the shard it holds and how much of it is
 * consumed.  A step is planned in two sweeps over the same routine: a dry run on scratch
 * copies of the small per-worker state that only counts ranges, then the committing run.
 *
 * A shard becomes DONE only once the gradients computed on its last samples have been pushed
 * (Section V-C.3).  The planner learns of a failed push through antdt_dds_requeue_worker, so the
 * shards a worker finished in the latest plan call stay on that worker's short "finished" list
 * until the next plan call: a requeue in between takes them back together with the DOING shard.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include "antdt.h"

#define MAX_WORKERS 1024
/* Shards one worker can finish in one step: the one it holds, then only shards no longer than
 * what is left of its batch (<= B), i.e. the short last shard of the dataset, or a whole shard
 * when B*M == B_i.  Two at most; the list has room for four, a fifth would simply stay DONE. */
#define MAX_FINISHED 4
#define DDS_MAGIC 0x53444454414E41ull /* "ANATDDS" */

struct antdt_dds {
  int64_t n_samples, global_batch;
  int32_t batches_per_shard, n_workers;
  uint64_t shuffle_seed;
  int64_t n_shards;
  int64_t* shard_start;
  int64_t* shard_len;
  int8_t* shard_state;
  int32_t* shard_owner;
  int64_t* queue; /* shard indices; live part is [q_head, q_tail) */
  int64_t q_head, q_tail, q_cap;
  int64_t* held;  /* [K] shard a worker is DOING, -1 if none */
  int64_t* used;  /* [K] samples of it already served */
  int64_t* fin;   /* [K][MAX_FINISHED] shards the worker finished in the latest plan call */
  int32_t* n_fin; /* [K] how many */
};

/* ---- splitmix64 stream (Steele, Lea, Flood 2014) for the shard shuffle --------------- */
static uint64_t sm64(uint64_t* s) {
  uint64_t z = (*s += 0x9E3779B97F4A7C15ull);
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

/* ====================================================================================== */
/* batch sizes                                                                            */
/* ====================================================================================== */

/* binary min-heap on (cost, worker) for the MINMAX rule */
typedef struct { double cost; int32_t w; } heap_item;
static int heap_less(heap_item a, heap_item b) {
  return a.cost < b.cost || (a.cost == b.cost && a.w < b.w);
}
static void heap_sift_down(heap_item* h, int n, int i) {
  for (;;) {
    int l = 2 * i + 1, r = l + 1, m = i;
    if (l < n && heap_less(h[l], h[m])) m = l;
    if (r < n && heap_less(h[r], h[m])) m = r;
    if (m == i) return;
    heap_item t = h[i]; h[i] = h[m]; h[m] = t;
    i = m;
  }
}

static int32_t minmax_sizes(const double* v, int32_t n, int64_t B, int64_t minb, int64_t* b) {
  /* Eq. 3 over integers.  Each of the B - n*minb free samples goes where the resulting
   * B_i/v_i is smallest; the heap keeps the next cost of every worker. */
  heap_item* h = (heap_item*)malloc(sizeof(heap_item) * (size_t)n);
  if (!h) return ANTDT_ERR_INVALID_ARG;
  for (int32_t i = 0; i < n; ++i) {
    b[i] = minb;
    h[i].cost = (double)(minb + 1) / v[i];
    h[i].w = i;
  }
  for (int i = n / 2 - 1; i >= 0; --i) heap_sift_down(h, n, i);
  for (int64_t left = B - minb * n; left > 0; --left) {
    int32_t w = h[0].w;
    b[w] += 1;
    h[0].cost = (double)(b[w] + 1) / v[w];
    heap_sift_down(h, n, 0);
  }
  free(h);
  return ANTDT_OK;
}

typedef struct { double frac; int32_t w; } frac_item;
static int frac_desc(const void* pa, const void* pb) {
  const frac_item* a = (const frac_item*)pa;
  const frac_item* b = (const frac_item*)pb;
  if (a->frac != b->frac) return a->frac > b->frac ? -1 : 1;
  return a->w < b->w ? -1 : (a->w > b->w ? 1 : 0);
}

static int32_t proportional_sizes(const double* v, int32_t n, int64_t B, int64_t minb,
                                  int64_t* b) {
  /* B_i = B v_i / sum v equalises B_i/v_i, the continuous optimum of Eq. 3.  Workers whose
   * share falls under min_batch are pinned there and the others share what remains. */
  double q[MAX_WORKERS];
  uint8_t pinned[MAX_WORKERS];
  frac_item fr[MAX_WORKERS];
  memset(pinned, 0, (size_t)n);
  int64_t budget;
  for (;;) {
    int64_t n_pinned = 0;
    double S = 0.0;
    for (int32_t i = 0; i < n; ++i) {
      if (pinned[i]) ++n_pinned; else S += v[i];
    }
    budget = B - minb * n_pinned;
    int newly = 0;
    for (int32_t i = 0; i < n; ++i) {
      if (pinned[i]) continue;
      q[i] = (double)budget * v[i] / S;
    }
    for (int32_t i = 0; i < n; ++i) {
      if (!pinned[i] && q[i] < (double)minb) { pinned[i] = 1; newly = 1; }
    }
    if (!newly) break;
  }
  int64_t given = 0;
  int32_t m = 0;
  for (int32_t i = 0; i < n; ++i) {
    if (pinned[i]) { b[i] = minb; continue; }
    double fl = floor(q[i]);
    b[i] = (int64_t)fl;
    given += b[i];
    fr[m].frac = q[i] - fl;
    fr[m].w = i;
    ++m;
  }
  int64_t left = budget - given;
  if (m == 0) return left == 0 ? ANTDT_OK : ANTDT_ERR_INVALID_ARG;
  qsort(fr, (size_t)m, sizeof(frac_item), frac_desc); /* largest remainder, then lower index */
  for (int64_t k = 0; left > 0; ++k, --left) b[fr[k % m].w] += 1;
  /* rounding slack in the other direction: give back from the smallest remainders,
   * the higher index first among equals */
  for (int64_t k = m - 1; left < 0;) {
    int32_t w = fr[k].w;
    if (b[w] > minb) { b[w] -= 1; ++left; }
    k = (k == 0) ? m - 1 : k - 1;
  }
  return ANTDT_OK;
}

int32_t antdt_batch_sizes(const double* speeds, int32_t n_workers, int64_t global_batch,
                          int32_t rule, int64_t min_batch, int64_t* batch_sizes) {
  if (!batch_sizes || n_workers < 1 || n_workers > MAX_WORKERS || global_batch < 1 ||
      min_batch < 0 || min_batch * n_workers > global_batch)
    return ANTDT_ERR_INVALID_ARG;
  if (!speeds) { /* Section VI-A step 1: B_i = B / n */
    int64_t base = global_batch / n_workers, rem = global_batch % n_workers;
    for (int32_t i = 0; i < n_workers; ++i) batch_sizes[i] = base + (i < rem ? 1 : 0);
    return ANTDT_OK;
  }
  for (int32_t i = 0; i < n_workers; ++i)
    if (!(speeds[i] > 0.0) || !isfinite(speeds[i])) return ANTDT_ERR_INVALID_ARG;
  if (rule == ANTDT_RULE_MINMAX)
    return minmax_sizes(speeds, n_workers, global_batch, min_batch, batch_sizes);
  if (rule == ANTDT_RULE_PROPORTIONAL)
    return proportional_sizes(speeds, n_workers, global_batch, min_batch, batch_sizes);
  return ANTDT_ERR_INVALID_ARG;
}

/* ====================================================================================== */
/* shard service                                                                          */
/* ====================================================================================== */

static void dds_free(antdt_dds* d) {
  if (!d) return;
  free(d->shard_start); free(d->shard_len); free(d->shard_state); free(d->shard_owner);
  free(d->queue); free(d->held); free(d->used); free(d->fin); free(d->n_fin);
  free(d);
}

static antdt_dds* dds_alloc(int64_t n_shards, int32_t K, int64_t q_cap) {
  antdt_dds* d = (antdt_dds*)calloc(1, sizeof(antdt_dds));
  if (!d) return NULL;
  size_t ns = (size_t)n_shards;
  d->shard_start = (int64_t*)malloc(8 * ns);
  d->shard_len = (int64_t*)malloc(8 * ns);
  d->shard_state = (int8_t*)malloc(ns);
  d->shard_owner = (int32_t*)malloc(4 * ns);
  d->queue = (int64_t*)malloc(8 * (size_t)q_cap);
  d->held = (int64_t*)malloc(8 * (size_t)K);
  d->used = (int64_t*)malloc(8 * (size_t)K);
  d->fin = (int64_t*)malloc(8 * (size_t)K * MAX_FINISHED);
  d->n_fin = (int32_t*)calloc((size_t)K, 4);
  d->q_cap = q_cap;
  d->n_shards = n_shards;
  d->n_workers = K;
  if (!d->shard_start || !d->shard_len || !d->shard_state || !d->shard_owner || !d->queue ||
      !d->held || !d->used || !d->fin || !d->n_fin) {
    dds_free(d);
    return NULL;
  }
  return d;
}

int32_t antdt_dds_create(antdt_dds** out, int64_t n_samples, int64_t global_batch,
                         int32_t batches_per_shard, int32_t n_workers, uint64_t shuffle_seed) {
  if (!out || n_samples < 1 || global_batch < 1 || batches_per_shard < 1 || n_workers < 1 ||
      n_workers > MAX_WORKERS)
    return ANTDT_ERR_INVALID_ARG;
  int64_t per = global_batch * (int64_t)batches_per_shard;
  int64_t n_shards = n_samples / per + (n_samples % per ? 1 : 0); /* ceil(N / (B*M)) */
  antdt_dds* d = dds_alloc(n_shards, n_workers, n_shards + 16);
  if (!d) return ANTDT_ERR_INVALID_ARG;
  d->n_samples = n_samples;
  d->global_batch = global_batch;
  d->batches_per_shard = batches_per_shard;
  d->shuffle_seed = shuffle_seed;
  for (int64_t j = 0; j < n_shards; ++j) {
    d->shard_start[j] = j * per;
    d->shard_len[j] = (j == n_shards - 1) ? n_samples - j * per : per;
    d->shard_state[j] = ANTDT_SHARD_TODO;
    d->shard_owner[j] = -1;
    d->queue[j] = j;
  }
  if (shuffle_seed != 0) { /* Fisher-Yates over the queue, from the back */
    uint64_t s = shuffle_seed;
    for (int64_t i = n_shards - 1; i >= 1; --i) {
      int64_t j = (int64_t)(sm64(&s) % (uint64_t)(i + 1));
      int64_t t = d->queue[i]; d->queue[i] = d->queue[j]; d->queue[j] = t;
    }
  }
  d->q_head = 0;
  d->q_tail = n_shards;
  for (int32_t i = 0; i < n_workers; ++i) { d->held[i] = -1; d->used[i] = 0; }
  *out = d;
  return ANTDT_OK;
}

void antdt_dds_destroy(antdt_dds* dds) { dds_free(dds); }

/* Serve the step.  commit == 0: touch nothing, only count ranges and served samples. */
static int64_t serve(antdt_dds* d, const int64_t* bsz, int commit, int64_t* range_offsets,
                     antdt_range* ranges, int64_t* counts, int64_t* total_served) {
  int64_t n_ranges = 0, q_head = d->q_head, total = 0;
  for (int32_t i = 0; i < d->n_workers; ++i) {
    int64_t held = d->held[i], used = d->used[i], need = bsz[i];
    if (commit) { range_offsets[i] = n_ranges; d->n_fin[i] = 0; }
    while (need > 0) {
      if (held < 0) {
        if (q_head == d->q_tail) break; /* nothing left to fetch: short batch */
        held = d->queue[q_head++];
        used = 0;
        if (commit) { d->shard_state[held] = ANTDT_SHARD_DOING; d->shard_owner[held] = i; }
      }
      int64_t avail = d->shard_len[held] - used;
      int64_t take = need < avail ? need : avail;
      if (commit) { ranges[n_ranges].start = d->shard_start[held] + used; ranges[n_ranges].len = take; }
      ++n_ranges;
      used += take;
      need -= take;
      if (used == d->shard_len[held]) { /* consumed: DONE, unless this step's push fails */
        if (commit) {
          d->shard_state[held] = ANTDT_SHARD_DONE;
          d->shard_owner[held] = -1;
          if (d->n_fin[i] < MAX_FINISHED) d->fin[(size_t)i * MAX_FINISHED + d->n_fin[i]++] = held;
        }
        held = -1;
        used = 0;
      }
    }
    if (commit) { d->held[i] = held; d->used[i] = used; counts[i] = bsz[i] - need; }
    total += bsz[i] - need;
  }
  if (commit) { range_offsets[d->n_workers] = n_ranges; d->q_head = q_head; }
  *total_served = total;
  return n_ranges;
}

int32_t antdt_shard_plan(antdt_dds* dds, const double* speeds, int32_t rule, int64_t min_batch,
                         int64_t* batch_sizes, int64_t* range_offsets, antdt_range* ranges,
                         int64_t ranges_cap, int64_t* counts) {
  if (!dds || !batch_sizes || !range_offsets || !counts || ranges_cap < 0 ||
      (!ranges && ranges_cap > 0))
    return ANTDT_ERR_INVALID_ARG;
  int32_t rc = antdt_batch_sizes(speeds, dds->n_workers, dds->global_batch, rule, min_batch,
                                 batch_sizes);
  if (rc != ANTDT_OK) return rc;
  int64_t total = 0;
  int64_t n_ranges = serve(dds, batch_sizes, 0, NULL, NULL, NULL, &total);
  if (total == 0) {
    for (int32_t i = 0; i <= dds->n_workers; ++i) range_offsets[i] = 0;
    for (int32_t i = 0; i < dds->n_workers; ++i) counts[i] = 0;
    return ANTDT_ERR_EXHAUSTED;
  }
  if (n_ranges > ranges_cap) return ANTDT_ERR_CAPACITY;
  serve(dds, batch_sizes, 1, range_offsets, ranges, counts, &total);
  return ANTDT_OK;
}

/* Appends shard j to the back of the queue (Section V-C.3) as TODO. */
static int32_t queue_push_back(antdt_dds* dds, int64_t j) {
  if (dds->q_tail == dds->q_cap) { /* compact the consumed prefix, grow if still full */
    int64_t live = dds->q_tail - dds->q_head;
    memmove(dds->queue, dds->queue + dds->q_head, 8 * (size_t)live);
    dds->q_head = 0;
    dds->q_tail = live;
    if (live + 1 > dds->q_cap) {
      int64_t cap = dds->q_cap * 2 + 16;
      int64_t* q = (int64_t*)realloc(dds->queue, 8 * (size_t)cap);
      if (!q) return ANTDT_ERR_STATE;
      dds->queue = q;
      dds->q_cap = cap;
    }
  }
  dds->queue[dds->q_tail++] = j;
  dds->shard_state[j] = ANTDT_SHARD_TODO;
  dds->shard_owner[j] = -1;
  return ANTDT_OK;
}

int32_t antdt_dds_requeue_worker(antdt_dds* dds, int32_t worker) {
  if (!dds || worker < 0 || worker >= dds->n_workers) return ANTDT_ERR_INVALID_ARG;
  /* the shards it finished in the latest plan call first, in the order it finished them ... */
  for (int32_t k = 0; k < dds->n_fin[worker]; ++k) {
    int32_t rc = queue_push_back(dds, dds->fin[(size_t)worker * MAX_FINISHED + k]);
    if (rc != ANTDT_OK) return rc;
  }
  dds->n_fin[worker] = 0;
  /* ... then the one it is DOING */
  int64_t j = dds->held[worker];
  if (j < 0) return ANTDT_OK;
  int32_t rc = queue_push_back(dds, j);
  if (rc != ANTDT_OK) return rc;
  dds->held[worker] = -1;
  dds->used[worker] = 0;
  return ANTDT_OK;
}

int64_t antdt_dds_num_shards(const antdt_dds* dds) { return dds ? dds->n_shards : -1; }

int32_t antdt_dds_counts(const antdt_dds* dds, int64_t* todo, int64_t* doing, int64_t* done) {
  if (!dds || !todo || !doing || !done) return ANTDT_ERR_INVALID_ARG;
  int64_t c[3] = {0, 0, 0};
  for (int64_t j = 0; j < dds->n_shards; ++j) c[dds->shard_state[j]] += 1;
  *todo = c[ANTDT_SHARD_TODO];
  *doing = c[ANTDT_SHARD_DOING];
  *done = c[ANTDT_SHARD_DONE];
  return ANTDT_OK;
}

int32_t antdt_dds_shard_info(const antdt_dds* dds, int64_t shard, int32_t* state, int32_t* owner,
                             antdt_range* r) {
  if (!dds || shard < 0 || shard >= dds->n_shards) return ANTDT_ERR_INVALID_ARG;
  if (state) *state = dds->shard_state[shard];
  if (owner) *owner = dds->shard_owner[shard];
  if (r) { r->start = dds->shard_start[shard]; r->len = dds->shard_len[shard]; }
  return ANTDT_OK;
}

/* ---- image: header of 10 int64, then state[n_shards] owner[n_shards] (as int64 each),
 * queue[live], held[K], used[K], n_fin[K], fin[K][MAX_FINISHED].  Shard (start, len) are
 * recomputed from the header. ---- */
#define DDS_IMAGE_VERSION 2
int32_t antdt_dds_save(const antdt_dds* dds, void* buf, size_t cap, size_t* used) {
  if (!dds || !used) return ANTDT_ERR_INVALID_ARG;
  int64_t live = dds->q_tail - dds->q_head;
  size_t words = 10 + 2 * (size_t)dds->n_shards + (size_t)live +
                 (3 + MAX_FINISHED) * (size_t)dds->n_workers;
  *used = words * 8;
  if (!buf) return ANTDT_OK;
  if (cap < *used) return ANTDT_ERR_CAPACITY;
  int64_t* w = (int64_t*)buf;
  size_t k = 0;
  w[k++] = (int64_t)DDS_MAGIC; w[k++] = DDS_IMAGE_VERSION;
  w[k++] = dds->n_samples; w[k++] = dds->global_batch; w[k++] = dds->batches_per_shard;
  w[k++] = dds->n_workers; w[k++] = (int64_t)dds->shuffle_seed; w[k++] = dds->n_shards;
  w[k++] = live; w[k++] = 0;
  for (int64_t j = 0; j < dds->n_shards; ++j) w[k++] = dds->shard_state[j];
  for (int64_t j = 0; j < dds->n_shards; ++j) w[k++] = dds->shard_owner[j];
  for (int64_t j = dds->q_head; j < dds->q_tail; ++j) w[k++] = dds->queue[j];
  for (int32_t i = 0; i < dds->n_workers; ++i) w[k++] = dds->held[i];
  for (int32_t i = 0; i < dds->n_workers; ++i) w[k++] = dds->used[i];
  for (int32_t i = 0; i < dds->n_workers; ++i) w[k++] = dds->n_fin[i];
  for (int32_t i = 0; i < dds->n_workers; ++i)
    for (int32_t f = 0; f < MAX_FINISHED; ++f)
      w[k++] = f < dds->n_fin[i] ? dds->fin[(size_t)i * MAX_FINISHED + f] : -1;
  return ANTDT_OK;
}

int32_t antdt_dds_load(antdt_dds** out, const void* buf, size_t len) {
  if (!out || !buf || len < 80 || len % 8) return ANTDT_ERR_INVALID_ARG;
  const int64_t* w = (const int64_t*)buf;
  if (w[0] != (int64_t)DDS_MAGIC || w[1] != DDS_IMAGE_VERSION) return ANTDT_ERR_INVALID_ARG;
  int64_t N = w[2], B = w[3], M = w[4], K = w[5], n_shards = w[7], live = w[8];
  if (N < 1 || B < 1 || M < 1 || K < 1 || K > MAX_WORKERS || live < 0 || live > n_shards)
    return ANTDT_ERR_INVALID_ARG;
  int64_t per = B * M;
  if (n_shards != N / per + (N % per ? 1 : 0)) return ANTDT_ERR_INVALID_ARG;
  if (len != 8 * (10 + 2 * (size_t)n_shards + (size_t)live + (3 + MAX_FINISHED) * (size_t)K))
    return ANTDT_ERR_INVALID_ARG;
  antdt_dds* d = dds_alloc(n_shards, (int32_t)K, n_shards + 16);
  if (!d) return ANTDT_ERR_INVALID_ARG;
  d->n_samples = N; d->global_batch = B; d->batches_per_shard = (int32_t)M;
  d->shuffle_seed = (uint64_t)w[6];
  size_t k = 10;
  int bad = 0;
  for (int64_t j = 0; j < n_shards; ++j) {
    d->shard_start[j] = j * per;
    d->shard_len[j] = (j == n_shards - 1) ? N - j * per : per;
    int64_t s = w[k++];
    if (s < 0 || s > 2) bad = 1;
    d->shard_state[j] = (int8_t)s;
  }
  for (int64_t j = 0; j < n_shards; ++j) {
    int64_t o = w[k++];
    if (o < -1 || o >= K) bad = 1;
    d->shard_owner[j] = (int32_t)o;
  }
  for (int64_t j = 0; j < live; ++j) {
    int64_t s = w[k++];
    if (s < 0 || s >= n_shards) { bad = 1; s = 0; }
    d->queue[j] = s;
  }
  d->q_head = 0;
  d->q_tail = live;
  for (int64_t i = 0; i < K; ++i) {
    int64_t h = w[k++];
    if (h < -1 || h >= n_shards) { bad = 1; h = -1; }
    d->held[i] = h;
  }
  for (int64_t i = 0; i < K; ++i) {
    int64_t u = w[k++];
    if (u < 0 || (d->held[i] >= 0 && u >= d->shard_len[d->held[i]])) bad = 1;
    d->used[i] = u;
  }
  for (int64_t i = 0; i < K; ++i) {
    int64_t nf = w[k++];
    if (nf < 0 || nf > MAX_FINISHED) { bad = 1; nf = 0; }
    d->n_fin[i] = (int32_t)nf;
  }
  for (int64_t i = 0; i < K; ++i)
    for (int32_t f = 0; f < MAX_FINISHED; ++f) {
      int64_t j = w[k++];
      if (f < d->n_fin[i] && (j < 0 || j >= n_shards || d->shard_state[j] != ANTDT_SHARD_DONE)) {
        bad = 1;
        j = 0;
      }
      d->fin[(size_t)i * MAX_FINISHED + f] = j;
    }
  if (bad) { dds_free(d); return ANTDT_ERR_INVALID_ARG; }
  *out = d;
  return ANTDT_OK;
}
