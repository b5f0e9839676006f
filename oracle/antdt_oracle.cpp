// TEST INFRASTRUCTURE ONLY -- the CPU checker of the BSP sparse-ranking step.
//
// A plain, slow, single-threaded statement of what each call of the step computes, with all
// floating-point accumulation in double and a rounding to float (or bf16) only where the
// contract stores one.  It shares no code with the CUDA library and must never be reachable
// from the product path: only the tests, the smoke check and the benchmark's CPU-baseline leg
// load it.
//
// Every function here is pinned by tests that do not re-use it: closed forms, brute force over
// dense count matrices, invariants of the paper (Section II / Eq. 1: sum_i B_i = B; Section
// V-C: every sample handed out once per epoch, #DONE shards = ceil(N/(B*M))) and exhaustive
// search over integer compositions for Eq. 3.
//
// Where the paper fixes the computation, the passage is cited beside the function; the
// embedding-bag, dedup, weighting and optimizer definitions are the textbook ones the paper
// leaves to its training substrate (Section II only says workers compute local gradients on
// B_i and that the servers combine them and apply the result to the parameters).
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <deque>
#include <limits>
#include <map>
#include <utility>
#include <vector>

namespace {

typedef int64_t i64;
typedef int32_t i32;

enum { OK = 0, E_ARG = 1, E_ID = 2, E_CAP = 4, E_EXHAUSTED = 7, E_OFFSETS = 9 };

// ---------------------------------------------------------------------------------------
// Batch sizes.  Section VI-A step 1 (B_i = B/n) and step 3 (Eq. 2-3: min z, z >= B_i/v_i,
// sum B_i = B).
// ---------------------------------------------------------------------------------------
bool speeds_ok(const double* v, int n) {
  for (int i = 0; i < n; ++i)
    if (!(v[i] > 0.0) || !std::isfinite(v[i])) return false;
  return true;
}

int batch_sizes(const double* v, int n, i64 B, int rule, i64 minb, i64* b) {
  if (n < 1 || B < 1 || minb < 0 || minb * n > B) return E_ARG;
  if (!v) {  // first iteration: even split, remainder to the lowest indices
    for (int i = 0; i < n; ++i) b[i] = B / n + (i < B % n ? 1 : 0);
    return OK;
  }
  if (!speeds_ok(v, n)) return E_ARG;
  if (rule == 1) {
    // Eq. 3 in integers.  The objective max_i B_i/v_i is separable and non-decreasing in
    // every B_i, so adding one sample at a time where it hurts least is optimal.
    for (int i = 0; i < n; ++i) b[i] = minb;
    for (i64 left = B - minb * n; left > 0; --left) {
      int best = 0;
      double bv = (double)(b[0] + 1) / v[0];
      for (int i = 1; i < n; ++i) {
        double c = (double)(b[i] + 1) / v[i];
        if (c < bv) { bv = c; best = i; }
      }
      b[best] += 1;
    }
    return OK;
  }
  if (rule != 0) return E_ARG;
  // Continuous optimum of Eq. 3 is B_i proportional to v_i (all B_i/v_i equal); round it.
  std::vector<char> pinned(n, 0);
  std::vector<double> q(n, 0.0);
  for (;;) {
    i64 npinned = 0;
    for (int i = 0; i < n; ++i) npinned += pinned[i];
    i64 budget = B - minb * npinned;
    double S = 0.0;
    for (int i = 0; i < n; ++i)
      if (!pinned[i]) S += v[i];
    bool again = false;
    for (int i = 0; i < n; ++i) {
      if (pinned[i]) continue;
      q[i] = (double)budget * v[i] / S;
      if (q[i] < (double)minb) again = true;
    }
    if (!again) {
      i64 given = 0;
      for (int i = 0; i < n; ++i) {
        b[i] = pinned[i] ? minb : (i64)std::floor(q[i]);
        if (!pinned[i]) given += b[i];
      }
      i64 left = budget - given;
      // largest remainder first, ties to the lower index; one unit each
      while (left > 0) {
        std::vector<char> used(n, 0);
        bool any = false;
        for (int i = 0; i < n; ++i) any = any || !pinned[i];
        if (!any) break;
        for (i64 round = 0; round < n && left > 0; ++round) {
          int best = -1;
          double bf = -1.0;
          for (int i = 0; i < n; ++i) {
            if (pinned[i] || used[i]) continue;
            double fr = q[i] - std::floor(q[i]);
            if (fr > bf) { bf = fr; best = i; }
          }
          if (best < 0) break;
          used[best] = 1;
          b[best] += 1;
          --left;
        }
      }
      // floating-point slack the other way: take back one unit each from the smallest
      // remainders, ties to the higher index
      while (left < 0) {
        std::vector<char> used(n, 0);
        bool progress = false;
        for (i64 round = 0; round < n && left < 0; ++round) {
          int best = -1;
          double bf = 2.0;
          for (int i = 0; i < n; ++i) {
            if (pinned[i] || used[i]) continue;
            double fr = q[i] - std::floor(q[i]);
            if (fr <= bf) { bf = fr; best = i; }
          }
          if (best < 0) break;
          used[best] = 1;
          if (b[best] > minb) { b[best] -= 1; ++left; progress = true; }
        }
        if (!progress) return E_ARG;
      }
      return OK;
    }
    for (int i = 0; i < n; ++i)
      if (!pinned[i] && q[i] < (double)minb) pinned[i] = 1;
  }
}

// ---------------------------------------------------------------------------------------
// Stateful Dynamic Data Sharding, Section V-C.
// ---------------------------------------------------------------------------------------
// done_by / done_plan / done_seq: who served the shard's last sample, in which plan call, and
// the position of that event among all such events (a global counter).
struct Shard { i64 start, len; int state; int owner; int done_by; i64 done_plan, done_seq; };

struct Dds {
  i64 N, B; int M, K;
  std::vector<Shard> shards;
  std::deque<i64> queue;         // TODO shards, head = next to hand out
  std::vector<i64> held, used;   // per worker: shard it is DOING (-1 none), samples consumed
  i64 plans = 0, seq = 0;        // committed plan calls; completion events so far
};

uint64_t sm64_next(uint64_t& s) {
  s += 0x9E3779B97F4A7C15ull;
  uint64_t z = s;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// bf16 <-> real
double bf16_to_double(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return (double)f;
}

uint16_t double_to_bf16_rne(double x) {
  if (x == 0.0 || !std::isfinite(x)) {
    float f = (float)x;
    uint32_t u;
    std::memcpy(&u, &f, 4);
    return (uint16_t)(u >> 16);
  }
  int e;
  double m = std::frexp(x, &e);          // x = m * 2^e, |m| in [0.5, 1)
  int q = e - 8;                          // 8 significant bits
  if (q < -133) q = -133;                 // bf16 subnormal quantum 2^-133
  double r = std::nearbyint(std::ldexp(x, -q));  // ties to even (default rounding mode)
  (void)m;
  float f = (float)std::ldexp(r, q);      // exactly representable (or overflow to inf)
  uint32_t u;
  std::memcpy(&u, &f, 4);
  return (uint16_t)(u >> 16);
}

double load_elem(const void* t, int dtype, i64 idx) {
  return dtype == 0 ? (double)((const float*)t)[idx] : bf16_to_double(((const uint16_t*)t)[idx]);
}
void store_elem(void* t, int dtype, i64 idx, double x) {
  if (dtype == 0) ((float*)t)[idx] = (float)x;
  else ((uint16_t*)t)[idx] = double_to_bf16_rne(x);
}

int check_bags(const i32* ids, const i64* off, i64 n_bags, i64 n_rows) {
  if (n_bags < 0 || off[0] != 0) return E_OFFSETS;
  for (i64 b = 0; b < n_bags; ++b)
    if (off[b + 1] < off[b]) return E_OFFSETS;
  if (n_rows >= 0)
    for (i64 j = 0; j < off[n_bags]; ++j)
      if (ids[j] < 0 || ids[j] >= n_rows) return E_ID;
  return OK;
}

}  // namespace

extern "C" {

int orc_batch_sizes(const double* speeds, int n, i64 B, int rule, i64 min_batch, i64* out) {
  return batch_sizes(speeds, n, B, rule, min_batch, out);
}

// Section V-C.1: K_sh = ceil(N / (B*M)) shards of B*M consecutive samples, each just (start,
// length); all TODO; queued in order, or shuffled between shards by a seeded Fisher-Yates.
void* orc_dds_create(i64 N, i64 B, int M, int K, uint64_t shuffle_seed) {
  if (N < 1 || B < 1 || M < 1 || K < 1 || K > 1024) return nullptr;
  Dds* d = new Dds;
  d->N = N; d->B = B; d->M = M; d->K = K;
  i64 per = B * (i64)M;
  i64 n_sh = (N + per - 1) / per;
  for (i64 j = 0; j < n_sh; ++j) {
    Shard s;
    s.start = j * per;
    s.len = std::min(per, N - s.start);
    s.state = 0; s.owner = -1;
    s.done_by = -1; s.done_plan = -1; s.done_seq = -1;
    d->shards.push_back(s);
  }
  std::vector<i64> order(n_sh);
  for (i64 j = 0; j < n_sh; ++j) order[j] = j;
  if (shuffle_seed != 0) {
    uint64_t st = shuffle_seed;
    for (i64 i = n_sh - 1; i >= 1; --i) {
      i64 j = (i64)(sm64_next(st) % (uint64_t)(i + 1));
      std::swap(order[i], order[j]);
    }
  }
  for (i64 j = 0; j < n_sh; ++j) d->queue.push_back(order[j]);
  d->held.assign(K, -1);
  d->used.assign(K, 0);
  return d;
}

void orc_dds_destroy(void* h) { delete (Dds*)h; }
i64 orc_dds_num_shards(void* h) { return (i64)((Dds*)h)->shards.size(); }

void orc_dds_counts(void* h, i64* todo, i64* doing, i64* done) {
  Dds* d = (Dds*)h;
  *todo = *doing = *done = 0;
  for (const Shard& s : d->shards) (s.state == 0 ? *todo : s.state == 1 ? *doing : *done) += 1;
}

void orc_dds_shard_info(void* h, i64 j, int* state, int* owner, i64* start, i64* len) {
  const Shard& s = ((Dds*)h)->shards[j];
  *state = s.state; *owner = s.owner; *start = s.start; *len = s.len;
}

// One BSP step of the service.  Workers are served in ascending index; a worker keeps the
// shard it is DOING until it has consumed all of it (Section V-C.2: it cannot fetch a new one
// before), then takes the queue head (TODO -> DOING).  A shard whose last sample was served is
// DONE once the step's gradients are pushed (Section V-C.3): it is marked DONE when this call
// returns, and orc_dds_requeue takes the mark back if the push turns out to have failed before
// the next call.
// ranges: int64 pairs (start, len), CSR by worker through range_offsets.
int orc_dds_plan(void* h, const double* speeds, int rule, i64 min_batch, i64* bsz,
                 i64* range_offsets, i64* ranges, i64 cap, i64* counts) {
  Dds* d = (Dds*)h;
  int rc = batch_sizes(speeds, d->K, d->B, rule, min_batch, bsz);
  if (rc != OK) return rc;
  Dds trial = *d;  // work on a copy; commit only if the ranges fit
  trial.plans += 1;
  std::vector<i64> out;
  i64 total = 0;
  for (int i = 0; i < trial.K; ++i) {
    range_offsets[i] = (i64)out.size() / 2;
    i64 need = bsz[i];
    while (need > 0) {
      if (trial.held[i] < 0) {
        if (trial.queue.empty()) break;
        i64 j = trial.queue.front();
        trial.queue.pop_front();
        trial.shards[j].state = 1;
        trial.shards[j].owner = i;
        trial.held[i] = j;
        trial.used[i] = 0;
      }
      Shard& s = trial.shards[trial.held[i]];
      i64 take = std::min(need, s.len - trial.used[i]);
      out.push_back(s.start + trial.used[i]);
      out.push_back(take);
      trial.used[i] += take;
      need -= take;
      if (trial.used[i] == s.len) {
        s.state = 2;
        s.owner = -1;
        s.done_by = i;
        s.done_plan = trial.plans;
        s.done_seq = trial.seq++;
        trial.held[i] = -1;
        trial.used[i] = 0;
      }
    }
    counts[i] = bsz[i] - need;
    total += counts[i];
  }
  range_offsets[trial.K] = (i64)out.size() / 2;
  if ((i64)out.size() / 2 > cap) return E_CAP;
  for (size_t k = 0; k < out.size(); ++k) ranges[k] = out[k];
  if (total == 0) return E_EXHAUSTED;
  *d = trial;
  return OK;
}

// Section V-C.3: the shards of a worker whose push failed go back to TODO at the END of the
// queue: those whose last sample it was served in the latest plan call (their gradients never
// arrived, so they are not DONE after all), oldest completion first, then the one it is DOING.
int orc_dds_requeue(void* h, int worker) {
  Dds* d = (Dds*)h;
  if (worker < 0 || worker >= d->K) return E_ARG;
  std::vector<std::pair<i64, i64>> undone;  // (completion order, shard)
  for (size_t j = 0; j < d->shards.size(); ++j) {
    const Shard& s = d->shards[j];
    if (s.state == 2 && s.done_by == worker && s.done_plan == d->plans)
      undone.push_back(std::make_pair(s.done_seq, (i64)j));
  }
  std::sort(undone.begin(), undone.end());
  for (const auto& e : undone) {
    Shard& s = d->shards[e.second];
    s.state = 0;
    s.owner = -1;
    s.done_by = -1;
    d->queue.push_back(e.second);
  }
  i64 j = d->held[worker];
  if (j < 0) return OK;
  d->shards[j].state = 0;
  d->shards[j].owner = -1;
  d->queue.push_back(j);
  d->held[worker] = -1;
  d->used[worker] = 0;
  return OK;
}

// Forward: pooled[b, c] = sum_{j in bag b} W[row_j, c]; repeated ids count each time.
int orc_embbag_fwd(const void* table, int dtype, i64 n_rows, int dim, const i32* ids,
                   const i64* off, i64 n_bags, float* pooled) {
  int rc = check_bags(ids, off, n_bags, n_rows);
  if (rc != OK) return rc;
  for (i64 b = 0; b < n_bags; ++b)
    for (int c = 0; c < dim; ++c) {
      double s = 0.0;
      for (i64 j = off[b]; j < off[b + 1]; ++j) s += load_elem(table, dtype, (i64)ids[j] * dim + c);
      pooled[b * dim + c] = (float)s;
    }
  return OK;
}

// Backward + dedup, one worker at a time: distinct rows ascending; the occurrences of a row in
// their original order (what a stable sort by row id yields); the worker's MEAN gradient
// G_w[u, c] = (sum_o dY[bag(o), c]) / b_w over its b_w samples.
// Returns the total number of unique (worker, row) pairs, or -(error code).
i64 orc_embbag_bwd_dedup(const i32* ids, const i64* off, i64 n_bags, int F, const float* dY,
                         int dim, i64 n_rows, int K, const i64* wso, i32* uniq_ids, i64* wuo,
                         i64* seg_off, i32* sorted_occ, float* uniq_grads, i64 cap) {
  int rc = check_bags(ids, off, n_bags, n_rows);
  if (rc != OK) return -rc;
  if (wso[0] != 0 || wso[K] * F != n_bags) return -E_ARG;
  i64 nu = 0;
  for (int w = 0; w < K; ++w) {
    wuo[w] = nu;
    i64 b0 = wso[w] * F, b1 = wso[w + 1] * F;
    double bw = (double)(wso[w + 1] - wso[w]);
    std::vector<std::pair<i32, i32> > occ;  // (row, bag), listed in occurrence order
    for (i64 b = b0; b < b1; ++b)
      for (i64 j = off[b]; j < off[b + 1]; ++j) occ.push_back(std::make_pair(ids[j], (i32)b));
    std::stable_sort(occ.begin(), occ.end(),
                     [](const std::pair<i32, i32>& a, const std::pair<i32, i32>& b) {
                       return a.first < b.first;
                     });
    i64 base = off[b0];
    size_t p = 0;
    while (p < occ.size()) {
      size_t e = p;
      while (e < occ.size() && occ[e].first == occ[p].first) ++e;
      if (nu >= cap) return -E_CAP;
      uniq_ids[nu] = occ[p].first;
      seg_off[nu] = base + (i64)p;
      for (int c = 0; c < dim; ++c) {
        double s = 0.0;
        for (size_t k = p; k < e; ++k) s += (double)dY[(i64)occ[k].second * dim + c];
        uniq_grads[nu * dim + c] = (float)(s / bw);
      }
      for (size_t k = p; k < e; ++k) sorted_occ[base + (i64)k] = occ[k].second;
      ++nu;
      p = e;
    }
  }
  wuo[K] = nu;
  seg_off[nu] = off[n_bags];
  return nu;
}

// AntDT-DD with gradient accumulation (Section VI-B, the paragraph before Eq. 4): a device whose
// plan is (B_w, C_w) runs C_w micro-batches of B_w samples between two synchronisations and
// pushes the accumulated gradient.  Worker w's samples [wso[w], wso[w+1]) are its C_w micro-batches
// back to back (so C_w divides their number); each micro-batch yields its own mean gradient over
// its B_w samples, and the pushed gradient is the mean of those C_w means.  A row that a
// micro-batch does not touch gets zero from it.  Distinct rows ascending per worker, as above.
// Returns the number of (worker, row) pairs, or -(error code).
i64 orc_embbag_bwd_accum(const i32* ids, const i64* off, i64 n_bags, int F, const float* dY, int dim,
                         i64 n_rows, int K, const i64* wso, const i64* micro, i32* uniq_ids,
                         i64* wuo, float* uniq_grads, i64 cap) {
  int rc = check_bags(ids, off, n_bags, n_rows);
  if (rc != OK) return -rc;
  if (wso[0] != 0 || wso[K] * F != n_bags) return -E_ARG;
  i64 nu = 0;
  for (int w = 0; w < K; ++w) {
    wuo[w] = nu;
    const i64 n_w = wso[w + 1] - wso[w], C = micro[w];
    if (C < 1 || n_w % C != 0) return -E_ARG;
    const i64 Bw = n_w / C;
    std::map<i32, std::vector<double> > pushed;  // sum over micro-batches of their mean gradients
    for (i64 c = 0; c < C; ++c) {
      std::map<i32, std::vector<double> > local;  // this micro-batch's gradient SUM per row
      const i64 s0 = wso[w] + c * Bw;
      for (i64 b = s0 * F; b < (s0 + Bw) * F; ++b)
        for (i64 j = off[b]; j < off[b + 1]; ++j) {
          std::vector<double>& g = local[ids[j]];
          if (g.empty()) g.assign(dim, 0.0);
          for (int e = 0; e < dim; ++e) g[e] += (double)dY[b * dim + e];
        }
      for (const auto& kv : local) {
        std::vector<double>& g = pushed[kv.first];
        if (g.empty()) g.assign(dim, 0.0);
        for (int e = 0; e < dim; ++e) g[e] += kv.second[e] / (double)Bw;  // the micro-batch mean
      }
    }
    for (const auto& kv : pushed) {
      if (nu >= cap) return -E_CAP;
      uniq_ids[nu] = kv.first;
      for (int e = 0; e < dim; ++e) uniq_grads[nu * dim + e] = (float)(kv.second[e] / (double)C);
      ++nu;
    }
  }
  wuo[K] = nu;
  return nu;
}

// Aggregation of mean gradients over unequal local batches: weights b_i / sum_j b_j, so that
// the result is the mean over the fixed global batch (Section II, Eq. 1: sum_i B_i = B).
// Union of the workers' row lists ascending; absent rows contribute nothing; ascending i.
// Returns the number of aggregated rows or -(error code).
i64 orc_aggregate_sparse(int dim, const i32* uniq_ids, const i64* wuo, const float* uniq_grads,
                         const i64* bsz, int K, i32* agg_ids, float* agg_grads, i64 cap) {
  double tot = 0.0;
  for (int i = 0; i < K; ++i) tot += (double)bsz[i];
  if (!(tot > 0.0)) return -E_ARG;
  std::vector<i32> all(uniq_ids, uniq_ids + wuo[K]);
  std::sort(all.begin(), all.end());
  all.erase(std::unique(all.begin(), all.end()), all.end());
  if ((i64)all.size() > cap) return -E_CAP;
  for (size_t u = 0; u < all.size(); ++u) {
    agg_ids[u] = all[u];
    std::vector<double> s(dim, 0.0);
    for (int i = 0; i < K; ++i) {
      const i32* lo = uniq_ids + wuo[i];
      const i32* hi = uniq_ids + wuo[i + 1];
      const i32* it = std::lower_bound(lo, hi, all[u]);
      if (it == hi || *it != all[u]) continue;
      double wi = (double)bsz[i] / tot;
      const float* g = uniq_grads + (i64)(it - uniq_ids) * dim;
      for (int c = 0; c < dim; ++c) s[c] += wi * (double)g[c];
    }
    for (int c = 0; c < dim; ++c) agg_grads[(i64)u * dim + c] = (float)s[c];
  }
  return (i64)all.size();
}

int orc_aggregate_dense(const float* grads, i64 n, i64 stride, const i64* bsz, int K, float* out) {
  double tot = 0.0;
  for (int i = 0; i < K; ++i) tot += (double)bsz[i];
  if (!(tot > 0.0)) return E_ARG;
  for (i64 e = 0; e < n; ++e) {
    double s = 0.0;
    for (int i = 0; i < K; ++i) s += ((double)bsz[i] / tot) * (double)grads[(i64)i * stride + e];
    out[e] = (float)s;
  }
  return OK;
}

// Sparse optimizer step on the listed rows only (lazy: untouched rows keep their state).
// Adagrad (Duchi et al. 2011): acc += g^2; w -= lr * g / (sqrt(acc) + eps).
// Adam (Kingma & Ba 2015) with bias correction by the global step t.
int orc_sparse_opt_update(void* table, int dtype, i64 n_rows, int dim, const i32* ids,
                          const float* grads, i64 n_ids, int opt, float lr, float eps, float b1,
                          float b2, i64 t, float* s0, float* s1) {
  for (i64 k = 0; k < n_ids; ++k)
    if (ids[k] < 0 || ids[k] >= n_rows) return E_ID;
  double c1 = 1.0 - std::pow((double)b1, (double)t), c2 = 1.0 - std::pow((double)b2, (double)t);
  for (i64 k = 0; k < n_ids; ++k)
    for (int c = 0; c < dim; ++c) {
      i64 at = (i64)ids[k] * dim + c;
      double g = (double)grads[k * dim + c];
      double w = load_elem(table, dtype, at);
      if (opt == 0) {
        double acc = (double)s0[at] + g * g;
        s0[at] = (float)acc;
        w -= (double)lr * g / (std::sqrt(acc) + (double)eps);
      } else {
        double m = (double)b1 * (double)s0[at] + (1.0 - (double)b1) * g;
        double v = (double)b2 * (double)s1[at] + (1.0 - (double)b2) * g * g;
        s0[at] = (float)m;
        s1[at] = (float)v;
        w -= (double)lr * (m / c1) / (std::sqrt(v / c2) + (double)eps);
      }
      store_elem(table, dtype, at, w);
    }
  return OK;
}

// Row-wise Adagrad: ONE accumulator per row, fed with the mean of the row's squared gradient
// elements:  acc_r += (1/D) sum_c g_c^2;  w_c -= lr * g_c / (sqrt(acc_r) + eps).
// s0 is [n_rows].  (The servers' update, Section II, with the accumulator shared by a row.)
int orc_sparse_rowwise_adagrad(void* table, int dtype, i64 n_rows, int dim, const i32* ids,
                               const float* grads, i64 n_ids, float lr, float eps, float* s0) {
  for (i64 k = 0; k < n_ids; ++k)
    if (ids[k] < 0 || ids[k] >= n_rows) return E_ID;
  for (i64 k = 0; k < n_ids; ++k) {
    double sq = 0.0;
    for (int c = 0; c < dim; ++c) {
      double g = (double)grads[k * dim + c];
      sq += g * g;
    }
    double acc = (double)s0[ids[k]] + sq / (double)dim;
    s0[ids[k]] = (float)acc;
    for (int c = 0; c < dim; ++c) {
      i64 at = (i64)ids[k] * dim + c;
      double w = load_elem(table, dtype, at);
      w -= (double)lr * (double)grads[k * dim + c] / (std::sqrt(acc) + (double)eps);
      store_elem(table, dtype, at, w);
    }
  }
  return OK;
}

// Optimizer step on a dense fp32 parameter vector with the aggregated dense gradient (Section
// II: the servers update the parameters after aggregating): the same element-wise Adagrad /
// Adam formulas as the sparse update, every element touched.
int orc_dense_opt_update(float* w, const float* grad, i64 n, int opt, float lr, float eps, float b1,
                         float b2, i64 t, float* s0, float* s1) {
  double c1 = 1.0 - std::pow((double)b1, (double)t), c2 = 1.0 - std::pow((double)b2, (double)t);
  for (i64 e = 0; e < n; ++e) {
    double g = (double)grad[e], x = (double)w[e];
    if (opt == 0) {
      double acc = (double)s0[e] + g * g;
      s0[e] = (float)acc;
      x -= (double)lr * g / (std::sqrt(acc) + (double)eps);
    } else {
      double m = (double)b1 * (double)s0[e] + (1.0 - (double)b1) * g;
      double v = (double)b2 * (double)s1[e] + (1.0 - (double)b2) * g * g;
      s0[e] = (float)m;
      s1[e] = (float)v;
      x -= (double)lr * (m / c1) / (std::sqrt(v / c2) + (double)eps);
    }
    w[e] = (float)x;
  }
  return OK;
}

// AntDT-ND controller, worker side (Section VI-A steps 2-5), stateless form: the whole report
// history is passed in.  reports: n_rep rows (worker, batch size, BPT seconds) in arrival order.
// Window means over each worker's last Lt / Lp reports; straggler if mean_i >= lambda * mean over
// workers; v_i = mean over the short window of batch / BPT.  action: 2 kill-restart if any
// persistent, else 1 adjust-bs if any transient, else 0.
int orc_ctl_decide(const double* reports, i64 n_rep, int K, int Lt, int Lp, double lambda,
                   double* speeds, int* trans, int* pers, int* action) {
  std::vector<std::vector<double> > bpt(K), rate(K);
  for (i64 r = 0; r < n_rep; ++r) {
    int w = (int)reports[3 * r];
    if (w < 0 || w >= K || !(reports[3 * r + 2] > 0.0)) return E_ARG;
    bpt[w].push_back(reports[3 * r + 2]);
    rate[w].push_back(reports[3 * r + 1] / reports[3 * r + 2]);
  }
  std::vector<double> mt(K), mp(K);
  double at = 0.0, ap = 0.0;
  for (int i = 0; i < K; ++i) {
    if (bpt[i].empty()) return 8;
    size_t n = bpt[i].size();
    size_t nt = std::min<size_t>(n, Lt), np_ = std::min<size_t>(n, Lp);
    double s = 0.0, sr = 0.0, sp = 0.0;
    for (size_t k = n - nt; k < n; ++k) { s += bpt[i][k]; sr += rate[i][k]; }
    for (size_t k = n - np_; k < n; ++k) sp += bpt[i][k];
    mt[i] = s / (double)nt;
    speeds[i] = sr / (double)nt;
    mp[i] = sp / (double)np_;
    at += mt[i];
    ap += mp[i];
  }
  at /= K;
  ap /= K;
  bool anyt = false, anyp = false;
  for (int i = 0; i < K; ++i) {
    trans[i] = mt[i] >= lambda * at;
    pers[i] = mp[i] >= lambda * ap;
    anyt = anyt || trans[i];
    anyp = anyp || pers[i];
  }
  *action = anyp ? 2 : (anyt ? 1 : 0);
  return OK;
}

// AntDT-DD, Eq. 4 (sum over the k device types): plain exhaustive search over every (C, B) in
// lexicographic order of (C_1..C_k, B_1..B_k); the first strictly better point is kept, so ties
// go to the lexicographically smallest.  Returns 10 when nothing is feasible.
int orc_dd_solve(int k, const int* n_dev, const double* v, i64 B, const i64* bmin, const i64* bmax,
                 int cmin, int cmax, i64* b_out, int* c_out, double* z_out) {
  if (k < 1 || k > 8) return E_ARG;
  std::vector<int> c(k, cmin);
  bool found = false;
  double best = 0.0;
  for (;;) {  // odometer over C, last index fastest
    std::vector<i64> b(bmin, bmin + k);
    for (;;) {  // odometer over B, last index fastest
      i64 total = 0;
      double z = 0.0;
      for (int i = 0; i < k; ++i) {
        total += (i64)n_dev[i] * c[i] * b[i];
        z = std::max(z, (double)(c[i] * b[i]) / v[i]);
      }
      if (total == B && (!found || z < best)) {
        found = true;
        best = z;
        for (int i = 0; i < k; ++i) { b_out[i] = b[i]; c_out[i] = c[i]; }
      }
      int i = k - 1;
      while (i >= 0 && b[i] == bmax[i]) { b[i] = bmin[i]; --i; }
      if (i < 0) break;
      b[i] += 1;
    }
    int i = k - 1;
    while (i >= 0 && c[i] == cmax) { c[i] = cmin; --i; }
    if (i < 0) break;
    c[i] += 1;
  }
  if (!found) return 10;
  *z_out = best;
  return OK;
}

// Backup-workers aggregation (Section VII-A.3): the dropped workers do not exist for this step.
// Union and weights over the surviving workers only, w_i = b_i / sum_{surviving} b_j.
i64 orc_aggregate_sparse_backup(int dim, const i32* uniq_ids, const i64* wuo, const float* uniq_grads,
                                const i64* bsz, const uint8_t* dropped, int K, i32* agg_ids,
                                float* agg_grads, i64 cap) {
  double tot = 0.0;
  for (int i = 0; i < K; ++i)
    if (!dropped[i]) tot += (double)bsz[i];
  if (!(tot > 0.0)) return -E_ARG;
  std::vector<i32> all;
  for (int i = 0; i < K; ++i)
    if (!dropped[i]) all.insert(all.end(), uniq_ids + wuo[i], uniq_ids + wuo[i + 1]);
  std::sort(all.begin(), all.end());
  all.erase(std::unique(all.begin(), all.end()), all.end());
  if ((i64)all.size() > cap) return -E_CAP;
  for (size_t u = 0; u < all.size(); ++u) {
    agg_ids[u] = all[u];
    std::vector<double> s(dim, 0.0);
    for (int i = 0; i < K; ++i) {
      if (dropped[i]) continue;
      const i32* lo = uniq_ids + wuo[i];
      const i32* hi = uniq_ids + wuo[i + 1];
      const i32* it = std::lower_bound(lo, hi, all[u]);
      if (it == hi || *it != all[u]) continue;
      double wi = (double)bsz[i] / tot;
      const float* g = uniq_grads + (i64)(it - uniq_ids) * dim;
      for (int c = 0; c < dim; ++c) s[c] += wi * (double)g[c];
    }
    for (int c = 0; c < dim; ++c) agg_grads[(i64)u * dim + c] = (float)s[c];
  }
  return (i64)all.size();
}

int orc_aggregate_dense_backup(const float* grads, i64 n, i64 stride, const i64* bsz,
                               const uint8_t* dropped, int K, float* out) {
  double tot = 0.0;
  for (int i = 0; i < K; ++i)
    if (!dropped[i]) tot += (double)bsz[i];
  if (!(tot > 0.0)) return E_ARG;
  for (i64 e = 0; e < n; ++e) {
    double s = 0.0;
    for (int i = 0; i < K; ++i)
      if (!dropped[i]) s += ((double)bsz[i] / tot) * (double)grads[(i64)i * stride + e];
    out[e] = (float)s;
  }
  return OK;
}

}  // extern "C"
