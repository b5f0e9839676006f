/*
 * Controller front end of AntDT-ND for worker stragglers (Section VI-A, steps 2-5), host C.
 *
 * Workers report (batch size, batch processing time) pairs; the controller keeps the last
 * L^trans and L^per reports of every worker (the paper's windows are minutes of reports; here a
 * window is a number of reports, which is the same thing at a fixed report rate), averages the
 * BPT over both, flags worker i as a transient / persistent straggler when its window mean is
 * at least lambda times the mean over all workers, and estimates the throughput v_i handed to
 * the batch-size solver as the mean over the short window of (batch size / BPT) of each report.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include "antdt.h"

struct antdt_ctl {
  int32_t n_workers, win_trans, win_per;
  double lambda;
  int32_t cap;        /* ring capacity per worker = max(win_trans, win_per) */
  double* bpt;        /* [K][cap] */
  double* rate;       /* [K][cap] batch / bpt */
  int64_t* count;     /* [K] reports seen */
};

int32_t antdt_ctl_create(antdt_ctl** out, int32_t n_workers, int32_t window_trans,
                         int32_t window_per, double lambda) {
  if (!out || n_workers < 1 || n_workers > 1024 || window_trans < 1 || window_per < 1 ||
      !(lambda > 1.0) || !isfinite(lambda))
    return ANTDT_ERR_INVALID_ARG;
  antdt_ctl* c = (antdt_ctl*)calloc(1, sizeof(antdt_ctl));
  if (!c) return ANTDT_ERR_INVALID_ARG;
  c->n_workers = n_workers;
  c->win_trans = window_trans;
  c->win_per = window_per;
  c->lambda = lambda;
  c->cap = window_trans > window_per ? window_trans : window_per;
  size_t n = (size_t)n_workers * (size_t)c->cap;
  c->bpt = (double*)calloc(n, sizeof(double));
  c->rate = (double*)calloc(n, sizeof(double));
  c->count = (int64_t*)calloc((size_t)n_workers, sizeof(int64_t));
  if (!c->bpt || !c->rate || !c->count) { antdt_ctl_destroy(c); return ANTDT_ERR_INVALID_ARG; }
  *out = c;
  return ANTDT_OK;
}

void antdt_ctl_destroy(antdt_ctl* c) {
  if (!c) return;
  free(c->bpt); free(c->rate); free(c->count); free(c);
}

int32_t antdt_ctl_report(antdt_ctl* c, int32_t worker, int64_t batch_size, double bpt_seconds) {
  if (!c || worker < 0 || worker >= c->n_workers || batch_size < 0 || !(bpt_seconds > 0.0) ||
      !isfinite(bpt_seconds))
    return ANTDT_ERR_INVALID_ARG;
  size_t slot = (size_t)worker * (size_t)c->cap + (size_t)(c->count[worker] % c->cap);
  c->bpt[slot] = bpt_seconds;
  c->rate[slot] = (double)batch_size / bpt_seconds;
  c->count[worker] += 1;
  return ANTDT_OK;
}

/* mean of the last `win` entries of worker w's ring (oldest first), in `arr` */
static double window_mean(const antdt_ctl* c, const double* arr, int32_t w, int32_t win, int64_t* used) {
  int64_t have = c->count[w] < win ? c->count[w] : win;
  double s = 0.0;
  for (int64_t k = have; k >= 1; --k) {
    int64_t idx = (c->count[w] - k) % c->cap;
    s += arr[(size_t)w * (size_t)c->cap + (size_t)idx];
  }
  *used = have;
  return have ? s / (double)have : 0.0;
}

int32_t antdt_ctl_decide(const antdt_ctl* c, double* speeds, int32_t* transient,
                         int32_t* persistent, int32_t* action) {
  if (!c || !speeds || !transient || !persistent || !action) return ANTDT_ERR_INVALID_ARG;
  const int32_t K = c->n_workers;
  double mt[1024], mp[1024];
  double all_t = 0.0, all_p = 0.0;
  for (int32_t i = 0; i < K; ++i) {
    int64_t used;
    mt[i] = window_mean(c, c->bpt, i, c->win_trans, &used);
    if (used == 0) return ANTDT_ERR_STATE; /* every worker must have reported at least once */
    mp[i] = window_mean(c, c->bpt, i, c->win_per, &used);
    speeds[i] = window_mean(c, c->rate, i, c->win_trans, &used);
    all_t += mt[i];
    all_p += mp[i];
  }
  all_t /= (double)K;
  all_p /= (double)K;
  int any_t = 0, any_p = 0;
  for (int32_t i = 0; i < K; ++i) {
    transient[i] = mt[i] >= c->lambda * all_t;
    persistent[i] = mp[i] >= c->lambda * all_p;
    any_t |= transient[i];
    any_p |= persistent[i];
  }
  *action = any_p ? ANTDT_ACTION_KILL_RESTART : (any_t ? ANTDT_ACTION_ADJUST_BS : ANTDT_ACTION_NONE);
  return ANTDT_OK;
}

/* ====================================================================================== */
/* AntDT-DD (Section VI-B, Eq. 4): batch size B_i and accumulation count C_i per device type */
/* ====================================================================================== */
typedef struct {
  int32_t k;
  const int32_t* n_dev;
  const double* v;
  const int64_t *bmin, *bmax;
  int64_t B;
  int32_t c[8];
  int64_t b[8], best_b[8];
  int32_t best_c[8];
  double best_z;
  int found;
} dd_state;

/* z of a full assignment under the current c: max_i c_i * b_i / v_i */
static double dd_cost(const dd_state* s, int32_t upto) {
  double z = 0.0;
  for (int32_t i = 0; i < upto; ++i) {
    double t = (double)(s->c[i] * s->b[i]) / s->v[i];
    if (t > z) z = t;
  }
  return z;
}

/* choose b[i..k-2] by enumeration (ascending, so the first optimum found is the
 * lexicographically smallest), the last type's batch follows from the equality constraint */
static void dd_search(dd_state* s, int32_t i, int64_t remaining) {
  const int32_t k = s->k;
  if (i == k - 1) {
    int64_t a = (int64_t)s->n_dev[i] * s->c[i];
    if (remaining % a) return;
    int64_t bi = remaining / a;
    if (bi < s->bmin[i] || bi > s->bmax[i]) return;
    s->b[i] = bi;
    double z = dd_cost(s, k);
    if (!s->found || z < s->best_z) {
      s->found = 1;
      s->best_z = z;
      memcpy(s->best_b, s->b, sizeof(s->b));
      memcpy(s->best_c, s->c, sizeof(s->c));
    }
    return;
  }
  int64_t a = (int64_t)s->n_dev[i] * s->c[i];
  for (int64_t bi = s->bmin[i]; bi <= s->bmax[i]; ++bi) {
    if (a * bi > remaining) break;
    /* this type alone already costs more than the best known: larger bi only cost more */
    if (s->found && (double)(s->c[i] * bi) / s->v[i] > s->best_z) break;
    s->b[i] = bi;
    dd_search(s, i + 1, remaining - a * bi);
  }
}

static void dd_enum_c(dd_state* s, int32_t i, int32_t cmin, int32_t cmax) {
  if (i == s->k) { dd_search(s, 0, s->B); return; }
  for (int32_t c = cmin; c <= cmax; ++c) {
    s->c[i] = c;
    dd_enum_c(s, i + 1, cmin, cmax);
  }
}

int32_t antdt_dd_solve(int32_t n_types, const int32_t* n_devices, const double* speeds,
                       int64_t global_batch, const int64_t* batch_min, const int64_t* batch_max,
                       int32_t accum_min, int32_t accum_max, int64_t* batch_out, int32_t* accum_out,
                       double* z_out) {
  if (n_types < 1 || n_types > 8 || !n_devices || !speeds || !batch_min || !batch_max ||
      !batch_out || !accum_out || global_batch < 1 || accum_min < 1 || accum_max < accum_min)
    return ANTDT_ERR_INVALID_ARG;
  for (int32_t i = 0; i < n_types; ++i)
    if (n_devices[i] < 1 || !(speeds[i] > 0.0) || !isfinite(speeds[i]) || batch_min[i] < 1 ||
        batch_max[i] < batch_min[i])
      return ANTDT_ERR_INVALID_ARG;
  dd_state s;
  memset(&s, 0, sizeof(s));
  s.k = n_types; s.n_dev = n_devices; s.v = speeds; s.bmin = batch_min; s.bmax = batch_max;
  s.B = global_batch;
  dd_enum_c(&s, 0, accum_min, accum_max);
  if (!s.found) return ANTDT_ERR_INFEASIBLE;
  for (int32_t i = 0; i < n_types; ++i) { batch_out[i] = s.best_b[i]; accum_out[i] = s.best_c[i]; }
  if (z_out) *z_out = s.best_z;
  return ANTDT_OK;
}
