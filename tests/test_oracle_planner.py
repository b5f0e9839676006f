"""Pins of the CPU checker's planner (shard service + batch sizes) against what the paper and
plain arithmetic fix: closed forms, the paper's printed numbers, exhaustive search, and the
data-integrity invariants of Section V-C / VII-D."""
import itertools

import numpy as np
import pytest

import oracle
from tests.util import read_golden

G = read_golden("paper_values.txt")


# ---- shard layout: K = ceil(N/(B*M)), shard = (start, length)  (Section V-C.1) ----------
def test_shard_count_and_layout_tiny():
    d = oracle.Dds(10, 2, 2, 3)
    assert d.num_shards() == 3
    got = [d.shard_info(j)[2:] for j in range(3)]
    assert got == [(0, 4), (4, 4), (8, 2)]
    assert d.counts() == (3, 0, 0)


def test_shard_count_paper_workload():
    N, B, M = G["criteo_records"], G["xdeepfm_global_batch"], G["batches_per_shard"]
    d = oracle.Dds(N, B, M, G["xdeepfm_workers"])
    assert d.num_shards() == G["xdeepfm_shards"] == -(-N // (B * M))
    total = sum(d.shard_info(j)[3] for j in range(d.num_shards()))
    assert total == N


# ---- batch sizes -----------------------------------------------------------------------
def test_equal_init_matches_paper_local_batch():
    # Section VI-A step 1 (B_i = B/n) on the paper's XDeepFM numbers: 81920 / 20 = 4096
    b = oracle.batch_sizes(None, G["xdeepfm_workers"], G["xdeepfm_global_batch"])
    assert b.tolist() == [G["xdeepfm_local_batch_avg"]] * G["xdeepfm_workers"]


def test_equal_init_remainder_to_low_indices():
    assert oracle.batch_sizes(None, 4, 10).tolist() == [3, 3, 2, 2]


def test_proportional_v100_p100_closed_form():
    v = [G["v100_over_p100"]] * G["cluster_b_v100"] + [1] * G["cluster_b_p100"]
    for rule in ("proportional", "minmax"):
        b = oracle.batch_sizes(v, 8, G["resnet_global_batch"], rule)
        assert b.tolist() == [G["cluster_b_batch_v100"]] * 4 + [G["cluster_b_batch_p100"]] * 4


def test_proportional_config2_closed_form():
    # quotas 16384*v/6.75: 2427.259.. x6, 1213.63, 606.81 -> floors sum to 16381, three units
    # left: largest remainders .81 (w7), .63 (w6), then .259 ties -> lowest index (w0)
    v = [1, 1, 1, 1, 1, 1, .5, .25]
    b = oracle.batch_sizes(v, 8, 16384, "proportional")
    assert b.tolist() == [2428, 2427, 2427, 2427, 2427, 2427, 1214, 607]


def test_minmax_config2():
    v = [1, 1, 1, 1, 1, 1, .5, .25]
    b = oracle.batch_sizes(v, 8, 16384, "minmax")
    assert b.sum() == 16384
    z = max(bi / vi for bi, vi in zip(b, v))
    # lower bound of Eq. 3: z >= B / sum(v) = 2427.26 and z*v_i must reach an integer
    assert z == 2428.0
    assert b.tolist() == [2428, 2428, 2428, 2427, 2427, 2427, 1213, 606]


def _compositions(total, n, lo):
    if n == 1:
        if total >= lo:
            yield (total,)
        return
    for first in range(lo, total - lo * (n - 1) + 1):
        for rest in _compositions(total - first, n - 1, lo):
            yield (first,) + rest


@pytest.mark.parametrize("n", [2, 3, 4])
def test_minmax_is_optimal_by_exhaustive_search(n):
    rng = np.random.default_rng(100 + n)
    for trial in range(12):
        B = int(rng.integers(n, 25))
        lo = int(rng.integers(0, B // n + 1)) if trial % 2 else 0
        v = rng.uniform(0.2, 3.0, size=n)
        b = oracle.batch_sizes(v, n, B, "minmax", lo)
        assert b.sum() == B and b.min() >= lo
        best = min(max(c[i] / v[i] for i in range(n)) for c in _compositions(B, n, lo))
        assert max(b[i] / v[i] for i in range(n)) == pytest.approx(best, rel=0, abs=0)


def test_proportional_within_one_unit_of_quota_and_monotone():
    rng = np.random.default_rng(7)
    for _ in range(50):
        n = int(rng.integers(2, 40))
        B = int(rng.integers(n, 100000))
        v = np.exp(rng.normal(0, 0.5, size=n))
        b = oracle.batch_sizes(v, n, B, "proportional")
        q = B * v / v.sum()
        assert b.sum() == B
        assert np.all(np.abs(b - q) < 1.0 + 1e-9)
        # faster worker never gets less (Section V-C.2 / VII-D.1: allocation follows throughput)
        order = np.argsort(v)
        assert np.all(np.diff(b[order]) >= 0)


def test_proportional_min_batch_clamp():
    v = [10.0, 10.0, 0.01, 0.01]
    b = oracle.batch_sizes(v, 4, 1000, "proportional", 100)
    assert b.sum() == 1000 and b.tolist() == [400, 400, 100, 100]
    # what is left after the clamped worker's share goes to the others in proportion to THEIR
    # speeds: 90 * 3/4 = 67.5 and 90 * 1/4 = 22.5, the odd unit to the lower index.  (Two equal
    # fast workers would hide a split of the whole batch instead of the remainder: 50 + 50 comes
    # back to 45 + 45 whichever way the surplus is taken off.)
    assert oracle.batch_sizes([3.0, 1.0, 0.02], 3, 100, "proportional", 10).tolist() == [68, 22, 10]
    with pytest.raises(oracle.OracleError):
        oracle.batch_sizes(v, 4, 1000, "proportional", 251)
    with pytest.raises(oracle.OracleError):
        oracle.batch_sizes([1.0, 0.0], 2, 10)
    with pytest.raises(oracle.OracleError):
        oracle.batch_sizes([1.0, float("nan")], 2, 10)


# ---- the data service ------------------------------------------------------------------
def _run_epoch(d, K, N, rng, speeds_fn, requeue_prob=0.0, rule="proportional"):
    cover = np.zeros(N, np.int64)
    steps = 0
    while True:
        rc, bsz, ro, rg, cnt = d.plan(speeds_fn(), rule, 0, cap=10000)
        if rc == 7:
            break
        assert rc == 0
        assert bsz.sum() == d_B(d)
        # a dropped worker's gradient never arrives: its samples of this step do not count
        dropped = int(rng.integers(0, K)) if requeue_prob and rng.random() < requeue_prob else -1
        for i in range(K):
            got = 0
            for s, n in rg[ro[i]:ro[i + 1]]:
                if i != dropped:
                    cover[s:s + n] += 1
                got += n
            assert got == cnt[i] <= bsz[i]
        steps += 1
        if dropped >= 0:
            d.requeue_worker(dropped)
        assert steps < 100000
    return cover, steps


def d_B(d):
    return d._B


def _mk(N, B, M, K, seed=0):
    d = oracle.Dds(N, B, M, K, seed)
    d._B = B
    return d


@pytest.mark.parametrize("shuffle", [0, 12345])
def test_every_sample_exactly_once_per_epoch(shuffle):
    rng = np.random.default_rng(3)
    for N, B, M, K in [(1000, 16, 3, 4), (997, 10, 1, 3), (50, 64, 2, 5), (640, 32, 2, 1)]:
        d = _mk(N, B, M, K, shuffle)
        cover, _ = _run_epoch(d, K, N, rng, lambda: np.exp(rng.normal(0, 0.7, size=K)))
        assert np.all(cover == 1)
        todo, doing, done = d.counts()
        assert (todo, doing, done) == (0, 0, -(-N // (B * M)))  # Section VII-D.2


def test_at_least_once_with_requeues_and_done_count():
    rng = np.random.default_rng(4)
    N, B, M, K = 2000, 20, 4, 5
    d = _mk(N, B, M, K, 99)
    cover, _ = _run_epoch(d, K, N, rng, lambda: np.exp(rng.normal(0, 0.7, size=K)), 0.3)
    assert np.all(cover >= 1) and cover.max() >= 2
    assert d.counts() == (0, 0, -(-N // (B * M)))


def test_drop_on_the_step_that_finishes_a_shard_loses_no_sample():
    # 6 shards of 100 samples (M = 1), speeds 3:1 -> batches 75 / 25.  Step 1: worker 0 takes
    # 0..74 of shard 0.  Step 2: it takes 75..99 (shard 0 finished) and 200..249 of shard 2; its
    # gradient is then dropped.  Samples 75..99 were in no gradient that arrived, so shard 0 must
    # come back although its last sample was served (Section V-C.3: DONE needs the push).
    N, B, M, K = 600, 100, 1, 2
    d = _mk(N, B, M, K)
    cover = np.zeros(N, np.int64)
    step = 0
    while True:
        rc, bsz, ro, rg, cnt = d.plan([3.0, 1.0])
        if rc == 7:
            break
        step += 1
        drop = 0 if step == 2 else -1
        if step == 2:
            assert rg[ro[0]:ro[1]].tolist() == [[75, 25], [200, 50]]
            assert d.shard_info(0)[0] == 2                       # provisionally DONE
        for i in range(K):
            for s, n in rg[ro[i]:ro[i + 1]]:
                if i != drop:
                    cover[s:s + n] += 1
        if drop >= 0:
            d.requeue_worker(drop)
            # both come back, the finished one first, behind the shards still queued
            assert d.shard_info(0)[:2] == (0, -1) and d.shard_info(2)[:2] == (0, -1)
    assert np.all(cover >= 1)
    assert cover[:75].tolist() == [2] * 75 and cover[75:100].tolist() == [1] * 25
    assert d.counts() == (0, 0, 6)
    # a requeue that comes after the NEXT plan call no longer touches what that worker finished
    d = _mk(N, B, M, K)
    d.plan([3.0, 1.0]); d.plan([3.0, 1.0]); d.plan([3.0, 1.0])
    assert d.shard_info(0)[0] == 2
    d.requeue_worker(0)
    assert d.shard_info(0)[0] == 2


def test_requeue_order_when_a_dropped_worker_finished_two_shards_in_one_step():
    # 33 samples, B = 10, M = 1: shards 0..2 of 10 samples and the short tail shard 3 = [30, 33).
    # A worker can only finish two shards in one step when the second is that tail.
    # Step 1 (speeds 8:1:1 -> batches 8/1/1): worker 0 holds shard 0 (8 used), worker 1 shard 1,
    # worker 2 shard 2; the queue is [3].  Workers 1 and 2 are dropped: queue [3, 1, 2].
    # Step 2 (only worker 0 gets samples): it finishes shard 0 (2 samples), takes and finishes the
    # tail (3 samples) and takes 5 of shard 1; the queue is [2].  Worker 0 is dropped: the shards it
    # finished in this step come back behind what is queued, the older completion first, then the
    # one it is DOING (Section V-C.3): [2, 0, 3, 1].
    d = _mk(33, 10, 1, 3)
    rc, bsz, ro, rg, cnt = d.plan([8.0, 1.0, 1.0])
    assert rc == 0 and bsz.tolist() == [8, 1, 1] and rg.tolist() == [[0, 8], [10, 1], [20, 1]]
    d.requeue_worker(1)
    d.requeue_worker(2)
    rc, bsz, ro, rg, cnt = d.plan([1.0, 1e-9, 1e-9])
    assert rc == 0 and bsz.tolist() == [10, 0, 0]
    assert rg[ro[0]:ro[1]].tolist() == [[8, 2], [30, 3], [10, 5]]
    assert d.shard_info(0)[0] == 2 and d.shard_info(3)[0] == 2 and d.shard_info(1)[:2] == (1, 0)
    d.requeue_worker(0)
    assert d.counts() == (4, 0, 0)
    served = []
    while True:                       # worker 1 alone drains the queue, a whole batch per step
        rc, bsz, ro, rg, cnt = d.plan([1e-9, 1.0, 1e-9])
        if rc == 7:
            break
        served += rg[ro[1]:ro[2]].tolist()
    assert served == [[20, 10], [0, 10], [30, 3], [10, 7], [17, 3]]


def test_shuffle_can_leave_a_shard_in_its_place():
    # A uniform shuffle of two shards keeps their order for about half of the seeds; a shuffle
    # that always moves every element (a cyclic permutation) would swap them for every seed.
    first = []
    for seed in range(1, 65):
        d = oracle.Dds(20, 10, 1, 1, seed)
        rc, bsz, ro, rg, cnt = d.plan(None)
        first.append(int(rg[0][0]))
    assert 16 <= first.count(0) <= 48 and first.count(0) + first.count(10) == 64


def test_doing_shard_is_exclusive_and_requeue_goes_to_queue_end():
    N, B, M, K = 6 * 8, 4, 2, 2   # 6 shards of 8 samples
    d = _mk(N, B, M, K)
    rc, bsz, ro, rg, cnt = d.plan(None)
    assert rc == 0 and bsz.tolist() == [2, 2]
    assert rg.tolist() == [[0, 2], [8, 2]]          # worker 0 holds shard 0, worker 1 shard 1
    assert d.shard_info(0)[:2] == (1, 0) and d.shard_info(1)[:2] == (1, 1)
    assert d.counts() == (4, 2, 0)
    d.requeue_worker(0)                              # shard 0 -> TODO, end of queue
    assert d.shard_info(0)[:2] == (0, -1)
    seen = []
    for _ in range(200):
        rc, bsz, ro, rg, cnt = d.plan(None)
        if rc == 7:
            break
        for s, n in rg[ro[0]:ro[1]]:
            seen.append(int(s) // 8)
    # worker 0 then works through shards 2.. and gets shard 0 back only after 2..5 were taken
    first_of_shard0 = seen.index(0)
    assert all(x != 0 for x in seen[:first_of_shard0]) and first_of_shard0 > 0
    taken_before = set(seen[:first_of_shard0])
    assert 2 in taken_before
    assert d.counts() == (0, 0, 6)


def test_batch_spans_two_shards_and_epoch_tail_is_short():
    d = _mk(20, 8, 1, 1)   # shards (0,8) (8,8) (16,4); one worker, batch 8
    got = []
    while True:
        rc, bsz, ro, rg, cnt = d.plan(None)
        if rc == 7:
            assert cnt.sum() == 0
            break
        got.append((rg.tolist(), int(cnt[0])))
    assert got == [([[0, 8]], 8), ([[8, 8]], 8), ([[16, 4]], 4)]
    d = _mk(20, 6, 1, 1)   # shards of 6: a batch of 6 never spans; use unequal speeds, K=2
    d = _mk(24, 6, 1, 2)
    rc, bsz, ro, rg, cnt = d.plan([5.0, 1.0])
    assert bsz.tolist() == [5, 1] and rg.tolist() == [[0, 5], [6, 1]]
    rc, bsz, ro, rg, cnt = d.plan([5.0, 1.0])
    # worker 0 finishes shard 0 (1 sample left) and continues in the next TODO shard
    assert rg[ro[0]:ro[1]].tolist() == [[5, 1], [12, 4]]
    assert d.shard_info(0)[0] == 2


def test_faster_worker_consumes_more_shards():
    # Section VII-D.1: shards consumed follow worker throughput
    N, B, M, K = 40000, 40, 5, 4
    d = _mk(N, B, M, K)
    v = [4.0, 2.0, 1.0, 1.0]
    served = np.zeros(K)
    while True:
        rc, bsz, ro, rg, cnt = d.plan(v)
        if rc == 7:
            break
        served += cnt
    assert served.sum() == N
    assert served[0] > served[1] > served[2] and served[2] == pytest.approx(served[3], rel=0.05)
    assert served[0] / served[2] == pytest.approx(4.0, rel=0.05)
