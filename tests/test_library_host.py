"""CPU-side tests of libantdt.so: it loads, exports every symbol the header declares, rejects
malformed arguments before touching a device, and its host planner reproduces the CPU checker's
plans bit for bit."""
import ctypes as C
import os
import re
import time

import numpy as np
import pytest

import oracle
from paper_2404_09679_b200 import binding as B
from paper_2404_09679_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "antdt.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(antdt_[a-z0-9_]+)\s*\(", hdr))
    assert len(declared) >= 20
    L = B.lib()
    for name in sorted(declared):
        assert hasattr(L, name), name
    assert declared == set(B.EXPORTS)
    assert "sm_100a" in B.antdt_version()


def test_device_calls_reject_bad_arguments_before_any_launch():
    L = B.lib()
    n0 = B.antdt_launch_count()
    one = C.c_void_p(256)  # never dereferenced: every call below fails validation first
    # dim not a multiple of 4
    assert L.antdt_embbag_fwd(one, B.F32, 10, 6, one, 1, one, 1, one, None, None) == B.ERR_INVALID_ARG
    # bf16 needs dim % 8
    assert L.antdt_embbag_fwd(one, B.BF16, 10, 12, one, 1, one, 1, one, None, None) == B.ERR_INVALID_ARG
    # unknown dtype, too many rows, misaligned table
    assert L.antdt_embbag_fwd(one, 7, 10, 8, one, 1, one, 1, one, None, None) == B.ERR_INVALID_ARG
    assert L.antdt_embbag_fwd(one, B.F32, 1 << 31, 8, one, 1, one, 1, one, None, None) == B.ERR_INVALID_ARG
    assert L.antdt_embbag_fwd(C.c_void_p(260), B.F32, 10, 8, one, 1, one, 1, one, None, None) == B.ERR_INVALID_ARG
    wso = (C.c_int64 * 3)(0, 2, 3)
    args = lambda ws_bytes, nb: (one, 8, one, nb, 2, one, 8, 10, 2, wso, one, one, one, one, one, 8,
                                 one, ws_bytes, None, None)
    assert L.antdt_embbag_bwd_dedup(*args(1 << 30, 5)) == B.ERR_INVALID_ARG      # 3*2 != 5 bags
    need = B.antdt_embbag_bwd_dedup_workspace_bytes(8, 6, 8, 2)
    assert need > 0
    assert L.antdt_embbag_bwd_dedup(*args(need - 1, 6)) == B.ERR_WORKSPACE_TOO_SMALL
    bad_wso = (C.c_int64 * 3)(0, 4, 3)
    a = list(args(need, 6))
    a[9] = bad_wso
    assert L.antdt_embbag_bwd_dedup(*a) == B.ERR_INVALID_ARG
    bsz = (C.c_int64 * 2)(0, 0)
    assert L.antdt_weighted_aggregate(None, None, bsz, 2, one, 1 << 20, None, None) == B.ERR_INVALID_ARG
    assert L.antdt_sparse_opt_update(one, B.F32, 10, 8, one, one, one, 4, 5, 0.1, 1e-8, 0.9, 0.999, 1,
                                     one, None, None, None) == B.ERR_INVALID_ARG   # unknown optimizer
    assert L.antdt_sparse_opt_update(one, B.F32, 10, 8, one, one, one, 4, B.OPT_ADAM, 0.1, 1e-8, 0.9,
                                     0.999, 1, one, None, None, None) == B.ERR_INVALID_ARG  # Adam, no v
    assert L.antdt_sparse_opt_update(one, B.F32, 10, 8, one, one, one, 4, B.OPT_ADAGRAD, 0.1, 1e-8, 0.9,
                                     0.999, 0, one, None, None, None) == B.ERR_INVALID_ARG  # step 0
    assert B.antdt_launch_count() == n0
    assert B.antdt_weighted_aggregate_workspace_bytes(100, 16, 4) > 0
    assert B.antdt_weighted_aggregate_workspace_bytes(100, 16, 2000) == 0
    # a step's workspace: room for both scratch areas side by side on a small batch (the
    # three-branch graph), the larger of the two on a large one, 0 when either figure is 0
    b = B.antdt_embbag_bwd_dedup_workspace_bytes(1000, 100, 16, 4)
    a = B.antdt_weighted_aggregate_workspace_bytes(1000, 16, 4)
    assert B.antdt_bsp_step_workspace_bytes(1000, 100, 16, 4, 1000) == (b + 255) // 256 * 256 + a
    big = 1 << 23
    b = B.antdt_embbag_bwd_dedup_workspace_bytes(big, big, 16, 4)
    a = B.antdt_weighted_aggregate_workspace_bytes(big, 16, 4)
    assert B.antdt_bsp_step_workspace_bytes(big, big, 16, 4, big) == max(a, b)
    assert B.antdt_bsp_step_workspace_bytes(1000, 100, 16, 2000, 1000) == 0


# ---- planner: library vs checker, bit for bit ---------------------------------------------
@pytest.mark.parametrize("rule", ["proportional", "minmax"])
def test_batch_sizes_match_checker(rule):
    rng = np.random.default_rng(1)
    for _ in range(300):
        n = int(rng.integers(1, 70))
        B_ = int(rng.integers(n, 300000))
        minb = int(rng.integers(0, B_ // n + 1)) if rng.random() < 0.5 else 0
        v = np.exp(rng.normal(0, rng.choice([0.1, 0.5, 2.0]), size=n))
        if rng.random() < 0.2:
            v = np.round(v * 4) / 4 + 0.25     # many exact ties
        want = oracle.batch_sizes(v, n, B_, rule, minb)
        got = B.antdt_batch_sizes(v, n, B_, B.RULES[rule], minb)
        assert got == want.tolist()
    assert B.antdt_batch_sizes(None, 4, 10) == [3, 3, 2, 2]
    for bad in ([1.0, -1.0], [1.0, float("inf")], [float("nan"), 1.0]):
        with pytest.raises(B.AntdtError):
            B.antdt_batch_sizes(bad, 2, 10)
    with pytest.raises(B.AntdtError):
        B.antdt_batch_sizes([1.0, 1.0], 2, 10, B.RULE_PROPORTIONAL, 6)


def test_paper_cases_on_the_library():
    assert B.antdt_batch_sizes([3, 3, 3, 3, 1, 1, 1, 1], 8, 768) == [144] * 4 + [48] * 4
    assert B.antdt_batch_sizes(None, 20, 81920) == [4096] * 20
    assert B.antdt_batch_sizes([1, 1, 1, 1, 1, 1, .5, .25], 8, 16384) == \
        [2428, 2427, 2427, 2427, 2427, 2427, 1214, 607]
    d = B.Dds(45_000_000, 81920, 100, 20)
    assert d.antdt_dds_num_shards() == 6


@pytest.mark.parametrize("seed", [0, 5, 77])
def test_shard_plans_match_checker_through_a_whole_epoch_with_requeues(seed):
    rng = np.random.default_rng(seed)
    N, B_, M, K = int(rng.integers(500, 5000)), int(rng.integers(8, 64)), int(rng.integers(1, 5)), \
        int(rng.integers(1, 9))
    shuffle = int(rng.integers(0, 2)) * 4242
    a, b = oracle.Dds(N, B_, M, K, shuffle), B.Dds(N, B_, M, K, shuffle)
    assert a.num_shards() == b.antdt_dds_num_shards()
    cover = np.zeros(N, np.int64)
    for step in range(100000):
        v = np.exp(rng.normal(0, 0.6, size=K)) if step else None
        rule = "minmax" if step % 3 == 2 else "proportional"
        minb = 1 if step % 5 == 4 and K <= B_ else 0
        rc_a, bs_a, ro_a, rg_a, cnt_a = a.plan(v, rule, minb, cap=1000)
        rc_b, bs_b, ro_b, rg_b, cnt_b = b.antdt_shard_plan(v, B.RULES[rule], minb, 1000)
        assert rc_a == rc_b
        assert bs_a.tolist() == bs_b and cnt_a.tolist() == cnt_b and ro_a.tolist() == ro_b
        assert rg_a.tolist() == [list(r) for r in rg_b]
        assert a.counts() == b.antdt_dds_counts()
        if rc_a == 7:
            break
        assert sum(bs_b) == B_
        # a dropped worker's samples of this step are in no gradient that arrived
        w = int(rng.integers(0, K)) if rng.random() < 0.15 else -1
        for i in range(K):
            if i != w:
                for s, n in rg_b[ro_b[i]:ro_b[i + 1]]:
                    cover[s:s + n] += 1
        if w >= 0:
            a.requeue_worker(w)
            b.antdt_dds_requeue_worker(w)
            for j in range(a.num_shards()):
                assert a.shard_info(j) == b.antdt_dds_shard_info(j)
    assert np.all(cover >= 1)
    assert b.antdt_dds_counts() == (0, 0, -(-N // (B_ * M)))


def test_exactly_once_without_loss_on_the_library():
    N, B_, M, K = 3001, 24, 3, 5
    d = B.Dds(N, B_, M, K, 9)
    cover = np.zeros(N, np.int64)
    rng = np.random.default_rng(2)
    while True:
        rc, bs, ro, rg, cnt = d.antdt_shard_plan(np.exp(rng.normal(0, 0.5, size=K)))
        if rc == B.ERR_EXHAUSTED:
            assert sum(cnt) == 0
            break
        for s, n in rg:
            cover[s:s + n] += 1
    assert np.all(cover == 1)


def test_plan_capacity_error_leaves_state_unchanged():
    d = B.Dds(1000, 10, 1, 4)
    before = d.antdt_dds_save()
    with pytest.raises(B.AntdtError) as e:
        d.antdt_shard_plan(None, ranges_cap=2)
    assert e.value.code == B.ERR_CAPACITY
    assert d.antdt_dds_save() == before and d.antdt_dds_counts() == (100, 0, 0)


def test_save_load_round_trip_mid_epoch():
    rng = np.random.default_rng(3)
    d = B.Dds(4000, 32, 2, 6, 17)
    for _ in range(20):
        d.antdt_shard_plan(np.exp(rng.normal(0, 0.5, size=6)))
    d.antdt_dds_requeue_worker(2)
    img = d.antdt_dds_save()
    e = B.Dds.antdt_dds_load(img, 6)
    assert e.antdt_dds_save() == img
    for _ in range(200):
        v = np.exp(rng.normal(0, 0.5, size=6))
        ra, rb = d.antdt_shard_plan(v), e.antdt_shard_plan(v)
        assert ra == rb
        if ra[0] == B.ERR_EXHAUSTED:
            break
    # the image carries the shards each worker finished in the latest plan call: a drop reported
    # after a restore takes them back exactly as it would have before the save
    d = B.Dds(600, 100, 1, 2)
    d.antdt_shard_plan([3.0, 1.0])
    d.antdt_shard_plan([3.0, 1.0])                 # worker 0 finishes shard 0 here
    e = B.Dds.antdt_dds_load(d.antdt_dds_save(), 2)
    d.antdt_dds_requeue_worker(0)
    e.antdt_dds_requeue_worker(0)
    assert d.antdt_dds_shard_info(0)[:2] == (B.SHARD_TODO, -1)
    assert e.antdt_dds_save() == d.antdt_dds_save()
    with pytest.raises(B.AntdtError):
        B.Dds.antdt_dds_load(img[:-8], 6)
    with pytest.raises(B.AntdtError):
        B.Dds.antdt_dds_load(b"\0" * len(img), 6)


def test_solver_is_millisecond_level_at_1000_workers():
    # Section VII-E: solving for the batch sizes takes milliseconds even with 1000 workers
    rng = np.random.default_rng(4)
    v = np.exp(rng.normal(0, 0.5, size=1000))
    arr = (C.c_double * 1000)(*v)
    out = (C.c_int64 * 1000)()
    for rule in (B.RULE_PROPORTIONAL, B.RULE_MINMAX):
        t0 = time.perf_counter()
        for _ in range(5):
            assert B.lib().antdt_batch_sizes(arr, 1000, 81920, rule, 16, out) == 0
        dt = (time.perf_counter() - t0) / 5
        assert sum(out) == 81920
        assert dt < 0.05, dt
