"""GPU parity: every device call of the C-ABI against the CPU checker on the same seeded inputs,
element by element.  Indices, offsets and orders must be bit-exact; fp32 values within
rel 1e-5 / abs 1e-6 per call on identical inputs; bf16 rows within rel 1e-2 after the update."""
import numpy as np
import pytest
import torch

import oracle
from paper_2404_09679_b200 import binding as B
from tests import gpu_util as G
from tests.util import random_bags

pytestmark = pytest.mark.gpu


def _bf16_bits(x):
    t = torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def _wso(rng, K, S, empties=False):
    cuts = np.sort(rng.integers(0, S + 1, size=K - 1))
    w = np.concatenate([[0], cuts, [S]]).astype(np.int64)
    if empties and K >= 3:
        w[1] = w[0]
        w[-2] = w[-1]
    return w


# ---- forward -------------------------------------------------------------------------------
@pytest.mark.parametrize("D,bf16", [(4, False), (8, False), (16, False), (32, False), (64, False),
                                    (128, False), (200, False), (512, False), (8, True), (64, True),
                                    (136, True), (1024, True)])
def test_fwd_matches_checker(D, bf16):
    rng = np.random.default_rng(D + bf16)
    V, n_bags = 5000, 3001                      # several CTAs and a ragged last one
    W = rng.normal(0, 0.01, size=(V, D)).astype(np.float32)
    Wt = _bf16_bits(W) if bf16 else W
    ids, off = random_bags(rng, n_bags, V, 70, zipf=1.2)   # bags longer than a lane group, empties
    got, code = G.gpu_fwd(Wt, ids, off)
    assert code == 0
    want = oracle.embbag_fwd(Wt, ids, off)
    G.close(got, want)
    assert np.all(got[np.diff(off) == 0] == 0)


@pytest.mark.parametrize("D,bf16", [(64, False), (64, True)])
def test_fwd_short_bags_over_several_turns(D, bf16):
    """Short bags (under 8 ids on average) take the kernel whose lane groups stride over the bags
    with a capped grid; 700 k bags of 16-lane rows are more than one turn for every group.  A few
    ids out of range are planted: flagged, and they contribute nothing."""
    rng = np.random.default_rng(7 + bf16)
    V, n_bags = 4000, 700_001
    W = rng.normal(0, 0.01, size=(V, D)).astype(np.float32)
    Wt = _bf16_bits(W) if bf16 else W
    ids, off = random_bags(rng, n_bags, V, 6)                # 0..6 ids per bag, empties included
    got, code = G.gpu_fwd(Wt, ids, off)
    assert code == 0
    want = oracle.embbag_fwd(Wt, ids, off)
    G.close(got, want)
    assert np.all(got[np.diff(off) == 0] == 0)
    bad = ids.copy()
    where = rng.choice(len(ids), size=50, replace=False)
    bad[where] = V + 3
    got2, code = G.gpu_fwd(Wt, bad, off)
    assert code == B.ERR_ID_OUT_OF_RANGE
    keep = np.ones(len(ids), bool)
    keep[where] = False
    off2 = np.concatenate([[0], np.cumsum(np.add.reduceat(keep, off[:-1].clip(max=len(ids) - 1)) *
                                          (np.diff(off) > 0))]).astype(np.int64)
    G.close(got2, oracle.embbag_fwd(Wt, ids[keep], off2))


def test_fwd_one_hot_is_bit_exact_and_empty_input_is_fine():
    rng = np.random.default_rng(1)
    V, D, n = 1000, 32, 777
    W = rng.normal(size=(V, D)).astype(np.float32)
    ids = rng.integers(0, V, size=n).astype(np.int32)
    got, code = G.gpu_fwd(W, ids, np.arange(n + 1, dtype=np.int64))
    assert code == 0 and np.array_equal(got, W[ids])
    got, code = G.gpu_fwd(W, np.zeros(0, np.int32), np.zeros(4, np.int64))
    assert code == 0 and got.shape == (3, D) and np.all(got == 0)
    got, code = G.gpu_fwd(W, np.zeros(0, np.int32), np.zeros(1, np.int64))
    assert code == 0 and got.shape == (0, D)


def test_fwd_flags_and_skips_bad_ids_and_offsets():
    V, D = 10, 8
    W = np.ones((V, D), np.float32)
    ids = np.array([1, 10, 2, -1, 3], np.int32)
    off = np.array([0, 2, 4, 5], np.int64)
    got, code = G.gpu_fwd(W, ids, off)
    assert code == B.ERR_ID_OUT_OF_RANGE
    assert np.array_equal(got[:, 0], [1.0, 1.0, 1.0])       # the bad ids contributed nothing
    off = np.array([0, 4, 2, 5], np.int64)                   # descending
    got, code = G.gpu_fwd(W, ids % V, off)
    assert code == B.ERR_BAD_OFFSETS and np.all(got[1] == 0)
    off = np.array([0, 2, 4, 9], np.int64)                   # runs past nnz
    got, code = G.gpu_fwd(W, ids % V, off)
    assert code == B.ERR_BAD_OFFSETS and np.all(got[2] == 0)


# ---- backward + dedup ------------------------------------------------------------------------
def _check_bwd(ids, off, F, dY, V, wso):
    got = G.gpu_bwd(ids, off, F, dY, V, wso)
    assert got["status"] == 0
    want = oracle.embbag_bwd_dedup(ids, off, F, dY, V, wso)
    assert np.array_equal(got["worker_uniq_offsets"], want["worker_uniq_offsets"])
    assert np.array_equal(got["uniq_ids"], want["uniq_ids"])
    assert np.array_equal(got["seg_offsets"], want["seg_offsets"])
    assert np.array_equal(got["sorted_occ"], want["sorted_occ"])
    G.close(got["uniq_grads"], want["uniq_grads"])
    return got, want


@pytest.mark.parametrize("V,D,K,F,S,maxlen,zipf", [
    (50, 16, 4, 3, 400, 6, 1.2),          # tiny vocabulary: runs of hundreds, many tiles each
    (1, 4, 2, 1, 300, 3, None),           # a single row: one run per worker
    (100_000, 64, 16, 7, 2000, 12, 1.1),  # 17-bit keys: two passes
    ((1 << 20) + 3, 32, 5, 4, 1500, 9, None),  # 21-bit keys: three passes, mostly distinct ids
    (3000, 8, 32, 2, 999, 5, 1.05),       # many workers, ragged everything
    (777, 128, 3, 2, 500, 4, 1.3),        # 32 lanes per row
    (777, 200, 3, 2, 300, 4, 1.3),        # rows wider than a warp's vector
])
def test_bwd_dedup_matches_checker(V, D, K, F, S, maxlen, zipf):
    rng = np.random.default_rng(V % 1000 + D + K)
    ids, off = random_bags(rng, S * F, V, maxlen, zipf=zipf)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    _check_bwd(ids, off, F, dY, V, _wso(rng, K, S, empties=(K >= 3)))


def test_bwd_dedup_large_multi_chunk_with_hot_rows():
    # > 592 chunks * 4096 so that chunks hold several tiles; Zipf head gives runs of ~1e5
    rng = np.random.default_rng(11)
    V, D, K, F, S = 200_000, 16, 6, 10, 30_000
    ids, off = random_bags(rng, S * F, V, 19, allow_empty=False, zipf=1.15)
    assert ids.shape[0] > 2_600_000
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    got, want = _check_bwd(ids, off, F, dY, V, _wso(rng, K, S))
    assert np.diff(want["seg_offsets"]).max() > 20_000


def test_bwd_with_the_minimum_workspace_walks_long_tiles():
    """Up to 2^20 occurrences the recommended workspace buys 16-entry reduction tiles; with the
    minimum workspace the same call walks 64-entry tiles.  Integer outputs identical, sums within
    tolerance of the checker either way; one byte less than the minimum is refused."""
    rng = np.random.default_rng(77)
    V, D, K, F, S = 20_000, 32, 5, 6, 9000
    ids, off = random_bags(rng, S * F, V, 9, zipf=1.2)        # ~270k occurrences, long hot runs
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    wso = _wso(rng, K, S)
    nnz = len(ids)
    rec = B.antdt_embbag_bwd_dedup_workspace_bytes(nnz, S * F, D, K)
    least = B.antdt_embbag_bwd_dedup_min_workspace_bytes(nnz, S * F, D, K)
    assert least < rec
    big = B.antdt_embbag_bwd_dedup_workspace_bytes(3 << 20, 1000, D, K)
    assert big == B.antdt_embbag_bwd_dedup_min_workspace_bytes(3 << 20, 1000, D, K)
    a = G.gpu_bwd(ids, off, F, dY, V, wso)
    b = G.gpu_bwd(ids, off, F, dY, V, wso, min_workspace=True)
    want = oracle.embbag_bwd_dedup(ids, off, F, dY, V, wso)
    for got in (a, b):
        assert got["status"] == 0
        for k in ("worker_uniq_offsets", "uniq_ids", "seg_offsets", "sorted_occ"):
            assert np.array_equal(got[k], want[k]), k
        G.close(got["uniq_grads"], want["uniq_grads"])
    # below the minimum: refused before any launch
    cap = max(1, nnz)
    t = lambda *shape, dt=torch.int32: torch.zeros(*shape, dtype=dt, device="cuda")
    with pytest.raises(B.AntdtError) as ei:
        B.antdt_embbag_bwd_dedup(G.dev(ids), G.dev(off), F, G.dev(dY), V, [int(x) for x in wso], t(cap),
                                 t(K + 1, dt=torch.int64), t(cap + 1, dt=torch.int64), t(nnz),
                                 t(cap, D, dt=torch.float32), t(least - 256, dt=torch.uint8), G.new_status())
    assert ei.value.code == B.ERR_WORKSPACE_TOO_SMALL


def test_bwd_is_bit_reproducible():
    rng = np.random.default_rng(12)
    V, D, K, F, S = 500, 32, 4, 5, 3000
    ids, off = random_bags(rng, S * F, V, 8, zipf=1.2)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    wso = _wso(rng, K, S)
    a = G.gpu_bwd(ids, off, F, dY, V, wso)
    b = G.gpu_bwd(ids, off, F, dY, V, wso)
    for k in ("uniq_ids", "seg_offsets", "sorted_occ", "worker_uniq_offsets"):
        assert np.array_equal(a[k], b[k])
    assert np.array_equal(a["uniq_grads"].view(np.uint32), b["uniq_grads"].view(np.uint32))


def test_bwd_empty_and_degenerate_inputs():
    D, F = 8, 2
    # no occurrences at all
    got = G.gpu_bwd(np.zeros(0, np.int32), np.zeros(2 * F * 3 + 1, np.int64), F,
                    np.zeros((2 * F * 3, D), np.float32), 10, np.array([0, 2, 6], np.int64))
    assert got["status"] == 0 and got["worker_uniq_offsets"].tolist() == [0, 0, 0]
    assert got["seg_offsets"].tolist() == [0]
    # all ids distinct: a scaled copy
    rng = np.random.default_rng(13)
    S = 40
    ids = rng.permutation(1000)[: S * F].astype(np.int32)
    off = np.arange(S * F + 1, dtype=np.int64)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    _check_bwd(ids, off, F, dY, 1000, np.array([0, 10, S], np.int64))


def test_bwd_flags_bad_ids_and_capacity():
    rng = np.random.default_rng(14)
    V, D, F, S = 100, 8, 2, 50
    ids, off = random_bags(rng, S * F, V, 4, allow_empty=False)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    wso = np.array([0, 20, S], np.int64)
    bad = ids.copy()
    bad[7] = V + 5
    assert G.gpu_bwd(bad, off, F, dY, V, wso)["status"] == B.ERR_ID_OUT_OF_RANGE
    want = oracle.embbag_bwd_dedup(ids, off, F, dY, V, wso)
    nu = int(want["worker_uniq_offsets"][-1])
    got = G.gpu_bwd(ids, off, F, dY, V, wso, out_cap=nu - 3)
    assert got["status"] == B.ERR_CAPACITY
    assert int(got["worker_uniq_offsets"][-1]) == nu          # the count is still reported
    assert np.array_equal(got["uniq_ids"], want["uniq_ids"][: nu - 3])   # nothing past the cap
    off_bad = off.copy()
    off_bad[5] = off_bad[6] + 1
    assert G.gpu_bwd(ids, off_bad, F, dY, V, wso)["status"] == B.ERR_BAD_OFFSETS
    # occurrences without a single bag to belong to: refused on the host, nothing is launched
    with pytest.raises(B.AntdtError) as ei:
        G.gpu_bwd(ids[:5], np.zeros(1, np.int64), F, np.zeros((1, D), np.float32), V,
                  np.array([0, 0], np.int64))
    assert ei.value.code == B.ERR_INVALID_ARG


# ---- aggregation ---------------------------------------------------------------------------
@pytest.mark.parametrize("V,D,K,n_per", [(500, 16, 4, 300), (100_000, 64, 16, 5000),
                                         (2_000_000, 32, 32, 3000), (64, 8, 1, 40),
                                         (5000, 200, 5, 1000)])
def test_sparse_aggregate_matches_checker(V, D, K, n_per):
    rng = np.random.default_rng(V % 997 + K)
    lists = [np.sort(rng.choice(V, size=min(V, int(rng.integers(0, n_per + 1))), replace=False))
             for _ in range(K)]
    if K >= 3:
        lists[1] = lists[1][:0]
    uid = np.concatenate(lists).astype(np.int32)
    wuo = np.concatenate([[0], np.cumsum([len(l) for l in lists])]).astype(np.int64)
    g = rng.normal(size=(len(uid), D)).astype(np.float32)
    bsz = rng.integers(1, 5000, size=K)
    ids, agg, na, _, code = G.gpu_aggregate(uid, wuo, g, bsz, V)
    assert code == 0
    want_ids, want = oracle.aggregate_sparse(uid, wuo, g, bsz)
    assert na == len(want_ids) and np.array_equal(ids, want_ids)
    G.close(agg, want)


def _lists_case(rng, K, make):
    lists = [np.unique(make(i)).astype(np.int64) for i in range(K)]
    uid = np.concatenate(lists).astype(np.int32)
    wuo = np.concatenate([[0], np.cumsum([len(l) for l in lists])]).astype(np.int64)
    return uid, wuo


def test_sparse_aggregate_clustered_and_dense_ranges():
    """Row ids that are NOT spread by a hash: every worker holds the same dense block (every
    4096-id range of it carries K entries per id), plus a thin tail; 32 workers fill every bit of
    the worker-set words; dim 4 puts one lane on a row."""
    rng = np.random.default_rng(61)
    for K, D, dense_to, V in [(32, 4, 20_000, 3_000_000), (8, 32, 70_000, 200_000), (17, 16, 9000, 9001)]:
        def make(i):
            tail = rng.integers(dense_to, V, size=500) if V > dense_to else np.zeros(0, np.int64)
            keep = rng.random(dense_to) < (1.0 if i % 3 == 0 else 0.8)
            return np.concatenate([np.nonzero(keep)[0], tail])
        uid, wuo = _lists_case(rng, K, make)
        g = rng.normal(size=(len(uid), D)).astype(np.float32)
        bsz = rng.integers(1, 4000, size=K)
        ids, agg, na, _, code = G.gpu_aggregate(uid, wuo, g, bsz, V)
        assert code == 0
        want_ids, want = oracle.aggregate_sparse(uid, wuo, g, bsz)
        assert na == len(want_ids) and np.array_equal(ids, want_ids)
        G.close(agg, want)


def test_sparse_aggregate_table_beyond_2_to_30_rows():
    """n_rows above 2^30 switches the merge to 8192-id ranges (the row count is only a bound here:
    no table is touched).  Ids sit at both ends of the id space and around a range boundary."""
    rng = np.random.default_rng(62)
    V = (1 << 31) - 1
    K, D = 6, 16
    edge = np.array([0, 1, 8191, 8192, 8193, V - 8193, V - 2, V - 1], np.int64)

    def make(i):
        return np.concatenate([edge[rng.random(len(edge)) < 0.7], rng.integers(0, V, size=20_000),
                               rng.integers(1 << 30, (1 << 30) + 50_000, size=10_000)])
    uid, wuo = _lists_case(rng, K, make)
    g = rng.normal(size=(len(uid), D)).astype(np.float32)
    bsz = rng.integers(1, 4000, size=K)
    ids, agg, na, _, code = G.gpu_aggregate(uid, wuo, g, bsz, V)
    assert code == 0
    want_ids, want = oracle.aggregate_sparse(uid, wuo, g, bsz)
    assert na == len(want_ids) and np.array_equal(ids, want_ids)
    G.close(agg, want)


def test_sparse_aggregate_flags_ids_outside_the_table():
    """An id >= n_rows is not part of the union: flagged, skipped, and every access stays inside
    the buffers (whatever else the flagged call returns is unspecified)."""
    rng = np.random.default_rng(63)
    V, K, D = 50_000, 4, 8
    uid, wuo = _lists_case(rng, K, lambda i: rng.integers(0, V, size=3000))
    g = rng.normal(size=(len(uid), D)).astype(np.float32)
    bad = uid.copy()
    bad[wuo[2] - 1] = V + 5            # last (largest) id of worker 1's list: still ascending
    _, _, _, _, code = G.gpu_aggregate(bad, wuo, g, [1] * K, V)
    assert code == B.ERR_ID_OUT_OF_RANGE
    bad[wuo[2] - 1] = 60_000_000       # far past the last range of the table
    _, _, _, _, code = G.gpu_aggregate(bad, wuo, g, [1] * K, V)
    assert code == B.ERR_ID_OUT_OF_RANGE
    ids, agg, na, _, code = G.gpu_aggregate(uid, wuo, g, [1] * K, V)   # the clean lists still work
    want_ids, want = oracle.aggregate_sparse(uid, wuo, g, [1] * K)
    assert code == 0 and np.array_equal(ids, want_ids)
    G.close(agg, want)


def test_sparse_aggregate_flags_a_list_that_repeats_ids():
    """A worker list must ascend strictly.  One that repeats an id 9000 times puts more entries
    into a 4096-id stretch than 2 workers can legitimately list there: flagged (only the status
    word is specified), every access stays inside the buffers."""
    D = 4
    uid = np.concatenate([np.full(9000, 7, np.int32), np.array([3, 9], np.int32)])
    wuo = np.array([0, 9000, 9002], np.int64)
    g = np.ones((len(uid), D), np.float32)
    _, _, _, _, code = G.gpu_aggregate(uid, wuo, g, [1, 1], 50_000)
    assert code == B.ERR_BAD_OFFSETS


def test_aggregate_invariants_on_gpu():
    rng = np.random.default_rng(21)
    V, D, F, K, S = 300, 16, 3, 4, 512
    ids, off = random_bags(rng, S * F, V, 4, zipf=1.2)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    wso = np.array([0, 64, 192, 320, 512], np.int64)     # 64/128/128/192
    bsz = np.diff(wso)
    b = G.gpu_bwd(ids, off, F, dY, V, wso)
    aid, agg, na, _, code = G.gpu_aggregate(b["uniq_ids"], b["worker_uniq_offsets"], b["uniq_grads"],
                                            bsz, V)
    assert code == 0
    # weighted aggregate of worker means == mean over the global batch (one worker holding all)
    whole = oracle.embbag_bwd_dedup(ids, off, F, dY, V, np.array([0, S], np.int64))
    assert np.array_equal(aid, whole["uniq_ids"])
    G.close(agg, whole["uniq_grads"], rtol=2e-5)
    # K = 1 is the identity, bit for bit
    w1 = G.gpu_bwd(ids, off, F, dY, V, np.array([0, S], np.int64))
    aid1, agg1, _, _, _ = G.gpu_aggregate(w1["uniq_ids"], w1["worker_uniq_offsets"], w1["uniq_grads"],
                                          [S], V)
    assert np.array_equal(aid1, w1["uniq_ids"]) and np.array_equal(agg1, w1["uniq_grads"])


def test_dense_aggregate_matches_checker_and_capacity_is_flagged():
    rng = np.random.default_rng(22)
    for K, n in [(4, 4096), (16, 100_000), (33, 1_000_004), (1, 8)]:
        g = (1e-2 * rng.normal(size=(K, n))).astype(np.float32)
        bsz = rng.integers(1, 9000, size=K)
        uid = np.array([3], np.int32)
        wuo = np.array([0] + [1] * K, np.int64)
        _, _, _, dout, code = G.gpu_aggregate(uid, wuo, np.ones((1, 4), np.float32), bsz, 10, dense=g)
        assert code == 0
        G.close(dout, oracle.aggregate_dense(g, bsz))
    # equal batches: plain mean
    g = rng.normal(size=(4, 64)).astype(np.float32)
    _, _, _, dout, _ = G.gpu_aggregate(np.array([3], np.int32), np.array([0, 1, 1, 1, 1], np.int64),
                                       np.ones((1, 4), np.float32), [7, 7, 7, 7], 10, dense=g)
    G.close(dout, g.astype(np.float64).mean(0))
    uid = np.array([1, 2, 3, 2, 5], np.int32)
    wuo = np.array([0, 3, 5], np.int64)
    aid, agg, na, _, code = G.gpu_aggregate(uid, wuo, np.ones((5, 4), np.float32), [1, 1], 10, out_cap=2)
    assert code == B.ERR_CAPACITY and na == 4 and aid.tolist() == [1, 2]


# ---- optimizers ------------------------------------------------------------------------------
@pytest.mark.parametrize("opt", ["adagrad", "adam"])
@pytest.mark.parametrize("D,bf16", [(16, False), (64, False), (200, False), (64, True), (8, True)])
def test_update_matches_checker(opt, D, bf16):
    rng = np.random.default_rng(D + (opt == "adam"))
    V, n = 4000, 1500
    W = rng.normal(0, 0.01, size=(V, D)).astype(np.float32)
    Wt = _bf16_bits(W) if bf16 else W
    s0 = np.abs(rng.normal(0, 0.1, size=(V, D))).astype(np.float32)
    s1 = np.abs(rng.normal(0, 0.01, size=(V, D))).astype(np.float32) if opt == "adam" else None
    ids = np.sort(rng.choice(V, size=n, replace=False)).astype(np.int32)
    g = rng.normal(0, 0.05, size=(n, D)).astype(np.float32)
    lr, eps, b1, b2, step = (0.01, 1e-8, 0.0, 0.0, 3) if opt == "adagrad" else (1e-3, 1e-8, 0.9, 0.999, 7)
    gw, g0, g1, code = G.gpu_update(Wt, ids, g, opt, lr, eps, b1, b2, step, s0, s1)
    assert code == 0
    w_ref, r0 = Wt.copy(), s0.copy()
    r1 = None if s1 is None else s1.copy()
    oracle.sparse_opt_update(w_ref, ids, g, opt, lr, eps, b1, b2, step, r0, r1)
    G.close(g0, r0)
    if r1 is not None:
        G.close(g1, r1)
    if bf16:
        a = (gw.astype(np.uint32) << 16).view(np.float32)
        b = (w_ref.astype(np.uint32) << 16).view(np.float32)
        G.close(a, b, rtol=G.BF16_RTOL, atol=1e-6)
        # RNE on both sides: almost every element identical, the rest one bf16 ulp apart
        assert (gw != w_ref).mean() < 0.02
    else:
        G.close(gw, w_ref)
    untouched = np.ones(V, bool)
    untouched[ids] = False
    assert np.array_equal(gw[untouched], Wt[untouched]) and np.array_equal(g0[untouched], s0[untouched])


def test_update_textbook_cases_and_flags():
    # Adam, first step from zero state: every element moves by -lr * g / (|g| + eps)
    V, D = 50, 8
    rng = np.random.default_rng(31)
    W = rng.normal(size=(V, D)).astype(np.float32)
    ids = np.arange(0, V, 3, dtype=np.int32)
    g = rng.normal(size=(len(ids), D)).astype(np.float32)
    z = np.zeros((V, D), np.float32)
    gw, m, v, code = G.gpu_update(W, ids, g, "adam", 1e-3, 1e-8, 0.9, 0.999, 1, z, z.copy())
    g64 = g.astype(np.float64)
    G.close(gw[ids], W[ids] - np.float32(1e-3) * g64 / (np.abs(g64) + 1e-8))
    # bf16 exact ties round to even (lr = 2^-8, eps = 0, g = -1 -> +lr exactly)
    start = np.array([[1.0, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -6, 2.0] * 2], np.float32)
    even = np.array([[1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -6, 2.0] * 2], np.float32)
    z = np.zeros((1, 8), np.float32)
    gw, _, _, _ = G.gpu_update(_bf16_bits(start), np.array([0], np.int32), -np.ones((1, 8), np.float32),
                               "adam", 2.0 ** -8, 0.0, 0.9, 0.999, 1, z, z.copy())
    assert np.array_equal(gw, _bf16_bits(even))
    # out-of-range id: flagged, skipped, the rest still updated
    W = np.ones((4, 8), np.float32)
    ids = np.array([1, 9, 2], np.int32)
    gw, acc, _, code = G.gpu_update(W, ids, np.ones((3, 8), np.float32), "adagrad", 0.5, 0.0, 0, 0, 1,
                                    np.zeros((4, 8), np.float32))
    assert code == B.ERR_ID_OUT_OF_RANGE
    assert np.all(gw[[0, 3]] == 1.0) and np.all(gw[[1, 2]] == 0.5) and np.all(acc[[1, 2]] == 1.0)


@pytest.mark.parametrize("D,bf16", [(4, False), (16, False), (64, False), (200, False), (64, True), (8, True)])
def test_rowwise_adagrad_matches_checker(D, bf16):
    rng = np.random.default_rng(100 + D)
    V, n = 3000, 1100
    W = rng.normal(0, 0.01, size=(V, D)).astype(np.float32)
    Wt = _bf16_bits(W) if bf16 else W
    acc = np.abs(rng.normal(0, 0.1, size=V)).astype(np.float32)
    ids = np.sort(rng.choice(V, size=n, replace=False)).astype(np.int32)
    g = rng.normal(0, 0.05, size=(n, D)).astype(np.float32)
    gw, g0, _, code = G.gpu_update(Wt, ids, g, "rowwise_adagrad", 0.01, 1e-8, 0.0, 0.0, 2, acc)
    assert code == 0
    w_ref, r0 = Wt.copy(), acc.copy()
    oracle.sparse_rowwise_adagrad(w_ref, ids, g, 0.01, 1e-8, r0)
    G.close(g0, r0)
    if bf16:
        a = (gw.astype(np.uint32) << 16).view(np.float32)
        b = (w_ref.astype(np.uint32) << 16).view(np.float32)
        G.close(a, b, rtol=G.BF16_RTOL, atol=1e-6)
        assert (gw != w_ref).mean() < 0.02
    else:
        G.close(gw, w_ref)
    untouched = np.ones(V, bool)
    untouched[ids] = False
    assert np.array_equal(gw[untouched], Wt[untouched]) and np.array_equal(g0[untouched], acc[untouched])
    # out-of-range id: flagged and skipped, the other rows still updated
    W1 = np.ones((4, 8), np.float32)
    gw, a1, _, code = G.gpu_update(W1, np.array([1, 9, 2], np.int32), np.ones((3, 8), np.float32),
                                   "rowwise_adagrad", 0.5, 0.0, 0, 0, 1, np.zeros(4, np.float32))
    assert code == B.ERR_ID_OUT_OF_RANGE
    assert np.all(gw[[0, 3]] == 1.0) and np.all(gw[[1, 2]] == 0.5) and a1.tolist() == [0, 1, 1, 0]


@pytest.mark.parametrize("opt", ["adagrad", "adam"])
@pytest.mark.parametrize("n", [4, 1000, 1 << 20, (1 << 22) + 12])
def test_dense_update_matches_checker(opt, n):
    rng = np.random.default_rng(n % 1000 + (opt == "adam"))
    w = rng.normal(0, 0.1, size=n).astype(np.float32)
    g = rng.normal(0, 0.01, size=n).astype(np.float32)
    s0 = np.abs(rng.normal(0, 0.1, size=n)).astype(np.float32)
    s1 = np.abs(rng.normal(0, 0.01, size=n)).astype(np.float32) if opt == "adam" else None
    lr, eps, b1, b2, step = (0.01, 1e-8, 0.0, 0.0, 3) if opt == "adagrad" else (1e-3, 1e-8, 0.9, 0.999, 5)
    dw, dg, d0 = G.dev(w), G.dev(g), G.dev(s0)
    d1 = None if s1 is None else G.dev(s1)
    B.antdt_dense_opt_update(dw, dg, B.OPTS[opt], lr, eps, b1, b2, step, d0, d1)
    torch.cuda.synchronize()
    oracle.dense_opt_update(w, g, opt, lr, eps, b1, b2, step, s0, s1)
    G.close(dw.cpu().numpy(), w)
    G.close(d0.cpu().numpy(), s0)
    if s1 is not None:
        G.close(d1.cpu().numpy(), s1)


def test_dense_update_argument_errors_and_empty():
    z = torch.zeros(8, device="cuda")
    B.antdt_dense_opt_update(z[:0], z[:0], B.OPT_ADAGRAD, 0.1, 1e-8, 0, 0, 1, z[:0])   # n = 0: nothing
    for bad in (lambda: B.antdt_dense_opt_update(z[:6], z[:6], B.OPT_ADAGRAD, 0.1, 1e-8, 0, 0, 1, z[:6]),
                lambda: B.antdt_dense_opt_update(z, z.clone(), B.OPT_ADAM, 0.1, 1e-8, .9, .99, 1, z.clone()),
                lambda: B.antdt_dense_opt_update(z, z.clone(), B.OPT_ROWWISE_ADAGRAD, 0.1, 1e-8, 0, 0, 1, z.clone()),
                lambda: B.antdt_dense_opt_update(z, z.clone(), B.OPT_ADAGRAD, 0.1, 1e-8, 0, 0, 0, z.clone())):
        with pytest.raises(B.AntdtError) as ei:
            bad()
        assert ei.value.code == B.ERR_INVALID_ARG


# ---- limits of the worker count, and the parts of the aggregate on their own ------------------
def test_a_thousand_workers():
    rng = np.random.default_rng(41)
    V, D, K, F, S = 5000, 16, 1000, 2, 3000
    ids, off = random_bags(rng, S * F, V, 6, zipf=1.2)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    wso = _wso(rng, K, S, empties=True)
    got, want = _check_bwd(ids, off, F, dY, V, wso)
    bsz = np.maximum(np.diff(wso), 0)
    aid, agg, na, _, code = G.gpu_aggregate(got["uniq_ids"], got["worker_uniq_offsets"],
                                            got["uniq_grads"], bsz, V)
    assert code == 0
    want_ids, want_agg = oracle.aggregate_sparse(want["uniq_ids"], want["worker_uniq_offsets"],
                                                 want["uniq_grads"], bsz)
    assert np.array_equal(aid, want_ids)
    G.close(agg, want_agg, rtol=3e-5, atol=2e-6)


def test_dense_part_alone_and_sparse_part_alone():
    rng = np.random.default_rng(42)
    K, n = 6, 40_000
    g = rng.normal(size=(K, n)).astype(np.float32)
    bsz = rng.integers(1, 100, size=K)
    dg, out = G.dev(g), torch.full((n,), float("nan"), device="cuda")
    ws = torch.empty(B.antdt_weighted_aggregate_workspace_bytes(0, 0, K), dtype=torch.uint8, device="cuda")
    st = G.new_status()
    B.antdt_weighted_aggregate([int(b) for b in bsz], ws, dense_grads=dg, dense_out=out, dev_status=st)
    assert B.antdt_read_status(st) == 0
    G.close(out.cpu().numpy(), oracle.aggregate_dense(g, bsz))
    # a strided view: worker vectors 2n apart
    wide = torch.zeros(K, 2 * n, device="cuda")
    wide[:, :n] = dg
    out.fill_(float("nan"))
    B.antdt_weighted_aggregate([int(b) for b in bsz], ws, dense_grads=wide[:, :n], dense_out=out,
                               dev_status=st)
    G.close(out.cpu().numpy(), oracle.aggregate_dense(g, bsz))


def test_backup_workers_aggregate_matches_checker():
    rng = np.random.default_rng(43)
    for V, D, K, n_per in [(500, 16, 6, 300), (200_000, 64, 16, 20_000), (3000, 32, 33, 500)]:
        lists = [np.sort(rng.choice(V, size=int(rng.integers(1, n_per + 1)), replace=False))
                 for _ in range(K)]
        uid = np.concatenate(lists).astype(np.int32)
        wuo = np.concatenate([[0], np.cumsum([len(l) for l in lists])]).astype(np.int64)
        g = rng.normal(size=(len(uid), D)).astype(np.float32)
        bsz = rng.integers(1, 5000, size=K)
        dropped = (rng.random(K) < 0.3).astype(np.uint8)
        dropped[0], dropped[1] = 1, 0
        dense = (1e-2 * rng.normal(size=(K, 4096))).astype(np.float32)
        dense[0] = np.nan                                # a dropped worker's vector is never read
        cap = len(uid)
        agg_ids = torch.full((cap,), -1, dtype=torch.int32, device="cuda")
        agg = torch.full((cap, D), float("nan"), device="cuda")
        n_agg = torch.zeros(1, dtype=torch.int64, device="cuda")
        dout = torch.full((4096,), float("nan"), device="cuda")
        ws = torch.empty(B.antdt_weighted_aggregate_workspace_bytes(cap, D, K), dtype=torch.uint8,
                         device="cuda")
        st = G.new_status()
        B.antdt_weighted_aggregate([int(b) for b in bsz], ws, n_rows=V, uniq_ids=G.dev(uid),
                                   worker_uniq_offsets=G.dev(wuo), uniq_grads=G.dev(g),
                                   agg_ids=agg_ids, agg_grads=agg, n_agg=n_agg,
                                   dense_grads=G.dev(dense), dense_out=dout, dev_status=st,
                                   dropped=dropped.tolist())
        assert B.antdt_read_status(st) == 0
        want_ids, want = oracle.aggregate_sparse_backup(uid, wuo, g, bsz, dropped)
        na = int(n_agg.item())
        assert na == len(want_ids) and np.array_equal(agg_ids[:na].cpu().numpy(), want_ids)
        G.close(agg[:na].cpu().numpy(), want)
        dense[0] = 0
        G.close(dout.cpu().numpy(), oracle.aggregate_dense_backup(dense, bsz, dropped))


def test_bwd_extreme_row_ids_and_widest_rows():
    # row ids up to 2^31 - 2: 31-bit keys, four radix passes (nothing here touches a table)
    rng = np.random.default_rng(44)
    V, D, K, F, S = (1 << 31) - 1, 8, 3, 2, 4000
    ids = rng.integers(V - 5000, V, size=S * F * 2).astype(np.int32)
    ids[::7] = rng.integers(0, 50, size=len(ids[::7]))           # and some at the low end
    off = np.arange(0, S * F * 2 + 1, 2, dtype=np.int64)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    _check_bwd(ids, off, F, dY, V, _wso(rng, K, S))
    # dim 1024: eight vectors per lane
    V, D, S = 300, 1024, 200
    ids, off = random_bags(rng, S * F, V, 3, zipf=1.2)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    got, want = _check_bwd(ids, off, F, dY, V, _wso(rng, K, S))
    bsz = np.maximum(np.diff(_wso(rng, K, S)), 1)
    aid, agg, na, _, code = G.gpu_aggregate(got["uniq_ids"], got["worker_uniq_offsets"],
                                            got["uniq_grads"], bsz, V)
    wid, wagg = oracle.aggregate_sparse(want["uniq_ids"], want["worker_uniq_offsets"],
                                        want["uniq_grads"], bsz)
    assert code == 0 and np.array_equal(aid, wid)
    G.close(agg, wagg, rtol=3e-5, atol=2e-6)


def test_probe_gather_sums_the_rows_it_is_given():
    rng = np.random.default_rng(91)
    for D, per_out in ((16, 3), (32, 8), (64, 20), (128, 9)):
        rows = rng.normal(size=(500, D)).astype(np.float32)
        idx = rng.integers(0, 500, size=77 * per_out).astype(np.int32)
        out = torch.full((77, D), float("nan"), device="cuda")
        B.antdt_probe_gather(G.dev(rows), G.dev(idx), per_out, out)
        want = rows.astype(np.float64)[idx.reshape(77, per_out)].sum(1)
        G.close(out.cpu().numpy(), want)
