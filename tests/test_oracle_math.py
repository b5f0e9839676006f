"""Pins of the CPU checker's device-step functions against definitions written another way:
dense count-matrix algebra in numpy float64, closed forms, special cases and the invariants
the aggregation must satisfy (weighted mean of worker means == mean over the global batch)."""
import numpy as np
import pytest

import oracle
from tests.util import bf16_bits_to_f64, count_matrix, f32_to_bf16_bits_trunc_exact, random_bags


def _workers(rng, K, n_samples):
    cuts = np.sort(rng.integers(0, n_samples + 1, size=K - 1))
    return np.concatenate([[0], cuts, [n_samples]]).astype(np.int64)


# ---- forward -----------------------------------------------------------------------------
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_fwd_equals_count_matrix_product(seed):
    rng = np.random.default_rng(seed)
    V, D, n_bags = 50, 8, 40
    W = rng.normal(0, 0.01, size=(V, D)).astype(np.float32)
    ids, off = random_bags(rng, n_bags, V, 6, zipf=1.3 if seed else None)
    got = oracle.embbag_fwd(W, ids, off)
    want = count_matrix(ids, off, V) @ W.astype(np.float64)
    assert np.array_equal(got, want.astype(np.float32)) or np.allclose(got, want, rtol=1e-7, atol=0)
    empty = np.flatnonzero(np.diff(off) == 0)
    assert np.all(got[empty] == 0)


def test_fwd_one_hot_returns_row_exactly_and_repeats_count():
    rng = np.random.default_rng(5)
    V, D = 30, 4
    W = rng.normal(size=(V, D)).astype(np.float32)
    ids = rng.integers(0, V, size=20).astype(np.int32)
    off = np.arange(21, dtype=np.int64)
    assert np.array_equal(oracle.embbag_fwd(W, ids, off), W[ids])
    # one bag holding the same id three times = 3 * row
    got = oracle.embbag_fwd(W, np.array([7, 7, 7], np.int32), np.array([0, 3], np.int64))
    assert np.array_equal(got[0], (3.0 * W[7].astype(np.float64)).astype(np.float32))


def test_fwd_bf16_rows_are_widened_exactly():
    rng = np.random.default_rng(6)
    V, D = 20, 8
    bits = (rng.normal(size=(V, D)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    ids, off = random_bags(rng, 15, V, 5)
    got = oracle.embbag_fwd(bits, ids, off)
    want = count_matrix(ids, off, V) @ bf16_bits_to_f64(bits)
    assert np.allclose(got, want, rtol=1e-7, atol=0)


def test_fwd_rejects_bad_inputs():
    W = np.zeros((4, 4), np.float32)
    with pytest.raises(oracle.OracleError) as e:
        oracle.embbag_fwd(W, np.array([4], np.int32), np.array([0, 1], np.int64))
    assert e.value.code == 2
    with pytest.raises(oracle.OracleError) as e:
        oracle.embbag_fwd(W, np.array([1, 1], np.int32), np.array([0, 2, 1], np.int64))
    assert e.value.code == 9


# ---- backward + dedup ----------------------------------------------------------------------
def _brute_bwd(ids, off, F, dY, V, wso):
    """Per worker: dW = A^T dY / b_w from the dense count matrix; lists from its columns."""
    A = count_matrix(ids, off, V)
    K = len(wso) - 1
    uniq, grads, segs, wuo, occ_sorted = [], [], [0], [0], []
    pos = 0
    bag_of = np.repeat(np.arange(len(off) - 1), np.diff(off))
    for w in range(K):
        b0, b1 = wso[w] * F, wso[w + 1] * F
        Aw = A[b0:b1]
        dW = Aw.T @ dY[b0:b1].astype(np.float64)
        cnt = Aw.sum(0)
        rows = np.flatnonzero(cnt)
        bw = float(wso[w + 1] - wso[w])
        for r in rows:
            uniq.append(r)
            grads.append(dW[r] / bw)
            pos += int(cnt[r])
            segs.append(pos)
        o0, o1 = off[b0], off[b1]
        o = np.arange(o0, o1)
        order = np.lexsort((o, ids[o0:o1]))       # by row id, then original position
        occ_sorted.extend(bag_of[o0:o1][order].tolist())
        wuo.append(len(uniq))
    return (np.array(uniq, np.int32), np.array(grads, np.float64).reshape(len(uniq), -1),
            np.array(segs, np.int64), np.array(wuo, np.int64), np.array(occ_sorted, np.int32))


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_bwd_dedup_equals_transposed_count_matrix(seed):
    rng = np.random.default_rng(10 + seed)
    V, D, F, K, S = 40, 4, 3, 4, 24
    ids, off = random_bags(rng, S * F, V, 5, zipf=1.2 if seed % 2 else None)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    wso = _workers(rng, K, S)
    if seed == 3:
        wso = np.array([0, 0, 10, 10, S], np.int64)   # empty workers
    r = oracle.embbag_bwd_dedup(ids, off, F, dY, V, wso)
    uniq, grads, segs, wuo, occ = _brute_bwd(ids, off, F, dY, V, wso)
    assert np.array_equal(r["uniq_ids"], uniq)
    assert np.array_equal(r["worker_uniq_offsets"], wuo)
    assert np.array_equal(r["seg_offsets"], segs)
    assert np.array_equal(r["sorted_occ"], occ)
    assert np.allclose(r["uniq_grads"], grads, rtol=1e-6, atol=1e-9)


def test_bwd_all_ids_distinct_is_a_scaled_copy():
    rng = np.random.default_rng(20)
    S, F, D, V = 10, 2, 4, 100
    ids = rng.permutation(V)[: S * F].astype(np.int32)
    off = np.arange(S * F + 1, dtype=np.int64)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    wso = np.array([0, 4, S], np.int64)
    r = oracle.embbag_bwd_dedup(ids, off, F, dY, V, wso)
    for w, bw in ((0, 4.0), (1, 6.0)):
        lo, hi = r["worker_uniq_offsets"][w], r["worker_uniq_offsets"][w + 1]
        bags = np.arange(wso[w] * F, wso[w + 1] * F)
        order = np.argsort(ids[bags])
        assert np.array_equal(r["uniq_ids"][lo:hi], ids[bags][order])
        want = (dY[bags][order].astype(np.float64) / bw).astype(np.float32)
        assert np.array_equal(r["uniq_grads"][lo:hi], want)


# ---- gradient accumulation (AntDT-DD, Section VI-B) ------------------------------------------
def test_accumulated_gradient_is_the_mean_over_all_micro_batch_samples():
    # C_w micro-batches of B_w samples each: the mean of the C_w means is the mean over the
    # C_w * B_w samples, which the dense count matrix gives without any notion of micro-batches
    rng = np.random.default_rng(30)
    V, D, F = 30, 4, 3
    micro = np.array([3, 1, 2, 4], np.int64)
    bsz = np.array([4, 7, 5, 2], np.int64)                 # B_w
    wso = np.concatenate([[0], np.cumsum(micro * bsz)]).astype(np.int64)
    S = int(wso[-1])
    ids, off = random_bags(rng, S * F, V, 4, zipf=1.3)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    r = oracle.embbag_bwd_accum(ids, off, F, dY, V, wso, micro)
    uniq, grads, _, wuo, _ = _brute_bwd(ids, off, F, dY, V, wso)
    assert np.array_equal(r["uniq_ids"], uniq) and np.array_equal(r["worker_uniq_offsets"], wuo)
    assert np.allclose(r["uniq_grads"], grads, rtol=1e-6, atol=1e-9)
    # without accumulation it IS the plain backward, value for value
    one = oracle.embbag_bwd_accum(ids, off, F, dY, V, wso, np.ones(4, np.int64))
    plain = oracle.embbag_bwd_dedup(ids, off, F, dY, V, wso)
    assert np.array_equal(one["uniq_ids"], plain["uniq_ids"])
    assert np.array_equal(one["uniq_grads"], plain["uniq_grads"])
    # a micro-batch count that does not divide the worker's samples is refused
    with pytest.raises(oracle.OracleError):
        oracle.embbag_bwd_accum(ids, off, F, dY, V, wso, np.array([5, 1, 2, 4], np.int64))


def test_accumulation_hand_case_with_a_row_missing_from_a_micro_batch():
    # one worker, 2 micro-batches of 2 samples, one bag per sample, dim 1.
    # row 5 occurs in samples 0, 1 and 3 (dY 1, 2, 8), row 9 only in sample 2 (dY 4):
    #   micro-batch means: row 5 -> (1+2)/2 = 1.5 and 8/2 = 4 ; row 9 -> 0 and 4/2 = 2
    #   pushed = mean of the two: row 5 -> 2.75, row 9 -> 1.0
    ids = np.array([5, 5, 9, 5], np.int32)
    off = np.arange(5, dtype=np.int64)
    dY = np.array([[1.0], [2.0], [4.0], [8.0]], np.float32)
    r = oracle.embbag_bwd_accum(ids, off, 1, dY, 10, np.array([0, 4], np.int64), np.array([2], np.int64))
    assert r["uniq_ids"].tolist() == [5, 9] and r["uniq_grads"][:, 0].tolist() == [2.75, 1.0]


# ---- aggregation ---------------------------------------------------------------------------
def test_weighted_aggregate_equals_full_batch_mean_gradient():
    rng = np.random.default_rng(30)
    V, D, F, K, S = 60, 4, 3, 5, 40
    ids, off = random_bags(rng, S * F, V, 4, zipf=1.3)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    wso = np.array([0, 3, 11, 11, 30, S], np.int64)      # unequal batches, one empty worker
    bsz = np.diff(wso)
    r = oracle.embbag_bwd_dedup(ids, off, F, dY, V, wso)
    agg_ids, agg = oracle.aggregate_sparse(r["uniq_ids"], r["worker_uniq_offsets"],
                                           r["uniq_grads"], bsz)
    # forget the workers altogether: mean over the global batch
    A = count_matrix(ids, off, V)
    full = A.T @ dY.astype(np.float64) / float(S)
    rows = np.flatnonzero(A.sum(0))
    assert np.array_equal(agg_ids, rows.astype(np.int32))
    assert np.allclose(agg, full[rows], rtol=2e-6, atol=1e-8)


def test_aggregate_equal_batches_is_plain_mean_and_single_worker_is_identity():
    rng = np.random.default_rng(31)
    D, K = 4, 3
    lists = [np.array([1, 4, 9], np.int32), np.array([4, 5], np.int32), np.array([0, 9], np.int32)]
    uid = np.concatenate(lists)
    wuo = np.array([0, 3, 5, 7], np.int64)
    g = rng.normal(size=(7, D)).astype(np.float32)
    ids, agg = oracle.aggregate_sparse(uid, wuo, g, [8, 8, 8])
    assert ids.tolist() == [0, 1, 4, 5, 9]
    g64 = g.astype(np.float64)
    want = {0: g64[5] / 3, 1: g64[0] / 3, 4: (g64[1] + g64[3]) / 3, 5: g64[4] / 3,
            9: (g64[2] + g64[6]) / 3}
    for k, r in enumerate(ids):
        assert np.allclose(agg[k], want[int(r)], rtol=1e-7, atol=0)
    # unequal weights: 1/8, 3/8, 4/8 (exact in binary)
    ids, agg = oracle.aggregate_sparse(uid, wuo, g, [1, 3, 4])
    assert np.array_equal(agg[2], (0.125 * g64[1] + 0.375 * g64[3]).astype(np.float32))
    # K = 1: identity, bit for bit
    ids, agg = oracle.aggregate_sparse(lists[0], np.array([0, 3], np.int64), g[:3], [5])
    assert np.array_equal(ids, lists[0]) and np.array_equal(agg, g[:3])


def test_dense_aggregate_constants_and_mean():
    bsz = np.array([64, 128, 128, 192], np.int64)
    c = np.array([1.0, -2.0, 0.5, 4.0])
    grads = np.repeat(c[:, None], 8, axis=1).astype(np.float32)
    out = oracle.aggregate_dense(grads, bsz)
    assert np.allclose(out, (bsz * c).sum() / bsz.sum(), rtol=1e-7)
    rng = np.random.default_rng(32)
    g = rng.normal(size=(4, 16)).astype(np.float32)
    assert np.allclose(oracle.aggregate_dense(g, [5, 5, 5, 5]), g.astype(np.float64).mean(0),
                       rtol=1e-6, atol=1e-9)
    assert np.array_equal(oracle.aggregate_dense(g[:1], [3]), g[0])


# ---- optimizers ----------------------------------------------------------------------------
def test_adagrad_closed_form_constant_gradient():
    V, D, T = 6, 4, 7
    lr, eps = 0.01, 1e-8
    W = np.full((V, D), 0.5, np.float32)
    acc = np.zeros((V, D), np.float32)
    g = np.array([[0.25, -0.5, 1.0, 2.0]], np.float32)
    ids = np.array([3], np.int32)
    for t in range(1, T + 1):
        oracle.sparse_opt_update(W, ids, g, "adagrad", lr, eps, 0, 0, t, acc)
    g64 = g[0].astype(np.float64)
    # acc_T = T g^2 ;  W_T = W_0 - lr * sum_t g / (sqrt(t) |g| + eps)
    assert np.allclose(acc[3], T * g64 ** 2, rtol=1e-6)
    want = 0.5 - np.float64(np.float32(lr)) * sum(
        g64 / (np.sqrt(t) * np.abs(g64) + np.float64(np.float32(eps))) for t in range(1, T + 1))
    assert np.allclose(W[3], want, rtol=1e-6)
    mask = np.ones(V, bool)
    mask[3] = False
    assert np.all(W[mask] == 0.5) and np.all(acc[mask] == 0)


def test_adagrad_eps_sits_outside_the_square_root():
    # One step from a zero accumulator with eps as large as |g|: acc = g^2, so the element moves by
    # -lr g / (|g| + eps) = -lr/2 exactly in binary arithmetic.  With eps under the root the move
    # would be -lr g / sqrt(g^2 + eps) = -lr / sqrt(1 + 2^10) ~ -0.0312 lr: a factor of 16 away.
    lr, eps = 0.5, 2.0 ** -10
    g = np.array([[2.0 ** -10, -(2.0 ** -10), 2.0 ** -10, -(2.0 ** -10)]], np.float32)
    W = np.zeros((2, 4), np.float32)
    acc = np.zeros((2, 4), np.float32)
    oracle.sparse_opt_update(W, np.array([1], np.int32), g, "adagrad", lr, eps, 0, 0, 1, acc)
    assert np.array_equal(acc[1], np.full(4, 2.0 ** -20, np.float32))
    assert np.array_equal(W[1], np.array([-0.25, 0.25, -0.25, 0.25], np.float32))
    assert np.all(W[0] == 0) and np.all(acc[0] == 0)
    # second step, same gradient: acc = 2 g^2, move = -lr g / (sqrt(2)|g| + eps) = -lr/(sqrt 2 + 1)
    oracle.sparse_opt_update(W, np.array([1], np.int32), g, "adagrad", lr, eps, 0, 0, 2, acc)
    want = -np.sign(g[0].astype(np.float64)) * (0.25 + 0.5 / (np.sqrt(2.0) + 1.0))
    assert np.allclose(W[1], want, rtol=1e-6)


def test_zero_gradient_row_is_unchanged():
    W = np.full((3, 4), 0.3, np.float32)
    acc = np.full((3, 4), 2.0, np.float32)
    oracle.sparse_opt_update(W, np.array([1], np.int32), np.zeros((1, 4), np.float32), "adagrad",
                             0.01, 1e-8, 0, 0, 1, acc)
    assert np.all(W == np.float32(0.3)) and np.all(acc == 2.0)


def test_adam_first_step_and_constant_gradient_property():
    V, D = 5, 4
    lr, eps, b1, b2 = 1e-3, 1e-8, 0.9, 0.999
    W = np.zeros((V, D), np.float32)
    m = np.zeros((V, D), np.float32)
    v = np.zeros((V, D), np.float32)
    g = np.array([[0.5, -0.25, 3.0, -1e-3], [1.0, 1.0, -1.0, 2.0]], np.float32)
    ids = np.array([0, 4], np.int32)
    g64 = g.astype(np.float64)
    step = -np.float64(np.float32(lr)) * g64 / (np.abs(g64) + np.float64(np.float32(eps)))
    for t in range(1, 6):
        oracle.sparse_opt_update(W, ids, g, "adam", lr, eps, b1, b2, t, m, v)
        # m_hat = g and v_hat = g^2 at every t when g is constant: every step moves the same
        assert np.allclose(W[ids], t * step, rtol=2e-6, atol=1e-10)
    assert np.all(W[1:4] == 0) and np.all(m[1:4] == 0) and np.all(v[1:4] == 0)
    b1d, b2d = np.float64(np.float32(b1)), np.float64(np.float32(b2))
    assert np.allclose(m[ids], (1 - b1d ** 5) * g64, rtol=1e-6)
    assert np.allclose(v[ids], (1 - b2d ** 5) * g64 ** 2, rtol=1e-6)


def test_bf16_store_rounds_to_nearest_even():
    # Adam, step 1, eps = 0, g = -1: the row moves by exactly +lr.  With lr = 2^-8 and bf16
    # rows at 1.0 (ulp 2^-7) the result is an exact tie: 1.0 + 2^-8 -> even neighbour.
    lr = 2.0 ** -8
    start = np.array([[1.0, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -6, 2.0]], np.float32)
    even = np.array([[1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -6, 2.0]], np.float32)
    W = f32_to_bf16_bits_trunc_exact(start)
    m = np.zeros((1, 4), np.float32)
    v = np.zeros((1, 4), np.float32)
    oracle.sparse_opt_update(W, np.array([0], np.int32), -np.ones((1, 4), np.float32), "adam", lr,
                             0.0, 0.9, 0.999, 1, m, v)
    assert np.array_equal(W, f32_to_bf16_bits_trunc_exact(even))
    # a non-tie: +0.75 ulp rounds up, +0.25 ulp rounds down
    for frac, up in ((0.75, True), (0.25, False)):
        W = f32_to_bf16_bits_trunc_exact(np.array([[1.0] * 4], np.float32))
        m[:] = 0
        v[:] = 0
        oracle.sparse_opt_update(W, np.array([0], np.int32), -np.ones((1, 4), np.float32), "adam",
                                 frac * 2.0 ** -7, 0.0, 0.9, 0.999, 1, m, v)
        want = 1.0 + 2.0 ** -7 if up else 1.0
        assert np.all(bf16_bits_to_f64(W) == want)


def test_update_rejects_out_of_range_id():
    W = np.zeros((3, 4), np.float32)
    with pytest.raises(oracle.OracleError):
        oracle.sparse_opt_update(W, np.array([3], np.int32), np.zeros((1, 4), np.float32),
                                 "adagrad", 0.01, 1e-8, 0, 0, 1, np.zeros((3, 4), np.float32))


# ---- row-wise Adagrad and the dense update -------------------------------------------------
def test_rowwise_adagrad_closed_form_constant_gradient():
    V, D, T = 5, 4, 6
    lr, eps = 0.05, 1e-8
    W = np.full((V, D), -0.25, np.float32)
    acc = np.zeros(V, np.float32)
    g = np.array([[0.25, -0.5, 1.0, 2.0]], np.float32)
    ids = np.array([2], np.int32)
    for _ in range(T):
        oracle.sparse_rowwise_adagrad(W, ids, g, lr, eps, acc)
    g64 = g[0].astype(np.float64)
    ms = (g64 ** 2).sum() / D                      # the row's mean square: 5.3125 / 4
    assert ms == 1.328125
    assert np.allclose(acc[2], T * ms, rtol=1e-6)
    want = -0.25 - np.float64(np.float32(lr)) * sum(
        g64 / (np.sqrt(t * ms) + np.float64(np.float32(eps))) for t in range(1, T + 1))
    assert np.allclose(W[2], want, rtol=1e-6)
    mask = np.arange(V) != 2
    assert np.all(W[mask] == np.float32(-0.25)) and np.all(acc[mask] == 0)


def test_rowwise_adagrad_eps_sits_outside_the_square_root():
    # |g_c| = 2^-10 for every element, eps = 2^-10, zero state: the row's mean square is 2^-20, its
    # root 2^-10 = eps, so every element moves by -lr sign(g)/2 exactly.  eps under the root would
    # give -lr sign(g) 2^-10 / sqrt(2^-20 + 2^-10), 16 times smaller.
    lr, eps = 0.5, 2.0 ** -10
    s = np.array([1, -1, -1, 1, 1, 1, -1, 1], np.float64)
    g = (s * 2.0 ** -10).astype(np.float32)[None, :]
    W = np.zeros((3, 8), np.float32)
    acc = np.zeros(3, np.float32)
    oracle.sparse_rowwise_adagrad(W, np.array([2], np.int32), g, lr, eps, acc)
    assert acc[2] == np.float32(2.0 ** -20) and acc[0] == 0 and acc[1] == 0
    assert np.array_equal(W[2], (-0.25 * s).astype(np.float32))
    assert np.all(W[:2] == 0)


def test_rowwise_adagrad_equals_elementwise_when_magnitudes_are_equal():
    # |g_c| = c for every element: the row's mean square is c^2, which is what every element's
    # own accumulator holds, so the two variants move the row identically (closed form of the
    # element-wise rule: acc = t c^2)
    lr, eps, c = 0.01, 1e-8, 0.75
    g = np.array([[c, -c, -c, c, c, -c, c, c]], np.float32)
    W = np.zeros((2, 8), np.float32)
    acc = np.zeros(2, np.float32)
    ids = np.array([1], np.int32)
    for _ in range(3):
        oracle.sparse_rowwise_adagrad(W, ids, g, lr, eps, acc)
    lr64, eps64 = np.float64(np.float32(lr)), np.float64(np.float32(eps))
    want = -lr64 * np.sign(g[0]) * sum(c / (np.sqrt(t) * c + eps64) for t in (1, 2, 3))
    assert np.allclose(W[1], want, rtol=1e-6)
    assert np.isclose(acc[1], 3 * c * c, rtol=1e-6)
    # dim 1: the row IS the element, so the stored state equals the element-wise call's
    W1, W2 = np.full((3, 1), 0.5, np.float32), np.full((3, 1), 0.5, np.float32)
    a1, a2 = np.zeros(3, np.float32), np.zeros((3, 1), np.float32)
    g1 = np.array([[0.3], [-2.0]], np.float32)
    i1 = np.array([0, 2], np.int32)
    for t in (1, 2):
        oracle.sparse_rowwise_adagrad(W1, i1, g1, lr, eps, a1)
        oracle.sparse_opt_update(W2, i1, g1, "adagrad", lr, eps, 0, 0, t, a2)
    assert np.array_equal(W1, W2) and np.array_equal(a1, a2[:, 0])


def test_rowwise_adagrad_zero_gradient_and_bad_id():
    W = np.full((3, 4), 0.3, np.float32)
    acc = np.full(3, 2.0, np.float32)
    oracle.sparse_rowwise_adagrad(W, np.array([1], np.int32), np.zeros((1, 4), np.float32), 0.01,
                                  1e-8, acc)
    assert np.all(W == np.float32(0.3)) and np.all(acc == 2.0)
    with pytest.raises(oracle.OracleError):
        oracle.sparse_rowwise_adagrad(W, np.array([3], np.int32), np.zeros((1, 4), np.float32),
                                      0.01, 1e-8, acc)


def test_dense_update_closed_forms():
    lr, eps, b1, b2 = 1e-2, 1e-8, 0.9, 0.999
    g = np.array([0.5, -0.25, 3.0, -1e-3, 0.0], np.float32)
    g64 = g.astype(np.float64)
    lr64, eps64 = np.float64(np.float32(lr)), np.float64(np.float32(eps))
    # Adagrad, constant gradient: acc_T = T g^2, w_T = w_0 - lr sum_t g / (sqrt(t)|g| + eps)
    w = np.full(5, 1.0, np.float32)
    acc = np.zeros(5, np.float32)
    for t in range(1, 5):
        oracle.dense_opt_update(w, g, "adagrad", lr, eps, 0, 0, t, acc)
    assert np.allclose(acc, 4 * g64 ** 2, rtol=1e-6)
    want = 1.0 - lr64 * sum(g64 / (np.sqrt(t) * np.abs(g64) + eps64) for t in range(1, 5))
    assert np.allclose(w, want, rtol=1e-6)
    assert w[4] == 1.0 and acc[4] == 0.0            # zero gradient: element untouched
    # Adam, constant gradient: every step moves -lr g / (|g| + eps)
    w = np.zeros(5, np.float32)
    m = np.zeros(5, np.float32)
    v = np.zeros(5, np.float32)
    step = -lr64 * g64 / (np.abs(g64) + eps64)
    for t in range(1, 5):
        oracle.dense_opt_update(w, g, "adam", lr, eps, b1, b2, t, m, v)
        assert np.allclose(w, t * step, rtol=2e-6, atol=1e-10)
    b1d, b2d = np.float64(np.float32(b1)), np.float64(np.float32(b2))
    assert np.allclose(m, (1 - b1d ** 4) * g64, rtol=1e-6)
    assert np.allclose(v, (1 - b2d ** 4) * g64 ** 2, rtol=1e-6)


# ---- backup-workers aggregation --------------------------------------------------------------
def test_backup_aggregate_is_the_mean_over_the_surviving_samples():
    rng = np.random.default_rng(40)
    V, D, F, K, S = 60, 4, 3, 5, 40
    ids, off = random_bags(rng, S * F, V, 4, zipf=1.3)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    wso = np.array([0, 3, 11, 20, 30, S], np.int64)
    bsz = np.diff(wso)
    dropped = np.array([0, 1, 0, 0, 1], np.uint8)            # workers 1 and 4 are the slowest
    r = oracle.embbag_bwd_dedup(ids, off, F, dY, V, wso)
    agg_ids, agg = oracle.aggregate_sparse_backup(r["uniq_ids"], r["worker_uniq_offsets"],
                                                  r["uniq_grads"], bsz, dropped)
    # forget workers: mean gradient over the samples of workers 0, 2, 3 only
    keep_bags = np.concatenate([np.arange(wso[w] * F, wso[w + 1] * F) for w in (0, 2, 3)])
    A = count_matrix(ids, off, V)[keep_bags]
    full = A.T @ dY[keep_bags].astype(np.float64) / float(bsz[[0, 2, 3]].sum())
    rows = np.flatnonzero(A.sum(0))
    assert np.array_equal(agg_ids, rows.astype(np.int32))
    assert np.allclose(agg, full[rows], rtol=2e-6, atol=1e-8)
    # nobody dropped: the plain aggregate, bit for bit
    a0, g0 = oracle.aggregate_sparse_backup(r["uniq_ids"], r["worker_uniq_offsets"], r["uniq_grads"],
                                            bsz, np.zeros(K, np.uint8))
    a1, g1 = oracle.aggregate_sparse(r["uniq_ids"], r["worker_uniq_offsets"], r["uniq_grads"], bsz)
    assert np.array_equal(a0, a1) and np.array_equal(g0, g1)
    dense = rng.normal(size=(K, 16)).astype(np.float32)
    d = oracle.aggregate_dense_backup(dense, bsz, dropped)
    w = bsz[[0, 2, 3]] / bsz[[0, 2, 3]].sum()
    assert np.allclose(d, (w[:, None] * dense[[0, 2, 3]].astype(np.float64)).sum(0), rtol=1e-6, atol=1e-9)
