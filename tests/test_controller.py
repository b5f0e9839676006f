"""AntDT-ND controller front end (Section VI-A steps 2-5): the checker pinned by hand-computed
cases and the paper's straggler pattern, then the library against the checker."""
import numpy as np
import pytest

import oracle
from paper_2404_09679_b200 import binding as B
from paper_2404_09679_b200 import build as libbuild


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()


def test_checker_hand_case():
    # 4 workers, batch 100 each; worker 3 takes 2 s, the others 1 s: mean BPT 1.25, lambda 1.5
    rep = [(w, 100, 2.0 if w == 3 else 1.0) for _ in range(3) for w in range(4)]
    v, t, p, a = oracle.ctl_decide(rep, 4, 2, 3, 1.5)
    assert v.tolist() == [100.0, 100.0, 100.0, 50.0]
    assert t.tolist() == [0, 0, 0, 1] and p.tolist() == [0, 0, 0, 1] and a == 2
    # lambda 1.7: 2.0 < 1.7 * 1.25 = 2.125 -> nobody is a straggler
    v, t, p, a = oracle.ctl_decide(rep, 4, 2, 3, 1.7)
    assert t.sum() == 0 and p.sum() == 0 and a == 0


def test_checker_transient_but_not_persistent():
    # the straggle only shows in the last 2 reports; the long window (10) dilutes it
    rep = [(w, 64, 1.0) for _ in range(8) for w in range(3)]
    rep += [(0, 64, 1.0), (1, 64, 1.0), (2, 64, 4.0)] * 2
    v, t, p, a = oracle.ctl_decide(rep, 3, 2, 10, 1.5)
    assert t.tolist() == [0, 0, 1] and p.tolist() == [0, 0, 0] and a == 1
    assert v.tolist() == [64.0, 64.0, 16.0]
    # the resulting speeds give the slow worker a quarter of the others' batch (Eq. 3)
    assert oracle.batch_sizes(v, 3, 576).tolist() == [256, 256, 64]


def test_lambda_test_flags_a_worker_exactly_at_the_threshold():
    # Section VI-A step 3 prints the test with ">=".  Batch-processing times 1, 1, 1, 3 (all exact
    # in binary): mean 1.5, lambda 2 -> threshold exactly 3.0, so worker 3 IS a straggler; a strict
    # comparison would let it pass.  One ulp below the threshold it is not.
    rep = [(w, 128, 3.0 if w == 3 else 1.0) for _ in range(4) for w in range(4)]
    v, t, p, a = oracle.ctl_decide(rep, 4, 2, 4, 2.0)
    assert t.tolist() == [0, 0, 0, 1] and p.tolist() == [0, 0, 0, 1] and a == 2
    below = float(np.nextafter(3.0, 0.0))
    rep = [(w, 128, below if w == 3 else 1.0) for _ in range(4) for w in range(4)]
    v, t, p, a = oracle.ctl_decide(rep, 4, 2, 4, 2.0)
    assert t.sum() == 0 and p.sum() == 0 and a == 0


def test_persistent_test_compares_with_the_mean_of_the_long_windows():
    # BPTs of worker 0: 1, 1, 1, 4; of worker 1: 2, 2, 2, 4.  Short window (1 report): 4 and 4, mean 4.
    # Long window (4 reports): 1.75 and 2.5, mean 2.125.  lambda = 1.1: worker 1 is a persistent
    # straggler (2.5 >= 1.1 * 2.125 = 2.3375) although nobody is a transient one (4 < 4.4); measured
    # against the short windows' mean (4.4) it would not be flagged.
    rep = []
    for k in range(4):
        rep += [(0, 32, 4.0 if k == 3 else 1.0), (1, 32, 4.0 if k == 3 else 2.0)]
    v, t, p, a = oracle.ctl_decide(rep, 2, 1, 4, 1.1)
    assert t.tolist() == [0, 0] and p.tolist() == [0, 1] and a == 2


def test_window_means_divide_by_the_reports_each_worker_has():
    # worker 1 joined late: two reports of 3 s against worker 0's four of 1 s; long window 4, short
    # window 1.  Its long-window MEAN is 3 (not 6/4, and not the sum 6): 3 >= 1.4 * mean(1, 3) = 2.8.
    rep = [(0, 16, 1.0), (0, 16, 1.0), (0, 16, 1.0), (1, 16, 3.0), (0, 16, 1.0), (1, 16, 3.0)]
    v, t, p, a = oracle.ctl_decide(rep, 2, 1, 4, 1.4)
    assert p.tolist() == [0, 1] and t.tolist() == [0, 1] and a == 2
    # with lambda 1.6 the threshold is 3.2: not flagged (a window mean of 6/1 or 6/2 * ... would be)
    v, t, p, a = oracle.ctl_decide(rep, 2, 1, 4, 1.6)
    assert p.sum() == 0 and t.sum() == 0 and a == 0
    # the same for the short window: two reports of 1 s against one report of 1.5 s, window 2:
    # means 1 and 1.5 (sums would be 2 and 1.5 and flag the wrong worker), threshold 1.1 * 1.25
    rep = [(0, 16, 1.0), (0, 16, 1.0), (1, 16, 1.5)]
    v, t, p, a = oracle.ctl_decide(rep, 2, 2, 2, 1.1)
    assert t.tolist() == [0, 1] and p.tolist() == [0, 1]


def test_throughput_is_mean_of_per_report_rates():
    rep = [(0, 100, 1.0), (0, 300, 2.0), (1, 100, 1.0), (1, 100, 1.0)]
    v, _, _, _ = oracle.ctl_decide(rep, 2, 5, 5, 1.5)
    assert v[0] == pytest.approx((100.0 + 150.0) / 2) and v[1] == 100.0


def test_library_matches_checker_on_the_papers_straggler_pattern():
    # Section VII-A.3: a delay of SleepDuration * Intensity added with probability 0.3 per node
    rng = np.random.default_rng(5)
    K, Lt, Lp, lam = 10, 5, 10, 1.5
    ctl = B.Ctl(K, Lt, Lp, lam)
    with pytest.raises(B.AntdtError):
        ctl.antdt_ctl_decide()                     # nobody has reported yet
    disturbed = rng.random(K) < 0.3
    disturbed[3] = True
    reports = []
    bsz = [512] * K
    for it in range(40):
        for w in range(K):
            bpt = 0.5 + 0.02 * rng.random() + (1.5 * 0.8 if disturbed[w] and 10 <= it < 30 else 0.0)
            ctl.antdt_ctl_report(w, bsz[w], bpt)
            reports.append((w, bsz[w], bpt))
        v, t, p, a = ctl.antdt_ctl_decide()
        ov, ot, op, oa = oracle.ctl_decide(reports, K, Lt, Lp, lam)
        assert np.allclose(v, ov, rtol=1e-12) and t == ot.tolist() and p == op.tolist() and a == oa
        if 16 <= it < 30:
            assert [bool(x) for x in t] == disturbed.tolist()
        if it >= 36:
            assert sum(t) == 0
        if a == B.ACTION_ADJUST_BS:
            bsz = B.antdt_batch_sizes(v, K, 512 * K)
            assert sum(bsz) == 512 * K
    for bad in ((K, 1, 1.0), (0, -1, 1.0), (0, 1, 0.0), (0, 1, float("nan"))):
        with pytest.raises(B.AntdtError):
            ctl.antdt_ctl_report(*bad)
    with pytest.raises(B.AntdtError):
        B.Ctl(4, 0, 1, 1.5)
    with pytest.raises(B.AntdtError):
        B.Ctl(4, 1, 1, 1.0)


# ---- AntDT-DD, Eq. 4 -------------------------------------------------------------------------
def test_dd_checker_on_the_papers_gpu_cluster():
    # Section VII-A: 4 V100 + 4 P100, V100 about 3x a P100 (Section I), B = 768.
    # Without accumulation (C = 1) and wide bounds Eq. 4 is Eq. 3: 144 / 48, z = 48.
    b, c, z = oracle.dd_solve([4, 4], [3.0, 1.0], 768, [1, 1], [768, 768], 1, 1)
    assert b.tolist() == [144, 48] and c.tolist() == [1, 1] and z == 48.0
    # P100 saturates below 96 samples (B_min), V100 holds at most 96 (B_max): accumulation is
    # needed: 4*C1*B1 + 4*C2*B2 = 768
    b, c, z = oracle.dd_solve([4, 4], [3.0, 1.0], 768, [32, 96], [96, 192], 1, 5)
    assert 4 * c[0] * b[0] + 4 * c[1] * b[1] == 768
    assert (b.tolist(), c.tolist()) == ([96, 96], [1, 1]) and z == 96.0
    with pytest.raises(oracle.OracleError) as e:
        oracle.dd_solve([4, 4], [3.0, 1.0], 770, [1, 1], [768, 768], 1, 5)   # 770 not a multiple of 4
    assert e.value.code == 10


def test_dd_optimum_is_a_lower_bound_witness():
    # z* can never beat the continuous bound B / sum_i n_i v_i, and for divisible cases meets it
    b, c, z = oracle.dd_solve([2, 2], [2.0, 1.0], 600, [1, 1], [1000, 1000], 1, 3)
    assert z == 600 / (2 * 2.0 + 2 * 1.0)
    assert 2 * c[0] * b[0] + 2 * c[1] * b[1] == 600 and c[0] * b[0] == 200 and c[1] * b[1] == 100


def test_dd_library_matches_checker():
    rng = np.random.default_rng(9)
    feasible = 0
    for _ in range(60):
        k = int(rng.integers(1, 4))
        n_dev = rng.integers(1, 5, size=k)
        v = np.round(rng.uniform(0.5, 4.0, size=k), 2)
        bmin = rng.integers(1, 8, size=k)
        bmax = bmin + rng.integers(0, 25, size=k)
        cmin, cmax = 1, int(rng.integers(1, 4))
        Bt = int(rng.integers(10, 400))
        try:
            ob, oc, oz = oracle.dd_solve(n_dev, v, Bt, bmin, bmax, cmin, cmax)
        except oracle.OracleError as e:
            assert e.code == 10
            with pytest.raises(B.AntdtError) as e2:
                B.antdt_dd_solve(n_dev, v, Bt, bmin, bmax, cmin, cmax)
            assert e2.value.code == B.ERR_INFEASIBLE
            continue
        feasible += 1
        b, c, z = B.antdt_dd_solve(n_dev, v, Bt, bmin, bmax, cmin, cmax)
        assert (b, c, z) == (ob.tolist(), oc.tolist(), oz)
        assert sum(int(n) * ci * bi for n, ci, bi in zip(n_dev, c, b)) == Bt
    assert feasible > 10
    assert B.antdt_dd_solve([4, 4], [3.0, 1.0], 768, [1, 1], [768, 768], 1, 1) == ([144, 48], [1, 1], 48.0)
    with pytest.raises(B.AntdtError):
        B.antdt_dd_solve([4, 0], [3.0, 1.0], 768, [1, 1], [768, 768], 1, 1)
