"""antdt_aggregate_update (Section II: the servers aggregate the local gradients and update the
parameters) against the CPU checker's two steps, and against the two separate device calls.

The call's weighted sums differ from the checker's float-rounded aggregate by rounding only, and
an Adagrad / Adam step divides by |g|-sized quantities, so the few elements whose aggregated
gradient is within rounding of zero may move by up to a learning rate (gpu_util.close_mostly); the
aggregate itself, when it is asked for, is checked at the fp32 tolerance."""
import numpy as np
import pytest
import torch

import oracle
from paper_2404_09679_b200 import binding as B
from tests import gpu_util as G
from tests.util import bf16_bits_to_f64

pytestmark = pytest.mark.gpu


def _lists(rng, K, V, n_per, hot):
    """Ascending id lists of K workers with a shared hot set, so rows have 1..K contributions."""
    ids, wuo = [], [0]
    for _ in range(K):
        cold = rng.integers(0, V, size=n_per)
        mine = np.unique(np.concatenate([cold, hot[rng.random(len(hot)) < 0.7]]))
        ids.append(mine.astype(np.int32))
        wuo.append(wuo[-1] + len(mine))
    return np.concatenate(ids), np.array(wuo, np.int64)


@pytest.mark.parametrize("opt,D,bf16,K,materialise", [
    ("adagrad", 64, True, 16, False), ("adagrad", 16, False, 4, True), ("adam", 32, False, 32, False),
    ("adam", 64, True, 7, True), ("adagrad", 256, False, 3, False), ("adam", 8, False, 40, True)])
def test_fused_aggregate_update_matches_the_checkers_two_steps(opt, D, bf16, K, materialise):
    rng = np.random.default_rng(1000 * D + 10 * K + len(opt))
    V, n_per = 60_000, 4000
    hot = rng.integers(0, V, size=300)
    uid, wuo = _lists(rng, K, V, n_per, hot)
    g = rng.normal(size=(len(uid), D)).astype(np.float32)
    bsz = rng.integers(1, 200, size=K)
    lr, eps, b1, b2, step = 0.05, 1e-8, 0.9, 0.999, 3
    t0 = rng.normal(0, 0.5, size=(V, D)).astype(np.float32)
    if bf16:
        t0 = ((t0.view(np.uint32) >> 16).astype(np.uint16))            # truncated: exact bf16 values
    s0 = np.abs(rng.normal(size=(V, D))).astype(np.float32) * 0.1
    s1 = np.abs(rng.normal(size=(V, D))).astype(np.float32) * 0.1 if opt == "adam" else None

    want_ids, want_agg = oracle.aggregate_sparse(uid, wuo, g, bsz)
    t_ref, s0_ref = t0.copy(), s0.copy()
    s1_ref = None if s1 is None else s1.copy()
    oracle.sparse_opt_update(t_ref, want_ids, want_agg, opt, lr, eps, b1, b2, step, s0_ref, s1_ref)

    table, d0 = G.table_to_dev(t0), G.dev(s0)
    d1 = None if s1 is None else G.dev(s1)
    n_in = len(uid)
    agg_ids = torch.full((n_in,), -1, dtype=torch.int32, device="cuda")
    agg = torch.full((n_in, D), float("nan"), device="cuda") if (materialise or K > 32) else None
    n_agg = torch.zeros(1, dtype=torch.int64, device="cuda")
    ws = torch.empty(B.antdt_weighted_aggregate_workspace_bytes(n_in, D, K), dtype=torch.uint8, device="cuda")
    st = G.new_status()
    B.antdt_aggregate_update([int(b) for b in bsz], ws, table, B.OPTS[opt], lr, eps, b1, b2, step, d0, d1,
                             uniq_ids=G.dev(uid), worker_uniq_offsets=G.dev(wuo), uniq_grads=G.dev(g),
                             agg_ids=agg_ids, n_agg=n_agg, agg_grads=agg, dev_status=st)
    assert B.antdt_read_status(st) == 0
    na = int(n_agg.item())
    assert na == len(want_ids) and np.array_equal(agg_ids[:na].cpu().numpy(), want_ids)
    if agg is not None:
        G.close(agg[:na].cpu().numpy(), want_agg)
    rows = want_ids.astype(np.int64)
    got_t = G.table_to_np(table)
    if bf16:
        G.close_mostly(bf16_bits_to_f64(got_t[rows]), bf16_bits_to_f64(t_ref[rows]), G.BF16_RTOL, 1e-6, 1e-3, 2 * lr)
    else:
        G.close_mostly(got_t[rows], t_ref[rows], 5e-5, 2e-6, 1e-3, 2 * lr)
    G.close_mostly(d0.cpu().numpy()[rows], s0_ref[rows], 1e-4, 1e-7, 1e-3, 1e-6 + 1e-4 * float(np.abs(s0_ref).max()))
    if s1 is not None:
        G.close_mostly(d1.cpu().numpy()[rows], s1_ref[rows], 1e-4, 1e-7, 1e-3, 1e-6 + 1e-4 * float(np.abs(s1_ref).max()))
    # rows outside the union: bit-identical
    mask = np.ones(V, bool)
    mask[rows] = False
    assert np.array_equal(got_t[mask], t0[mask]) and np.array_equal(d0.cpu().numpy()[mask], s0[mask])


def test_fused_call_rejects_bad_arguments():
    z = torch.zeros(4, 8, device="cuda")
    ids = torch.zeros(4, dtype=torch.int32, device="cuda")
    wuo = torch.zeros(3, dtype=torch.int64, device="cuda")
    n_agg = torch.zeros(1, dtype=torch.int64, device="cuda")
    ws = torch.empty(B.antdt_weighted_aggregate_workspace_bytes(4, 8, 2), dtype=torch.uint8, device="cuda")
    common = dict(uniq_ids=ids, worker_uniq_offsets=wuo, uniq_grads=z, agg_ids=ids.clone(), n_agg=n_agg)
    with pytest.raises(B.AntdtError) as e:      # row-wise Adagrad is not offered in one pass
        B.antdt_aggregate_update([1, 1], ws, z.clone(), B.OPT_ROWWISE_ADAGRAD, 0.1, 1e-8, 0.9, 0.999, 1,
                                 torch.zeros(4, device="cuda"), None, **common)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.AntdtError) as e:      # Adam needs its second state
        B.antdt_aggregate_update([1, 1], ws, z.clone(), B.OPT_ADAM, 0.1, 1e-8, 0.9, 0.999, 1, z.clone(), None,
                                 **common)
    assert e.value.code == B.ERR_INVALID_ARG
