"""Full-size steps (configs 2-5 as stated: tables up to 1e8 rows, up to 1.05e8 occurrences) in
the launch configuration bench.py times.  The CPU checker cannot run these whole, so:

  * integer outputs are checked completely against properties that fix them uniquely, using
    torch's own stable sort / unique on the device as the independent reference (ascending ids,
    run starts, stable occurrence order, union of the workers' rows);
  * floating-point outputs are checked against the checker on sampled outputs it can compute one
    by one: pooled rows of sampled bags, and -- for a sample of table rows that always includes
    the hottest ones -- the worker gradients, the aggregate and the updated table / state rows,
    obtained by running the checker on the sub-problem that keeps only the occurrences of those
    rows (every stage is independent per row, so the sub-problem's results are the full
    problem's results for those rows);
  * rows the step must not touch are compared bit for bit with their initial values.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2404_09679_b200 import binding as B
from paper_2404_09679_b200 import synth
from paper_2404_09679_b200.step import OptConfig, StepBuffers, run_step
from tests import gpu_util as G
from tests.step_harness import plan_steps, table_np

pytestmark = pytest.mark.gpu


def _rows_np(t):
    return table_np(t)


@pytest.mark.parametrize("cfg", [2, 3, 4, 5])
def test_full_size_step(cfg):
    w = synth.WORKLOADS[cfg]
    dev = torch.device("cuda")
    free, total = torch.cuda.mem_get_info()
    need = w.V * w.D * ((2 if w.table_dtype == "bf16" else 4) + (8 if w.opt == "adam" else 4)) + 30e9
    if free < need:
        pytest.skip(f"needs {need / 1e9:.0f} GB of device memory")
    plan = plan_steps(w, 1)[0]
    bm = synth.BatchMaker(w, dev)
    idx = synth.sample_indices(plan["ranges"], dev)
    ids, off = bm.bags(idx)
    dY = bm.d_pooled(idx)
    dense = bm.dense_grads(0)
    counts = np.asarray(plan["counts"], np.int64)
    wso = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    nnz, n_bags = ids.numel(), off.numel() - 1
    table = bm.table()
    s0 = torch.zeros(w.V, w.D, device=dev)
    s1 = torch.zeros(w.V, w.D, device=dev) if w.opt == "adam" else None
    oc = OptConfig(B.OPTS[w.opt], w.lr, w.eps, w.beta1, w.beta2)
    rng = np.random.default_rng(cfg)

    # ---- references that must be taken before the step changes the table ---------------------
    ids64 = ids.to(torch.int64)
    all_rows = torch.unique(ids64)                                   # ascending
    hot = torch.bincount(ids64 % (1 << 22), minlength=1 << 22)       # cheap heavy-hitter screen
    cand = torch.topk(hot, 4).indices
    hot_rows = []
    for c in cand.tolist():
        m = ids64[(ids64 % (1 << 22)) == c]
        vals, cnt = torch.unique(m, return_counts=True)
        hot_rows.append(int(vals[cnt.argmax()]))
    pick = all_rows[torch.from_numpy(rng.choice(all_rows.numel(), size=2500, replace=False)).to(dev)]
    R = torch.unique(torch.cat([pick, torch.tensor(hot_rows, device=dev)]))
    untouched_probe = torch.from_numpy(rng.integers(0, w.V, size=200_000)).to(dev)
    untouched_probe = untouched_probe[~torch.isin(untouched_probe, all_rows)]
    t_before_R, t_before_probe = table[R].clone(), table[untouched_probe].clone()
    bag_sample = torch.from_numpy(np.sort(rng.choice(n_bags, size=3000, replace=False))).to(dev)

    # forward sample: compact sub-problem of the sampled bags
    lens = (off[1:] - off[:-1])[bag_sample]
    sub_off = torch.zeros(bag_sample.numel() + 1, dtype=torch.int64, device=dev)
    torch.cumsum(lens, 0, out=sub_off[1:])
    pos = torch.repeat_interleave(off[bag_sample], lens) + (
        torch.arange(int(sub_off[-1]), device=dev) - torch.repeat_interleave(sub_off[:-1], lens))
    sub_ids = ids64[pos]
    sub_rows = torch.unique(sub_ids)
    fwd_want = oracle.embbag_fwd(_rows_np(table[sub_rows]),
                                 torch.searchsorted(sub_rows, sub_ids).to(torch.int32).cpu().numpy(),
                                 sub_off.cpu().numpy())

    # ---- the step, as bench.py launches it --------------------------------------------------------
    buf = StepBuffers(w.D, w.K, nnz, n_bags, w.dense_n, uniq_cap=nnz // (2 if cfg == 4 else 1),
                      device=dev)
    run_step(buf, table, s0, s1, oc, 1, ids, off, w.F, dY, wso.tolist(), counts.tolist(), dense)
    assert B.antdt_read_status(buf.status) == 0

    # ---- forward ------------------------------------------------------------------------------------
    G.close(buf.pooled[bag_sample].cpu().numpy(), fwd_want)

    # ---- dedup: complete integer check against torch's stable sort per worker --------------------
    wuo = buf.worker_uniq_offsets.cpu().numpy()
    nu = int(wuo[w.K])
    uid, so, occ = buf.uniq_ids[:nu], buf.seg_offsets[:nu + 1], buf.sorted_occ[:nnz]
    assert int(so[0]) == 0 and int(so[nu]) == nnz
    assert bool((so[1:] > so[:-1]).all())
    bag_of = torch.repeat_interleave(torch.arange(n_bags, device=dev, dtype=torch.int32),
                                     off[1:] - off[:-1], output_size=nnz)
    occ_bounds = off[torch.from_numpy(wso * w.F).to(dev)].cpu().numpy()
    run_rows = torch.repeat_interleave(uid, so[1:] - so[:-1], output_size=nnz)   # row of each sorted slot
    for i in range(w.K):
        a, b = int(occ_bounds[i]), int(occ_bounds[i + 1])
        srt, perm = torch.sort(ids[a:b], stable=True)
        assert torch.equal(run_rows[a:b], srt), f"worker {i}: sorted row sequence"
        assert torch.equal(occ[a:b], bag_of[a:b][perm]), f"worker {i}: stable occurrence order"
        u = uid[int(wuo[i]):int(wuo[i + 1])]
        assert torch.equal(u.to(torch.int64), torch.unique(ids64[a:b])), f"worker {i}: distinct rows"
        assert int(so[int(wuo[i])]) == a if wuo[i] < wuo[i + 1] else True
        del srt, perm
    na = int(buf.n_agg.item())
    assert torch.equal(buf.agg_ids[:na].to(torch.int64), all_rows)

    # ---- sampled rows through the checker on the filtered sub-problem ----------------------------
    keep = torch.isin(ids64, R)
    kept_per_bag = torch.zeros(n_bags + 1, dtype=torch.int64, device=dev)
    torch.cumsum(torch.segment_reduce(keep.to(torch.float32), "sum", lengths=off[1:] - off[:-1]).to(torch.int64),
                 0, out=kept_per_bag[1:])
    f_ids = torch.searchsorted(R, ids64[keep]).to(torch.int32).cpu().numpy()      # compact row numbers
    f_off = kept_per_bag.cpu().numpy()
    dY_h = dY.cpu().numpy()
    ref = oracle.embbag_bwd_dedup(f_ids, f_off, w.F, dY_h, R.numel(), wso)
    R_h = R.cpu().numpy()
    for i in range(w.K):
        lo, hi = ref["worker_uniq_offsets"][i], ref["worker_uniq_offsets"][i + 1]
        if lo == hi:
            continue
        rows_i = torch.from_numpy(R_h[ref["uniq_ids"][lo:hi]]).to(dev)
        u = uid[int(wuo[i]):int(wuo[i + 1])].to(torch.int64)
        at = torch.searchsorted(u, rows_i)
        assert torch.equal(u[at], rows_i)
        G.close(buf.uniq_grads[int(wuo[i]) + at].cpu().numpy(), ref["uniq_grads"][lo:hi])
        # run lengths of the sampled rows
        want_len = np.diff(ref["seg_offsets"][lo:hi + 1]) if hi < len(ref["seg_offsets"]) else None
        got_len = (so[int(wuo[i]) + at + 1] - so[int(wuo[i]) + at]).cpu().numpy()
        assert want_len is None or np.array_equal(got_len, want_len)
    agg_ids_r, agg_r = oracle.aggregate_sparse(ref["uniq_ids"], ref["worker_uniq_offsets"],
                                               ref["uniq_grads"], counts)
    assert np.array_equal(agg_ids_r, np.arange(R.numel(), dtype=np.int32))      # every sampled row occurs
    at = torch.searchsorted(all_rows, R)
    G.close(buf.agg_grads[at].cpu().numpy(), agg_r, rtol=3e-5, atol=2e-6)
    if w.dense_n:
        e = rng.integers(0, w.dense_n, size=50_000)
        cols = torch.from_numpy(e).to(dev)
        want = oracle.aggregate_dense(np.ascontiguousarray(dense[:, cols].cpu().numpy()), counts)
        G.close(buf.dense_out[cols].cpu().numpy(), want)
    # update of the sampled rows, on the checker's aggregate (identical inputs)
    tR = _rows_np(t_before_R)
    r0 = np.zeros(tR.shape, np.float32)
    r1 = np.zeros(tR.shape, np.float32) if w.opt == "adam" else None
    oracle.sparse_opt_update(tR, agg_ids_r, agg_r, w.opt, w.lr, w.eps, w.beta1, w.beta2, 1, r0, r1)
    got = _rows_np(table[R])
    if w.table_dtype == "bf16":
        a = (got.astype(np.uint32) << 16).view(np.float32)
        b = (tR.astype(np.uint32) << 16).view(np.float32)
        G.close_mostly(a, b, G.BF16_RTOL, 1e-6, 1e-3, 2 * w.lr)
    else:
        G.close_mostly(got, tR, 5e-5, 2e-6, 1e-3, 2 * w.lr)
    # the state is well conditioned: no element may leave a band of the tolerance's own size
    G.close_mostly(s0[R].cpu().numpy(), r0, 1e-4, 1e-7, 1e-3, 1e-6 + 1e-4 * float(np.abs(r0).max()))
    # rows outside the batch: bit-identical
    assert torch.equal(table[untouched_probe].view(torch.int16 if w.table_dtype == "bf16" else torch.int32),
                       t_before_probe.view(torch.int16 if w.table_dtype == "bf16" else torch.int32))
    assert bool((s0[untouched_probe] == 0).all())
