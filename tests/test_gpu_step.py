"""Whole BSP steps of the five workload shapes on the GPU against the CPU checker: every stage
per step from identical state (the GPU is fed the checker's current table and optimizer state),
plus the free-running trajectory over all steps.  Configs 1 and 2 run at their stated batch and
field sizes; 2-5 use smaller tables / batches here so the checker finishes in seconds (the
full-size cases are in test_gpu_fullsize.py)."""
import numpy as np
import pytest
import torch

from paper_2404_09679_b200 import binding as B
from paper_2404_09679_b200 import synth
from paper_2404_09679_b200.step import OptConfig, StepBuffers, run_step
from tests import gpu_util as G
from tests.step_harness import OracleState, make_batch, plan_steps, table_np

pytestmark = pytest.mark.gpu

CASES = {
    "c1": (synth.WORKLOADS[1], 10),
    "c2": (synth.WORKLOADS[2].scaled(V=26 * 100_000), 10),
    "c3": (synth.WORKLOADS[3].scaled(B=2048, V=200_000, dense_n=65_536), 5),
    "c4": (synth.WORKLOADS[4].scaled(B=2048, V=1_000_000), 5),
    "c5": (synth.WORKLOADS[5].scaled(B=16_384, V=500_000, dense_n=131_072), 5),
}


def _to_dev(table_np_, bf16):
    return G.table_to_dev(table_np_)


@pytest.mark.parametrize("name", list(CASES))
def test_steps_match_checker(name):
    w, n_steps = CASES[name]
    plans = plan_steps(w, n_steps)
    if name == "c1":
        assert plans[0]["batch_sizes"] == [64, 128, 128, 192]
    if name == "c2":
        assert plans[0]["batch_sizes"] == [2428, 2427, 2427, 2427, 2427, 2427, 1214, 607]
    bm = synth.BatchMaker(w, "cuda")
    table0 = bm.table()
    ref = OracleState(w, table0)
    oc = OptConfig(B.OPTS[w.opt], w.lr, w.eps, w.beta1, w.beta2)
    bf16 = w.table_dtype == "bf16"

    # free-running GPU state
    free_t = table0.clone()
    free_s0 = torch.zeros(w.V, w.D, device="cuda")
    free_s1 = torch.zeros(w.V, w.D, device="cuda") if w.opt == "adam" else None
    buf = None
    for s in range(n_steps):
        batch = make_batch(bm, plans[s], s)
        nnz, n_bags = batch["row_ids"].numel(), batch["bag_offsets"].numel() - 1
        if buf is None or nnz > buf.max_nnz:
            buf = StepBuffers(w.D, w.K, int(nnz * 1.2), n_bags, w.dense_n)
        # --- (1) per call from the checker's state -------------------------------------------
        t = _to_dev(ref.table, bf16)
        s0 = G.dev(ref.s0)
        s1 = None if ref.s1 is None else G.dev(ref.s1)
        state_before = (ref.table.copy(), ref.s0.copy(), None if ref.s1 is None else ref.s1.copy())
        want = ref.step(batch, s + 1)           # advances the checker
        buf.status.zero_()
        run_step(buf, t, s0, s1, oc, s + 1, batch["row_ids"], batch["bag_offsets"], w.F,
                 batch["d_pooled"], batch["wso"].tolist(), batch["counts"].tolist(), batch["dense"])
        assert B.antdt_read_status(buf.status) == 0
        G.close(buf.pooled[:n_bags].cpu().numpy(), want["pooled"])
        bw = want["bwd"]
        nu = len(bw["uniq_ids"])
        assert np.array_equal(buf.worker_uniq_offsets.cpu().numpy(), bw["worker_uniq_offsets"])
        assert np.array_equal(buf.uniq_ids[:nu].cpu().numpy(), bw["uniq_ids"])
        assert np.array_equal(buf.seg_offsets[:nu + 1].cpu().numpy(), bw["seg_offsets"])
        assert np.array_equal(buf.sorted_occ[:nnz].cpu().numpy(), bw["sorted_occ"])
        G.close(buf.uniq_grads[:nu].cpu().numpy(), bw["uniq_grads"])
        na = int(buf.n_agg.item())
        assert na == len(want["agg_ids"])
        assert np.array_equal(buf.agg_ids[:na].cpu().numpy(), want["agg_ids"])
        # chained stages: inputs differ from the checker's by the previous stage's rounding
        G.close(buf.agg_grads[:na].cpu().numpy(), want["agg"], rtol=3e-5, atol=2e-6)
        if w.dense_n:
            G.close(buf.dense_out.cpu().numpy(), want["dense"])
        # the update, on the checker's own aggregate (identical inputs) from the same state
        t2, s0b = _to_dev(state_before[0], bf16), G.dev(state_before[1])
        s1b = None if state_before[2] is None else G.dev(state_before[2])
        n_dev = torch.tensor([na], dtype=torch.int64, device="cuda")
        B.antdt_sparse_opt_update(t2, G.dev(want["agg_ids"]), G.dev(want["agg"]), n_dev, oc.opt,
                                  oc.lr, oc.eps, oc.beta1, oc.beta2, s + 1, s0b, s1b, buf.status)
        assert B.antdt_read_status(buf.status) == 0
        if bf16:
            a = (table_np(t2).astype(np.uint32) << 16).view(np.float32)
            b = (ref.table.astype(np.uint32) << 16).view(np.float32)
            G.close(a, b, rtol=G.BF16_RTOL, atol=1e-6)
        else:
            G.close(table_np(t2), ref.table)
        G.close(s0b.cpu().numpy(), ref.s0)
        if s1b is not None:
            G.close(s1b.cpu().numpy(), ref.s1)
        # and the chained update (fed the GPU's own aggregate)
        rows = torch.from_numpy(want["agg_ids"].astype(np.int64)).cuda()
        got_rows = table_np(t[rows])
        if bf16:
            a = (got_rows.astype(np.uint32) << 16).view(np.float32)
            b = (ref.table[want["agg_ids"]].astype(np.uint32) << 16).view(np.float32)
            G.close_mostly(a, b, G.BF16_RTOL, 1e-6, 1e-3, 2 * w.lr)
        else:
            G.close_mostly(got_rows, ref.table[want["agg_ids"]], 5e-5, 2e-6, 1e-3, 2 * w.lr)
        # the state is well conditioned (acc += g^2 and m += (1-b1) g move by at most 2|g| dg + dg^2
        # and dg for a gradient off by dg): no element may leave a band of the tolerance's own size
        s0_want = ref.s0[want["agg_ids"]]
        G.close_mostly(s0[rows].cpu().numpy(), s0_want, 1e-4, 1e-7, 1e-3,
                       1e-6 + 1e-4 * float(np.abs(s0_want).max()))
        # --- (2) free-running trajectory -----------------------------------------------------
        run_step(buf, free_t, free_s0, free_s1, oc, s + 1, batch["row_ids"], batch["bag_offsets"],
                 w.F, batch["d_pooled"], batch["wso"].tolist(), batch["counts"].tolist(),
                 batch["dense"])
        assert B.antdt_read_status(buf.status) == 0
    got = table_np(free_t)
    if bf16:
        a = (got.astype(np.uint32) << 16).view(np.float32)
        b = (ref.table.astype(np.uint32) << 16).view(np.float32)
        G.close_mostly(a, b, 2 * G.BF16_RTOL, 1e-5, 1e-3, 2 * w.lr * n_steps)
    else:
        G.close_mostly(got, ref.table, 1e-3, 1e-5, 1e-3, 2 * w.lr * n_steps)
    touched = np.flatnonzero(np.any(ref.s0 != 0, axis=1))
    assert np.array_equal(np.flatnonzero(np.any(free_s0.cpu().numpy() != 0, axis=1)), touched)
