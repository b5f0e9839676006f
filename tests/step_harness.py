"""Drives whole BSP steps of a workload through the CPU checker (numpy) and, where a GPU is
present, through the C-ABI, from the same planner output and the same seeded inputs."""
import numpy as np
import torch

import oracle
from paper_2404_09679_b200 import binding as B
from paper_2404_09679_b200 import synth


def plan_steps(w: synth.Workload, n_steps: int):
    """Library planner (the checker's planner is compared elsewhere): per step
    (batch_sizes, counts, ranges, range_offsets, speeds)."""
    dds = B.Dds(w.n_samples, w.B, w.M, w.K)
    out = []
    for s in range(n_steps):
        v = synth.speeds_for_step(w, s)
        rc, bsz, ro, rg, cnt = dds.antdt_shard_plan(v, B.RULES[w.rule], w.min_batch)
        assert rc == B.OK
        out.append(dict(batch_sizes=bsz, counts=cnt, ranges=rg, range_offsets=ro, speeds=v))
    return out


def make_batch(bm: synth.BatchMaker, plan, step: int):
    """Inputs of one step on bm.device: ids, offsets, d_pooled, dense grads, worker offsets."""
    idx = synth.sample_indices(plan["ranges"], bm.device)
    ids, off = bm.bags(idx)
    dY = bm.d_pooled(idx)
    wso = np.concatenate([[0], np.cumsum(plan["counts"])]).astype(np.int64)
    return dict(row_ids=ids, bag_offsets=off, d_pooled=dY, dense=bm.dense_grads(step), wso=wso,
                counts=np.asarray(plan["counts"], np.int64))


def table_np(t: torch.Tensor):
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16).copy()
    return t.cpu().numpy().copy()


class OracleState:
    def __init__(self, w: synth.Workload, table_t: torch.Tensor):
        self.w = w
        self.table = table_np(table_t)
        self.s0 = np.zeros(self.table.shape, np.float32)
        self.s1 = np.zeros(self.table.shape, np.float32) if w.opt == "adam" else None

    def step(self, batch, t: int):
        """One checker step; returns every stage's outputs."""
        w = self.w
        ids, off = batch["row_ids"].cpu().numpy(), batch["bag_offsets"].cpu().numpy()
        dY = batch["d_pooled"].cpu().numpy()
        pooled = oracle.embbag_fwd(self.table, ids, off)
        bwd = oracle.embbag_bwd_dedup(ids, off, w.F, dY, w.V, batch["wso"])
        agg_ids, agg = oracle.aggregate_sparse(bwd["uniq_ids"], bwd["worker_uniq_offsets"],
                                               bwd["uniq_grads"], batch["counts"])
        dense = None
        if batch["dense"] is not None:
            dense = oracle.aggregate_dense(batch["dense"].cpu().numpy(), batch["counts"])
        before = (self.table[agg_ids].copy(), self.s0[agg_ids].copy(),
                  None if self.s1 is None else self.s1[agg_ids].copy())
        oracle.sparse_opt_update(self.table, agg_ids, agg, w.opt, w.lr, w.eps, w.beta1, w.beta2, t,
                                 self.s0, self.s1)
        return dict(pooled=pooled, bwd=bwd, agg_ids=agg_ids, agg=agg, dense=dense, before=before)
