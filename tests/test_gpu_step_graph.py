"""antdt_bsp_step_graph (the step replayed as one CUDA graph launch) against
antdt_bsp_step_device (plain launches) and the CPU checker.

The kernels are deterministic, so the two launch forms must agree bit for bit on every output
and on the table and optimizer state after every step.  The cases cover the three ways a call
meets the graph store: a descriptor seen before (replay), a new descriptor while slots are free
(instantiate), and a new descriptor once the 8 slots are taken (least recently used graph
updated in place) - including batches whose sizes differ from step to step - and Adam, which
the entry point issues as plain launches (its step number changes kernel parameters every
step, so no graph could be replayed)."""
import numpy as np
import pytest
import torch

from paper_2404_09679_b200 import binding as B
from paper_2404_09679_b200 import synth
from paper_2404_09679_b200.step import DeviceStep, OptConfig, StepBuffers
from tests import gpu_util as G
from tests.step_harness import OracleState, make_batch, plan_steps

pytestmark = pytest.mark.gpu

CASES = {
    # 12 steps with a different occurrence count each: more distinct descriptors than slots
    "c1_varying_sizes": (synth.WORKLOADS[1], 12, 12),
    # fixed sizes, two batches in rotation: every step after the first two is a replay
    "c2_replay": (synth.WORKLOADS[2].scaled(V=26 * 50_000), 8, 2),
    # Adagrad with a dense part: the three-branch graph with the dense weighted sum behind the join
    "c1_dense_adagrad": (synth.WORKLOADS[1].scaled(dense_n=8192), 6, 3),
    # Adam + dense part: issued as plain launches by the entry point
    "c3_adam_dense": (synth.WORKLOADS[3].scaled(B=2048, V=200_000, dense_n=65_536), 10, 3),
}


class _Side:
    """One copy of the model state and buffers, stepped through one of the two entry points."""

    def __init__(self, w, table0, max_nnz, max_bags, graph, fuse_update=False):
        self.table = table0.clone()
        self.s0 = torch.zeros(w.V, w.D, device="cuda")
        self.s1 = torch.zeros(w.V, w.D, device="cuda") if w.opt == "adam" else None
        self.buf = StepBuffers(w.D, w.K, max_nnz, max_bags, w.dense_n)
        oc = OptConfig(B.OPTS[w.opt], w.lr, w.eps, w.beta1, w.beta2)
        self.step = DeviceStep(self.buf, self.table, self.s0, self.s1, oc, w.K, fuse_update=fuse_update)
        self.graph = graph

    def run(self, t, b, F):
        self.step.run(t, b["row_ids"], b["bag_offsets"], F, b["d_pooled"], b["wso"].tolist(),
                      b["counts"].tolist(), b["dense"], graph=self.graph)


def _same(a, b, what):
    assert torch.equal(a, b), what


@pytest.mark.parametrize("name", list(CASES))
def test_graph_step_equals_plain_step(name):
    w, n_steps, n_batches = CASES[name]
    plans = plan_steps(w, n_batches)
    bm = synth.BatchMaker(w, "cuda")
    table0 = bm.table()
    batches = [make_batch(bm, plans[j], j) for j in range(n_batches)]
    max_nnz = max(b["row_ids"].numel() for b in batches)
    max_bags = max(b["bag_offsets"].numel() - 1 for b in batches)
    plain = _Side(w, table0, max_nnz, max_bags, graph=False)
    graph = _Side(w, table0, max_nnz, max_bags, graph=True)
    ref = OracleState(w, table0) if name == "c1_varying_sizes" else None
    B.antdt_bsp_step_graph_reset()
    launches = []
    for s in range(n_steps):
        b = batches[s % n_batches]
        nnz, n_bags = b["row_ids"].numel(), b["bag_offsets"].numel() - 1
        l0 = B.antdt_launch_count()
        plain.run(s + 1, b, w.F)
        l1 = B.antdt_launch_count()
        graph.run(s + 1, b, w.F)
        l2 = B.antdt_launch_count()
        launches.append((l1 - l0, l2 - l1))
        torch.cuda.synchronize()
        assert B.antdt_read_status(plain.buf.status) == 0
        assert B.antdt_read_status(graph.buf.status) == 0
        p, g = plain.buf, graph.buf
        _same(p.pooled[:n_bags], g.pooled[:n_bags], f"pooled, step {s}")
        _same(p.worker_uniq_offsets, g.worker_uniq_offsets, f"worker_uniq_offsets, step {s}")
        nu = int(p.worker_uniq_offsets[w.K].item())
        _same(p.uniq_ids[:nu], g.uniq_ids[:nu], f"uniq_ids, step {s}")
        _same(p.seg_offsets[:nu + 1], g.seg_offsets[:nu + 1], f"seg_offsets, step {s}")
        _same(p.sorted_occ[:nnz], g.sorted_occ[:nnz], f"sorted_occ, step {s}")
        _same(p.uniq_grads[:nu], g.uniq_grads[:nu], f"uniq_grads, step {s}")
        _same(p.n_agg, g.n_agg, f"n_agg, step {s}")
        na = int(p.n_agg.item())
        _same(p.agg_ids[:na], g.agg_ids[:na], f"agg_ids, step {s}")
        _same(p.agg_grads[:na], g.agg_grads[:na], f"agg_grads, step {s}")
        if w.dense_n:
            _same(p.dense_out, g.dense_out, f"dense_out, step {s}")
        _same(plain.table, graph.table, f"table, step {s}")
        _same(plain.s0, graph.s0, f"state0, step {s}")
        if plain.s1 is not None:
            _same(plain.s1, graph.s1, f"state1, step {s}")
        if ref is not None and s == 0:      # the graph side against the checker, first step
            want = ref.step(b, 1)
            G.close(g.pooled[:n_bags].cpu().numpy(), want["pooled"])
            assert np.array_equal(g.uniq_ids[:nu].cpu().numpy(), want["bwd"]["uniq_ids"])
            assert np.array_equal(g.seg_offsets[:nu + 1].cpu().numpy(), want["bwd"]["seg_offsets"])
            G.close(g.uniq_grads[:nu].cpu().numpy(), want["bwd"]["uniq_grads"])
            assert np.array_equal(g.agg_ids[:na].cpu().numpy(), want["agg_ids"])
            G.close(g.agg_grads[:na].cpu().numpy(), want["agg"], rtol=3e-5, atol=2e-6)
    # a replayed or freshly captured graph accounts for the same kernels as the plain launches
    assert all(a == b and a > 0 for a, b in launches), launches
    B.antdt_bsp_step_graph_reset()


@pytest.mark.parametrize("name", ["c1_varying_sizes", "c2_replay", "c1_dense_adagrad"])
def test_one_pass_server_step_as_graph_equals_plain_and_agrees_with_the_two_kernel_step(name):
    """fuse_update: aggregation and update in one kernel.  As a graph (three branches on these
    sizes) it must equal its plain launches bit for bit; against the two-kernel step the table and
    the accumulator agree to rounding (the weighted sum is formed with fused multiply-adds in the
    one-pass kernel), step after step on free-running state."""
    w, n_steps, n_batches = CASES[name]
    n_steps = min(n_steps, 6)
    plans = plan_steps(w, n_batches)
    bm = synth.BatchMaker(w, "cuda")
    table0 = bm.table()
    batches = [make_batch(bm, plans[j], j) for j in range(n_batches)]
    max_nnz = max(b["row_ids"].numel() for b in batches)
    max_bags = max(b["bag_offsets"].numel() - 1 for b in batches)
    two = _Side(w, table0, max_nnz, max_bags, graph=False)
    plain = _Side(w, table0, max_nnz, max_bags, graph=False, fuse_update=True)
    graph = _Side(w, table0, max_nnz, max_bags, graph=True, fuse_update=True)
    B.antdt_bsp_step_graph_reset()
    for s in range(n_steps):
        b = batches[s % n_batches]
        n_bags = b["bag_offsets"].numel() - 1
        for side in (two, plain, graph):
            side.run(s + 1, b, w.F)
        torch.cuda.synchronize()
        for side in (two, plain, graph):
            assert B.antdt_read_status(side.buf.status) == 0
        _same(plain.buf.pooled[:n_bags], graph.buf.pooled[:n_bags], f"pooled, step {s}")
        _same(plain.buf.n_agg, graph.buf.n_agg, f"n_agg, step {s}")
        na = int(plain.buf.n_agg.item())
        _same(plain.buf.agg_ids[:na], graph.buf.agg_ids[:na], f"agg_ids, step {s}")
        _same(plain.table, graph.table, f"table, step {s}")
        _same(plain.s0, graph.s0, f"state0, step {s}")
        if w.dense_n:
            _same(plain.buf.dense_out, graph.buf.dense_out, f"dense_out, step {s}")
            _same(two.buf.dense_out, plain.buf.dense_out, f"dense_out vs two-kernel step, step {s}")
        _same(two.buf.agg_ids[:na], plain.buf.agg_ids[:na], f"agg_ids vs two-kernel step, step {s}")
        rows = plain.buf.agg_ids[:na].long()
        G.close_mostly(plain.table[rows].cpu().numpy(), two.table[rows].cpu().numpy(), 5e-5, 2e-6, 1e-3, 2 * w.lr)
        G.close_mostly(plain.s0[rows].cpu().numpy(), two.s0[rows].cpu().numpy(), 1e-4, 1e-7, 1e-3,
                       1e-6 + 1e-4 * float(two.s0.abs().max().item()))
    B.antdt_bsp_step_graph_reset()


def test_graph_step_reports_argument_errors():
    w = synth.WORKLOADS[1]
    plans = plan_steps(w, 1)
    bm = synth.BatchMaker(w, "cuda")
    b = make_batch(bm, plans[0], 0)
    side = _Side(w, bm.table(), b["row_ids"].numel(), b["bag_offsets"].numel() - 1, graph=True)
    bad = b["wso"].copy()
    bad[-1] += 1                      # worker offsets that do not cover the batch
    with pytest.raises(B.AntdtError) as ei:
        side.step.run(1, b["row_ids"], b["bag_offsets"], w.F, b["d_pooled"], bad.tolist(),
                      b["counts"].tolist(), None, graph=True)
    assert ei.value.code == B.ERR_INVALID_ARG
    # the stream is usable and not left capturing: a correct call goes through afterwards
    side.run(1, b, w.F)
    torch.cuda.synchronize()
    assert B.antdt_read_status(side.buf.status) == 0
    B.antdt_bsp_step_graph_reset()
