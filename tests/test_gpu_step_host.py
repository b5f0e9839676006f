"""antdt_bsp_step_host (the call bench.py's end-to-end leg times): one step from page-locked host
buffers must leave the same results as the four device calls issued one by one, and both must
match the CPU checker."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2404_09679_b200 import binding as B
from paper_2404_09679_b200 import synth
from paper_2404_09679_b200.step import OptConfig, StepBuffers, run_step
from tests import gpu_util as G
from tests.step_harness import OracleState, make_batch, plan_steps

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,scale", [(1, {}), (3, dict(B=1024, V=50_000, dense_n=8192)),
                                       (4, dict(B=1024, V=200_000))])
def test_host_buffer_step_matches_device_calls_and_checker(cfg, scale):
    w = synth.WORKLOADS[cfg].scaled(**scale)
    plans = plan_steps(w, 2)
    bm = synth.BatchMaker(w, "cuda")
    table0 = bm.table()
    ref = OracleState(w, table0)
    oc = OptConfig(B.OPTS[w.opt], w.lr, w.eps, w.beta1, w.beta2)
    t_a, t_b = table0.clone(), table0.clone()
    s0_a, s0_b = torch.zeros(w.V, w.D, device="cuda"), torch.zeros(w.V, w.D, device="cuda")
    adam = w.opt == "adam"
    s1_a = torch.zeros(w.V, w.D, device="cuda") if adam else None
    s1_b = torch.zeros(w.V, w.D, device="cuda") if adam else None
    stream = torch.cuda.current_stream()
    for s in range(2):
        batch = make_batch(bm, plans[s], s)
        nnz, n_bags = batch["row_ids"].numel(), batch["bag_offsets"].numel() - 1
        buf_a = StepBuffers(w.D, w.K, nnz, n_bags, w.dense_n)
        buf_b = StepBuffers(w.D, w.K, nnz, n_bags, w.dense_n)
        want = ref.step(batch, s + 1)
        run_step(buf_a, t_a, s0_a, s1_a, oc, s + 1, batch["row_ids"], batch["bag_offsets"], w.F,
                 batch["d_pooled"], batch["wso"].tolist(), batch["counts"].tolist(), batch["dense"])
        # the same step from host memory
        pin = lambda t: None if t is None else t.cpu().pin_memory()  # noqa: E731
        h_ids, h_off, h_dY, h_dense = pin(batch["row_ids"]), pin(batch["bag_offsets"]), \
            pin(batch["d_pooled"]), pin(batch["dense"])
        d_ids = torch.empty(nnz, dtype=torch.int32, device="cuda")
        d_off = torch.empty(n_bags + 1, dtype=torch.int64, device="cuda")
        d_dY = torch.empty(n_bags, w.D, device="cuda")
        d_dense = torch.empty(w.K, w.dense_n, device="cuda") if w.dense_n else None
        h_pooled = torch.empty(n_bags, w.D).pin_memory()
        h_dense_out = torch.empty(w.dense_n).pin_memory() if w.dense_n else None
        h_n_agg = torch.zeros(1, dtype=torch.int64).pin_memory()
        h_status = torch.full((1,), -1, dtype=torch.int32).pin_memory()
        wso = (C.c_int64 * (w.K + 1))(*[int(x) for x in batch["wso"]])
        bsz = (C.c_int64 * w.K)(*[int(x) for x in batch["counts"]])
        p = lambda t: None if t is None else t.data_ptr()  # noqa: E731
        d = B.StepDesc()
        d.table, d.dtype, d.n_rows, d.dim = p(t_b), (B.BF16 if t_b.dtype == torch.bfloat16 else B.F32), w.V, w.D
        d.state0, d.state1 = p(s0_b), p(s1_b)
        d.opt, d.lr, d.eps, d.beta1, d.beta2, d.step = oc.opt, oc.lr, oc.eps, oc.beta1, oc.beta2, s + 1
        d.h_row_ids, d.nnz, d.h_bag_offsets, d.n_bags, d.bags_per_sample = p(h_ids), nnz, p(h_off), n_bags, w.F
        d.h_d_pooled, d.h_dense_grads, d.dense_n, d.n_workers = p(h_dY), p(h_dense), w.dense_n, w.K
        d.worker_sample_offsets, d.batch_sizes = C.cast(wso, C.c_void_p), C.cast(bsz, C.c_void_p)
        d.d_row_ids, d.d_bag_offsets, d.d_pooled_out, d.d_d_pooled = p(d_ids), p(d_off), p(buf_b.pooled), p(d_dY)
        d.d_dense_grads, d.d_dense_out = p(d_dense), p(buf_b.dense_out)
        d.d_uniq_ids, d.d_worker_uniq_offsets = p(buf_b.uniq_ids), p(buf_b.worker_uniq_offsets)
        d.d_seg_offsets, d.d_sorted_occ, d.d_uniq_grads, d.uniq_cap = \
            p(buf_b.seg_offsets), p(buf_b.sorted_occ), p(buf_b.uniq_grads), buf_b.uniq_cap
        d.d_agg_ids, d.d_agg_grads, d.d_n_agg, d.agg_cap = p(buf_b.agg_ids), p(buf_b.agg_grads), p(buf_b.n_agg), buf_b.agg_cap
        d.ws, d.ws_bytes, d.d_status = p(buf_b.ws), buf_b.ws.numel(), p(buf_b.status)
        d.h_pooled, d.h_dense_out, d.h_n_agg, d.h_status = p(h_pooled), p(h_dense_out), p(h_n_agg), p(h_status)
        B.antdt_bsp_step_host(d, stream)
        stream.synchronize()                      # the caller's stream alone is waited on
        assert int(h_status[0]) == 0
        na = int(h_n_agg[0])
        assert na == len(want["agg_ids"]) == int(buf_a.n_agg.item())
        # identical kernels on identical inputs: bit-identical to the call-by-call path
        assert torch.equal(h_pooled.cuda(), buf_a.pooled[:n_bags])
        assert torch.equal(buf_b.agg_grads[:na], buf_a.agg_grads[:na])
        assert torch.equal(buf_b.agg_ids[:na], buf_a.agg_ids[:na])
        eq = lambda x, y: torch.equal(x.view(torch.int16) if x.dtype == torch.bfloat16 else x,  # noqa: E731
                                      y.view(torch.int16) if y.dtype == torch.bfloat16 else y)
        assert eq(t_b, t_a) and eq(s0_b, s0_a)
        if w.dense_n:
            assert torch.equal(h_dense_out.cuda(), buf_a.dense_out)
            G.close(h_dense_out.numpy(), want["dense"])
        # and the checker (from step 2 on the GPU table is free-running: the optimizer's
        # conditioning lets a few elements drift by up to a learning rate, see gpu_util.close_mostly)
        if s == 0:
            G.close(h_pooled.numpy(), want["pooled"])
            G.close(buf_b.agg_grads[:na].cpu().numpy(), want["agg"], rtol=3e-5, atol=2e-6)
        else:
            G.close_mostly(h_pooled.numpy(), want["pooled"], 1e-4, 1e-5, 1e-3, 2 * w.lr * w.len_hi)


def test_single_call_device_step_equals_the_four_calls():
    from paper_2404_09679_b200.step import DeviceStep
    w = synth.WORKLOADS[3].scaled(B=1024, V=50_000, dense_n=8192)
    plans = plan_steps(w, 2)
    bm = synth.BatchMaker(w, "cuda")
    table0 = bm.table()
    oc = OptConfig(B.OPTS[w.opt], w.lr, w.eps, w.beta1, w.beta2)
    t_a, t_b = table0.clone(), table0.clone()
    z = lambda: torch.zeros(w.V, w.D, device="cuda")  # noqa: E731
    s0_a, s1_a, s0_b, s1_b = z(), z(), z(), z()
    buf_a = buf_b = ds = None
    for s in range(2):
        batch = make_batch(bm, plans[s], s)
        nnz, n_bags = batch["row_ids"].numel(), batch["bag_offsets"].numel() - 1
        if buf_a is None:
            buf_a = StepBuffers(w.D, w.K, 2 * nnz, n_bags, w.dense_n)
            buf_b = StepBuffers(w.D, w.K, 2 * nnz, n_bags, w.dense_n)
            ds = DeviceStep(buf_b, t_b, s0_b, s1_b, oc, w.K)
        args = (batch["row_ids"], batch["bag_offsets"], w.F, batch["d_pooled"], batch["wso"].tolist(),
                batch["counts"].tolist(), batch["dense"])
        run_step(buf_a, t_a, s0_a, s1_a, oc, s + 1, *args)
        ds.run(s + 1, *args)
        assert B.antdt_read_status(buf_a.status) == 0 and B.antdt_read_status(buf_b.status) == 0
        na = int(buf_a.n_agg.item())
        assert int(buf_b.n_agg.item()) == na
        assert torch.equal(buf_b.pooled[:n_bags], buf_a.pooled[:n_bags])
        assert torch.equal(buf_b.agg_grads[:na], buf_a.agg_grads[:na])
        assert torch.equal(buf_b.dense_out, buf_a.dense_out)
        assert torch.equal(t_b, t_a) and torch.equal(s0_b, s0_a) and torch.equal(s1_b, s1_a)


@pytest.mark.parametrize("fuse_update", [False, True])
def test_two_host_steps_in_flight_equal_one_at_a_time(fuse_update):
    """(fuse_update: the server step in one pass, as bench.py's end-to-end leg runs it.)
    Two staging sets alternated with staging_idle: the copies of a step run under the kernels
    of the step before it.  Results (host outputs of every step, table and state at the end) must
    be bit-identical to the same steps issued one at a time."""
    from paper_2404_09679_b200.step import HostStaging, HostStep
    w = synth.WORKLOADS[4].scaled(B=4096, V=400_000)
    n_steps = 5
    plans = plan_steps(w, n_steps)
    bm = synth.BatchMaker(w, "cuda")
    table0 = bm.table()
    oc = OptConfig(B.OPTS[w.opt], w.lr, w.eps, w.beta1, w.beta2)
    batches = [make_batch(bm, plans[s], s) for s in range(n_steps)]
    pin = lambda t: None if t is None else t.cpu().pin_memory()  # noqa: E731
    host = [dict(ids=pin(b["row_ids"]), off=pin(b["bag_offsets"]), dY=pin(b["d_pooled"]),
                 dense=pin(b["dense"])) for b in batches]
    max_nnz = max(b["row_ids"].numel() for b in batches)
    max_bags = max(b["bag_offsets"].numel() - 1 for b in batches)
    stream = torch.cuda.Stream()
    results = {}
    for mode in ("serial", "overlap"):
        table = table0.clone()
        s0 = torch.zeros(w.V, w.D, device="cuda")
        buf = StepBuffers(w.D, w.K, max_nnz, max_bags, w.dense_n)
        sets = [HostStaging(w.D, w.K, max_nnz, max_bags, w.dense_n) for _ in range(2)]
        hs = HostStep(buf, table, s0, None, oc, w.K, fuse_update)
        torch.cuda.synchronize()
        outs, pending = [], None

        def collect(st, s):
            st.done.synchronize()
            assert int(st.h_status[0]) == 0
            nb = batches[s]["bag_offsets"].numel() - 1
            outs.append((int(st.h_n_agg[0]), st.h_pooled[:nb].clone()))

        for s in range(n_steps):
            b, h = batches[s], host[s]
            st = sets[s % 2]
            hs.run(st, s + 1, h["ids"], h["off"], w.F, h["dY"], b["wso"].tolist(), b["counts"].tolist(),
                   h["dense"], stream=stream, staging_idle=(mode == "overlap"))
            if mode == "serial":
                collect(st, s)
            else:
                if pending is not None:
                    collect(*pending)
                pending = (st, s)
        if pending is not None:
            collect(*pending)
        torch.cuda.synchronize()
        results[mode] = (outs, table.view(torch.int16).clone(), s0.clone())
    (o_a, t_a, s_a), (o_b, t_b, s_b) = results["serial"], results["overlap"]
    assert [n for n, _ in o_a] == [n for n, _ in o_b]
    for (_, pa), (_, pb) in zip(o_a, o_b):
        assert torch.equal(pa, pb)
    assert torch.equal(t_a, t_b) and torch.equal(s_a, s_b)


def test_device_step_forward_in_field_major_order_on_a_ragged_batch():
    """The step knows the number of fields, so its forward walks the bags field by field (a CTA
    takes one field of consecutive samples).  A sample count that fills neither the last CTA nor
    the workers evenly, bags of 1..100 ids: pooled must equal the checker's and the bag-major
    antdt_embbag_fwd's bit for bit."""
    from paper_2404_09679_b200.step import DeviceStep
    w = synth.WORKLOADS[4].scaled(B=1003, V=300_000)
    plans = plan_steps(w, 1)
    bm = synth.BatchMaker(w, "cuda")
    table = bm.table()
    batch = make_batch(bm, plans[0], 0)
    nnz, n_bags = batch["row_ids"].numel(), batch["bag_offsets"].numel() - 1
    assert n_bags == 1003 * w.F and nnz >= 8 * n_bags
    oc = OptConfig(B.OPTS[w.opt], w.lr, w.eps, w.beta1, w.beta2)
    buf = StepBuffers(w.D, w.K, nnz, n_bags, w.dense_n)
    want = OracleState(w, table).step(batch, 1)["pooled"]
    plain = torch.full((n_bags, w.D), float("nan"), device="cuda")
    B.antdt_embbag_fwd(table, batch["row_ids"], batch["bag_offsets"], plain, buf.status)
    ds = DeviceStep(buf, table.clone(), torch.zeros(w.V, w.D, device="cuda"), None, oc, w.K)
    buf.pooled.fill_(float("nan"))
    ds.run(1, batch["row_ids"], batch["bag_offsets"], w.F, batch["d_pooled"], batch["wso"].tolist(),
           batch["counts"].tolist(), batch["dense"])
    assert B.antdt_read_status(buf.status) == 0
    assert torch.equal(buf.pooled[:n_bags], plain)
    G.close(buf.pooled[:n_bags].cpu().numpy(), want)
