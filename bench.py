#!/usr/bin/env python
"""Benchmark of the BSP sparse-ranking step: training samples/s per step on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]
                  [--launch auto|graph|stream]

One step = planner call + embbag_fwd + embbag_bwd_dedup + weighted_aggregate + sparse_opt_update
over one batch of seeded synthetic input.  `value` is measured with the batch resident in HBM
(plain launches through antdt_bsp_step_device; the launch-bound configurations 1 and 2 as one CUDA
graph per step through antdt_bsp_step_graph);
`e2e` goes through antdt_bsp_step_host with page-locked HOST buffers (copies inside the timed
region).  The path does not shard (one GPU holds the whole table): with N > 1 every rank runs an
independent replica and the job value is the sum of the replicas' samples over the slowest time.
Rank 0 prints one JSON line.
"""
import argparse
import ctypes as C
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

METRIC = "training samples/s per BSP step"
UNIT = "samples/s"
DEFAULT_CONFIG = 4          # largest single-GPU configuration (100M x 64 bf16 table, B = 131072)


# ------------------------------------------------------------------------------------------
# rank plumbing (torch.distributed only when launched with more than one rank)
# ------------------------------------------------------------------------------------------
def dist_setup(backend: str):
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1 and not dist.is_initialized():
        dist.init_process_group(backend=backend)
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), world


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(x: float, device="cpu") -> float:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        t = torch.tensor([x], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())
    return x


def sum_over_ranks(x: float, device="cpu") -> float:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        t = torch.tensor([x], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())
    return x


# ------------------------------------------------------------------------------------------
# clocks during the timed region
# ------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("uuid,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.uuid = str(torch.cuda.get_device_properties(device_index).uuid)
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def count(self):
        """Samples written so far."""
        try:
            with open(self.f.name) as g:
                return sum(1 for ln in g if ln.strip())
        except OSError:
            return 0

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        rows = [[c.strip() for c in ln.split(",")] for ln in self.f.read().splitlines() if ln.strip()]
        mine = [r for r in rows if len(r) >= 8 and r[0].endswith(self.uuid[-12:])] or \
               [r for r in rows if len(r) >= 8]
        sm, names = [], ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = set()
        for r in mine:
            try:
                sm.append(float(r[1]))
                out["sm_max_mhz"] = float(r[2])
            except ValueError:
                continue
            for k, nm in enumerate(names):
                if r[4 + k].lower().startswith("active"):
                    reasons.add(nm)
        if sm:
            busy = sorted(sm)[len(sm) // 4:]          # drop idle samples around the region
            out["sm_mhz"] = statistics.median(busy)
        out["reasons"] = sorted(reasons)
        out["samples"] = len(sm)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        return out


# ------------------------------------------------------------------------------------------
# workload set-up shared by both arms
# ------------------------------------------------------------------------------------------
def plan_all(w, n_steps):
    from paper_2404_09679_b200 import binding as B
    from paper_2404_09679_b200 import synth
    dds = B.Dds(w.n_samples, w.B, w.M, w.K)
    plans = []
    for s in range(n_steps):
        v = synth.speeds_for_step(w, s)
        rc, bsz, ro, rg, cnt = dds.antdt_shard_plan(v, B.RULES[w.rule], w.min_batch)
        assert rc == B.OK and sum(bsz) == w.B
        plans.append(dict(speeds=v, batch_sizes=bsz, counts=cnt, ranges=rg))
    return plans


def plan_all_checker(w, n_steps):
    """The same plans from the CPU checker's own planner: the reference arm never loads the
    CUDA library."""
    import oracle
    from paper_2404_09679_b200 import synth
    dds = oracle.Dds(w.n_samples, w.B, w.M, w.K, 0)
    plans = []
    for s in range(n_steps):
        v = synth.speeds_for_step(w, s)
        rc, bsz, ro, rg, cnt = dds.plan(v, w.rule, w.min_batch, cap=4 * w.K + 16)
        assert rc == 0 and int(bsz.sum()) == w.B
        plans.append(dict(speeds=v, batch_sizes=[int(x) for x in bsz], counts=[int(x) for x in cnt],
                          ranges=[(int(a), int(b)) for a, b in rg]))
    return plans


def host_info():
    """CPU model and core counts of the box the checker is timed on."""
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as f:
            for ln in f:
                if ln.lower().startswith("model name"):
                    model = ln.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    try:
        usable = len(os.sched_getaffinity(0))
    except (AttributeError, OSError):
        usable = os.cpu_count() or 1
    return {"cpu_model": model, "cores_total": os.cpu_count() or 1, "cores_usable": usable}


class PinnedToOneCore:
    """Pins this process to one of its allowed cores for the checker's timed leg (the checker is
    single-threaded; pinning keeps the scheduler from migrating it) and restores the mask."""

    def __enter__(self):
        self.old, self.core = None, None
        try:
            self.old = os.sched_getaffinity(0)
            self.core = sorted(self.old)[-1]
            os.sched_setaffinity(0, {self.core})
        except (AttributeError, OSError):
            self.old = None
        return self

    def __exit__(self, *exc):
        if self.old is not None:
            try:
                os.sched_setaffinity(0, self.old)
            except OSError:
                pass
        return False


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) come from ncu captures
# summarised in profiles/dram_traffic.json, which records for every kernel the hash of the source
# files it was compiled from: a kernel whose sources have changed since reports no traffic.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.json")
CSRC = os.path.join(ROOT, "paper_2404_09679_b200", "csrc")


def sources_hash(files):
    import hashlib
    h = hashlib.sha256()
    for f in sorted(files):
        try:
            with open(os.path.join(CSRC, f), "rb") as g:
                h.update(g.read())
        except OSError:
            h.update(b"missing:" + f.encode())
    return h.hexdigest()[:16]


def load_traffic(cfg):
    """-> {kernel: bytes per launch} for this config, only kernels whose sources are unchanged."""
    try:
        rec = json.load(open(TRAFFIC_FILE))
    except (OSError, ValueError):
        return {}, None
    out = {}
    for name, k in rec.get("configs", {}).get(str(cfg), {}).items():
        if sources_hash(k.get("sources", [])) == k.get("sources_sha"):
            out[name] = float(k["dram_bytes_per_launch"])
    return out, rec.get("commit")


def scaled_workload(w, scale):
    if scale == 1.0:
        return w
    B_ = max(w.K * max(w.min_batch, 1), int(w.B * scale) // w.K * w.K)
    V = max(w.F, int(w.V * scale) // w.F * w.F)
    return w.scaled(B=B_, V=V, dense_n=int(w.dense_n * scale) // 4 * 4,
                    name=f"{w.name} scaled x{scale:g}")


def algorithmic_bytes(w, nnz, n_bags, sum_u, u):
    """Bytes each kernel of the step has to move per launch (per step for the radix kernels'
    sum), from the counts of the batch: the gathers at full multiplicity, every output once."""
    D, ew = w.D, (2 if w.table_dtype == "bf16" else 4)
    S = 2 if w.opt == "adam" else 1
    return {
        "radix_hist": 4 * nnz, "radix_scatter": 16 * nnz, "runs_count": 4 * nnz,
        "runs_emit": 4 * nnz + nnz // 8 + 12 * sum_u,
        "agg_radix_hist": 4 * sum_u, "agg_radix_scatter": 16 * sum_u, "agg_runs_count": 4 * sum_u,
        "agg_runs_emit": 4 * sum_u + sum_u // 8 + 12 * u,
        # range-partitioned merge (up to 32 workers): ids read by both passes; merge order, head
        # bits and the distinct ids written once
        "agg_range_count": 4 * sum_u, "agg_range_emit": 8 * sum_u + sum_u // 8 + 4 * u,
        "embbag_fwd": 4 * nnz + 8 * (n_bags + 1) + nnz * D * ew + n_bags * D * 4,
        "expand_bags": 8 * (n_bags + 1) + 4 * nnz,
        "seg_reduce_tiles": 4 * nnz + nnz // 8 + nnz * D * 4 + sum_u * D * 4,
        "agg_reduce": sum_u * (4 * D + 4) + u * (4 * D + 8),
        # one pass: contributions in, table and state in and out; no aggregated gradient in between
        "agg_update": sum_u * (4 * D + 4) + u * 8 + 2 * u * D * ew + 2 * S * u * D * 4,
        "sparse_adagrad": u * (4 + 4 * D) + 2 * u * D * ew + 2 * S * u * D * 4,
        "sparse_adam": u * (4 + 4 * D) + 2 * u * D * ew + 2 * S * u * D * 4,
        "dense_wsum": (w.K + 1) * w.dense_n * 4,
    }


def step_bytes(w, nnz, n_bags, sum_u, u, passes_bwd, passes_agg, fused=False):
    b = algorithmic_bytes(w, nnz, n_bags, sum_u, u)
    upd = b["sparse_adam"] if w.opt == "adam" else b["sparse_adagrad"]
    if fused and w.K <= 32:   # the one-pass server step: no aggregated gradient in between
        upd = b["agg_update"] - b["agg_reduce"]
    sort = passes_bwd * (b["radix_hist"] + b["radix_scatter"]) + b["runs_count"] + b["runs_emit"]
    if w.K <= 32:       # the aggregation's merge order comes from the range pass, not a sort
        sort += b["agg_range_count"] + b["agg_range_emit"]
    else:
        sort += (passes_agg * (b["agg_radix_hist"] + b["agg_radix_scatter"]) + b["agg_runs_count"] +
                 b["agg_runs_emit"])
    return (b["embbag_fwd"] + b["expand_bags"] + b["seg_reduce_tiles"] + b["agg_reduce"] + upd +
            (b["dense_wsum"] if w.dense_n else 0) + sort)


# ------------------------------------------------------------------------------------------
# CPU baseline: the checker, as it stands, on a bounded sample of the workload
# ------------------------------------------------------------------------------------------
class OracleSample:
    """First `per_worker` samples of every worker of one batch, on a compact copy of the rows
    they touch (ids renumbered in order, so every id comparison is preserved)."""

    def __init__(self, w, bm, plan, table, per_worker):
        from paper_2404_09679_b200 import synth
        idx_parts, counts = [], []
        ranges = list(plan["ranges"])
        # walk the plan's ranges worker by worker
        pos = 0
        for i, c in enumerate(plan["counts"]):
            take, got = min(per_worker, c), []
            left = c
            while left > 0:
                s, n = ranges[pos]
                pos += 1
                left -= n
                if take > 0:
                    k = min(take, n)
                    got.append((s, k))
                    take -= k
            idx_parts += got
            counts.append(sum(n for _, n in got))
        idx = synth.sample_indices(idx_parts, bm.device)
        ids, off = bm.bags(idx)
        dY = bm.d_pooled(idx)
        rows = torch.unique(ids.to(torch.int64))          # ascending
        self.ids = torch.searchsorted(rows, ids.to(torch.int64)).to(torch.int32).cpu().numpy()
        self.off = off.cpu().numpy()
        self.dY = dY.cpu().numpy()
        t = table[rows.to(table.device)]
        self.table = (t.view(torch.int16).cpu().numpy().view(np.uint16).copy()
                      if t.dtype == torch.bfloat16 else t.cpu().numpy().copy())
        self.s0 = np.zeros(self.table.shape, np.float32)
        self.s1 = np.zeros(self.table.shape, np.float32) if w.opt == "adam" else None
        self.counts = np.asarray(counts, np.int64)
        self.wso = np.concatenate([[0], np.cumsum(self.counts)]).astype(np.int64)
        dn = min(w.dense_n, 1 << 18)                    # dense part sampled in proportion
        self.dense_frac = dn / w.dense_n if w.dense_n else 0.0
        self.dense = None
        if w.dense_n:
            e = torch.arange(dn, dtype=torch.int64, device=bm.device)
            g = [synth.normal01(synth.hash_coords(w.seed, synth.TAG_DENSE, 0, i, e)) * w.dense_std
                 for i in range(w.K)]
            self.dense = torch.stack(g).to(torch.float32).cpu().numpy()
        self.w = w
        self.n_samples = int(self.counts.sum())

    def run(self, step):
        import oracle
        w = self.w
        t0 = time.perf_counter()
        oracle.embbag_fwd(self.table, self.ids, self.off)
        b = oracle.embbag_bwd_dedup(self.ids, self.off, w.F, self.dY, self.table.shape[0], self.wso)
        ai, ag = oracle.aggregate_sparse(b["uniq_ids"], b["worker_uniq_offsets"], b["uniq_grads"],
                                         self.counts)
        if self.dense is not None:
            oracle.aggregate_dense(self.dense, self.counts)
        oracle.sparse_opt_update(self.table, ai, ag, w.opt, w.lr, w.eps, w.beta1, w.beta2, step,
                                 self.s0, self.s1)
        return time.perf_counter() - t0


# samples per worker in the bounded sample: about 15 s of checker time for the baseline leg of
# our arm, about 5 s per step for the reference arm (which runs warmup + steps of them)
CPU_SAMPLE_PER_WORKER = {1: 1 << 30, 2: 1 << 30, 3: 1536, 4: 2048, 5: 8192}
REF_SAMPLE_PER_WORKER = {1: 1 << 30, 2: 1 << 30, 3: 256, 4: 256, 5: 1536}


def cpu_baseline(w, cfg, bm, plan, table):
    repeats = 5 if cfg <= 2 else 1
    smp = OracleSample(w, bm, plan, table, CPU_SAMPLE_PER_WORKER[cfg])
    with PinnedToOneCore() as pin:
        ts = [smp.run(s + 1) for s in range(repeats)]
    t = statistics.median(ts)
    return {"value": smp.n_samples / t, "unit": UNIT, "cores": 1, "kind": "oracle",
            "pinned_to_core": pin.core, **host_info(),
            "sample": f"first {min(CPU_SAMPLE_PER_WORKER[cfg], max(plan['counts']))} samples of each "
                      f"of the {w.K} workers of one batch ({smp.n_samples} samples, "
                      f"{len(smp.ids)} occurrences, touched rows only"
                      + (f", dense vector cut to {smp.dense.shape[1]} elements" if w.dense_n else "")
                      + f"), {repeats} step(s), {t:.2f} s per step"}, smp


# ------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------
def run_ours(args):
    from paper_2404_09679_b200 import binding as B
    from paper_2404_09679_b200 import synth
    from paper_2404_09679_b200.step import DeviceStep, OptConfig, StepBuffers

    rank, local_rank, world = dist_setup("nccl")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    B.lib()
    cfg = args.config
    w = scaled_workload(synth.WORKLOADS[cfg], args.scale)
    if world > 1:
        w = w.scaled(seed=w.seed + 1000 * rank)           # independent replicas
    W, K_steps = args.warmup, args.steps
    # the one-pass server step measures faster on all five configs; it needs at most 32 workers
    args.fuse_update = args.fuse_update or (w.K <= 32 and not args.no_fuse_update)
    n_batches = min(3, W + K_steps)
    plans = plan_all(w, max(n_batches, 1))
    bm = synth.BatchMaker(w, dev)
    table = bm.table()
    state0 = torch.zeros(w.V, w.D, dtype=torch.float32, device=dev)
    state1 = torch.zeros(w.V, w.D, dtype=torch.float32, device=dev) if w.opt == "adam" else None
    oc = OptConfig(B.OPTS[w.opt], w.lr, w.eps, w.beta1, w.beta2)

    batches = []
    for j in range(n_batches):
        idx = synth.sample_indices(plans[j]["ranges"], dev)
        ids, off = bm.bags(idx)
        batches.append(dict(ids=ids, off=off, dY=bm.d_pooled(idx), dense=bm.dense_grads(j),
                            wso=[0] + list(np.cumsum(plans[j]["counts"])),
                            counts=list(plans[j]["counts"])))
        del idx
    max_nnz = max(b["ids"].numel() for b in batches)
    max_bags = max(b["off"].numel() - 1 for b in batches)

    # CPU baseline first (rank 0, N = 1 only): it needs the initial table rows
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu, _ = cpu_baseline(w, cfg, bm, plans[0], table)

    # sizing pass: count the (worker, row) pairs of every batch with capacity 0
    ws0 = torch.empty(B.antdt_embbag_bwd_dedup_workspace_bytes(max_nnz, max_bags, w.D, w.K),
                      dtype=torch.uint8, device=dev)
    wuo = torch.zeros(w.K + 1, dtype=torch.int64, device=dev)
    so = torch.zeros(1, dtype=torch.int64, device=dev)
    occ = torch.empty(max_nnz, dtype=torch.int32, device=dev)
    dummy = torch.empty(0, w.D, dtype=torch.float32, device=dev)
    sum_us = []
    for b in batches:
        B.antdt_embbag_bwd_dedup(b["ids"], b["off"], w.F, b["dY"], w.V, b["wso"],
                                 torch.empty(0, dtype=torch.int32, device=dev), wuo, so,
                                 occ[: b["ids"].numel()], dummy, ws0, None)
        sum_us.append(int(wuo[w.K].item()))
    del ws0, occ
    cap = int(max(sum_us) * 1.05) + 1024
    buf = StepBuffers(w.D, w.K, max_nnz, max_bags, w.dense_n, uniq_cap=cap, agg_cap=cap, device=dev)

    dds = B.Dds(w.n_samples, w.B, w.M, w.K)                # the live planner of the timed loop
    # the device calls behind one C call; --fuse-update: aggregate and update in one pass
    dstep = DeviceStep(buf, table, state0, state1, oc, w.K, fuse_update=args.fuse_update)

    # Launch form of the timed steps.  A step is 30-40 launches; on the small configurations
    # they, not the kernels, are the step time, so there the step is replayed as one CUDA graph.
    # (auto: wherever the entry point can replay a graph, i.e. not for Adam, whose step number
    # changes kernel parameters every step; on the large configurations it saves the launch gaps.)
    use_graph = args.launch == "graph" or (args.launch == "auto" and w.opt != "adam")

    def one_step(s, graph=use_graph):
        b = batches[s % n_batches]
        v = synth.speeds_for_step(w, s)
        rc, bsz, _, _, cnt = dds.antdt_shard_plan(v, B.RULES[w.rule], w.min_batch)
        if s < len(plans):
            assert rc == B.OK and cnt == plans[s]["counts"]
        dstep.run(s + 1, b["ids"], b["off"], w.F, b["dY"], b["wso"], b["counts"], b["dense"],
                  graph=graph)

    # torch's default stream is the legacy stream, which cannot be captured
    torch.cuda.synchronize()
    stream = torch.cuda.Stream() if use_graph else torch.cuda.current_stream()
    torch.cuda.set_stream(stream)
    # the sampler runs from before the warm-up to after the timed region: a timed region of a few
    # milliseconds (small configurations) would otherwise fall between two samples
    clocks = ClockSampler(local_rank)
    clocks.start()
    for s in range(W):
        one_step(s)
    # nvidia-smi takes a moment to deliver its first sample: keep stepping (untimed) until it has,
    # so that the clocks are seen under this load even when the timed region lasts milliseconds
    extra, t_wait = 0, time.time()
    while clocks.p is not None and clocks.count() < 2 and time.time() - t_wait < 3.0:
        one_step(W + extra)
        extra += 1
        if extra % 8 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    assert B.antdt_read_status(buf.status) == 0, "device status after warm-up"
    u_seen = int(buf.n_agg.item())
    sum_u_seen = int(buf.worker_uniq_offsets[w.K].item())

    barrier()
    torch.cuda.synchronize()
    # the timed steps carry no per-kernel events (an event pair around each of a step's 22 launches
    # costs about 0.15 ms per step on the large configurations)
    launches0 = B.antdt_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for s in range(W, W + K_steps):
        one_step(s)
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    ms_local = e0.elapsed_time(e1)
    launches = B.antdt_launch_count() - launches0
    # the per-kernel times come from the same K steps issued once more as plain launches with an
    # event pair around every launch (the DDS handle keeps advancing: same shapes)
    B.antdt_profile_enable(True)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record(stream)
    for s in range(W + K_steps, W + 2 * K_steps):
        one_step(s, graph=False)
    p1.record(stream)
    torch.cuda.synchronize()
    prof_ms = p0.elapsed_time(p1)
    prof = B.antdt_profile_get()
    B.antdt_profile_enable(False)
    clk = clocks.stop()
    assert B.antdt_read_status(buf.status) == 0, "device status after the timed region"
    samples_local = sum(sum(batches[s % n_batches]["counts"]) for s in range(W, W + K_steps))
    ms = max_over_ranks(ms_local, dev)
    samples = sum_over_ranks(float(samples_local), dev)

    # ---- end to end through antdt_bsp_step_host, page-locked host buffers ---------------------
    if args.no_e2e:
        e2e = {"ms": float("nan"), "samples": 0, "h2d": 0, "d2h": 0}
    else:
        e2e = run_e2e(B, w, batches, buf, table, state0, state1, oc, W, K_steps, dev, stream,
                      args.fuse_update)
    e2e_ms = max_over_ranks(e2e["ms"], dev)
    e2e_samples = sum_over_ranks(float(e2e["samples"]), dev)

    if rank != 0:
        return
    # ---- roofline of the dominant kernel ---------------------------------------------------------
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except (OSError, ValueError):
        pass
    peak_gbs = float(peaks.get("hbm_gbs", 6650.0))
    nnz_avg = sum(b["ids"].numel() for b in batches) / n_batches
    bags_avg = sum(b["off"].numel() - 1 for b in batches) / n_batches
    alg = algorithmic_bytes(w, int(nnz_avg), int(bags_avg), sum_u_seen, u_seen)
    traffic, traffic_commit = load_traffic(cfg) if (args.scale == 1.0 and world == 1) else ({}, None)
    D, ew = w.D, (2 if w.table_dtype == "bf16" else 4)
    # the two gathering kernels: bytes their gathers pull (at full multiplicity) and what a perfect
    # cache would leave for DRAM (every distinct input row once + ids + outputs)
    gathers = {"embbag_fwd": (nnz_avg * D * ew, D * ew,
                              4 * nnz_avg + 8 * (bags_avg + 1) + u_seen * D * ew + bags_avg * D * 4),
               "seg_reduce_tiles": (nnz_avg * D * 4, D * 4,
                                    4 * nnz_avg + nnz_avg / 8 + bags_avg * D * 4 + sum_u_seen * D * 4)}
    kern = {}
    step_dram, step_dram_missing = 0.0, []
    for name, (n, tms) in prof.items():
        d = {"launches": n, "ms_total": round(tms, 4), "share": round(tms / max(prof_ms, 1e-9), 4)}
        if name in alg and n:
            d["algorithmic_GBps"] = round(alg[name] / (tms / n * 1e-3) / 1e9, 1)
        if name in traffic and n:
            d["dram_GBps"] = round(traffic[name] / (tms / n * 1e-3) / 1e9, 1)
            d["dram_frac"] = round(d["dram_GBps"] / peak_gbs, 4)
            step_dram += traffic[name] * n / K_steps
        elif tms / max(prof_ms, 1e-9) > 0.005:
            step_dram_missing.append(name)
        kern[name] = d
    top = max(prof.items(), key=lambda kv: kv[1][1])[0]
    top_n, top_ms = prof[top]
    top_s = top_ms / top_n * 1e-3
    roof = {"kernel": top, "bound": "hbm", "unit": "GB/s", "peak": peak_gbs,
            "peak_source": "MEASURED_PEAKS.json hbm_gbs (measured copy)" if peaks else "fallback 6650",
            "achieved": None, "frac": None, "traffic": traffic.get(top),
            "algorithmic_bytes_per_launch": alg.get(top), "avg_launch_ms": round(top_ms / top_n, 4)}
    if top in alg:
        roof["achieved_algorithmic"] = round(alg[top] / top_s / 1e9, 1)
        roof["frac_algorithmic"] = round(roof["achieved_algorithmic"] / peak_gbs, 4)
    if top in gathers:
        roof["compulsory_bytes_per_launch"] = int(gathers[top][2])
        roof["frac_compulsory"] = round(gathers[top][2] / top_s / 1e9 / peak_gbs, 4)
    # `frac` is what DRAM did: measured DRAM bytes where a capture of this kernel exists; else, for
    # a gathering kernel (whose repeats are served by L1/L2, so its algorithmic rate is not a DRAM
    # rate), the compulsory bytes; else the algorithmic bytes (streaming kernels: the same thing)
    if roof["traffic"]:
        roof["achieved"] = round(roof["traffic"] / top_s / 1e9, 1)
        roof["frac_source"] = (f"ncu dram bytes per launch (profiles/dram_traffic.json, commit "
                               f"{traffic_commit}) / CUDA-event launch time")
    elif top in gathers:
        roof["achieved"] = round(gathers[top][2] / top_s / 1e9, 1)
        roof["frac_source"] = ("compulsory bytes (every distinct input row once, ids, outputs): a lower "
                               "bound of the DRAM traffic; no current ncu capture of this kernel here")
    elif top in alg:
        roof["achieved"] = roof["achieved_algorithmic"]
        roof["frac_source"] = "algorithmic bytes (a streaming kernel: every byte is touched once)"
    if roof["achieved"] is not None:
        roof["frac"] = round(roof["achieved"] / peak_gbs, 4)
    # secondary roof of the gathering kernels: the rate at which the SMs pull scattered rows of the
    # same width out of an L2-resident matrix (measured here with the library's plain probe)
    l2 = None
    if not args.no_l2_probe:
        l2 = {}
        for name, (gbytes, row_bytes, _) in gathers.items():
            if name not in prof or not prof[name][0]:
                continue
            rate = measure_l2_gather(B, dev, row_bytes, stream)
            n, tms = prof[name]
            ach = gbytes / (tms / n * 1e-3) / 1e9
            l2[name] = {"row_bytes": row_bytes, "l2_gather_peak_GBps": round(rate, 1),
                        "gathered_GBps": round(ach, 1), "frac_of_l2_gather_peak": round(ach / rate, 4)}
            kern[name]["frac_of_l2_gather_peak"] = l2[name]["frac_of_l2_gather_peak"]
        roof["l2_gather"] = l2.get(top)
    rowbits = max(1, (w.V - 1).bit_length())
    passes = -(-rowbits // 9)
    sb = step_bytes(w, int(nnz_avg), int(bags_avg), sum_u_seen, u_seen, passes, passes, args.fuse_update)
    line = {
        "metric": METRIC, "value": samples / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": K_steps, "warmup": W, "ms_per_step": ms / K_steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"configs[{cfg - 1}] {w.name}: K={w.K} workers, B={w.B}, F={w.F}, "
                               f"V={w.V} x D={w.D} {w.table_dtype}, {w.opt}",
                   "nnz_per_step": int(nnz_avg), "bags_per_step": int(bags_avg),
                   "uniq_worker_rows": sum_u_seen, "uniq_rows": u_seen,
                   "l2": "no flush: per-step working set (table + state + batch) is far above the "
                         "126 MB L2", "batches_rotated": n_batches,
                   "launch": ("one CUDA graph per step (antdt_bsp_step_graph)" if use_graph
                              else "plain launches (antdt_bsp_step_device)"),
                   "server_step": ("one pass (antdt_aggregate_update)" if args.fuse_update
                                   else "aggregate, then update"),
                   "parallelism": "replicas" if world > 1 else "single"},
        "clocks": {"sm_mhz": clk["sm_mhz"], "sm_max_mhz": clk["sm_max_mhz"], "reasons": clk["reasons"],
                   "samples": clk["samples"], "extra_warmup_steps": extra},
        "e2e": None if args.no_e2e else {
            "value": e2e_samples / (e2e_ms * 1e-3), "unit": UNIT,
            "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
            "ms_per_step": e2e_ms / K_steps,
            "h2d_GBps": round(e2e["h2d"] / (e2e_ms / K_steps * 1e-3) / 1e9, 2),
            "link": e2e.get("link"),
            "frac_of_link": (round(e2e["h2d"] / (e2e_ms / K_steps * 1e-3) / 1e9 /
                                   e2e["link"]["h2d_beside_d2h_GBps"], 4) if e2e.get("link") else None),
            "how": "antdt_bsp_step_host, two staging sets alternated: the copies of step s+1 run "
                   "under the kernels of step s; the host reads every step's results"},
        "gpu_launches": launches,
        "roofline": roof,
        "step_algorithmic_GB": round(sb / 1e9, 3),
        "step_GBps_algorithmic": round(sb / (ms / K_steps * 1e-3) / 1e9, 1),
        "step_dram_GB": round(step_dram / 1e9, 3) if traffic else None,
        "step_frac_dram": (round(step_dram / (ms / K_steps * 1e-3) / 1e9 / peak_gbs, 4)
                           if traffic else None),
        "step_dram_kernels_without_capture": step_dram_missing if traffic else None,
        "l2_gather": l2,
        "kernels": kern,
        "kernels_timed_in": (f"the same {K_steps} steps issued again as plain launches with an event pair "
                             f"around every launch, {prof_ms / K_steps:.4f} ms per step there"),
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)


def measure_l2_gather(B, dev, row_bytes, stream, _cache={}):
    """GB/s at which antdt_probe_gather pulls uniformly random rows of `row_bytes` out of a 32 MB
    matrix (L2 resident after the first touch); best of 5 launches of about 4 GB each."""
    if row_bytes in _cache:
        return _cache[row_bytes]
    dim = row_bytes // 4
    if dim not in (16, 32, 64, 128):
        dim = 64
    n_rows = (32 << 20) // (dim * 4)
    per_out, n_out = 32, (1 << 24) // 32 * (64 // min(dim, 64))
    g = torch.Generator(device=dev)
    g.manual_seed(12345)
    rows = torch.randn(n_rows, dim, device=dev, generator=g)
    idx = torch.randint(0, n_rows, (n_out * per_out,), device=dev, generator=g, dtype=torch.int32)
    out = torch.empty(n_out, dim, device=dev)
    best = float("inf")
    for i in range(8):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        B.antdt_probe_gather(rows, idx, per_out, out, stream=stream)
        e1.record(stream)
        e1.synchronize()
        if i >= 3:
            best = min(best, e0.elapsed_time(e1))
    _cache[row_bytes] = n_out * per_out * dim * 4 / (best * 1e-3) / 1e9
    del rows, idx, out
    return _cache[row_bytes]


def run_e2e(B, w, batches, buf, table, state0, state1, oc, W, K_steps, dev, stream, fuse_update=False):
    """K steps through antdt_bsp_step_host; every step copies its inputs from page-locked host
    memory and its results back, and the host reads every step's results.  Two staging sets are
    alternated so that the copies of step s+1 run under the kernels of step s; the host reads step
    s's results while step s+1 is in flight."""
    from paper_2404_09679_b200.step import HostStaging, HostStep

    def pin(t):
        return None if t is None else t.cpu().pin_memory()

    host = [dict(ids=pin(b["ids"]), off=pin(b["off"]), dY=pin(b["dY"]), dense=pin(b["dense"]))
            for b in batches]
    max_nnz = max(b["ids"].numel() for b in batches)
    max_bags = max(b["off"].numel() - 1 for b in batches)
    sets = [HostStaging(w.D, w.K, max_nnz, max_bags, w.dense_n, dev) for _ in range(2)]
    hs = HostStep(buf, table, state0, state1, oc, w.K, fuse_update)
    n_b = len(batches)

    def issue(s, step, idle):
        j = s % n_b
        b, h, st = batches[j], host[j], sets[s % 2]
        hs.run(st, step, h["ids"], h["off"], w.F, h["dY"], b["wso"], b["counts"], h["dense"],
               stream=stream, staging_idle=idle)
        return st

    def collect(st):
        st.done.synchronize()                             # the caller reads the step's results
        assert int(st.h_status[0]) == 0 and int(st.h_n_agg[0]) > 0

    step0 = 10_000
    for s in range(min(W, 3)):
        collect(issue(s, step0 + s, False))
    barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    samples, pending = 0, None
    for s in range(K_steps):
        st = issue(s, step0 + 3 + s, True)                # its set was collected two steps ago
        if pending is not None:
            collect(pending)
        pending = st
        samples += sum(batches[s % n_b]["counts"])
    collect(pending)
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    b = batches[0]
    h2d = (b["ids"].numel() * 4 + b["off"].numel() * 8 + b["dY"].numel() * 4 +
           (b["dense"].numel() * 4 if b["dense"] is not None else 0))
    d2h = (b["off"].numel() - 1) * w.D * 4 + w.dense_n * 4 + 12
    return {"ms": e0.elapsed_time(e1), "samples": samples, "h2d": h2d, "d2h": d2h,
            "link": measure_link(host[0]["dY"], sets[0], stream)}


def measure_link(h_src, st, stream):
    """The host link the end-to-end step rides on: the largest input copied host-to-device alone,
    then with the largest result going device-to-host at the same time (as in a step).  Plain
    cudaMemcpyAsync through torch, page-locked on the host side; GB/s of the host-to-device copy."""
    n = min(h_src.numel(), st.d_d_pooled.numel(), st.h_pooled.numel())
    if n * 4 < (1 << 20):
        return None
    src, dst = h_src.reshape(-1)[:n], st.d_d_pooled.reshape(-1)[:n]
    back_src, back_dst = st.d_pooled_out.reshape(-1)[:n], st.h_pooled.reshape(-1)[:n]
    side = torch.cuda.Stream()
    out = {}
    for name, both in (("h2d_alone_GBps", False), ("h2d_beside_d2h_GBps", True)):
        best = 0.0
        for _ in range(3):
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if both:
                with torch.cuda.stream(side):
                    back_dst.copy_(back_src, non_blocking=True)
                    back_dst.copy_(back_src, non_blocking=True)   # still running when the other ends
            with torch.cuda.stream(stream):
                e0.record(stream)
                dst.copy_(src, non_blocking=True)
                e1.record(stream)
            torch.cuda.synchronize()
            best = max(best, n * 4 / (e0.elapsed_time(e1) * 1e-3) / 1e9)
        out[name] = round(best, 2)
    return out


# ------------------------------------------------------------------------------------------
# reference arm: the CPU checker timed on the host cores
# ------------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2404_09679_b200 import synth
    cfg = args.config
    w = scaled_workload(synth.WORKLOADS[cfg], args.scale)
    dev = torch.device("cuda", 0) if torch.cuda.is_available() else torch.device("cpu")
    plans = plan_all_checker(w, 1)
    bm = synth.BatchMaker(w, dev)

    class _LazyTable:                     # rows of the initial table, produced on demand
        device = dev
        dtype = torch.float32 if w.table_dtype == "f32" else torch.bfloat16

        def __getitem__(self, rows):
            c = torch.arange(w.D, dtype=torch.int64, device=dev)
            h = synth.hash_coords(w.seed, synth.TAG_TABLE, rows[:, None], c[None, :])
            return (w.init_std * synth.normal01(h)).to(torch.float32).to(self.dtype)

    smp = OracleSample(w, bm, plans[0], _LazyTable(), REF_SAMPLE_PER_WORKER[cfg])
    with PinnedToOneCore() as pin:
        for s in range(args.warmup):
            smp.run(s + 1)
        t0 = time.perf_counter()
        for s in range(args.steps):
            smp.run(args.warmup + s + 1)
        dt = time.perf_counter() - t0
    value = smp.n_samples * args.steps / dt
    sample = (f"each step = first {min(REF_SAMPLE_PER_WORKER[cfg], max(plans[0]['counts']))} samples of "
              f"each of the {w.K} workers of one batch ({smp.n_samples} samples, {len(smp.ids)} "
              f"occurrences, touched rows only)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": f"configs[{cfg - 1}] {w.name}: K={w.K} workers, B={w.B}, F={w.F}, "
                               f"V={w.V} x D={w.D} {w.table_dtype}, {w.opt}", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "pinned_to_core": pin.core, **host_info()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=DEFAULT_CONFIG, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--launch", default="auto", choices=["auto", "graph", "stream"],
                    help="timed steps as one CUDA graph each or as plain launches (auto: graph "
                         "except for Adam, which the graph entry point issues as plain launches)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--fuse-update", action="store_true",
                    help="server step through antdt_aggregate_update (aggregated gradients not "
                         "materialised); the default")
    ap.add_argument("--no-fuse-update", action="store_true",
                    help="server step as antdt_weighted_aggregate + antdt_sparse_opt_update on every config")
    ap.add_argument("--no-l2-probe", action="store_true",
                    help="skip the L2 gather-rate probe (profiling runs)")
    ap.add_argument("--scale", type=float, default=1.0,
                    help="shrink batch, table rows and dense vector by this factor (profiling "
                         "captures on a small case); the JSON line says so")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
