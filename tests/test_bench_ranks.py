"""The rank plumbing of bench.py (barrier, max and sum over ranks) with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import bench
    r, lr, w = bench.dist_setup("gloo")
    assert (r, lr, w) == (rank, rank, world)
    bench.barrier()
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)       # slowest replica sets the time
    samples = bench.sum_over_ranks(1000.0 * (rank + 1))  # every replica's samples count
    out[rank] = (ms, samples)
    bench.barrier()
    torch.distributed.destroy_process_group()


def test_two_ranks_agree_on_job_time_and_samples():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert dict(out) == {0: (15.0, 3000.0), 1: (15.0, 3000.0)}


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5 and bench.sum_over_ranks(2.0) == 2.0
    bench.barrier()


def test_reference_arm_runs_the_checker_only():
    """`bench.py --impl reference` times the CPU checker and must not map the CUDA library: it
    plans with the checker's own planner.  Run as a child process that lists what it mapped."""
    import json
    import subprocess
    code = (
        "import sys, json; sys.argv = ['bench.py', '--impl', 'reference', '--config', '1', "
        "'--steps', '1', '--warmup', '0']; sys.path.insert(0, %r); import bench; bench.main(); "
        "maps = open('/proc/self/maps').read(); "
        "print(json.dumps({'antdt': 'libantdt' in maps, 'oracle': 'liboracle' in maps}))" % ROOT)
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env,
                         timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    line, loaded = json.loads(lines[0]), json.loads(lines[1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["cores"] == 1
    assert line["cpu_baseline"]["cpu_model"] and line["cpu_baseline"]["cores_total"] >= 1
    assert loaded == {"antdt": False, "oracle": True}
    # its plan equals the library planner's (the two arms time the same batch)
    sys.path.insert(0, ROOT)
    import bench
    from paper_2404_09679_b200 import synth
    w = synth.WORKLOADS[2]
    a, b = bench.plan_all(w, 2), bench.plan_all_checker(w, 2)
    for pa, pb in zip(a, b):
        assert list(pa["batch_sizes"]) == pb["batch_sizes"] and list(pa["counts"]) == pb["counts"]
        assert [tuple(r) for r in pa["ranges"]] == pb["ranges"]
