"""Times single C-ABI calls that the five benchmark configurations do not reach, on synthetic
inputs of a given size, with CUDA events:

  python -m paper_2404_09679_b200.kernel_bench --case dense_adam --n 33554432
  python -m paper_2404_09679_b200.kernel_bench --case aggregate_k33 --rows 4000000 --dim 32

cases: dense_adagrad, dense_adam            antdt_dense_opt_update on an n-element vector
       rowwise_adagrad, rowwise_adagrad_bf16 antdt_sparse_opt_update, one accumulator per row
       aggregate_k33                         antdt_weighted_aggregate with 33 workers (the
                                             sort-based merge used beyond 32 workers)
       aggregate_backup                      antdt_weighted_aggregate_backup, 16 workers, 2 dropped
       fused_adagrad_bf16, fused_adam        antdt_aggregate_update, 16 workers
Prints one JSON line: the case, its sizes, milliseconds per call and the per-kernel times the
library recorded.  Marshalling only; every kernel is the library's.
"""
import argparse
import json

import torch

from . import binding as B


def _timed(fn, reps, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    B.antdt_profile_enable(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    prof = B.antdt_profile_get()
    B.antdt_profile_enable(False)
    return e0.elapsed_time(e1) / reps, {k: round(ms / max(n, 1), 4) for k, (n, ms) in prof.items()}


def _worker_lists(K, V, per_worker, gen):
    """K ascending id lists (distinct ids inside a list) and their offsets."""
    ids, wuo = [], [0]
    for _ in range(K):
        mine = torch.unique(torch.randint(0, V, (per_worker,), device="cuda", generator=gen))
        ids.append(mine.to(torch.int32))
        wuo.append(wuo[-1] + mine.numel())
    return torch.cat(ids), torch.tensor(wuo, dtype=torch.int64, device="cuda")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", required=True)
    ap.add_argument("--n", type=int, default=1 << 25, help="elements of the dense vector")
    ap.add_argument("--rows", type=int, default=2_000_000, help="ids per call / per worker list")
    ap.add_argument("--table-rows", type=int, default=20_000_000)
    ap.add_argument("--dim", type=int, default=64)
    ap.add_argument("--reps", type=int, default=5)
    a = ap.parse_args()
    assert torch.cuda.is_available(), "needs a CUDA device"
    B.lib()
    gen = torch.Generator(device="cuda")
    gen.manual_seed(7)
    f32 = torch.float32
    info = {"case": a.case}
    if a.case in ("dense_adagrad", "dense_adam"):
        n = a.n // 4 * 4
        p, g = torch.randn(n, device="cuda", generator=gen), torch.randn(n, device="cuda", generator=gen)
        s0 = torch.zeros(n, device="cuda")
        s1 = torch.zeros(n, device="cuda") if a.case == "dense_adam" else None
        opt = B.OPT_ADAM if s1 is not None else B.OPT_ADAGRAD
        step = [0]

        def fn():
            step[0] += 1
            B.antdt_dense_opt_update(p, g, opt, 1e-3, 1e-8, 0.9, 0.999, step[0], s0, s1)
        info.update(n=n, bytes=n * 4 * (7 if s1 is not None else 5))
    elif a.case in ("rowwise_adagrad", "rowwise_adagrad_bf16"):
        V, D = a.table_rows, a.dim
        dt = torch.bfloat16 if a.case.endswith("bf16") else f32
        table = (0.01 * torch.randn(V, D, device="cuda", generator=gen)).to(dt)
        ids = torch.unique(torch.randint(0, V, (a.rows,), device="cuda", generator=gen)).to(torch.int32)
        g = torch.randn(ids.numel(), D, device="cuda", generator=gen)
        s0 = torch.zeros(V, device="cuda")
        n_ids = torch.tensor([ids.numel()], dtype=torch.int64, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")

        def fn():
            B.antdt_sparse_opt_update(table, ids, g, n_ids, B.OPT_ROWWISE_ADAGRAD, 0.01, 1e-8, 0, 0, 1, s0,
                                      None, st)
        u = ids.numel()
        info.update(rows=u, dim=D, bytes=u * (4 + 4 * D + 8) + 2 * u * D * table.element_size())
    elif a.case in ("aggregate_k33", "aggregate_backup", "fused_adagrad_bf16", "fused_adam"):
        K = 33 if a.case == "aggregate_k33" else 16
        V, D = a.table_rows, a.dim
        uid, wuo = _worker_lists(K, V, a.rows // K, gen)
        n_in = uid.numel()
        g = torch.randn(n_in, D, device="cuda", generator=gen)
        agg_ids = torch.empty(n_in, dtype=torch.int32, device="cuda")
        agg = torch.empty(n_in, D, device="cuda")
        n_agg = torch.zeros(1, dtype=torch.int64, device="cuda")
        ws = torch.empty(B.antdt_weighted_aggregate_workspace_bytes(n_in, D, K), dtype=torch.uint8,
                         device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        bsz = [100 + 3 * i for i in range(K)]
        if a.case.startswith("fused"):
            adam = a.case == "fused_adam"
            table = (0.01 * torch.randn(V, D, device="cuda", generator=gen)).to(f32 if adam else torch.bfloat16)
            s0 = torch.zeros(V, D, device="cuda")
            s1 = torch.zeros(V, D, device="cuda") if adam else None
            step = [0]

            def fn():
                step[0] += 1
                B.antdt_aggregate_update(bsz, ws, table, B.OPT_ADAM if adam else B.OPT_ADAGRAD, 1e-3, 1e-8,
                                         0.9, 0.999, step[0], s0, s1, uniq_ids=uid, worker_uniq_offsets=wuo,
                                         uniq_grads=g, agg_ids=agg_ids, n_agg=n_agg, dev_status=st)
        else:
            dropped = [i in (3, 11) for i in range(K)] if a.case == "aggregate_backup" else None

            def fn():
                B.antdt_weighted_aggregate(bsz, ws, n_rows=V, uniq_ids=uid, worker_uniq_offsets=wuo,
                                           uniq_grads=g, agg_ids=agg_ids, agg_grads=agg, n_agg=n_agg,
                                           dev_status=st, dropped=dropped)
        info.update(workers=K, entries=n_in, dim=D)
    else:
        raise SystemExit(f"unknown case {a.case}")
    ms, kernels = _timed(fn, a.reps)
    info.update(ms_per_call=round(ms, 4), kernels_ms_per_launch=kernels)
    if "bytes" in info:
        info["GBps"] = round(info["bytes"] / (ms * 1e-3) / 1e9, 1)
    print(json.dumps(info), flush=True)


if __name__ == "__main__":
    main()
