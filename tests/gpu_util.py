"""Helpers of the GPU parity tests: numpy in, C-ABI call on cuda:0, numpy out."""
import numpy as np
import torch

from paper_2404_09679_b200 import binding as B

RTOL, ATOL = 1e-5, 1e-6          # fp32 values (per call, identical inputs)
BF16_RTOL = 1e-2                 # bf16 table rows after the update


def close(got, want, rtol=RTOL, atol=ATOL):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    err = np.abs(got - want)
    ok = err <= atol + rtol * np.abs(want)
    if not ok.all():
        i = np.argmax(err - (atol + rtol * np.abs(want)))
        raise AssertionError(f"{(~ok).sum()} of {ok.size} outside tolerance; worst at flat index {i}: "
                             f"got {got.flat[i]!r} want {want.flat[i]!r}")
    return True


def close_mostly(got, want, rtol, atol, max_frac, max_abs):
    """Chained stages: an Adagrad/Adam step divides by |g|-sized quantities, so the few elements
    whose aggregated gradient is within rounding of zero amplify the previous stage's last-bit
    differences.  All but max_frac of the elements must be inside (rtol, atol); none may be off
    by more than max_abs (a learning-rate sized bound)."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    err = np.abs(got - want)
    bad = err > atol + rtol * np.abs(want)
    assert bad.mean() <= max_frac, f"{bad.sum()} of {bad.size} outside tolerance"
    assert err.max() <= max_abs, f"max abs error {err.max()} > {max_abs}"
    return True


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def table_to_dev(table_np):
    """float32 array -> f32 tensor; uint16 array (bf16 bits) -> bf16 tensor."""
    if table_np.dtype == np.uint16:
        return torch.from_numpy(table_np.view(np.int16).copy()).cuda().view(torch.bfloat16)
    return dev(table_np)


def table_to_np(table_t):
    if table_t.dtype == torch.bfloat16:
        return table_t.view(torch.int16).cpu().numpy().view(np.uint16)
    return table_t.cpu().numpy()


def new_status():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


def gpu_fwd(table_np, ids, off, status=None):
    t = table_to_dev(table_np)
    n_bags = off.shape[0] - 1
    pooled = torch.full((max(n_bags, 1), t.shape[1]), float("nan"), device="cuda")
    st = status if status is not None else new_status()
    B.antdt_embbag_fwd(t, dev(ids), dev(off), pooled[:n_bags], st)
    code = B.antdt_read_status(st)
    return pooled[:n_bags].cpu().numpy(), code


def gpu_bwd(ids, off, F, dY, n_rows, wso, out_cap=None, min_workspace=False):
    nnz, n_bags, D, K = ids.shape[0], off.shape[0] - 1, dY.shape[1], len(wso) - 1
    cap = max(1, nnz if out_cap is None else out_cap)
    uid = torch.full((cap,), -1, dtype=torch.int32, device="cuda")
    wuo = torch.full((K + 1,), -1, dtype=torch.int64, device="cuda")
    so = torch.full((cap + 1,), -1, dtype=torch.int64, device="cuda")
    occ = torch.full((max(nnz, 1),), -1, dtype=torch.int32, device="cuda")
    ug = torch.full((cap, D), float("nan"), device="cuda")
    size = (B.antdt_embbag_bwd_dedup_min_workspace_bytes if min_workspace
            else B.antdt_embbag_bwd_dedup_workspace_bytes)(nnz, n_bags, D, K)
    ws = torch.empty(size, dtype=torch.uint8, device="cuda")
    st = new_status()
    B.antdt_embbag_bwd_dedup(dev(ids), dev(off), F, dev(dY), n_rows, [int(x) for x in wso], uid, wuo,
                             so, occ[:nnz], ug, ws, st)
    code = B.antdt_read_status(st)
    wuo_h = wuo.cpu().numpy()
    nu = int(wuo_h[K])
    nu_w = min(nu, cap)
    return dict(uniq_ids=uid[:nu_w].cpu().numpy(), worker_uniq_offsets=wuo_h,
                seg_offsets=so[: nu_w + 1].cpu().numpy(), sorted_occ=occ[:nnz].cpu().numpy(),
                uniq_grads=ug[:nu_w].cpu().numpy(), status=code,
                dev=dict(uniq_ids=uid, worker_uniq_offsets=wuo, uniq_grads=ug))


def gpu_aggregate(uniq_ids, wuo, uniq_grads, bsz, n_rows, dense=None, out_cap=None):
    K = len(bsz)
    n_in = int(wuo[K])
    D = uniq_grads.shape[1]
    cap = max(1, n_in if out_cap is None else out_cap)
    uid = dev(uniq_ids) if n_in else torch.zeros(1, dtype=torch.int32, device="cuda")
    ug = dev(uniq_grads) if n_in else torch.zeros(1, D, device="cuda")
    agg_ids = torch.full((cap,), -1, dtype=torch.int32, device="cuda")
    agg = torch.full((cap, D), float("nan"), device="cuda")
    n_agg = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    ws = torch.empty(B.antdt_weighted_aggregate_workspace_bytes(ug.shape[0], D, K), dtype=torch.uint8,
                     device="cuda")
    st = new_status()
    dg = dout = None
    if dense is not None:
        dg = dev(dense)
        dout = torch.full((dense.shape[1],), float("nan"), device="cuda")
    B.antdt_weighted_aggregate([int(b) for b in bsz], ws, n_rows=n_rows, uniq_ids=uid,
                               worker_uniq_offsets=dev(wuo), uniq_grads=ug, agg_ids=agg_ids,
                               agg_grads=agg, n_agg=n_agg, dense_grads=dg, dense_out=dout,
                               dev_status=st)
    code = B.antdt_read_status(st)
    na = int(n_agg.item())
    k = min(na, cap)
    return (agg_ids[:k].cpu().numpy(), agg[:k].cpu().numpy(), na,
            None if dout is None else dout.cpu().numpy(), code)


def gpu_update(table_np, ids, grads, opt, lr, eps, b1, b2, step, s0, s1=None):
    t = table_to_dev(table_np)
    d0 = dev(s0)
    d1 = None if s1 is None else dev(s1)
    st = new_status()
    n = torch.tensor([ids.shape[0]], dtype=torch.int64, device="cuda")
    ids_t = dev(ids) if ids.shape[0] else torch.zeros(1, dtype=torch.int32, device="cuda")
    g_t = dev(grads) if ids.shape[0] else torch.zeros(1, t.shape[1], device="cuda")
    B.antdt_sparse_opt_update(t, ids_t, g_t, n, B.OPTS[opt], lr, eps, b1, b2, step, d0, d1, st)
    code = B.antdt_read_status(st)
    return table_to_np(t), d0.cpu().numpy(), None if d1 is None else d1.cpu().numpy(), code
