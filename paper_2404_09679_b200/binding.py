"""ctypes binding of libantdt.so: the same names as the C entry points, argument marshalling
only (tensor -> pointer, Python list -> C array).  Every step of the path runs in the CUDA
library; there is no fallback: if the library is missing or a call fails, an exception is raised.

Device buffers are torch CUDA tensors (torch is used for device memory and streams only).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

OK, ERR_INVALID_ARG, ERR_ID_OUT_OF_RANGE, ERR_WORKSPACE_TOO_SMALL, ERR_CAPACITY, ERR_CUDA, \
    ERR_TIMEOUT, ERR_EXHAUSTED, ERR_STATE, ERR_BAD_OFFSETS, ERR_INFEASIBLE = range(11)
F32, BF16 = 0, 1
RULE_PROPORTIONAL, RULE_MINMAX = 0, 1
OPT_ADAGRAD, OPT_ADAM, OPT_ROWWISE_ADAGRAD = 0, 1, 2
SHARD_TODO, SHARD_DOING, SHARD_DONE = 0, 1, 2
RULES = {"proportional": RULE_PROPORTIONAL, "minmax": RULE_MINMAX}
OPTS = {"adagrad": OPT_ADAGRAD, "adam": OPT_ADAM, "rowwise_adagrad": OPT_ROWWISE_ADAGRAD}

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libantdt.so")
_lib = None

EXPORTS = [
    "antdt_dds_create", "antdt_dds_destroy", "antdt_batch_sizes", "antdt_shard_plan",
    "antdt_dds_requeue_worker", "antdt_dds_num_shards", "antdt_dds_counts", "antdt_dds_shard_info",
    "antdt_dds_save", "antdt_dds_load", "antdt_ctl_create", "antdt_ctl_destroy",
    "antdt_ctl_report", "antdt_ctl_decide", "antdt_dd_solve", "antdt_embbag_fwd",
    "antdt_embbag_bwd_dedup_workspace_bytes", "antdt_embbag_bwd_dedup_min_workspace_bytes",
    "antdt_embbag_bwd_dedup",
    "antdt_embbag_bwd_dedup_static",
    "antdt_weighted_aggregate_workspace_bytes", "antdt_weighted_aggregate",
    "antdt_bsp_step_workspace_bytes",
    "antdt_weighted_aggregate_backup", "antdt_aggregate_update",
    "antdt_sparse_opt_update", "antdt_dense_opt_update", "antdt_bsp_step_host", "antdt_bsp_step_device", "antdt_bsp_step_graph", "antdt_bsp_step_graph_reset",
    "antdt_read_status", "antdt_launch_count",
    "antdt_profile_enable", "antdt_profile_kernels", "antdt_profile_get", "antdt_probe_gather",
    "antdt_version",
]


class AntdtError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: status {code}")
        self.code = code


class Range(C.Structure):
    _fields_ = [("start", C.c_int64), ("len", C.c_int64)]


class SparsePart(C.Structure):
    _fields_ = [("dim", C.c_int32), ("n_rows", C.c_int64), ("uniq_ids", C.c_void_p),
                ("worker_uniq_offsets", C.c_void_p), ("uniq_grads", C.c_void_p),
                ("in_cap", C.c_int64), ("agg_ids", C.c_void_p), ("agg_grads", C.c_void_p),
                ("n_agg", C.c_void_p), ("out_cap", C.c_int64)]


class DensePart(C.Structure):
    _fields_ = [("grads", C.c_void_p), ("n", C.c_int64), ("stride", C.c_int64),
                ("out", C.c_void_p)]


class StepDesc(C.Structure):
    _fields_ = [
        ("table", C.c_void_p), ("dtype", C.c_int32), ("n_rows", C.c_int64), ("dim", C.c_int32),
        ("state0", C.c_void_p), ("state1", C.c_void_p),
        ("opt", C.c_int32), ("lr", C.c_float), ("eps", C.c_float), ("beta1", C.c_float),
        ("beta2", C.c_float), ("step", C.c_int64),
        ("h_row_ids", C.c_void_p), ("nnz", C.c_int64),
        ("h_bag_offsets", C.c_void_p), ("n_bags", C.c_int64), ("bags_per_sample", C.c_int32),
        ("h_d_pooled", C.c_void_p), ("h_dense_grads", C.c_void_p), ("dense_n", C.c_int64),
        ("n_workers", C.c_int32), ("worker_sample_offsets", C.c_void_p),
        ("batch_sizes", C.c_void_p),
        ("d_row_ids", C.c_void_p), ("d_bag_offsets", C.c_void_p), ("d_pooled_out", C.c_void_p),
        ("d_d_pooled", C.c_void_p), ("d_dense_grads", C.c_void_p), ("d_dense_out", C.c_void_p),
        ("d_uniq_ids", C.c_void_p), ("d_worker_uniq_offsets", C.c_void_p),
        ("d_seg_offsets", C.c_void_p), ("d_sorted_occ", C.c_void_p), ("d_uniq_grads", C.c_void_p),
        ("uniq_cap", C.c_int64),
        ("d_agg_ids", C.c_void_p), ("d_agg_grads", C.c_void_p), ("d_n_agg", C.c_void_p),
        ("agg_cap", C.c_int64),
        ("ws", C.c_void_p), ("ws_bytes", C.c_size_t), ("d_status", C.c_void_p),
        ("h_pooled", C.c_void_p), ("h_dense_out", C.c_void_p), ("h_n_agg", C.c_void_p),
        ("h_status", C.c_void_p), ("staging_idle", C.c_int32), ("fuse_update", C.c_int32),
    ]


def lib() -> C.CDLL:
    """Loads libantdt.so (once).  A missing library is an error: build it with
    `python -m paper_2404_09679_b200.build`."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise AntdtError(ERR_STATE, f"{_LIB_PATH} is not built (python -m paper_2404_09679_b200.build)")
        L = C.CDLL(_LIB_PATH)
        P, I32, I64, F, D, SZ = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_double, C.c_size_t
        L.antdt_dds_create.argtypes = [C.POINTER(P), I64, I64, I32, I32, C.c_uint64]
        L.antdt_dds_destroy.argtypes = [P]
        L.antdt_dds_destroy.restype = None
        L.antdt_batch_sizes.argtypes = [P, I32, I64, I32, I64, P]
        L.antdt_shard_plan.argtypes = [P, P, I32, I64, P, P, P, I64, P]
        L.antdt_dds_requeue_worker.argtypes = [P, I32]
        L.antdt_dds_num_shards.argtypes = [P]
        L.antdt_dds_num_shards.restype = I64
        L.antdt_dds_counts.argtypes = [P, P, P, P]
        L.antdt_dds_shard_info.argtypes = [P, I64, P, P, P]
        L.antdt_dds_save.argtypes = [P, P, SZ, C.POINTER(SZ)]
        L.antdt_dds_load.argtypes = [C.POINTER(P), P, SZ]
        L.antdt_ctl_create.argtypes = [C.POINTER(P), I32, I32, I32, D]
        L.antdt_ctl_destroy.argtypes = [P]
        L.antdt_ctl_destroy.restype = None
        L.antdt_ctl_report.argtypes = [P, I32, I64, D]
        L.antdt_ctl_decide.argtypes = [P, P, P, P, P]
        L.antdt_dd_solve.argtypes = [I32, P, P, I64, P, P, I32, I32, P, P, P]
        L.antdt_dd_solve.restype = I32
        L.antdt_embbag_fwd.argtypes = [P, I32, I64, I32, P, I64, P, I64, P, P, P]
        L.antdt_embbag_bwd_dedup_workspace_bytes.argtypes = [I64, I64, I32, I32]
        L.antdt_embbag_bwd_dedup_workspace_bytes.restype = SZ
        L.antdt_embbag_bwd_dedup_min_workspace_bytes.argtypes = [I64, I64, I32, I32]
        L.antdt_embbag_bwd_dedup_min_workspace_bytes.restype = SZ
        L.antdt_embbag_bwd_dedup.argtypes = [P, I64, P, I64, I32, P, I32, I64, I32, P, P, P, P, P, P,
                                             I64, P, SZ, P, P]
        L.antdt_embbag_bwd_dedup_static.argtypes = [P, I64, P, I64, I32, P, I32, I64, I32, P, P, P, P,
                                                    P, P, I64, P, P]
        L.antdt_embbag_bwd_dedup_static.restype = I32
        L.antdt_weighted_aggregate_workspace_bytes.argtypes = [I64, I32, I32]
        L.antdt_weighted_aggregate_workspace_bytes.restype = SZ
        L.antdt_bsp_step_workspace_bytes.argtypes = [I64, I64, I32, I32, I64]
        L.antdt_bsp_step_workspace_bytes.restype = SZ
        L.antdt_weighted_aggregate.argtypes = [P, P, P, I32, P, SZ, P, P]
        L.antdt_weighted_aggregate_backup.argtypes = [P, P, P, P, I32, P, SZ, P, P]
        L.antdt_weighted_aggregate_backup.restype = I32
        L.antdt_aggregate_update.argtypes = [P, P, P, I32, P, I32, I32, C.c_float, C.c_float, C.c_float,
                                             C.c_float, I64, P, P, P, SZ, P, P]
        L.antdt_aggregate_update.restype = I32
        L.antdt_sparse_opt_update.argtypes = [P, I32, I64, I32, P, P, P, I64, I32, F, F, F, F, I64,
                                              P, P, P, P]
        L.antdt_dense_opt_update.argtypes = [P, P, I64, I32, F, F, F, F, I64, P, P, P]
        L.antdt_dense_opt_update.restype = I32
        L.antdt_bsp_step_host.argtypes = [P, P]
        L.antdt_bsp_step_device.argtypes = [P, P]
        L.antdt_bsp_step_device.restype = I32
        L.antdt_bsp_step_graph.argtypes = [P, P]
        L.antdt_bsp_step_graph.restype = I32
        L.antdt_bsp_step_graph_reset.argtypes = []
        L.antdt_bsp_step_graph_reset.restype = I32
        L.antdt_read_status.argtypes = [P, P]
        L.antdt_launch_count.restype = I64
        L.antdt_profile_enable.argtypes = [I32]
        L.antdt_profile_get.argtypes = [I32, C.c_char_p, SZ, C.POINTER(I64), C.POINTER(D)]
        L.antdt_version.restype = C.c_char_p
        L.antdt_probe_gather.argtypes = [P, I64, I32, P, I64, I32, P, P]
        L.antdt_probe_gather.restype = I32
        for fn in ("antdt_ctl_create", "antdt_ctl_report", "antdt_ctl_decide",
                   "antdt_dds_create", "antdt_batch_sizes", "antdt_shard_plan",
                   "antdt_dds_requeue_worker", "antdt_dds_counts", "antdt_dds_shard_info",
                   "antdt_dds_save", "antdt_dds_load", "antdt_ctl_create", "antdt_ctl_destroy",
    "antdt_ctl_report", "antdt_ctl_decide", "antdt_dd_solve", "antdt_embbag_fwd", "antdt_embbag_bwd_dedup",
                   "antdt_weighted_aggregate", "antdt_sparse_opt_update", "antdt_bsp_step_host", "antdt_bsp_step_device",
                   "antdt_read_status", "antdt_profile_enable", "antdt_profile_kernels",
                   "antdt_profile_get"):
            getattr(L, fn).restype = I32
        _lib = L
    return _lib


def _check(rc: int, where: str):
    if rc != OK:
        raise AntdtError(rc, where)


def _dp(t: Optional[torch.Tensor]):
    """Device (or pinned host) tensor -> raw pointer; None -> NULL."""
    if t is None:
        return None
    assert t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _i64s(xs: Sequence[int]):
    return (C.c_int64 * len(xs))(*[int(x) for x in xs])


def _f64s(xs: Sequence[float]):
    return (C.c_double * len(xs))(*[float(x) for x in xs])


def _dtype_code(table: torch.Tensor) -> int:
    if table.dtype == torch.float32:
        return F32
    if table.dtype == torch.bfloat16:
        return BF16
    raise AntdtError(ERR_INVALID_ARG, "table dtype must be float32 or bfloat16")


# ---- host planner --------------------------------------------------------------------------
def antdt_batch_sizes(speeds, n_workers: int, global_batch: int, rule: int = RULE_PROPORTIONAL,
                      min_batch: int = 0):
    out = (C.c_int64 * n_workers)()
    v = None if speeds is None else _f64s(speeds)
    _check(lib().antdt_batch_sizes(v, n_workers, global_batch, rule, min_batch, out),
           "antdt_batch_sizes")
    return list(out)


class Dds:
    """Handle of the shard service (antdt_dds_* calls)."""

    def __init__(self, n_samples: int, global_batch: int, batches_per_shard: int, n_workers: int,
                 shuffle_seed: int = 0, _handle=None):
        self.K = n_workers
        if _handle is not None:
            self._h = _handle
            return
        h = C.c_void_p()
        _check(lib().antdt_dds_create(C.byref(h), n_samples, global_batch, batches_per_shard,
                                      n_workers, shuffle_seed), "antdt_dds_create")
        self._h = h

    def __del__(self):
        if getattr(self, "_h", None):
            lib().antdt_dds_destroy(self._h)
            self._h = None

    def antdt_shard_plan(self, speeds=None, rule: int = RULE_PROPORTIONAL, min_batch: int = 0,
                         ranges_cap: Optional[int] = None):
        """-> (status, batch_sizes, range_offsets, ranges [(start, len)...], counts).
        status is OK or ERR_EXHAUSTED; anything else raises."""
        K = self.K
        cap = ranges_cap if ranges_cap is not None else 4 * K + 64
        bsz, ro, cnt = (C.c_int64 * K)(), (C.c_int64 * (K + 1))(), (C.c_int64 * K)()
        rg = (Range * max(cap, 1))()
        v = None if speeds is None else _f64s(speeds)
        rc = lib().antdt_shard_plan(self._h, v, rule, min_batch, bsz, ro, rg, cap, cnt)
        if rc not in (OK, ERR_EXHAUSTED):
            raise AntdtError(rc, "antdt_shard_plan")
        ranges = [(rg[i].start, rg[i].len) for i in range(ro[K])]
        return rc, list(bsz), list(ro), ranges, list(cnt)

    def antdt_dds_requeue_worker(self, worker: int):
        _check(lib().antdt_dds_requeue_worker(self._h, worker), "antdt_dds_requeue_worker")

    def antdt_dds_num_shards(self) -> int:
        return lib().antdt_dds_num_shards(self._h)

    def antdt_dds_counts(self):
        a = [C.c_int64() for _ in range(3)]
        _check(lib().antdt_dds_counts(self._h, *[C.byref(x) for x in a]), "antdt_dds_counts")
        return tuple(x.value for x in a)

    def antdt_dds_shard_info(self, shard: int):
        st, ow, r = C.c_int32(), C.c_int32(), Range()
        _check(lib().antdt_dds_shard_info(self._h, shard, C.byref(st), C.byref(ow), C.byref(r)),
               "antdt_dds_shard_info")
        return st.value, ow.value, r.start, r.len

    def antdt_dds_save(self) -> bytes:
        used = C.c_size_t()
        _check(lib().antdt_dds_save(self._h, None, 0, C.byref(used)), "antdt_dds_save")
        buf = C.create_string_buffer(used.value)
        _check(lib().antdt_dds_save(self._h, buf, used.value, C.byref(used)), "antdt_dds_save")
        return buf.raw[: used.value]

    @staticmethod
    def antdt_dds_load(image: bytes, n_workers: int) -> "Dds":
        h = C.c_void_p()
        _check(lib().antdt_dds_load(C.byref(h), image, len(image)), "antdt_dds_load")
        return Dds(0, 0, 0, n_workers, _handle=h)


ACTION_NONE, ACTION_ADJUST_BS, ACTION_KILL_RESTART = 0, 1, 2


class Ctl:
    """Handle of the AntDT-ND controller front end (antdt_ctl_* calls)."""

    def __init__(self, n_workers: int, window_trans: int, window_per: int, lam: float):
        self.K = n_workers
        h = C.c_void_p()
        _check(lib().antdt_ctl_create(C.byref(h), n_workers, window_trans, window_per, lam),
               "antdt_ctl_create")
        self._h = h

    def __del__(self):
        if getattr(self, "_h", None):
            lib().antdt_ctl_destroy(self._h)
            self._h = None

    def antdt_ctl_report(self, worker: int, batch_size: int, bpt_seconds: float):
        _check(lib().antdt_ctl_report(self._h, worker, batch_size, bpt_seconds), "antdt_ctl_report")

    def antdt_ctl_decide(self):
        """-> (speeds [K], transient [K], persistent [K], action)"""
        K = self.K
        v, t, p, a = (C.c_double * K)(), (C.c_int32 * K)(), (C.c_int32 * K)(), C.c_int32()
        _check(lib().antdt_ctl_decide(self._h, v, t, p, C.byref(a)), "antdt_ctl_decide")
        return list(v), list(t), list(p), a.value


def antdt_dd_solve(n_devices, speeds, global_batch: int, batch_min, batch_max, accum_min: int,
                   accum_max: int):
    """-> (B_i list, C_i list, z) of Eq. 4; raises AntdtError(ERR_INFEASIBLE) if there is none."""
    k = len(n_devices)
    nd = (C.c_int32 * k)(*[int(x) for x in n_devices])
    b, c, z = (C.c_int64 * k)(), (C.c_int32 * k)(), C.c_double()
    _check(lib().antdt_dd_solve(k, nd, _f64s(speeds), global_batch, _i64s(batch_min),
                                _i64s(batch_max), accum_min, accum_max, b, c, C.byref(z)),
           "antdt_dd_solve")
    return list(b), list(c), z.value


# ---- device path ---------------------------------------------------------------------------
def antdt_embbag_fwd(table, row_ids, bag_offsets, pooled, dev_status=None, stream=None):
    V, D = table.shape
    n_bags = bag_offsets.numel() - 1
    _check(lib().antdt_embbag_fwd(_dp(table), _dtype_code(table), V, D, _dp(row_ids),
                                  row_ids.numel(), _dp(bag_offsets), n_bags, _dp(pooled),
                                  _dp(dev_status), _stream(stream)), "antdt_embbag_fwd")


def antdt_embbag_bwd_dedup_workspace_bytes(nnz: int, n_bags: int, dim: int, n_workers: int) -> int:
    return lib().antdt_embbag_bwd_dedup_workspace_bytes(nnz, n_bags, dim, n_workers)


def antdt_embbag_bwd_dedup_min_workspace_bytes(nnz: int, n_bags: int, dim: int, n_workers: int) -> int:
    return lib().antdt_embbag_bwd_dedup_min_workspace_bytes(nnz, n_bags, dim, n_workers)


def antdt_embbag_bwd_dedup(row_ids, bag_offsets, bags_per_sample: int, d_pooled, n_rows: int,
                           worker_sample_offsets: Sequence[int], uniq_ids, worker_uniq_offsets,
                           seg_offsets, sorted_occ, uniq_grads, ws, dev_status=None, stream=None):
    n_bags = bag_offsets.numel() - 1
    K = len(worker_sample_offsets) - 1
    _check(lib().antdt_embbag_bwd_dedup(
        _dp(row_ids), row_ids.numel(), _dp(bag_offsets), n_bags, bags_per_sample, _dp(d_pooled),
        d_pooled.shape[1], n_rows, K, _i64s(worker_sample_offsets), _dp(uniq_ids),
        _dp(worker_uniq_offsets), _dp(seg_offsets), _dp(sorted_occ), _dp(uniq_grads),
        uniq_grads.shape[0], _dp(ws), ws.numel() * ws.element_size(), _dp(dev_status),
        _stream(stream)), "antdt_embbag_bwd_dedup")


STATIC_SCRATCH_BYTES = 24 << 20


def antdt_embbag_bwd_dedup_static(row_ids, bag_offsets, bags_per_sample: int, d_pooled, n_rows: int,
                                  worker_sample_offsets: Sequence[int], uniq_ids, worker_uniq_offsets,
                                  seg_offsets, sorted_occ, uniq_grads, dev_status=None, stream=None):
    """antdt_embbag_bwd_dedup for callers that cannot allocate device memory: no workspace
    argument, the scratch is a fixed STATIC_SCRATCH_BYTES array inside the library (shared by
    all calls on a device, so calls must not overlap).  Raises with ERR_CAPACITY when the
    problem needs more scratch than that."""
    n_bags = bag_offsets.numel() - 1
    K = len(worker_sample_offsets) - 1
    _check(lib().antdt_embbag_bwd_dedup_static(
        _dp(row_ids), row_ids.numel(), _dp(bag_offsets), n_bags, bags_per_sample, _dp(d_pooled),
        d_pooled.shape[1], n_rows, K, _i64s(worker_sample_offsets), _dp(uniq_ids),
        _dp(worker_uniq_offsets), _dp(seg_offsets), _dp(sorted_occ), _dp(uniq_grads),
        uniq_grads.shape[0], _dp(dev_status), _stream(stream)), "antdt_embbag_bwd_dedup_static")


def antdt_weighted_aggregate_workspace_bytes(in_cap: int, dim: int, n_workers: int) -> int:
    return lib().antdt_weighted_aggregate_workspace_bytes(in_cap, dim, n_workers)


def antdt_bsp_step_workspace_bytes(nnz: int, n_bags: int, dim: int, n_workers: int, uniq_cap: int) -> int:
    return lib().antdt_bsp_step_workspace_bytes(nnz, n_bags, dim, n_workers, uniq_cap)


def antdt_weighted_aggregate(batch_sizes: Sequence[int], ws, *, n_rows: int = 0, uniq_ids=None,
                             worker_uniq_offsets=None, uniq_grads=None, agg_ids=None,
                             agg_grads=None, n_agg=None, dense_grads=None, dense_out=None,
                             dev_status=None, stream=None, dropped=None):
    """Sparse part when uniq_ids is given, dense part when dense_grads ([K, n]) is given.
    dropped (list of K flags) selects antdt_weighted_aggregate_backup."""
    K = len(batch_sizes)
    sp = dp = None
    if uniq_ids is not None:
        sp = SparsePart(uniq_grads.shape[1], n_rows, uniq_ids.data_ptr(),
                        worker_uniq_offsets.data_ptr(), uniq_grads.data_ptr(), uniq_grads.shape[0],
                        agg_ids.data_ptr(), agg_grads.data_ptr(), n_agg.data_ptr(),
                        agg_grads.shape[0])
    if dense_grads is not None:
        dp = DensePart(dense_grads.data_ptr(), dense_grads.shape[1], dense_grads.stride(0),
                       dense_out.data_ptr())
    if dropped is not None:
        flags = (C.c_uint8 * K)(*[1 if d else 0 for d in dropped])
        _check(lib().antdt_weighted_aggregate_backup(
            C.byref(sp) if sp else None, C.byref(dp) if dp else None, _i64s(batch_sizes), flags, K,
            _dp(ws), ws.numel() * ws.element_size(), _dp(dev_status), _stream(stream)),
            "antdt_weighted_aggregate_backup")
        return
    _check(lib().antdt_weighted_aggregate(
        C.byref(sp) if sp else None, C.byref(dp) if dp else None, _i64s(batch_sizes), K, _dp(ws),
        ws.numel() * ws.element_size(), _dp(dev_status), _stream(stream)),
        "antdt_weighted_aggregate")


def antdt_aggregate_update(batch_sizes: Sequence[int], ws, table, opt: int, lr: float, eps: float,
                           beta1: float, beta2: float, step: int, state0, state1=None, *,
                           uniq_ids, worker_uniq_offsets, uniq_grads, agg_ids, n_agg, agg_grads=None,
                           dense_grads=None, dense_out=None, dev_status=None, stream=None):
    """antdt_weighted_aggregate + antdt_sparse_opt_update in one call (one pass for <= 32 workers);
    agg_grads=None: the aggregated gradients are not materialised."""
    K = len(batch_sizes)
    V, D = table.shape
    sp = SparsePart(D, V, uniq_ids.data_ptr(), worker_uniq_offsets.data_ptr(), uniq_grads.data_ptr(),
                    uniq_grads.shape[0], agg_ids.data_ptr(),
                    None if agg_grads is None else agg_grads.data_ptr(), n_agg.data_ptr(),
                    agg_ids.shape[0])
    dp = None
    if dense_grads is not None:
        dp = DensePart(dense_grads.data_ptr(), dense_grads.shape[1], dense_grads.stride(0),
                       dense_out.data_ptr())
    _check(lib().antdt_aggregate_update(
        C.byref(sp), C.byref(dp) if dp else None, _i64s(batch_sizes), K, _dp(table), _dtype_code(table),
        opt, lr, eps, beta1, beta2, step, _dp(state0), _dp(state1), _dp(ws),
        ws.numel() * ws.element_size(), _dp(dev_status), _stream(stream)), "antdt_aggregate_update")


def antdt_sparse_opt_update(table, ids, grads, n_ids_dev, opt: int, lr: float, eps: float,
                            beta1: float, beta2: float, step: int, state0, state1=None,
                            dev_status=None, stream=None):
    V, D = table.shape
    _check(lib().antdt_sparse_opt_update(
        _dp(table), _dtype_code(table), V, D, _dp(ids), _dp(grads), _dp(n_ids_dev), ids.numel(),
        opt, lr, eps, beta1, beta2, step, _dp(state0), _dp(state1), _dp(dev_status),
        _stream(stream)), "antdt_sparse_opt_update")


def antdt_dense_opt_update(params, grad, opt: int, lr: float, eps: float, beta1: float,
                           beta2: float, step: int, state0, state1=None, stream=None):
    _check(lib().antdt_dense_opt_update(_dp(params), _dp(grad), params.numel(), opt, lr, eps, beta1,
                                        beta2, step, _dp(state0), _dp(state1), _stream(stream)),
           "antdt_dense_opt_update")


def antdt_bsp_step_host(desc: StepDesc, stream=None):
    _check(lib().antdt_bsp_step_host(C.byref(desc), _stream(stream)), "antdt_bsp_step_host")


def antdt_bsp_step_device(desc: StepDesc, stream=None):
    _check(lib().antdt_bsp_step_device(C.byref(desc), _stream(stream)), "antdt_bsp_step_device")


def antdt_bsp_step_graph(desc: StepDesc, stream=None):
    _check(lib().antdt_bsp_step_graph(C.byref(desc), _stream(stream)), "antdt_bsp_step_graph")


def antdt_bsp_step_graph_reset():
    _check(lib().antdt_bsp_step_graph_reset(), "antdt_bsp_step_graph_reset")


def antdt_read_status(dev_status, stream=None) -> int:
    return lib().antdt_read_status(_dp(dev_status), _stream(stream))


def antdt_launch_count() -> int:
    return lib().antdt_launch_count()


def antdt_profile_enable(on: bool):
    _check(lib().antdt_profile_enable(1 if on else 0), "antdt_profile_enable")


def antdt_profile_get():
    """-> {kernel name: (launches, total_ms)} since antdt_profile_enable(True)."""
    out = {}
    n = lib().antdt_profile_kernels()
    for i in range(n):
        name = C.create_string_buffer(64)
        launches, ms = C.c_int64(), C.c_double()
        _check(lib().antdt_profile_get(i, name, 64, C.byref(launches), C.byref(ms)),
               "antdt_profile_get")
        out[name.value.decode()] = (launches.value, ms.value)
    return out


def antdt_probe_gather(rows, idx, per_out: int, out, stream=None):
    """out[o] = sum of rows[idx[o*per_out : (o+1)*per_out]]: the gather-rate probe."""
    _check(lib().antdt_probe_gather(_dp(rows), rows.shape[0], rows.shape[1], _dp(idx), out.shape[0],
                                    per_out, _dp(out), _stream(stream)), "antdt_probe_gather")


def antdt_version() -> str:
    return lib().antdt_version().decode()
