"""TEST INFRASTRUCTURE ONLY: numpy-facing loader of the CPU checker (liboracle.so).

Imported by the tests, the smoke check and the benchmark's CPU-baseline leg; never by the
product package.  Arrays are numpy, contiguous, of the exact dtypes the C++ side expects.
bf16 tables travel as uint16 bit patterns.
"""
import ctypes as C

import numpy as np

from .build import build as _build

_lib = C.CDLL(_build())
_i64, _i32, _f32, _f64 = np.int64, np.int32, np.float32, np.float64
_p = C.c_void_p


def _ptr(a):
    return None if a is None else a.ctypes.data_as(_p)


def _chk(a, dt):
    assert a.dtype == dt and a.flags["C_CONTIGUOUS"], (a.dtype, dt)
    return a


_lib.orc_batch_sizes.argtypes = [_p, C.c_int, C.c_int64, C.c_int, C.c_int64, _p]
_lib.orc_dds_create.restype = _p
_lib.orc_dds_create.argtypes = [C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_uint64]
_lib.orc_dds_destroy.argtypes = [_p]
_lib.orc_dds_num_shards.restype = C.c_int64
_lib.orc_dds_num_shards.argtypes = [_p]
_lib.orc_dds_counts.argtypes = [_p, _p, _p, _p]
_lib.orc_dds_shard_info.argtypes = [_p, C.c_int64, _p, _p, _p, _p]
_lib.orc_dds_plan.argtypes = [_p, _p, C.c_int, C.c_int64, _p, _p, _p, C.c_int64, _p]
_lib.orc_dds_requeue.argtypes = [_p, C.c_int]
_lib.orc_embbag_fwd.argtypes = [_p, C.c_int, C.c_int64, C.c_int, _p, _p, C.c_int64, _p]
_lib.orc_embbag_bwd_dedup.restype = C.c_int64
_lib.orc_embbag_bwd_dedup.argtypes = [_p, _p, C.c_int64, C.c_int, _p, C.c_int, C.c_int64, C.c_int,
                                      _p, _p, _p, _p, _p, _p, C.c_int64]
_lib.orc_embbag_bwd_accum.restype = C.c_int64
_lib.orc_embbag_bwd_accum.argtypes = [_p, _p, C.c_int64, C.c_int, _p, C.c_int, C.c_int64, C.c_int,
                                      _p, _p, _p, _p, _p, C.c_int64]
_lib.orc_aggregate_sparse.restype = C.c_int64
_lib.orc_aggregate_sparse.argtypes = [C.c_int, _p, _p, _p, _p, C.c_int, _p, _p, C.c_int64]
_lib.orc_aggregate_dense.argtypes = [_p, C.c_int64, C.c_int64, _p, C.c_int, _p]
_lib.orc_sparse_opt_update.argtypes = [_p, C.c_int, C.c_int64, C.c_int, _p, _p, C.c_int64, C.c_int,
                                       C.c_float, C.c_float, C.c_float, C.c_float, C.c_int64, _p, _p]
_lib.orc_sparse_rowwise_adagrad.argtypes = [_p, C.c_int, C.c_int64, C.c_int, _p, _p, C.c_int64,
                                            C.c_float, C.c_float, _p]
_lib.orc_dense_opt_update.argtypes = [_p, _p, C.c_int64, C.c_int, C.c_float, C.c_float, C.c_float,
                                      C.c_float, C.c_int64, _p, _p]

_lib.orc_ctl_decide.argtypes = [_p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_double, _p, _p, _p, _p]

_lib.orc_dd_solve.argtypes = [C.c_int, _p, _p, C.c_int64, _p, _p, C.c_int, C.c_int, _p, _p, _p]

_lib.orc_aggregate_sparse_backup.restype = C.c_int64
_lib.orc_aggregate_sparse_backup.argtypes = [C.c_int, _p, _p, _p, _p, _p, C.c_int, _p, _p, C.c_int64]
_lib.orc_aggregate_dense_backup.argtypes = [_p, C.c_int64, C.c_int64, _p, _p, C.c_int, _p]

RULES = {"proportional": 0, "minmax": 1}
OPTS = {"adagrad": 0, "adam": 1}


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle status {code}")
        self.code = code


def batch_sizes(speeds, n, B, rule="proportional", min_batch=0):
    v = None if speeds is None else np.ascontiguousarray(speeds, dtype=_f64)
    out = np.zeros(n, dtype=_i64)
    rc = _lib.orc_batch_sizes(_ptr(v), n, B, RULES[rule], min_batch, _ptr(out))
    if rc:
        raise OracleError(rc)
    return out


class Dds:
    """Section V-C shard service, checker side."""

    def __init__(self, N, B, M, K, shuffle_seed=0):
        self.K = K
        self._h = _lib.orc_dds_create(N, B, M, K, shuffle_seed)
        if not self._h:
            raise OracleError(1)

    def __del__(self):
        if getattr(self, "_h", None):
            _lib.orc_dds_destroy(self._h)
            self._h = None

    def num_shards(self):
        return _lib.orc_dds_num_shards(self._h)

    def counts(self):
        a = [C.c_int64() for _ in range(3)]
        _lib.orc_dds_counts(self._h, *[C.byref(x) for x in a])
        return tuple(x.value for x in a)

    def shard_info(self, j):
        st, ow, s, n = C.c_int(), C.c_int(), C.c_int64(), C.c_int64()
        _lib.orc_dds_shard_info(self._h, j, C.byref(st), C.byref(ow), C.byref(s), C.byref(n))
        return st.value, ow.value, s.value, n.value

    def plan(self, speeds=None, rule="proportional", min_batch=0, cap=None):
        """-> (status, batch_sizes[K], range_offsets[K+1], ranges[n,2], counts[K])"""
        K = self.K
        v = None if speeds is None else np.ascontiguousarray(speeds, dtype=_f64)
        cap = cap if cap is not None else 4 * K + 64
        bsz = np.zeros(K, _i64)
        ro = np.zeros(K + 1, _i64)
        rg = np.zeros((max(cap, 1), 2), _i64)
        cnt = np.zeros(K, _i64)
        rc = _lib.orc_dds_plan(self._h, _ptr(v), RULES[rule], min_batch, _ptr(bsz), _ptr(ro),
                               _ptr(rg), cap, _ptr(cnt))
        return rc, bsz, ro, rg[: ro[K]] if rc in (0, 7) else rg[:0], cnt

    def requeue_worker(self, w):
        rc = _lib.orc_dds_requeue(self._h, w)
        if rc:
            raise OracleError(rc)


def _table_view(table):
    """numpy float32 [V,D] -> (array, 0); numpy uint16 [V,D] (bf16 bits) -> (array, 1)."""
    if table.dtype == _f32:
        return _chk(table, _f32), 0
    return _chk(table, np.uint16), 1


def embbag_fwd(table, row_ids, bag_offsets):
    t, dt = _table_view(table)
    V, D = t.shape
    n_bags = bag_offsets.shape[0] - 1
    out = np.zeros((n_bags, D), _f32)
    rc = _lib.orc_embbag_fwd(_ptr(t), dt, V, D, _ptr(_chk(row_ids, _i32)),
                             _ptr(_chk(bag_offsets, _i64)), n_bags, _ptr(out))
    if rc:
        raise OracleError(rc)
    return out


def embbag_bwd_dedup(row_ids, bag_offsets, F, d_pooled, n_rows, worker_sample_offsets):
    """-> dict(uniq_ids, worker_uniq_offsets, seg_offsets, sorted_occ, uniq_grads)"""
    n_bags = bag_offsets.shape[0] - 1
    nnz = int(bag_offsets[-1])
    D = d_pooled.shape[1]
    K = worker_sample_offsets.shape[0] - 1
    cap = max(nnz, 1)
    uid = np.zeros(cap, _i32)
    wuo = np.zeros(K + 1, _i64)
    so = np.zeros(cap + 1, _i64)
    occ = np.zeros(max(nnz, 1), _i32)
    ug = np.zeros((cap, D), _f32)
    nu = _lib.orc_embbag_bwd_dedup(_ptr(_chk(row_ids, _i32)), _ptr(_chk(bag_offsets, _i64)), n_bags,
                                   F, _ptr(_chk(d_pooled, _f32)), D, n_rows, K,
                                   _ptr(_chk(worker_sample_offsets, _i64)), _ptr(uid), _ptr(wuo),
                                   _ptr(so), _ptr(occ), _ptr(ug), cap)
    if nu < 0:
        raise OracleError(-nu)
    return dict(uniq_ids=uid[:nu].copy(), worker_uniq_offsets=wuo, seg_offsets=so[: nu + 1].copy(),
                sorted_occ=occ[:nnz].copy(), uniq_grads=ug[:nu].copy())


def embbag_bwd_accum(row_ids, bag_offsets, F, d_pooled, n_rows, worker_sample_offsets, micro_batches):
    """Gradient accumulation (Section VI-B): worker w's samples are micro_batches[w] micro-batches
    back to back; -> dict(uniq_ids, worker_uniq_offsets, uniq_grads), the mean of the micro-batch
    mean gradients."""
    n_bags = bag_offsets.shape[0] - 1
    nnz = int(bag_offsets[-1])
    D = d_pooled.shape[1]
    K = worker_sample_offsets.shape[0] - 1
    cap = max(nnz, 1)
    uid = np.zeros(cap, _i32)
    wuo = np.zeros(K + 1, _i64)
    ug = np.zeros((cap, D), _f32)
    nu = _lib.orc_embbag_bwd_accum(_ptr(_chk(row_ids, _i32)), _ptr(_chk(bag_offsets, _i64)), n_bags,
                                   F, _ptr(_chk(d_pooled, _f32)), D, n_rows, K,
                                   _ptr(_chk(worker_sample_offsets, _i64)),
                                   _ptr(np.ascontiguousarray(micro_batches, _i64)), _ptr(uid),
                                   _ptr(wuo), _ptr(ug), cap)
    if nu < 0:
        raise OracleError(-nu)
    return dict(uniq_ids=uid[:nu].copy(), worker_uniq_offsets=wuo, uniq_grads=ug[:nu].copy())


def aggregate_sparse(uniq_ids, worker_uniq_offsets, uniq_grads, batch_sizes_):
    K = worker_uniq_offsets.shape[0] - 1
    n = int(worker_uniq_offsets[K])
    D = uniq_grads.shape[1]
    ids = np.zeros(max(n, 1), _i32)
    g = np.zeros((max(n, 1), D), _f32)
    na = _lib.orc_aggregate_sparse(D, _ptr(_chk(uniq_ids, _i32)), _ptr(_chk(worker_uniq_offsets, _i64)),
                                   _ptr(_chk(uniq_grads, _f32)),
                                   _ptr(np.ascontiguousarray(batch_sizes_, _i64)), K, _ptr(ids),
                                   _ptr(g), max(n, 1))
    if na < 0:
        raise OracleError(-na)
    return ids[:na].copy(), g[:na].copy()


def aggregate_dense(grads, batch_sizes_):
    K, n = grads.shape
    out = np.zeros(n, _f32)
    rc = _lib.orc_aggregate_dense(_ptr(_chk(grads, _f32)), n, n,
                                  _ptr(np.ascontiguousarray(batch_sizes_, _i64)), K, _ptr(out))
    if rc:
        raise OracleError(rc)
    return out


def sparse_opt_update(table, ids, grads, opt, lr, eps, beta1, beta2, step, state0, state1=None):
    """In place on table / state0 / state1 (numpy arrays)."""
    t, dt = _table_view(table)
    V, D = t.shape
    rc = _lib.orc_sparse_opt_update(_ptr(t), dt, V, D, _ptr(_chk(ids, _i32)), _ptr(_chk(grads, _f32)),
                                    ids.shape[0], OPTS[opt], lr, eps, beta1, beta2, step,
                                    _ptr(_chk(state0, _f32)),
                                    _ptr(None if state1 is None else _chk(state1, _f32)))
    if rc:
        raise OracleError(rc)


def sparse_rowwise_adagrad(table, ids, grads, lr, eps, state0):
    """In place on table and state0 (numpy [n_rows] float32: one accumulator per row)."""
    t, dt = _table_view(table)
    V, D = t.shape
    assert state0.shape == (V,)
    rc = _lib.orc_sparse_rowwise_adagrad(_ptr(t), dt, V, D, _ptr(_chk(ids, _i32)),
                                         _ptr(_chk(grads, _f32)), ids.shape[0], lr, eps,
                                         _ptr(_chk(state0, _f32)))
    if rc:
        raise OracleError(rc)


def dense_opt_update(params, grad, opt, lr, eps, beta1, beta2, step, state0, state1=None):
    """In place on params / state0 / state1 (numpy float32 vectors of one length)."""
    n = params.shape[0]
    assert grad.shape == (n,) and state0.shape == (n,)
    rc = _lib.orc_dense_opt_update(_ptr(_chk(params, _f32)), _ptr(_chk(grad, _f32)), n, OPTS[opt],
                                   lr, eps, beta1, beta2, step, _ptr(_chk(state0, _f32)),
                                   _ptr(None if state1 is None else _chk(state1, _f32)))
    if rc:
        raise OracleError(rc)


def ctl_decide(reports, K, Lt, Lp, lam):
    """reports: rows (worker, batch size, BPT seconds) -> (speeds, transient, persistent, action)"""
    r = np.ascontiguousarray(reports, dtype=_f64).reshape(-1, 3)
    v = np.zeros(K, _f64)
    t = np.zeros(K, np.int32)
    p = np.zeros(K, np.int32)
    a = C.c_int()
    rc = _lib.orc_ctl_decide(_ptr(r), r.shape[0], K, Lt, Lp, lam, _ptr(v), _ptr(t), _ptr(p), C.byref(a))
    if rc:
        raise OracleError(rc)
    return v, t, p, a.value


def dd_solve(n_dev, v, B, bmin, bmax, cmin, cmax):
    k = len(n_dev)
    nd = np.ascontiguousarray(n_dev, dtype=np.int32)
    vv = np.ascontiguousarray(v, dtype=_f64)
    lo, hi = np.ascontiguousarray(bmin, dtype=_i64), np.ascontiguousarray(bmax, dtype=_i64)
    b = np.zeros(k, _i64)
    c = np.zeros(k, np.int32)
    z = C.c_double()
    rc = _lib.orc_dd_solve(k, _ptr(nd), _ptr(vv), B, _ptr(lo), _ptr(hi), cmin, cmax, _ptr(b), _ptr(c),
                           C.byref(z))
    if rc:
        raise OracleError(rc)
    return b, c, z.value


def aggregate_sparse_backup(uniq_ids, worker_uniq_offsets, uniq_grads, batch_sizes_, dropped):
    K = worker_uniq_offsets.shape[0] - 1
    n = int(worker_uniq_offsets[K])
    D = uniq_grads.shape[1]
    ids = np.zeros(max(n, 1), _i32)
    g = np.zeros((max(n, 1), D), _f32)
    d = np.ascontiguousarray(dropped, dtype=np.uint8)
    na = _lib.orc_aggregate_sparse_backup(D, _ptr(_chk(uniq_ids, _i32)), _ptr(_chk(worker_uniq_offsets, _i64)),
                                          _ptr(_chk(uniq_grads, _f32)),
                                          _ptr(np.ascontiguousarray(batch_sizes_, _i64)), _ptr(d), K,
                                          _ptr(ids), _ptr(g), max(n, 1))
    if na < 0:
        raise OracleError(-na)
    return ids[:na].copy(), g[:na].copy()


def aggregate_dense_backup(grads, batch_sizes_, dropped):
    K, n = grads.shape
    out = np.zeros(n, _f32)
    d = np.ascontiguousarray(dropped, dtype=np.uint8)
    rc = _lib.orc_aggregate_dense_backup(_ptr(_chk(grads, _f32)), n, n,
                                         _ptr(np.ascontiguousarray(batch_sizes_, _i64)), _ptr(d), K, _ptr(out))
    if rc:
        raise OracleError(rc)
    return out
