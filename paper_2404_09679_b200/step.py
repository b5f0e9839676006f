"""Buffer set and call sequence of one BSP step (marshalling only; all compute is in libantdt).

`StepBuffers` owns the device tensors a step needs (torch = device memory only) and `run_step`
issues the four device calls in order on the current stream.  Nothing here touches the data.
"""
from __future__ import annotations

import dataclasses
from typing import Optional, Sequence

import torch

from . import binding as B


@dataclasses.dataclass
class OptConfig:
    opt: int
    lr: float
    eps: float = 1e-8
    beta1: float = 0.9
    beta2: float = 0.999


class StepBuffers:
    """Outputs, intermediates and workspace of a step, sized for at most max_nnz occurrences,
    max_bags bags and uniq_cap (worker, row) pairs."""

    def __init__(self, dim: int, n_workers: int, max_nnz: int, max_bags: int, dense_n: int = 0,
                 uniq_cap: Optional[int] = None, agg_cap: Optional[int] = None, device="cuda"):
        dev = torch.device(device)
        self.dim, self.K, self.max_nnz, self.max_bags = dim, n_workers, max_nnz, max_bags
        self.uniq_cap = max(1, uniq_cap if uniq_cap is not None else max_nnz)
        self.agg_cap = max(1, agg_cap if agg_cap is not None else self.uniq_cap)
        i32, i64, f32 = torch.int32, torch.int64, torch.float32
        self.pooled = torch.empty(max(max_bags, 1), dim, dtype=f32, device=dev)
        self.uniq_ids = torch.empty(self.uniq_cap, dtype=i32, device=dev)
        self.worker_uniq_offsets = torch.zeros(n_workers + 1, dtype=i64, device=dev)
        self.seg_offsets = torch.empty(self.uniq_cap + 1, dtype=i64, device=dev)
        self.sorted_occ = torch.empty(max(max_nnz, 1), dtype=i32, device=dev)
        self.uniq_grads = torch.empty(self.uniq_cap, dim, dtype=f32, device=dev)
        self.agg_ids = torch.empty(self.agg_cap, dtype=i32, device=dev)
        self.agg_grads = torch.empty(self.agg_cap, dim, dtype=f32, device=dev)
        self.n_agg = torch.zeros(1, dtype=i64, device=dev)
        self.status = torch.zeros(1, dtype=i32, device=dev)
        self.dense_out = torch.empty(dense_n, dtype=f32, device=dev) if dense_n else None
        ws_bytes = B.antdt_bsp_step_workspace_bytes(max_nnz, max_bags, dim, n_workers, self.uniq_cap)
        self.ws = torch.empty((ws_bytes + 255) // 256 * 256, dtype=torch.uint8, device=dev)


def run_step(buf: StepBuffers, table, state0, state1, oc: OptConfig, step: int, row_ids,
             bag_offsets, bags_per_sample: int, d_pooled, worker_sample_offsets: Sequence[int],
             batch_sizes: Sequence[int], dense_grads=None, stream=None):
    """fwd -> bwd_dedup -> weighted_aggregate -> sparse_opt_update, asynchronous."""
    n_bags = bag_offsets.numel() - 1
    nnz = row_ids.numel()
    B.antdt_embbag_fwd(table, row_ids, bag_offsets, buf.pooled[:n_bags], buf.status, stream)
    B.antdt_embbag_bwd_dedup(row_ids, bag_offsets, bags_per_sample, d_pooled, table.shape[0],
                             worker_sample_offsets, buf.uniq_ids, buf.worker_uniq_offsets,
                             buf.seg_offsets, buf.sorted_occ[:max(nnz, 1)] if nnz else buf.sorted_occ[:0],
                             buf.uniq_grads, buf.ws, buf.status, stream)
    B.antdt_weighted_aggregate(batch_sizes, buf.ws, n_rows=table.shape[0], uniq_ids=buf.uniq_ids,
                               worker_uniq_offsets=buf.worker_uniq_offsets,
                               uniq_grads=buf.uniq_grads, agg_ids=buf.agg_ids,
                               agg_grads=buf.agg_grads, n_agg=buf.n_agg, dense_grads=dense_grads,
                               dense_out=buf.dense_out, dev_status=buf.status, stream=stream)
    B.antdt_sparse_opt_update(table, buf.agg_ids, buf.agg_grads, buf.n_agg, oc.opt, oc.lr, oc.eps,
                              oc.beta1, oc.beta2, step, state0, state1, buf.status, stream)


class DeviceStep:
    """One antdt_bsp_step_device call per step: the descriptor is filled once for a buffer set and
    a model state, only the batch pointers and the step number change."""

    def __init__(self, buf: StepBuffers, table, state0, state1, oc: OptConfig, n_workers: int,
                 fuse_update: bool = False):
        import ctypes as C
        self.buf, self.K = buf, n_workers
        d = B.StepDesc()
        d.fuse_update = 1 if fuse_update else 0
        p = lambda t: None if t is None else t.data_ptr()  # noqa: E731
        d.table, d.dtype = p(table), (B.BF16 if table.dtype == torch.bfloat16 else B.F32)
        d.n_rows, d.dim = table.shape
        d.state0, d.state1 = p(state0), p(state1)
        d.opt, d.lr, d.eps, d.beta1, d.beta2 = oc.opt, oc.lr, oc.eps, oc.beta1, oc.beta2
        d.n_workers = n_workers
        d.d_pooled_out, d.d_dense_out = p(buf.pooled), p(buf.dense_out)
        d.d_uniq_ids, d.d_worker_uniq_offsets = p(buf.uniq_ids), p(buf.worker_uniq_offsets)
        d.d_seg_offsets, d.d_sorted_occ = p(buf.seg_offsets), p(buf.sorted_occ)
        d.d_uniq_grads, d.uniq_cap = p(buf.uniq_grads), buf.uniq_cap
        d.d_agg_ids, d.d_agg_grads, d.d_n_agg, d.agg_cap = p(buf.agg_ids), p(buf.agg_grads), p(buf.n_agg), buf.agg_cap
        d.ws, d.ws_bytes, d.d_status = p(buf.ws), buf.ws.numel(), p(buf.status)
        self.desc = d
        self._wso = (C.c_int64 * (n_workers + 1))()
        self._bsz = (C.c_int64 * n_workers)()
        d.worker_sample_offsets = C.cast(self._wso, C.c_void_p)
        d.batch_sizes = C.cast(self._bsz, C.c_void_p)

    def run(self, step: int, row_ids, bag_offsets, bags_per_sample: int, d_pooled,
            worker_sample_offsets: Sequence[int], batch_sizes: Sequence[int], dense_grads=None,
            stream=None, graph: bool = False):
        """graph=True replays the step as one CUDA graph launch (antdt_bsp_step_graph)."""
        d = self.desc
        d.step = step
        d.d_row_ids, d.nnz = row_ids.data_ptr(), row_ids.numel()
        d.d_bag_offsets, d.n_bags = bag_offsets.data_ptr(), bag_offsets.numel() - 1
        d.bags_per_sample = bags_per_sample
        d.d_d_pooled = d_pooled.data_ptr()
        d.d_dense_grads = None if dense_grads is None else dense_grads.data_ptr()
        d.dense_n = 0 if dense_grads is None else dense_grads.shape[1]
        self._wso[:] = [int(x) for x in worker_sample_offsets]
        self._bsz[:] = [int(x) for x in batch_sizes]
        if graph:
            B.antdt_bsp_step_graph(d, stream)
        else:
            B.antdt_bsp_step_device(d, stream)


class HostStaging:
    """One set of the buffers antdt_bsp_step_host copies through: device staging for the inputs,
    device and page-locked host buffers for the results.  A caller that keeps two of these and
    alternates them may have two steps in flight (staging_idle in the descriptor)."""

    def __init__(self, dim: int, n_workers: int, max_nnz: int, max_bags: int, dense_n: int = 0,
                 device="cuda"):
        dev = torch.device(device)
        i32, i64, f32 = torch.int32, torch.int64, torch.float32
        self.d_row_ids = torch.empty(max(max_nnz, 1), dtype=i32, device=dev)
        self.d_bag_offsets = torch.empty(max_bags + 1, dtype=i64, device=dev)
        self.d_d_pooled = torch.empty(max(max_bags, 1), dim, dtype=f32, device=dev)
        self.d_dense_grads = torch.empty(n_workers, dense_n, dtype=f32, device=dev) if dense_n else None
        self.d_pooled_out = torch.empty(max(max_bags, 1), dim, dtype=f32, device=dev)
        self.d_dense_out = torch.empty(dense_n, dtype=f32, device=dev) if dense_n else None
        self.d_n_agg = torch.zeros(1, dtype=i64, device=dev)
        self.d_status = torch.zeros(1, dtype=i32, device=dev)
        self.h_pooled = torch.empty(max(max_bags, 1), dim, dtype=f32).pin_memory()
        self.h_dense_out = torch.empty(dense_n, dtype=f32).pin_memory() if dense_n else None
        self.h_n_agg = torch.zeros(1, dtype=i64).pin_memory()
        self.h_status = torch.zeros(1, dtype=i32).pin_memory()
        self.done = torch.cuda.Event()   # recorded by HostStep.run after the call


class HostStep:
    """antdt_bsp_step_host for a model state and a buffer set; `run` fills the descriptor for one
    batch given as page-locked host tensors and one HostStaging set."""

    def __init__(self, buf: StepBuffers, table, state0, state1, oc: OptConfig, n_workers: int,
                 fuse_update: bool = False):
        import ctypes as C
        self._inner = DeviceStep(buf, table, state0, state1, oc, n_workers, fuse_update)
        self._C = C

    def run(self, st: HostStaging, step: int, h_row_ids, h_bag_offsets, bags_per_sample: int,
            h_d_pooled, worker_sample_offsets: Sequence[int], batch_sizes: Sequence[int],
            h_dense_grads=None, stream=None, staging_idle: bool = False):
        d = self._inner.desc
        p = lambda t: None if t is None else t.data_ptr()  # noqa: E731
        d.step = step
        d.h_row_ids, d.nnz = p(h_row_ids), h_row_ids.numel()
        d.h_bag_offsets, d.n_bags = p(h_bag_offsets), h_bag_offsets.numel() - 1
        d.bags_per_sample = bags_per_sample
        d.h_d_pooled, d.h_dense_grads = p(h_d_pooled), p(h_dense_grads)
        d.dense_n = 0 if h_dense_grads is None else h_dense_grads.shape[1]
        self._inner._wso[:] = [int(x) for x in worker_sample_offsets]
        self._inner._bsz[:] = [int(x) for x in batch_sizes]
        d.d_row_ids, d.d_bag_offsets, d.d_d_pooled = p(st.d_row_ids), p(st.d_bag_offsets), p(st.d_d_pooled)
        d.d_dense_grads, d.d_pooled_out, d.d_dense_out = p(st.d_dense_grads), p(st.d_pooled_out), p(st.d_dense_out)
        d.d_n_agg, d.d_status = p(st.d_n_agg), p(st.d_status)
        d.h_pooled, d.h_dense_out = p(st.h_pooled), p(st.h_dense_out)
        d.h_n_agg, d.h_status = p(st.h_n_agg), p(st.h_status)
        d.staging_idle = 1 if staging_idle else 0
        B.antdt_bsp_step_host(d, stream)
        st.done.record(stream if stream is not None else torch.cuda.current_stream())
