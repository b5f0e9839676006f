"""Seeded synthetic inputs for the BSP sparse-ranking step.

Everything here is input generation only: counter-based hashing, the samplers that shape the
ids (Zipf ranks, bag lengths), normal draws for gradients and table initialisation, worker
speeds.  None of the method's arithmetic (pooling, dedup, aggregation, optimizer) lives here.

All draws are pure functions of (seed, stream tag, coordinates), built from the splitmix64
finaliser (Steele, Lea, Flood 2014), so a dataset sample's content depends on its global index
only -- whichever worker the shard service hands it to -- and any slice of a tensor can be
produced without producing the rest.  The functions are written with torch integer/float64
ops and take a `device`, so the large workloads can be produced directly in GPU memory; the
tensors they return are the inputs of BOTH the CUDA path and the CPU checker.

The inputs stand in for the workloads the paper trains on (Section VII-A.2: XDeepFM on the
Criteo click logs, and a production ranking model); no record of either is reproduced.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence, Tuple

import torch

# stream tags
TAG_LEN, TAG_ID, TAG_ROW, TAG_DY, TAG_DENSE, TAG_TABLE, TAG_SPEED, TAG_SLOW = range(1, 9)

_M64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Python int -> the signed 64-bit value with the same bits."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_GAMMA = _s64(0x9E3779B97F4A7C15)
_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 lanes (torch's >> is arithmetic)."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def mix64(z: torch.Tensor) -> torch.Tensor:
    """splitmix64 output function on int64 lanes (wrap-around arithmetic)."""
    z = z + _GAMMA
    z = (z ^ _lsr(z, 30)) * _C1
    z = (z ^ _lsr(z, 27)) * _C2
    return z ^ _lsr(z, 31)


def mix64_int(z: int) -> int:
    """The same function on one Python integer (unsigned result)."""
    z = (z + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def hash_coords(seed: int, tag: int, *coords) -> torch.Tensor:
    """Hash of (seed, tag, c0, c1, ...); coords are int64 tensors (broadcast) or ints."""
    h0 = _s64(mix64_int(((seed & 0xFFFFFFFF) << 8) ^ tag))
    h: Optional[torch.Tensor] = None
    for c in coords:
        if h is None:
            if not torch.is_tensor(c):
                h0 = _s64(mix64_int((h0 ^ c) & _M64))
                continue
            h = mix64(c ^ h0)
        else:
            h = mix64(h ^ c)
    if h is None:
        raise ValueError("at least one tensor coordinate is needed")
    return h


def uniform01(h: torch.Tensor) -> torch.Tensor:
    """Top 53 bits of a hash as a float64 in [0, 1)."""
    return _lsr(h, 11).to(torch.float64) * (2.0 ** -53)


def normal01(h: torch.Tensor) -> torch.Tensor:
    """Standard normal (float64) from one hash by Box-Muller on two derived uniforms."""
    u1 = uniform01(mix64(h ^ 0x5851F42D4C957F2D))
    u2 = uniform01(mix64(h ^ 0x14057B7EF767814F))
    return torch.sqrt(-2.0 * torch.log1p(-u1)) * torch.cos((2.0 * math.pi) * u2)


class ZipfTable:
    """Exact inverse-CDF sampler of P(r) ~ r^-s on the finite support r = 1..V."""

    def __init__(self, V: int, s: float, device):
        r = torch.arange(1, V + 1, dtype=torch.float64, device=device)
        w = r.pow_(-s)
        self.cdf = torch.cumsum(w, 0)
        self.cdf /= self.cdf[-1].clone()
        self.V = V

    def rank(self, u: torch.Tensor) -> torch.Tensor:
        """u in [0,1) -> rank in 1..V (int64)."""
        r = torch.searchsorted(self.cdf, u, right=True) + 1
        return r.clamp_(max=self.V)


class LengthSampler:
    """Bag-length distributions: uniform on lo..hi, fixed, or Poisson(mean) clamped to lo..hi."""

    def __init__(self, kind: str, lo: int, hi: int, mean: float, device):
        self.kind, self.lo, self.hi = kind, lo, hi
        if kind == "poisson":
            kmax = max(hi, int(mean * 4) + 20)
            k = torch.arange(0, kmax + 1, dtype=torch.float64)
            logp = k * math.log(mean) - mean - torch.lgamma(k + 1.0)
            self.cdf = torch.cumsum(torch.exp(logp), 0).to(device)

    def sample(self, h: torch.Tensor) -> torch.Tensor:
        if self.kind == "fixed":
            return torch.full_like(h, self.lo)
        u = uniform01(h)
        if self.kind == "uniform":
            n = self.hi - self.lo + 1
            return (u * n).floor().to(torch.int64).clamp_(max=n - 1) + self.lo
        k = torch.searchsorted(self.cdf, u, right=True)
        return k.clamp_(min=self.lo, max=self.hi)  # clamp, not rejection


@dataclasses.dataclass(frozen=True)
class Workload:
    """One of the five step configurations (sizes and distributions only)."""
    name: str
    seed: int
    K: int                       # simulated workers
    B: int                       # global batch
    F: int                       # fields = bags per sample
    V: int                       # total table rows
    D: int                       # embedding dim
    table_dtype: str             # "f32" | "bf16"
    shared_table: bool           # True: fields hashed into one table; False: V/F rows per field
    len_kind: str                # "uniform" | "fixed" | "poisson"
    len_lo: int
    len_hi: int
    len_mean: float
    zipf_s: float
    dense_n: int                 # 0: no dense part
    opt: str                     # "adagrad" | "adam"
    lr: float
    eps: float
    beta1: float
    beta2: float
    steps: int
    speed_kind: str              # "fixed" | "lognormal_once" | "lognormal_step" | "equal"
    speed_sigma: float
    fixed_speeds: Tuple[float, ...]
    n_slowed: int                # workers divided by 4 each step (straggler sweep)
    rule: str                    # "proportional" | "minmax"
    min_batch: int
    M: int = 100                 # batches per shard (the paper's default, Section VII-A.4)
    init_std: float = 0.01
    dense_std: float = 1e-2

    @property
    def n_samples(self) -> int:
        """Virtual dataset: long enough that no measured step falls in the epoch tail."""
        return 8 * self.K * self.B * self.M

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _cfg(**kw) -> Workload:
    base = dict(dense_n=0, lr=0.01, eps=1e-8, beta1=0.9, beta2=0.999, speed_sigma=0.0,
                fixed_speeds=(), n_slowed=0, rule="proportional", min_batch=0, len_mean=0.0)
    base.update(kw)
    return Workload(**base)


WORKLOADS = {
    1: _cfg(name="c1_tiny", seed=0, K=4, B=512, F=8, V=80_000, D=16, table_dtype="f32",
            shared_table=False, len_kind="uniform", len_lo=1, len_hi=4, zipf_s=1.1,
            opt="adagrad", steps=10, speed_kind="fixed", fixed_speeds=(64., 128., 128., 192.)),
    2: _cfg(name="c2_onehot_ctr", seed=1, K=8, B=16_384, F=26, V=26_000_000, D=32,
            table_dtype="f32", shared_table=False, len_kind="fixed", len_lo=1, len_hi=1,
            zipf_s=1.05, opt="adagrad", steps=50, speed_kind="fixed",
            fixed_speeds=(1., 1., 1., 1., 1., 1., .5, .25)),
    3: _cfg(name="c3_multihot_adam", seed=2, K=16, B=65_536, F=100, V=10_000_000, D=64,
            table_dtype="f32", shared_table=True, len_kind="poisson", len_lo=1, len_hi=50,
            len_mean=10.0, zipf_s=1.1, dense_n=4_194_304, opt="adam", lr=1e-3, steps=20,
            speed_kind="lognormal_once", speed_sigma=0.3),
    4: _cfg(name="c4_hotrow_bf16", seed=3, K=16, B=131_072, F=40, V=100_000_000, D=64,
            table_dtype="bf16", shared_table=True, len_kind="poisson", len_lo=1, len_hi=100,
            len_mean=20.0, zipf_s=1.2, opt="adagrad", steps=10, speed_kind="equal"),
    5: _cfg(name="c5_straggler_sweep", seed=4, K=32, B=262_144, F=30, V=50_000_000, D=32,
            table_dtype="f32", shared_table=True, len_kind="uniform", len_lo=1, len_hi=8,
            zipf_s=1.05, dense_n=16_777_216, opt="adam", lr=1e-3, steps=20,
            speed_kind="lognormal_step", speed_sigma=0.5, n_slowed=2, min_batch=256),
}


def speeds_for_step(w: Workload, step: int) -> Optional[List[float]]:
    """Worker throughputs v_i handed to the planner for `step` (None = equal split)."""
    if w.speed_kind == "equal":
        return None
    if w.speed_kind == "fixed":
        return list(w.fixed_speeds)
    st = 0 if w.speed_kind == "lognormal_once" else step
    i = torch.arange(w.K, dtype=torch.int64)
    v = torch.exp(w.speed_sigma * normal01(hash_coords(w.seed, TAG_SPEED, st, i)))
    if w.n_slowed:
        order = torch.argsort(_lsr(hash_coords(w.seed, TAG_SLOW, step, i), 1), stable=True)
        v[order[: w.n_slowed]] /= 4.0
    return [float(x) for x in v]


def sample_indices(ranges: Sequence[Tuple[int, int]], device) -> torch.Tensor:
    """Concatenate (start, len) ranges of dataset indices into one int64 tensor."""
    parts = [torch.arange(s, s + n, dtype=torch.int64, device=device) for s, n in ranges if n > 0]
    if not parts:
        return torch.empty(0, dtype=torch.int64, device=device)
    return torch.cat(parts)


class BatchMaker:
    """Materialises bags, ids and upstream gradients of dataset samples for one workload."""

    def __init__(self, w: Workload, device="cpu"):
        self.w, self.device = w, torch.device(device)
        per = w.V if w.shared_table else w.V // w.F
        self.ranks = per
        self.zipf = ZipfTable(per, w.zipf_s, self.device)
        self.lens = LengthSampler(w.len_kind, w.len_lo, w.len_hi, w.len_mean, self.device)

    def bags(self, sample_idx: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
        """-> (row_ids int32 [nnz], bag_offsets int64 [n_bags+1]); bag = sample*F + field."""
        w, dev = self.w, self.device
        S = sample_idx.numel()
        f = torch.arange(w.F, dtype=torch.int64, device=dev)
        lens = self.lens.sample(hash_coords(w.seed, TAG_LEN, sample_idx[:, None], f[None, :]))
        lens = lens.reshape(-1)
        off = torch.zeros(S * w.F + 1, dtype=torch.int64, device=dev)
        torch.cumsum(lens, 0, out=off[1:])
        nnz = int(off[-1]) if S else 0
        bag = torch.repeat_interleave(torch.arange(S * w.F, dtype=torch.int64, device=dev), lens,
                                      output_size=nnz)
        slot = torch.arange(nnz, dtype=torch.int64, device=dev) - off[bag]
        smp = sample_idx[bag // w.F]
        fld = bag % w.F
        del bag
        rank = self.zipf.rank(uniform01(hash_coords(w.seed, TAG_ID, smp, fld, slot)))
        del smp, slot
        if w.shared_table:
            # field-salted hash of the rank into the shared table
            rows = _lsr(hash_coords(w.seed, TAG_ROW, fld, rank), 1) % w.V
        else:
            rows = fld * self.ranks + (rank - 1)
        return rows.to(torch.int32), off

    def d_pooled(self, sample_idx: torch.Tensor, chunk: int = 1 << 16) -> torch.Tensor:
        """Upstream gradient of the pooled output, N(0,1), fp32 [n_bags, D]."""
        w, dev = self.w, self.device
        S = sample_idx.numel()
        out = torch.empty(S * w.F, w.D, dtype=torch.float32, device=dev)
        f = torch.arange(w.F, dtype=torch.int64, device=dev)
        c = torch.arange(w.D, dtype=torch.int64, device=dev)
        for s0 in range(0, S, chunk):
            s = sample_idx[s0:s0 + chunk]
            h = hash_coords(w.seed, TAG_DY, s[:, None, None], f[None, :, None], c[None, None, :])
            out[s0 * w.F:(s0 + s.numel()) * w.F] = normal01(h).reshape(-1, w.D).to(torch.float32)
        return out

    def dense_grads(self, step: int, chunk: int = 1 << 22) -> Optional[torch.Tensor]:
        """Per-worker dense gradients N(0, dense_std), fp32 [K, dense_n]."""
        w, dev = self.w, self.device
        if not w.dense_n:
            return None
        out = torch.empty(w.K, w.dense_n, dtype=torch.float32, device=dev)
        for i in range(w.K):
            for e0 in range(0, w.dense_n, chunk):
                e = torch.arange(e0, min(e0 + chunk, w.dense_n), dtype=torch.int64, device=dev)
                h = hash_coords(w.seed, TAG_DENSE, step, i, e)
                out[i, e0:e0 + e.numel()] = (w.dense_std * normal01(h)).to(torch.float32)
        return out

    def table(self, chunk_rows: int = 1 << 20) -> torch.Tensor:
        """Initial table N(0, init_std) as a pure function of (row, col); f32 or bf16."""
        w, dev = self.w, self.device
        dt = torch.float32 if w.table_dtype == "f32" else torch.bfloat16
        out = torch.empty(w.V, w.D, dtype=dt, device=dev)
        c = torch.arange(w.D, dtype=torch.int64, device=dev)
        for r0 in range(0, w.V, chunk_rows):
            r = torch.arange(r0, min(r0 + chunk_rows, w.V), dtype=torch.int64, device=dev)
            h = hash_coords(w.seed, TAG_TABLE, r[:, None], c[None, :])
            out[r0:r0 + r.numel()] = (w.init_std * normal01(h)).to(torch.float32).to(dt)
        return out
