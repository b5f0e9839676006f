"""antdt_embbag_bwd_dedup_static -- the variant for callers that cannot allocate device memory
(allocator-free serving loops, plug-ins with a fixed memory budget, processes whose device memory
another framework owns) -- must give what antdt_embbag_bwd_dedup gives.  Its scratch is one
array inside the library that every call re-uses, so the check runs two different problems back
to back: the second call finds the first one's leftovers in the scratch.  This file sorts last on
purpose, so a run that stops at the first failure has already run every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_2404_09679_b200 import binding as B
from tests import gpu_util as G
from tests.util import random_bags

pytestmark = pytest.mark.gpu


def _static_bwd(ids, off, F, dY, n_rows, wso):
    nnz, D, K = ids.shape[0], dY.shape[1], len(wso) - 1
    cap = max(1, nnz)
    uid = torch.full((cap,), -1, dtype=torch.int32, device="cuda")
    wuo = torch.full((K + 1,), -1, dtype=torch.int64, device="cuda")
    so = torch.full((cap + 1,), -1, dtype=torch.int64, device="cuda")
    occ = torch.full((max(nnz, 1),), -1, dtype=torch.int32, device="cuda")
    ug = torch.full((cap, D), float("nan"), device="cuda")
    st = G.new_status()
    B.antdt_embbag_bwd_dedup_static(G.dev(ids), G.dev(off), F, G.dev(dY), n_rows,
                                    [int(x) for x in wso], uid, wuo, so, occ[:nnz], ug, st)
    assert B.antdt_read_status(st) == 0
    wuo_h = wuo.cpu().numpy()
    nu = int(wuo_h[K])
    return dict(uniq_ids=uid[:nu].cpu().numpy(), worker_uniq_offsets=wuo_h,
                seg_offsets=so[: nu + 1].cpu().numpy(), sorted_occ=occ[:nnz].cpu().numpy(),
                uniq_grads=ug[:nu].cpu().numpy())


def _problem(seed, V, D, K, F, S, maxlen, zipf):
    rng = np.random.default_rng(seed)
    ids, off = random_bags(rng, S * F, V, maxlen, zipf=zipf)
    dY = rng.normal(size=(S * F, D)).astype(np.float32)
    cuts = np.sort(rng.integers(0, S + 1, size=K - 1))
    wso = np.concatenate([[0], cuts, [S]]).astype(np.int64)
    return ids, off, F, dY, V, wso


def test_static_scratch_variant_matches_the_workspace_variant_twice_in_a_row():
    # first a large problem (long runs, many tiles), then a smaller, differently shaped one
    for n, args in enumerate((_problem(1, 3000, 64, 8, 6, 20_000, 9, 1.15),
                              _problem(2, 50_000, 16, 3, 4, 5000, 5, None))):
        want = G.gpu_bwd(*args)
        assert want["status"] == 0
        got = _static_bwd(*args)
        for k in ("worker_uniq_offsets", "uniq_ids", "seg_offsets", "sorted_occ"):
            assert np.array_equal(got[k], want[k]), k
        G.close(got["uniq_grads"], want["uniq_grads"])
        if n == 1:
            # the call that found leftovers in the scratch, against the CPU checker as well, so
            # that this file stands on its own
            ids, off, F, dY, V, wso = args
            ref = oracle.embbag_bwd_dedup(ids, off, F, dY, V, wso)
            for k in ("worker_uniq_offsets", "uniq_ids", "seg_offsets", "sorted_occ"):
                assert np.array_equal(got[k], ref[k]), k
            G.close(got["uniq_grads"], ref["uniq_grads"])


def test_static_scratch_variant_rejects_what_does_not_fit():
    L = B.lib()
    one = C.c_void_p(256)          # never dereferenced: the size check comes first
    wso = (C.c_int64 * 2)(0, 1)
    n0 = B.antdt_launch_count()
    too_many = 4_000_000           # needs far more than the 24 MiB array at dim 64
    assert B.antdt_embbag_bwd_dedup_min_workspace_bytes(too_many, 1, 64, 1) > B.STATIC_SCRATCH_BYTES
    rc = L.antdt_embbag_bwd_dedup_static(one, too_many, one, 1, 1, one, 64, 10, 1, wso, one, one, one,
                                         one, one, too_many, None, None)
    assert rc == B.ERR_CAPACITY
    assert B.antdt_launch_count() == n0
