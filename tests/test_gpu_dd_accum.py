"""AntDT-DD with gradient accumulation (Section VI-B, Eq. 4) end to end on the device.

antdt_dd_solve gives every device type its micro-batch size B_i and accumulation count C_i;
a device of that type enters the step with a local batch of C_i * B_i samples.  The device path
(antdt_embbag_bwd_dedup, then antdt_weighted_aggregate with weights C_i * B_i / B) must give
what the accumulating checker gives: per device the mean of its C_i micro-batch mean gradients,
then the mean over the global batch."""
import numpy as np
import pytest

import oracle
from paper_2404_09679_b200 import binding as B
from tests import gpu_util as G
from tests.util import random_bags

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bmax", [(48, 48), (48, 24)])
def test_dd_plan_with_accumulation_through_the_device_path(bmax):
    # the paper's GPU cluster: 4 V100 + 4 P100, V100 about 3x a P100, global batch 768; micro-batch
    # caps below the shares 144 / 48 force accumulation
    n_dev, speeds, Bg = [4, 4], [3.0, 1.0], 768
    b, c, z = B.antdt_dd_solve(n_dev, speeds, Bg, [8, 8], list(bmax), 1, 6)
    ob, oc, oz = oracle.dd_solve(n_dev, speeds, Bg, [8, 8], list(bmax), 1, 6)
    assert (b, c, z) == (ob.tolist(), oc.tolist(), oz)
    assert max(c) > 1 and sum(n * ci * bi for n, ci, bi in zip(n_dev, c, b)) == Bg
    assert [ci * bi for ci, bi in zip(c, b)] == [144, 48]       # the continuous optimum is met

    # one simulated worker per device: local batch C_i * B_i, C_i micro-batches back to back
    micro = np.array([c[0]] * 4 + [c[1]] * 4, np.int64)
    local = np.array([c[0] * b[0]] * 4 + [c[1] * b[1]] * 4, np.int64)
    wso = np.concatenate([[0], np.cumsum(local)]).astype(np.int64)
    rng = np.random.default_rng(71)
    V, D, F, K = 5000, 32, 6, 8
    ids, off = random_bags(rng, Bg * F, V, 6, allow_empty=False, zipf=1.15)
    dY = rng.normal(size=(Bg * F, D)).astype(np.float32)

    want = oracle.embbag_bwd_accum(ids, off, F, dY, V, wso, micro)
    got = G.gpu_bwd(ids, off, F, dY, V, wso)
    assert got["status"] == 0
    assert np.array_equal(got["worker_uniq_offsets"], want["worker_uniq_offsets"])
    assert np.array_equal(got["uniq_ids"], want["uniq_ids"])
    G.close(got["uniq_grads"], want["uniq_grads"])

    # server side, per call on identical inputs: the checker's accumulated gradients in
    want_ids, want_agg = oracle.aggregate_sparse(want["uniq_ids"], want["worker_uniq_offsets"],
                                                 want["uniq_grads"], local)
    a_ids, a_g, na, _, code = G.gpu_aggregate(want["uniq_ids"], want["worker_uniq_offsets"],
                                              want["uniq_grads"], local, V)
    assert code == 0 and na == len(want_ids) and np.array_equal(a_ids, want_ids)
    G.close(a_g, want_agg)
    # and the chain on the device's own gradients equals the mean over the global batch, which
    # needs no notion of devices or micro-batches at all
    c_ids, c_g, _, _, code = G.gpu_aggregate(got["uniq_ids"], got["worker_uniq_offsets"],
                                             got["uniq_grads"], local, V)
    one = oracle.embbag_bwd_dedup(ids, off, F, dY, V, np.array([0, Bg], np.int64))
    assert code == 0 and np.array_equal(c_ids, one["uniq_ids"])
    G.close(c_g, one["uniq_grads"], rtol=3e-5, atol=2e-6)
