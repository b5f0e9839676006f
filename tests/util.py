"""Shared helpers of the tests: golden-file reader and small brute-force builders (numpy)."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            k, v = [s.strip() for s in line.split("=", 1)]
            out[k] = float(v) if "." in v else int(v)
    return out


def random_bags(rng, n_bags, V, max_len, allow_empty=True, zipf=None):
    """Random CSR bags: -> (row_ids int32, bag_offsets int64)."""
    lo = 0 if allow_empty else 1
    lens = rng.integers(lo, max_len + 1, size=n_bags)
    off = np.zeros(n_bags + 1, np.int64)
    off[1:] = np.cumsum(lens)
    nnz = int(off[-1])
    if zipf:
        ids = np.minimum(rng.zipf(zipf, size=nnz) - 1, V - 1)
    else:
        ids = rng.integers(0, V, size=nnz)
    return ids.astype(np.int32), off


def count_matrix(row_ids, bag_offsets, V):
    """A[b, r] = number of times row r occurs in bag b (dense, float64)."""
    n_bags = bag_offsets.shape[0] - 1
    A = np.zeros((n_bags, V), np.float64)
    for b in range(n_bags):
        for j in range(bag_offsets[b], bag_offsets[b + 1]):
            A[b, row_ids[j]] += 1.0
    return A


def bf16_bits_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f32_to_bf16_bits_trunc_exact(x):
    """For values already representable in bf16: their bit pattern."""
    u = np.asarray(x, np.float32).view(np.uint32)
    assert np.all((u & 0xFFFF) == 0)
    return (u >> 16).astype(np.uint16)
