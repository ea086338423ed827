"""Shared test helpers (no method arithmetic of the CUDA path, none of the oracle's)."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            out[k] = float(v)
    return out


def csr_to_dense(row_ptr, col_idx, vals, D, dtype=np.float64):
    B = len(row_ptr) - 1
    X = np.zeros((B, D), dtype=dtype)
    for s in range(B):
        for i in range(row_ptr[s], row_ptr[s + 1]):
            X[s, col_idx[i]] = vals[i]
    return X


def label_matrix(label_ptr, labels, N, dtype=np.float64):
    """Y[s, j] = 1/|Y_s| for the distinct labels of sample s."""
    B = len(label_ptr) - 1
    Y = np.zeros((B, N), dtype=dtype)
    for s in range(B):
        ys = np.unique(labels[label_ptr[s]:label_ptr[s + 1]])
        Y[s, ys] = 1.0 / len(ys)
    return Y


def small_batch(rng, B, D, N, nnz, max_labels=3, dtype=np.float64):
    cols, vals, labs = [], [], []
    row_ptr = np.zeros(B + 1, dtype=np.int32)
    label_ptr = np.zeros(B + 1, dtype=np.int32)
    for s in range(B):
        n = int(rng.integers(1, nnz + 1))
        ids = np.sort(rng.choice(D, size=n, replace=False)).astype(np.int32)
        cols.append(ids)
        vals.append((rng.standard_normal(n)).astype(dtype))
        ny = int(rng.integers(1, max_labels + 1))
        labs.append(rng.choice(N, size=ny, replace=False).astype(np.int32))
        row_ptr[s + 1] = row_ptr[s] + n
        label_ptr[s + 1] = label_ptr[s] + ny
    return row_ptr, np.concatenate(cols), np.concatenate(vals), label_ptr, np.concatenate(labs)


def max_rel_err(a, b, floor_frac=1e-3):
    """max_i |a_i - b_i| / max(|a_i|, |b_i|, floor), floor = floor_frac * the tensor's largest magnitude.

    The floor keeps elements that are (near) zero through cancellation from turning a
    rounding-level absolute difference into a huge relative one.
    """
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    assert a.shape == b.shape
    if a.size == 0:
        return 0.0
    scale = max(np.max(np.abs(a)), np.max(np.abs(b)), 1e-30)
    den = np.maximum(np.maximum(np.abs(a), np.abs(b)), floor_frac * scale)
    return float(np.max(np.abs(a - b) / den))
