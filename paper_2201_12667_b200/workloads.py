"""Seeded synthetic workloads shaped like the paper's extreme-classification data.

This module only draws inputs (CSR feature rows and label lists) and names
the model shapes they go with.  It holds none of the method's arithmetic and
is the one module both the CUDA path's callers and the CPU oracle's tests
use.  The real datasets of the paper (Table 1) are not available; these
batches have their shapes and statistics only: feature and label ids follow
a Zipf law through a seeded permutation, values are lognormal and rows are
L2-normalised.
"""
import numpy as np

SIMHASH, DWTA = 0, 1

# name -> model shape + hashing + batch statistics
CONFIGS = {
    # small case the CPU oracle finishes in seconds
    "tiny": dict(D=1000, H=32, N=2000, family=SIMHASH, K=4, L=8, bin_size=8, srp_nnz=0, bucket_cap=64,
                 batch=32, mean_nnz=20, mean_labels=2, dist="uniform", lr=1e-3, max_labels=3),
    # the headline shape (Table 1, first dataset: 135,909 features, 670,091 labels)
    "670k": dict(D=135909, H=128, N=670091, family=DWTA, K=6, L=50, bin_size=8, srp_nnz=0, bucket_cap=128,
                 batch=256, mean_nnz=76, mean_labels=5, dist="zipf", lr=1e-4, max_labels=16),
    "325k": dict(D=1617899, H=128, N=325056, family=SIMHASH, K=9, L=50, bin_size=8, srp_nnz=0, bucket_cap=128,
                 batch=256, mean_nnz=42, mean_labels=3, dist="zipf", lr=1e-4, max_labels=16),
    "1b": dict(D=200000, H=256, N=4000000, family=DWTA, K=7, L=64, bin_size=8, srp_nnz=0, bucket_cap=256,
               batch=512, mean_nnz=100, mean_labels=4, dist="zipf", lr=1e-4, max_labels=16),
    # the paper's second dataset (Table 1: 253,855 words in and out, about one nonzero per sample; Table 3: hidden
    # layer 200, batch 1024 or 2048): one-hot inputs, a few context words as labels
    "text8": dict(D=253855, H=200, N=253855, family=SIMHASH, K=9, L=50, bin_size=8, srp_nnz=0, bucket_cap=128,
                  batch=1024, mean_nnz=1, fixed_nnz=1, mean_labels=4, dist="zipf", lr=1e-4, max_labels=16),
    # the 670K shape with the large hidden layer and batch of Table 3
    "670k-h1024": dict(D=135909, H=1024, N=670091, family=DWTA, K=6, L=50, bin_size=8, srp_nnz=0, bucket_cap=128,
                       batch=1024, mean_nnz=76, mean_labels=5, dist="zipf", lr=1e-4, max_labels=16),
    # the shape of the low-bandwidth experiment (Section 4.7: hidden layer 256, batch 2048) on the first dataset's dimensions
    "670k-h256-b2048": dict(D=135909, H=256, N=670091, family=DWTA, K=6, L=50, bin_size=8, srp_nnz=0, bucket_cap=128,
                            batch=2048, mean_nnz=76, mean_labels=5, dist="zipf", lr=1e-4, max_labels=16),
    # Table 3's batch of 2048 with the large hidden layer
    "670k-h1024-b2048": dict(D=135909, H=1024, N=670091, family=DWTA, K=6, L=50, bin_size=8, srp_nnz=0, bucket_cap=128,
                             batch=2048, mean_nnz=76, mean_labels=5, dist="zipf", lr=1e-4, max_labels=16),
    "text8-b2048": dict(D=253855, H=200, N=253855, family=SIMHASH, K=9, L=50, bin_size=8, srp_nnz=0, bucket_cap=128,
                        batch=2048, mean_nnz=1, fixed_nnz=1, mean_labels=4, dist="zipf", lr=1e-4, max_labels=16),
    # a mid-size shape for parity tests: several tiles, ragged tails, both dedup paths
    "mid": dict(D=5003, H=128, N=20011, family=DWTA, K=3, L=10, bin_size=8, srp_nnz=0, bucket_cap=16,
                batch=48, mean_nnz=30, mean_labels=3, dist="zipf", lr=1e-3, max_labels=16),
}

ZIPF_S = 1.1


def config(name, **overrides):
    c = dict(CONFIGS[name])
    c.update(overrides)
    c["name"] = name
    return c


class _Zipf:
    """ids in [0, M) with P(rank k) ~ k^-s, rank -> id through a seeded permutation."""

    def __init__(self, M, s, seed):
        w = np.arange(1, M + 1, dtype=np.float64) ** (-s)
        self.cdf = np.cumsum(w)
        self.cdf /= self.cdf[-1]
        self.perm = np.random.Generator(np.random.PCG64(seed)).permutation(M).astype(np.int32)
        self.M = M

    def distinct(self, rng, n):
        """n distinct ids, in order of first appearance."""
        n = min(n, self.M)
        out = np.zeros(0, dtype=np.int32)
        while len(out) < n:
            r = np.searchsorted(self.cdf, rng.random(3 * n + 8), side="right")
            r = np.minimum(r, self.M - 1)
            cand = np.concatenate([out, self.perm[r]])
            _, first = np.unique(cand, return_index=True)
            out = cand[np.sort(first)]
        return out[:n]


class Workload:
    """Batches for one named config.  batch(i) is a pure function of (config, seed, i)."""

    def __init__(self, cfg, seed=0):
        self.cfg = cfg
        self.seed = seed
        if cfg["dist"] == "zipf":
            self.feat = _Zipf(cfg["D"], ZIPF_S, seed * 7919 + 11)
            self.lab = _Zipf(cfg["N"], ZIPF_S, seed * 7919 + 13)

    def batch(self, i, batch_size=None):
        """-> row_ptr[B+1] i32, col_idx i32 (ascending in a row), vals f32, label_ptr[B+1] i32, labels i32."""
        c = self.cfg
        B = batch_size or c["batch"]
        rng = np.random.Generator(np.random.PCG64([self.seed, i, 0x5EED]))
        cols, vals, labs = [], [], []
        row_ptr = np.zeros(B + 1, dtype=np.int32)
        label_ptr = np.zeros(B + 1, dtype=np.int32)
        for s in range(B):
            if c["dist"] == "uniform":
                nnz = min(c["mean_nnz"], c["D"])
                ids = rng.choice(c["D"], size=nnz, replace=False).astype(np.int32)
                v = (1.0 - rng.random(nnz)).astype(np.float32)          # U(0,1]
                ny = int(rng.integers(1, c["max_labels"] + 1))
                y = rng.choice(c["N"], size=ny, replace=False).astype(np.int32)
            else:
                nnz = c.get("fixed_nnz") or int(np.clip(rng.poisson(c["mean_nnz"]), 1, min(4 * c["mean_nnz"], c["D"])))
                ids = self.feat.distinct(rng, nnz)
                v = np.exp(rng.standard_normal(nnz))
                v = (v / np.sqrt(np.sum(v * v))).astype(np.float32)
                ny = int(np.clip(rng.poisson(c["mean_labels"] - 1) + 1, 1, c["max_labels"]))
                y = self.lab.distinct(rng, ny)
            order = np.argsort(ids, kind="stable")
            cols.append(ids[order])
            vals.append(v[order])
            labs.append(y)
            row_ptr[s + 1] = row_ptr[s] + len(ids)
            label_ptr[s + 1] = label_ptr[s] + len(y)
        return (row_ptr, np.concatenate(cols).astype(np.int32), np.concatenate(vals).astype(np.float32),
                label_ptr, np.concatenate(labs).astype(np.int32))
