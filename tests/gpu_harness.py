"""Pairs a CUDA context (through the C ABI binding) with the CPU oracle on the same state and inputs."""
import numpy as np
import torch

from oracle.oracle import Oracle
from paper_2201_12667_b200 import binding as ds

WEIGHTS = ["W1", "b1", "W2", "b2"]
MOMENTS = ["mW1", "vW1", "mb1", "vb1", "mW2", "vW2", "mb2", "vb2"]


def to_dev(batch):
    return [torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in batch]


class Pair:
    """oracle (fp32) + GPU context with identical configuration; the GPU gets the oracle's weights."""

    def __init__(self, D, H, N, family, K, L, bucket_cap, max_batch, bin_size=8, srp_nnz=0, max_labels=16,
                 rebuild_period0=0, rebuild_lambda=0.0, redraw=1, force_dense=0, max_active=0, lr=1e-3,
                 init_std=0.05, seed=0, dedup_mode=0, sync_weights=True, densify=0, budget=0, budget_fill=0,
                 inputs_ready=0, oracle_build="float", hidden_K=0, hidden_L=0, hidden_cap=0):
        self.o = Oracle(oracle_build, D=D, H=H, N=N, family=family, K=K, L=L, bin_size=bin_size, srp_nnz=srp_nnz,
                        bucket_cap=bucket_cap, rebuild_period0=rebuild_period0, rebuild_lambda=rebuild_lambda,
                        redraw=redraw, force_dense=force_dense, max_active=max_active, lr=lr, init_std=init_std,
                        seed=seed, densify=densify, budget=budget, budget_fill=budget_fill, hidden_K=hidden_K,
                        hidden_L=hidden_L, hidden_cap=hidden_cap)
        self.cfg = ds.make_config(input_dim=D, hidden_dim=H, output_dim=N, hash_family=family, K=K, L=L,
                                  dwta_bin_size=bin_size, srp_nnz=srp_nnz, bucket_cap=bucket_cap,
                                  rebuild_period0=rebuild_period0, rebuild_growth_lambda=rebuild_lambda,
                                  redraw_hash_fns=redraw, force_dense=force_dense, max_batch=max_batch,
                                  max_labels=max_labels, max_active_per_sample=max_active, lr=lr, init_std=init_std,
                                  seed=seed, dedup_mode=dedup_mode, dwta_densify=densify, sample_budget=budget, budget_fill=budget_fill,
                                  inputs_ready=inputs_ready, hidden_K=hidden_K, hidden_L=hidden_L, hidden_cap=hidden_cap)
        self.ctx = ds.dslide_init(self.cfg)
        self.D, self.H, self.N, self.L, self.K = D, H, N, L, K
        self.dense = bool(force_dense)
        self.max_batch = max_batch
        if sync_weights:
            self.push_state()

    def close(self):
        if self.ctx is not None:
            ds.dslide_destroy(self.ctx)
            self.ctx = None
        self.o.close()

    def push_state(self, moments=False, counters=False):
        """oracle -> GPU: weights (and optionally Adam moments and counters), then rebuild the GPU tables."""
        for n in WEIGHTS + (MOMENTS if moments else []):
            ds.dslide_set_tensor(self.ctx, n, self.o.view(n))
        if not self.dense:
            ds.dslide_set_tensor(self.ctx, "hash_idx", self.o.view("hash_idx"))
            if len(self.o.view("hash_sign")):
                ds.dslide_set_tensor(self.ctx, "hash_sign", self.o.view("hash_sign"))
        if len(self.o.view("proj1")):
            ds.dslide_set_tensor(self.ctx, "proj1", self.o.view("proj1"))
        if counters:
            ds.dslide_set_tensor(self.ctx, "counters", np.array([self.o.t, self.o.r, self.o.next_rebuild], dtype=np.int64))
        ds.dslide_build_tables(self.ctx)
        ds.dslide_sync(self.ctx)

    def gpu_step(self, batch, host=False):
        B = len(batch[0]) - 1
        if host:
            return ds.dslide_train_step_host(self.ctx, B, *batch)
        dev = to_dev(batch)
        loss = torch.zeros(1, device="cuda")
        ds.dslide_train_step(self.ctx, B, *dev, loss)
        ds.dslide_sync(self.ctx)
        return float(loss.item())

    def gpu_active_sets(self, B):
        cnt = ds.dslide_get_last(self.ctx, "act_count", B)
        if self.dense:
            return [np.arange(self.N, dtype=np.int32) for _ in range(B)], cnt
        ids = ds.dslide_get_last(self.ctx, "act_ids", B)
        return [ids[s, :cnt[s]].copy() for s in range(B)], cnt

    def gpu_ragged(self, name, B, cnt):
        a = ds.dslide_get_last(self.ctx, name, B)
        return np.concatenate([a[s, :cnt[s]] for s in range(B)]) if B else a
