"""The step learns: precision@1 on planted data rises far above chance (run with -m gpu).

The paper's measure is accuracy on its datasets, which are not available; here the labels come from a hidden
teacher (each class owns a few characteristic features, a sample is drawn from one class), so that a
correct training step must drive precision@1 up.  This runs the whole path for a few hundred steps: sparse
forward, LSH sampling with scheduled rebuilds (new hash functions every time), sparse back-propagation, Adam on the
touched rows, and dslide_predict_topk both through the tables and over all classes.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2201_12667_b200 import binding as ds


def planted_batch(rng, B, D, N, proto, noise=4):
    """Sample s belongs to class y_s; its row holds that class's prototype features plus a few random ones."""
    cols, vals = [], []
    row_ptr = np.zeros(B + 1, dtype=np.int32)
    y = rng.integers(0, N, size=B).astype(np.int32)
    for s in range(B):
        ids = np.union1d(proto[y[s]], rng.choice(D, size=noise, replace=False)).astype(np.int32)
        v = (1.0 + 0.1 * rng.standard_normal(len(ids))).astype(np.float32)
        cols.append(ids)
        vals.append(v / np.sqrt(np.sum(v * v)))
        row_ptr[s + 1] = row_ptr[s] + len(ids)
    label_ptr = np.arange(B + 1, dtype=np.int32)
    return row_ptr, np.concatenate(cols), np.concatenate(vals), label_ptr, y


def precision_at_1(ctx, batch, dense):
    B = len(batch[0]) - 1
    dev = [torch.from_numpy(a).cuda() for a in batch[:3]]
    ids = torch.empty(B, dtype=torch.int32, device="cuda")
    sc = torch.empty(B, dtype=torch.float32, device="cuda")
    ds.dslide_predict_topk(ctx, B, *dev, 1, dense, ids, sc)
    ds.dslide_sync(ctx)
    return float((ids.cpu().numpy() == batch[4]).mean())


@pytest.mark.parametrize("family,K,L,hidden", [(1, 2, 24, None), (0, 4, 24, None),
                                                (1, 2, 24, dict(hidden_K=2, hidden_L=10, hidden_cap=32))])
def test_precision_rises_on_planted_data(family, K, L, hidden):
    """The third case samples the hidden layer too (tables over the hidden neurons, queried with the sparse input)."""
    D, H, N, B = 1000, 64, 1000, 128
    rng = np.random.default_rng(0)
    proto = [rng.choice(D, size=6, replace=False) for _ in range(N)]
    cfg = ds.make_config(input_dim=D, hidden_dim=H, output_dim=N, hash_family=family, K=K, L=L, bucket_cap=64,
                         rebuild_period0=25, rebuild_growth_lambda=0.05, redraw_hash_fns=1, max_batch=B, max_labels=2,
                         lr=5e-3, init_std=0.05, seed=3, **(hidden or {}))
    ctx = ds.dslide_init(cfg)
    try:
        test = planted_batch(np.random.default_rng(1), B, D, N, proto)
        before = precision_at_1(ctx, test, dense=1)
        losses = []
        for step in range(600):
            losses.append(ds.dslide_train_step_host(ctx, B, *planted_batch(rng, B, D, N, proto)))
        after_dense = precision_at_1(ctx, test, dense=1)
        after_lsh = precision_at_1(ctx, test, dense=0)
        assert ds.dslide_get_tensor(ctx, "counters")[1] >= 8            # the schedule rebuilt the tables many times
        assert before < 0.03                                             # chance is 1 / 1000
        assert np.mean(losses[-20:]) < 0.7 * np.mean(losses[:20]), (np.mean(losses[:20]), np.mean(losses[-20:]))
        assert after_dense > (0.5 if hidden is None else 0.3), (before, after_dense, after_lsh)
        assert after_lsh > (0.3 if hidden is None else 0.2), (before, after_dense, after_lsh)   # retrieval through the tables finds the class too
    finally:
        ds.dslide_destroy(ctx)
