"""GPU-vs-oracle parity on shapes chosen to reach every path of the two step kernels (run with -m gpu).

The forward kernel switches between three ways of removing duplicate candidates (counting ranks, bitonic
sort, bitmap) by the size of the candidate set, stages the active rows of W2 in shared memory in one or
several chunks, and hands rows to the update kernel through slots, masks and two lists whose capacity is
bounded; the update kernel has code paths per touch count (1, up to the slots, listed, listed hot and cut
in slices) and per hidden width.  Each case below states which of these it drives.  Bars as in
test_gpu_parity.py.
"""
import numpy as np
import pytest
import torch

from tests.helpers import max_rel_err

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2201_12667_b200 import binding as ds
    from paper_2201_12667_b200 import workloads
    from tests.gpu_harness import Pair
    from tests.test_gpu_parity import ACT_TOL, W_TOL, compare_forward, compare_weights

SIMHASH, DWTA = 0, 1


def dense_features_batch(rng, B, D, N, nnz, nlab):
    """Every sample draws nnz of only D features, so every feature row is touched by about B*nnz/D samples."""
    cols, vals, labs = [], [], []
    row_ptr = np.zeros(B + 1, dtype=np.int32)
    label_ptr = np.zeros(B + 1, dtype=np.int32)
    for s in range(B):
        ids = np.sort(rng.choice(D, size=nnz, replace=False)).astype(np.int32)
        cols.append(ids)
        v = rng.standard_normal(nnz).astype(np.float32)
        vals.append(v / np.sqrt(np.sum(v * v)))
        labs.append(rng.choice(N, size=nlab, replace=False).astype(np.int32))
        row_ptr[s + 1] = row_ptr[s] + nnz
        label_ptr[s + 1] = label_ptr[s] + nlab
    return row_ptr, np.concatenate(cols), np.concatenate(vals), label_ptr, np.concatenate(labs)


def one_and_two_steps(pr, batches):
    for i, batch in enumerate(batches):
        lo = pr.o.train_step(*batch)
        lg = pr.gpu_step(batch)
        tol = ACT_TOL if i == 0 else W_TOL
        assert abs(lo - lg) <= tol * abs(lo), (i, lo, lg)
        compare_forward(pr, batch, bit_exact_hidden=(i == 0), tol=tol)
    compare_weights(pr)


@pytest.mark.parametrize("H", [64, 256, 512, 1024])
def test_hidden_widths(H):
    """H = 64: two groups of threads per hidden unit in the back-propagation; 256 / 512 / 1024: the wider
    register layouts of the update kernel and several hidden units per thread in the forward kernel."""
    c = workloads.config("mid")
    pr = Pair(D=c["D"], H=H, N=8009, family=DWTA, K=3, L=6, bucket_cap=16, max_batch=24, max_labels=16, lr=1e-3, seed=2)
    try:
        wl = workloads.Workload(workloads.config("mid", N=8009), seed=11)
        one_and_two_steps(pr, [wl.batch(i, batch_size=24) for i in range(2)])
    finally:
        pr.close()


@pytest.mark.parametrize("family,K,L,cap,dedup_mode", [
    (SIMHASH, 3, 12, 40, 0),     # 300-480 candidates per sample: ranks counted with two or more values per thread
    (SIMHASH, 2, 30, 64, 0),     # up to 1,920 candidates: past the counting limit, bitmap (N bits fit in shared memory)
    (SIMHASH, 2, 30, 64, 2),     # the same through the bitonic sort
    (DWTA, 1, 16, 48, 0),        # 8 buckets per table: about 770 candidates, chunked staging of the active rows
])
def test_large_candidate_sets(family, K, L, cap, dedup_mode):
    """Active sets of several hundred to a thousand neurons: every dedup path, active rows staged in more than one
    chunk (the staging space holds about 190 rows of 128 floats), logits and errors beyond the shared-memory mirror."""
    pr = Pair(D=3001, H=128, N=12007, family=family, K=K, L=L, bucket_cap=cap, max_batch=16, max_labels=16, lr=1e-3,
              seed=3, dedup_mode=dedup_mode)
    try:
        wl = workloads.Workload(workloads.config("mid", D=3001, N=12007), seed=12)
        batches = [wl.batch(i, batch_size=16) for i in range(2)]
        one_and_two_steps(pr, batches)
        cnt = ds.dslide_get_last(pr.ctx, "act_count", 16)
        assert cnt.max() > 256
    finally:
        pr.close()


def test_batch_beyond_256_and_rows_touched_by_most_samples():
    """Batch 300 (ten mask words per row, so a slice of a hot row covers two words and some slices are empty) with
    only 400 features, 60 per sample: every row of W1 is touched by about 45 samples -> the hot list and its slices."""
    rng = np.random.default_rng(5)
    pr = Pair(D=400, H=128, N=6007, family=DWTA, K=3, L=8, bucket_cap=16, max_batch=300, max_labels=4, lr=1e-3, seed=4)
    try:
        batches = [dense_features_batch(rng, 300, 400, 6007, 60, 2) for _ in range(2)]
        one_and_two_steps(pr, batches)
        st = ds.dslide_last_stats(pr.ctx)
        assert st["touched_w1"] == 400
    finally:
        pr.close()


def test_more_hot_rows_than_the_hot_list_holds():
    """2,000 features, 200 per sample, batch 512: each of the 2,000 rows of W1 is touched by about 51 samples, more
    rows than the hot list holds (1,024): the rest must be summed through the list of rows past the slots."""
    rng = np.random.default_rng(6)
    pr = Pair(D=2000, H=32, N=3001, family=DWTA, K=2, L=4, bucket_cap=8, max_batch=512, max_labels=4, lr=1e-3, seed=5)
    try:
        batch = dense_features_batch(rng, 512, 2000, 3001, 200, 1)
        lo = pr.o.train_step(*batch)
        lg = pr.gpu_step(batch)
        assert abs(lo - lg) <= ACT_TOL * abs(lo)
        compare_weights(pr, names=["W1", "mW1", "vW1", "W2", "b2", "b1"])
        # a second step proves that counters, masks and lists were left clean
        batch = dense_features_batch(rng, 512, 2000, 3001, 200, 1)
        lo = pr.o.train_step(*batch)
        lg = pr.gpu_step(batch)
        assert abs(lo - lg) <= W_TOL * abs(lo)
        compare_weights(pr, names=["W1", "W2", "b2", "b1"])
    finally:
        pr.close()


def test_more_listed_rows_than_the_list_holds():
    """One table with two buckets and no cap: every sample retrieves about half of 140,000 neurons, so with 16
    samples some 70,000 rows of W2 are touched by more samples than a row has slots -- more than the list of such
    rows holds (65,536); the rest are found and summed by the walk over the ordinary row list."""
    N = 140000
    pr = Pair(D=200, H=32, N=N, family=SIMHASH, K=1, L=1, bucket_cap=N, max_batch=16, max_labels=2, lr=1e-3, seed=6,
              init_std=0.05)
    try:
        wl = workloads.Workload(workloads.config("tiny", D=200, N=N, max_labels=2), seed=13)
        for i in range(2):
            batch = wl.batch(i, batch_size=16)
            lo = pr.o.train_step(*batch)
            lg = pr.gpu_step(batch)
            assert abs(lo - lg) <= (ACT_TOL if i == 0 else W_TOL) * abs(lo)
            sets, cnt = pr.gpu_active_sets(16)
            for s, a in enumerate(pr.o.active_sets()):
                assert np.array_equal(sets[s], a)
            if i == 0:
                touches = np.bincount(np.concatenate(sets), minlength=N)
                assert (touches > 6).sum() > 65536
        for n in ("W2", "b2", "mW2", "vW2", "W1"):
            assert max_rel_err(ds.dslide_get_tensor(pr.ctx, n), pr.o.get(n), 1e-2) < W_TOL, n
    finally:
        pr.close()


def test_neuron_ids_too_long_to_sort_packed():
    """More than 2^22 neurons: an id and its position among the candidates no longer share a 32-bit word, so the
    candidates are ranked by comparing ids and positions separately."""
    N = (1 << 22) + 5003
    pr = Pair(D=300, H=8, N=N, family=SIMHASH, K=12, L=4, bucket_cap=32, max_batch=8, max_labels=2, lr=1e-3, seed=7,
              init_std=0.05)
    try:
        wl = workloads.Workload(workloads.config("tiny", D=300, N=N, max_labels=2), seed=14)
        for i in range(2):
            batch = wl.batch(i, batch_size=8)
            lo = pr.o.train_step(*batch)
            lg = pr.gpu_step(batch)
            assert abs(lo - lg) <= (ACT_TOL if i == 0 else W_TOL) * abs(lo)
            sets, cnt = pr.gpu_active_sets(8)
            for s, a in enumerate(pr.o.active_sets()):
                assert np.array_equal(sets[s], a)
        for n in ("W2", "b2", "W1"):
            assert max_rel_err(ds.dslide_get_tensor(pr.ctx, n), pr.o.get(n), 1e-2) < W_TOL, n
    finally:
        pr.close()


@pytest.mark.parametrize("H", [128, 1024])
def test_same_step_repeated_gives_the_same_outputs(H):
    """With a vanishing learning rate the weights do not move, so repeating a batch must reproduce every per-sample
    output of the forward kernel bit for bit (H = 1024: the active rows are streamed in several chunks).  A barrier
    missing between two uses of a shared array shows up here as an occasional difference."""
    pr = Pair(D=workloads.config("mid")["D"], H=H, N=8009, family=DWTA, K=3, L=6, bucket_cap=16, max_batch=24,
              max_labels=16, lr=1e-30, seed=2)
    try:
        wl = workloads.Workload(workloads.config("mid", N=8009), seed=11)
        batch = wl.batch(0, batch_size=24)
        names = ("hidden", "codes", "act_count", "act_logit", "act_err", "loss", "dhidden")
        ref = None
        for it in range(150):
            pr.gpu_step(batch)
            cur = {n: ds.dslide_get_last(pr.ctx, n, 24).copy() for n in names}
            if ref is None:
                ref = cur
                continue
            for n in names:
                assert np.array_equal(cur[n], ref[n]), (it, n)
    finally:
        pr.close()


def test_one_hot_inputs_and_hidden_layer_of_200():
    """The shape of the paper's second dataset at a reduced vocabulary (Table 1, Table 3): one nonzero per sample,
    hidden layer 200 (fifty 16-byte pieces per row: the two-piece register layout of the update kernel with a
    ragged second piece), batch 64 -- words repeat within a batch, so rows of W1 are shared by several samples."""
    V = 20011
    pr = Pair(D=V, H=200, N=V, family=SIMHASH, K=6, L=8, bucket_cap=32, max_batch=64, max_labels=16, lr=1e-3, seed=8)
    try:
        wl = workloads.Workload(workloads.config("text8", D=V, N=V), seed=15)
        batches = [wl.batch(i, batch_size=64) for i in range(2)]
        assert all(np.all(np.diff(b[0]) == 1) for b in batches)
        one_and_two_steps(pr, batches)
    finally:
        pr.close()


def test_densified_dwta_queries():
    """Most hidden units off (a negative hidden bias): about a quarter of the bins of a query are all zero and borrow
    a position along the probe sequence; a scheduled rebuild after the first step draws a new sequence.  Codes and
    active sets must match the oracle bit for bit, with the flag and without it."""
    for densify in (1, 0):
        pr = Pair(D=5003, H=128, N=20011, family=DWTA, K=3, L=10, bucket_cap=16, max_batch=48, max_labels=16, lr=1e-3,
                  seed=9, densify=densify, rebuild_period0=1)
        try:
            pr.o.set("b1", np.full(128, -0.05, dtype=np.float32))
            pr.push_state()
            wl = workloads.Workload(workloads.config("mid"), seed=16)
            batches = [wl.batch(i, batch_size=48) for i in range(3)]
            one_and_two_steps(pr, batches)
            if densify:
                h = ds.dslide_get_last(pr.ctx, "hidden", 48).reshape(48, 128)
                idx = ds.dslide_get_tensor(pr.ctx, "hash_idx").reshape(30, 8)
                empty = np.all(h[:, idx] == 0, axis=2)
                assert 0.05 < empty.mean() < 0.9
        finally:
            pr.close()


@pytest.mark.parametrize("family,K,L,cap,budget", [
    (SIMHASH, 3, 12, 40, 100),     # 300-480 retrieved per sample, 100 kept
    (SIMHASH, 2, 12, 400, 1100),   # well over a thousand retrieved: sets past the shared-memory mirror of the ids
    (DWTA, 3, 10, 16, 40),         # some samples over, some under the budget
    (DWTA, 3, 10, 16, 2),          # fewer than some label lists: those samples keep their labels only
])
def test_sampling_budget(family, K, L, cap, budget):
    """Section 3.7: reservoir sampling over the retrieved neurons.  The kept sets must be the oracle's bit for bit
    (the same draws decide), at two consecutive steps (the draws are numbered by step), and the step built on
    them must match as usual."""
    pr = Pair(D=3001, H=128, N=12007, family=family, K=K, L=L, bucket_cap=cap, max_batch=16, max_labels=16, lr=1e-3,
              seed=10, budget=budget)
    try:
        wl = workloads.Workload(workloads.config("mid", D=3001, N=12007), seed=17)
        batches = [wl.batch(i, batch_size=16) for i in range(2)]
        one_and_two_steps(pr, batches)
        cnt = ds.dslide_get_last(pr.ctx, "act_count", 16)
        nlab = np.array([len(np.unique(batches[1][4][batches[1][3][s]:batches[1][3][s + 1]])) for s in range(16)])
        assert np.all(cnt <= np.maximum(budget, nlab))
        if budget >= 40:
            assert np.any(cnt == budget)                 # the budget was reached by some sample
        # inference applies the same budget
        k = 5
        ids_o, sc_o = pr.o.predict_topk(*batches[1][:3], k)
        dev = [torch.from_numpy(a).cuda() for a in batches[1][:3]]
        out_ids = torch.zeros(16 * k, dtype=torch.int32, device="cuda")
        out_sc = torch.zeros(16 * k, dtype=torch.float32, device="cuda")
        ds.dslide_predict_topk(pr.ctx, 16, *dev, k, False, out_ids, out_sc)
        ds.dslide_sync(pr.ctx)
        assert np.array_equal(out_ids.cpu().numpy().reshape(16, k), ids_o)
    finally:
        pr.close()


@pytest.mark.parametrize("family,K,L,cap,budget", [
    (DWTA, 3, 10, 16, 200),        # every sample under the budget: 40-150 retrieved, topped up to 200
    (DWTA, 3, 10, 16, 60),         # some over (reservoir), some under (fill)
    (SIMHASH, 2, 12, 400, 1100),   # sets topped up past the shared-memory mirror of the ids
])
def test_sampling_budget_with_fill(family, K, L, cap, budget):
    """Section 3.7's other option: sets below the budget are filled with uniform draws.  Same bar as above: the sets
    are the oracle's bit for bit at two consecutive steps and at inference."""
    pr = Pair(D=3001, H=128, N=12007, family=family, K=K, L=L, bucket_cap=cap, max_batch=16, max_labels=16, lr=1e-3,
              seed=11, budget=budget, budget_fill=1)
    try:
        wl = workloads.Workload(workloads.config("mid", D=3001, N=12007), seed=18)
        batches = [wl.batch(i, batch_size=16) for i in range(2)]
        one_and_two_steps(pr, batches)
        cnt = ds.dslide_get_last(pr.ctx, "act_count", 16)
        assert np.all(cnt == budget)                      # far from N, the draws always suffice
        k = 5
        ids_o, sc_o = pr.o.predict_topk(*batches[1][:3], k)
        dev = [torch.from_numpy(a).cuda() for a in batches[1][:3]]
        out_ids = torch.zeros(16 * k, dtype=torch.int32, device="cuda")
        out_sc = torch.zeros(16 * k, dtype=torch.float32, device="cuda")
        ds.dslide_predict_topk(pr.ctx, 16, *dev, k, False, out_ids, out_sc)
        ds.dslide_sync(pr.ctx)
        assert np.array_equal(out_ids.cpu().numpy().reshape(16, k), ids_o)
    finally:
        pr.close()


def test_fill_that_cannot_reach_the_budget():
    """A budget of all N neurons: the draws run out (2 * missing + 64 of them) before every neuron has come up."""
    pr = Pair(D=300, H=32, N=257, family=SIMHASH, K=2, L=2, bucket_cap=8, max_batch=8, max_labels=4, lr=1e-3, seed=12,
              budget=257, budget_fill=1)
    try:
        wl = workloads.Workload(workloads.config("tiny", D=300, N=257, max_labels=3), seed=19)
        batches = [wl.batch(i, batch_size=8) for i in range(2)]
        one_and_two_steps(pr, batches)
        cnt = ds.dslide_get_last(pr.ctx, "act_count", 8)
        assert np.all(cnt < 257) and np.all(cnt > 128)
    finally:
        pr.close()


@pytest.mark.parametrize("name", ["670k-h256-b2048", "670k-h1024-b2048", "text8-b2048"])
def test_paper_shapes_with_batch_2048_at_reduced_vocabulary(name):
    """The hidden widths, batch of 2,048 and hashing of the paper's large-batch and low-bandwidth experiments
    (Table 3; Section 4.7: hidden layer 256, batch 2048) on a vocabulary the oracle steps through in seconds: every
    row of W1 is touched by dozens of samples (hot rows, sample masks of 64 words)."""
    c = workloads.config(name, D=4001, N=30011)
    pr = Pair(D=c["D"], H=c["H"], N=c["N"], family=c["family"], K=c["K"] if c["family"] == SIMHASH else 4, L=12,
              bucket_cap=32, max_batch=c["batch"], max_labels=c["max_labels"], lr=1e-3, seed=5, oracle_build="float_omp")
    try:
        wl = workloads.Workload(c, seed=17)
        one_and_two_steps(pr, [wl.batch(i) for i in range(2)])
    finally:
        pr.close()


def test_tables_whose_counters_exceed_the_cache_are_counted_table_by_table():
    """21-bit codes x 9 tables: 75 MB of bucket counters, beyond what the table build counts while it hashes; the
    counting then runs as a pass of its own.  Tables must not change by a bit, two rebuilds in a row."""
    pr = Pair(D=64, H=64, N=30011, family=DWTA, K=7, L=9, bucket_cap=16, max_batch=8)
    try:
        for trial in range(2):
            assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "bucket_off"), pr.o.view("bucket_off"))
            assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "bucket_ids"), pr.o.view("bucket_ids"))
            ds.dslide_rebuild_tables(pr.ctx)
            ds.dslide_sync(pr.ctx)
            pr.o.rebuild_tables()
    finally:
        pr.close()
