"""GPU-vs-oracle parity through the C ABI (run with -m gpu on a B200).

Bars: hash functions, bucket codes, tables and active sets bit-exact; the hidden layer bit-exact on
identical weights (its summation order is part of the definition); logits, probabilities, loss and
back-propagated errors within 1e-4 relative; weights after 10 Adam steps within 1e-3 relative.
Relative error is |a-b| / max(|a|,|b|,floor) with floor = 1e-2 of the tensor's largest magnitude, so
that entries that cancel to nearly zero are judged on an absolute scale.  (Adam divides by the
gradient's magnitude, so fp32 rounding in a cancelling gradient sum moves a weight by a fraction of
lr whatever the weight's size: the fp32 and fp64 builds of the oracle themselves differ by 2e-4 under
this measure after 10 steps, and by more than 1e-3 with a floor ten times smaller.)
"""
import numpy as np
import pytest
import torch

from tests.helpers import max_rel_err, small_batch

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2201_12667_b200 import binding as ds
    from paper_2201_12667_b200 import workloads
    from tests.gpu_harness import MOMENTS, WEIGHTS, Pair, to_dev

SIMHASH, DWTA = 0, 1
ACT_TOL = 1e-4
W_TOL = 1e-3


def tiny_pair(**kw):
    c = workloads.config("tiny")
    d = dict(D=c["D"], H=c["H"], N=c["N"], family=c["family"], K=c["K"], L=c["L"], bucket_cap=c["bucket_cap"],
             max_batch=c["batch"], max_labels=c["max_labels"], lr=c["lr"], seed=0)
    d.update(kw)
    return Pair(**d)


def mid_pair(**kw):
    c = workloads.config("mid")
    d = dict(D=c["D"], H=c["H"], N=c["N"], family=c["family"], K=c["K"], L=c["L"], bucket_cap=c["bucket_cap"],
             max_batch=c["batch"], max_labels=c["max_labels"], lr=c["lr"], seed=1)
    d.update(kw)
    return Pair(**d)


def compare_forward(pr, batch, bit_exact_hidden=True, tol=ACT_TOL):
    """Snapshot of the last step on both sides (the oracle's was taken with the same pre-update weights)."""
    B = len(batch[0]) - 1
    o = pr.o
    h_g = ds.dslide_get_last(pr.ctx, "hidden", B)
    h_o = o.get("h").reshape(B, pr.H)
    if bit_exact_hidden:
        assert np.array_equal(h_g.view(np.uint32), h_o.view(np.uint32)), "hidden layer not bit-exact"
    else:
        assert max_rel_err(h_g, h_o, 1e-2) < tol
    sets_g, cnt = pr.gpu_active_sets(B)
    sets_o = o.active_sets()
    if not pr.dense:
        assert np.array_equal(ds.dslide_get_last(pr.ctx, "codes", B), o.get("codes").reshape(B, pr.L)), "codes differ"
    for s in range(B):
        assert np.array_equal(sets_g[s], sets_o[s]), "active set of sample %d differs" % s
    ptr = o.get("act_ptr")
    for name, oname in (("act_logit", "act_z"), ("act_prob", "act_p"), ("act_err", "act_g")):
        g = pr.gpu_ragged(name, B, cnt)
        ref = o.get(oname)
        for s in range(B):      # per sample, so that the floor follows the sample's own scale
            assert max_rel_err(g[ptr[s]:ptr[s + 1]], ref[ptr[s]:ptr[s + 1]], 1e-2) < tol, (name, s)
    assert max_rel_err(ds.dslide_get_last(pr.ctx, "loss", B), o.get("loss"), 1e-2) < tol
    assert max_rel_err(ds.dslide_get_last(pr.ctx, "dhidden", B), o.get("dh").reshape(B, pr.H), 1e-2) < tol


def compare_weights(pr, tol=W_TOL, names=None):
    for n in names or (WEIGHTS + MOMENTS):
        e = max_rel_err(ds.dslide_get_tensor(pr.ctx, n), pr.o.get(n), 1e-2)
        assert e < tol, (n, e)


# ------------------------------------------------------------------ hash functions and tables
@pytest.mark.parametrize("family,K,H", [(SIMHASH, 4, 32), (SIMHASH, 9, 128), (DWTA, 2, 32), (DWTA, 6, 128), (DWTA, 3, 1024)])
def test_hash_functions_match_for_every_rebuild_count(family, K, H):
    pr = Pair(D=64, H=H, N=500, family=family, K=K, L=7, bucket_cap=8, max_batch=8, sync_weights=False)
    try:
        for r in range(3):
            assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "hash_idx"), pr.o.get("hash_idx")), r
            assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "hash_sign"), pr.o.get("hash_sign")), r
            assert ds.dslide_get_tensor(pr.ctx, "counters")[1] == pr.o.r == r
            ds.dslide_rebuild_tables(pr.ctx)
            ds.dslide_sync(pr.ctx)
            pr.o.rebuild_tables()
    finally:
        pr.close()


@pytest.mark.parametrize("family,K,L,N,H", [
    (SIMHASH, 4, 8, 2000, 32),        # one radix pass, 16 buckets
    (SIMHASH, 9, 5, 20011, 128),      # one 9-bit pass, ragged last tile
    (DWTA, 3, 10, 20011, 128),        # 9 bits
    (DWTA, 6, 4, 30000, 128),         # 18 bits: two passes
    (DWTA, 7, 2, 9000, 64),           # 21 bits: three passes
])
def test_tables_bit_exact(family, K, L, N, H):
    pr = Pair(D=100, H=H, N=N, family=family, K=K, L=L, bucket_cap=16, max_batch=8)
    try:
        for trial in range(2):
            assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "bucket_off"), pr.o.get("bucket_off"))
            assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "bucket_ids"), pr.o.get("bucket_ids"))
            ds.dslide_rebuild_tables(pr.ctx)          # new hash functions, same weights
            ds.dslide_sync(pr.ctx)
            pr.o.rebuild_tables()
    finally:
        pr.close()


@pytest.mark.parametrize("K", [4, 6])
def test_tables_with_crowded_buckets(K):
    """Codes wider than one radix digit take the place-then-order table build.  5,000 all-zero rows land in one
    bucket per table (larger than a block sorts: the ordered pass over the codes), 600 copies of one random row in
    another (the block-wide sort), the other rows in buckets of a few ids (ordered in registers)."""
    N, H = 9000, 64
    pr = Pair(D=50, H=H, N=N, family=DWTA, K=K, L=3, bucket_cap=16, max_batch=8)
    try:
        rng = np.random.default_rng(9)
        W2 = pr.o.get("W2").reshape(N, H)
        perm = rng.permutation(N)
        W2[perm[:5000]] = 0.0
        W2[perm[5000:5600]] = rng.standard_normal(H).astype(np.float32)
        pr.o.set("W2", W2)
        pr.o.build_tables()
        pr.push_state()
        for trial in range(2):
            off_o = pr.o.get("bucket_off").reshape(3, -1)
            assert np.diff(off_o, axis=1).max() >= 5000
            assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "bucket_off"), pr.o.get("bucket_off"))
            assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "bucket_ids"), pr.o.get("bucket_ids"))
            ds.dslide_rebuild_tables(pr.ctx)
            ds.dslide_sync(pr.ctx)
            pr.o.rebuild_tables()
    finally:
        pr.close()


def test_initial_weights_have_the_stated_distribution():
    pr = Pair(D=300, H=64, N=4000, family=DWTA, K=2, L=3, bucket_cap=8, max_batch=8, init_std=0.02,
              sync_weights=False)
    try:
        for n in ("W1", "W2"):
            g, o = ds.dslide_get_tensor(pr.ctx, n), pr.o.get(n)
            # same counter-based uniforms and the same Box-Muller formula: equal up to libm rounding
            assert max_rel_err(g, o, 1e-3) < 1e-5
            assert abs(g.std() - 0.02) < 2e-4 and abs(g.mean()) < 2e-4
        for n in ("b1", "b2", "mW1", "vW2"):
            assert not ds.dslide_get_tensor(pr.ctx, n).any()
    finally:
        pr.close()


# ------------------------------------------------------------------ one step
@pytest.mark.parametrize("dedup_mode", [1, 2])
def test_single_step_tiny(dedup_mode):
    pr = tiny_pair(dedup_mode=dedup_mode)
    try:
        wl = workloads.Workload(workloads.config("tiny"), seed=0)
        batch = wl.batch(0)
        lo = pr.o.train_step(*batch)
        lg = pr.gpu_step(batch)
        assert abs(lo - lg) <= ACT_TOL * abs(lo)
        compare_forward(pr, batch)
        compare_weights(pr)
        st = ds.dslide_last_stats(pr.ctx)
        assert st["sum_active"] == pr.o.get("act_ptr")[-1]
        assert st["touched_w2"] == len(np.unique(pr.o.get("act_ids")))
        assert st["touched_w1"] == len(np.unique(batch[1])) and st["nnz"] == len(batch[1])
    finally:
        pr.close()


@pytest.mark.parametrize("family,K,dedup_mode", [(DWTA, 3, 1), (DWTA, 3, 2), (SIMHASH, 7, 1), (SIMHASH, 7, 2)])
def test_single_step_mid(family, K, dedup_mode):
    """Zipf inputs, H = 128, several radix tiles, ragged active sets, repeated hot labels and features."""
    pr = mid_pair(family=family, K=K, dedup_mode=dedup_mode)
    try:
        wl = workloads.Workload(workloads.config("mid"), seed=3)
        batch = wl.batch(0)
        lo = pr.o.train_step(*batch)
        lg = pr.gpu_step(batch)
        assert abs(lo - lg) <= ACT_TOL * abs(lo)
        compare_forward(pr, batch)
        compare_weights(pr)
    finally:
        pr.close()


def test_untouched_rows_keep_their_bits():
    pr = mid_pair()
    try:
        wl = workloads.Workload(workloads.config("mid"), seed=4)
        batch = wl.batch(0)
        before = {n: ds.dslide_get_tensor(pr.ctx, n) for n in ("W2", "mW2", "vW2", "b2", "W1", "mW1", "vW1")}
        pr.gpu_step(batch)
        sets, _ = pr.gpu_active_sets(len(batch[0]) - 1)
        act = np.unique(np.concatenate(sets))
        rows2 = np.setdiff1d(np.arange(pr.N), act)
        rows1 = np.setdiff1d(np.arange(pr.D), np.unique(batch[1]))
        for n, rows, width in (("W2", rows2, pr.H), ("mW2", rows2, pr.H), ("vW2", rows2, pr.H), ("b2", rows2, 1),
                               ("W1", rows1, pr.H), ("mW1", rows1, pr.H), ("vW1", rows1, pr.H)):
            a = before[n].reshape(-1, width)[rows]
            b = ds.dslide_get_tensor(pr.ctx, n).reshape(-1, width)[rows]
            assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), n
        moved = ds.dslide_get_tensor(pr.ctx, "W2").reshape(-1, pr.H)[act] != before["W2"].reshape(-1, pr.H)[act]
        assert moved.any(axis=1).all()
    finally:
        pr.close()


def test_two_runs_are_bit_identical():
    outs = []
    for _ in range(2):
        pr = mid_pair()
        try:
            wl = workloads.Workload(workloads.config("mid"), seed=5)
            for i in range(3):
                pr.gpu_step(wl.batch(i))
            outs.append([ds.dslide_get_tensor(pr.ctx, n) for n in WEIGHTS + MOMENTS])
        finally:
            pr.close()
    for a, b in zip(*outs):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


# ------------------------------------------------------------------ ten steps
def run_steps(pr, wl, steps, host=False):
    """Both sides step on their own weights.  The first step starts from identical state and is held to the
    activation tolerance; later steps run on weights that agree only within the weight tolerance, so their
    activations are compared at that tolerance.  Codes and active sets must stay identical throughout."""
    for i in range(steps):
        batch = wl.batch(i)
        tol = ACT_TOL if i == 0 else W_TOL
        lo = pr.o.train_step(*batch)
        lg = pr.gpu_step(batch, host=host)
        assert abs(lo - lg) <= tol * abs(lo), (i, lo, lg)
        compare_forward(pr, batch, bit_exact_hidden=(i == 0), tol=tol)
        c = ds.dslide_get_tensor(pr.ctx, "counters")
        assert (c[0], c[1], c[2]) == (pr.o.t, pr.o.r, pr.o.next_rebuild)


def test_ten_adam_steps_tiny_config():
    """The tiny reference configuration: batch 32, 10 Adam steps, lr 1e-3, seed 0."""
    pr = tiny_pair()
    try:
        run_steps(pr, workloads.Workload(workloads.config("tiny"), seed=0), 10)
        compare_weights(pr)
    finally:
        pr.close()


def test_ten_steps_with_scheduled_rebuilds():
    pr = tiny_pair(rebuild_period0=3, rebuild_lambda=0.3, redraw=1)
    try:
        run_steps(pr, workloads.Workload(workloads.config("tiny"), seed=1), 10)
        assert pr.o.r >= 2
        assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "hash_idx"), pr.o.get("hash_idx"))
        compare_weights(pr)
    finally:
        pr.close()


def test_ten_steps_mid_through_host_entry_point():
    pr = mid_pair(rebuild_period0=4)
    try:
        run_steps(pr, workloads.Workload(workloads.config("mid"), seed=6), 10, host=True)
        compare_weights(pr)
    finally:
        pr.close()


def test_pipelined_host_steps_match_synchronous_ones():
    """dslide_train_step_host_async hands out each step's loss one call late; losses and weights must be the very
    bits the synchronous entry point produces (the kernels and their order are the same)."""
    wl = workloads.Workload(workloads.config("mid"), seed=8)
    batches = [wl.batch(i) for i in range(7)]
    B = len(batches[0][0]) - 1
    a, b = mid_pair(rebuild_period0=3), mid_pair(rebuild_period0=3)
    try:
        sync_losses = [ds.dslide_train_step_host(a.ctx, B, *bt) for bt in batches]
        got = []
        for bt in batches:
            prev = ds.dslide_train_step_host_async(b.ctx, B, *[x.copy() for x in bt])   # the arrays may be reused at once
            if prev is not None:
                got.append(prev)
        got.append(ds.dslide_host_result(b.ctx))
        assert ds.dslide_host_result(b.ctx) is None
        assert np.array_equal(np.array(got, dtype=np.float32), np.array(sync_losses, dtype=np.float32))
        for n in WEIGHTS + MOMENTS:
            x, y = ds.dslide_get_tensor(a.ctx, n), ds.dslide_get_tensor(b.ctx, n)
            assert np.array_equal(x.view(np.uint32), y.view(np.uint32)), n
        # an out-of-range feature id is reported with the step it belongs to (one call late) and cleared by the collect
        bad = [x.copy() for x in batches[0]]
        bad[1][3] = a.D + 7
        assert ds.dslide_train_step_host_async(b.ctx, B, *bad) is None
        with pytest.raises(ds.DslideError) as e:
            ds.dslide_host_result(b.ctx)
        assert e.value.status == ds.ERR_BAD_INDEX
        assert ds.dslide_sync(b.ctx, check=False) == ds.OK
    finally:
        a.close()
        b.close()


# ------------------------------------------------------------------ dense limit
def test_force_dense_matches_oracle_and_dense_softmax():
    pr = tiny_pair(force_dense=1)
    try:
        wl = workloads.Workload(workloads.config("tiny"), seed=2)
        run_steps(pr, wl, 3)
        compare_weights(pr)
    finally:
        pr.close()


# ------------------------------------------------------------------ inference
# over all neurons: k <= 8 runs on the tensor pipe when the hidden width allows it (32 .. 256 in steps of 32; one, two or
# three tiles of W2 in flight), else the fp32 scan with 32, 16, 8 samples per block
@pytest.mark.parametrize("dense,k,H", [(0, 5, 128), (1, 5, 128), (1, 12, 128), (1, 40, 128), (1, 3, 32), (1, 8, 96), (1, 5, 192),
                                       (1, 5, 256), (1, 5, 104)])
def test_predict_topk(dense, k, H):
    pr = mid_pair(H=H)
    try:
        check_predict(pr, workloads.Workload(workloads.config("mid"), seed=7).batch(0), dense, k)
    finally:
        pr.close()


def test_predict_topk_over_all_neurons_with_five_groups_of_samples():
    """600 samples: five blocks of 128 samples share every tile of W2 (the last group ragged), fewer slices of the
    neurons per group, larger candidate buffers."""
    pr = mid_pair(max_batch=600)
    try:
        check_predict(pr, workloads.Workload(workloads.config("mid"), seed=8).batch(0, 600), 1, 5)
    finally:
        pr.close()


def test_predict_topk_over_all_neurons_when_the_filter_cannot_decide():
    """Every output neuron a copy of one of three rows and no bias: thousands of neurons tie at every cut, the candidate
    buffers run over and the error bound cannot separate the k-th score from the rest, so every sample goes through
    the exact fp32 scan inside the exact pass.  Ties are ordered by id (ascending), as the oracle's full sort does."""
    pr = mid_pair()
    try:
        r = np.random.default_rng(3)
        rows = (r.standard_normal((3, pr.H)) * 0.05).astype(np.float32)
        pr.o.set("W2", rows[np.arange(pr.N) % 3].ravel())
        check_predict(pr, workloads.Workload(workloads.config("mid"), seed=9).batch(0), 1, 5, b2=np.zeros(pr.N, dtype=np.float32), same_ids=True)
    finally:
        pr.close()


def check_predict(pr, batch, dense, k, b2=None, same_ids=False):
    pr.o.set("b2", np.random.default_rng(0).standard_normal(pr.N).astype(np.float32) * 0.05 if b2 is None else b2)
    pr.push_state()
    B = len(batch[0]) - 1
    ids_o, sc_o = pr.o.predict_topk(batch[0], batch[1], batch[2], k, dense=bool(dense))
    dev = to_dev(batch[:3])
    ids_g = torch.empty(B * k, dtype=torch.int32, device="cuda")
    sc_g = torch.empty(B * k, dtype=torch.float32, device="cuda")
    ds.dslide_predict_topk(pr.ctx, B, *dev, k, dense, ids_g, sc_g)
    ds.dslide_sync(pr.ctx)
    ids_g = ids_g.cpu().numpy().reshape(B, k)
    sc_g = sc_g.cpu().numpy().reshape(B, k)
    if same_ids:
        assert np.array_equal(ids_g, ids_o)
    for s in range(B):
        valid = ids_o[s] >= 0
        assert np.array_equal(ids_g[s] >= 0, valid)
        assert max_rel_err(sc_g[s][valid], sc_o[s][valid], 1e-2) < ACT_TOL
        assert np.all(np.isneginf(sc_g[s][~valid]))
        # ids must agree wherever the scores are separated by more than the tolerance
        for q in range(k):
            if not valid[q]:
                continue
            near = np.abs(sc_o[s][valid] - sc_o[s][q]) <= 2 * ACT_TOL * np.abs(sc_o[s][q])
            if near.sum() == 1:
                assert ids_g[s][q] == ids_o[s][q]
            else:
                assert ids_g[s][q] in ids_o[s][valid][near]


# ------------------------------------------------------------------ error paths: status codes, never a fault
def test_device_detected_errors_are_reported_and_skipped():
    pr = tiny_pair()
    try:
        wl = workloads.Workload(workloads.config("tiny"), seed=3)
        good = wl.batch(0)
        B = len(good[0]) - 1
        before = ds.dslide_get_tensor(pr.ctx, "W2").copy()
        # feature id out of range in sample 3
        bad = [a.copy() for a in good]
        bad[1][good[0][3 + 1] - 1] = pr.D + 5
        dev = to_dev(bad)
        ds.dslide_train_step(pr.ctx, B, *dev, None)
        assert ds.dslide_sync(pr.ctx, check=False) == ds.ERR_BAD_INDEX
        assert ds.dslide_sync(pr.ctx, check=False) == ds.OK          # sticky status is cleared by the read
        cnt = ds.dslide_get_last(pr.ctx, "act_count", B)
        assert cnt[3] == 0 and np.all(np.delete(cnt, 3) > 0)          # only the offending sample is skipped
        assert ds.dslide_get_last(pr.ctx, "loss", B)[3] == 0
        # label out of range
        bad = [a.copy() for a in good]
        bad[4][0] = pr.N
        ds.dslide_train_step(pr.ctx, B, *to_dev(bad), None)
        assert ds.dslide_sync(pr.ctx, check=False) == ds.ERR_BAD_INDEX
        # negative label, unsorted columns
        bad = [a.copy() for a in good]
        bad[4][1] = -1
        bad[1][[0, 1]] = bad[1][[1, 0]]
        ds.dslide_train_step(pr.ctx, B, *to_dev(bad), None)
        assert ds.dslide_sync(pr.ctx, check=False) == ds.ERR_BAD_INDEX
        # too many labels for one sample
        bad = [a.copy() for a in good]
        bad[3] = np.concatenate([[0], np.full(B, 5, dtype=np.int32)]).astype(np.int32)
        bad[4] = np.arange(5, dtype=np.int32)
        ds.dslide_train_step(pr.ctx, B, *to_dev(bad), None)
        assert ds.dslide_sync(pr.ctx, check=False) == ds.ERR_OVERFLOW
        # the context still works
        ds.dslide_train_step(pr.ctx, B, *to_dev(good), None)
        assert ds.dslide_sync(pr.ctx, check=False) == ds.OK
        assert np.any(ds.dslide_get_tensor(pr.ctx, "W2") != before)
    finally:
        pr.close()


def test_active_set_overflow_is_reported():
    pr = tiny_pair(max_active=4)
    try:
        wl = workloads.Workload(workloads.config("tiny"), seed=3)
        good = wl.batch(0)
        ds.dslide_train_step(pr.ctx, len(good[0]) - 1, *to_dev(good), None)
        assert ds.dslide_sync(pr.ctx, check=False) == ds.ERR_OVERFLOW
    finally:
        pr.close()


def test_host_detected_errors():
    pr = tiny_pair()
    try:
        wl = workloads.Workload(workloads.config("tiny"), seed=3)
        dev = to_dev(wl.batch(0))
        with pytest.raises(ds.DslideError) as e:
            ds.dslide_train_step(pr.ctx, 33, *dev, None)               # max_batch is 32
        assert e.value.status == ds.ERR_OVERFLOW
        with pytest.raises(ds.DslideError) as e:
            ds.dslide_train_step(pr.ctx, 0, *dev, None)
        assert e.value.status == ds.ERR_INVALID_ARG
        with pytest.raises(ds.DslideError):
            ds.dslide_set_tensor(pr.ctx, "W1", np.zeros(3, dtype=np.float32))   # wrong size
        with pytest.raises(ds.DslideError):
            ds.dslide_set_tensor(pr.ctx, "hash_idx", np.full(pr.K * pr.L * pr.o.idx_per_fn, pr.H, dtype=np.int32))
        for kw in (dict(hidden_dim=30), dict(K=0), dict(hash_family=7), dict(max_batch=5000), dict(dwta_bin_size=6, hash_family=1),
                   dict(K=30, hash_family=0)):
            base = dict(input_dim=10, hidden_dim=32, output_dim=100, hash_family=0, K=4, L=2, bucket_cap=4, max_batch=8)
            base.update(kw)
            with pytest.raises(ds.DslideError) as e:
                ds.dslide_init(ds.make_config(**base))
            assert e.value.status == ds.ERR_INVALID_ARG
    finally:
        pr.close()


# ------------------------------------------------------------------ full size, in the benchmark's launch configuration
def test_full_size_670k_step_against_oracle():
    """One step at the headline shape (D 135,909, H 128, N 670,091, DWTA K=6 L=50, cap 128, batch 256)."""
    c = workloads.config("670k")
    pr = Pair(D=c["D"], H=c["H"], N=c["N"], family=c["family"], K=c["K"], L=c["L"], bucket_cap=c["bucket_cap"],
              max_batch=c["batch"], max_labels=c["max_labels"], lr=c["lr"], init_std=0.01, seed=0,
              inputs_ready=1)                    # as the benchmark launches it: batches resident before the call
    try:
        assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "bucket_off"), pr.o.get("bucket_off"))
        assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "bucket_ids"), pr.o.get("bucket_ids"))
        wl = workloads.Workload(c, seed=0)
        batch = wl.batch(0)
        lo = pr.o.train_step(*batch)
        lg = pr.gpu_step(batch)
        assert abs(lo - lg) <= ACT_TOL * abs(lo)
        compare_forward(pr, batch)
        # rows touched by the step (sampled densely: all of them) and a sample of untouched ones
        act = np.unique(pr.o.get("act_ids"))
        W2g = ds.dslide_get_tensor(pr.ctx, "W2").reshape(pr.N, pr.H)
        W2o = pr.o.view("W2").reshape(pr.N, pr.H)
        assert max_rel_err(W2g[act], W2o[act], 1e-2) < W_TOL
        rest = np.setdiff1d(np.arange(0, pr.N, 97), act)
        assert np.array_equal(W2g[rest].view(np.uint32), W2o[rest].view(np.uint32))
        feats = np.unique(batch[1])
        W1g = ds.dslide_get_tensor(pr.ctx, "W1").reshape(pr.D, pr.H)
        assert max_rel_err(W1g[feats], pr.o.view("W1").reshape(pr.D, pr.H)[feats], 1e-2) < W_TOL
    finally:
        pr.close()


# ------------------------------------------------------------------ batch arrays produced on the stream just before the step
@pytest.mark.parametrize("inputs_ready_after_sync", [False, True])
def test_batch_written_by_a_kernel_on_the_same_stream_right_before_the_step(inputs_ready_after_sync):
    """The five batch arrays live in fixed device buffers that a copy kernel on the context's stream overwrites
    immediately before every step (no synchronisation in between): the step must see the new batch, not the one
    the buffers held before.  With inputs_ready = 1 the caller has to finish the producer first (here: a
    synchronize), and the early-reading path must then give the same results."""
    pr = mid_pair(inputs_ready=1 if inputs_ready_after_sync else 0)
    try:
        wl = workloads.Workload(workloads.config("mid"), seed=21)
        batches = [wl.batch(i) for i in range(6)]
        cap = [max(len(b[k]) for b in batches) for k in range(5)]
        bufs = [torch.zeros(cap[k], dtype=torch.float32 if k == 2 else torch.int32, device="cuda") for k in range(5)]
        staged = [to_dev(b) for b in batches]
        torch.cuda.synchronize()
        loss = torch.zeros(1, device="cuda")
        for i, b in enumerate(batches):
            B = len(b[0]) - 1
            lo = pr.o.train_step(*b)
            for k in range(5):
                bufs[k][:len(b[k])].copy_(staged[i][k])          # a kernel on the same stream, just before the step
            if inputs_ready_after_sync:
                torch.cuda.synchronize()
            ds.dslide_train_step(pr.ctx, B, *bufs, loss)
            ds.dslide_sync(pr.ctx)
            assert abs(float(loss.item()) - lo) <= 1e-3 * abs(lo)
            sets_g, _ = pr.gpu_active_sets(B)
            for s, ref in enumerate(pr.o.active_sets()):
                assert np.array_equal(sets_g[s], ref), (i, s)
    finally:
        pr.close()


def test_training_snapshot_is_whole_again_after_a_predict_call():
    """A predict call borrows the per-sample work space; the next training step must rewrite all of it."""
    pr = mid_pair()
    try:
        wl = workloads.Workload(workloads.config("mid"), seed=5)
        b0, b1 = wl.batch(0), wl.batch(1)
        pr.o.train_step(*b0)
        pr.gpu_step(b0)
        B = len(b1[0]) - 1
        dev = to_dev(b1)
        out_ids = torch.zeros(B * 4, dtype=torch.int32, device="cuda")
        out_sc = torch.zeros(B * 4, dtype=torch.float32, device="cuda")
        for dense in (0, 1):
            ds.dslide_predict_topk(pr.ctx, B, dev[0], dev[1], dev[2], 4, dense, out_ids, out_sc)
        ds.dslide_sync(pr.ctx)
        pr.o.train_step(*b1)
        pr.gpu_step(b1)
        compare_forward(pr, b1, bit_exact_hidden=False, tol=1e-3)     # second step: each side on its own weights
    finally:
        pr.close()
