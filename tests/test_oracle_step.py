"""Pins for the oracle's forward pass, gradients and Adam update (CPU only).

* With every neuron forced active ("sparsity is 1", Section 3.6) the step must be the dense
  softmax-cross-entropy step of a two-layer perceptron: checked against torch's CPU
  log_softmax + autograd + torch.optim.Adam (library routines).
* Gradients must match central finite differences of the loss with the active sets as retrieved.
* The softmax over each active set sums to one; neurons outside it get no gradient and keep
  their weights bit for bit (Section 2.1: other neurons are no-ops).
* The first Adam step has the closed form lr * g / (|g| + eps) with the constants of Section 4.1.
"""
import numpy as np
import pytest
import torch

from oracle.oracle import DWTA, SIMHASH, Oracle
from tests.helpers import csr_to_dense, label_matrix, read_golden, small_batch

HYPER = read_golden("section4_1_hyperparameters.txt")


def tiny(real="double", **kw):
    d = dict(D=20, H=8, N=30, family=SIMHASH, K=2, L=3, bucket_cap=4, seed=5, init_std=0.3,
             lr=HYPER["learning_rate"], beta1=HYPER["adam_beta1"], beta2=HYPER["adam_beta2"], eps=HYPER["adam_eps"])
    d.update(kw)
    return Oracle(real, **d)


def torch_dense_model(o, batch):
    """An independent dense statement of the same network in torch (fp64, CPU)."""
    X = torch.tensor(csr_to_dense(batch[0], batch[1], batch[2], o.D))
    Y = torch.tensor(label_matrix(batch[3], batch[4], o.N))
    p = {n: torch.tensor(o.get(n).astype(np.float64).reshape(shape), requires_grad=True)
         for n, shape in (("W1", (o.D, o.H)), ("b1", (o.H,)), ("W2", (o.N, o.H)), ("b2", (o.N,)))}

    def loss_fn():
        h = torch.relu(X @ p["W1"] + p["b1"])
        z = h @ p["W2"].T + p["b2"]
        return -(Y * torch.log_softmax(z, dim=1)).sum(dim=1).mean()
    return p, loss_fn


def test_all_active_step_is_the_dense_softmax_cross_entropy_step():
    o = tiny(force_dense=1, lr=1e-2)
    o.set("b1", np.linspace(-0.2, 0.4, o.H))         # non-trivial biases
    o.set("b2", np.linspace(-0.5, 0.5, o.N))
    r = np.random.default_rng(0)
    batch = small_batch(r, 6, o.D, o.N, 7)
    p, loss_fn = torch_dense_model(o, batch)
    opt = torch.optim.Adam(list(p.values()), lr=1e-2, betas=(HYPER["adam_beta1"], HYPER["adam_beta2"]),
                           eps=HYPER["adam_eps"])
    for step in range(3):                            # same batch: the touched rows stay the same
        opt.zero_grad()
        loss = loss_fn()
        loss.backward()
        o.forward(*batch)
        assert abs(o.get("loss").mean() - loss.item()) < 1e-12
        o.backward()
        for n in ("W1", "b1", "W2", "b2"):
            np.testing.assert_allclose(o.get("d" + n), p[n].grad.numpy().ravel(), rtol=1e-10, atol=1e-14)
        o.adam()
        opt.step()
        for n in ("W1", "b1", "W2", "b2"):
            np.testing.assert_allclose(o.get(n), p[n].detach().numpy().ravel(), rtol=1e-9, atol=1e-12)
    assert o.t == 3


@pytest.mark.parametrize("family", [SIMHASH, DWTA])
def test_gradients_match_finite_differences(family):
    o = tiny(family=family, K=2, L=3)
    o.set("b1", np.linspace(0.05, 0.3, o.H))
    r = np.random.default_rng(1)
    batch = small_batch(r, 5, o.D, o.N, 6)
    o.forward(*batch)
    sets0 = [a.copy() for a in o.active_sets()]
    assert any(len(a) < o.N for a in sets0)          # genuinely sparse
    o.backward()
    grads = {n: o.get("d" + n) for n in ("W1", "b1", "W2", "b2")}
    eps = 1e-6
    for n in ("W1", "b1", "W2", "b2"):
        w = o.view(n)
        nz = np.nonzero(grads[n])[0]
        zero = np.nonzero(grads[n] == 0)[0]
        picks = list(r.choice(nz, size=min(25, len(nz)), replace=False)) + list(zero[:5])
        for e in picks:
            keep = w[e]
            vals = []
            for sgn in (+1, -1):
                w[e] = keep + sgn * eps
                o.forward(*batch)
                assert all(np.array_equal(a, b) for a, b in zip(o.active_sets(), sets0))
                vals.append(o.get("loss").mean())
            w[e] = keep
            fd = (vals[0] - vals[1]) / (2 * eps)
            assert abs(fd - grads[n][e]) < 1e-7 + 1e-5 * abs(fd), (n, e, fd, grads[n][e])


@pytest.mark.parametrize("real", ["float", "double"])
def test_softmax_over_active_set_is_a_distribution(real):
    o = tiny(real=real, N=200, L=5)
    r = np.random.default_rng(2)
    batch = small_batch(r, 16, o.D, o.N, 6, dtype=o.dtype)
    o.forward(*batch)
    ptr, p, z, g = o.get("act_ptr"), o.get("act_p"), o.get("act_z"), o.get("act_g")
    ids = o.get("act_ids")
    assert np.all(o.get("loss") >= 0)
    for s in range(16):
        ps = p[ptr[s]:ptr[s + 1]].astype(np.float64)
        assert np.all(ps > 0) and abs(ps.sum() - 1) < (1e-6 if real == "float" else 1e-12)
        # logits recomputed densely for the active ids
        h = o.get("h").reshape(16, o.H)[s].astype(np.float64)
        W2 = o.get("W2").reshape(o.N, o.H).astype(np.float64)
        zz = W2[ids[ptr[s]:ptr[s + 1]]] @ h + o.get("b2")[ids[ptr[s]:ptr[s + 1]]]
        np.testing.assert_allclose(z[ptr[s]:ptr[s + 1]], zz, rtol=1e-5, atol=1e-6)
        # errors sum to zero over the active set: sum(p) - sum(1/|Y|) = 0, scaled by 1/B
        assert abs(g[ptr[s]:ptr[s + 1]].astype(np.float64).sum()) < 1e-6
        labs = set(batch[4][batch[3][s]:batch[3][s + 1]].tolist())
        assert labs <= set(ids[ptr[s]:ptr[s + 1]].tolist())          # labels are always active


def test_hidden_layer_is_relu_of_sparse_affine_map():
    o = tiny(real="double")
    o.set("b1", np.linspace(-0.3, 0.3, o.H))
    r = np.random.default_rng(3)
    batch = small_batch(r, 9, o.D, o.N, 8)
    o.forward(*batch)
    X = csr_to_dense(batch[0], batch[1], batch[2], o.D)
    want = np.maximum(X @ o.get("W1").reshape(o.D, o.H) + o.get("b1"), 0)
    np.testing.assert_allclose(o.get("h").reshape(9, o.H), want, rtol=1e-12, atol=1e-15)
    assert np.any(want == 0) and np.any(want > 0)


def test_duplicate_labels_count_once():
    o = tiny()
    row_ptr = np.array([0, 2], dtype=np.int32)
    cols = np.array([1, 4], dtype=np.int32)
    vals = np.array([0.5, -1.0])
    o.forward(row_ptr, cols, vals, np.array([0, 3], dtype=np.int32), np.array([7, 7, 9], dtype=np.int32))
    l_dup = o.get("loss")[0]
    o.forward(row_ptr, cols, vals, np.array([0, 2], dtype=np.int32), np.array([7, 9], dtype=np.int32))
    assert l_dup == o.get("loss")[0]


def test_first_adam_step_closed_form_and_untouched_rows():
    """At t = 1 the bias-corrected moments are g and g^2, so the step is lr * g / (|g| + eps)."""
    lr, eps = 1e-3, HYPER["adam_eps"]
    o = tiny(real="double", N=200, L=3, lr=lr)
    r = np.random.default_rng(4)
    batch = small_batch(r, 4, o.D, o.N, 5)
    before = {n: o.get(n) for n in ("W1", "b1", "W2", "b2", "mW2", "vW2", "mW1", "vW1")}
    o.forward(*batch)
    o.backward()
    g = {n: o.get("d" + n) for n in ("W1", "b1", "W2", "b2")}
    active = np.unique(o.get("act_ids"))
    feats = np.unique(batch[1])
    assert len(active) < o.N and len(feats) < o.D
    o.adam()
    assert o.t == 1
    for n in ("W1", "b1", "W2", "b2"):
        step = before[n] - o.get(n)
        np.testing.assert_allclose(step, lr * g[n] / (np.abs(g[n]) + eps), rtol=1e-9, atol=1e-18)
        assert np.all(o.get("d" + n) == 0)                             # gradient buffers cleared
    # rows outside the active sets / the batch's features: weights and moments bit-identical
    rows2 = np.setdiff1d(np.arange(o.N), active)
    rows1 = np.setdiff1d(np.arange(o.D), feats)
    for n, rows, width in (("W2", rows2, o.H), ("mW2", rows2, o.H), ("vW2", rows2, o.H),
                           ("W1", rows1, o.H), ("mW1", rows1, o.H), ("vW1", rows1, o.H)):
        a = before[n].reshape(-1, width)[rows]
        b = o.get(n).reshape(-1, width)[rows]
        assert np.array_equal(a, b)
    # touched rows did move (a touched row with a zero gradient entry still only decays its moments)
    assert np.any(o.get("W2").reshape(o.N, o.H)[active] != before["W2"].reshape(o.N, o.H)[active])
    # moments after one step: m = (1-b1) g, v = (1-b2) g^2
    np.testing.assert_allclose(o.get("mW2"), (1 - HYPER["adam_beta1"]) * g["W2"], rtol=1e-12)
    np.testing.assert_allclose(o.get("vW2"), (1 - HYPER["adam_beta2"]) * g["W2"] ** 2, rtol=1e-9)


def test_adam_second_step_uses_global_step_in_bias_correction():
    """Two steps on the same batch against torch.optim.Adam restricted to touched rows (sparse active sets)."""
    o = tiny(real="double", lr=1e-2, redraw=0)
    r = np.random.default_rng(5)
    batch = small_batch(r, 5, o.D, o.N, 6)
    w = torch.tensor(o.get("b1"), requires_grad=True)
    opt = torch.optim.Adam([w], lr=1e-2, betas=(HYPER["adam_beta1"], HYPER["adam_beta2"]), eps=HYPER["adam_eps"])
    for _ in range(2):
        o.forward(*batch)
        o.backward()
        w.grad = torch.tensor(o.get("db1"))
        o.adam()
        opt.step()
        np.testing.assert_allclose(o.get("b1"), w.detach().numpy(), rtol=1e-10, atol=1e-14)


def test_predict_topk_dense_is_a_full_sort_and_sparse_is_a_subset():
    o = tiny(real="double", N=120, L=4)
    o.set("b2", np.random.default_rng(6).standard_normal(o.N) * 0.1)
    r = np.random.default_rng(7)
    batch = small_batch(r, 7, o.D, o.N, 6)
    ids, sc = o.predict_topk(batch[0], batch[1], batch[2], 5, dense=True)
    X = csr_to_dense(batch[0], batch[1], batch[2], o.D)
    h = np.maximum(X @ o.get("W1").reshape(o.D, o.H) + o.get("b1"), 0)
    Z = h @ o.get("W2").reshape(o.N, o.H).T + o.get("b2")
    for s in range(7):
        order = np.lexsort((np.arange(o.N), -Z[s]))[:5]                # by logit descending, id ascending
        assert ids[s].tolist() == order.tolist()
        np.testing.assert_allclose(sc[s], Z[s, order], rtol=1e-12)
    ids_s, sc_s = o.predict_topk(batch[0], batch[1], batch[2], 5, dense=False)
    sets = o.active_sets()
    for s in range(7):
        got = [i for i in ids_s[s] if i >= 0]
        assert set(got) <= set(sets[s].tolist())
        assert len(got) == min(5, len(sets[s]))
        assert np.all(np.diff(sc_s[s][:len(got)]) <= 0)
        assert np.all(ids_s[s][len(got):] == -1) and np.all(np.isneginf(sc_s[s][len(got):]))
        np.testing.assert_allclose(sc_s[s][:len(got)], Z[s, got], rtol=1e-12)


def test_active_set_overflow_is_an_error():
    o = tiny(max_active=2)
    r = np.random.default_rng(8)
    batch = small_batch(r, 3, o.D, o.N, 5, max_labels=3)
    batch = (batch[0], batch[1], batch[2], np.array([0, 3, 6, 9], dtype=np.int32),
             np.arange(9, dtype=np.int32))
    with pytest.raises(RuntimeError):
        o.forward(*batch)


def test_out_of_range_ids_are_errors():
    o = tiny()
    with pytest.raises(RuntimeError):
        o.forward(np.array([0, 1], dtype=np.int32), np.array([o.D], dtype=np.int32), np.array([1.0]),
                  np.array([0, 1], dtype=np.int32), np.array([0], dtype=np.int32))
    with pytest.raises(RuntimeError):
        o.forward(np.array([0, 1], dtype=np.int32), np.array([0], dtype=np.int32), np.array([1.0]),
                  np.array([0, 1], dtype=np.int32), np.array([o.N], dtype=np.int32))


def test_float_and_double_oracles_agree():
    kw = dict(D=40, H=16, N=100, K=3, L=4, init_std=0.2, lr=1e-3)
    of, od = tiny(real="float", **kw), tiny(real="double", **kw)
    od.set("W1", of.get("W1")); od.set("W2", of.get("W2"))
    od.build_tables(); of.build_tables()
    r = np.random.default_rng(9)
    batch = small_batch(r, 8, 40, 100, 8, dtype=np.float32)
    lf = of.train_step(*batch)
    ld = od.train_step(*batch)
    if all(np.array_equal(a, b) for a, b in zip(of.active_sets(), od.active_sets())):
        assert abs(lf - ld) < 1e-5 * abs(ld)
        np.testing.assert_allclose(of.get("W2"), od.get("W2"), rtol=2e-3, atol=1e-6)


# ---------------------------------------------------------------- sampling budget (Section 3.7)
def _sets_with_and_without_budget(budget, seed=4, t=0, B=6, **kw):
    rs = np.random.default_rng(21)
    cfg = dict(D=60, H=16, N=400, family=SIMHASH, K=2, L=6, bucket_cap=40, seed=seed, init_std=0.5)
    cfg.update(kw)
    batch = small_batch(rs, B, 60, 400, 8, max_labels=3, dtype=np.float32)
    free = Oracle("float", **cfg)
    capped = Oracle("float", budget=budget, **cfg)
    capped.set_counters(t, 0, 0)
    free.set_counters(t, 0, 0)
    free.forward(*batch)
    capped.forward(*batch)
    labels = [np.unique(batch[4][batch[3][s]:batch[3][s + 1]]) for s in range(B)]
    return free.active_sets(), capped.active_sets(), labels, capped


def test_budget_keeps_labels_and_the_reservoir_of_the_other_candidates():
    """Algorithm R written out in Python over the candidates in ascending order, with the oracle's generator."""
    from oracle.oracle import rng as orc_rng
    budget, seed, t = 30, 4, 7
    full, capped, labels, _ = _sets_with_and_without_budget(budget, seed=seed, t=t)
    over = 0
    for s, (a0, a1, y) in enumerate(zip(full, capped, labels)):
        cand = [j for j in a0 if j not in set(y)]
        m = max(0, budget - len(y))
        if len(cand) <= m:
            assert np.array_equal(a0, a1)
            continue
        over += 1
        res = cand[:m]
        for i in range(m, len(cand)):
            j = orc_rng(seed, 4, t, (s << 32) + i) % (i + 1)
            if j < m:
                res[j] = cand[i]
        want = np.array(sorted(set(res) | set(y)), dtype=np.int32)
        assert np.array_equal(a1, want)
        assert len(a1) == budget and set(y) <= set(a1) and set(a1) <= set(a0)
        assert np.all(np.diff(a1) > 0)
    assert over >= 3                                     # the case was exercised


def test_budget_above_the_retrieved_count_changes_nothing_and_below_the_labels_keeps_labels_only():
    full, capped, labels, _ = _sets_with_and_without_budget(10 ** 6)
    for a0, a1 in zip(full, capped):
        assert np.array_equal(a0, a1)
    full, capped, labels, _ = _sets_with_and_without_budget(1)
    for a1, y in zip(capped, labels):
        assert np.array_equal(a1, y)                     # m = max(0, 1 - |Y|) = 0 other neurons


def test_reservoir_keeps_every_candidate_with_probability_m_over_n():
    """The property the reservoir algorithm is known for, over 400 values of the step counter (each draws afresh)."""
    budget = 12
    counts, ncand, m = None, None, None
    for t in range(400):
        full, capped, labels, _ = _sets_with_and_without_budget(budget, t=t, B=1, bucket_cap=60)
        y = set(labels[0])
        cand = [j for j in full[0] if j not in y]
        if counts is None:
            ncand, m = len(cand), budget - len(y)
            assert ncand > 3 * m
            counts = {j: 0 for j in cand}
        for j in capped[0]:
            if j not in y:
                counts[j] += 1
    freq = np.array(list(counts.values())) / 400.0
    p = m / ncand
    sigma = np.sqrt(p * (1 - p) / 400)
    assert abs(freq.mean() - p) < 1e-12                  # exactly m kept every time
    assert np.all(np.abs(freq - p) < 5 * sigma)          # no candidate favoured (first or last positions included)


def test_budget_fill_tops_an_under_full_set_up_with_uniform_draws():
    """The fill written out in Python: draws in order, already-present ids passed over, stop when full or after
    2 * missing + 64 draws."""
    from oracle.oracle import rng as orc_rng
    seed, t = 4, 3
    for budget, N in ((150, 400), (395, 400), (10 ** 4, 400)):
        free, filled, labels, _ = _sets_with_and_without_budget(budget, seed=seed, t=t, budget_fill=1, N=N)
        nofill, _, _, _ = _sets_with_and_without_budget(budget, seed=seed, t=t, N=N)
        topped = 0
        for s, (a0, a1) in enumerate(zip(free, filled)):
            target = min(budget, N)
            if len(a0) >= target:
                continue                                  # over the budget: the reservoir's business
            have = list(a0)
            need = target - len(a0)
            for k in range(2 * need + 64):
                if len(have) == target:
                    break
                j = orc_rng(seed, 5, t, (s << 32) + k) % N
                if j not in have:
                    have.append(j)
            assert np.array_equal(a1, np.array(sorted(have), dtype=np.int32))
            assert set(a0) <= set(a1) and np.all(np.diff(a1) > 0)
            topped += 1
            if budget == 150:
                assert len(a1) == 150                     # far from N, the draws always suffice
        assert topped >= 3


def test_budget_fill_off_leaves_under_full_sets_alone():
    free, capped, labels, _ = _sets_with_and_without_budget(150)
    for a0, a1 in zip(free, capped):
        if len(a0) <= 150:
            assert np.array_equal(a0, a1)


# ---------------------------------------------------------------- the weight bar's floor, measured
def test_fp32_rounding_alone_moves_weights_by_the_floor_the_gpu_bar_uses():
    """The GPU parity bar for weights after 10 Adam steps is 1e-3 of max(|a|, |b|, 0.01 * largest magnitude).
    Why 0.01 and not 0.001: Adam divides by the gradient's magnitude, so fp32 rounding in a cancelling gradient
    sum moves a weight by a fixed fraction of lr whatever the weight's size.  Measured here with the oracle alone:
    its fp32 and fp64 builds, same start, same batches, same active sets, differ by about 2e-4 under the 0.01
    floor and by more than the 1e-3 bar under a 0.001 floor -- i.e. that floor would be below fp32 noise."""
    from paper_2201_12667_b200 import workloads
    from tests.helpers import max_rel_err
    c = workloads.config("mid")
    kw = dict(D=c["D"], H=c["H"], N=c["N"], family=c["family"], K=c["K"], L=c["L"], bucket_cap=c["bucket_cap"],
              lr=c["lr"], init_std=0.05, seed=0)
    a, b = Oracle("float", **kw), Oracle("double", **kw)
    try:
        for n in ("W1", "W2"):
            b.set(n, a.view(n).astype(np.float64))
        b.build_tables()
        wl = workloads.Workload(c, seed=0)
        for i in range(10):
            bt = wl.batch(i)
            a.train_step(*bt)
            b.train_step(*bt)
            assert np.array_equal(a.get("act_ids"), b.get("act_ids"))     # no code flipped: same rows touched
        names = ("W1", "b1", "W2", "b2")
        wide = max(max_rel_err(a.view(n), b.view(n), 1e-2) for n in names)
        narrow = max(max_rel_err(a.view(n), b.view(n), 1e-3) for n in names)
        assert 1e-4 < wide < 4e-4           # fp32 noise sits a factor 3-10 inside the 1e-3 bar
        assert narrow > 1e-3                # with the smaller floor the noise alone would break the bar
    finally:
        a.close()
        b.close()


# ---------------------------------------------------------------- the all-cores build is the same oracle
def test_openmp_build_is_bit_identical_to_the_plain_build():
    """The build that times the oracle on all host cores runs the same source with its loops over samples, neurons
    and touched rows shared out between threads; every accumulator receives the same addends in the same order, so
    tables, snapshots and weights must be identical bit for bit."""
    from paper_2201_12667_b200 import workloads
    c = workloads.config("mid")
    kw = dict(D=c["D"], H=c["H"], N=c["N"], family=c["family"], K=c["K"], L=c["L"], bucket_cap=c["bucket_cap"],
              lr=c["lr"], init_std=0.05, seed=4, rebuild_period0=2)
    a, b = Oracle("float", **kw), Oracle("float_omp", **kw)
    try:
        assert a.threads == 1 and b.threads >= 1
        wl = workloads.Workload(c, seed=4)
        for i in range(3):                       # a scheduled rebuild falls after the second step
            bt = wl.batch(i)
            la, lb = a.train_step(*bt), b.train_step(*bt)
            assert la == lb
            for n in ("h", "dh", "codes", "act_ptr", "act_ids", "act_z", "act_p", "act_g", "loss"):
                assert np.array_equal(a.get(n), b.get(n)), (i, n)
        for n in ("W1", "b1", "W2", "b2", "mW1", "vW1", "mW2", "vW2", "mb2", "vb2", "bucket_off", "bucket_ids", "hash_idx"):
            assert np.array_equal(a.get(n), b.get(n)), n
    finally:
        a.close()
        b.close()
