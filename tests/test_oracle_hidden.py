"""Pins of the oracle's LSH-sampled hidden layer (Algorithm 1: active neurons are retrieved for every layer;
Section 3.6: the second kind of layer, of which the dense layer is the case "sparsity is 1"; Section 2.1: a neuron
that is not retrieved is a NoOp with activation 0 and receives no gradient).

  * the first layer's sparse random projections against their definition on the pinned generator and their 1/6, 2/3,
    1/6 statistics,
  * codes of inputs and of hidden neurons against dense +1/0/-1 projections in fp64 (brute force on the definition),
  * tables over the hidden neurons: a partition, ascending, right bucket; the active set against a scan without tables,
  * inactive neurons exactly 0, active ones bit-equal to the dense layer's activation,
  * every neuron active  ==  the dense-hidden-layer oracle, bit for bit, through a whole Adam step,
  * finite differences of the loss with the sets as retrieved; untouched weights (input zero, or neuron inactive for
    every sample that has the input) keep weight and moments bit-identical.
"""
import numpy as np
import pytest

from oracle import oracle as orc
from oracle.oracle import SIMHASH, Oracle
from tests.helpers import csr_to_dense, small_batch


def make(real="double", **kw):
    d = dict(D=40, H=16, N=50, family=SIMHASH, K=2, L=3, bucket_cap=6, seed=3, init_std=0.3, lr=1e-3,
             hidden_K=2, hidden_L=3, hidden_cap=5)
    d.update(kw)
    return Oracle(real, **d)


def test_first_layer_projections_follow_their_definition():
    o = make(D=3000, hidden_K=3, hidden_L=4)
    KL = 12
    P = o.get("proj1").reshape(3000, KL)
    assert set(np.unique(P).tolist()) == {-1, 0, 1}
    n = P.size
    for v, prob in ((1, 1 / 6), (-1, 1 / 6), (0, 2 / 3)):
        assert abs(np.mean(P == v) - prob) < 4 * np.sqrt(prob * (1 - prob) / n)
    for c, p in ((0, 0), (17, 5), (2999, 11), (1234, 7)):
        u = orc.rng(3, 6, 0, c * KL + p) % 6                 # stream 6, rebuild count 0 (generator pinned in test_oracle_rng)
        assert P[c, p] == (1 if u == 0 else (-1 if u == 1 else 0))
    o.draw_hash1(1)
    assert not np.array_equal(P, o.get("proj1").reshape(3000, KL))          # redrawn with the rebuild count
    o.draw_hash1(0)
    assert np.array_equal(P, o.get("proj1").reshape(3000, KL))
    o.close()


def codes_from_sums(S, K, L):
    bits = (S >= 0).reshape(L, K)
    return (bits * (1 << np.arange(K))).sum(axis=1).astype(np.uint32)


def test_codes_of_inputs_and_neurons_by_brute_force():
    o = make(D=60, H=12, hidden_K=3, hidden_L=5, hidden_cap=12)
    K, L = 3, 5
    P = o.get("proj1").reshape(60, K * L).astype(np.float64)
    W1 = o.get("W1").reshape(60, 12)
    r = np.random.default_rng(0)
    batch = small_batch(r, 7, 60, o.N, 9)
    o.forward(*batch)
    X = csr_to_dense(batch[0], batch[1], batch[2], 60)
    codes1 = o.get("codes1").reshape(7, L)
    for s in range(7):
        S = P.T @ X[s]
        assert np.min(np.abs(S[S != 0])) > 1e-9 if np.any(S != 0) else True
        assert np.array_equal(codes1[s], codes_from_sums(S, K, L)), s
    # the all-zero input: every sum is exactly 0 -> every bit 1
    z = (np.array([0, 0], dtype=np.int32), np.zeros(0, dtype=np.int32), np.zeros(0), np.array([0, 1], dtype=np.int32),
         np.array([3], dtype=np.int32))
    o.forward(*z)
    assert np.all(o.get("codes1") == (1 << K) - 1)
    # neurons: bucket t of neuron k is the code of column k of W1
    off = o.get("bucket1_off").reshape(L, -1)
    ids = o.get("bucket1_ids").reshape(L, 12)
    for t in range(L):
        assert sorted(ids[t].tolist()) == list(range(12))                      # a partition
        assert off[t, 0] == 0 and off[t, -1] == 12
        for b in range(1 << K):
            mem = ids[t, off[t, b]:off[t, b + 1]]
            assert np.all(np.diff(mem) > 0)                                    # ascending
            for k in mem:
                S = P.T @ W1[:, k]
                assert codes_from_sums(S, K, L)[t] == b
    o.close()


def test_active_hidden_set_is_the_union_of_capped_buckets_and_the_rest_are_noops():
    o = make(D=50, H=24, hidden_K=2, hidden_L=3, hidden_cap=4)
    dense = make(D=50, H=24, hidden_L=0)
    K, L, cap = 2, 3, 4
    r = np.random.default_rng(1)
    batch = small_batch(r, 9, 50, o.N, 8)
    o.forward(*batch)
    dense.forward(*batch)
    P = o.get("proj1").reshape(50, K * L).astype(np.float64)
    W1 = o.get("W1").reshape(50, 24)
    X = csr_to_dense(batch[0], batch[1], batch[2], 50)
    ncodes = np.array([codes_from_sums(P.T @ W1[:, k], K, L) for k in range(24)])     # [H][L]
    hact = o.get("hact").reshape(9, 24)
    h, hd = o.get("h").reshape(9, 24), dense.get("h").reshape(9, 24)
    capped = False
    for s in range(9):
        q = codes_from_sums(P.T @ X[s], K, L)
        want = np.zeros(24, dtype=np.uint8)
        for t in range(L):
            same = np.nonzero(ncodes[:, t] == q[t])[0]          # ascending ids; a query reads the `cap` lowest
            capped = capped or len(same) > cap
            want[same[:cap]] = 1
        assert np.array_equal(hact[s], want), s
        assert np.all(h[s][want == 0] == 0)                      # not retrieved: NoOp, activation 0
        assert np.array_equal(h[s][want == 1], hd[s][want == 1]) # retrieved: the dense layer's value, bit for bit
    assert capped and 0 < hact.mean() < 1
    o.close()
    dense.close()


def test_every_neuron_active_equals_the_dense_hidden_layer():
    """Section 3.6: the dense layer is the sparse layer with sparsity 1.  One-bit codes, many tables, no cap: every
    neuron is retrieved by some table for every sample here, and the whole training step must then be the dense one."""
    kw = dict(D=30, H=8, N=40, seed=9, rebuild_period0=2)
    o = make(hidden_K=1, hidden_L=24, hidden_cap=8, **kw)
    dense = make(hidden_L=0, **kw)
    r = np.random.default_rng(2)
    for i in range(3):                        # a scheduled rebuild (both layers' tables) falls after step 2
        batch = small_batch(r, 6, 30, 40, 7)
        la, lb = o.train_step(*batch), dense.train_step(*batch)
        assert np.all(o.get("hact") == 1), "choose another seed: a neuron was missed by all tables"
        assert la == lb
        for n in ("h", "dh", "act_ids", "act_g"):
            assert np.array_equal(o.get(n), dense.get(n)), (i, n)
    for n in ("W1", "b1", "W2", "b2", "mW1", "vW1", "mb1", "vb1", "mW2", "vW2"):
        assert np.array_equal(o.get(n), dense.get(n)), n
    o.close()
    dense.close()


def test_gradients_with_a_sampled_hidden_layer_match_finite_differences():
    o = make(D=20, H=10, N=30, hidden_K=2, hidden_L=2, hidden_cap=3, seed=4)
    o.set("b1", np.linspace(0.05, 0.4, o.H))
    r = np.random.default_rng(5)
    batch = small_batch(r, 5, o.D, o.N, 6)
    o.forward(*batch)
    sets0 = [a.copy() for a in o.active_sets()]
    hact0 = o.get("hact").copy()
    assert 0 < hact0.mean() < 1
    o.backward()
    grads = {n: o.get("d" + n) for n in ("W1", "b1", "W2")}
    # an inactive neuron passes no gradient on
    dh = o.get("dh").reshape(5, o.H)
    assert np.all(dh[hact0.reshape(5, o.H) == 0] == 0)
    eps = 1e-6
    for n in ("W1", "b1", "W2"):
        w = o.view(n)
        nz = np.nonzero(grads[n])[0]
        zero = np.nonzero(grads[n] == 0)[0]
        picks = list(r.choice(nz, size=min(25, len(nz)), replace=False)) + list(zero[:8])
        for e in picks:
            keep = w[e]
            vals = []
            for sgn in (+1, -1):
                w[e] = keep + sgn * eps        # tables are not rebuilt: the hidden sets stay as retrieved
                o.forward(*batch)
                assert all(np.array_equal(a, b) for a, b in zip(o.active_sets(), sets0))
                assert np.array_equal(o.get("hact"), hact0)
                vals.append(o.get("loss").mean())
            w[e] = keep
            fd = (vals[0] - vals[1]) / (2 * eps)
            assert abs(fd - grads[n][e]) < 1e-7 + 1e-5 * abs(fd), (n, e, fd, grads[n][e])
    o.close()


def test_only_touched_weights_of_the_first_layer_move():
    """Weight (c, k) is touched when some sample has input c nonzero AND hidden neuron k active; bias k when some
    sample has neuron k active.  Everything else keeps weight and moments bit-identical (lazy Adam)."""
    o = make("float", D=40, H=16, hidden_K=2, hidden_L=2, hidden_cap=3, seed=6)
    r = np.random.default_rng(7)
    batch = small_batch(r, 6, 40, o.N, 5, dtype=np.float32)
    before = {n: o.get(n) for n in ("W1", "mW1", "vW1", "b1", "mb1", "vb1")}
    o.train_step(*batch)
    hact = o.get("hact").reshape(6, 16).astype(bool)
    touched = np.zeros((40, 16), dtype=bool)
    for s in range(6):
        for c in batch[1][batch[0][s]:batch[0][s + 1]]:
            touched[c] |= hact[s]
    assert 0 < touched.mean() < 0.5
    for n in ("W1", "mW1", "vW1"):
        a, b = before[n].reshape(40, 16), o.get(n).reshape(40, 16)
        assert np.array_equal(a[~touched].view(np.uint32), b[~touched].view(np.uint32)), n
    v = o.get("vW1").reshape(40, 16)
    moved = o.get("W1").reshape(40, 16) != before["W1"].reshape(40, 16)
    assert np.all(touched[moved])                          # nothing untouched moved ...
    assert moved[touched].mean() > 0.2                     # ... and touched weights with a gradient did
    assert np.all(v[~touched] == 0)
    any_active = hact.any(axis=0)
    assert not any_active.all()
    for n in ("b1", "mb1", "vb1"):
        assert np.array_equal(before[n][~any_active].view(np.uint32), o.get(n)[~any_active].view(np.uint32)), n
    o.close()
