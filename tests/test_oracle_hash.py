"""Pins for the oracle's hash functions and tables (CPU only).

The paper names the two families (Section 4.1: sparse random projections with
K = 9, densified winner-take-all with K = 6) and says weight vectors are
indexed into L tables that are queried with the layer input, the union of the
retrieved buckets being the active set (Section 2.1, Fig. 1).  These tests
evaluate those definitions by brute force, without the oracle's tables or its
hash routine, and compare.
"""
import numpy as np
import pytest

from oracle.oracle import DWTA, SIMHASH, Oracle, rng as orc_rng


def make(family, real="float", **kw):
    d = dict(D=50, H=24, N=300, family=family, K=4 if family == SIMHASH else 2, L=6, bin_size=8,
             bucket_cap=5, seed=3, init_std=0.5)
    d.update(kw)
    return Oracle(real, **d)


# ---------------------------------------------------------------- parameters
def test_simhash_parameters_are_sparse_sign_projections():
    o = make(SIMHASH, H=31, K=5, L=7)
    m = o.idx_per_fn
    assert m == (31 + 2) // 3                       # a third of the coordinates
    idx = o.get("hash_idx").reshape(5 * 7, m)
    sign = o.get("hash_sign").reshape(5 * 7, m)
    assert np.all((idx >= 0) & (idx < 31))
    assert np.all(np.diff(idx, axis=1) > 0)         # distinct and ascending
    assert set(np.unique(sign)) == {-1, 1}
    assert len({tuple(r) for r in idx}) > 30        # projections differ


def test_dwta_parameters_are_concatenated_permutations():
    o = make(DWTA, H=24, K=3, L=5, bin_size=8)      # 15 bins * 8 = 120 entries = 5 permutations of 24
    idx = o.get("hash_idx")
    assert len(idx) == 120
    for q in range(5):
        assert sorted(idx[q * 24:(q + 1) * 24]) == list(range(24))
    assert o.bits == 9


def test_redraw_changes_functions_and_is_reproducible():
    o = make(SIMHASH)
    a0 = o.get("hash_idx"), o.get("hash_sign")
    o.draw_hash(1)
    a1 = o.get("hash_idx"), o.get("hash_sign")
    assert not (np.array_equal(a0[0], a1[0]) and np.array_equal(a0[1], a1[1]))
    o.draw_hash(0)
    assert np.array_equal(o.get("hash_idx"), a0[0]) and np.array_equal(o.get("hash_sign"), a0[1])


def test_counter_rng_is_a_function_of_all_four_words():
    base = orc_rng(1, 2, 3, 4)
    assert base == orc_rng(1, 2, 3, 4)
    assert len({base, orc_rng(0, 2, 3, 4), orc_rng(1, 0, 3, 4), orc_rng(1, 2, 0, 4), orc_rng(1, 2, 3, 0)}) == 5
    bits = np.array([bin(orc_rng(7, 2, 0, i)).count("1") for i in range(2000)])
    assert abs(bits.mean() - 32.0) < 0.5            # outputs look uniform over 64 bits


# ---------------------------------------------------------------- codes, brute force on the definition
def brute_simhash(o, v):
    """Each projection expanded to a dense +1/0/-1 vector; exact dot product in fp64."""
    K, L, H, m = o.K, o.L, o.H, o.idx_per_fn
    idx = o.get("hash_idx").reshape(K * L, m)
    sign = o.get("hash_sign").reshape(K * L, m)
    P = np.zeros((K * L, H))
    for p in range(K * L):
        P[p, idx[p]] = sign[p]
    s = P @ np.asarray(v, dtype=np.float64)
    return s.reshape(L, K), np.abs(P) @ np.abs(np.asarray(v, dtype=np.float64))


def test_simhash_codes_match_dense_projection_signs():
    o = make(SIMHASH, real="float")
    r = np.random.default_rng(0)
    checked = 0
    for _ in range(200):
        v = r.standard_normal(o.H).astype(np.float32)
        codes = o.hash_vec(v)
        s, l1 = brute_simhash(o, v)
        l1 = l1.reshape(o.L, o.K)
        for t in range(o.L):
            for k in range(o.K):
                if abs(s[t, k]) > 1e-5 * l1[t, k]:   # away from a rounding-level tie
                    assert ((codes[t] >> k) & 1) == (1 if s[t, k] >= 0 else 0)
                    checked += 1
    assert checked > 4000


def test_simhash_sequential_fp32_sum_second_loop():
    """The bit is decided by the sequential fp32 sum in stored order; redo that sum with numpy float32 scalars."""
    o = make(SIMHASH, real="float")
    K, L, m = o.K, o.L, o.idx_per_fn
    idx = o.get("hash_idx").reshape(K * L, m)
    sign = o.get("hash_sign").reshape(K * L, m)
    r = np.random.default_rng(1)
    for _ in range(50):
        v = (r.standard_normal(o.H) * 10 ** r.uniform(-3, 3)).astype(np.float32)
        codes = o.hash_vec(v)
        for t in range(L):
            code = 0
            for k in range(K):
                p = t * K + k
                acc = np.float32(0)
                for i in range(m):
                    acc = np.float32(acc + (v[idx[p, i]] if sign[p, i] > 0 else -v[idx[p, i]]))
                code |= int(acc >= 0) << k
            assert code == codes[t]


def test_simhash_zero_vector_gives_all_ones():
    o = make(SIMHASH)
    assert np.all(o.hash_vec(np.zeros(o.H, dtype=np.float32)) == (1 << o.K) - 1)


def test_dwta_codes_match_first_maximum_of_each_bin():
    o = make(DWTA, H=24, K=3, L=5)
    idx = o.get("hash_idx").reshape(15, 8)
    r = np.random.default_rng(2)
    for trial in range(200):
        v = r.standard_normal(24).astype(np.float32)
        if trial % 3 == 0:
            v = np.maximum(v, 0)                    # ReLU-like: many exact ties at 0
        if trial % 7 == 0:
            v = np.round(v)                         # ties among positive values too
        codes = o.hash_vec(v)
        for t in range(5):
            code = 0
            for k in range(3):
                code |= int(np.argmax(v[idx[t * 3 + k]])) << (3 * k)   # np.argmax returns the first maximum
            assert code == codes[t]


def test_dwta_all_equal_bins_give_zero():
    o = make(DWTA, H=24, K=3, L=5)
    assert np.all(o.hash_vec(np.zeros(24, dtype=np.float32)) == 0)
    assert np.all(o.hash_vec(np.full(24, 2.5, dtype=np.float32)) == 0)


# ---------------------------------------------------------------- invariances the families must have
@pytest.mark.parametrize("family", [SIMHASH, DWTA])
def test_codes_invariant_under_power_of_two_scaling(family):
    o = make(family)
    r = np.random.default_rng(4)
    for _ in range(50):
        v = r.standard_normal(o.H).astype(np.float32)
        c = o.hash_vec(v)
        for e in (-20, -3, 5, 30):
            assert np.array_equal(o.hash_vec(np.ldexp(v, e).astype(np.float32)), c)


def test_dwta_invariant_under_increasing_maps():
    o = make(DWTA, real="double")
    r = np.random.default_rng(5)
    for _ in range(50):
        v = r.standard_normal(o.H)
        c = o.hash_vec(v)
        assert np.array_equal(o.hash_vec(np.exp(v)), c)
        assert np.array_equal(o.hash_vec(v ** 3 + 7.0), c)


def test_simhash_collision_rate_follows_the_angle():
    """A sign random projection collides with probability 1 - angle/pi (loose statistical check)."""
    o = make(SIMHASH, real="double", H=96, K=8, L=40, N=10, srp_nnz=32)
    r = np.random.default_rng(6)
    for theta in (0.3, 1.0, 2.0):
        agree = total = 0
        for _ in range(60):
            a = r.standard_normal(96)
            b = r.standard_normal(96)
            b -= a * (a @ b) / (a @ a)
            u = a / np.linalg.norm(a) * np.cos(theta) + b / np.linalg.norm(b) * np.sin(theta)
            x = o.hash_vec(a) ^ o.hash_vec(u)
            agree += sum(8 - bin(int(w)).count("1") for w in x)
            total += 8 * 40
        assert abs(agree / total - (1 - theta / np.pi)) < 0.04


def test_dwta_collision_rate_grows_with_similarity():
    o = make(DWTA, real="double", H=64, K=2, L=40, N=10)
    r = np.random.default_rng(7)
    rates = []
    for noise in (0.1, 1.0, 10.0):
        hit = tot = 0
        for _ in range(100):
            a = r.standard_normal(64)
            b = a + noise * r.standard_normal(64)
            hit += int(np.sum(o.hash_vec(a) == o.hash_vec(b)))
            tot += 40
        rates.append(hit / tot)
    assert rates[0] > rates[1] > rates[2]
    assert rates[0] > 0.5 and rates[2] < 0.2


# ---------------------------------------------------------------- tables
@pytest.mark.parametrize("family", [SIMHASH, DWTA])
def test_tables_partition_the_neurons(family):
    o = make(family)
    N, L, nb = o.N, o.L, 1 << o.bits
    off = o.get("bucket_off").reshape(L, nb + 1)
    ids = o.get("bucket_ids").reshape(L, N)
    W2 = o.get("W2").reshape(N, o.H)
    codes = np.stack([o.hash_vec(W2[j]) for j in range(N)])          # [N][L]
    for t in range(L):
        assert off[t, 0] == 0 and off[t, nb] == N
        assert np.all(np.diff(off[t]) >= 0)
        assert sorted(ids[t]) == list(range(N))                      # every neuron exactly once
        for b in range(nb):
            seg = ids[t, off[t, b]:off[t, b + 1]]
            assert np.all(np.diff(seg) > 0)                          # ascending ids
            assert np.all(codes[seg, t] == b)                        # and in the right bucket


@pytest.mark.parametrize("family", [SIMHASH, DWTA])
def test_active_set_equals_scan_over_all_neurons(family):
    """Active set recomputed without the tables: scan every neuron, keep those that share a code with the
    query in some table and are among the `cap` lowest ids with that code, then add the labels."""
    from tests.helpers import small_batch
    o = make(family, bucket_cap=3)
    r = np.random.default_rng(8)
    batch = small_batch(r, 12, o.D, o.N, 10, dtype=np.float32)
    o.forward(*batch)
    W2 = o.get("W2").reshape(o.N, o.H)
    ncode = np.stack([o.hash_vec(W2[j]) for j in range(o.N)])
    h = o.get("h").reshape(12, o.H)
    got = o.active_sets()
    capped_somewhere = False
    for s in range(12):
        q = o.hash_vec(h[s])
        assert np.array_equal(q, o.get("codes").reshape(12, o.L)[s])
        want = set(batch[4][batch[3][s]:batch[3][s + 1]].tolist())
        for t in range(o.L):
            same = np.nonzero(ncode[:, t] == q[t])[0]                 # ascending ids
            capped_somewhere |= len(same) > 3
            want |= set(same[:3].tolist())
        assert got[s].tolist() == sorted(want)
    assert capped_somewhere                                           # the cap was exercised


def test_rebuild_without_redraw_and_unchanged_weights_is_identity():
    o = make(DWTA, redraw=0)
    off, ids = o.get("bucket_off"), o.get("bucket_ids")
    o.rebuild_tables()
    assert o.r == 1
    assert np.array_equal(off, o.get("bucket_off")) and np.array_equal(ids, o.get("bucket_ids"))


def test_rebuild_schedule_closed_form():
    """gap_i = max(1, floor(p0 * exp(lambda * i))): lambda = 0 gives 50, 100, 150, ...; enumerate lambda = 0.5 by hand."""
    from tests.helpers import small_batch
    r = np.random.default_rng(9)
    for lam, want in ((0.0, [5, 10, 15, 20]), (0.5, [5, 13, 26])):     # 5 + floor(5e^.5)=8 -> 13, + floor(5e^1)=13 -> 26
        o = make(SIMHASH, rebuild_period0=5, rebuild_lambda=lam, lr=1e-3)
        seen = []
        for step in range(1, 28 if lam else 21):
            before = o.r
            o.train_step(*small_batch(r, 4, o.D, o.N, 6, dtype=np.float32))
            assert o.t == step
            if o.r != before:
                seen.append(step)
        assert seen == want


# ---------------------------------------------------------------- densification of all-zero DWTA bins
def brute_densified_codes(o, v, K, L, bs, seed, r, attempts=16, stream=3):
    """The definition written out: positions of all bins first, then every all-zero bin borrows."""
    idx = o.get("hash_idx").reshape(K * L, bs)
    vals = v[idx]                                       # [KL][bs]
    pos = np.argmax(vals, axis=1)                       # first maximum = lowest position on ties
    empty = np.all(vals == 0, axis=1)
    KL = K * L
    out = pos.copy()
    for p in np.nonzero(empty)[0]:
        out[p] = 0
        for a in range(attempts):
            g = (int(p) + 1 + orc_rng(seed, stream, r, int(p) * attempts + a) % (KL - 1)) % KL
            if not empty[g]:
                out[p] = pos[g]
                break
    lg = int(np.log2(bs))
    return np.array([sum(int(out[t * K + k]) << (k * lg) for k in range(K)) for t in range(L)], dtype=np.uint32)


def test_densified_query_codes_match_the_definition_written_out():
    rs = np.random.default_rng(11)
    o = make(DWTA, H=64, K=3, L=7, bin_size=8, densify=1, seed=5)
    saw_empty = saw_borrow = 0
    for trial in range(40):
        v = np.maximum(rs.standard_normal(64), 0).astype(np.float32)
        v[rs.random(64) < 0.6] = 0.0                    # ReLU output with most units off
        want = brute_densified_codes(o, v, 3, 7, 8, 5, 0)
        got = o.hash_query(v)
        assert np.array_equal(got, want)
        plain = o.hash_vec(v)                           # neurons' rows are never densified
        idx = o.get("hash_idx").reshape(21, 8)
        empty = np.all(v[idx] == 0, axis=1)
        saw_empty += int(empty.sum())
        saw_borrow += int(np.any(got != plain))
        # a function whose own bin is not empty keeps its position
        for t in range(7):
            for k in range(3):
                if not empty[t * 3 + k]:
                    assert (got[t] >> (3 * k)) & 7 == (plain[t] >> (3 * k)) & 7
    assert saw_empty > 20 and saw_borrow > 5


def test_densification_needs_the_flag_and_a_nonzero_bin_somewhere():
    v = np.zeros(64, dtype=np.float32)
    on = make(DWTA, H=64, K=3, L=7, bin_size=8, densify=1, seed=5)
    off = make(DWTA, H=64, K=3, L=7, bin_size=8, densify=0, seed=5)
    assert np.all(on.hash_query(v) == 0)                # every probe finds an empty bin
    v[on.get("hash_idx")[0]] = 2.0                      # one unit on: only the bins holding it are not empty
    assert np.array_equal(off.hash_query(v), off.hash_vec(v))
    assert np.array_equal(on.hash_vec(v), off.hash_vec(v))
    # the probe sequence is drawn again with the hash functions
    on.draw_hash(1)
    on.set_counters(0, 1, 0)
    assert np.array_equal(on.hash_query(v), brute_densified_codes(on, v, 3, 7, 8, 5, 1))
