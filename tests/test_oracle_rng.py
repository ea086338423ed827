"""Pins of the oracle's random numbers and weight initialisation (Algorithm 1, "Initialize layers with
randomly generated weights"; the counter-based generator feeds the hash functions, the sampling budget
and the densification probes as well).

  * the generator's output function against the published outputs of splitmix64 (tests/golden/),
  * orc_rng(seed, stream, r, ctr) against the three rounds expanded by hand for fixed tuples,
  * the initial weights against N(0, sigma^2): moments, a Kolmogorov-Smirnov distance, independence of
    the W1 and W2 streams and of neighbouring draws, and the draw at position i not depending on the
    size of the array.
"""
import os

import numpy as np
import pytest
from scipy import stats

from oracle import oracle as orc
from oracle.oracle import Oracle

from tests.helpers import GOLDEN

M64 = (1 << 64) - 1
GOLD = 0x9E3779B97F4A7C15


def golden_splitmix():
    out = []
    with open(os.path.join(GOLDEN, "splitmix64_reference.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(int(line.split()[1]))
    return out


def test_output_function_reproduces_published_splitmix64_outputs():
    """Output k of splitmix64 seeded with s is mix(s + k * GOLD): a wrong constant or shift fails here."""
    want = golden_splitmix()
    assert len(want) == 5
    seed = 1234567
    got = [orc.mix64((seed + (k + 1) * GOLD) & M64) for k in range(5)]
    assert got == want


def test_first_round_of_the_counter_generator_is_a_splitmix_output():
    """orc_rng's first round is output (stream + 1) of splitmix64(seed); with that value as the next
    round's seed the same holds for r and for the counter: three nested published sequences."""
    want = golden_splitmix()
    seed = 1234567
    for stream in range(5):
        a = want[stream]                                  # published: output stream + 1 of seed 1234567
        for r in (0, 3):
            b = orc.mix64((a + (r + 1) * GOLD) & M64)     # output function, pinned above
            for ctr in (0, 1, 77):
                assert orc.rng(seed, stream, r, ctr) == orc.mix64((b + (ctr + 1) * GOLD) & M64)


def test_counter_generator_hand_expanded_tuple():
    """(seed 1234567, stream 0, r 0, ctr 0): every round is the FIRST output of a splitmix64 generator seeded
    with the previous round's value; the first round's value is the published 6457827717110365317."""
    def first_output(seed):
        z = (seed + GOLD) & M64
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
        return z ^ (z >> 31)
    a = first_output(1234567)
    assert a == 6457827717110365317
    assert orc.rng(1234567, 0, 0, 0) == first_output(first_output(a))
    # words must not be interchangeable
    assert len({orc.rng(1, 2, 3, 4), orc.rng(2, 1, 3, 4), orc.rng(1, 3, 2, 4), orc.rng(1, 2, 4, 3)}) == 4


@pytest.fixture(scope="module")
def big():
    # 2 x 524,288 draws: W1[4096][128] and W2[4096][128]
    o = Oracle("double", D=4096, H=128, N=4096, family=orc.SIMHASH, K=2, L=1, init_std=0.05, seed=11)
    yield o
    o.close()


def test_initial_weights_are_gaussian(big):
    sigma = 0.05
    for name in ("W1", "W2"):
        w = big.get(name)
        n = w.size
        assert n == 4096 * 128
        assert abs(w.mean()) < 5 * sigma / np.sqrt(n)
        assert abs(w.std() / sigma - 1.0) < 5 / np.sqrt(2 * n)
        z = w / sigma
        assert abs(np.mean(z ** 3)) < 5 * np.sqrt(15.0 / n)              # skewness 0
        assert abs(np.mean(z ** 4) - 3.0) < 5 * np.sqrt(96.0 / n)        # kurtosis 3
        d, p = stats.kstest(z, "norm")
        assert d < 1.95 / np.sqrt(n)                                     # 0.1 % critical value of the KS distance
        # tails: a uniform mapped wrongly (a missing +0.5, a clipped log) shows here
        assert 2e-3 < np.mean(np.abs(z) > 3.0) < 3.4e-3                  # 2 * (1 - Phi(3)) = 2.70e-3
    assert np.all(big.get("b1") == 0) and np.all(big.get("b2") == 0)
    for m in ("mW1", "vW1", "mW2", "vW2", "mb1", "vb1", "mb2", "vb2"):
        assert np.all(big.get(m) == 0)


def test_initial_weight_streams_are_independent(big):
    w1, w2 = big.get("W1"), big.get("W2")
    n = w1.size
    bound = 5 / np.sqrt(n)
    assert abs(np.corrcoef(w1, w2)[0, 1]) < bound                        # the two layers use different streams
    for lag in (1, 2, 128):
        assert abs(np.corrcoef(w1[:-lag], w1[lag:])[0, 1]) < bound       # neighbouring draws (cos/sin pairs, rows)
    assert not np.array_equal(w1, w2)


def test_initial_weight_at_position_i_does_not_depend_on_the_array_size(big):
    small = Oracle("double", D=50, H=128, N=70, family=orc.SIMHASH, K=2, L=1, init_std=0.05, seed=11)
    try:
        assert np.array_equal(small.get("W1"), big.get("W1")[:50 * 128])
        assert np.array_equal(small.get("W2"), big.get("W2")[:70 * 128])
    finally:
        small.close()
    other = Oracle("double", D=50, H=128, N=70, family=orc.SIMHASH, K=2, L=1, init_std=0.05, seed=12)
    try:
        assert not np.array_equal(other.get("W1"), big.get("W1")[:50 * 128])
    finally:
        other.close()


def test_initial_weight_from_the_pinned_generator(big):
    """Element i is sigma * sqrt(-2 ln u1) * cos(2 pi u2) with u = (x >> 11 + 1/2) / 2^53 of draws 2i and 2i + 1
    of the layer's stream: rebuilt here from the generator pinned above, for a few positions."""
    for name, stream in (("W1", 0), ("W2", 1)):
        w = big.view(name)
        for i in (0, 1, 12345, w.size - 1):
            u1 = ((orc.rng(11, stream, 0, 2 * i) >> 11) + 0.5) / 2.0 ** 53
            u2 = ((orc.rng(11, stream, 0, 2 * i + 1) >> 11) + 0.5) / 2.0 ** 53
            want = 0.05 * np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
            assert abs(w[i] - want) <= 1e-15 + 1e-12 * abs(want)
