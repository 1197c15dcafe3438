"""Pins for the oracle's nucleus sampler (Section 2: smallest set of tokens whose cumulative probability
reaches p, one token drawn from it in proportion to probability)."""
import itertools
import math

import numpy as np
import pytest

from oracle import spd_oracle as so


def _softmax(z, t):
    e = np.exp(z / t - np.max(z / t))
    return e / e.sum()


def _brute_nucleus(prob, p):
    """The definition by exhaustive search: among all subsets with mass >= p, the fewest tokens; among those,
    the largest mass; ids as a set."""
    v = len(prob)
    for size in range(1, v + 1):
        best = None
        for sub in itertools.combinations(range(v), size):
            mass = math.fsum(prob[list(sub)])
            if mass >= p and (best is None or mass > best[0]):
                best = (mass, set(sub))
        if best is not None:
            return best
    return math.fsum(prob), set(range(v))


@pytest.mark.parametrize("seed", range(6))
def test_nucleus_is_the_smallest_sufficient_subset(seed):
    rng = np.random.default_rng(seed)
    v = 9
    z = rng.normal(0.0, 2.0, v)
    t = [0.7, 1.0, 1.6][seed % 3]
    prob = _softmax(z, t)
    for p in (0.05, 0.3, 0.55, 0.8, 0.95, 1.0):
        mass, members = _brute_nucleus(prob, min(p, math.fsum(prob)))
        _, info = so.nucleus(z, t, p, 0.0)
        assert info["size"] == len(members)
        assert info["mass"] == pytest.approx(mass, rel=1e-12)
        # every draw lands inside the set, and every member wider than the grid of draws is drawn
        seen = {so.nucleus(z, t, p, u)[0] for u in np.linspace(0.0, 0.999999, 4001)}
        assert seen <= members
        assert {i for i in members if prob[i] / mass > 2.0 / 4000} <= seen


def test_uniform_logits_closed_form():
    """All probabilities equal 1/V: the nucleus is the first ceil(p V) ids, draw u takes id floor(u * size)."""
    v = 10
    z = np.full(v, 0.37)
    for p, size in ((0.05, 1), (0.11, 2), (0.45, 5), (0.55, 6), (0.95, 10), (1.0, 10)):   # away from multiples of 1/V
        for u in (0.0, 0.09, 0.31, 0.52, 0.77, 0.999):                                        # away from multiples of 1/size
            tok, info = so.nucleus(z, 1.3, p, u)
            assert info["size"] == size
            assert tok == int(math.floor(u * size))


def test_two_point_distribution():
    """Probabilities (a, 1-a) with a > 1/2: p <= a keeps only token 0; above it both, split at u = a."""
    a = 0.8
    z = np.array([math.log(a), math.log(1 - a)])
    assert so.nucleus(z, 1.0, 0.5, 0.99)[0] == 0
    assert so.nucleus(z, 1.0, 0.79, 0.99)[1]["size"] == 1
    assert so.nucleus(z, 1.0, 0.81, 0.0)[1]["size"] == 2
    assert so.nucleus(z, 1.0, 0.9, 0.79)[0] == 0
    assert so.nucleus(z, 1.0, 0.9, 0.81)[0] == 1
    # temperature 1/2 squares the odds: 16 : 1
    assert so.nucleus(z, 0.5, 0.9, 0.93)[0] == 0 and so.nucleus(z, 0.5, 0.99, 0.95)[0] == 1


def test_small_p_is_greedy_and_ties_go_to_the_lower_id():
    rng = np.random.default_rng(3)
    z = rng.normal(0, 1, 50)
    assert so.nucleus(z, 1.0, 1e-6, 0.9)[0] == int(np.argmax(z))
    z[7] = z[31] = z.max() + 1.0
    assert so.nucleus(z, 1.0, 1e-6, 0.9)[0] == 7
    tok, info = so.nucleus(z, 0.01, 0.75, 0.9)   # two tokens hold all the mass, half each
    assert info["size"] == 2 and tok == 31


def test_draw_frequencies_follow_the_renormalised_probabilities():
    rng = np.random.default_rng(11)
    z = rng.normal(0, 1.5, 12)
    prob = _softmax(z, 1.0)
    order = np.argsort(-prob, kind="stable")
    p = 0.9
    size = int(np.searchsorted(np.cumsum(prob[order]), p) + 1)
    keep = order[:size]
    n = 200000
    us = (np.arange(n) + 0.5) / n
    counts = np.zeros(12)
    for u in us[::20]:
        counts[so.nucleus(z, 1.0, p, float(u))[0]] += 1
    freq = counts / counts.sum()
    want = np.zeros(12)
    want[keep] = prob[keep] / prob[keep].sum()
    assert np.max(np.abs(freq - want)) < 2e-4
    assert set(np.nonzero(counts)[0]) == set(keep.tolist())


def test_margins_report_the_distance_to_the_decision_boundaries():
    z = np.log(np.array([0.5, 0.3, 0.2]))
    tok, info = so.nucleus(z, 1.0, 0.7, 0.5)          # nucleus {0, 1}, mass 0.8, target 0.4 -> token 0
    assert tok == 0 and info["size"] == 2
    assert info["mass"] == pytest.approx(0.8) and info["gap_cut"] == pytest.approx(0.1)
    assert info["gap_draw"] == pytest.approx(0.1)
