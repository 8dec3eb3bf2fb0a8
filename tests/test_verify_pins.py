"""Pins for the oracle's tree verification (Algorithm 3): properties the mathematics fixes.

The central one: whatever the draft distribution and the tree, the first emitted token is distributed
exactly as the target distribution at the root, provided the branches of a node are drawn from the
draft distribution without replacement (which is how the tree is built, Sec. 4.1).  Checked by Monte
Carlo with the oracle as a black box; a wrong residual, a missing renormalisation, a swapped ratio or
a wrong inverse CDF all break it."""
import numpy as np
import pytest

from oracle import dyspec_oracle as orc


def _draw_children(rng, D, k):
    """k tokens from D without replacement, each from the renormalised remainder."""
    D = D.copy()
    out = []
    for _ in range(k):
        if D.sum() <= 0:
            break
        D = D / D.sum()
        y = int(rng.choice(len(D), p=D))
        out.append(y)
        D[y] = 0.0
    return out


def _random_dist(rng, V, zero=0):
    p = rng.dirichlet(np.full(V, 0.7))
    if zero:
        p[rng.choice(V, size=zero, replace=False)] = 0.0
        p = p / p.sum()
    return p


@pytest.mark.parametrize("V,k,seed", [(4, 1, 0), (4, 2, 1), (5, 3, 2), (3, 3, 3), (6, 2, 4)])
def test_first_token_follows_the_target_distribution(V, k, seed):
    rng = np.random.default_rng(seed)
    D0 = _random_dist(rng, V, zero=1 if V > 4 else 0)
    T0 = _random_dist(rng, V)
    trials = 40000
    counts = np.zeros(V)
    for _ in range(trials):
        toks = _draw_children(rng, D0, k)
        n = 1 + len(toks)
        parents = [-1] + [0] * len(toks)
        tokens = [0] + toks
        Dm = np.tile(D0, (n, 1))
        Tm = np.tile(T0, (n, 1))
        A, nodes, _ = orc.verify_tree(parents, tokens, Dm, Tm, rng.random(n), rng.random(n))
        counts[A[0]] += 1
    freq = counts / trials
    sigma = np.sqrt(T0 * (1 - T0) / trials)
    assert np.all(np.abs(freq - T0) <= 4.5 * sigma + 1e-9), (freq, T0)


def test_two_levels_follow_the_target_chain():
    """Depth 2: P(first = a, second = b) = T(root, a) * T(child a, b) whenever a was speculated."""
    rng = np.random.default_rng(11)
    V = 3
    D0, T0 = _random_dist(rng, V), _random_dist(rng, V)
    D1 = [_random_dist(rng, V) for _ in range(V)]      # distributions after token a
    T1 = [_random_dist(rng, V) for _ in range(V)]
    trials = 60000
    pair = np.zeros((V, V))
    first_only = np.zeros(V)
    for _ in range(trials):
        parents, tokens, Dm, Tm = [-1], [0], [D0], [T0]
        for a in _draw_children(rng, D0, 2):
            node = len(parents)
            parents.append(0); tokens.append(a); Dm.append(D1[a]); Tm.append(T1[a])
        for node in (1, 2):
            a = tokens[node]
            for b in _draw_children(rng, D1[a], 2):
                parents.append(node); tokens.append(b); Dm.append(D0); Tm.append(T0)
        n = len(parents)
        A, nodes, _ = orc.verify_tree(parents, tokens, np.array(Dm), np.array(Tm), rng.random(n), rng.random(n))
        if len(nodes) >= 1:                        # the first token was a speculated one: a second token follows
            assert len(A) >= 2
            pair[A[0], A[1]] += 1
        else:
            first_only[A[0]] += 1
    first = (pair.sum(axis=1) + first_only) / trials
    assert np.all(np.abs(first - T0) <= 4.5 * np.sqrt(T0 * (1 - T0) / trials))
    for a in range(V):
        m = pair[a].sum()
        if m > 2000:
            cond = pair[a] / m
            assert np.all(np.abs(cond - T1[a]) <= 4.5 * np.sqrt(T1[a] * (1 - T1[a]) / m) + 1e-9)


def test_draft_equal_to_target_accepts_every_first_branch():
    rng = np.random.default_rng(5)
    V = 7
    parents = [-1, 0, 0, 1, 1, 3]
    tokens = [0, 2, 5, 1, 4, 6]
    P = np.array([_random_dist(rng, V) for _ in parents])
    P[:, tokens] += 0.05                                 # every speculated token has mass
    P = P / P.sum(axis=1, keepdims=True)
    A, nodes, _ = orc.verify_tree(parents, tokens, P, P, rng.random(6) * 0.999, rng.random(6))
    assert nodes == [1, 3, 5] and A == [2, 1, 6]          # first child each time; node 5 is a leaf: the walk ends
    A2, nodes2, _ = orc.verify_tree(parents, tokens, P, P, rng.random(6) * 0.999, rng.random(6), bonus_at_leaf=True)
    assert nodes2 == [1, 3, 5] and A2[:3] == [2, 1, 6] and len(A2) == 4


def test_single_branch_acceptance_rate_is_min_1_ratio():
    D = np.array([[0.8, 0.2], [0.5, 0.5]])
    T = np.array([[0.4, 0.6], [0.5, 0.5]])
    us = (np.arange(2000) + 0.5) / 2000
    acc = sum(len(orc.verify_tree([-1, 0], [0, 0], D, T, [0.0, u], [0.3, 0.3])[1]) for u in us)
    assert abs(acc / 2000 - 0.5) < 1e-3                  # token 0: T/D = 0.5
    acc = sum(len(orc.verify_tree([-1, 0], [0, 1], D, T, [0.0, u], [0.3, 0.3])[1]) for u in us)
    assert acc == 2000                                    # token 1: T/D = 3 > 1: always accepted
    # rejected token 0: residual = norm(max(T - D, 0)) = (0, 1): the emitted token is 1 whatever sample_u is
    for su in (0.0, 0.4, 0.999):
        A, nodes, _ = orc.verify_tree([-1, 0], [0, 0], D, T, [0.0, 0.9], [su, su])
        assert A == [1] and nodes == []


def test_zero_target_mass_is_never_accepted_and_all_zero_draft_stops():
    D = np.array([[0.0, 1.0, 0.0], [1 / 3, 1 / 3, 1 / 3], [1 / 3, 1 / 3, 1 / 3]])
    T = np.array([[0.5, 0.0, 0.5], [1 / 3, 1 / 3, 1 / 3], [1 / 3, 1 / 3, 1 / 3]])
    # child 1 carries token 1 (target mass 0): rejected for any c > 0; the draft is then all zero -> stop,
    # child 2 is never tried; the residual is norm(max(T - D, 0)) = (0.5, 0, 0.5)
    A, nodes, _ = orc.verify_tree([-1, 0, 0], [0, 1, 0], D, T, [0.0, 1e-9, 0.0], [0.6, 0.0, 0.0])
    assert nodes == [] and A == [2]
    A, nodes, _ = orc.verify_tree([-1, 0, 0], [0, 1, 0], D, T, [0.0, 1e-9, 0.0], [0.4, 0.0, 0.0])
    assert A == [0]


def test_inverse_cdf_sampling_order():
    T = np.array([[0.1, 0.2, 0.3, 0.4]])
    D = T.copy()
    for u, want in [(0.0, 0), (0.0999, 0), (0.1001, 1), (0.2999, 1), (0.3001, 2), (0.6001, 3), (0.9999, 3)]:
        A, _, _ = orc.verify_tree([-1], [0], D, T, [0.0], [u], bonus_at_leaf=True)
        assert A == [want]
    assert orc.verify_tree([-1], [0], D, T, [0.0], [0.5])[0] == []     # as printed: a lone root emits nothing
