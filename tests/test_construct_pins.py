"""Pins for the oracle's tree construction (Algorithms 1 and 2): what the paper states about them.

* values come out in non-increasing order (Sec. 4.2 / App. B: "tokens with decreasing acceptance rate");
* the estimated acceptance rate of a node is the product of its ancestors' probabilities times the
  probability that all earlier guesses at its position failed (App. B) -- which telescopes to a
  closed form in the RAW draft probabilities, recomputed here from the output tree alone;
* with the threshold set to the value of the last node, Algorithm 2 gives exactly the tree of
  Algorithm 1 (App. B);
* the first guess at a position is distributed as the draft row, the second as the row with the first
  removed and renormalised (sampling without replacement, Sec. 4.1)."""
import numpy as np
import pytest

from oracle import dyspec_oracle as orc


def _table(seed, T, V, sharp):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, V)) * sharp
    e = np.exp(x - x.max(axis=1, keepdims=True))
    return e / e.sum(axis=1, keepdims=True), rng.random(997)


def _paths(res):
    out = {}
    for k in range(1, len(res["parents"])):
        path, j = [], k
        while j > 0:
            path.append(int(res["tokens"][j]))
            j = int(res["parents"][j])
        out[tuple(reversed(path))] = k
    return out


@pytest.mark.parametrize("seed,T,V,sharp,m", [(0, 16, 50, 1.5, 40), (1, 64, 300, 2.5, 120), (2, 8, 12, 0.5, 30)])
def test_greedy_values_decrease_and_match_closed_form(seed, T, V, sharp, m):
    rows, uni = _table(seed, T, V, sharp)
    res = orc.build_tree_greedy(rows, uni, m)
    par, tok, val, cval, nrow = res["parents"], res["tokens"], res["values"], res["child_values"], res["rows"]
    assert len(par) == m + 1 and par[0] == -1
    assert all(0 <= par[k] < k for k in range(1, m + 1))
    assert np.all(np.diff(val[1:]) <= 1e-15)                       # pop order = decreasing estimated acceptance rate
    for p in range(m + 1):                                           # siblings carry different tokens
        sib = [int(tok[k]) for k in range(1, m + 1) if par[k] == p]
        assert len(sib) == len(set(sib))
    # closed forms in the raw probabilities: cv(k) = product of D[token] along the path;
    # v(k) = cv(parent) * (1 - sum of the raw probabilities of the earlier siblings)
    prod = np.ones(m + 1)
    for k in range(1, m + 1):
        p = int(par[k])
        prod[k] = prod[p] * rows[nrow[p]][tok[k]]
        earlier = [int(tok[s]) for s in range(1, k) if par[s] == p]
        assert abs(val[k] - prod[p] * (1.0 - rows[nrow[p]][earlier].sum())) <= 1e-12
        assert abs(cval[k] - prod[k]) <= 1e-12
        assert nrow[k] == orc.draft_row_of_child(int(nrow[p]), int(tok[k]), T)


@pytest.mark.parametrize("seed,T,V,sharp,m", [(3, 32, 80, 2.0, 25), (4, 32, 400, 3.0, 64), (5, 8, 10, 0.3, 40)])
def test_threshold_at_last_value_reproduces_the_greedy_tree(seed, T, V, sharp, m):
    rows, uni = _table(seed, T, V, sharp)
    a = orc.build_tree_greedy(rows, uni, m)
    t = a["values"][-1]
    if np.sum(np.isclose(a["values"][1:], t, rtol=1e-12, atol=0)) > 1:
        pytest.skip("tie at the threshold")
    b = orc.build_tree_threshold(rows, uni, t, 10 * m)
    pa, pb = _paths(a), _paths(b)
    assert set(pa) == set(pb)
    for path, k in pa.items():
        assert abs(a["values"][k] - b["values"][pb[path]]) <= 1e-12
    # a slightly higher threshold drops exactly the last node
    c = orc.build_tree_threshold(rows, uni, np.nextafter(t, 1.0) * (1 + 1e-9), 10 * m)
    assert len(c["parents"]) <= len(a["parents"]) - 1
    assert set(_paths(c)) <= set(pa)


def test_threshold_tree_layer_order_and_cap():
    rows, uni = _table(6, 16, 40, 2.0)
    res = orc.build_tree_threshold(rows, uni, 0.02, 1000)
    par, val = res["parents"], res["values"]
    assert all(0 <= par[k] < k for k in range(1, len(par)))
    assert np.all(val[1:] >= 0.02)
    depth = np.zeros(len(par), int)
    for k in range(1, len(par)):
        depth[k] = depth[par[k]] + 1
    assert np.all(np.diff(depth) >= 0)                             # layer by layer
    capped = orc.build_tree_threshold(rows, uni, 0.02, 7)
    assert len(capped["parents"]) == 8
    assert np.array_equal(capped["parents"], par[:8]) and np.array_equal(capped["tokens"], res["tokens"][:8])


def test_guesses_at_a_position_are_draws_without_replacement():
    V = 5
    rng = np.random.default_rng(12)
    row = rng.dirichlet(np.ones(V))
    rows = np.tile(row, (4, 1))
    first = np.zeros(V)
    second = np.zeros((V, V))
    trials = 30000
    for _ in range(trials):
        res = orc.build_tree_threshold(rows, rng.random(64), 0.0, 2)        # two guesses at the root
        y1, y2 = int(res["tokens"][1]), int(res["tokens"][2])
        assert res["parents"][2] == 0 and y1 != y2
        first[y1] += 1
        second[y1, y2] += 1
    f = first / trials
    assert np.all(np.abs(f - row) <= 4.5 * np.sqrt(row * (1 - row) / trials))
    for a in range(V):
        n_a = second[a].sum()
        cond = row.copy(); cond[a] = 0; cond /= cond.sum()
        if n_a > 1500:
            assert np.all(np.abs(second[a] / n_a - cond) <= 4.5 * np.sqrt(cond * (1 - cond) / n_a) + 1e-9)
