"""Pins for the token-reorder functions of the oracle (App. C): the paper's printed block counts
(Table 5), closed forms, and the invariance of attention under the renumbering."""
import os

import numpy as np
import pytest

from oracle import dyspec_oracle as orc
from paper_2410_11744_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table5_block_counts.txt")


def _table5():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                n, a, b = line.split()
                rows.append((int(n), float(a), float(b)))
    return rows


@pytest.mark.parametrize("n,paper_orig,paper_dfs", _table5())
def test_block_counts_reproduce_table5(n, paper_orig, paper_dfs):
    """Uniform random recursive trees (parent of node i uniform in [0, i)), block 32: the mean block
    count in creation order and after DFS renumbering matches the paper's Table 5."""
    rng = np.random.default_rng(1000 + n)
    trials = 24 if n <= 1024 else 8
    orig, dfs = [], []
    for _ in range(trials):
        p = wl.random_tree(rng, n)
        orig.append(orc.mask_block_count(p, 32))
        new_p, _ = orc.relabel_tree(p, orc.dfs_order(p))
        dfs.append(orc.mask_block_count(new_p, 32))
    t = n // 32
    assert max(orig) <= t * (t + 1) // 2                       # never more than the full lower triangle
    assert abs(np.mean(orig) - paper_orig) <= 0.015 * paper_orig + 0.5
    # Children visited in index order is the reading that fits: within 5 % up to 1024 nodes and about
    # 8 % low at 2048 (sample std there is ~10 blocks and the paper does not give its sample count);
    # visiting children in reverse index order lands 27 % high, ordering children by subtree size 15 % low.
    assert abs(np.mean(dfs) - paper_dfs) <= (0.05 if n <= 1024 else 0.10) * paper_dfs
    assert np.mean(dfs) < np.mean(orig)


def test_block_count_closed_forms():
    # chain: the mask is the full lower triangle -> T (T + 1) / 2 blocks; star: the diagonal -> T blocks
    assert orc.mask_block_count(wl.chain_tree(96), 32) == 6
    assert orc.mask_block_count(wl.chain_tree(100), 32) == 10
    assert orc.mask_block_count(wl.star_forest(100), 32) == 4
    # hand example, block 2: parents -1 0 0 1 -> mask rows {0},{0,1},{0,2},{0,1,3}: blocks (0,0),(1,0),(1,1)
    assert orc.mask_block_count([-1, 0, 0, 1], 2) == 3


def test_dfs_order_hand_example():
    #        0            7
    #       / \           |
    #      1   2          8          pre-order, children by index: 0 1 3 6 4 2 5 7 8
    #     / \   \
    #    3   4   5
    #    |
    #    6
    parents = [-1, 0, 0, 1, 1, 2, 3, -1, 7]
    order = orc.dfs_order(parents)
    assert order == [0, 1, 3, 6, 4, 2, 5, 7, 8]
    new_p, new_of_old = orc.relabel_tree(parents, order)
    assert new_p.tolist() == [-1, 0, 1, 2, 1, 0, 5, -1, 7]
    assert new_of_old.tolist() == [0, 1, 5, 2, 4, 6, 3, 7, 8]


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_dfs_order_properties(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 300))
    p = wl.random_tree(rng, n, p_root=0.05)
    order = orc.dfs_order(p)
    assert sorted(order) == list(range(n))
    new_p, new_of_old = orc.relabel_tree(p, order)
    assert all(new_p[k] < k for k in range(n))                  # still a valid creation order
    # a DFS numbering makes every subtree a contiguous index range [k, k + size)
    size = np.ones(n, dtype=np.int64)
    for k in range(n - 1, -1, -1):
        if new_p[k] >= 0:
            size[new_p[k]] += size[k]
    _, depth_new = orc.build_tree_mask(new_p, 4 * ((n + 127) // 128))
    for k in range(n):
        for d in range(k + 1, k + int(size[k])):
            j = d
            while depth_new[j] > depth_new[k]:
                j = new_p[j]
            assert j == k
    # depths are carried along
    _, depth_old = orc.build_tree_mask(p, 4 * ((n + 127) // 128))
    assert [int(depth_old[o]) for o in order] == depth_new.tolist()


def test_attention_is_invariant_under_dfs_renumbering():
    rng = np.random.default_rng(5)
    p = wl.greedy_tree(rng, 40, 4, 0.3)
    L = 9
    w = wl.make_custom(6, 4, 2, 16, [L], [p])
    base = orc.tree_attention(w.q, w.k, w.v, L, p)
    order = orc.dfs_order(p)
    new_p, _ = orc.relabel_tree(p, order)
    k2 = np.concatenate([w.k[:L], w.k[L:][order]])
    v2 = np.concatenate([w.v[:L], w.v[L:][order]])
    out2 = orc.tree_attention(w.q[order], k2, v2, L, new_p)
    assert np.abs(out2 - base[order]).max() < 1e-13
