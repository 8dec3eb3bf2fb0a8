"""Pins for the oracle's accepted-path KV compaction."""
import numpy as np

from oracle import dyspec_oracle as orc
from paper_2410_11744_b200 import workloads as wl


def test_hand_example_and_noop():
    cache = np.arange(12 * 2, dtype=np.int64).reshape(12, 2)           # row r = (2r, 2r+1)
    ref = cache.copy()
    new_L = orc.compact_kv(cache, kv_row0=2, prefix_len=3, accepted_nodes=[1, 3, 4, -1])
    assert new_L == 6
    # prefix rows 2..4 untouched; rows 5, 6, 7 = old rows of nodes 1, 3, 4 = old rows 6, 8, 9
    assert np.array_equal(cache[:5], ref[:5])
    assert np.array_equal(cache[5], ref[6]) and np.array_equal(cache[6], ref[8]) and np.array_equal(cache[7], ref[9])
    assert np.array_equal(cache[8:], ref[8:])                           # rows past the new prefix keep their old content
    c2 = ref.copy()
    assert orc.compact_kv(c2, 2, 3, [0, 1, 2]) == 6 and np.array_equal(c2, ref)   # a chain prefix is already in place
    assert orc.compact_kv(c2, 2, 3, []) == 3 and np.array_equal(c2, ref)


def test_overlapping_moves_are_a_gather():
    # path 1, 2, 3: node 1's row moves to slot 0, node 2's to slot 1 (which node 1 occupied), ...
    cache = np.arange(8, dtype=np.int64).reshape(8, 1)
    orc.compact_kv(cache, 0, 2, [1, 2, 3])
    assert cache[:, 0].tolist() == [0, 1, 3, 4, 5, 5, 6, 7]


def test_next_step_attention_sees_the_accepted_path():
    """A token decoded after the step must attend to prefix + accepted path: a one-node tree over the
    compacted cache gives what the last path node's query would get from the tree attention over the
    original cache, if its query is reused (same visible keys in the same order)."""
    rng = np.random.default_rng(8)
    parents = wl.greedy_tree(rng, 24, 4, 0.3)
    L = 7
    w = wl.make_custom(5, 4, 2, 16, [L], [parents])
    path, j = [], 23
    while j >= 0:
        path.append(j)
        j = int(parents[j])
    path = path[::-1]                                                    # root .. node 23
    full = orc.tree_attention(w.q, w.k, w.v, L, parents)
    k2, v2 = w.k.copy(), w.v.copy()
    new_L = orc.compact_kv(k2, 0, L, path)
    assert orc.compact_kv(v2, 0, L, path) == new_L == L + len(path)
    # query of node 23 as a single new "tree" whose own K/V row is the last path row
    one = orc.tree_attention(w.q[23:24], k2[:new_L], v2[:new_L], new_L - 1, [-1])
    assert np.abs(one[0] - full[23]).max() < 1e-13
