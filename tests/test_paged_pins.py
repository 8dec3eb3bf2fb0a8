"""Pins for the oracle's paged-cache forms: the address rule on a hand-written page table, and the fact
that the layout of the pool cannot change what attention or compaction compute."""
import numpy as np

from oracle import dyspec_oracle as orc
from paper_2410_11744_b200 import workloads as wl


def test_address_rule_hand_example():
    # pages of 4 rows; the request owns pages 5, 0, 2 in this order
    assert orc.paged_prefix_rows([5, 0, 2], 4, 10) == [20, 21, 22, 23, 0, 1, 2, 3, 8, 9]
    assert orc.paged_prefix_rows([7], 128, 0) == []
    assert orc.paged_prefix_rows([3, 1], 2, 4) == [6, 7, 2, 3]


def _cases():
    rng = np.random.default_rng(21)
    return [
        wl.make_custom(1, 4, 2, 16, [9], [wl.greedy_tree(rng, 12, 3, 0.3)]),
        wl.make_custom(2, 2, 2, 8, [0, 17, 5, 8], [wl.random_tree(rng, 7), wl.chain_tree(5), np.zeros(0, np.int32),
                                                   wl.star_forest(6)]),
    ]


def test_identity_table_is_the_contiguous_layout():
    """One request whose pages are 0, 1, 2, ... and whose tree rows follow the prefix directly is the
    contiguous cache itself."""
    w = wl.make_custom(3, 4, 1, 16, [11], [wl.chain_tree(6)])
    table = np.arange(4, dtype=np.int32)[None, :]
    got = orc.tree_attention_paged(w.q, w.k, w.v, table, 4, w.prefix_len, w.n_nodes, [11], w.parents)
    ref = orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents)
    assert np.array_equal(got, ref)


def test_scattering_the_pages_changes_nothing():
    for w in _cases():
        ref = orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents)
        for page_size, seed in ((4, 0), (8, 1), (16, 2)):
            pw = wl.to_paged(w, page_size, seed)
            # the scatter really moved things: the filler and the shuffled pages make the pools differ
            assert pw.pool_rows > w.k.shape[0]
            got = orc.tree_attention_paged(w.q, pw.k, pw.v, pw.page_table, page_size, w.prefix_len, w.n_nodes,
                                           pw.tree_row_offset, w.parents)
            assert np.array_equal(got, ref)                     # same keys in the same order: bit-identical


def test_filler_rows_are_never_read():
    """Rows of a page past the prefix and the pages nobody owns hold other values in two pools; the
    result is the same."""
    w = _cases()[1]
    pw = wl.to_paged(w, 8, 5)
    k2, v2 = pw.k.copy(), pw.v.copy()
    used = np.zeros(pw.pool_rows, bool)
    for r in range(w.n_req):
        used[orc.paged_prefix_rows(pw.page_table[r], 8, int(w.prefix_len[r]))] = True
        t = int(pw.tree_row_offset[r])
        used[t:t + int(w.n_nodes[r])] = True
    assert (~used).sum() > 0
    k2[~used] ^= 0x0101
    v2[~used] ^= 0x0101
    a = orc.tree_attention_paged(w.q, pw.k, pw.v, pw.page_table, 8, w.prefix_len, w.n_nodes, pw.tree_row_offset, w.parents)
    b = orc.tree_attention_paged(w.q, k2, v2, pw.page_table, 8, w.prefix_len, w.n_nodes, pw.tree_row_offset, w.parents)
    assert np.array_equal(a, b)


def test_compaction_hand_example():
    pool = np.arange(40, dtype=np.int64).reshape(20, 2)
    ref = pool.copy()
    # pages of 4 rows, the request owns pages 3 then 1; prefix 3 tokens; tree rows start at pool row 16
    new_L = orc.compact_kv_paged(pool, [3, 1], 4, 16, 3, [0, 2, -1, 3])
    assert new_L == 6
    # token 3 -> page 3 row 3 = pool row 15; tokens 4, 5 -> page 1 rows 0, 1 = pool rows 4, 5
    assert np.array_equal(pool[15], ref[16]) and np.array_equal(pool[4], ref[18]) and np.array_equal(pool[5], ref[19])
    untouched = [i for i in range(20) if i not in (15, 4, 5)]
    assert np.array_equal(pool[untouched], ref[untouched])


def test_compaction_matches_the_contiguous_one_read_through_the_table():
    rng = np.random.default_rng(4)
    parents = wl.greedy_tree(rng, 20, 3, 0.3)
    L = 13
    w = wl.make_custom(6, 2, 2, 8, [L], [parents])
    path, j = [], 19
    while j >= 0:
        path.append(j)
        j = int(parents[j])
    path = path[::-1] + [-1]
    cont = w.k.copy()
    new_L = orc.compact_kv(cont, 0, L, path)
    pw = wl.to_paged(w, 4, 9)
    pool = pw.k.copy()
    assert orc.compact_kv_paged(pool, pw.page_table[0], 4, int(pw.tree_row_offset[0]), L, path) == new_L
    rows = orc.paged_prefix_rows(pw.page_table[0], 4, new_L)
    assert np.array_equal(pool[rows], cont[:new_L])
    # nothing else moved
    others = np.setdiff1d(np.arange(pw.pool_rows), rows[L:])
    assert np.array_equal(pool[others], pw.k[others])


def test_paged_compaction_keeps_the_root_like_the_contiguous_one():
    rng = np.random.default_rng(4)
    L, n = 6, 12
    w = wl.make_custom(71, 2, 2, 8, [L], [wl.chain_tree(n)])
    pw = wl.to_paged(w, 4, 3)
    listed = [2, 5, 9, -1]
    cont = w.k.copy()
    pool = pw.k.copy()
    new_L = orc.compact_kv(cont, 0, L, listed, keep_root=True)
    assert orc.compact_kv_paged(pool, pw.page_table[0], 4, int(pw.tree_row_offset[0]), L, listed, keep_root=True) == new_L == L + 4
    rows = orc.paged_prefix_rows(pw.page_table[0], 4, new_L)
    assert np.array_equal(pool[rows], cont[:new_L])
    assert np.array_equal(pool[rows[L]], w.k[L])                          # token L is the root's row


# ---- tree rows inside the paged sequence (tokens L .. L + n - 1 of the request's pages) ----------------
def test_tree_rows_inside_the_pages_change_nothing():
    """The same keys in the same order, whatever pages the tree rows lie in: bit-identical to the
    contiguous form, also when a tree crosses page boundaries at an odd offset."""
    for w in _cases():
        ref = orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents)
        for page_size, seed in ((4, 0), (8, 1), (16, 2)):
            pw = wl.to_paged(w, page_size, seed, tree_in_pages=True)
            assert pw.tree_row_offset is None
            got = orc.tree_attention_paged(w.q, pw.k, pw.v, pw.page_table, page_size, w.prefix_len, w.n_nodes,
                                           None, w.parents)
            assert np.array_equal(got, ref)


def test_tree_rows_inside_the_pages_hand_example():
    """Pages of 4 rows, the request owns pages 2 then 0; prefix 3 tokens, 3 nodes: node 0 is token 3
    (pool row 11), nodes 1 and 2 are tokens 4, 5 (pool rows 0, 1).  A star forest sees prefix + self only:
    V of the node's own row leaks into its output and nobody else's."""
    w = wl.make_custom(5, 1, 1, 8, [3], [wl.star_forest(3)])
    pw = wl.to_paged(w, 4, 0, tree_in_pages=True)
    table = pw.page_table[0]
    rows = [int(table[t // 4]) * 4 + t % 4 for t in range(6)]
    assert np.array_equal(pw.k[rows], w.k[:6]) and np.array_equal(pw.v[rows], w.v[:6])
    base = orc.tree_attention_paged(w.q, pw.k, pw.v, pw.page_table, 4, w.prefix_len, w.n_nodes, None, w.parents)
    v2 = pw.v.copy()
    v2[rows[4]] ^= 0x0040                                    # node 1's own V row
    moved = orc.tree_attention_paged(w.q, pw.k, v2, pw.page_table, 4, w.prefix_len, w.n_nodes, None, w.parents)
    assert not np.array_equal(moved[1], base[1])
    assert np.array_equal(moved[0], base[0]) and np.array_equal(moved[2], base[2])


def test_in_sequence_compaction_is_the_contiguous_one_read_through_the_table():
    """Source and destination rows overlap here (token L + 1 receives node 2 after node 1 ... was read):
    the definition is a gather, as in the contiguous form."""
    L, n = 6, 12
    w = wl.make_custom(72, 2, 2, 8, [L], [wl.chain_tree(n)])
    for listed, keep_root in (([1, 2, 3, -1], False), ([1, 2, 3, -1], True), ([2, 5, 9], True), ([0, 1, 2], False), ([], True)):
        cont = w.k.copy()
        new_L = orc.compact_kv(cont, 0, L, listed, keep_root=keep_root)
        pw = wl.to_paged(w, 4, 3, tree_in_pages=True)
        pool = pw.k.copy()
        assert orc.compact_kv_paged(pool, pw.page_table[0], 4, None, L, listed, keep_root=keep_root) == new_L
        rows = orc.paged_prefix_rows(pw.page_table[0], 4, L + n)
        assert np.array_equal(pool[rows], cont[:L + n])       # kept rows moved, everything behind them as it was
        others = np.setdiff1d(np.arange(pw.pool_rows), rows)
        assert np.array_equal(pool[others], pw.k[others])
