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
