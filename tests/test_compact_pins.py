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


def test_keep_root_hand_example():
    """What dyspec_verify_tree hands over lists only the accepted children (and -1 for a drawn token); the
    walk's start node, tree row 0, stays in front of them."""
    cache = np.arange(12 * 2, dtype=np.int64).reshape(12, 2)
    ref = cache.copy()
    new_L = orc.compact_kv(cache, kv_row0=2, prefix_len=3, accepted_nodes=[2, 5, -1], keep_root=True)
    assert new_L == 3 + 1 + 2
    assert np.array_equal(cache[:6], ref[:6])                          # prefix rows 2..4 and the root's row 5 stay
    assert np.array_equal(cache[6], ref[7]) and np.array_equal(cache[7], ref[10])
    assert np.array_equal(cache[8:], ref[8:])
    c2 = ref.copy()
    assert orc.compact_kv(c2, 2, 3, [], keep_root=True) == 3 and np.array_equal(c2, ref)     # nothing emitted: nothing kept
    assert orc.compact_kv(c2, 2, 3, [-1], keep_root=True) == 4 and np.array_equal(c2, ref)   # only a drawn token: the root stays
    assert orc.kept_nodes([3, -1, 7], True) == [0, 3, 7] and orc.kept_nodes([3, -1, 7], False) == [3, 7]


def test_verify_then_compact_gives_the_causal_sequence_prefix_root_path():
    """Algorithm 3 walks from the root; the sequence the NEXT decoding step must attend to is the old
    prefix, the root (the last decoded token, whose K/V the verification pass computed as tree row 0)
    and the accepted path.  Pin: after verify -> compact (keep_root) a new token's attention over the
    compacted cache equals library causal attention (torch SDPA, fp64) over that sequence assembled by
    hand from the ORIGINAL cache, last row."""
    import torch
    rng = np.random.default_rng(17)
    parents = wl.greedy_tree(rng, 40, 5, 0.4)
    L, hq, hkv, d = 9, 4, 2, 16
    w = wl.make_custom(6, hq, hkv, d, [L], [parents])
    case = wl.make_verify_case(3, 64, [parents], sharpness=2.0, disagreement=0.3)
    tokens, nodes, _ = orc.verify_tree(parents, case.tokens[0], case.draft_probs, case.target_probs, case.accept_u,
                                       case.sample_u, bonus_at_leaf=True)
    assert len(nodes) >= 1 and 0 not in nodes                           # children only, as the kernel writes them
    listed = list(nodes) + [-1] * (len(tokens) - len(nodes))
    k2, v2 = w.k.copy(), w.v.copy()
    new_L = orc.compact_kv(k2, 0, L, listed, keep_root=True)
    assert orc.compact_kv(v2, 0, L, listed, keep_root=True) == new_L == L + 1 + len(nodes)
    # the next token: its own K/V row follows the new prefix
    q_new = wl.f32_to_bf16_bits(rng.standard_normal((1, hq, d)).astype(np.float32))
    kv_new = wl.f32_to_bf16_bits(rng.standard_normal((2, hkv, d)).astype(np.float32))
    k3 = np.concatenate([k2[:new_L], kv_new[0:1]])
    v3 = np.concatenate([v2[:new_L], kv_new[1:2]])
    got = orc.tree_attention(q_new, k3, v3, new_L, [-1])[0]              # [hq][d]
    # by hand, from the original cache: prefix rows, root row, path rows, the new row
    rows = list(range(L)) + [L + 0] + [L + a for a in nodes]
    f = orc.bf16_bits_to_f64
    K = torch.from_numpy(np.concatenate([f(w.k[rows]), f(kv_new[0:1])]))   # [T][hkv][d]
    V = torch.from_numpy(np.concatenate([f(w.v[rows]), f(kv_new[1:2])]))
    T = K.shape[0]
    g = hq // hkv
    for h in range(hq):
        qs = torch.zeros((1, 1, T, d), dtype=torch.float64)
        qs[0, 0, T - 1] = torch.from_numpy(f(q_new)[0, h])
        ref = torch.nn.functional.scaled_dot_product_attention(qs, K[:, h // g].reshape(1, 1, T, d), V[:, h // g].reshape(1, 1, T, d),
                                                               is_causal=True)[0, 0, T - 1].numpy()
        assert np.abs(got[h] - ref).max() < 1e-12
