"""Pins for the fp64 oracle: each test checks it against something other than itself.

The paper prints no worked numeric example of an attention output or a mask, so the pins are
what its definitions and the mathematics fix: a hand-written mask fixture (Sec. 2, mask(A)),
library causal attention for a chain, prefix+self for a star, pure-Python brute force over each
root-to-node path (parallel verification == decoding each path autoregressively, Sec. 2), closed
forms, and relabelling invariance (App. C: reordering tokens must not change the result).
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import dyspec_oracle as orc
from paper_2410_11744_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- helpers (independent of the oracle)
def _bf16_to_float(bits: int) -> float:
    import struct
    return struct.unpack("<f", struct.pack("<I", (int(bits) & 0xFFFF) << 16))[0]


def _decode(arr):
    return np.vectorize(_bf16_to_float, otypes=[np.float64])(arr)


def _path(parents, i):
    p = []
    while i != -1:
        p.append(i)
        i = int(parents[i])
    return p[::-1]  # root first


def _causal_last_row_python(qrows, krows, vrows, scale):
    """Textbook full causal attention over a sequence, pure Python floats; returns the last position's output.

    qrows/krows/vrows: lists of lists (positions x D)."""
    T = len(krows)
    D = len(krows[0])
    outs = []
    for t in range(T):
        s = [scale * sum(qrows[t][d] * krows[u][d] for d in range(D)) for u in range(t + 1)]
        m = max(s)
        e = [math.exp(x - m) for x in s]
        z = sum(e)
        outs.append([sum(e[u] / z * vrows[u][d] for u in range(t + 1)) for d in range(D)])
    return outs[-1]


def _small(seed, hq, hkv, d, L, parents):
    return wl.make_custom(seed, hq, hkv, d, [L], [np.asarray(parents, dtype=np.int32)])


# ----------------------------------------------------------------------------- bf16 decode
def test_bf16_decode_known_patterns():
    bits = np.array([0x3F80, 0xC000, 0x0000, 0x8000, 0x3DCD, 0x7F7F, 0x0080, 0x4049], dtype=np.uint16)
    want = [1.0, -2.0, 0.0, -0.0, 0.10009765625, 3.3895313892515355e38, 1.1754943508222875e-38, 3.140625]
    got = orc.bf16_bits_to_f64(bits)
    assert got.tolist() == want
    assert math.copysign(1.0, got[3]) == -1.0


def test_generator_rounding_is_rne():
    # 1 + 2^-8 is exactly halfway between bf16 1.0 (even mantissa) and 1.0078125 -> rounds to even (1.0);
    # 1.0078125 + 2^-8 is halfway between odd 0x3F81 and even 0x3F82 -> rounds up to 0x3F82.
    x = np.array([1.0 + 2.0 ** -8, 1.0078125 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -3.0], dtype=np.float32)
    assert wl.f32_to_bf16_bits(x).tolist() == [0x3F80, 0x3F82, 0x3F81, 0xC040]


# ----------------------------------------------------------------------------- mask
def _read_mask_fixture():
    parents, rows = None, {}
    with open(os.path.join(GOLDEN, "mask_small_tree.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("parents"):
                parents = [int(t) for t in line.split()[1:]]
            elif line.startswith("row"):
                head, vis, depth, word = [t.strip() for t in line[3:].replace(":", ";", 1).split(";")]
                rows[int(head)] = ([int(t) for t in vis.split()], int(depth), int(word, 16))
    return parents, rows


def test_mask_matches_hand_written_fixture():
    parents, rows = _read_mask_fixture()
    bits, depths = orc.build_tree_mask(parents, 4)
    assert bits.shape == (9, 4) and bits.dtype == np.uint32
    for i, (vis, depth, word) in rows.items():
        assert sorted(orc.visible_nodes(parents, i)) == vis
        assert int(bits[i, 0]) == word, f"row {i}"
        assert bits[i, 1:].tolist() == [0, 0, 0]
        assert int(depths[i]) == depth
        # the hex word and the list in the fixture agree with each other (guards the fixture itself)
        assert sum(1 << j for j in vis) == word
    m = orc.tree_mask_matrix(parents)
    for i, (vis, _, _) in rows.items():
        assert np.flatnonzero(m[i]).tolist() == vis


def test_mask_crosses_word_boundaries():
    # chain of 70 nodes: row i = bits 0..i; check the words by closed form.
    parents = wl.chain_tree(70)
    bits, depths = orc.build_tree_mask(parents, 4)
    for i in range(70):
        full = (1 << (i + 1)) - 1
        assert [int(x) for x in bits[i]] == [(full >> (32 * w)) & 0xFFFFFFFF for w in range(4)]
        assert depths[i] == i
    # star: only the self bit
    bits, depths = orc.build_tree_mask(wl.star_forest(40), 4)
    for i in range(40):
        assert int(bits[i, i // 32]) == 1 << (i % 32) and int(bits[i].astype(np.uint64).sum()) == 1 << (i % 32)
        assert depths[i] == 0


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_mask_invariants_random_trees(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 200))
    parents = wl.random_tree(rng, n, p_root=0.1)
    W = 8
    bits, depths = orc.build_tree_mask(parents, W)
    as_int = [sum(int(bits[i, w]) << (32 * w) for w in range(W)) for i in range(n)]
    total = 0
    for i in range(n):
        row = as_int[i]
        assert (row >> i) & 1 == 1                       # self bit
        assert row >> (i + 1) == 0                       # nothing beyond self: bit j set => j <= i
        p = int(parents[i])
        if p >= 0:
            assert row == as_int[p] | (1 << i)           # recurrence
            assert depths[i] == depths[p] + 1
        else:
            assert row == 1 << i and depths[i] == 0
        assert bin(row).count("1") == depths[i] + 1
        total += depths[i] + 1
    assert sum(bin(r).count("1") for r in as_int) == total


def test_bad_parents_rejected():
    for bad in ([-1, 1], [-1, 0, 2], [-2], [0]):
        with pytest.raises(ValueError):
            orc.build_tree_mask(bad, 4)
    with pytest.raises(ValueError):
        orc.build_tree_mask(wl.chain_tree(33), 1)


# ----------------------------------------------------------------------------- attention pins
def test_chain_equals_library_causal_attention():
    """parents[i] = i-1: the tree is a plain continuation, so the result is the last n rows of causal attention."""
    L, n, hq, hkv, d = 37, 21, 4, 2, 32
    w = _small(11, hq, hkv, d, L, wl.chain_tree(n))
    got = orc.tree_attention(w.q, w.k, w.v, L, w.parents[0])
    k = torch.from_numpy(_decode(w.k)).permute(1, 0, 2)              # [hkv][T][d]
    v = torch.from_numpy(_decode(w.v)).permute(1, 0, 2)
    k = k.repeat_interleave(hq // hkv, dim=0)                        # consecutive query heads share a KV head
    v = v.repeat_interleave(hq // hkv, dim=0)
    qfull = torch.zeros(hq, L + n, d, dtype=torch.float64)
    qfull[:, L:, :] = torch.from_numpy(_decode(w.q)).permute(1, 0, 2)
    ref = torch.nn.functional.scaled_dot_product_attention(qfull[None], k[None], v[None], is_causal=True)[0]
    ref = ref[:, L:, :].permute(1, 0, 2).numpy()
    assert np.abs(got - ref).max() < 1e-12


def test_star_is_prefix_plus_self():
    L, n, hq, hkv, d = 9, 6, 2, 1, 8
    w = _small(5, hq, hkv, d, L, wl.star_forest(n))
    got = orc.tree_attention(w.q, w.k, w.v, L, w.parents[0])
    q, k, v = _decode(w.q), _decode(w.k), _decode(w.v)
    scale = 1 / math.sqrt(d)
    for i in range(n):
        for h in range(hq):
            rows = list(range(L)) + [L + i]
            s = [scale * float(np.dot(q[i, h], k[t, 0])) for t in rows]
            m = max(s)
            e = [math.exp(x - m) for x in s]
            ref = sum(ei / sum(e) * v[t, 0] for ei, t in zip(e, rows))
            assert np.abs(got[i, h] - ref).max() < 1e-12


@pytest.mark.parametrize("case", [
    dict(seed=1, hq=2, hkv=2, d=8, L=5, parents=[-1, 0, 0, 1, 1, 2, 3]),
    dict(seed=2, hq=4, hkv=2, d=4, L=0, parents=[-1, 0, 1, 0, -1, 4]),       # empty prefix, forest, GQA
    dict(seed=3, hq=8, hkv=1, d=4, L=3, parents=[-1]),                       # single node, g = 8
    dict(seed=4, hq=2, hkv=1, d=16, L=12, parents=None),                     # greedy tree (config-1 recipe, smaller)
])
def test_brute_force_per_path(case):
    """Each node's output == last position of ordinary causal attention over prefix + its root-to-node path."""
    parents = case["parents"]
    if parents is None:
        parents = wl.greedy_tree(np.random.default_rng(99), 12, 4, 0.3).tolist()
    hq, hkv, d, L = case["hq"], case["hkv"], case["d"], case["L"]
    w = _small(case["seed"], hq, hkv, d, L, parents)
    got = orc.tree_attention(w.q, w.k, w.v, L, parents)
    sampled = orc.tree_attention_nodes(w.q, w.k, w.v, L, parents, range(len(parents)))
    assert np.abs(got - sampled).max() < 1e-13
    q, k, v = _decode(w.q), _decode(w.k), _decode(w.v)
    g = hq // hkv
    scale = 1 / math.sqrt(d)
    for i in range(len(parents)):
        path = _path(parents, i)
        seq = list(range(L)) + [L + j for j in path]
        for h in range(hq):
            krows = [k[t, h // g].tolist() for t in seq]
            vrows = [v[t, h // g].tolist() for t in seq]
            # queries of earlier positions do not influence the last row; use zeros for the prefix, the path's own q after
            qrows = [[0.0] * d for _ in range(L)] + [q[j, h].tolist() for j in path]
            ref = _causal_last_row_python(qrows, krows, vrows, scale)
            assert np.abs(got[i, h] - np.array(ref)).max() < 1e-12, (i, h)


def test_closed_form_constant_v():
    parents = [-1, 0, 0, 1, 2, 2]
    w = _small(21, 4, 2, 16, 10, parents)
    vconst = wl.f32_to_bf16_bits(np.linspace(-2, 2, 16, dtype=np.float32))
    w.v[:] = vconst[None, None, :]
    got = orc.tree_attention(w.q, w.k, w.v, 10, parents)
    assert np.abs(got - _decode(vconst)[None, None, :]).max() < 1e-14


def test_closed_form_zero_k_gives_mean_of_visible_rows():
    """K = 0 -> uniform weights -> mean of the L + depth + 1 visible V rows: pins the visible set per node."""
    parents = [-1, 0, 1, 1, 0, 4, -1, 6]
    L = 7
    w = _small(22, 2, 1, 8, L, parents)
    w.k[:] = 0
    got = orc.tree_attention(w.q, w.k, w.v, L, parents)
    v = _decode(w.v)
    for i in range(len(parents)):
        rows = list(range(L)) + [L + j for j in _path(parents, i)]
        ref = v[rows, 0, :].mean(axis=0)
        for h in range(2):
            assert np.abs(got[i, h] - ref).max() < 1e-14


def test_spike_pins_masking():
    """A key with an overwhelming score captures the output iff it is visible."""
    parents = [-1, 0, 0, 1, 2]           # node 3: path 0-1-3 ; node 2 is NOT an ancestor of 3
    L, d = 6, 8
    w = _small(23, 1, 1, d, L, parents)
    base = orc.tree_attention(w.q, w.k, w.v, L, parents)
    big = wl.f32_to_bf16_bits(np.float32(64.0) * np.sign(_decode(w.q[3, 0]).astype(np.float32)))
    # spike on node 2's key, aligned with node 3's query: node 3 must not move, node 4 (child of 2) has its own q
    w2 = _small(23, 1, 1, d, L, parents)
    w2.k[L + 2, 0] = big
    moved = orc.tree_attention(w2.q, w2.k, w2.v, L, parents)
    assert np.array_equal(moved[3], base[3])
    assert np.array_equal(moved[1], base[1]) and np.array_equal(moved[0], base[0])
    # same spike on node 1 (an ancestor of 3): output of node 3 collapses onto V row of node 1
    w3 = _small(23, 1, 1, d, L, parents)
    w3.k[L + 1, 0] = big
    cap = orc.tree_attention(w3.q, w3.k, w3.v, L, parents)
    assert np.abs(cap[3, 0] - _decode(w3.v[L + 1, 0])).max() < 1e-9
    # and a spike on a prefix key is seen by that query too
    w4 = _small(23, 1, 1, d, L, parents)
    w4.k[2, 0] = big
    cap = orc.tree_attention(w4.q, w4.k, w4.v, L, parents)
    assert np.abs(cap[3, 0] - _decode(w4.v[2, 0])).max() < 1e-9


def test_scale_is_inverse_sqrt_head_dim_and_overridable():
    # one prefix key + self, D = 4, hand-computable: q = k_self = (1,1,1,1), k_prefix = 0, v = e0 / e1
    L, d = 1, 4
    w = _small(0, 1, 1, d, L, [-1])
    one = 0x3F80
    w.q[:] = one
    w.k[0] = 0
    w.k[1] = one
    w.v[:] = 0
    w.v[0, 0, 0] = one
    w.v[1, 0, 1] = one
    got = orc.tree_attention(w.q, w.k, w.v, L, [-1])          # scores: 0 and 4/sqrt(4) = 2
    p_self = math.exp(2.0) / (1.0 + math.exp(2.0))
    assert abs(got[0, 0, 1] - p_self) < 1e-15 and abs(got[0, 0, 0] - (1 - p_self)) < 1e-15
    got = orc.tree_attention(w.q, w.k, w.v, L, [-1], scale=0.25)   # scores 0 and 1
    assert abs(got[0, 0, 1] - math.e / (1 + math.e)) < 1e-15


def test_relabelling_invariance():
    """Renumbering nodes in another topological order (e.g. DFS, App. C) permutes the outputs and nothing else."""
    rng = np.random.default_rng(3)
    parents = wl.greedy_tree(rng, 24, 4, 0.3)
    L = 11
    w = _small(31, 4, 2, 8, L, parents)
    base = orc.tree_attention(w.q, w.k, w.v, L, parents)
    # DFS preorder
    children = {i: [] for i in range(-1, 24)}
    for i, p in enumerate(parents):
        children[int(p)].append(i)
    order, stack = [], children[-1][::-1]
    while stack:
        u = stack.pop()
        order.append(u)
        stack.extend(children[u][::-1])
    new_of_old = {old: new for new, old in enumerate(order)}
    new_parents = [-1 if parents[old] < 0 else new_of_old[int(parents[old])] for old in order]
    q2 = w.q[order]
    k2 = np.concatenate([w.k[:L], w.k[L:][order]])
    v2 = np.concatenate([w.v[:L], w.v[L:][order]])
    out2 = orc.tree_attention(q2, k2, v2, L, new_parents)
    assert np.abs(out2 - base[order]).max() < 1e-13


def test_ragged_is_independent_requests():
    rng = np.random.default_rng(8)
    trees = [wl.greedy_tree(rng, 7, 4, 0.3), np.zeros(0, np.int32), wl.chain_tree(3)]
    w = wl.make_custom(9, 4, 2, 8, [5, 4, 0], trees)
    full = orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents)
    assert full.shape == (10, 4, 8)
    for r in (0, 2):
        q, k, v, p, L = w.request(r)
        no = w.node_offsets
        assert np.array_equal(full[no[r]:no[r + 1]], orc.tree_attention(q, k, v, L, p))
    bits, depths = orc.build_tree_mask_ragged(w.parents, 4)
    assert bits.shape == (10, 4) and depths.tolist()[7:] == [0, 1, 2]


# ----------------------------------------------------------------------------- visible (query, key) pairs (what the flop count of the roofline is built on)
def test_visible_pair_count_closed_forms_and_brute_force():
    """The number of (query, key) pairs the definition of Sec. 2 / App. C uses: every node sees the L
    prefix keys, its ancestors and itself.  Chain of n nodes: n L + n (n + 1) / 2.  Forest of n roots
    (star): n (L + 1).  A perfect binary tree with levels 0 .. d: sum over levels 2^k (L + k + 1).
    Brute force: count, pair by pair, the keys j <= i that lie on node i's root path."""
    for L, n in ((0, 1), (5, 1), (7, 9), (128, 16), (1000, 33)):
        assert orc.visible_pair_count([L], [wl.chain_tree(n)]) == n * L + n * (n + 1) // 2
        assert orc.visible_pair_count([L], [wl.star_forest(n)]) == n * (L + 1)
    d, L = 4, 11
    binary = np.array([-1] + [(i - 1) // 2 for i in range(1, 2 ** (d + 1) - 1)], dtype=np.int32)
    assert orc.visible_pair_count([L], [binary]) == sum(2 ** k * (L + k + 1) for k in range(d + 1))
    # ragged: the sum over requests; an empty request adds nothing
    assert orc.visible_pair_count([3, 9, 2], [wl.chain_tree(4), np.zeros(0, np.int32), wl.star_forest(5)]) == \
        (4 * 3 + 10) + 0 + 5 * 3
    rng = np.random.default_rng(12)
    for n in (1, 6, 40):
        p = wl.random_tree(rng, n, p_root=0.2)
        L = int(rng.integers(0, 20))
        brute = 0
        for i in range(n):
            path = set(_path(p, i))
            brute += L + sum(1 for j in range(n) if j in path)
        assert orc.visible_pair_count([L], [p]) == brute


# ----------------------------------------------------------------------------- workload structure (Sec. 4.3: shallow trees)
def test_generator_trees_are_valid_and_shallow():
    """Sec. 4.3: depth is typically < 10 at N = 64 and < 30 at N = 768; greedy trees keep parent[i] < i."""
    for n, alpha, bound in ((64, 0.3, 10), (768, 0.3, 30)):
        p = wl.greedy_tree(np.random.default_rng(n), n, 8, alpha)
        assert p[0] == -1 and all(0 <= p[i] < i for i in range(1, n))
        _, depths = orc.build_tree_mask(p, 24)
        assert depths.max() < bound


def test_configs_have_stated_shapes():
    w = wl.make_config(1)
    assert (w.n_q_heads, w.n_kv_heads, w.head_dim, int(w.prefix_len[0]), int(w.n_nodes[0])) == (4, 4, 64, 128, 16)
    assert w.q.shape == (16, 4, 64) and w.k.shape == (144, 4, 64) and w.q.dtype == np.uint16
    w2 = wl.make_config(1)
    assert np.array_equal(w.q, w2.q) and np.array_equal(w.parents[0], w2.parents[0])
    w = wl.make_config(5)
    assert w.n_req == 8 and w.prefix_len.min() >= 512 and w.prefix_len.max() <= 8192
    assert w.n_nodes.min() >= 32 and w.n_nodes.max() <= 768
    assert w.k.shape[0] == int((w.prefix_len + w.n_nodes).sum())
