"""GPU parity of the token-reorder path (App. C): DFS renumbering, per-node tile sets, the block count
and the attention call that skips empty tree tiles, each against the oracle.  Index and bit outputs
must match exactly; attention within the tolerance of the dense path."""
import numpy as np
import pytest

from oracle import dyspec_oracle as orc
from paper_2410_11744_b200 import workloads as wl

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


@pytest.fixture(scope="module")
def rt():
    import torch
    assert torch.cuda.is_available()
    from paper_2410_11744_b200 import build
    build.build()
    from paper_2410_11744_b200 import binding, runner
    return binding, runner


def _trees():
    rng = np.random.default_rng(77)
    out = {
        "single": np.array([-1], np.int32),
        "pair": np.array([-1, 0], np.int32),
        "chain33": wl.chain_tree(33),
        "chain2048": wl.chain_tree(2048),
        "star100": wl.star_forest(100),
        "star2048": wl.star_forest(2048),
        "root_fan": np.concatenate([[-1], np.zeros(2047, np.int32)]).astype(np.int32),       # one root, 2047 children
        "random64": wl.random_tree(rng, 64),
        "random257": wl.random_tree(rng, 257),
        "random1000": wl.random_tree(rng, 1000),
        "random1024": wl.random_tree(rng, 1024),
        "random1025": wl.random_tree(rng, 1025),
        "random2048": wl.random_tree(rng, 2048),
        "forest1500": wl.random_tree(rng, 1500, p_root=0.02),
        "greedy768": wl.greedy_tree(rng, 768, 8, 0.05),
        "sparse_sibs": np.array([-1] + [0 if i % 97 == 1 else i - 1 for i in range(1, 1200)], np.int32),
    }
    return out


TREES = _trees()


def _tiles_from_bits(bits):
    """Bit t of a node's word = some bit set in words 2t, 2t+1 of its mask row (64 columns per tile)."""
    n, W = bits.shape
    pairs = (bits.reshape(n, W // 2, 2) != 0).any(axis=2)
    out = np.zeros(n, dtype=np.uint32)
    for t in range(W // 2):
        out |= pairs[:, t].astype(np.uint32) << np.uint32(t)
    return out


@pytest.mark.parametrize("name", sorted(TREES))
def test_dfs_reorder_single_request(rt, name):
    import torch
    B, _ = rt
    parents = TREES[name]
    n = len(parents)
    dev = "cuda:0"
    d_par = torch.from_numpy(parents).to(dev)
    order = torch.full((n,), -7, dtype=torch.int32, device=dev)
    new_of_old = torch.full((n,), -7, dtype=torch.int32, device=dev)
    new_parents = torch.full((n,), -7, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.dyspec_dfs_reorder(d_par, n, order, new_of_old, new_parents, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref_order = orc.dfs_order(parents)
    ref_parents, ref_new_of_old = orc.relabel_tree(parents, ref_order)
    assert np.array_equal(order.cpu().numpy(), np.asarray(ref_order, np.int32))
    assert np.array_equal(new_of_old.cpu().numpy(), ref_new_of_old)
    assert np.array_equal(new_parents.cpu().numpy(), ref_parents)


@pytest.mark.parametrize("name", ["chain2048", "random1025", "random2048", "forest1500", "random1000", "star2048"])
def test_mask_tiles_and_block_count_large_trees(rt, name):
    """Mask builder beyond 1024 nodes (column chunks), per-node tile sets, and the block count."""
    import torch
    B, _ = rt
    parents = TREES[name]
    n = len(parents)
    W = B.dyspec_words_per_row(n)
    dev = "cuda:0"
    d_par = torch.from_numpy(parents).to(dev)
    bits = torch.full((n, W), -1, dtype=torch.int32, device=dev)
    depths = torch.full((n,), -1, dtype=torch.int32, device=dev)
    tiles = torch.full((n,), -1, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    count = torch.zeros(1, dtype=torch.int64, device=dev)
    B.dyspec_build_tree_mask_tiles(d_par, n, bits, depths, tiles, W, status)
    ref_bits, ref_depths = orc.build_tree_mask(parents, W)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got_bits = bits.cpu().numpy().view(np.uint32)
    assert np.array_equal(got_bits, ref_bits)
    assert np.array_equal(depths.cpu().numpy(), ref_depths)
    assert np.array_equal(tiles.cpu().numpy().view(np.uint32), _tiles_from_bits(ref_bits))
    # the plain entry point gives the same mask
    bits2 = torch.full((n, W), -1, dtype=torch.int32, device=dev)
    B.dyspec_build_tree_mask(d_par, n, bits2, None, W, status)
    torch.cuda.synchronize()
    assert np.array_equal(bits2.cpu().numpy().view(np.uint32), ref_bits)
    for block in (32, 64, 128):
        B.dyspec_mask_block_count(bits, n, W, block, count)
        torch.cuda.synchronize()
        assert int(count.item()) == orc.mask_block_count(parents, block)


def test_block_counts_before_and_after_reorder(rt):
    """End to end on the GPU: reorder -> mask -> block count equals the oracle's count on the oracle's
    relabelled tree, and the reorder lowers the count (Table 5)."""
    import torch
    B, _ = rt
    dev = "cuda:0"
    for n in (256, 512, 1024, 2048):
        parents = wl.make_random_tree_case(n, n_heads=1, head_dim=64).parents[0]
        W = B.dyspec_words_per_row(n)
        d_par = torch.from_numpy(parents).to(dev)
        new_parents = torch.zeros(n, dtype=torch.int32, device=dev)
        bits = torch.zeros((n, W), dtype=torch.int32, device=dev)
        count = torch.zeros(1, dtype=torch.int64, device=dev)
        counts = []
        for par in (d_par, new_parents):
            if par is new_parents:
                B.dyspec_dfs_reorder(d_par, n, None, None, new_parents, None)
            B.dyspec_build_tree_mask(par, n, bits, None, W, None)
            B.dyspec_mask_block_count(bits, n, W, 32, count)
            torch.cuda.synchronize()
            counts.append(int(count.item()))
        ref_new, _ = orc.relabel_tree(parents, orc.dfs_order(parents))
        assert counts == [orc.mask_block_count(parents, 32), orc.mask_block_count(ref_new, 32)]
        assert counts[1] < counts[0]


def _reordered(rt, w):
    """Reorders w's trees with the GPU kernel and returns the renumbered workload."""
    _, R = rt
    batch = R.DeviceBatch(w)
    order, _, new_parents = batch.dfs_reorder()
    no = w.node_offsets
    orders = [order[no[r]:no[r + 1]] for r in range(w.n_req)]
    news = [new_parents[no[r]:no[r + 1]] for r in range(w.n_req)]
    for r in range(w.n_req):
        assert np.array_equal(orders[r], np.asarray(orc.dfs_order(w.parents[r]), np.int32))
    return wl.permute_tree_tokens(w, orders, news), orders


def _check_sparse(rt, w, sample=None, regime=-1, ctas=0):
    """Sparse mask + attention on w against the oracle (all rows, or `sample` nodes per request)."""
    B, R = rt
    B.dyspec_set_tuning(regime, ctas, 2)
    try:
        batch = R.DeviceBatch(w, sparse=True)
    finally:
        B.dyspec_set_tuning(-1, 0, 2)
    batch.step()
    bits, depths, out_bits, status = batch.results()
    assert status == 0
    ref_bits, ref_depths = orc.build_tree_mask_ragged(w.parents, batch.W)
    assert np.array_equal(bits, ref_bits) and np.array_equal(depths, ref_depths)
    assert np.array_equal(batch.node_tiles[:w.total_nodes].cpu().numpy().view(np.uint32), _tiles_from_bits(ref_bits))
    got = orc.bf16_bits_to_f64(out_bits)
    assert np.isfinite(got).all()
    if sample is None:
        ref = orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents)
        err = np.abs(got - ref)
    else:
        rng = np.random.default_rng(3)
        errs = []
        no = w.node_offsets
        for r in range(w.n_req):
            n = int(w.n_nodes[r])
            if n == 0:
                continue
            nodes = sorted(set([0, n - 1] + [int(x) for x in rng.integers(0, n, size=sample)]))
            q, k, v, parents, L = w.request(r)
            ref = orc.tree_attention_nodes(q, k, v, L, parents, nodes)
            errs.append(np.abs(got[no[r] + np.asarray(nodes)] - ref).ravel())
        err = np.concatenate(errs)
    assert err.max() <= MAX_ABS, f"max abs err {err.max()}"
    assert err.mean() <= MEAN_ABS, f"mean abs err {err.mean()}"
    return batch, got


@pytest.mark.parametrize("n,heads,L", [(300, 4, 0), (700, 2, 100), (1024, 2, 0), (1500, 1, 37), (2048, 1, 0)])
def test_sparse_attention_on_reordered_random_trees(rt, n, heads, L):
    """The paper's random-tree experiment (App. C.1) at reduced head count: creation order dense ==
    oracle, DFS order with tile skipping == oracle on the renumbered problem, and the two outputs are
    the same rows in a different order."""
    w = wl.make_random_tree_case(n, n_heads=heads, head_dim=128, prefix_len=L)
    w2, orders = _reordered(rt, w)
    _, got2 = _check_sparse(rt, w2, regime=1)
    _, got1 = _check_sparse(rt, w, regime=1)
    assert np.abs(got2 - got1[orders[0]]).max() <= 2 * MAX_ABS


def test_sparse_attention_ragged_batch_and_gqa(rt):
    rng = np.random.default_rng(11)
    trees = [wl.random_tree(rng, 900), wl.greedy_tree(rng, 300, 8, 0.1), np.zeros(0, np.int32), wl.chain_tree(260),
             wl.random_tree(rng, 1100, p_root=0.01)]
    w = wl.make_custom(21, 8, 2, 128, [0, 700, 5, 129, 64], trees)
    w2, _ = _reordered(rt, w)
    for ctas in (0, 7):
        _check_sparse(rt, w2, regime=1, ctas=ctas)
    w3 = wl.make_custom(22, 4, 4, 64, [0, 300], [wl.random_tree(rng, 800), wl.random_tree(rng, 513)])
    w4, _ = _reordered(rt, w3)
    _check_sparse(rt, w4, regime=1)
    _check_sparse(rt, w4)              # scheduler's own choice of regime


def test_sparse_full_size_random_tree_sampled(rt):
    """Table 5's largest case at full size (64 heads x 128, 2048 tokens, no prefix), DFS order, tile
    skipping on; sampled rows against the oracle."""
    w = wl.make_random_tree_case(2048)
    w2, _ = _reordered(rt, w)
    _check_sparse(rt, w2, sample=6)


def test_sparse_call_ignores_tiles_in_small_tree_regime(rt):
    w = wl.make_config(2)
    _check_sparse(rt, w)
    _check_sparse(rt, w, regime=0)


def test_reorder_reports_bad_parent(rt):
    import torch
    B, _ = rt
    parents = np.array([-1, 0, 5, 1, -3, 2], np.int32)            # entries 2 and 4 are invalid
    fixed = np.array([-1, 0, -1, 1, -1, 2], np.int32)             # treated as roots
    dev = "cuda:0"
    d_par = torch.from_numpy(parents).to(dev)
    order = torch.zeros(6, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.dyspec_dfs_reorder(d_par, 6, order, None, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == -5
    assert order.cpu().numpy().tolist() == orc.dfs_order(fixed)
