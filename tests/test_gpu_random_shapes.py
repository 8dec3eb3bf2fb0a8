"""GPU parity on randomly drawn small batches: head grouping, head size, prefix lengths around the tile
boundaries, tree shapes and sizes on both sides of the regime boundary, empty requests, forced CTA counts
and both ways of merging split-KV partials; every case runs twice on the same buffers and is compared
with the oracle element by element."""
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


def _draw(rng, index):
    g = int(rng.choice([1, 2, 4, 8]))
    hkv = int(rng.choice([1, 2, 4]))
    d = int(rng.choice([64, 128]))
    n_req = int(rng.integers(1, 6))
    Ls = [int(x) for x in rng.choice([0, 1, 5, 63, 64, 65, 127, 128, 129, 200, 500, 900], n_req)]
    max_n = 64 // g if rng.random() < 0.6 else 300
    trees = []
    for _ in range(n_req):
        n = int(rng.integers(0, max_n + 1))
        kind = int(rng.integers(0, 4))
        if n == 0:
            trees.append(np.zeros(0, np.int32))
        elif kind == 0:
            trees.append(wl.chain_tree(n))
        elif kind == 1:
            trees.append(wl.star_forest(n))
        elif kind == 2:
            trees.append(wl.random_tree(rng, n))
        else:
            trees.append(wl.greedy_tree(rng, n, 4, 0.3))
    w = wl.make_custom(9000 + index, hkv * g, hkv, d, Ls, trees)
    return w, int(rng.choice([0, 0, 0, 1, 3, 7, 148])), int(rng.choice([2, 2, 0]))


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_small_batches(rt, seed):
    B, R = rt
    rng = np.random.default_rng(seed)
    for index in range(24):
        w, ctas, combine = _draw(rng, 100 * seed + index)
        B.dyspec_set_tuning(-1, ctas, combine)
        try:
            batch = R.DeviceBatch(w)
        finally:
            B.dyspec_set_tuning(-1, 0, 2)
        for _ in range(2):
            batch.step()
        bits, depths, out_bits, status = batch.results()
        what = dict(heads=(w.n_q_heads, w.n_kv_heads), d=w.head_dim, L=w.prefix_len.tolist(), n=w.n_nodes.tolist(),
                    ctas=ctas, combine=combine, plan=batch.plan.describe())
        assert status == 0, what
        ref_bits, ref_depths = orc.build_tree_mask_ragged(w.parents, batch.W)
        assert np.array_equal(bits, ref_bits) and np.array_equal(depths, ref_depths), what
        ref = orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents)
        if ref.size:
            got = orc.bf16_bits_to_f64(out_bits)
            assert np.isfinite(got).all(), what
            err = np.abs(got - ref)
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (what, err.max(), err.mean())


def _draw_large(rng, index):
    g = int(rng.choice([1, 2, 4, 8]))
    hkv = int(rng.choice([1, 2, 4, 8]))
    d = int(rng.choice([64, 128]))
    n_req = int(rng.integers(1, 10))
    Ls = [int(np.exp(rng.uniform(0.0, np.log(6000.0)))) for _ in range(n_req)]
    trees = []
    for _ in range(n_req):
        n = int(rng.choice([1, 17, 64, 65, 128, 129, 255, 256, 257, 511, 700, 1024, 1500, 2048]))
        kind = int(rng.integers(0, 3))
        if kind == 0 and n <= 300:
            trees.append(wl.chain_tree(n))
        elif kind <= 1:
            trees.append(wl.random_tree(rng, n))
        else:
            trees.append(wl.greedy_tree(rng, n, 8, 0.2))
    w = wl.make_custom(20000 + index, hkv * g, hkv, d, Ls, trees)
    return w, bool(rng.integers(0, 2)), int(rng.choice([0, 0, 1, 2]))


@pytest.mark.parametrize("seed", [21, 22])
def test_random_large_ragged_batches_on_sampled_rows(rt, seed):
    """Trees up to 2048 nodes, prefixes up to 6000 keys, up to 9 requests: split plans, whole-group plans and
    the shared queue, with and without tile skipping.  Masks and depths are compared in full, the attention
    on sampled query nodes of every request (the oracle evaluates those one by one)."""
    B, R = rt
    rng = np.random.default_rng(seed)
    for index in range(8):
        w, sparse, whole = _draw_large(rng, 100 * seed + index)
        B.dyspec_set_tuning(-1, 0, 2 + 16 * whole)
        try:
            batch = R.DeviceBatch(w, sparse=sparse)
        finally:
            B.dyspec_set_tuning(-1, 0, 2)
        for _ in range(2):
            batch.step()
        bits, depths, out_bits, status = batch.results()
        what = dict(heads=(w.n_q_heads, w.n_kv_heads), d=w.head_dim, L=w.prefix_len.tolist(), n=w.n_nodes.tolist(),
                    sparse=sparse, whole=whole, plan=batch.plan.describe())
        assert status == 0, what
        ref_bits, ref_depths = orc.build_tree_mask_ragged(w.parents, batch.W)
        assert np.array_equal(bits, ref_bits) and np.array_equal(depths, ref_depths), what
        got = orc.bf16_bits_to_f64(out_bits)
        assert np.isfinite(got).all(), what
        qo = 0
        for r in range(w.n_req):
            n, o, L = int(w.n_nodes[r]), int(w.kv_row_offset[r]), int(w.prefix_len[r])
            nodes = sorted(set(rng.integers(0, n, size=min(n, 24)).tolist() + [0, n - 1]))
            ref = orc.tree_attention_nodes(w.q[qo:qo + n], w.k[o:o + L + n], w.v[o:o + L + n], L, w.parents[r], nodes)
            err = np.abs(got[qo:qo + n][nodes] - ref)
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (what, r, err.max(), err.mean())
            qo += n


def _draw_few_long(rng, index):
    """One to three requests with long prefixes: the shapes that get cluster plans, even pieces merged through
    the workspace, or the combine launch, depending on the merge mode."""
    g = int(rng.choice([1, 2, 4, 8]))
    hkv = int(rng.choice([1, 2, 4, 8, 16]))
    d = int(rng.choice([64, 128]))
    n_req = int(rng.choice([1, 1, 1, 2, 3]))
    Ls = [int(np.exp(rng.uniform(np.log(100.0), np.log(7000.0)))) for _ in range(n_req)]
    ns = [int(rng.choice([5, 12, 33, 64, 100, 129, 256, 300, 512])) for _ in range(n_req)]
    trees = [wl.greedy_tree(rng, k, 6, 0.3) if rng.random() < 0.7 else wl.random_tree(rng, k) for k in ns]
    return wl.make_custom(30000 + index, hkv * g, hkv, d, Ls, trees)


def test_random_plans_merge_modes_and_cache_layouts(rt):
    """Few long requests under every merge mode (0 combine launch, 1 through the workspace inside the kernel,
    2 clusters where the plan allows), either regime, and the three cache layouts (contiguous, paged with the
    tree rows outside the pages, paged with the tree rows inside); sampled rows against the oracle."""
    B, R = rt
    seen = set()
    for seed, index in [(s_, i) for s_ in (31, 32) for i in range(24)]:
        if index == 0:
            rng = np.random.default_rng(seed)
        w = _draw_few_long(rng, 100 * seed + index)
        layout = int(rng.integers(0, 3))
        page = int(rng.choice([128, 256, 1024]))
        paged = None if layout == 0 else wl.to_paged(w, page, seed=seed, tree_in_pages=(layout == 2))
        combine, regime = int(rng.choice([2, 2, 2, 1, 0])), int(rng.choice([-1, -1, 1]))
        B.dyspec_set_tuning(regime, 0, combine)
        try:
            batch = R.DeviceBatch(w, paged=paged)
        finally:
            B.dyspec_set_tuning(-1, 0, 2)
        for _ in range(2):
            batch.step()
        _, _, out_bits, status = batch.results()
        info = batch.plan.describe()
        what = dict(heads=(w.n_q_heads, w.n_kv_heads), d=w.head_dim, L=w.prefix_len.tolist(), n=w.n_nodes.tolist(),
                    layout=layout, page=page, combine=combine, regime=regime, plan=info)
        seen.add((info["regime"], info["cluster"] > 1, info["split_groups"] > 0))
        assert status == 0, what
        got = orc.bf16_bits_to_f64(out_bits)
        assert np.isfinite(got).all(), what
        qo = 0
        for r in range(w.n_req):
            n, o, L = int(w.n_nodes[r]), int(w.kv_row_offset[r]), int(w.prefix_len[r])
            nodes = sorted(set(rng.integers(0, n, size=min(n, 6)).tolist() + [0, n - 1]))
            ref = orc.tree_attention_nodes(w.q[qo:qo + n], w.k[o:o + L + n], w.v[o:o + L + n], L, w.parents[r], nodes)
            err = np.abs(got[qo:qo + n][nodes] - ref)
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (what, r, err.max(), err.mean())
            qo += n
    assert (1, True, False) in seen and (1, False, True) in seen, seen      # cluster plans and workspace merges both ran
