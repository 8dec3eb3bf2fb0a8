"""GPU parity with the oracle for the paged cache whose tree rows are part of the paged sequence (node j =
token L + j): key tiles follow the sequence, so a row's mask slice is shifted by L modulo the tile size.
Both kernel regimes, every word / tile boundary of that shift, split plans, and the in-place compaction."""
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


def _check(rt, w, page_size, seed=0, regime=-1, ctas=0, combine=2, sample=None, sparse=False):
    B, R = rt
    pw = wl.to_paged(w, page_size, seed, tree_in_pages=True)
    B.dyspec_set_tuning(regime, ctas, combine)
    try:
        batch = R.DeviceBatch(w, paged=pw, sparse=sparse)
    finally:
        B.dyspec_set_tuning(-1, 0, 2)
    batch.step()
    _, _, out_bits, status = batch.results()
    assert status == 0
    got = orc.bf16_bits_to_f64(out_bits)
    assert np.isfinite(got).all()
    if sample is None:
        ref = orc.tree_attention_paged(w.q, pw.k, pw.v, pw.page_table, page_size, w.prefix_len, w.n_nodes, None, w.parents)
        err = np.abs(got - ref)
    else:
        rng = np.random.default_rng(5)
        errs, no = [], w.node_offsets
        for r in range(w.n_req):
            n, L = int(w.n_nodes[r]), int(w.prefix_len[r])
            if n == 0:
                continue
            nodes = sorted(set([0, n - 1] + [int(x) for x in rng.integers(0, n, size=sample)]))
            rows = orc.paged_prefix_rows(pw.page_table[r], page_size, L + n)
            ref = orc.tree_attention_nodes(w.q[no[r]:no[r + 1]], pw.k[rows], pw.v[rows], L, w.parents[r], nodes)
            errs.append(np.abs(got[no[r] + np.asarray(nodes)] - ref).ravel())
        err = np.concatenate(errs)
    assert err.max() <= MAX_ABS, f"max abs err {err.max()}"
    assert err.mean() <= MEAN_ABS, f"mean abs err {err.mean()}"
    return batch


# prefix lengths whose remainder modulo 128 (and 64) sits on and around every 32-bit word boundary
SHIFTS = [0, 1, 31, 32, 33, 63, 64, 65, 95, 96, 97, 127]


@pytest.mark.parametrize("regime", [0, 1])
def test_every_shift_of_the_mask_window(rt, regime):
    rng = np.random.default_rng(300 + regime)
    n = 40 if regime == 0 else 200
    for base in (0, 256):
        prefix = [base + s for s in SHIFTS]
        trees = [wl.greedy_tree(rng, int(rng.integers(n // 2, n + 1)), 5, 0.3) for _ in prefix]
        w = wl.make_custom(80 + regime, 8, 2, 128, prefix, trees)
        _check(rt, w, 128, seed=base + regime, regime=regime)


@pytest.mark.parametrize("regime", [0, 1])
def test_trees_that_end_exactly_on_or_just_past_a_mask_group(rt, regime):
    """n a multiple of the tile size with a non-zero shift: the last tile starts in the row's last bit group,
    and the group behind it does not exist (it must read as zeros, not as the next row's bits)."""
    rng = np.random.default_rng(310 + regime)
    if regime == 0:      # forced small tiles (64 keys): 128 nodes = 2 groups of 64 bits, W = 4
        w = wl.make_custom(82, 2, 2, 64, [5, 64 + 63, 1], [wl.random_tree(rng, 128), wl.chain_tree(128), wl.star_forest(64)])
    else:
        w = wl.make_custom(83, 4, 1, 128, [5, 128 + 127, 300], [wl.random_tree(rng, 128), wl.chain_tree(256),
                                                                wl.greedy_tree(rng, 384, 4, 0.3)])
    _check(rt, w, 128, seed=2, regime=regime)
    _check(rt, w, 512, seed=3, regime=regime, ctas=3)


def test_chain_and_star_closed_forms_through_the_pages(rt):
    """Chain = causal attention over the sequence, star = prefix + self: both through shifted windows."""
    w = wl.make_custom(84, 8, 8, 64, [77, 130, 0], [wl.chain_tree(150), wl.star_forest(90), wl.chain_tree(33)])
    _check(rt, w, 128, seed=4)
    _check(rt, w, 256, seed=5, regime=0)


def test_largest_trees(rt):
    rng = np.random.default_rng(320)
    w = wl.make_custom(85, 2, 1, 128, [1000, 19], [wl.random_tree(rng, 2048), wl.greedy_tree(rng, 1024, 8, 0.2)])
    _check(rt, w, 1024, seed=6, sample=6)
    _check(rt, w, 128, seed=7, sample=6, sparse=True)       # the tile sets are ignored by such a plan


@pytest.mark.parametrize("combine", [0, 2])
def test_split_plans(rt, combine):
    """A long prefix cut across CTAs: cluster merge / merge inside the tensor-core kernel / combine launch."""
    rng = np.random.default_rng(330)
    w0 = wl.make_custom(86, 32, 32, 128, [3001], [wl.greedy_tree(rng, 64, 8, 0.2)])
    _check(rt, w0, 256, seed=8, regime=0, combine=combine)
    w1 = wl.make_custom(87, 16, 16, 128, [4001], [wl.greedy_tree(rng, 256, 8, 0.1)])
    _check(rt, w1, 256, seed=9, regime=1, combine=combine, sample=8)
    w2 = wl.make_custom(88, 8, 1, 64, [2100, 901], [wl.greedy_tree(rng, 8, 3, 0.2), wl.greedy_tree(rng, 5, 2, 0.2)])
    _check(rt, w2, 128, seed=10, combine=combine)


def test_full_size_sampled(rt):
    """The benchmark's configurations 2 and 5 with prefix AND tree in 256-row pages; sampled rows."""
    _check(rt, wl.make_config(2), 256, seed=11, sample=4)
    _check(rt, wl.make_config(5), 256, seed=12, sample=2)


def test_table_must_cover_prefix_and_tree(rt):
    import torch
    B, R = rt
    w = wl.make_custom(89, 4, 4, 64, [120], [wl.chain_tree(16)])      # 136 tokens: two pages of 128
    pw = wl.to_paged(w, 128, 0, tree_in_pages=True)
    batch = R.DeviceBatch(w, paged=pw)
    batch.build_mask()
    with pytest.raises(B.DyspecError):
        B.dyspec_tree_attention_paged(batch.plan, batch.q, batch.k, batch.v, batch.page_table, 1, batch.bits, None,
                                      batch.out, batch.workspace, batch.status)
    torch.cuda.synchronize()


@pytest.mark.parametrize("keep_root", [False, True])
@pytest.mark.parametrize("hkv,d,page_size", [(8, 128, 128), (2, 64, 16), (1, 8, 4)])
def test_compaction_in_place_matches_oracle(rt, hkv, d, page_size, keep_root):
    import torch
    B, _ = rt
    rng = np.random.default_rng(hkv + d + page_size + 1)
    n_req, max_out = 6, 12
    Ls = rng.integers(0, 3 * page_size, size=n_req).astype(np.int32)
    Ls[1] = page_size - 1
    Ls[2] = page_size
    ns = rng.integers(2, 40, size=n_req).astype(np.int32)
    w = wl.make_custom(90, hkv, hkv, d, Ls, [wl.chain_tree(int(n)) for n in ns])
    pw = wl.to_paged(w, page_size, 14, tree_in_pages=True)
    acc = np.full((n_req, max_out), -7, dtype=np.int32)
    cnt = np.zeros(n_req, dtype=np.int32)
    for r in range(n_req):
        lo = 1 if keep_root else 0
        m = int(rng.integers(0, min(max_out - 2, ns[r] - lo) + 1))
        acc[r, :m] = np.sort(lo + rng.choice(ns[r] - lo, size=m, replace=False))
        acc[r, m] = -1
        cnt[r] = m + 1
    # overlapping moves: token L + 1 receives node 2 after node 1 was taken from it
    acc[5, :4] = [1, 2, 3, -1] if ns[5] > 3 else [1, -1, -7, -7]
    cnt[5] = 4 if ns[5] > 3 else 2
    rk, rv = pw.k.copy(), pw.v.copy()
    want_L = np.zeros(n_req, np.int32)
    for r in range(n_req):
        want_L[r] = orc.compact_kv_paged(rk, pw.page_table[r], page_size, None, Ls[r], acc[r, :cnt[r]], keep_root=keep_root)
        orc.compact_kv_paged(rv, pw.page_table[r], page_size, None, Ls[r], acc[r, :cnt[r]], keep_root=keep_root)
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    dk, dv = t(pw.k.view(np.int16)), t(pw.v.view(np.int16))
    newL = torch.zeros(n_req, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.dyspec_compact_kv_paged(dk, dv, None, t(pw.page_table), pw.pages_per_req, page_size, t(Ls), t(acc), t(cnt), n_req,
                              max_out, hkv, d, newL, status, keep_root=keep_root)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(dk.cpu().numpy().view(np.uint16), rk)
    assert np.array_equal(dv.cpu().numpy().view(np.uint16), rv)
    assert np.array_equal(newL.cpu().numpy(), want_L)
