"""GPU parity of the paged-cache forms with the oracle: tree attention whose prefix keys come through a
page table (both kernel regimes, split and unsplit plans, tile skipping), and the accepted-path
compaction into the prefix pages (bit exact)."""
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


def _check_paged(rt, w, page_size, seed=0, sparse=False, regime=-1, ctas=0, combine=2, sample=None):
    B, R = rt
    pw = wl.to_paged(w, page_size, seed)
    B.dyspec_set_tuning(regime, ctas, combine)
    try:
        batch = R.DeviceBatch(w, sparse=sparse, paged=pw)
    finally:
        B.dyspec_set_tuning(-1, 0, 2)
    batch.step()
    bits, depths, out_bits, status = batch.results()
    assert status == 0
    got = orc.bf16_bits_to_f64(out_bits)
    assert np.isfinite(got).all()
    if sample is None:
        ref = orc.tree_attention_paged(w.q, pw.k, pw.v, pw.page_table, page_size, w.prefix_len, w.n_nodes,
                                       pw.tree_row_offset, w.parents)
        err = np.abs(got - ref)
    else:
        rng = np.random.default_rng(5)
        errs = []
        no = w.node_offsets
        for r in range(w.n_req):
            n, L = int(w.n_nodes[r]), int(w.prefix_len[r])
            if n == 0:
                continue
            nodes = sorted(set([0, n - 1] + [int(x) for x in rng.integers(0, n, size=sample)]))
            rows = orc.paged_prefix_rows(pw.page_table[r], page_size, L) + [int(pw.tree_row_offset[r]) + j for j in range(n)]
            ref = orc.tree_attention_nodes(w.q[no[r]:no[r + 1]], pw.k[rows], pw.v[rows], L, w.parents[r], nodes)
            errs.append(np.abs(got[no[r] + np.asarray(nodes)] - ref).ravel())
        err = np.concatenate(errs)
    assert err.max() <= MAX_ABS, f"max abs err {err.max()}"
    assert err.mean() <= MEAN_ABS, f"mean abs err {err.mean()}"
    return batch


@pytest.mark.parametrize("page_size", [128, 256, 1024])
@pytest.mark.parametrize("regime", [0, 1])
def test_paged_attention_ragged_batch(rt, page_size, regime):
    rng = np.random.default_rng(100 + page_size + regime)
    n_max = 60 if regime == 0 else 200
    trees = [wl.greedy_tree(rng, n_max, 6, 0.2), wl.chain_tree(17), np.zeros(0, np.int32), wl.random_tree(rng, 33),
             wl.star_forest(9), wl.greedy_tree(rng, 48, 4, 0.3)]
    prefix = [700, 0, 50, 129, 128, 1025]            # ragged tails, exactly one tile, one row into a new page
    w = wl.make_custom(40 + regime, 8, 2, 128, prefix, trees)
    for ctas in (0, 5):
        _check_paged(rt, w, page_size, seed=page_size, regime=regime, ctas=ctas)


@pytest.mark.parametrize("combine", [0, 2])
def test_paged_attention_split_kv_small_trees(rt, combine):
    """One long-prefix request: the prefix is cut across CTAs (cluster merge or the combine kernel)."""
    rng = np.random.default_rng(7)
    w = wl.make_custom(50, 32, 32, 128, [3000], [wl.greedy_tree(rng, 64, 8, 0.2)])
    _check_paged(rt, w, 256, seed=1, regime=0, combine=combine)
    w2 = wl.make_custom(51, 8, 1, 64, [2100, 900], [wl.greedy_tree(rng, 8, 3, 0.2), wl.greedy_tree(rng, 5, 2, 0.2)])
    _check_paged(rt, w2, 128, seed=2, combine=combine)


def test_paged_attention_tensor_core_regime_with_tile_skipping(rt):
    rng = np.random.default_rng(9)
    w = wl.make_custom(52, 8, 2, 128, [1500, 300], [wl.random_tree(rng, 700), wl.random_tree(rng, 300)])
    B, R = rt
    plain = R.DeviceBatch(w)
    order, _, new_parents = plain.dfs_reorder()
    no = w.node_offsets
    w2 = wl.permute_tree_tokens(w, [order[no[r]:no[r + 1]] for r in range(2)],
                                [new_parents[no[r]:no[r + 1]] for r in range(2)])
    _check_paged(rt, w2, 512, seed=3, sparse=True, regime=1)
    _check_paged(rt, w2, 128, seed=4, sparse=False, regime=1)


def test_paged_equals_contiguous_bit_for_bit(rt):
    """Same keys in the same order: the paged call and the contiguous call return identical bits."""
    B, R = rt
    for cfg in (2, 3):
        w = wl.make_config(cfg)
        a = R.DeviceBatch(w)
        a.step()
        _, _, out_a, st_a = a.results()
        for page_size in (128, 2048):
            b = R.DeviceBatch(w, paged=wl.to_paged(w, page_size, 11))
            b.step()
            _, _, out_b, st_b = b.results()
            assert st_a == 0 and st_b == 0
            assert np.array_equal(out_a, out_b)


def test_paged_full_size_sampled(rt):
    """The headline configuration with its cache in 256-row pages; sampled rows against the oracle."""
    _check_paged(rt, wl.make_config(2), 256, seed=6, sample=4)
    _check_paged(rt, wl.make_config(4), 256, seed=7, sample=3)


def test_paged_argument_checks(rt):
    import torch
    B, R = rt
    w = wl.make_config(1)
    pw = wl.to_paged(w, 128, 0)
    paged = R.DeviceBatch(w, paged=pw)
    cont = R.DeviceBatch(w)
    paged.build_mask()
    cont.build_mask()
    with pytest.raises(B.DyspecError):       # contiguous call on a paged plan
        B.dyspec_tree_attention_ragged(paged.plan, paged.q, paged.k, paged.v, paged.bits, paged.out, paged.workspace,
                                       paged.workspace_bytes, paged.status)
    with pytest.raises(B.DyspecError):       # paged call on a contiguous plan
        B.dyspec_tree_attention_paged(cont.plan, cont.q, cont.k, cont.v, paged.page_table, pw.pages_per_req, cont.bits,
                                      None, cont.out, cont.workspace, cont.status)
    with pytest.raises(B.DyspecError):       # table too narrow for the prefix
        B.dyspec_tree_attention_paged(paged.plan, paged.q, paged.k, paged.v, paged.page_table, 0, paged.bits, None,
                                      paged.out, paged.workspace, paged.status)
    for bad in (0, 100, 64, 192):            # not a power of two >= 128
        with pytest.raises(B.DyspecError):
            B.dyspec_plan_create_paged(8, 8, 128, [10], [4], [0], 1000, bad, 4)
    torch.cuda.synchronize()


@pytest.mark.parametrize("keep_root", [False, True])
@pytest.mark.parametrize("hkv,d,page_size", [(8, 128, 128), (2, 64, 16), (1, 8, 4)])
def test_paged_compaction_matches_oracle(rt, hkv, d, page_size, keep_root):
    import torch
    B, _ = rt
    rng = np.random.default_rng(hkv + d + page_size)
    n_req, max_out = 5, 12
    Ls = rng.integers(0, 3 * page_size, size=n_req).astype(np.int32)
    Ls[1] = page_size - 1                                               # the accepted tokens cross into the next page
    Ls[2] = page_size
    ns = rng.integers(1, 40, size=n_req).astype(np.int32)
    w = wl.make_custom(60, hkv, hkv, d, Ls, [wl.chain_tree(int(n)) for n in ns])
    pw = wl.to_paged(w, page_size, 13)
    acc = np.full((n_req, max_out), -7, dtype=np.int32)
    cnt = np.zeros(n_req, dtype=np.int32)
    for r in range(n_req):
        lo = 1 if keep_root else 0
        m = int(rng.integers(0, min(max_out - 2, ns[r] - lo) + 1))
        acc[r, :m] = np.sort(lo + rng.choice(ns[r] - lo, size=m, replace=False))
        acc[r, m] = -1
        cnt[r] = m + 1
    rk, rv = pw.k.copy(), pw.v.copy()
    want_L = np.zeros(n_req, np.int32)
    for r in range(n_req):
        want_L[r] = orc.compact_kv_paged(rk, pw.page_table[r], page_size, pw.tree_row_offset[r], Ls[r], acc[r, :cnt[r]],
                                         keep_root=keep_root)
        orc.compact_kv_paged(rv, pw.page_table[r], page_size, pw.tree_row_offset[r], Ls[r], acc[r, :cnt[r]], keep_root=keep_root)
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    dk, dv = t(pw.k.view(np.int16)), t(pw.v.view(np.int16))
    newL = torch.zeros(n_req, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.dyspec_compact_kv_paged(dk, dv, t(pw.tree_row_offset), t(pw.page_table), pw.pages_per_req, page_size, t(Ls), t(acc),
                              t(cnt), n_req, max_out, hkv, d, newL, status, keep_root=keep_root)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(dk.cpu().numpy().view(np.uint16), rk)
    assert np.array_equal(dv.cpu().numpy().view(np.uint16), rv)
    assert np.array_equal(newL.cpu().numpy(), want_L)


def test_paged_compaction_without_a_page_reports_it(rt):
    import torch
    B, _ = rt
    w = wl.make_custom(61, 2, 2, 8, [6], [wl.chain_tree(10)])
    pw = wl.to_paged(w, 4, 1, room_for_accepted=False)                  # pages for 6 tokens only: 2 pages = 8 rows
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    dk, dv = t(pw.k.view(np.int16)), t(pw.v.view(np.int16))
    acc = np.array([[0, 1, 2, 3, 4]], np.int32)
    newL = torch.zeros(1, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.dyspec_compact_kv_paged(dk, dv, t(pw.tree_row_offset), t(pw.page_table), pw.pages_per_req, 4, t(w.prefix_len),
                              t(acc), t(np.array([5], np.int32)), 1, 5, 2, 8, newL, status)
    torch.cuda.synchronize()
    assert int(status.item()) == -1
    assert int(newL.item()) == 8                                        # two tokens fitted into the last page
    rk = pw.k.copy()
    orc.compact_kv_paged(rk, pw.page_table[0], 4, pw.tree_row_offset[0], 6, [0, 1])
    assert np.array_equal(dk.cpu().numpy().view(np.uint16), rk)
