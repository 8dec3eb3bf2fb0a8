"""Host logic of the ragged scheduler (no GPU): every key tile of every (request, kv head, query
tile) group is covered exactly once, split groups get distinct partial slots, CTAs get contiguous,
roughly equal shares."""
import numpy as np
import pytest

from paper_2410_11744_b200 import workloads as wl


@pytest.fixture(scope="module")
def B():
    from paper_2410_11744_b200 import build
    build.build()
    from paper_2410_11744_b200 import binding
    return binding


def cluster_workspace_per_cta(d, c):
    """Tensor-core regime, cluster of c CTAs: a CTA merges 256 / c rows and gets its c - 1 peers' shares of them
    through the workspace (a row: d floats and two scalars)."""
    return (c - 1) * (256 // c) * (d * 4 + 8)


def check_schedule(B, hq, hkv, d, Ls, ns, regime=-1, ctas=0, fuse=2):
    B.dyspec_set_tuning(regime, ctas, fuse)
    try:
        W = B.dyspec_words_per_row(max(list(ns) + [0]))
        items, cta_begin, info = B.dyspec_schedule_dry_run(hq, hkv, d, Ls, ns, W)
    finally:
        B.dyspec_set_tuning(-1, 0, 2)
    g = hq // hkv
    bm, bn = info["rows_per_tile"], info["keys_per_tile"]
    npt = bm // g
    # expected groups and their tile counts, from the definition of the tile list
    expect = {}
    for r, (L, n) in enumerate(zip(Ls, ns)):
        for kvh in range(hkv):
            for qt in range((n + npt - 1) // npt):
                last = min(n, (qt + 1) * npt)
                expect[(r, kvh, qt * bm)] = (L + bn - 1) // bn + (last + bn - 1) // bn
    assert info["groups"] == len(expect)
    assert info["key_tiles"] == sum(expect.values())
    covered = {k: [] for k in expect}
    slots = set()
    for req, kvh, row0, tb, te, slot, group, nsp in items.tolist():
        assert te > tb >= 0
        covered[(req, kvh, row0)].append((tb, te, slot, nsp))
    for key, pieces in covered.items():
        pieces.sort()
        assert pieces[0][0] == 0 and pieces[-1][1] == expect[key]
        for a, b in zip(pieces, pieces[1:]):
            assert a[1] == b[0]
        if info["cluster"] > 1:
            # cluster mode: every group is cut into `cluster` pieces merged on chip, no global slots
            assert len(pieces) == info["cluster"]
            assert all(slot == -1 and nsp == info["cluster"] for _, _, slot, nsp in pieces)
        elif len(pieces) == 1:
            assert pieces[0][2] == -1 and pieces[0][3] == 1
        else:
            for _, _, slot, nsp in pieces:
                assert slot >= 0 and slot not in slots and nsp == len(pieces)
                slots.add(slot)
    # a plan that runs from the shared queue (whole groups, more of them than CTAs, tensor-core regime)
    # keeps the queue's two words (256 bytes) behind the partials
    # (only when the scheduler chose that plan itself, i.e. no CTA count was forced)
    queue = 256 if (ctas == 0 and info["regime"] == 1 and info["split_groups"] == 0 and info["groups"] > info["ctas"]) else 0
    # ... and the split groups' counter pairs (two words each, padded to 256 bytes) right behind the partials
    pad = lambda x: (x + 255) & ~255
    n_split = len([1 for pieces in covered.values() if len(pieces) > 1]) if info["cluster"] == 1 else 0
    want = len(slots) * bm * (d + 2) * 4
    if info["cluster"] > 1 and info["regime"] == 1:
        want = info["ctas"] * cluster_workspace_per_cta(d, info["cluster"])
    if n_split:
        want = pad(want) + pad(8 * n_split)
    if queue:
        want = pad(want) + queue
    assert info["workspace_bytes"] == want
    assert sorted(slots) == list(range(len(slots)))
    # CTA ranges partition the item list
    assert cta_begin[0] == 0 and cta_begin[-1] == len(items) and (np.diff(cta_begin) > 0).all()
    loads = [int(sum(items[i][4] - items[i][3] for i in range(a, b))) for a, b in zip(cta_begin, cta_begin[1:])]
    return info, loads


def test_five_configs_schedule(B):
    for idx in range(1, 6):
        w = wl.make_config(idx)
        info, loads = check_schedule(B, w.n_q_heads, w.n_kv_heads, w.head_dim, w.prefix_len.tolist(), w.n_nodes.tolist())
        assert info["ctas"] <= (2 if info["regime"] == 0 else 1) * 148 + 8
        if idx >= 2:
            assert max(loads) <= 1.5 * (sum(loads) / len(loads)) + 4


@pytest.mark.parametrize("ctas", [1, 2, 7, 148, 5000])
def test_forced_cta_counts(B, ctas):
    check_schedule(B, 8, 2, 128, [700, 45, 0, 9000], [90, 33, 5, 1024], ctas=ctas)


def test_degenerate_batches(B):
    info, loads = check_schedule(B, 4, 4, 64, [], [])
    assert info["items"] == 0 and info["ctas"] == 0
    info, _ = check_schedule(B, 4, 4, 64, [10, 0], [0, 0])
    assert info["items"] == 0
    info, _ = check_schedule(B, 4, 4, 64, [0], [1])
    assert info["items"] == 4 and info["key_tiles"] == 4


def test_regime_1_tiles(B):
    info, _ = check_schedule(B, 64, 8, 128, [2048], [512], regime=1)
    assert info["rows_per_tile"] == 256 and info["keys_per_tile"] == 128 and info["regime"] == 1


def test_cluster_mode_is_used_for_uniform_small_batches(B):
    # Llama2-7B shape, 64 nodes: 32 groups x 17 tiles -> clusters of 4 (128 CTAs), no workspace
    info, loads = check_schedule(B, 32, 32, 128, [1024], [64])
    assert info["cluster"] == 4 and info["ctas"] == 128 and info["workspace_bytes"] == 0
    assert max(loads) - min(loads) <= 1
    # forcing a separate combine kernel switches it off
    info, _ = check_schedule(B, 32, 32, 128, [1024], [64], fuse=0)
    assert info["cluster"] == 1 and info["workspace_bytes"] > 0
    # very uneven groups do not qualify
    info, _ = check_schedule(B, 8, 8, 128, [64, 4096], [16, 16])
    assert info["cluster"] == 1


def test_regime_is_chosen_from_packed_rows(B):
    # nodes x group <= 64 rows: warp-level tiles; more: tcgen05 tiles
    assert check_schedule(B, 32, 32, 128, [1024], [64])[0]["regime"] == 0
    assert check_schedule(B, 64, 8, 128, [1024], [8])[0]["regime"] == 0
    assert check_schedule(B, 64, 8, 128, [1024], [9])[0]["regime"] == 1
    assert check_schedule(B, 32, 32, 128, [4096], [256])[0]["regime"] == 1


def test_whole_group_plan_is_chosen_when_cheaper(B):
    """Many groups of similar length (Llama2-70B shape, 512-node tree: 128 groups of 17 - 20 key tiles):
    dealing whole groups needs no partials and no combine launch, and the cost model prefers it; a few
    long groups (Llama2-7B, 4096-token prefix: 32 groups of 34 tiles) must still be split."""
    w = wl.make_config(4)
    args = (w.n_q_heads, w.n_kv_heads, w.head_dim, w.prefix_len.tolist(), w.n_nodes.tolist())
    info, loads = check_schedule(B, *args)
    assert info["split_groups"] == 0 and info["ctas"] == 128 and max(loads) == 20
    info_never, _ = check_schedule(B, *args, fuse=2 + 16)          # whole groups switched off
    assert info_never["split_groups"] > 0
    w3 = wl.make_config(3)
    args3 = (w3.n_q_heads, w3.n_kv_heads, w3.head_dim, w3.prefix_len.tolist(), w3.n_nodes.tolist())
    info3, loads3 = check_schedule(B, *args3)
    # few long groups of equal length: one cluster of 4 CTAs per group, merged through distributed shared memory
    assert info3["cluster"] == 4 and info3["split_groups"] == 0 and info3["ctas"] == 128 == info3["items"]
    assert max(loads3) == 9 and info3["workspace_bytes"] == 128 * 3 * 64 * 520 and info3["combine_launch"] == 0   # three peers' shares per CTA
    # without clusters: even pieces, one per CTA, on as many CTAs as there are SMs (20 groups in 5, 12 in 4),
    # merged inside the kernel through the workspace
    info3e, loads3e = check_schedule(B, *args3, fuse=1)
    assert info3e["cluster"] == 1 and info3e["split_groups"] == 32 and info3e["ctas"] == 148 == info3e["items"]
    assert max(loads3e) == 9 and info3e["combine_launch"] == 0
    info3_always, loads3 = check_schedule(B, *args3, fuse=2 + 32)   # forced: 32 CTAs with 34 tiles each
    assert info3_always["split_groups"] == 0 and info3_always["ctas"] == 32 and set(loads3) == {34}


def test_whole_group_plan_balances_a_ragged_batch(B):
    """Ragged batch: groups sorted by length and dealt to the least loaded CTA; no CTA ends up with more
    than the mean plus the longest group."""
    w = wl.make_config(5)
    info, loads = check_schedule(B, w.n_q_heads, w.n_kv_heads, w.head_dim, w.prefix_len.tolist(), w.n_nodes.tolist(),
                                 fuse=2 + 32)
    assert info["split_groups"] == 0 and info["ctas"] == 148
    longest = max(-(-int(L) // 128) + -(-int(n) // 128) for L, n in zip(w.prefix_len, w.n_nodes))
    assert max(loads) <= sum(loads) / len(loads) + longest


def test_merge_in_kernel_only_when_the_grid_is_one_wave(B):
    """The items of a split group wait for each other inside the tensor-core kernel, so that plan is only
    made when all CTAs are resident at once (no more CTAs than SMs); a forced larger grid, the small-tile
    regime and combine mode 0 keep the combine launch."""
    shape = (8, 1, 128, [60000], [40])                              # 2 groups of 470 key tiles
    info, _ = check_schedule(B, *shape, regime=1)
    assert info["ctas"] <= 148 and info["split_groups"] == 2 and info["combine_launch"] == 0
    info_big, _ = check_schedule(B, *shape, regime=1, ctas=200, fuse=2 + 16)
    assert info_big["ctas"] > 148 and info_big["split_groups"] == 2 and info_big["combine_launch"] == 1
    assert check_schedule(B, *shape, regime=1, fuse=0)[0]["combine_launch"] == 1
    small = check_schedule(B, 32, 32, 128, [4096] * 8, [64] * 8)[0]  # regime 0, split, not uniform enough for clusters
    assert small["regime"] == 0 and small["split_groups"] > 0 and small["combine_launch"] == 1


def test_cluster_plans_of_the_tensor_core_regime(B):
    """Few groups of similar length in the tensor-core regime: one cluster of C CTAs per group (C the same
    for all groups, at least two tiles per piece, all CTAs in one wave), a workspace for the peers' shares but no
    counters; merge mode 1 keeps the
    merge through the workspace; too many groups, or groups too short, get no clusters."""
    for shape, want in (((8, 8, 128, [2000], [256]), 8), ((16, 16, 128, [1500], [200]), 4), ((64, 64, 64, [700], [130]), 2),
                        ((8, 1, 128, [3000], [12]), 8)):
        info, loads = check_schedule(B, *shape, regime=1)
        assert info["cluster"] == want and info["combine_launch"] == 0, (shape, info)
        assert info["workspace_bytes"] == info["ctas"] * cluster_workspace_per_cta(shape[2], want)
        assert info["ctas"] == info["groups"] * want and min(loads) >= 2 and max(loads) - min(loads) <= 1
        never = check_schedule(B, *shape, regime=1, fuse=1)[0]
        assert never["cluster"] == 1 and never["combine_launch"] == 0
    # 128 groups: two CTAs each would not fit in one wave
    assert check_schedule(B, 64, 8, 128, [2048], [512], regime=1)[0]["cluster"] == 1
    # one group of three tiles: a piece would have fewer than two
    assert check_schedule(B, 8, 1, 128, [200], [16], regime=1)[0]["cluster"] == 1
    # two requests of very different length: the cost model decides, every tile is still covered once (check_schedule)
    check_schedule(B, 16, 16, 128, [6000, 300], [200, 200], regime=1)
